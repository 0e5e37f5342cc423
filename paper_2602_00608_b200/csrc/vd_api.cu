// C ABI of libvd.so: argument validation, the per-configuration launch plan (layer list ->
// kernel launches and workspace offsets), weight repacking at create time, and the decode loop.
#include <stdio.h>
#include <string.h>

#include <map>
#include <string>
#include <vector>

#include "vd_internal.h"

using namespace vd;

namespace {

thread_local std::string g_last_error;

struct Step {
    vd_step_info info;
    int kind;
    bool use_tc;
    ConvArgs conv;
    GnArgs gn;
    AttnArgs attn;
    IngestArgs ing;
    ConvTcPlan tc;
    AttnTcPlan attn_tc;
    // batch-dependent pointers are rebased per call: strides per frame
    bool has_residual;
};

// A tensor-core convolution whose output only ever meets a GroupNorm, another convolution's residual add or the
// fused shortcut leaves its bias out (its epilogue warps pace the narrow layers, and the additions are 40 of their
// 70 instructions per pass).  The tensor then stands for "stored value + pending[c]", and the per-channel vector
// `pending` is accounted for downstream: the statistics pass adds it on the fly and folds it into `shift`, a residual add
// carries it along, the fused 1x1 shortcut contributes W * pending, and a convolution that reads the tensor without a
// normalisation gets it as a unit-scale prologue.  The vectors depend on the weights alone: computed once in vd_create.
constexpr size_t kNone = (size_t)-1;
struct FoldJob {             // out[c] = in[c] + b[c] + b2[c] + sum_k w2[c][k] * pin[k]   (absent terms: kNone)
    size_t out_off, in_off, b_off, b2_off, w2_off, pin_off;
    int Cin2, Cout;
};
struct FillJob {             // dst[n][c] = src[c] (src kNone: 1.0) for n < B
    size_t dst_off, src_off;
    int C, B;
};

struct WeightJob {           // repack work done once in vd_create
    std::string name;        // source tensor
    int kind;                // 0 conv weight (packed), 1 vector -> fp32, 2 matrix [Cout][Cin] -> fp32 (same layout)
    bool tc;
    bool phase;              // tensor-core weights of the phase-collapsed upsampling form
    int Cout, Cin, taps;
    int cout_total, cout_offset;
    size_t dst_off;
};

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
constexpr size_t kGuardBytes = 256;
constexpr int kGuardByte = 0xA5;
int elt(int dtype) { return dtype == VD_BF16 ? 2 : 4; }

}  // namespace

struct vd_handle_s {
    vd_config cfg;
    char* ws = nullptr;
    size_t ws_bytes = 0;
    std::vector<Step> steps;
    std::vector<WeightJob> jobs;
    std::vector<FoldJob> folds;          // run once after the weight jobs, in order
    std::vector<FillJob> fills;          // then these
    std::vector<size_t> guards;          // offsets of the guard regions (VD_FLAG_CANARY)
    std::string err;
    int stop_after = -1;
    size_t status_off = 0, lat_stage_off[2] = {0, 0}, frm_stage_off[2] = {0, 0}, gn_counter_off = 0, stat_off = 0, stat_bytes = 0;
    size_t total = 0;
    // host-transport pipeline (vd_decode_host_stream): two copy streams and the events that order
    // copies and decodes; created on first use, destroyed with the handle
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_dec[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    bool pipe_ready = false;
    size_t frame_bytes(int batch) const {
        const size_t px = (size_t)batch * cfg.out_channels * cfg.latent_h * cfg.latent_w * 64;
        return (cfg.flags & VD_FLAG_OUT_U8) ? px : px * (cfg.dtype == VD_BF16 ? 2 : 4);
    }
    size_t latent_bytes(int batch) const {
        return (size_t)batch * cfg.latent_channels * cfg.latent_h * cfg.latent_w * (cfg.dtype == VD_BF16 ? 2 : 4);
    }
    ~vd_handle_s() {
        for (int i = 0; i < 2; ++i) {
            if (ev_in[i]) cudaEventDestroy(ev_in[i]);
            if (ev_dec[i]) cudaEventDestroy(ev_dec[i]);
            if (ev_out[i]) cudaEventDestroy(ev_out[i]);
        }
        if (copy_in) cudaStreamDestroy(copy_in);
        if (copy_out) cudaStreamDestroy(copy_out);
    }
};

namespace {

// Walks the layer list of a layout and lays out workspace + steps.  With base == nullptr only
// sizes/offsets are computed (all pointers are offsets from 0).
class Planner {
  public:
    Planner(vd_handle_s* h, char* base) : h_(h), base_(base), cfg_(h->cfg) {}

    // With VD_FLAG_CANARY every region is followed by a 256-byte guard that vd_create fills with a pattern
    // and vd_debug_check_canaries verifies: a kernel that writes past the end of its buffer (or before the start of
    // the next one) is caught even if the overrun lands in memory that a later layer overwrites.
    size_t alloc(size_t bytes) {
        const size_t off = align_up(cur_, 256);
        cur_ = off + bytes;
        if (cfg_.flags & VD_FLAG_CANARY) {
            const size_t g = align_up(cur_, 256);
            h_->guards.push_back(g);
            cur_ = g + kGuardBytes;
        }
        return off;
    }
    template <typename T> T* ptr(size_t off) const { return (T*)(base_ + off); }

    bool bf16() const { return cfg_.dtype == VD_BF16; }
    int act_dtype() const { return bf16() ? VD_BF16 : VD_F32; }   // intra-block tensors

    struct ConvW { size_t w_off, b_off; bool tc; };

    // registers the repack of a conv weight (possibly a stack of several source tensors along Cout)
    ConvW conv_weight(const std::vector<std::string>& names, int Cout_each, int Cin, int taps, bool tc, bool phase = false) {
        const int Cout = Cout_each * (int)names.size();
        ConvW r;
        r.tc = tc;
        const size_t wbytes = tc ? conv_tc_packed_bytes(Cout, Cin, taps, phase) : (size_t)taps * Cin * Cout * 4;
        r.w_off = alloc(wbytes);
        r.b_off = alloc((size_t)Cout * 4);
        for (size_t i = 0; i < names.size(); ++i) {
            h_->jobs.push_back({names[i] + ".weight", 0, tc, phase, Cout_each, Cin, taps, Cout, (int)i * Cout_each, r.w_off});
            h_->jobs.push_back({names[i] + ".bias", 1, false, false, Cout_each, 0, 0, 0, 0, r.b_off + (size_t)i * Cout_each * 4});
        }
        return r;
    }
    void norm_weight(const std::string& name, int C, size_t& g_off, size_t& b_off) {
        g_off = alloc((size_t)C * 4);
        b_off = alloc((size_t)C * 4);
        h_->jobs.push_back({name + ".weight", 1, false, false, C, 0, 0, 0, 0, g_off});
        h_->jobs.push_back({name + ".bias", 1, false, false, C, 0, 0, 0, 0, b_off});
    }

    void add_gn(const std::string& name, size_t x_off, int dtype, int H, int W, int C, const std::string& wname) {
        size_t g_off, b_off;
        norm_weight(wname, C, g_off, b_off);
        // scale/shift buffers alternate, so a convolution can read one set in its prologue while
        // its epilogue writes the next normalisation's set
        gn_toggle_ ^= 1;
        scale_off_ = scale_buf_[gn_toggle_];
        shift_off_ = shift_buf_[gn_toggle_];
        // On request: where the step before is the tensor-core convolution that writes this very tensor, its epilogue
        // takes the statistics and the normalisation needs no pass of its own.
        if ((cfg_.flags & VD_FLAG_FUSED_STATS) && !h_->steps.empty()) {
            Step& prev = h_->steps.back();
            ConvArgs probe = prev.conv;
            probe.B = 1;
            if (prev.kind == VD_STEP_CONV && prev.use_tc && prev.conv.y == ptr<void>(x_off) && prev.conv.Cout == C &&
                prev.conv.H == H && prev.conv.W == W && !prev.conv.stat_sum && conv_tc_stats_supported(probe, cfg_.norm_groups)) {
                ConvArgs& a = prev.conv;
                a.stat_sum = ptr<unsigned long long>(stat_off_);
                a.stat_counter = ptr<unsigned int>(stat_off_ + conv_stat_sum_bytes(cfg_.max_batch, cfg_.norm_groups));
                a.stat_gamma = ptr<float>(g_off); a.stat_beta = ptr<float>(b_off);
                a.stat_scale = ptr<float>(scale_off_); a.stat_shift = ptr<float>(shift_off_);
                a.stat_G = cfg_.norm_groups; a.stat_eps = cfg_.norm_eps;
                prev.info.stats_fused = 1;
                return;
            }
        }
        Step s{};
        s.kind = VD_STEP_GN_STATS;
        s.gn = GnArgs{ptr<void>(x_off), dtype, 0, H * W, C, cfg_.norm_groups, cfg_.norm_eps, ptr<float>(g_off),
                      ptr<float>(b_off), ptr<float>(scale_off_), ptr<float>(shift_off_), ptr<float>(partial_off_),
                      ptr<unsigned int>(partial_off_ + gn_partial_bytes(cfg_.max_batch, cfg_.norm_groups)),
                      pending(x_off) != kNone ? ptr<float>(pending(x_off)) : nullptr};
        fill_info(s, name, 0, C, C, 0, 0, H, W, C, VD_F32, 0, -1);
        s.info.launches = 1;
        s.info.bytes_per_frame = (double)H * W * C * elt(dtype);
        h_->steps.push_back(s);
    }

    // conv step; x at source resolution Hs x Ws
    void add_conv(const std::string& name, const std::vector<std::string>& wnames, int Cout_each, size_t x_off,
                  int in_dtype, int Hs, int Ws, int Cin, int ksize, bool upsample, bool prologue, bool silu,
                  long residual_off, size_t y_off, int out_dtype, bool out_nchw, bool y_is_frames,
                  const std::string& shortcut_name = std::string(), size_t x2_off = 0, int Cin2 = 0, bool out_u8 = false) {
        Step s{};
        s.kind = VD_STEP_CONV;
        const int Cout = Cout_each * (int)wnames.size();
        const int H = upsample ? 2 * Hs : Hs, W = upsample ? 2 * Ws : Ws;
        ConvArgs a{};
        a.x = ptr<void>(x_off);
        a.scale = prologue ? ptr<float>(scale_off_) : nullptr;
        a.shift = prologue ? ptr<float>(shift_off_) : nullptr;
        a.residual = residual_off >= 0 ? ptr<float>((size_t)residual_off) : nullptr;
        a.y = y_is_frames ? nullptr : ptr<void>(y_off);
        a.B = 0; a.Hs = Hs; a.Ws = Ws; a.H = H; a.W = W;
        a.Cin = Cin; a.Cout = Cout; a.ksize = ksize; a.upsample = upsample ? 1 : 0; a.silu = silu;
        a.in_dtype = in_dtype; a.out_dtype = out_dtype; a.out_nchw = out_nchw; a.bf16_operands = bf16();
        if (!shortcut_name.empty()) { a.x2 = ptr<void>(x2_off); a.Cin2 = Cin2; }
        a.out_u8 = out_u8 ? 1 : 0;
        const bool tc_on = bf16() && !(cfg_.flags & VD_FLAG_FORCE_SIMT);
        ConvArgs probe = a;
        probe.B = 1;
        // an upsampling 3x3 runs in the phase-collapsed form (4/9 of the products) where the tensor-core kernel has it
        bool phase = false;
        if (tc_on && upsample && !(cfg_.flags & VD_FLAG_UPSAMPLE_9TAP)) {
            probe.upsample = 2;
            phase = conv_tc_supported(probe);
            if (!phase) probe.upsample = 1;
        }
        if (phase) a.upsample = 2;
        const bool tc = tc_on && conv_tc_supported(probe);
        ConvW cw = conv_weight(wnames, Cout_each, Cin, ksize * ksize, tc, phase);
        a.w = ptr<void>(cw.w_off);
        a.bias = ptr<float>(cw.b_off);
        if (!shortcut_name.empty()) {          // only requested when the tensor-core kernel takes this layer
            // the fused shortcut multiplies in tf32: its weight stays an fp32 [Cout][Cin2] matrix
            const size_t w2_off = alloc((size_t)Cout * Cin2 * 4), b2_off = alloc((size_t)Cout * 4);
            h_->jobs.push_back({shortcut_name + ".weight", 2, false, false, Cout, Cin2, 1, 0, 0, w2_off});
            h_->jobs.push_back({shortcut_name + ".bias", 1, false, false, Cout, 0, 0, 0, 0, b2_off});
            a.w2 = ptr<void>(w2_off);
            a.bias2 = ptr<float>(b2_off);
        }
        // ---- pending biases (see FoldJob)
        const bool want_defer = defer_;
        defer_ = false;
        const size_t pin_x = pending(x_off);
        const size_t pres = residual_off >= 0 ? pending((size_t)residual_off) : kNone;
        const size_t px2 = !shortcut_name.empty() ? pending(x2_off) : kNone;
        if (!prologue && pin_x != kNone) {       // no normalisation in front: the pending bias enters as x * 1 + pending
            if (ones_off_ == kNone) {
                ones_off_ = alloc((size_t)cfg_.max_batch * max_c_ * 4);
                h_->fills.push_back({ones_off_, kNone, max_c_ * cfg_.max_batch, 1});
            }
            const size_t sh = alloc((size_t)cfg_.max_batch * Cin * 4);
            h_->fills.push_back({sh, pin_x, Cin, cfg_.max_batch});
            a.scale = ptr<float>(ones_off_);
            a.shift = ptr<float>(sh);
        }
        const size_t b2_off = a.bias2 ? (size_t)((const char*)a.bias2 - base_) : kNone;
        const size_t w2_off = a.w2 ? (size_t)((const char*)a.w2 - base_) : kNone;
        if (!y_is_frames) {
            if (tc && want_defer && !(cfg_.flags & VD_FLAG_FUSED_STATS)) {
                const size_t v = alloc((size_t)Cout * 4);
                h_->folds.push_back({v, pres, cw.b_off, b2_off, px2 != kNone ? w2_off : kNone, px2, Cin2, Cout});
                a.bias = nullptr;
                a.bias2 = nullptr;
                pending_[y_off] = v;
            } else {
                if (px2 != kNone) {               // the shortcut's share of its input's pending bias joins the shortcut bias
                    const size_t v2 = alloc((size_t)Cout * 4);
                    h_->folds.push_back({v2, kNone, kNone, b2_off, w2_off, px2, Cin2, Cout});
                    a.bias2 = ptr<float>(v2);
                }
                if (pres != kNone) pending_[y_off] = pres;      // accumulated in place: what was pending stays pending
                else pending_.erase(y_off);
            }
        }
        s.conv = a;
        s.use_tc = tc;
        s.has_residual = residual_off >= 0;
        fill_info(s, name, tc, Cin, Cout, ksize, upsample, H, W, Cout, out_dtype, out_nchw, y_is_frames ? -1 : (long)y_off);
        const double P = (double)H * W;
        s.info.flops_per_frame = 2.0 * ksize * ksize * Cin * (double)Cout * P;
        s.info.out_u8 = out_u8 ? 1 : 0;
        s.info.bytes_per_frame = (double)Hs * Ws * Cin * elt(in_dtype) + P * Cout * (out_u8 ? 1 : elt(out_dtype)) +
                                 (residual_off >= 0 ? P * Cout * 4.0 : 0.0);
        s.info.weight_bytes = (double)ksize * ksize * Cin * Cout * elt(cfg_.dtype);
        s.info.has_residual = residual_off >= 0;
        s.info.phase_collapsed = phase ? 1 : 0;
        if (!y_is_frames && pending(y_off) != kNone) s.info.out_pending_offset = (int64_t)pending(y_off);
        if (!shortcut_name.empty()) {
            s.info.c_in2 = Cin2;
            s.info.flops_per_frame += 2.0 * Cin2 * (double)Cout * P;
            s.info.bytes_per_frame += P * Cin2 * 4.0;
            s.info.weight_bytes += (double)Cin2 * Cout * elt(cfg_.dtype);
        }
        h_->steps.push_back(s);
    }

    void fill_info(Step& s, const std::string& name, int impl, int cin, int cout, int ksize, int up, int H, int W,
                   int oc, int odt, int nchw, long off) {
        memset(&s.info, 0, sizeof(s.info));
        snprintf(s.info.name, sizeof(s.info.name), "%s", name.c_str());
        s.info.kind = s.kind; s.info.impl = impl; s.info.launches = 1;
        s.info.c_in = cin; s.info.c_out = cout; s.info.ksize = ksize; s.info.upsample = up;
        s.info.out_h = H; s.info.out_w = W; s.info.out_channels = oc; s.info.out_dtype = odt;
        s.info.out_nchw = nchw; s.info.out_offset = off;
        s.info.out_pending_offset = -1;
    }

    // x -> shortcut(x) + conv2(silu(gn2(conv1(silu(gn1(x))))))
    void resblock(const std::string& p, int Cin, int Cout, int H, int W) {
        const size_t x = xs_[cur_x_], y = xs_[cur_x_ ^ 1];
        add_gn(p + ".norm1", x, VD_F32, H, W, Cin, p + ".norm1");
        defer_ = true;
        add_conv(p + ".conv1", {p + ".conv1"}, Cout, x, VD_F32, H, W, Cin, 3, false, true, true, -1, hbuf_, act_dtype(),
                 false, false);
        add_gn(p + ".norm2", hbuf_, act_dtype(), H, W, Cout, p + ".norm2");
        if (Cin == Cout) {
            // identity skip: conv2 accumulates into the residual stream in place (x += conv2(...))
            defer_ = true;
            add_conv(p + ".conv2", {p + ".conv2"}, Cout, hbuf_, act_dtype(), H, W, Cout, 3, false, true, true, (long)x, x,
                     VD_F32, false, false);
            return;
        }
        const bool fuse = bf16() && !(cfg_.flags & VD_FLAG_FORCE_SIMT) && Cout % 128 == 0 && Cin % 32 == 0;
        if (fuse) {      // the 1x1 shortcut rides along as extra K of conv2: no tensor of its own
            defer_ = true;
            add_conv(p + ".conv2", {p + ".conv2"}, Cout, hbuf_, act_dtype(), H, W, Cout, 3, false, true, true, -1, y,
                     VD_F32, false, false, p + ".shortcut", x, Cin);
        } else {
            add_conv(p + ".shortcut", {p + ".shortcut"}, Cout, x, VD_F32, H, W, Cin, 1, false, false, false, -1, y, VD_F32,
                     false, false);
            defer_ = true;
            add_conv(p + ".conv2", {p + ".conv2"}, Cout, hbuf_, act_dtype(), H, W, Cout, 3, false, true, true, (long)y, y,
                     VD_F32, false, false);
        }
        cur_x_ ^= 1;
    }

    void attention(const std::string& p, int C, int H, int W) {
        const size_t x = xs_[cur_x_];
        add_gn(p + ".norm", x, VD_F32, H, W, C, p + ".norm");
        add_conv(p + ".qkv", {p + ".q", p + ".k", p + ".v"}, C, x, VD_F32, H, W, C, 1, false, true, false, -1, qkv_,
                 act_dtype(), false, false);
        Step s{};
        s.kind = VD_STEP_ATTENTION;
        const int es = elt(act_dtype());
        s.attn = AttnArgs{ptr<void>(qkv_), ptr<void>(qkv_ + (size_t)C * es), ptr<void>(qkv_ + (size_t)2 * C * es),
                          ptr<void>(attno_), act_dtype(), 0, H * W, C, 3 * C, C, 1.0f / sqrtf((float)C), ptr<void>(vt_)};
        s.use_tc = bf16() && !(cfg_.flags & VD_FLAG_FORCE_SIMT) && attn_tc_supported(s.attn);
        fill_info(s, p + ".core", s.use_tc, C, C, 0, 0, H, W, C, act_dtype(), 0, (long)attno_);
        if (s.use_tc) s.info.launches = 2;               // V transpose + attention core
        const double T = (double)H * W;
        s.info.flops_per_frame = 4.0 * T * T * C;
        s.info.bytes_per_frame = 4.0 * T * C * es;
        h_->steps.push_back(s);
        defer_ = true;
        add_conv(p + ".o", {p + ".o"}, C, attno_, act_dtype(), H, W, C, 1, false, false, false, (long)x, x, VD_F32,
                 false, false);          // x += Wo o + bo, in place
    }

    void upconv(const std::string& p, int Cin, int Cout, int Hs, int Ws) {
        defer_ = true;
        add_conv(p, {p}, Cout, xs_[cur_x_], VD_F32, Hs, Ws, Cin, 3, true, false, false, -1, xs_[cur_x_ ^ 1], VD_F32,
                 false, false);
        cur_x_ ^= 1;
    }

    vd_status plan() {
        const int h = cfg_.latent_h, w = cfg_.latent_w, B = cfg_.max_batch;
        const int lc = cfg_.latent_channels;
        const size_t P0 = (size_t)h * w;
        // ---- sizes of the shared activation buffers (per frame), by walking the widths
        size_t max_x = 0, max_h = 0, max_s = 0, max_c = 0, qkv = 0, ao = 0;
        if (cfg_.arch == VD_ARCH_SDVAE) {
            const int ch[4] = {512, 512, 256, 128};
            size_t P = P0;
            max_x = P * 512;
            max_h = P * 512;
            max_c = 512;
            int prev = 512;
            for (int i = 0; i < 4; ++i) {
                max_x = std::max(max_x, P * (size_t)std::max(prev, ch[i]));
                max_h = std::max(max_h, P * (size_t)ch[i]);
                if (prev != ch[i]) max_s = std::max(max_s, P * (size_t)ch[i]);
                prev = ch[i];
                if (i < 3) { P *= 4; max_x = std::max(max_x, P * (size_t)ch[i]); }
            }
            qkv = P0 * 1536;
            ao = P0 * 512;
        } else {
            const int st[3][2] = {{64, 64}, {64, 32}, {32, 32}};
            size_t P = P0;
            max_x = P * 64; max_h = P * 64; max_c = 64;
            for (int i = 0; i < 3; ++i) {
                P *= 4;
                max_x = std::max(max_x, P * (size_t)st[i][1]);
                max_h = std::max(max_h, P * (size_t)st[i][1]);
            }
        }
        const int ae = elt(act_dtype());
        max_c_ = (int)max_c;
        h_->status_off = alloc(256);
        for (int i = 0; i < 2; ++i) {
            scale_buf_[i] = alloc((size_t)B * max_c * 4);
            shift_buf_[i] = alloc((size_t)B * max_c * 4);
        }
        scale_off_ = scale_buf_[0];
        shift_off_ = shift_buf_[0];
        partial_off_ = alloc(vd_gn_scratch_bytes(B, cfg_.norm_groups));
        h_->gn_counter_off = partial_off_ + gn_partial_bytes(B, cfg_.norm_groups);
        stat_off_ = alloc(conv_stat_scratch_bytes(B, cfg_.norm_groups));
        h_->stat_off = stat_off_;
        h_->stat_bytes = conv_stat_scratch_bytes(B, cfg_.norm_groups);
        zbuf_ = alloc((size_t)B * P0 * lc * 4);
        xs_[0] = alloc((size_t)B * max_x * 4);
        xs_[1] = alloc((size_t)B * max_x * 4);
        hbuf_ = alloc((size_t)B * max_h * ae);
        qkv_ = qkv ? alloc((size_t)B * qkv * ae) : 0;
        attno_ = ao ? alloc((size_t)B * ao * ae) : 0;
        vt_ = ao ? alloc(attn_tc_scratch_bytes(B, (int)P0, 512)) : 0;
        for (int i = 0; i < 2; ++i) {        // two of each: a copy runs while the other buffer is decoded from / into
            h_->lat_stage_off[i] = alloc((size_t)B * P0 * lc * elt(cfg_.dtype));
            h_->frm_stage_off[i] = alloc((size_t)B * P0 * 64 * cfg_.out_channels * elt(cfg_.dtype));
        }

        // ---- steps
        {
            Step s{};
            s.kind = VD_STEP_INGEST;
            s.ing = IngestArgs{nullptr, nullptr, nullptr, nullptr, 0.f, ptr<float>(zbuf_), cfg_.dtype, 0, lc, h, w};
            fill_info(s, "ingest", 0, lc, lc, 0, 0, h, w, lc, VD_F32, 0, (long)zbuf_);
            s.info.bytes_per_frame = (double)P0 * lc * (elt(cfg_.dtype) + 4);
            h_->steps.push_back(s);
        }
        cur_x_ = 0;
        int H = h, W = w;
        if (cfg_.arch == VD_ARCH_SDVAE) {
            add_conv("conv_in", {"conv_in"}, 512, zbuf_, VD_F32, H, W, lc, 3, false, false, false, -1, xs_[0], VD_F32, false, false);
            resblock("mid.res0", 512, 512, H, W);
            attention("mid.attn", 512, H, W);
            resblock("mid.res1", 512, 512, H, W);
            const int ch[4] = {512, 512, 256, 128};
            int prev = 512;
            for (int i = 0; i < 4; ++i) {
                for (int j = 0; j < 3; ++j) {
                    char nm[32];
                    snprintf(nm, sizeof(nm), "up%d.res%d", i, j);
                    resblock(nm, j == 0 ? prev : ch[i], ch[i], H, W);
                }
                prev = ch[i];
                if (i < 3) {
                    char nm[32];
                    snprintf(nm, sizeof(nm), "up%d.upconv", i);
                    upconv(nm, ch[i], ch[i], H, W);
                    H *= 2; W *= 2;
                }
            }
            head(prev, H, W);
        } else {
            add_conv("conv_in", {"conv_in"}, 64, zbuf_, VD_F32, H, W, lc, 3, false, false, false, -1, xs_[0], VD_F32, false, false);
            resblock("mid.res0", 64, 64, H, W);
            const int st[3][2] = {{64, 64}, {64, 32}, {32, 32}};
            for (int i = 0; i < 3; ++i) {
                char nm[32];
                snprintf(nm, sizeof(nm), "up%d.upconv", i);
                upconv(nm, st[i][0], st[i][1], H, W);
                H *= 2; W *= 2;
                snprintf(nm, sizeof(nm), "up%d.res0", i);
                resblock(nm, st[i][1], st[i][1], H, W);
            }
            head(32, H, W);
        }
        h_->total = align_up(cur_, 256);
        return VD_OK;
    }

    void head(int C, int H, int W) {
        add_gn("norm_out", xs_[cur_x_], VD_F32, H, W, C, "norm_out");
        const bool u8 = (cfg_.flags & VD_FLAG_OUT_U8) != 0;
        add_conv("conv_out", {"conv_out"}, cfg_.out_channels, xs_[cur_x_], VD_F32, H, W, C, 3, false, true, true, -1, 0,
                 cfg_.dtype, !u8, true, std::string(), 0, 0, u8);
    }

  private:
    vd_handle_s* h_;
    char* base_;
    const vd_config& cfg_;
    size_t cur_ = 0;
    size_t stat_off_ = 0;
    std::map<size_t, size_t> pending_;   // tensor offset -> offset of its pending-bias vector
    size_t pending(size_t off) const { auto it = pending_.find(off); return it == pending_.end() ? kNone : it->second; }
    bool defer_ = false;                 // set by the caller of add_conv: this layer's bias may be left pending
    size_t ones_off_ = kNone;
    int max_c_ = 0;
    size_t scale_off_ = 0, shift_off_ = 0, partial_off_ = 0, zbuf_ = 0, hbuf_ = 0, qkv_ = 0, attno_ = 0, vt_ = 0;
    size_t xs_[2] = {0, 0};
    size_t scale_buf_[2] = {0, 0}, shift_buf_[2] = {0, 0};
    int gn_toggle_ = 0;
    int cur_x_ = 0;
};

vd_status validate_cfg(const vd_config* cfg, std::string& err) {
    if (!cfg) { err = "config is NULL"; return VD_ERR_INVALID_ARG; }
    if (cfg->struct_size != sizeof(vd_config)) { err = "config.struct_size does not match this library"; return VD_ERR_INVALID_ARG; }
    if (cfg->arch != VD_ARCH_TINY && cfg->arch != VD_ARCH_SDVAE) { err = "unknown arch"; return VD_ERR_INVALID_ARG; }
    if (cfg->dtype != VD_F32 && cfg->dtype != VD_BF16) { err = "unknown dtype"; return VD_ERR_INVALID_ARG; }
    if (cfg->latent_channels != 4 || cfg->out_channels != 3) { err = "latent_channels must be 4 and out_channels 3"; return VD_ERR_UNSUPPORTED; }
    if (cfg->latent_h < 1 || cfg->latent_w < 1 || cfg->latent_h > 4096 || cfg->latent_w > 4096) { err = "latent size out of range"; return VD_ERR_INVALID_ARG; }
    if (cfg->max_batch < 1 || cfg->max_batch > 1024) { err = "max_batch out of range"; return VD_ERR_INVALID_ARG; }
    const int cmin = cfg->arch == VD_ARCH_SDVAE ? 128 : 32;
    if (cfg->norm_groups < 1 || cmin % cfg->norm_groups != 0 || (cmin / cfg->norm_groups) % 4 != 0) {
        err = "norm_groups must divide every width into groups of a multiple of 4 channels";
        return VD_ERR_INVALID_ARG;
    }
    if (!(cfg->norm_eps > 0.f) || !(cfg->norm_eps < 1.f)) { err = "norm_eps must be in (0,1)"; return VD_ERR_INVALID_ARG; }
    if (cfg->flags & ~(VD_FLAG_FORCE_SIMT | VD_FLAG_UPSAMPLE_9TAP | VD_FLAG_OUT_U8 | VD_FLAG_CANARY | VD_FLAG_FUSED_STATS)) { err = "unknown flag bits"; return VD_ERR_INVALID_ARG; }
    return VD_OK;
}

vd_status fail(vd_handle h, vd_status st, const std::string& msg) {
    if (h) h->err = msg;
    g_last_error = msg;
    return st;
}
vd_status cuda_fail(vd_handle h, cudaError_t e, const char* where) {
    return fail(h, VD_ERR_CUDA, std::string(where) + ": " + cudaGetErrorString(e));
}

const vd_tensor* find_tensor(const vd_tensor* t, int n, const std::string& name) {
    for (int i = 0; i < n; ++i)
        if (t[i].name && name == t[i].name) return &t[i];
    return nullptr;
}

cudaError_t launch_step(const vd_handle_s* h, const Step& st, int B, const void* latents, const void* v_prev,
                        float lambda, void* z_out, void* v_out, void* frames, cudaStream_t s) {
    unsigned int* status = (unsigned int*)(h->ws + h->status_off);
    switch (st.kind) {
        case VD_STEP_INGEST: {
            IngestArgs a = st.ing;
            a.B = B; a.z = latents; a.v_prev = v_prev; a.lambda = lambda; a.z_out = z_out; a.v_out = v_out;
            return launch_ingest(a, s);
        }
        case VD_STEP_GN_STATS: {
            GnArgs a = st.gn;
            a.B = B;
            return launch_gn_stats(a, s);
        }
        case VD_STEP_CONV: {
            ConvArgs a = st.conv;
            a.B = B;
            if (!a.y) a.y = frames;
            return st.use_tc ? launch_conv_tc(a, st.tc, status, s) : launch_conv_simt(a, s);
        }
        case VD_STEP_ATTENTION: {
            AttnArgs a = st.attn;
            a.B = B;
            return st.use_tc ? launch_attn_tc(a, &st.attn_tc, status, s) : launch_attn_simt(a, s);
        }
    }
    return cudaErrorInvalidValue;
}

}  // namespace

namespace vd {
static thread_local bool t_pdl_active = false;
bool pdl_enabled() { return t_pdl_active; }
PdlScope::PdlScope(bool on) : prev(t_pdl_active) { t_pdl_active = on; }
PdlScope::~PdlScope() { t_pdl_active = prev; }
}  // namespace vd

namespace {

vd_status decode_impl(vd_handle h, const void* latents, const void* v_prev, float lambda, void* z_out, void* v_out,
                      void* frames, int32_t batch, void* stream, float* ms, int n_ms) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    if (!latents || !frames) return fail(h, VD_ERR_INVALID_ARG, "latents/frames must not be NULL");
    if (batch < 1 || batch > h->cfg.max_batch) return fail(h, VD_ERR_INVALID_ARG, "batch must be in [1, max_batch]");
    const size_t al = h->cfg.dtype == VD_BF16 ? 2 : 4;
    const size_t fal = (h->cfg.flags & VD_FLAG_OUT_U8) ? 1 : al;
    if (((uintptr_t)latents % al) || ((uintptr_t)frames % fal)) return fail(h, VD_ERR_INVALID_ARG, "latents/frames are misaligned for their dtype");
    cudaStream_t s = (cudaStream_t)stream;
    const int n = h->stop_after >= 0 ? std::min((int)h->steps.size(), h->stop_after + 1) : (int)h->steps.size();
    std::vector<cudaEvent_t> ev;
    if (ms) {
        if (n_ms < (int)h->steps.size()) return fail(h, VD_ERR_INVALID_ARG, "ms array shorter than the number of steps");
        ev.resize(n + 1);
        for (auto& e : ev) {
            cudaError_t ce = cudaEventCreate(&e);
            if (ce != cudaSuccess) return cuda_fail(h, ce, "cudaEventCreate");
        }
        cudaEventRecord(ev[0], s);
    }
    PdlScope pdl(true);
    for (int i = 0; i < n; ++i) {
        cudaError_t e = launch_step(h, h->steps[i], batch, latents, v_prev, lambda, z_out, v_out, frames, s);
        if (e != cudaSuccess) {
            for (auto& x : ev) cudaEventDestroy(x);
            return cuda_fail(h, e, h->steps[i].info.name);
        }
        if (ms) cudaEventRecord(ev[i + 1], s);
    }
    if (ms) {
        cudaError_t e = cudaStreamSynchronize(s);
        for (int i = 0; i < (int)h->steps.size(); ++i) ms[i] = 0.f;
        if (e == cudaSuccess)
            for (int i = 0; i < n; ++i) cudaEventElapsedTime(&ms[i], ev[i], ev[i + 1]);
        for (auto& x : ev) cudaEventDestroy(x);
        if (e != cudaSuccess) return cuda_fail(h, e, "vd_profile synchronise");
    }
    return VD_OK;
}

}  // namespace

namespace vd {
void set_last_error(const char* msg) { g_last_error = msg ? msg : ""; }
}  // namespace vd

extern "C" {

vd_status vd_query_workspace(const vd_config* cfg, size_t* bytes) {
    std::string err;
    vd_status st = validate_cfg(cfg, err);
    if (st != VD_OK) return fail(nullptr, st, err);
    if (!bytes) return fail(nullptr, VD_ERR_INVALID_ARG, "bytes is NULL");
    vd_handle_s tmp;
    tmp.cfg = *cfg;
    Planner p(&tmp, nullptr);
    p.plan();
    *bytes = tmp.total;
    return VD_OK;
}

vd_status vd_create(const vd_config* cfg, const vd_tensor* weights, int32_t n_weights, void* workspace,
                    size_t workspace_bytes, void* cuda_stream, vd_handle* out) {
    if (out) *out = nullptr;
    std::string err;
    vd_status st = validate_cfg(cfg, err);
    if (st != VD_OK) return fail(nullptr, st, err);
    if (!out) return fail(nullptr, VD_ERR_INVALID_ARG, "out is NULL");
    if (!weights || n_weights <= 0) return fail(nullptr, VD_ERR_INVALID_ARG, "weights list is empty");
    if (!workspace || ((uintptr_t)workspace % 256)) return fail(nullptr, VD_ERR_INVALID_ARG, "workspace must be non-NULL and 256-byte aligned");

    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "device query");
    if (major != 10) return fail(nullptr, VD_ERR_UNSUPPORTED, "this library runs on sm_100 devices only");

    vd_handle_s* h = new vd_handle_s();
    h->cfg = *cfg;
    h->ws = (char*)workspace;
    h->ws_bytes = workspace_bytes;
    Planner p(h, h->ws);
    p.plan();
    if (workspace_bytes < h->total) {
        char msg[128];
        snprintf(msg, sizeof(msg), "workspace too small: %zu bytes given, %zu needed", workspace_bytes, h->total);
        delete h;
        return fail(nullptr, VD_ERR_WORKSPACE, msg);
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    e = cudaMemsetAsync(h->ws + h->status_off, 0, 256, s);
    // arrival counters of the GroupNorm statistics kernel: zero once, every launch leaves them zero
    if (e == cudaSuccess) e = cudaMemsetAsync(h->ws + h->gn_counter_off, 0, (size_t)cfg->max_batch * 4, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->ws + h->stat_off, 0, h->stat_bytes, s);   // likewise the sums and the counter of the convolutions that take statistics
    for (size_t g : h->guards)
        if (e == cudaSuccess) e = cudaMemsetAsync(h->ws + g, kGuardByte, kGuardBytes, s);
    if (e != cudaSuccess) { delete h; return cuda_fail(nullptr, e, "status memset"); }
    for (const WeightJob& j : h->jobs) {
        const vd_tensor* t = find_tensor(weights, n_weights, j.name);
        if (!t) { std::string m = "missing weight tensor: " + j.name; delete h; return fail(nullptr, VD_ERR_INVALID_ARG, m); }
        if (!t->dptr) { std::string m = "NULL pointer for " + j.name; delete h; return fail(nullptr, VD_ERR_INVALID_ARG, m); }
        if (t->dtype != cfg->dtype) { std::string m = "dtype of " + j.name + " differs from config.dtype"; delete h; return fail(nullptr, VD_ERR_INVALID_ARG, m); }
        int64_t want = j.kind == 1 ? j.Cout : (int64_t)j.Cout * j.Cin * j.taps;
        int64_t have = 1;
        if (t->ndim < 1 || t->ndim > 4) { std::string m = "bad ndim for " + j.name; delete h; return fail(nullptr, VD_ERR_INVALID_ARG, m); }
        for (int d = 0; d < t->ndim; ++d) have *= t->shape[d];
        bool ok = have == want && t->shape[0] == j.Cout;
        if (ok && j.kind != 1) ok = t->ndim >= 2 && t->shape[1] == j.Cin;
        if (!ok) { std::string m = "shape mismatch for " + j.name; delete h; return fail(nullptr, VD_ERR_INVALID_ARG, m); }
        if (j.kind == 1 || j.kind == 2) {
            e = launch_to_f32(t->dptr, t->dtype, (float*)(h->ws + j.dst_off), j.kind == 1 ? j.Cout : (int64_t)j.Cout * j.Cin, s);
        } else if (j.tc) {
            e = launch_pack_weight_tc(t->dptr, t->dtype, h->ws + j.dst_off, j.Cout, j.Cin, j.taps, j.cout_total, j.cout_offset, j.phase, s);
        } else {
            e = launch_pack_weight_simt(t->dptr, t->dtype, (float*)(h->ws + j.dst_off), j.Cout, j.Cin, j.taps, j.cout_total, j.cout_offset, s);
        }
        if (e != cudaSuccess) { delete h; return cuda_fail(nullptr, e, j.name.c_str()); }
    }
    auto at = [&](size_t off) -> float* { return off == kNone ? nullptr : (float*)(h->ws + off); };
    for (const FoldJob& f : h->folds) {
        e = launch_fold_bias(at(f.out_off), at(f.in_off), at(f.b_off), at(f.b2_off), at(f.w2_off), at(f.pin_off), f.Cin2, f.Cout, s);
        if (e != cudaSuccess) { delete h; return cuda_fail(nullptr, e, "bias fold"); }
    }
    for (const FillJob& f : h->fills) {
        e = launch_fill_rows(at(f.dst_off), at(f.src_off), f.C, f.B, s);
        if (e != cudaSuccess) { delete h; return cuda_fail(nullptr, e, "bias rows"); }
    }
    for (Step& st : h->steps) {
        if (st.kind == VD_STEP_CONV && st.use_tc) {
            ConvArgs pa = st.conv;
            pa.B = cfg->max_batch;
            e = conv_tc_prepare(pa, &st.tc);
            if (e == cudaErrorInvalidConfiguration && pa.upsample == 2) {
                delete h;
                return fail(nullptr, VD_ERR_UNSUPPORTED, "this device cannot co-schedule the CTA pairs of the phase-collapsed "
                                                         "upsampling convolution; set VD_FLAG_UPSAMPLE_9TAP");
            }
            if (e != cudaSuccess) { delete h; return cuda_fail(nullptr, e, "weight tensor map"); }
        }
    }
    for (Step& st : h->steps) {
        if (st.kind == VD_STEP_ATTENTION && st.use_tc) {
            AttnArgs pa = st.attn;
            pa.B = cfg->max_batch;
            e = attn_tc_prepare(pa, &st.attn_tc);
            if (e != cudaSuccess) { delete h; return cuda_fail(nullptr, e, "attention tensor maps"); }
        }
    }
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { delete h; return cuda_fail(nullptr, e, "vd_create synchronise"); }
    *out = h;
    return VD_OK;
}

vd_status vd_decode(vd_handle h, const void* latents, void* frames, int32_t batch, void* cuda_stream) {
    return decode_impl(h, latents, nullptr, 0.f, nullptr, nullptr, frames, batch, cuda_stream, nullptr, 0);
}

vd_status vd_decode_extrapolated(vd_handle h, const void* z_prev, const void* v_prev, float lambda, void* z_out,
                                 void* v_out, void* frames, int32_t batch, void* cuda_stream) {
    if (h && !v_prev) return fail(h, VD_ERR_INVALID_ARG, "v_prev must not be NULL");
    return decode_impl(h, z_prev, v_prev, lambda, z_out, v_out, frames, batch, cuda_stream, nullptr, 0);
}

vd_status vd_decode_host(vd_handle h, const void* latents_host, void* frames_host, int32_t batch, void* cuda_stream) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    if (!latents_host || !frames_host) return fail(h, VD_ERR_INVALID_ARG, "host buffers must not be NULL");
    if (batch < 1 || batch > h->cfg.max_batch) return fail(h, VD_ERR_INVALID_ARG, "batch must be in [1, max_batch]");
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t lat_bytes = h->latent_bytes(batch), frm_bytes = h->frame_bytes(batch);
    void* dl = h->ws + h->lat_stage_off[0];
    void* df = h->ws + h->frm_stage_off[0];
    cudaError_t e = cudaMemcpyAsync(dl, latents_host, lat_bytes, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(h, e, "latents host-to-device copy");
    vd_status st = decode_impl(h, dl, nullptr, 0.f, nullptr, nullptr, df, batch, cuda_stream, nullptr, 0);
    if (st != VD_OK) return st;
    e = cudaMemcpyAsync(frames_host, df, frm_bytes, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(h, e, "frames device-to-host copy");
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(h, e, "vd_decode_host synchronise");
    return VD_OK;
}

vd_status vd_decode_host_stream(vd_handle h, const void* latents_host, void* frames_host, int32_t n_frames,
                                int32_t batch, void* cuda_stream) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    if (!latents_host || !frames_host) return fail(h, VD_ERR_INVALID_ARG, "host buffers must not be NULL");
    if (batch < 1 || batch > h->cfg.max_batch) return fail(h, VD_ERR_INVALID_ARG, "batch must be in [1, max_batch]");
    if (n_frames < 0) return fail(h, VD_ERR_INVALID_ARG, "n_frames must not be negative");
    if (n_frames == 0) return VD_OK;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaSuccess;
    if (!h->pipe_ready) {
        e = cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking);
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_dec[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_out[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) return cuda_fail(h, e, "vd_decode_host_stream set-up");
        h->pipe_ready = true;
    }
    const int steps = (n_frames + batch - 1) / batch;
    const size_t lat1 = h->latent_bytes(1), frm1 = h->frame_bytes(1);
    auto frames_of = [&](int t) { return std::min(batch, n_frames - t * batch); };
    // Work of earlier calls on `cuda_stream` (and whatever it waits for) comes first: the copy streams join it.
    e = cudaEventRecord(h->ev_dec[0], s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_in, h->ev_dec[0], 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_out, h->ev_dec[0], 0);
    auto copy_in = [&](int t) -> cudaError_t {        // latents of step t -> device buffer t & 1
        const int k = t & 1;
        cudaError_t ce = cudaSuccess;
        if (t >= 2) ce = cudaStreamWaitEvent(h->copy_in, h->ev_dec[k], 0);          // the decode that read this buffer is done
        if (ce == cudaSuccess)
            ce = cudaMemcpyAsync(h->ws + h->lat_stage_off[k], (const char*)latents_host + (size_t)t * batch * lat1,
                                 lat1 * frames_of(t), cudaMemcpyHostToDevice, h->copy_in);
        if (ce == cudaSuccess) ce = cudaEventRecord(h->ev_in[k], h->copy_in);
        return ce;
    };
    if (e == cudaSuccess) e = copy_in(0);
    for (int t = 0; t < steps && e == cudaSuccess; ++t) {
        const int k = t & 1;
        if (t + 1 < steps) e = copy_in(t + 1);                                       // next latents travel during this decode
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, h->ev_in[k], 0);
        if (e == cudaSuccess && t >= 2) e = cudaStreamWaitEvent(s, h->ev_out[k], 0); // the copy that read this frame buffer is done
        if (e != cudaSuccess) break;
        vd_status st = decode_impl(h, h->ws + h->lat_stage_off[k], nullptr, 0.f, nullptr, nullptr, h->ws + h->frm_stage_off[k],
                                   frames_of(t), cuda_stream, nullptr, 0);
        if (st != VD_OK) { cudaStreamSynchronize(h->copy_in); cudaStreamSynchronize(h->copy_out); cudaStreamSynchronize(s); return st; }
        e = cudaEventRecord(h->ev_dec[k], s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_out, h->ev_dec[k], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync((char*)frames_host + (size_t)t * batch * frm1, h->ws + h->frm_stage_off[k], frm1 * frames_of(t),
                                cudaMemcpyDeviceToHost, h->copy_out);                // previous frames travel during the next decode
        if (e == cudaSuccess) e = cudaEventRecord(h->ev_out[k], h->copy_out);
    }
    // one wait at the end: every frame has reached the host, and `cuda_stream` is idle again
    cudaError_t e2 = cudaStreamSynchronize(h->copy_out);
    cudaError_t e3 = cudaStreamSynchronize(s);
    cudaError_t e4 = cudaStreamSynchronize(h->copy_in);
    if (e == cudaSuccess) e = e2 != cudaSuccess ? e2 : (e3 != cudaSuccess ? e3 : e4);
    return e == cudaSuccess ? VD_OK : cuda_fail(h, e, "vd_decode_host_stream");
}

vd_status vd_get_status(vd_handle h) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    unsigned int word[4] = {0, 0, 0, 0};
    cudaError_t e = cudaMemcpy(word, h->ws + h->status_off, sizeof(word), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(h, e, "status read");
    if (word[0] != 0) {
        char msg[160];
        const char* who = word[0] == kStatusConvTimeout ? "convolution" : word[0] == kStatusAttnTimeout ? "attention"
                          : word[0] == kStatusWaitProbe ? "wait probe" : "unknown";
        snprintf(msg, sizeof(msg), "a %s kernel gave up on a bounded wait (code 0x%x, block %u, detail 0x%x)", who, word[0], word[1], word[2]);
        return fail(h, VD_ERR_DEVICE_TIMEOUT, msg);
    }
    return VD_OK;
}

vd_status vd_clear_status(vd_handle h, void* cuda_stream) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    cudaError_t e = cudaMemsetAsync(h->ws + h->status_off, 0, 256, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? VD_OK : cuda_fail(h, e, "status clear");
}

const char* vd_last_error(vd_handle h) { return h ? h->err.c_str() : g_last_error.c_str(); }

vd_status vd_destroy(vd_handle h) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    delete h;
    return VD_OK;
}

vd_status vd_num_steps(vd_handle h, int32_t* n) {
    if (!h || !n) return fail(h, VD_ERR_INVALID_ARG, "NULL argument");
    *n = (int32_t)h->steps.size();
    return VD_OK;
}

vd_status vd_get_step(vd_handle h, int32_t index, vd_step_info* info) {
    if (!h || !info) return fail(h, VD_ERR_INVALID_ARG, "NULL argument");
    if (index < 0 || index >= (int)h->steps.size()) return fail(h, VD_ERR_INVALID_ARG, "step index out of range");
    *info = h->steps[index].info;
    return VD_OK;
}

vd_status vd_profile(vd_handle h, const void* latents, void* frames, int32_t batch, void* cuda_stream, float* ms,
                     int32_t n_steps) {
    if (!ms) return fail(h, VD_ERR_INVALID_ARG, "ms is NULL");
    return decode_impl(h, latents, nullptr, 0.f, nullptr, nullptr, frames, batch, cuda_stream, ms, n_steps);
}

vd_status vd_debug_status_offset(vd_handle h, int64_t* offset) {
    if (!h || !offset) return fail(h, VD_ERR_INVALID_ARG, "NULL argument");
    *offset = (int64_t)h->status_off;
    return VD_OK;
}

vd_status vd_debug_wait_probe(vd_handle h, int64_t limit_cycles, void* cuda_stream) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    if (limit_cycles < 1000 || limit_cycles > 2000000000LL)
        return fail(h, VD_ERR_INVALID_ARG, "limit_cycles must be in [1e3, 2e9]");
    cudaError_t e = launch_wait_probe((unsigned int*)(h->ws + h->status_off), (long long)limit_cycles, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? VD_OK : cuda_fail(h, e, "vd_debug_wait_probe");
}

vd_status vd_debug_check_canaries(vd_handle h, int32_t* n_guards) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    if (n_guards) *n_guards = (int32_t)h->guards.size();
    if (h->guards.empty()) return VD_OK;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(h, e, "vd_debug_check_canaries synchronise");
    std::vector<unsigned char> host(kGuardBytes);
    for (size_t i = 0; i < h->guards.size(); ++i) {
        e = cudaMemcpy(host.data(), h->ws + h->guards[i], kGuardBytes, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return cuda_fail(h, e, "vd_debug_check_canaries copy");
        for (size_t k = 0; k < kGuardBytes; ++k)
            if (host[k] != (unsigned char)kGuardByte) {
                char msg[160];
                snprintf(msg, sizeof(msg), "workspace guard %zu (offset %zu) was overwritten at byte %zu: a kernel wrote outside its buffer",
                         i, h->guards[i], k);
                return fail(h, VD_ERR_WORKSPACE, msg);
            }
    }
    return VD_OK;
}

vd_status vd_debug_stop_after(vd_handle h, int32_t index) {
    if (!h) return fail(nullptr, VD_ERR_INVALID_ARG, "handle is NULL");
    if (index < -1 || index >= (int)h->steps.size()) return fail(h, VD_ERR_INVALID_ARG, "step index out of range");
    h->stop_after = index;
    return VD_OK;
}

// ------------------------------------------------------------------ operator-level entry points
static vd_status check_conv_desc(const vd_conv_desc* d) {
    if (!d || d->struct_size != sizeof(vd_conv_desc)) return fail(nullptr, VD_ERR_INVALID_ARG, "bad conv descriptor");
    if (d->batch < 0 || d->in_h < 1 || d->in_w < 1 || d->c_in < 1 || d->c_out < 1) return fail(nullptr, VD_ERR_INVALID_ARG, "bad conv sizes");
    if (d->ksize != 1 && d->ksize != 3) return fail(nullptr, VD_ERR_INVALID_ARG, "ksize must be 1 or 3");
    if ((d->in_dtype != VD_F32 && d->in_dtype != VD_BF16) || (d->out_dtype != VD_F32 && d->out_dtype != VD_BF16))
        return fail(nullptr, VD_ERR_INVALID_ARG, "bad dtype");
    if (d->impl < VD_IMPL_AUTO || d->impl > VD_IMPL_TC) return fail(nullptr, VD_ERR_INVALID_ARG, "bad impl");
    if (d->upsample < 0 || d->upsample > 2) return fail(nullptr, VD_ERR_INVALID_ARG, "upsample must be 0, 1 or 2");
    return VD_OK;
}

static ConvArgs conv_args_from_desc(const vd_conv_desc* d) {
    ConvArgs a{};
    a.B = d->batch; a.Hs = d->in_h; a.Ws = d->in_w;
    a.H = d->upsample ? 2 * d->in_h : d->in_h;
    a.W = d->upsample ? 2 * d->in_w : d->in_w;
    a.Cin = d->c_in; a.Cout = d->c_out; a.ksize = d->ksize; a.upsample = d->upsample; a.silu = d->silu ? 1 : 0;
    a.in_dtype = d->in_dtype; a.out_dtype = d->out_dtype; a.out_nchw = d->out_nchw ? 1 : 0;
    a.bf16_operands = d->bf16_operands ? 1 : 0;
    return a;
}

static vd_status resolve_impl(const vd_conv_desc* d, const ConvArgs& a, bool* tc) {
    ConvArgs probe = a;
    probe.B = 1;
    const bool can = a.bf16_operands && conv_tc_supported(probe);
    if (d->impl == VD_IMPL_TC && !can) return fail(nullptr, VD_ERR_UNSUPPORTED, "the tensor-core convolution does not support this shape");
    *tc = d->impl == VD_IMPL_TC || (d->impl == VD_IMPL_AUTO && can);
    if (!*tc && a.upsample == 2) return fail(nullptr, VD_ERR_UNSUPPORTED, "the phase-collapsed upsampling form exists in the tensor-core kernel only");
    return VD_OK;
}

vd_status vd_conv_packed_weight_bytes(const vd_conv_desc* d, size_t* bytes) {
    vd_status st = check_conv_desc(d);
    if (st != VD_OK) return st;
    if (!bytes) return fail(nullptr, VD_ERR_INVALID_ARG, "bytes is NULL");
    bool tc;
    st = resolve_impl(d, conv_args_from_desc(d), &tc);
    if (st != VD_OK) return st;
    const int taps = d->ksize * d->ksize;
    *bytes = tc ? conv_tc_packed_bytes(d->c_out, d->c_in, taps, d->upsample == 2) : (size_t)taps * d->c_in * d->c_out * 4;
    return VD_OK;
}

vd_status vd_conv_pack_weight(const vd_conv_desc* d, const void* w_oihw, int32_t w_dtype, void* packed, void* cuda_stream) {
    vd_status st = check_conv_desc(d);
    if (st != VD_OK) return st;
    if (!w_oihw || !packed) return fail(nullptr, VD_ERR_INVALID_ARG, "NULL pointer");
    if (w_dtype != VD_F32 && w_dtype != VD_BF16) return fail(nullptr, VD_ERR_INVALID_ARG, "bad dtype");
    bool tc;
    st = resolve_impl(d, conv_args_from_desc(d), &tc);
    if (st != VD_OK) return st;
    const int taps = d->ksize * d->ksize;
    cudaError_t e = tc ? launch_pack_weight_tc(w_oihw, w_dtype, packed, d->c_out, d->c_in, taps, d->c_out, 0, d->upsample == 2, (cudaStream_t)cuda_stream)
                       : launch_pack_weight_simt(w_oihw, w_dtype, (float*)packed, d->c_out, d->c_in, taps, d->c_out, 0, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? VD_OK : cuda_fail(nullptr, e, "vd_conv_pack_weight");
}

vd_status vd_op_conv2d(const vd_conv_desc* d, const void* x, const void* w_packed, const float* bias, const float* scale,
                       const float* shift, const float* residual, void* y, void* cuda_stream) {
    vd_status st = check_conv_desc(d);
    if (st != VD_OK) return st;
    if (!x || !w_packed || !y) return fail(nullptr, VD_ERR_INVALID_ARG, "NULL pointer");
    if ((scale == nullptr) != (shift == nullptr)) return fail(nullptr, VD_ERR_INVALID_ARG, "scale and shift go together");
    if (d->batch == 0) return VD_OK;
    ConvArgs a = conv_args_from_desc(d);
    a.x = x; a.w = w_packed; a.bias = bias; a.scale = scale; a.shift = shift; a.residual = residual; a.y = y;
    bool tc;
    st = resolve_impl(d, a, &tc);
    if (st != VD_OK) return st;
    cudaError_t e;
    if (tc) {
        ConvTcPlan plan{};
        if (a.residual && a.residual != (const float*)a.y) {
            // the tensor-core kernel accumulates into its output: seed it with the residual
            const size_t n = (size_t)a.B * a.H * a.W * a.Cout * sizeof(float);
            e = a.out_dtype == VD_F32 ? cudaMemcpyAsync(a.y, a.residual, n, cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream)
                                      : cudaErrorInvalidValue;
            if (e != cudaSuccess) return cuda_fail(nullptr, e, "vd_op_conv2d (a residual needs an fp32 output)");
            a.residual = (const float*)a.y;
        }
        e = conv_tc_prepare(a, &plan);
        if (e == cudaSuccess) e = launch_conv_tc(a, plan, nullptr, (cudaStream_t)cuda_stream);
    } else {
        e = launch_conv_simt(a, (cudaStream_t)cuda_stream);
    }
    return e == cudaSuccess ? VD_OK : cuda_fail(nullptr, e, "vd_op_conv2d");
}

size_t vd_conv_stats_scratch_bytes(int32_t batch, int32_t groups) {
    if (batch < 1 || groups < 1) return 0;
    return conv_stat_scratch_bytes(batch, groups);
}

vd_status vd_op_conv2d_stats(const vd_conv_desc* d, const void* x, const void* w_packed, const float* bias, const float* scale,
                             const float* shift, void* y, int32_t groups, float eps, const float* gamma, const float* beta,
                             float* out_scale, float* out_shift, void* scratch, void* cuda_stream) {
    vd_status st = check_conv_desc(d);
    if (st != VD_OK) return st;
    if (!x || !w_packed || !y || !gamma || !beta || !out_scale || !out_shift || !scratch) return fail(nullptr, VD_ERR_INVALID_ARG, "NULL pointer");
    if ((scale == nullptr) != (shift == nullptr)) return fail(nullptr, VD_ERR_INVALID_ARG, "scale and shift go together");
    if (groups < 1) return fail(nullptr, VD_ERR_INVALID_ARG, "bad group count");
    if (d->batch == 0) return VD_OK;
    ConvArgs a = conv_args_from_desc(d);
    a.x = x; a.w = w_packed; a.bias = bias; a.scale = scale; a.shift = shift; a.y = y;
    bool tc;
    st = resolve_impl(d, a, &tc);
    if (st != VD_OK) return st;
    if (!tc || !conv_tc_stats_supported(a, groups))
        return fail(nullptr, VD_ERR_UNSUPPORTED, "this layer's epilogue cannot take GroupNorm statistics");
    a.stat_sum = (unsigned long long*)scratch;
    a.stat_counter = (unsigned int*)((char*)scratch + conv_stat_sum_bytes(a.B, groups));
    a.stat_gamma = gamma; a.stat_beta = beta; a.stat_scale = out_scale; a.stat_shift = out_shift;
    a.stat_G = groups; a.stat_eps = eps;
    cudaError_t e = cudaMemsetAsync(scratch, 0, conv_stat_scratch_bytes(a.B, groups), (cudaStream_t)cuda_stream);
    ConvTcPlan plan{};
    if (e == cudaSuccess) e = conv_tc_prepare(a, &plan);
    if (e == cudaSuccess) e = launch_conv_tc(a, plan, nullptr, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? VD_OK : cuda_fail(nullptr, e, "vd_op_conv2d_stats");
}

size_t vd_gn_scratch_bytes(int32_t batch, int32_t groups) {
    if (batch < 1 || groups < 1) return 0;
    return gn_scratch_bytes(batch, groups);
}

vd_status vd_op_gn_stats(const void* x, int32_t dtype, int32_t batch, int32_t h, int32_t w, int32_t c, int32_t groups,
                         float eps, const float* gamma, const float* beta, const float* offset, float* scale, float* shift,
                         void* scratch, void* cuda_stream) {
    if (!x || !gamma || !beta || !scale || !shift || !scratch) return fail(nullptr, VD_ERR_INVALID_ARG, "NULL pointer");
    if (dtype != VD_F32 && dtype != VD_BF16) return fail(nullptr, VD_ERR_INVALID_ARG, "bad dtype");
    if (batch < 0 || h < 1 || w < 1 || c < 1 || groups < 1 || c % groups != 0 || (c / groups) % 4 != 0 || c > 1024)
        return fail(nullptr, VD_ERR_INVALID_ARG, "bad GroupNorm sizes (groups must hold a multiple of 4 channels)");
    if ((long long)h * w > 0x7fffffffLL || (long long)batch * h * w * c > (1LL << 40))
        return fail(nullptr, VD_ERR_INVALID_ARG, "tensor too large (h*w must fit 31 bits, batch*h*w*c 40 bits)");
    if (batch == 0) return VD_OK;
    unsigned int* counters = (unsigned int*)((char*)scratch + gn_partial_bytes(batch, groups));
    GnArgs a{x, dtype, batch, h * w, c, groups, eps, gamma, beta, scale, shift, (float*)scratch, counters, offset};
    cudaError_t e = cudaMemsetAsync(counters, 0, (size_t)batch * sizeof(unsigned int), (cudaStream_t)cuda_stream);
    if (e == cudaSuccess) e = launch_gn_stats(a, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? VD_OK : cuda_fail(nullptr, e, "vd_op_gn_stats");
}

size_t vd_attention_scratch_bytes(int32_t batch, int32_t tokens, int32_t channels) {
    if (batch < 1 || tokens < 1 || channels < 1) return 0;
    return attn_tc_scratch_bytes(batch, tokens, channels);
}

vd_status vd_op_attention(const void* q, const void* k, const void* v, void* o, int32_t dtype, int32_t batch,
                          int32_t tokens, int32_t channels, int32_t ld_qkv, int32_t ld_o, float scale, int32_t impl,
                          void* scratch, void* cuda_stream) {
    if (!q || !k || !v || !o) return fail(nullptr, VD_ERR_INVALID_ARG, "NULL pointer");
    if (dtype != VD_F32 && dtype != VD_BF16) return fail(nullptr, VD_ERR_INVALID_ARG, "bad dtype");
    if (batch < 0 || tokens < 1 || channels < 32 || channels % 32 != 0 || channels > 512 || ld_qkv < channels || ld_o < channels)
        return fail(nullptr, VD_ERR_INVALID_ARG, "bad attention sizes");
    if (impl < VD_IMPL_AUTO || impl > VD_IMPL_TC) return fail(nullptr, VD_ERR_INVALID_ARG, "bad impl");
    if (batch == 0) return VD_OK;
    AttnArgs a{q, k, v, o, dtype, batch, tokens, channels, ld_qkv, ld_o, scale, scratch};
    const bool can = attn_tc_supported(a) && scratch != nullptr;
    if (impl == VD_IMPL_TC && !can) return fail(nullptr, VD_ERR_UNSUPPORTED, "the tensor-core attention does not support this shape");
    const bool tc = impl == VD_IMPL_TC || (impl == VD_IMPL_AUTO && can);
    cudaError_t e = tc ? launch_attn_tc(a, nullptr, nullptr, (cudaStream_t)cuda_stream) : launch_attn_simt(a, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? VD_OK : cuda_fail(nullptr, e, "vd_op_attention");
}

}  // extern "C"
