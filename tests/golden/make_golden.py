"""Writes the oracle frames of the full-size workloads that the GPU parity tests compare with.

Calls only the oracle (`oracle/`) and the seeded input generators.

    python tests/golden/make_golden.py 3 4 5          # frames_cfg{3,4,5}.npz
    python tests/golden/make_golden.py --full 3 4 5   # frame_cfg{3,4,5}_full.npz

Without --full: for every frame of the workload the whole decoder is run by the oracle; kept are
all three channels at a fixed set of pixel positions (image corners, points along the four
borders, and seeded random positions), plus each frame's mean, standard deviation and L2 norm.
With --full: the LAST frame of the workload is kept whole (every pixel, fp32), so that the
max-abs bar can be checked over the complete frame.

About 90 s of an 8-core host per 720x480 frame, 280 s per 1280x720 one.
"""
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import ref                                # noqa: E402
from paper_2602_00608_b200 import synth               # noqa: E402

N_RANDOM = 2048


def sample_positions(h: int, w: int) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=777))
    pos = [(0, 0), (0, w - 1), (h - 1, 0), (h - 1, w - 1)]
    for t in np.linspace(0, 1, 33)[1:-1]:
        i, j = int(t * (h - 1)), int(t * (w - 1))
        pos += [(0, j), (h - 1, j), (i, 0), (i, w - 1)]
    ri = rng.integers(0, h, size=N_RANDOM)
    rj = rng.integers(0, w, size=N_RANDOM)
    pos += list(zip(ri.tolist(), rj.tolist()))
    return np.asarray(pos, dtype=np.int32)


def main(indices):
    for idx in indices:
        wl = synth.WORKLOADS[idx]
        wts = synth.workload_weights(wl)
        z = synth.workload_latents(wl)
        pos = sample_positions(wl.out_h, wl.out_w)
        vals = np.empty((wl.batch, wl.out_channels, len(pos)), np.float32)
        stats = np.empty((wl.batch, 3), np.float64)
        for b in range(wl.batch):
            t0 = time.time()
            y = ref.decode(wl.arch, wts, z[b:b + 1], wl.groups, wl.eps)[0]
            vals[b] = y[:, pos[:, 0], pos[:, 1]]
            y64 = y.astype(np.float64)
            stats[b] = (y64.mean(), y64.std(), np.sqrt((y64 * y64).sum()))
            print(f"cfg {idx} frame {b}: {time.time() - t0:.1f} s, std {stats[b, 1]:.4f}", flush=True)
        out = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"frames_cfg{idx}.npz")
        np.savez_compressed(out, positions=pos, values=vals, stats=stats)
        print("wrote", out, os.path.getsize(out), "bytes", flush=True)


def main_full(indices):
    for idx in indices:
        wl = synth.WORKLOADS[idx]
        wts = synth.workload_weights(wl)
        z = synth.workload_latents(wl)
        b = wl.batch - 1
        t0 = time.time()
        y = ref.decode(wl.arch, wts, z[b:b + 1], wl.groups, wl.eps)[0]
        print(f"cfg {idx} frame {b}: {time.time() - t0:.1f} s", flush=True)
        out = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"frame_cfg{idx}_full.npz")
        np.savez_compressed(out, frame=y.astype(np.float32), index=np.int32(b))
        print("wrote", out, os.path.getsize(out), "bytes", flush=True)


if __name__ == "__main__":
    argv = sys.argv[1:]
    full = "--full" in argv
    idxs = [int(a) for a in argv if a != "--full"] or [3, 4, 5]
    (main_full if full else main)(idxs)
