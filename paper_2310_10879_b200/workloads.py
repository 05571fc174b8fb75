"""Seeded synthetic inputs: sequence lengths and frame payloads.

This module holds no arithmetic of the packing method.  It only draws the
inputs that both the GPU library and the CPU checker are fed with, so that the
two can be compared on identical data.  The five workloads follow the shapes of
the evaluation configurations (toy video, per-frame features, raw frames,
token sequences, heavy-tailed feature sequences); a sixth has the shape of the
video dataset used in the paper's experiments (N=7,464 clips of 3..94 frames)
and is a synthetic stand-in, not that dataset; a seventh ("random_chunks") is a
probe of the memory system, not a workload of the paper.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    index: int          # position in the list of evaluation configurations (0-based), -1 for extras
    n: int              # number of sequences
    t_block: int        # block length in frames
    frame_bytes: int    # bytes of one frame in the ragged store
    out_frame_bytes: int  # bytes of one frame of the per-frame model output that is unpacked
    batch_blocks: int   # blocks per training batch
    dist: str           # length distribution
    payload: str        # element type / distribution of the payload
    pad_byte: int = 0

    @property
    def seed(self) -> int:
        return 1000 + self.index


WORKLOADS = {
    "toy_video": Workload("toy_video", 0, 64, 64, 3 * 64 * 64, 3 * 64 * 64, 8, "uniform[2,64]", "u8"),
    "features_fp16": Workload("features_fp16", 1, 1000, 1000, 1024 * 2, 1024 * 2, 16,
                              "lognormal(median 30, sigma 1) clip [1,1000]", "f16"),
    "raw_frames": Workload("raw_frames", 2, 500, 900, 3 * 224 * 224, 3 * 224 * 224, 4,
                           "geometric(mean 60) clip [1,900]", "u8"),
    "tokens": Workload("tokens", 3, 1_000_000, 4096, 4, 4, 64, "zipf(1.2) clip [8,4096]", "i32"),
    "heavy_tail_bf16": Workload("heavy_tail_bf16", 4, 20_000, 10_000, 2048 * 2, 2048 * 4, 8,
                                "pareto(1.5, min 20) clip [1,10000]", "bf16"),
    # shape of the paper's training set (Experiments section): N clips, 3..94 frames, mean about 22.3
    "video_dataset_shape": Workload("video_dataset_shape", 5, 7464, 94, 64, 64, 8,
                                    "3 + geometric(mean 19.3) clip [3,94]", "u8"),
    # Not one of the evaluation configurations: a probe of the memory system.  Every sequence is one frame and every block
    # one slot, so the plan is a random permutation and pack / unpack copy equal-sized, 16-byte aligned chunks in random
    # order.  It measures what a copy of chunks of that size can reach on the device, whichever kernel moves them; other
    # chunk sizes with bench.py's --frame-bytes (and --n to keep the total at a few GB).
    "random_chunks": Workload("random_chunks", 6, 262_144, 1, 16384, 16384, 256, "all 1 (one frame per sequence and block)", "u8"),
}

# The toy dataset of the paper's problem statement: 8 videos of 2..6 frames, two of
# length 2 and two of length 6.  The figure that lists them is not available; the four
# middle values here are a stand-in (tests also run every other completion).
TOY8_LENGTHS = np.array([2, 2, 3, 3, 4, 5, 6, 6], dtype=np.int32)
TOY8_T_BLOCK = 6


def scaled(w: Workload, n: int) -> Workload:
    """Same distributions, fewer sequences (for quick checks)."""
    return replace(w, n=n)


def lengths(w: Workload, seed: int | None = None) -> np.ndarray:
    """int32[n] sequence lengths, 1 <= T_i <= t_block, from numpy's PCG64."""
    rng = np.random.Generator(np.random.PCG64(w.seed if seed is None else seed))
    n = w.n
    if w.name == "toy_video":
        t = rng.integers(2, 65, size=n)
    elif w.name == "features_fp16":
        t = np.clip(np.rint(rng.lognormal(np.log(30.0), 1.0, size=n)), 1, 1000)
    elif w.name == "raw_frames":
        t = np.clip(rng.geometric(1.0 / 60.0, size=n), 1, 900)
    elif w.name == "tokens":
        t = np.clip(rng.zipf(1.2, size=n), 8, 4096)
    elif w.name == "heavy_tail_bf16":
        t = np.clip(np.floor(20.0 * (1.0 + rng.pareto(1.5, size=n))), 1, 10_000)
    elif w.name == "video_dataset_shape":
        t = np.clip(2 + rng.geometric(1.0 / 20.3, size=n), 3, 94)
    elif w.name == "random_chunks":
        t = np.ones(n)
    else:
        raise KeyError(w.name)
    t = np.minimum(t, w.t_block)
    return np.ascontiguousarray(t, dtype=np.int32)


def payload_bytes_numpy(n_bytes: int, seed: int) -> np.ndarray:
    """uint8[n_bytes] of uniform random bytes (host).  Payload values never steer control flow;
    any bit pattern is a legal frame, so raw bytes also stand in for fp16/bf16/int32 payloads
    in bit-exactness checks (NaN patterns included on purpose)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, 256, size=n_bytes, dtype=np.uint8)


def payload_torch(w: Workload, n_frames: int, device, seed: int | None = None, out: bool = False):
    """Typed payload on `device` with the value distribution of the workload:
    u8 uniform, f16/bf16 ~ N(0,1), i32 token ids uniform in [0, 50000).  With out=True the
    tensor has the shape of the per-frame model output (fp32 for the bf16 workload).
    Returns a 2-D tensor [n_frames, elements_per_frame]."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed((w.seed if seed is None else seed) * 7919 + (1 if out else 0))
    fb = w.out_frame_bytes if out else w.frame_bytes
    kind = w.payload
    if out and w.out_frame_bytes != w.frame_bytes:
        kind = "f32"
    if kind == "u8":
        return torch.randint(0, 256, (n_frames, fb), dtype=torch.uint8, device=device, generator=g)
    if kind == "i32":
        return torch.randint(0, 50000, (n_frames, fb // 4), dtype=torch.int32, device=device, generator=g)
    dt = {"f16": torch.float16, "bf16": torch.bfloat16, "f32": torch.float32}[kind]
    esz = {"f16": 2, "bf16": 2, "f32": 4}[kind]
    x = torch.empty((n_frames, fb // esz), dtype=dt, device=device)
    # fill in slabs to bound the temporary memory of the normal sampler
    step = max(1, (256 << 20) // max(1, fb))
    for lo in range(0, n_frames, step):
        x[lo:lo + step].normal_(0.0, 1.0, generator=g)
    return x
