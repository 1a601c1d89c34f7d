"""Seeded synthetic inputs shared by the CUDA path's tests/bench and by the CPU
oracle's tests.  Holds no attention arithmetic: only shapes, seeds and random
draws.  Both sides receive the same bf16 bytes.

Workload shapes: the five benchmark configurations (tiny, 8K, 32K, 128K
training, 128K decode).  Values: Q/K/V/dO ~ N(0,1) drawn in fp32 from a seeded
torch generator and rounded once to bf16; softmax scale 1/sqrt(D).  Seeds are
config_index*1000 + tensor_index (Q 0, K 1, V 2, dO 3, lens 4).  Decode cache
positions at or beyond lens[b] hold NaN so that an over-read shows up.
"""
from __future__ import annotations

import math

import torch

CONFIGS = {
    "tiny": dict(index=0, B=1, T=1024, Hq=4, Hkv=2, D=64, sink=64, local=128, block=64),
    "8k": dict(index=1, B=2, T=8192, Hq=16, Hkv=4, D=128, sink=128, local=1024, block=128),
    "32k": dict(index=2, B=1, T=32768, Hq=32, Hkv=8, D=128, sink=128, local=2048, block=128),
    "128k": dict(index=3, B=1, T=131072, Hq=32, Hkv=8, D=128, sink=128, local=4096, block=128),
    "decode128k": dict(index=4, B=8, Tmax=131072, Hq=32, Hkv=8, D=128, sink=128, local=4096,
                       block=128, len_lo=98304, len_hi=131072),
}


def softmax_scale(D):
    return 1.0 / math.sqrt(D)


def _normal_bf16(shape, seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    # Drawn in chunks along the first axis to bound the fp32 temporary.
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(shape[0], -1)
    for i in range(shape[0]):
        flat[i] = torch.randn(flat.shape[1], generator=g, dtype=torch.float32,
                              device=device).to(torch.bfloat16)
    return out


def make_train_inputs(index, B, T, Hq, Hkv, D, device="cpu"):
    """q, k, v, d_o as bf16 tensors [B,H,T,D] (head-major, D contiguous)."""
    q = _normal_bf16((B, Hq, T, D), index * 1000 + 0, device)
    k = _normal_bf16((B, Hkv, T, D), index * 1000 + 1, device)
    v = _normal_bf16((B, Hkv, T, D), index * 1000 + 2, device)
    d_o = _normal_bf16((B, Hq, T, D), index * 1000 + 3, device)
    return q, k, v, d_o


def make_decode_inputs(index, B, Tmax, Hq, Hkv, D, len_lo, len_hi, device="cpu"):
    """q [B,Hq,D], kcache/vcache [B,Hkv,Tmax,D] bf16, lens int32 [B] in
    [len_lo, len_hi]; cache rows >= lens[b] are NaN."""
    q = _normal_bf16((B, Hq, D), index * 1000 + 0, device)
    kc = _normal_bf16((B, Hkv, Tmax, D), index * 1000 + 1, device)
    vc = _normal_bf16((B, Hkv, Tmax, D), index * 1000 + 2, device)
    g = torch.Generator(device="cpu")
    g.manual_seed(index * 1000 + 4)
    lens = torch.randint(int(len_lo), int(len_hi) + 1, (B,), generator=g, dtype=torch.int64)
    lens = lens.to(torch.int32)
    for b in range(B):
        n = int(lens[b])
        if n < Tmax:
            kc[b, :, n:] = float("nan")
            vc[b, :, n:] = float("nan")
    return q, kc, vc, lens.to(device)


def to_f64(t):
    """bf16 tensor -> float64 numpy array with the same values (for the oracle)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
