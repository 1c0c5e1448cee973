"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds none of the method's arithmetic: it only draws numbers.  Values are
drawn in fp32 on the CPU from a seeded ``torch.Generator`` and rounded to the I/O dtype
first, so the oracle and the GPU library see identical bits.

The five workload recipes (stand-ins for the shapes of BERT / GPT attention tensors; the
paper states no activation distribution, so entries are iid standard normal):
  1  tiny causal fp32      B=1  H=2  N=256   d=32 ; Q,K rows times exp(N(0,1))
  2  bidirectional bf16    B=32 H=12 N=512   d=64
  3  causal bf16           B=8  H=12 N=1024  d=64 ; 5 % of K rows exactly zero
  4  causal fwd+bwd bf16   B=4  H=16 N=4096  d=64 ; plus dO ~ N(0,1)
  5  long causal bf16      B=1  H=16 N in {4096,16384,65536,131072} d=128,
     and decode: B=64 H=16 d=128, prefill 8192 then 1024 single-token steps
"""
from __future__ import annotations

import torch

CONFIGS = {
    1: dict(B=1, H=2, N=256, d=32, dtype=torch.float32, causal=True),
    2: dict(B=32, H=12, N=512, d=64, dtype=torch.bfloat16, causal=False),
    3: dict(B=8, H=12, N=1024, d=64, dtype=torch.bfloat16, causal=True),
    4: dict(B=4, H=16, N=4096, d=64, dtype=torch.bfloat16, causal=True),
    5: dict(B=1, H=16, N=4096, d=128, dtype=torch.bfloat16, causal=True),
}
C5_SWEEP_N = (4096, 16384, 65536, 131072)
C5_DECODE = dict(B=64, H=16, d=128, prefill=8192, steps=1024)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def normal(shape, dtype, gen: torch.Generator) -> torch.Tensor:
    return torch.randn(shape, generator=gen, dtype=torch.float32).to(dtype)


def make_qkv(B, H, N, d, dtype, seed, row_lognormal=False, zero_k_frac=0.0, with_do=False, d_v=None):
    """Returns a dict with q,k,v (and d_o) ``[B,H,N,d]`` in ``dtype`` and m ``[H]`` fp32.
    ``d_v``: value size when it differs from the key size d (v and d_o are ``[B,H,N,d_v]``)."""
    g = _gen(seed)
    d_v = d if d_v is None else d_v
    q = torch.randn((B, H, N, d), generator=g, dtype=torch.float32)
    k = torch.randn((B, H, N, d), generator=g, dtype=torch.float32)
    v = torch.randn((B, H, N, d_v), generator=g, dtype=torch.float32)
    m = torch.randn((H,), generator=g, dtype=torch.float32)
    if row_lognormal:  # exercises the normalisation: rows of wildly different length
        q = q * torch.exp(torch.randn((B, H, N, 1), generator=g, dtype=torch.float32))
        k = k * torch.exp(torch.randn((B, H, N, 1), generator=g, dtype=torch.float32))
    if zero_k_frac > 0.0:  # exactly-zero key rows exercise the norm floor
        n_zero = int(zero_k_frac * N)
        for b in range(B):
            for h in range(H):
                idx = torch.randperm(N, generator=g)[:n_zero]
                k[b, h, idx, :] = 0.0
    out = {"q": q.to(dtype), "k": k.to(dtype), "v": v.to(dtype), "m": m}
    if with_do:
        out["d_o"] = torch.randn((B, H, N, d_v), generator=g, dtype=torch.float32).to(dtype)
    return out


def make_config(idx: int, N: int | None = None, B: int | None = None, with_do: bool | None = None):
    """Inputs of workload ``idx`` (1..5); ``N`` / ``B`` override the size (config 5 sweep,
    reduced parity cases).  Seed is ``1000 + idx`` (plus N for the sweep)."""
    c = dict(CONFIGS[idx])
    if N is not None:
        c["N"] = N
    if B is not None:
        c["B"] = B
    seed = 1000 + idx + (c["N"] if idx == 5 else 0)
    data = make_qkv(c["B"], c["H"], c["N"], c["d"], c["dtype"], seed,
                    row_lognormal=(idx == 1), zero_k_frac=(0.05 if idx == 3 else 0.0),
                    with_do=(idx == 4) if with_do is None else with_do)
    data["causal"] = c["causal"]
    return data


def make_decode_steps(B, H, d, steps, dtype, seed):
    """q,k,v ``[steps,B,H,d]`` for a run of single-token decode steps."""
    g = _gen(seed)
    return tuple(torch.randn((steps, B, H, d), generator=g, dtype=torch.float32).to(dtype)
                 for _ in range(3))


def make_onehot_case(B, H, N, d, dtype, seed, vmax=3):
    """Exactly representable inputs for bit-exact indexing tests: every Q and K row is a
    signed power of two on one axis (norm and reciprocal exact), V holds small integers on
    a sparse set of rows, so every partial sum is a small integer.  Use with s = 1."""
    g = _gen(seed)

    def onehot_rows():
        idx = torch.randint(0, d, (B, H, N), generator=g)
        sign = torch.randint(0, 2, (B, H, N), generator=g) * 2 - 1
        expo = torch.randint(-2, 3, (B, H, N), generator=g)
        x = torch.zeros((B, H, N, d), dtype=torch.float32)
        x.scatter_(3, idx.unsqueeze(-1), (sign * (2.0 ** expo)).unsqueeze(-1).float())
        return x

    q, k = onehot_rows(), onehot_rows()
    v = torch.randint(-vmax, vmax + 1, (B, H, N, d), generator=g).float()
    keep = torch.rand((B, H, N, 1), generator=g) < (8.0 / max(N, 8))  # ~8 live rows per head
    v = v * keep
    m = torch.randn((H,), generator=g, dtype=torch.float32)
    return {"q": q.to(dtype), "k": k.to(dtype), "v": v.to(dtype), "m": m}
