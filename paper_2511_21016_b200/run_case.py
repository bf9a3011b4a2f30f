"""Run one small case of the hot path a few times (seeded, device-generated inputs).

    python -m paper_2511_21016_b200.run_case fwd    B heads T n_iter reps
    python -m paper_2511_21016_b200.run_case decode N heads reps
    python -m paper_2511_21016_b200.run_case tokens N heads T reps

Used for profiling captures (a case of a few hundred MB that ends by itself) and as a usage example
of the binding: inputs with the benchmark's distributions, one workspace allocation, repeated calls.
"""
from __future__ import annotations

import sys

import torch

from . import gka


def _unit(shape, gen, dev):
    x = torch.randn(shape, device=dev, generator=gen)
    return (x / x.norm(dim=-1, keepdim=True)).bfloat16()


def run_fwd(B: int, heads: int, T: int, n_iter: int, reps: int, d: int = 128, dev: str = "cuda:0") -> float:
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    q, k = _unit((B, T, heads, d), gen, dev), _unit((B, T, heads, d), gen, dev)
    v = torch.randn(B, T, heads, d, device=dev, generator=gen).bfloat16()
    gate = torch.sigmoid(torch.randn(B, T, heads, device=dev, generator=gen) + 2)
    lam = torch.nn.functional.softplus(torch.randn(B, T, heads, device=dev, generator=gen)) + 1e-2
    ws = gka.alloc_workspace(B, T, heads, d, dev)
    out = torch.empty_like(v)
    state = torch.empty(B, heads, 2 * d * d, device=dev)
    for _ in range(reps):
        gka.gka_fwd_chunked(q, k, v, gate, lam, n_iter, 64, out=out, state_out=state, workspace=ws)
    torch.cuda.synchronize()
    return float(out.float().abs().mean())


def run_decode(N: int, heads: int, reps: int, d: int = 128, dev: str = "cuda:0") -> float:
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    state = torch.randn(N, heads, 2 * d * d, device=dev, generator=gen) * 0.05
    q, k = _unit((N, heads, d), gen, dev), _unit((N, heads, d), gen, dev)
    v = torch.randn(N, heads, d, device=dev, generator=gen).bfloat16()
    gate = torch.sigmoid(torch.randn(N, heads, device=dev, generator=gen) + 2)
    lam = torch.nn.functional.softplus(torch.randn(N, heads, device=dev, generator=gen)) + 1e-2
    out = torch.empty_like(v)
    for _ in range(reps):
        gka.gka_decode_step(state, q, k, v, gate, lam, 10, out=out)
    torch.cuda.synchronize()
    return float(out.float().abs().mean())


def run_tokens(N: int, heads: int, T: int, reps: int, d: int = 128, dev: str = "cuda:0") -> float:
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    state = torch.randn(N, heads, 2 * d * d, device=dev, generator=gen) * 0.05
    q, k = _unit((N, T, heads, d), gen, dev), _unit((N, T, heads, d), gen, dev)
    v = torch.randn(N, T, heads, d, device=dev, generator=gen).bfloat16()
    gate = torch.sigmoid(torch.randn(N, T, heads, device=dev, generator=gen) + 2)
    lam = torch.nn.functional.softplus(torch.randn(N, T, heads, device=dev, generator=gen)) + 1e-2
    out = torch.empty_like(v)
    for _ in range(reps):
        gka.gka_decode_tokens(state, q, k, v, gate, lam, 10, out=out)
    torch.cuda.synchronize()
    return float(out.float().abs().mean())


def main(argv) -> int:
    if len(argv) >= 6 and argv[0] == "fwd":
        print("ok", run_fwd(*(int(x) for x in argv[1:6])))
    elif len(argv) >= 4 and argv[0] == "decode":
        print("ok", run_decode(*(int(x) for x in argv[1:4])))
    elif len(argv) >= 5 and argv[0] == "tokens":
        print("ok", run_tokens(*(int(x) for x in argv[1:5])))
    else:
        print(__doc__)
        return 2
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv[1:]))
