"""A seeded sweep of shapes and options through the tensor-core path of the chunked forward against the fp64 oracle:
head dimension, batch, heads, sequence lengths around the tile and work-item boundaries, iteration counts, the adaptive
rule, write strengths, the alpha-connection, the solve alone, and initial states taken from a prefix of the recurrence
(the state a caller would pass on)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21016_b200 import gka, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def rel(a, b):
    return float(np.linalg.norm(np.asarray(a, np.float64) - b) / max(np.linalg.norm(b), 1e-300))


def dev(x, bf16=False):
    t = torch.from_numpy(np.ascontiguousarray(x)).to(DEV)
    return t.to(torch.bfloat16) if bf16 else t


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_seeded_sweep_of_shapes_and_options(seed):
    rng = np.random.default_rng(1000 + seed)
    for case in range(25):
        d = int(rng.choice([64, 128]))
        B, H = int(rng.integers(1, 4)), int(rng.integers(1, 6))
        T = int(rng.choice([16, 17, 64, 100, 128, 129, 300, 1000, 2500, 128 * int(rng.integers(1, 40)) + int(rng.integers(0, 128))]))
        r = int(rng.choice([0, 1, 2, 5, 10, 30]))
        adaptive, use_b, use_a = (bool(rng.integers(0, 2)) for _ in range(3))
        solve, use_state = bool(rng.integers(0, 4) == 0), bool(rng.integers(0, 2))
        cfg = synth.shrink(synth.CONFIGS[1], B=B, heads=H, T=T, d=d, n_iter=r, seed=int(rng.integers(0, 10 ** 6)))
        inp = synth.make_inputs(cfg)
        lam = np.full_like(inp["lam"], 0.02) if adaptive else inp["lam"]
        beta = rng.uniform(0.2, 1.0, lam.shape).astype(np.float32) if use_b else None
        alpha = rng.uniform(0.0, 1.0, lam.shape).astype(np.float32) if (use_a and not solve) else None
        s_in = None
        if use_state:
            pin = synth.make_inputs(synth.shrink(cfg, T=int(rng.integers(1, 200)), seed=cfg.seed + 7))
            s_in = oracle.fwd(pin["q"], pin["k"], pin["v"], pin["gate"], pin["lam"], 0)["state"].astype(np.float32)
        ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], lam, r, state_in=s_in, lam_mode=1 if adaptive else 0,
                         beta=beta, alpha=alpha, want_x=True)
        q, k, v = (dev(inp[m], True) for m in ("q", "k", "v"))
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        kw = dict(flags=gka.GKA_FLAG_ADAPTIVE_LAMBDA if adaptive else 0, device_status=status,
                  state_in=None if s_in is None else dev(s_in), beta=None if beta is None else dev(beta))
        what = dict(d=d, B=B, H=H, T=T, r=r, adaptive=adaptive, beta=use_b, alpha=use_a, solve=solve, state=use_state)
        if solve:
            x = gka.gka_solve_chunked(q, k, dev(inp["gate"]), dev(lam), r, 64, **kw)
            torch.cuda.synchronize()
            assert int(status.item()) == 0, what
            assert rel(x.float().cpu().numpy(), ref["x"]) <= 2e-2, what
        else:
            out, st = gka.gka_fwd_chunked(q, k, v, dev(inp["gate"]), dev(lam), r, 64,
                                          alpha=None if alpha is None else dev(alpha), **kw)
            torch.cuda.synchronize()
            assert int(status.item()) == 0, what
            assert rel(out.float().cpu().numpy(), ref["out"]) <= 2e-2, what
            assert rel(st.cpu().numpy(), ref["state"]) <= 5e-3, what
