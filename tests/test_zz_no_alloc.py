"""The allocation-free entry point against the regular one, through the C ABI.

gka_fwd_chunked_noalloc is for callers that cannot allocate device memory around the call (code
inside stream-ordered regions where allocation is forbidden or synchronises, runtime plugins whose
memory is pre-planned, hosts without a tensor framework): it uses the scratch array built into the
library instead of a caller workspace.  It must give the same result as gka_fwd_chunked, also when
it is called twice in a row (the second call sees the first call's stale scratch contents).
This file sorts last so that a failure here cannot hide a failure elsewhere.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2511_21016_b200 import gka, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev(x, bf16=False):
    t = torch.from_numpy(np.ascontiguousarray(x)).to(DEV)
    return t.to(torch.bfloat16) if bf16 else t


def _rel(a, b):
    a = a.double().cpu().numpy()
    b = b.double().cpu().numpy()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


@pytest.mark.parametrize("name,cfg,tol", [
    # fp32 path, d = 64: several work items, sequences cut between items (scan scratch is used)
    ("f32_d64", synth.GkaConfig("na0", B=1, heads=3, T=64 * 50, d=64, chunk=64, n_iter=3,
                                io_dtype="f32", seed=11), 1e-4),
    # tensor-core path, d = 128, 20 tiles of 128 tokens: below the built-in scratch limit of 51 tiles
    ("bf16_d128", synth.GkaConfig("na1", B=1, heads=2, T=64 * 20, d=128, chunk=64, n_iter=4,
                                  io_dtype="bf16", seed=12), 2e-2),
])
def test_noalloc_matches_regular_entry_point_twice(name, cfg, tol):
    inp = synth.make_inputs(cfg)
    bf16 = cfg.io_dtype == "bf16"
    q, k, v = (_dev(inp[n], bf16) for n in ("q", "k", "v"))
    gate, lam = _dev(inp["gate"]), _dev(inp["lam"])
    ref_out, ref_state = gka.gka_fwd_chunked(q, k, v, gate, lam, cfg.n_iter, cfg.chunk)
    torch.cuda.synchronize()
    want = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], cfg.n_iter)     # and both against the oracle
    for call in range(2):
        out = torch.full_like(ref_out, float("nan"))
        state = torch.full_like(ref_state, float("nan"))
        gka.gka_fwd_chunked_noalloc(q, k, v, gate, lam, cfg.n_iter, cfg.chunk, out=out, state_out=state)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all() and torch.isfinite(state).all()
        assert _rel(out, ref_out) <= tol, f"{name}: call {call}: out differs"
        assert _rel(state, ref_state) <= tol, f"{name}: call {call}: state differs"
        e = float(np.linalg.norm(out.double().cpu().numpy() - want["out"]) / np.linalg.norm(want["out"]))
        assert e <= tol, f"{name}: call {call}: rel L2 {e:.3e} against the oracle"


def test_noalloc_rejects_problems_beyond_the_builtin_scratch():
    lib = gka.load_library()
    limit = int(lib.gka_noalloc_scratch_bytes())
    assert limit == 16 << 20
    B, T, heads, d = 1, 64 * 64, 2, 128          # 128 chunks of d = 128: needs far more than 16 MiB
    assert gka.gka_fwd_workspace_bytes(B, T, heads, d) > limit
    q = torch.zeros(B, T, heads, d, dtype=torch.bfloat16, device=DEV)
    g = torch.ones(B, T, heads, device=DEV)
    with pytest.raises(gka.GkaError) as ei:
        gka.gka_fwd_chunked_noalloc(q, q, q, g, g, 1)
    assert ei.value.status == 5                   # GKA_ERR_WORKSPACE, nothing was launched
    # argument errors are still named by their own status
    desc = gka.make_desc(1, 0, 1, 64, 64, gka.GKA_F32)       # no token: rejected before any pointer is used
    rc = lib.gka_fwd_chunked_noalloc(ctypes.byref(desc), 256, 256, 256, 256, 256, 1, 64, 256, None)
    assert rc == 2
