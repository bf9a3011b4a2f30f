"""The five benchmark configurations at full size, in the launch configuration bench.py times.

The oracle cannot recompute a whole full-size tensor in a test, so whole (batch, head) pairs are
sampled: every pair is an independent problem whose outputs the oracle computes one by one from the
same seeded inputs (per-(b,h) substreams make a pair's inputs identical whether drawn alone or with
the rest).  Tolerances: relative L2 of 1e-4 (fp32 I/O) and 2e-2 (bf16 I/O) over each compared pair, and the same
bound over every 128-token tile of a compared pair, so that one wrong tile cannot hide in a long sequence.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21016_b200 import gka, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def rel(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def dev(x, bf16=False):
    t = torch.from_numpy(np.ascontiguousarray(x)).to(DEV)
    return t.to(torch.bfloat16) if bf16 else t


def tile_max(out, ref, tile=128):
    """Largest relative L2 error over the 128-token tiles of a [T, d] sequence."""
    out = np.asarray(out, np.float64)
    ref = np.asarray(ref, np.float64)
    T = ref.shape[0] // tile * tile
    num = np.sqrt(((out[:T] - ref[:T]) ** 2).reshape(-1, tile * ref.shape[1]).sum(1))
    den = np.sqrt((ref[:T] ** 2).reshape(-1, tile * ref.shape[1]).sum(1))
    return float((num / np.maximum(den, 1e-300)).max())


def head_inputs(inp, pairs):
    """[1, T, len(pairs), d] slices of the sampled pairs, in oracle layout."""
    return {n: np.stack([a[b, :, h] for (b, h) in pairs], 1)[None] for n, a in inp.items()}


def run_full(cfg, inp, precision=gka.GKA_PREC_NATIVE, n_iter=None):
    bf16 = cfg.io_dtype == "bf16"
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out, st = gka.gka_fwd_chunked(dev(inp["q"], bf16), dev(inp["k"], bf16), dev(inp["v"], bf16),
                                  dev(inp["gate"]), dev(inp["lam"]),
                                  cfg.n_iter if n_iter is None else n_iter, cfg.chunk,
                                  precision=precision, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.float().cpu().numpy(), st.cpu().numpy()


def test_config1_full_size_sampled_pairs():
    """B=4, heads=16, T=4096, d=128, n_iter=10, bf16: the benchmark's launch; 4 sampled pairs."""
    cfg = synth.CONFIGS[1]
    inp = synth.make_inputs(cfg)
    out, st = run_full(cfg, inp)
    assert np.all(np.isfinite(out))
    pairs = [(0, 0), (1, 7), (2, 15), (3, 9)]
    hi = head_inputs(inp, pairs)
    ref = oracle.fwd(hi["q"], hi["k"], hi["v"], hi["gate"], hi["lam"], cfg.n_iter)
    got = np.stack([out[b, :, h] for (b, h) in pairs], 1)[None]
    got_st = np.stack([st[b, h] for (b, h) in pairs], 0)[None]
    e, es = rel(got, ref["out"]), rel(got_st, ref["state"])
    print("config1 sampled rel L2 out %.3e state %.3e" % (e, es))
    assert e <= 2e-2 and es <= 5e-3
    # per-pair too: no pair hides behind the others
    for i in range(len(pairs)):
        assert rel(got[0, :, i], ref["out"][0, :, i]) <= 2e-2
        et = tile_max(got[0, :, i], ref["out"][0, :, i])
        assert et <= 2e-2, f"pair {pairs[i]}: worst 128-token tile rel L2 {et:.3e}"


def test_config3_long_context_three_heads_of_32():
    """T=131072, d=128, bf16, slow-fading gates, B=1, heads=32: the benchmark's launch with real inputs for every
    head (drawn on the device with the configuration's distributions; the host recipe would take minutes).  Every
    head is spread over several work items; the oracle recomputes three whole heads (first, middle, last) from the
    same inputs, and every 128-token tile of each is bounded."""
    cfg = synth.CONFIGS[3]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(cfg.seed)
    B, T, Hh, d = cfg.B, cfg.T, cfg.heads, cfg.d

    def unit(shape):
        x = torch.randn(shape, generator=gen, device=DEV)
        return (x / x.norm(dim=-1, keepdim=True)).to(torch.bfloat16)

    q, k = unit((B, T, Hh, d)), unit((B, T, Hh, d))
    v = torch.randn((B, T, Hh, d), generator=gen, device=DEV).to(torch.bfloat16)
    gate = torch.sigmoid(torch.randn((B, T, Hh), generator=gen, device=DEV) + 4.0)
    lam = torch.nn.functional.softplus(torch.randn((B, T, Hh), generator=gen, device=DEV) - 1.0) + 1e-3
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out, st = gka.gka_fwd_chunked(q, k, v, gate, lam, cfg.n_iter, cfg.chunk, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert bool(torch.isfinite(out.float()).all())
    heads = [0, 13, 31]
    f64 = lambda t: np.ascontiguousarray(t.float().cpu().numpy().astype(np.float64))
    ref = oracle.fwd(f64(q[:, :, heads]), f64(k[:, :, heads]), f64(v[:, :, heads]), f64(gate[:, :, heads]),
                     f64(lam[:, :, heads]), cfg.n_iter)
    for i, h in enumerate(heads):
        got = out[0, :, h].float().cpu().numpy()
        e = rel(got, ref["out"][0, :, i])
        et = tile_max(got, ref["out"][0, :, i])
        es = rel(st[0, h].cpu().numpy(), ref["state"][0, i])
        print("config3 head %d rel L2 out %.3e (worst tile %.3e) state %.3e" % (h, e, et, es))
        assert e <= 2e-2 and es <= 5e-3
        assert et <= 2e-2


def test_config2_decode_full_size_sampled_heads():
    """256 sequences x 32 heads, d=128, fp32 state from a 2048-token prefix, n_iter=10.  The prefix runs
    through gka_fwd_chunked (state_out) for all 8192 heads; for sampled heads the oracle recomputes the
    prefix state and the step from the same inputs."""
    cfg = synth.CONFIGS[2]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(cfg.seed)
    N, Hh, d, Tp = cfg.B, cfg.heads, cfg.d, cfg.prefix_T

    def unit(shape):
        x = torch.randn(shape, generator=gen, device=DEV)
        return (x / x.norm(dim=-1, keepdim=True)).to(torch.bfloat16)

    pq, pk = unit((N, Tp, Hh, d)), unit((N, Tp, Hh, d))
    pv = torch.randn((N, Tp, Hh, d), generator=gen, device=DEV).to(torch.bfloat16)
    pg = torch.sigmoid(torch.randn((N, Tp, Hh), generator=gen, device=DEV) + 2.0)
    pl = torch.nn.functional.softplus(torch.randn((N, Tp, Hh), generator=gen, device=DEV)) + 1e-2
    sq, sk = unit((N, Hh, d)), unit((N, Hh, d))
    sv = torch.randn((N, Hh, d), generator=gen, device=DEV).to(torch.bfloat16)
    sg = torch.sigmoid(torch.randn((N, Hh), generator=gen, device=DEV) + 2.0)
    sl = torch.nn.functional.softplus(torch.randn((N, Hh), generator=gen, device=DEV)) + 1e-2
    _, state = gka.gka_fwd_chunked(pq, pk, pv, pg, pl, 0, cfg.chunk)
    out = gka.gka_decode_step(state, sq, sk, sv, sg, sl, cfg.n_iter)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    pairs = [(0, 0), (17, 3), (128, 31), (255, 16)]
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    for (b, h) in pairs:
        ref_pre = oracle.fwd(f64(pq[b:b + 1, :, h:h + 1]), f64(pk[b:b + 1, :, h:h + 1]), f64(pv[b:b + 1, :, h:h + 1]),
                             f64(pg[b:b + 1, :, h:h + 1]), f64(pl[b:b + 1, :, h:h + 1]), 0)
        ref = oracle.decode(ref_pre["state"], f64(sq[b:b + 1, h:h + 1]), f64(sk[b:b + 1, h:h + 1]),
                            f64(sv[b:b + 1, h:h + 1]), f64(sg[b:b + 1, h:h + 1]), f64(sl[b:b + 1, h:h + 1]),
                            cfg.n_iter)
        e = rel(out[b, h].float().cpu().numpy(), ref["out"][0, 0])
        es = rel(state[b, h].cpu().numpy(), ref["state"][0, 0])
        assert e <= 2e-2, f"decode out ({b},{h}) rel L2 {e:.3e}"
        assert es <= 5e-3, f"decode state ({b},{h}) rel L2 {es:.3e}"


def test_config4_conditioning_stress_table():
    """Keys close to a rank-8 subspace, lambda ~ 1e-4, gates near 1: kappa ~ 1e6.  Sweep n_iter; the fp32
    arithmetic mode must track the fp64 Chebyshev oracle (1e-4 for fp32 I/O, 2e-2 for bf16 I/O); bf16
    operands are reported, must stay finite, and are not expected to meet 2e-2 (epsilon * kappa).
    Errors against the exact Cholesky solve are reported: at this kappa Chebyshev has not converged
    after 32 steps, whatever the precision."""
    cfg = synth.CONFIGS[4]
    inp = synth.make_inputs(cfg)
    pairs = [(0, 0), (1, 5)]
    hi = head_inputs(inp, pairs)
    inp32 = dict(inp)
    cfg32 = synth.shrink(cfg, io_dtype="f32")
    rows = []
    exact = None
    for r in (4, 8, 16, 32):
        ref = oracle.fwd(hi["q"], hi["k"], hi["v"], hi["gate"], hi["lam"], r, exact=exact is None)
        if exact is None:
            exact = ref["out_exact"]          # the exact solve does not depend on n_iter
        pick = lambda o: np.stack([o[b, :, h] for (b, h) in pairs], 1)[None]
        o_f32, _ = run_full(cfg32, inp32, n_iter=r)                                   # fp32 I/O, fp32 math
        o_hi, _ = run_full(cfg, inp, precision=gka.GKA_PREC_HIGH, n_iter=r)           # bf16 I/O, fp32 math
        o_nat, _ = run_full(cfg, inp, n_iter=r)                                       # bf16 operands
        e_f32, e_hi, e_nat = (rel(pick(o), ref["out"]) for o in (o_f32, o_hi, o_nat))
        x_ch = rel(ref["out"], exact)
        x_f32 = rel(pick(o_f32), exact)
        rows.append((r, e_f32, e_hi, e_nat, x_ch, x_f32))
        assert np.all(np.isfinite(o_nat))
        assert e_f32 <= 1e-4, f"fp32 I/O n_iter={r}: {e_f32:.3e}"
        assert e_hi <= 2e-2, f"bf16 I/O fp32 math n_iter={r}: {e_hi:.3e}"
    print("\nconfig4: n_iter | vs CH oracle: f32 io, bf16 io (fp32 math), bf16 operands | vs Cholesky: oracle CH, f32 kernel")
    for row in rows:
        print("  %2d | %.2e %.2e %.2e | %.4f %.4f" % row)
