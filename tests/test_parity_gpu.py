"""Parity of the CUDA path (through the C ABI) against the fp64 CPU oracle, element by element
on the same seeded inputs.  Tolerances: relative L2 over the whole tensor of 1e-4 for fp32 I/O
and 2e-2 for bf16 I/O, and, so that no single stretch of tokens hides behind the rest, a bound on the
relative L2 of every 128-token tile of every (batch, head) pair: the same two figures (measured: the
worst tile sits within a factor of two of the whole-tensor error)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21016_b200 import gka, synth

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 2e-2
TILE_TOL_F32 = 1e-4
TILE_TOL_BF16 = 2e-2
DEV = "cuda:0"


def tile_max(out, ref, tile=128):
    """Largest relative L2 error over the 128-token tiles of every (batch, head) pair; [B, T, heads, d] arrays."""
    out = np.asarray(out, np.float64)
    ref = np.asarray(ref, np.float64)
    worst = 0.0
    for t0 in range(0, ref.shape[1], tile):
        num = np.sqrt(((out[:, t0:t0 + tile] - ref[:, t0:t0 + tile]) ** 2).sum(axis=(1, 3)))
        den = np.sqrt((ref[:, t0:t0 + tile] ** 2).sum(axis=(1, 3)))
        worst = max(worst, float((num / np.maximum(den, 1e-300)).max()))
    return worst


def rel(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def to_dev(x, bf16=False):
    t = torch.from_numpy(np.ascontiguousarray(x)).to(DEV)
    return t.to(torch.bfloat16) if bf16 else t


def run_fwd(inp, n_iter, bf16, precision=gka.GKA_PREC_NATIVE, state_in=None, flags=0, want_fro=True):
    q, k, v = (to_dev(inp[n], bf16) for n in ("q", "k", "v"))
    gate, lam = to_dev(inp["gate"]), to_dev(inp["lam"])
    B, T, Hh, d = q.shape
    fro = torch.zeros(B, T, Hh, dtype=torch.float32, device=DEV) if want_fro else None
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    s_in = None if state_in is None else to_dev(np.asarray(state_in, np.float32))
    out, st = gka.gka_fwd_chunked(q, k, v, gate, lam, n_iter, 64, state_in=s_in, precision=precision,
                                  flags=flags, fro_out=fro, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return (out.float().cpu().numpy(), st.cpu().numpy(),
            None if fro is None else fro.cpu().numpy())


def check_fwd(cfg, n_iter=None, precision=gka.GKA_PREC_NATIVE, flags=0, tol=None, state_tol=None,
              T=None):
    n_iter = cfg.n_iter if n_iter is None else n_iter
    bf16 = cfg.io_dtype == "bf16"
    inp = synth.make_inputs(cfg, T=T)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], n_iter,
                     lam_mode=1 if flags & gka.GKA_FLAG_ADAPTIVE_LAMBDA else 0)
    out, st, fro = run_fwd(inp, n_iter, bf16, precision, flags=flags)
    tol = tol if tol is not None else (TOL_BF16 if bf16 else TOL_F32)
    fp32_math = (not bf16) or precision == gka.GKA_PREC_HIGH     # bf16 I/O in native precision: tensor cores, d = 64 or 128
    state_tol = state_tol if state_tol is not None else (1e-5 if fp32_math else 5e-3)
    assert np.all(np.isfinite(out))
    e_out, e_st, e_fro = rel(out, ref["out"]), rel(st, ref["state"]), rel(fro, ref["fro"])
    assert e_out <= tol, f"out rel L2 {e_out:.3e} > {tol}"
    e_tile = tile_max(out, ref["out"])
    assert e_tile <= (TILE_TOL_BF16 if bf16 else TILE_TOL_F32), f"worst 128-token tile rel L2 {e_tile:.3e}"
    assert e_st <= state_tol, f"state rel L2 {e_st:.3e} > {state_tol}"
    assert e_fro <= (1e-5 if fp32_math else 5e-3), f"fro rel L2 {e_fro:.3e}"
    return e_out, e_st, e_fro, e_tile


SMALL = synth.GkaConfig("small", B=2, heads=3, T=128, d=64, chunk=64, n_iter=4, io_dtype="f32", seed=7)


@pytest.mark.parametrize("n_iter", [0, 1, 2, 8])
@pytest.mark.parametrize("T", [64, 128, 320])
def test_fwd_f32_small(T, n_iter):
    check_fwd(synth.shrink(SMALL, T=T), n_iter=n_iter)


def test_fwd_config0():
    """Config 0 exactly: fp32 I/O, B=1, heads=2, T=256, d=64, chunk=64, n_iter=8, seed 0."""
    e = check_fwd(synth.CONFIGS[0])
    print("config0 rel L2 (out, state, fro):", e)


def test_fwd_f32_d128():
    check_fwd(synth.shrink(SMALL, d=128, T=256, heads=2, n_iter=6))


def test_fwd_f32_items_cut_sequences():
    """More chunks than SMs, chunk count not a multiple of the item count: every work item starts
    or ends inside a sequence, so the summary kernel and the cross-item scan carry the state."""
    cfg = synth.shrink(SMALL, B=1, heads=3, T=64 * 101, n_iter=2)
    check_fwd(cfg)


@pytest.mark.parametrize("io,d", [("f32", 64), ("f32", 128), ("bf16", 128)])
def test_fwd_slow_fading_state_crosses_many_items(io, d):
    """Gates close to 1 (sigmoid(N(6,1))): the state of a sequence start is still alive many work items
    later, so a wrong start state of any item shows (fast-fading gates would hide it).  Several sequences
    whose boundaries fall inside items."""
    cfg = synth.GkaConfig("slow", B=2, heads=3, T=64 * 70, d=d, chunk=64, n_iter=2, io_dtype=io, seed=21,
                          gate_mean=6.0)
    check_fwd(cfg)


def test_fwd_f32_long_runs_d128():
    cfg = synth.shrink(SMALL, B=1, heads=2, d=128, T=64 * 160, n_iter=3)
    check_fwd(cfg)


def test_fwd_bf16_io_high_precision():
    """bf16 I/O with fp32 arithmetic: the error is the final rounding of the output to bf16."""
    cfg = synth.shrink(synth.CONFIGS[1], B=1, heads=2, T=512)
    e = check_fwd(cfg, precision=gka.GKA_PREC_HIGH)
    assert e[0] < 5e-3


def test_fwd_bf16_native_small():
    """bf16 I/O, native precision (tensor-core operands in bf16), several chunks and heads."""
    cfg = synth.shrink(synth.CONFIGS[1], B=2, heads=3, T=640)
    e = check_fwd(cfg)
    print("bf16 native rel L2 (out, state, fro):", e)


@pytest.mark.parametrize("n_iter", [0, 1, 3])
def test_fwd_bf16_native_iteration_counts(n_iter):
    cfg = synth.shrink(synth.CONFIGS[1], B=1, heads=2, T=192)
    check_fwd(cfg, n_iter=n_iter)


@pytest.mark.parametrize("d", [128, 64])
def test_fwd_bf16_native_items_cut_sequences(d):
    cfg = synth.shrink(synth.CONFIGS[1], B=1, heads=3, T=64 * 101, n_iter=4, d=d)
    check_fwd(cfg)


def test_fwd_bf16_native_head_dimension_64_every_option():
    """Head dimension 64 on the tensor-core path (bf16 I/O, native precision): several heads side by side (a head's
    upper half on chip must read as zeros, not as the next head's channels), write strengths, alpha-connection,
    adaptive lambda at the paper's iteration count, the solve alone, and a 1e-4 comparison of the final state's
    layout against the fp32 path."""
    cfg = synth.shrink(synth.CONFIGS[1], B=2, heads=5, T=64 * 9 + 30, n_iter=10, d=64)
    inp = synth.make_inputs(cfg)
    rng = np.random.default_rng(5)
    beta = rng.uniform(0.2, 1.0, inp["gate"].shape).astype(np.float32)
    alpha = rng.uniform(0.0, 1.0, inp["gate"].shape).astype(np.float32)
    q, k, v = (to_dev(inp[n], True) for n in ("q", "k", "v"))
    gate, lam = to_dev(inp["gate"]), to_dev(inp["lam"])
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 10, beta=beta, alpha=alpha, want_x=True)
    out, st = gka.gka_fwd_chunked(q, k, v, gate, lam, 10, 64, beta=to_dev(beta), alpha=to_dev(alpha), device_status=status)
    x = gka.gka_solve_chunked(q, k, gate, lam, 10, 64, beta=to_dev(beta), device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert rel(out.float().cpu().numpy(), ref["out"]) <= TOL_BF16
    assert tile_max(out.float().cpu().numpy(), ref["out"]) <= TILE_TOL_BF16
    assert rel(st.cpu().numpy(), ref["state"]) <= 5e-3
    assert rel(x.float().cpu().numpy(), ref["x"]) <= TOL_BF16
    lam_a = np.full_like(inp["lam"], 0.02)
    ref_a = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], lam_a, 30, lam_mode=1)
    out_a, _ = gka.gka_fwd_chunked(q, k, v, gate, to_dev(lam_a), 30, 64, flags=gka.GKA_FLAG_ADAPTIVE_LAMBDA, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert rel(out_a.float().cpu().numpy(), ref_a["out"]) <= TOL_BF16


def test_fwd_state_in_split_prefill_equals_whole():
    cfg = synth.shrink(SMALL, B=1, heads=2, T=384, n_iter=5)
    inp = synth.make_inputs(cfg)
    whole, st_whole, _ = run_fwd(inp, 5, False)
    first = {n: a[:, :128] for n, a in inp.items()}
    second = {n: a[:, 128:] for n, a in inp.items()}
    o1, st1, _ = run_fwd(first, 5, False)
    o2, st2, _ = run_fwd(second, 5, False, state_in=st1)
    assert rel(np.concatenate([o1, o2], axis=1), whole) < 1e-5
    assert rel(st2, st_whole) < 1e-5
    ref = oracle.fwd(second["q"], second["k"], second["v"], second["gate"], second["lam"], 5,
                     state_in=st1)
    assert rel(o2, ref["out"]) < TOL_F32


def test_fwd_adaptive_lambda_mode():
    """lambda_t = a ||H_t||_F (Section 4.1): kappa bound (a+1)/a = 51 for a = 0.02."""
    cfg = synth.shrink(SMALL, T=192, n_iter=10)
    inp = synth.make_inputs(cfg)
    inp["lam"] = np.full_like(inp["lam"], 0.02)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 10, lam_mode=1)
    out, st, fro = run_fwd(inp, 10, False, flags=gka.GKA_FLAG_ADAPTIVE_LAMBDA)
    assert rel(out, ref["out"]) < TOL_F32


@pytest.mark.parametrize("T,n_iter", [(256, 8), (457, 8), (64 * 30, 30)])
def test_fwd_adaptive_lambda_mode_bf16(T, n_iter):
    """The adaptive rule with the paper's a = 0.02 makes every solve as ill-conditioned as the rule allows
    (kappa = 51), and the paper runs 30 iterations: the tensor-core path (bf16 operands on the increments,
    fp32 iterate, two-term read) meets the bf16 bar there, and so does the fp32-arithmetic mode of the same call."""
    cfg = synth.shrink(synth.CONFIGS[1], B=3, heads=5, T=T, n_iter=n_iter, seed=49)
    inp = synth.make_inputs(cfg)
    inp["lam"] = np.full_like(inp["lam"], 0.02)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], n_iter, lam_mode=1)
    out, _, _ = run_fwd(inp, n_iter, True, flags=gka.GKA_FLAG_ADAPTIVE_LAMBDA)
    e, et = rel(out, ref["out"]), tile_max(out, ref["out"])
    print("adaptive a=0.02 T=%d r=%d tensor path: rel L2 %.3e, worst tile %.3e" % (T, n_iter, e, et))
    assert e <= TOL_BF16 and et <= TILE_TOL_BF16
    out, _, _ = run_fwd(inp, n_iter, True, precision=gka.GKA_PREC_HIGH, flags=gka.GKA_FLAG_ADAPTIVE_LAMBDA)
    assert rel(out, ref["out"]) <= 5e-3


def test_fwd_bf16_native_paper_iteration_count():
    """30 iterations (the paper's setting in every experiment) on configuration-1-like inputs, sequences cut by
    work items: tensor-core path against the oracle."""
    cfg = synth.shrink(synth.CONFIGS[1], B=2, heads=3, T=64 * 70, n_iter=30)
    e = check_fwd(cfg)
    print("bf16 native r=30 rel L2 (out, state, fro, worst tile):", e)


def test_fwd_degenerate_inputs():
    """Unit gates, a hard reset gate, zero keys (H = 0, so L = mu) and a zero gate."""
    cfg = synth.shrink(SMALL, B=1, heads=2, T=128, n_iter=4)
    inp = synth.make_inputs(cfg)
    inp["gate"][:, :, 0] = 1.0                       # head 0: no forgetting
    inp["gate"][:, 70, 1] = 1e-30                    # head 1: reset in the middle of chunk 2
    inp["k"][:, :5, 1] = 0.0                         # head 1: H stays zero for five tokens
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 4)
    out, st, fro = run_fwd(inp, 4, False)
    assert np.all(np.isfinite(out))
    assert rel(out, ref["out"]) < TOL_F32
    assert rel(st, ref["state"]) < 1e-5
    inp["gate"][:, 40, 1] = 0.0                      # exact zero gate: clamped at exp(-80) on device
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 4)
    out, st, fro = run_fwd(inp, 4, False)
    assert np.all(np.isfinite(out)) and rel(out, ref["out"]) < TOL_F32


def test_fwd_is_deterministic():
    cfg = synth.shrink(synth.CONFIGS[1], B=1, heads=3, T=64 * 60, n_iter=3)
    inp = synth.make_inputs(cfg)
    a = run_fwd(inp, 3, True)
    b = run_fwd(inp, 3, True)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_fwd_back_to_back_calls_share_a_workspace():
    """Two different problems enqueued back to back on one stream with the same workspace: the second result must not
    see the first call's segment summaries (the main kernel starts under the summary kernel's tail and waits for the
    summaries only where it reads them)."""
    cfg = synth.shrink(synth.CONFIGS[1], B=2, heads=5, T=64 * 60, n_iter=3)
    a = synth.make_inputs(cfg)
    b = synth.make_inputs(synth.shrink(cfg, seed=77))
    ws = gka.alloc_workspace(cfg.B, cfg.T, cfg.heads, cfg.d, DEV)
    dev_a = [to_dev(a[n], n in ("q", "k", "v")) for n in ("q", "k", "v", "gate", "lam")]
    dev_b = [to_dev(b[n], n in ("q", "k", "v")) for n in ("q", "k", "v", "gate", "lam")]
    alone, st_alone = gka.gka_fwd_chunked(*dev_b, 3, 64, workspace=ws)
    torch.cuda.synchronize()
    for _ in range(5):
        gka.gka_fwd_chunked(*dev_a, 3, 64, workspace=ws)
        after, st_after = gka.gka_fwd_chunked(*dev_b, 3, 64, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(alone, after) and torch.equal(st_alone, st_after)


@pytest.mark.parametrize("B,heads,T,d", [(2, 5, 640, 128), (2, 5, 640, 64), (1, 40, 2000, 128), (8, 16, 1000, 128),
                                         (2, 5, 3840, 128), (4, 40, 200, 128)])
def test_fwd_bf16_native_repeated_calls_are_bit_identical(B, heads, T, d):
    """The same problem several times over, one workspace: outputs and final states must agree bit for bit in every
    decomposition of the state pass (whole sequences with one block per master, whole sequences with one block each,
    ranges that cut sequences, more pairs than SMs with two whole sequences per work item), and the first call must
    agree with the oracle."""
    cfg = synth.shrink(synth.CONFIGS[1], B=B, heads=heads, T=T, d=d, n_iter=3, seed=31)
    inp = synth.make_inputs(cfg)
    dev = [to_dev(inp[n], n in ("q", "k", "v")) for n in ("q", "k", "v", "gate", "lam")]
    ws = gka.alloc_workspace(B, T, heads, d, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    first, st_first = gka.gka_fwd_chunked(*dev, 3, 64, workspace=ws, device_status=status)
    torch.cuda.synchronize()
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 3)
    assert rel(first.float().cpu().numpy(), ref["out"]) <= TOL_BF16
    for _ in range(6):
        again, st_again = gka.gka_fwd_chunked(*dev, 3, 64, workspace=ws, device_status=status)
        torch.cuda.synchronize()
        assert torch.equal(first, again) and torch.equal(st_first, st_again)
    assert int(status.item()) == 0


def test_work_items_follow_the_decomposition_rule():
    """Number of work items of the state pass on this device: whole sequences where that is cheaper than cutting them
    (fewer pairs than SMs and short enough sequences; more pairs than SMs with a small divisor), one range per SM
    otherwise; the fp32 path always takes one range per SM (or one per chunk for small problems)."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n = gka.gka_fwd_num_work_items
    assert n(4, 4096, 16, 128) == 64                       # configuration 1: the 64 pairs
    assert n(1, 131072, 32, 128) == min(sms, 32 * 1024)    # configuration 3: long sequences are cut
    if sms == 148:
        assert n(16, 2048, 16, 128) == 128                 # 256 pairs: 128 items of two sequences
        assert n(2, 3840, 5, 128) == 148                   # 10 pairs of 30 tiles: cut
    assert n(4, 4096, 16, 128, io_dtype=gka.GKA_F32) == min(sms, 4 * 16 * 64)
    for B, T, heads in ((4, 4096, 16), (16, 2048, 16), (2, 640, 5)):
        G = n(B, T, heads, 128)
        if G < sms and (B * heads) % G == 0:               # whole sequences: nothing is cut
            for i in range(G):
                assert gka.gka_fwd_work_range(B, T, heads, 128, G, i)[2:] == (0, 0)


def test_fwd_gpu_argument_errors():
    q = torch.zeros(1, 100, 1, 64, device=DEV)
    v = torch.zeros(1, 100, 1, 128, device=DEV)
    g = torch.ones(1, 100, 1, device=DEV)
    with pytest.raises(ValueError, match="shape"):
        gka.gka_fwd_chunked(q, q, v, g, g, 1)          # d_k != d_v: stopped by the binding (the library answers status 2)
    q = torch.zeros(1, 128, 1, 64, device=DEV)
    g = torch.ones(1, 128, 1, device=DEV)
    ws = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(gka.GkaError) as ei:
        gka.gka_fwd_chunked(q, q, q, g, g, 1, workspace=ws)
    assert ei.value.status == 5


# ------------------------------------------------------------------------------------------ decode
def decode_case(N, heads, d, n_iter, bf16, seed, prefix_T=96):
    cfg = synth.GkaConfig("dec", B=N, heads=heads, T=prefix_T, d=d, chunk=64, n_iter=n_iter,
                          io_dtype="bf16" if bf16 else "f32", seed=seed)
    pre = synth.make_inputs(cfg)
    state = oracle.fwd(pre["q"], pre["k"], pre["v"], pre["gate"], pre["lam"], 0)["state"]
    state32 = state.astype(np.float32)
    step = synth.make_inputs(cfg, T=1, stream=1)
    sq, sk, sv = (step[n][:, 0] for n in ("q", "k", "v"))
    sg, sl = step["gate"][:, 0], step["lam"][:, 0]
    ref = oracle.decode(state32, sq, sk, sv, sg, sl, n_iter)
    st_dev = to_dev(state32)
    out = gka.gka_decode_step(st_dev, to_dev(sq, bf16), to_dev(sk, bf16), to_dev(sv, bf16),
                              to_dev(sg), to_dev(sl), n_iter)
    torch.cuda.synchronize()
    return out.float().cpu().numpy(), st_dev.cpu().numpy(), ref


@pytest.mark.parametrize("d,bf16", [(128, True), (128, False), (64, False), (64, True), (32, False), (32, True), (16, False), (16, True)])
@pytest.mark.parametrize("n_iter", [0, 1, 10])
def test_decode_step(d, bf16, n_iter):
    out, st, ref = decode_case(5, 3, d, n_iter, bf16, seed=31)
    assert rel(st, ref["state"]) < 1e-6
    assert rel(out, ref["out"]) < (5e-3 if bf16 else TOL_F32)


def test_decode_continues_chunked_forward():
    """T tokens through gka_fwd_chunked, then 64 decode steps on its state_out, equals T + 64
    tokens through gka_fwd_chunked (one recurrence, eq. (CH)); both match the oracle."""
    cfg = synth.shrink(SMALL, B=2, heads=2, T=192, n_iter=6)
    inp = synth.make_inputs(cfg)
    whole, st_whole, _ = run_fwd(inp, 6, False)
    head = {n: a[:, :128] for n, a in inp.items()}
    _, st, _ = run_fwd(head, 6, False)
    st_dev = to_dev(st)
    outs = []
    for t in range(128, 192):
        o = gka.gka_decode_step(st_dev, to_dev(inp["q"][:, t]), to_dev(inp["k"][:, t]),
                                to_dev(inp["v"][:, t]), to_dev(inp["gate"][:, t]),
                                to_dev(inp["lam"][:, t]), 6)
        outs.append(o.cpu().numpy())
    torch.cuda.synchronize()
    dec = np.stack(outs, axis=1)
    assert rel(dec, whole[:, 128:]) < 1e-5
    assert rel(st_dev.cpu().numpy(), st_whole) < 1e-5
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 6)
    assert rel(dec, ref["out"][:, 128:]) < TOL_F32


def test_decode_adaptive_lambda():
    cfg = synth.GkaConfig("dec", B=3, heads=2, T=64, d=128, chunk=64, n_iter=8, io_dtype="f32", seed=5)
    pre = synth.make_inputs(cfg)
    state32 = oracle.fwd(pre["q"], pre["k"], pre["v"], pre["gate"], pre["lam"], 0)["state"].astype(np.float32)
    step = synth.make_inputs(cfg, T=1, stream=1)
    a = np.full_like(step["lam"][:, 0], 0.02)
    ref = oracle.decode(state32, step["q"][:, 0], step["k"][:, 0], step["v"][:, 0], step["gate"][:, 0],
                        a, 8, lam_mode=1)
    st_dev = to_dev(state32)
    out = gka.gka_decode_step(st_dev, to_dev(step["q"][:, 0]), to_dev(step["k"][:, 0]),
                              to_dev(step["v"][:, 0]), to_dev(step["gate"][:, 0]), to_dev(a), 8,
                              flags=gka.GKA_FLAG_ADAPTIVE_LAMBDA)
    assert rel(out.cpu().numpy(), ref["out"]) < TOL_F32


# --------------------------------------------------------------------------- the solve alone (backward solve for dq)
def run_solve(inp, rhs, n_iter, bf16, precision=gka.GKA_PREC_NATIVE, flags=0):
    r_, k = to_dev(rhs, bf16), to_dev(inp["k"], bf16)
    gate, lam = to_dev(inp["gate"]), to_dev(inp["lam"])
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    x = gka.gka_solve_chunked(r_, k, gate, lam, n_iter, 64, precision=precision, flags=flags, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return x.float().cpu().numpy()


@pytest.mark.parametrize("d,n_iter", [(64, 6), (128, 0), (128, 8)])
def test_solve_f32_matches_the_oracle_iterates(d, n_iter):
    """x_t = CH(H_t + lambda_t I, rhs_t, r) for an arbitrary right-hand side (not unit norm: a gradient)."""
    cfg = synth.shrink(synth.CONFIGS[0], d=d, T=320, heads=3)
    inp = synth.make_inputs(cfg)
    rhs = np.random.default_rng(5).standard_normal(inp["q"].shape).astype(np.float32)
    ref = oracle.fwd(rhs, inp["k"], inp["v"], inp["gate"], inp["lam"], n_iter, want_x=True)["x"]
    x = run_solve(inp, rhs, n_iter, bf16=False)
    assert rel(x, ref) <= TOL_F32


@pytest.mark.parametrize("n_iter", [0, 1, 10])
def test_solve_bf16_native_matches_the_oracle_iterates(n_iter):
    """Tensor-core path; several work items cut the sequences so the start states come through the summaries."""
    cfg = synth.shrink(synth.CONFIGS[1], B=2, heads=3, T=64 * 70)
    inp = synth.make_inputs(cfg)
    rng = np.random.default_rng(6)
    rhs = synth.round_bf16(rng.standard_normal(inp["q"].shape).astype(np.float32))
    ref = oracle.fwd(rhs, inp["k"], inp["v"], inp["gate"], inp["lam"], n_iter, want_x=True)["x"]
    x = run_solve(inp, rhs, n_iter, bf16=True)
    assert np.all(np.isfinite(x))
    e = rel(x, ref)
    print("solve bf16 n_iter %d rel L2 %.3e" % (n_iter, e))
    assert e <= TOL_BF16


def test_solve_with_q_gives_the_forward_output_through_u():
    """Consistency of the two entry points: U_t x_t from the forward equals the oracle's U_t applied to the
    iterate that gka_solve_chunked returns for rhs = q (fp32 path, where both are accurate to 1e-4)."""
    cfg = synth.shrink(synth.CONFIGS[0], d=64, T=192, heads=2)
    inp = synth.make_inputs(cfg)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], cfg.n_iter, want_x=True)
    x = run_solve(inp, inp["q"], cfg.n_iter, bf16=False)
    assert rel(x, ref["x"]) <= TOL_F32
    out, _, _ = run_fwd(inp, cfg.n_iter, bf16=False)
    assert rel(out, ref["out"]) <= TOL_F32


# --------------------------------------------------------------------------- beta-augmented write
def _beta_for(inp, seed):
    rng = np.random.default_rng(seed)
    return (1.0 / (1.0 + np.exp(-rng.standard_normal(inp["gate"].shape)))).astype(np.float32)


@pytest.mark.parametrize("d", [64, 128])
def test_fwd_beta_write_f32(d):
    """H_t = gamma_t H_{t-1} + beta_t k k^T, U_t = gamma_t U_{t-1} + beta_t v k^T (Remark on the beta-augmented
    variant, Section 4.1), fp32 path, sequences cut by work items."""
    cfg = synth.shrink(synth.CONFIGS[0], d=d, T=384, heads=3)
    inp = synth.make_inputs(cfg)
    beta = _beta_for(inp, 7)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], cfg.n_iter, beta=beta)
    q, k, v = (to_dev(inp[n]) for n in ("q", "k", "v"))
    out, st = gka.gka_fwd_chunked(q, k, v, to_dev(inp["gate"]), to_dev(inp["lam"]), cfg.n_iter, 64, beta=to_dev(beta))
    torch.cuda.synchronize()
    assert rel(out.cpu().numpy(), ref["out"]) <= TOL_F32
    assert rel(st.cpu().numpy(), ref["state"]) <= 1e-5


def test_fwd_beta_write_bf16_native():
    """Tensor-core path with write strengths; the run crosses several work items."""
    cfg = synth.shrink(synth.CONFIGS[1], B=2, heads=3, T=64 * 70)
    inp = synth.make_inputs(cfg)
    beta = _beta_for(inp, 8)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], cfg.n_iter, beta=beta, want_x=True)
    q, k, v = (to_dev(inp[n], True) for n in ("q", "k", "v"))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out, st = gka.gka_fwd_chunked(q, k, v, to_dev(inp["gate"]), to_dev(inp["lam"]), cfg.n_iter, 64,
                                  beta=to_dev(beta), device_status=status)
    x = gka.gka_solve_chunked(q, k, to_dev(inp["gate"]), to_dev(inp["lam"]), cfg.n_iter, 64, beta=to_dev(beta))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    e, es, ex = rel(out.float().cpu().numpy(), ref["out"]), rel(st.cpu().numpy(), ref["state"]), \
        rel(x.float().cpu().numpy(), ref["x"])
    print("beta bf16 rel L2 out %.3e state %.3e solve %.3e" % (e, es, ex))
    assert e <= TOL_BF16 and es <= 5e-3 and ex <= TOL_BF16


def test_decode_beta_write():
    cfg = synth.shrink(synth.CONFIGS[2], B=6, heads=4)
    rng = np.random.default_rng(9)
    N, Hh, d = cfg.B, cfg.heads, cfg.d
    state = (0.05 * rng.standard_normal((N, Hh, 2 * d * d))).astype(np.float32)
    # a valid H block: symmetric positive semi-definite
    for n in range(N):
        for h in range(Hh):
            A = rng.standard_normal((d, 8)) * 0.2
            state[n, h, :d * d] = (A @ A.T).astype(np.float32).ravel()
    unit = lambda x: x / np.linalg.norm(x, axis=-1, keepdims=True)
    q = synth.round_bf16(unit(rng.standard_normal((N, Hh, d))).astype(np.float32))
    k = synth.round_bf16(unit(rng.standard_normal((N, Hh, d))).astype(np.float32))
    v = synth.round_bf16(rng.standard_normal((N, Hh, d)).astype(np.float32))
    gate = (1 / (1 + np.exp(-rng.normal(2, 1, (N, Hh))))).astype(np.float32)
    lam = (np.log1p(np.exp(rng.standard_normal((N, Hh)))) + 1e-2).astype(np.float32)
    beta = (1 / (1 + np.exp(-rng.standard_normal((N, Hh))))).astype(np.float32)
    ref = oracle.decode(state, q, k, v, gate, lam, 10, beta=beta)
    s_dev = to_dev(state)
    out = gka.gka_decode_step(s_dev, to_dev(q, True), to_dev(k, True), to_dev(v, True), to_dev(gate), to_dev(lam), 10,
                              beta=to_dev(beta))
    torch.cuda.synchronize()
    assert rel(out.float().cpu().numpy(), ref["out"]) <= TOL_BF16
    assert rel(s_dev.cpu().numpy(), ref["state"]) <= 1e-5


# --------------------------------------------------------------------------- alpha-connection
@pytest.mark.parametrize("bf16,n_iter", [(False, 8), (True, 10), (True, 0), (True, 3)])
def test_fwd_alpha_connection(bf16, n_iter):
    """out_t = U_t (alpha_t x_t + (1 - alpha_t) q_t) (Section 4.3, "Architectural Consideration"), both forward paths, with write strengths too."""
    cfg = synth.shrink(synth.CONFIGS[1 if bf16 else 0], B=2, heads=3, T=64 * 9, d=128)
    inp = synth.make_inputs(cfg)
    alpha, beta = _beta_for(inp, 11), _beta_for(inp, 12)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], n_iter, alpha=alpha, beta=beta)
    q, k, v = (to_dev(inp[n], bf16) for n in ("q", "k", "v"))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out, st = gka.gka_fwd_chunked(q, k, v, to_dev(inp["gate"]), to_dev(inp["lam"]), n_iter, 64,
                                  alpha=to_dev(alpha), beta=to_dev(beta), device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    e = rel(out.float().cpu().numpy(), ref["out"])
    print("alpha bf16=%s n_iter %d rel L2 %.3e" % (bf16, n_iter, e))
    assert e <= (TOL_BF16 if bf16 else TOL_F32)
    assert rel(st.cpu().numpy(), ref["state"]) <= (5e-3 if bf16 else 1e-5)


def test_decode_alpha_connection():
    cfg = synth.shrink(synth.CONFIGS[2], B=5, heads=3)
    rng = np.random.default_rng(13)
    N, Hh, d = cfg.B, cfg.heads, cfg.d
    state = np.zeros((N, Hh, 2 * d * d), np.float32)
    for n in range(N):
        for h in range(Hh):
            A = rng.standard_normal((d, 8)) * 0.2
            state[n, h, :d * d] = (A @ A.T).astype(np.float32).ravel()
            state[n, h, d * d:] = (0.05 * rng.standard_normal(d * d)).astype(np.float32)
    unit = lambda x: x / np.linalg.norm(x, axis=-1, keepdims=True)
    q = unit(rng.standard_normal((N, Hh, d))).astype(np.float32)
    k = unit(rng.standard_normal((N, Hh, d))).astype(np.float32)
    v = rng.standard_normal((N, Hh, d)).astype(np.float32)
    gate = (1 / (1 + np.exp(-rng.normal(2, 1, (N, Hh))))).astype(np.float32)
    lam = (np.log1p(np.exp(rng.standard_normal((N, Hh)))) + 1e-2).astype(np.float32)
    alpha = (1 / (1 + np.exp(-rng.standard_normal((N, Hh))))).astype(np.float32)
    ref = oracle.decode(state, q, k, v, gate, lam, 10, alpha=alpha)
    s_dev = to_dev(state)
    out = gka.gka_decode_step(s_dev, to_dev(q), to_dev(k), to_dev(v), to_dev(gate), to_dev(lam), 10, alpha=to_dev(alpha))
    torch.cuda.synchronize()
    assert rel(out.cpu().numpy(), ref["out"]) <= TOL_F32
    assert rel(s_dev.cpu().numpy(), ref["state"]) <= 1e-5


# --------------------------------------------------------------------------- sequence lengths that are not multiples of the chunk
@pytest.mark.parametrize("bf16,d,B,heads,T", [
    (True, 128, 2, 3, 1), (True, 128, 2, 3, 63), (True, 128, 1, 2, 65), (True, 128, 2, 2, 127), (True, 128, 2, 3, 129),
    (True, 128, 3, 2, 64 * 5 + 17), (True, 128, 1, 3, 64 * 70 + 33), (True, 128, 1, 1, 64 * 301 + 1),
    (False, 64, 2, 3, 1), (False, 64, 2, 2, 50), (False, 128, 2, 3, 100), (False, 128, 1, 5, 64 * 5 + 17),
    (True, 64, 2, 2, 64 * 3 + 5)])
def test_fwd_ragged_sequence_length(bf16, d, B, heads, T):
    """The last chunk of every sequence holds T mod 64 tokens: outputs, norms and final state follow the token
    recurrence (eq. (CH)) for exactly T tokens, and nothing past a sequence's last token is written."""
    cfg = synth.shrink(synth.CONFIGS[1 if bf16 else 0], B=B, heads=heads, T=T, d=d, n_iter=5)
    inp = synth.make_inputs(cfg)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 5, want_x=True)
    q, k, v = (to_dev(inp[n], bf16) for n in ("q", "k", "v"))
    pad = 3 * heads * d
    big = torch.full((B * T * heads * d + pad,), 7.0, dtype=q.dtype, device=DEV)
    out = big[:B * T * heads * d].view(B, T, heads, d)
    fbig = torch.full((B * T * heads + 8,), -3.0, dtype=torch.float32, device=DEV)
    fro = fbig[:B * T * heads].view(B, T, heads)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    _, st = gka.gka_fwd_chunked(q, k, v, to_dev(inp["gate"]), to_dev(inp["lam"]), 5, 64, out=out, fro_out=fro,
                                device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert bool((big[B * T * heads * d:] == 7.0).all()) and bool((fbig[B * T * heads:] == -3.0).all())
    tensor_path = bf16 and T >= 16
    o = out.float().cpu().numpy()
    assert rel(o, ref["out"]) <= (TOL_BF16 if bf16 else TOL_F32)
    assert rel(fro.cpu().numpy(), ref["fro"]) <= (5e-3 if tensor_path else 1e-5)
    assert rel(st.cpu().numpy(), ref["state"]) <= (5e-3 if tensor_path else 1e-5)


@pytest.mark.parametrize("bf16", [False, True])
def test_ragged_length_with_every_option(bf16):
    """Write strengths, alpha-connection, a caller's initial state and the solve alone on a ragged length."""
    B, heads, T, d = 2, 3, 64 * 9 + 40, 128
    cfg = synth.shrink(synth.CONFIGS[1 if bf16 else 0], B=B, heads=heads, T=T, d=d, n_iter=4)
    inp = synth.make_inputs(cfg)
    alpha, beta = _beta_for(inp, 5), _beta_for(inp, 6)
    rng = np.random.default_rng(17)
    s_in = np.zeros((B, heads, 2 * d * d), np.float32)
    for b in range(B):
        for h in range(heads):
            A = rng.standard_normal((d, 6)) * 0.3
            s_in[b, h, :d * d] = (A @ A.T).astype(np.float32).ravel()
            s_in[b, h, d * d:] = (0.1 * rng.standard_normal(d * d)).astype(np.float32)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 4, state_in=s_in, alpha=alpha, beta=beta,
                     want_x=True)
    q, k, v = (to_dev(inp[n], bf16) for n in ("q", "k", "v"))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out, st = gka.gka_fwd_chunked(q, k, v, to_dev(inp["gate"]), to_dev(inp["lam"]), 4, 64, state_in=to_dev(s_in),
                                  alpha=to_dev(alpha), beta=to_dev(beta), device_status=status)
    x = gka.gka_solve_chunked(q, k, to_dev(inp["gate"]), to_dev(inp["lam"]), 4, 64, state_in=to_dev(s_in),
                              beta=to_dev(beta), device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert rel(out.float().cpu().numpy(), ref["out"]) <= (TOL_BF16 if bf16 else TOL_F32)
    assert rel(x.float().cpu().numpy(), ref["x"]) <= (TOL_BF16 if bf16 else TOL_F32)
    assert rel(st.cpu().numpy(), ref["state"]) <= (5e-3 if bf16 else 1e-5)


# --------------------------------------------------------------------------- very short sequences
@pytest.mark.parametrize("T", [1, 2, 4, 7, 15, 16, 24])
@pytest.mark.parametrize("d", [64, 128])
def test_fwd_bf16_very_short_sequences_under_the_adaptive_rule(T, d):
    """From a zero state the first tokens have an all but rank-one H_t, the hardest case for bf16 operands (x_t is
    dominated by q_t / lambda_t off the key direction, the read takes its key component).  Sequences of fewer than 16
    tokens run in fp32 arithmetic whatever the precision asked for; from 16 tokens on the tensor-core path meets the
    same bar, at the paper's a = 0.02 and at 1, 10 and 30 iterations."""
    for n_iter in (1, 10, 30):
        for seed in (100, 101, 102):
            cfg = synth.shrink(synth.CONFIGS[1], B=2, heads=3, T=T, d=d, n_iter=n_iter, seed=seed)
            inp = synth.make_inputs(cfg)
            lam = np.full_like(inp["lam"], 0.02)
            ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], lam, n_iter, lam_mode=1)
            q, k, v = (to_dev(inp[n], True) for n in ("q", "k", "v"))
            status = torch.zeros(1, dtype=torch.int32, device=DEV)
            out, st = gka.gka_fwd_chunked(q, k, v, to_dev(inp["gate"]), to_dev(lam), n_iter, 64,
                                          flags=gka.GKA_FLAG_ADAPTIVE_LAMBDA, device_status=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert rel(out.float().cpu().numpy(), ref["out"]) <= TOL_BF16, (T, d, n_iter, seed)
            assert rel(st.cpu().numpy(), ref["state"]) <= 5e-3


# --------------------------------------------------------------------------- head dimensions 16 and 32
@pytest.mark.parametrize("d,bf16,precision", [(16, False, 0), (32, False, 0), (16, True, 0), (32, True, 0), (32, True, 1)])
def test_fwd_small_head_dimensions(d, bf16, precision):
    """Head dimensions 16 and 32 run on the 64-channel fp32 kernels, zero-extended on chip (whatever the I/O dtype and
    precision): several heads side by side, a ragged last chunk, work items that cut sequences, a caller-supplied
    initial state in the caller's d x d layout, write strengths and the alpha-connection; outputs, norms, final state
    and the solve alone against the oracle."""
    B, heads, T = 2, 5, 64 * 40 + 23
    cfg = synth.shrink(synth.CONFIGS[1 if bf16 else 0], B=B, heads=heads, T=T, d=d, n_iter=6)
    inp = synth.make_inputs(cfg)
    alpha, beta = _beta_for(inp, 8), _beta_for(inp, 9)
    rng = np.random.default_rng(23)
    s_in = np.zeros((B, heads, 2 * d * d), np.float32)
    for b in range(B):
        for h in range(heads):
            A = rng.standard_normal((d, 4)) * 0.3
            s_in[b, h, :d * d] = (A @ A.T).astype(np.float32).ravel()
            s_in[b, h, d * d:] = (0.1 * rng.standard_normal(d * d)).astype(np.float32)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 6, state_in=s_in, alpha=alpha, beta=beta,
                     want_x=True)
    q, k, v = (to_dev(inp[n], bf16) for n in ("q", "k", "v"))
    gate, lam = to_dev(inp["gate"]), to_dev(inp["lam"])
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    fro = torch.zeros(B, T, heads, dtype=torch.float32, device=DEV)
    out, st = gka.gka_fwd_chunked(q, k, v, gate, lam, 6, 64, state_in=to_dev(s_in), alpha=to_dev(alpha), beta=to_dev(beta),
                                  precision=precision, fro_out=fro, device_status=status)
    x = gka.gka_solve_chunked(q, k, gate, lam, 6, 64, state_in=to_dev(s_in), beta=to_dev(beta), precision=precision,
                              device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    tol = TOL_BF16 if bf16 else TOL_F32          # bf16 I/O: the output is rounded to bf16, the arithmetic is fp32
    assert rel(out.float().cpu().numpy(), ref["out"]) <= tol
    assert rel(x.float().cpu().numpy(), ref["x"]) <= tol
    assert rel(fro.cpu().numpy(), ref["fro"]) <= 1e-5
    assert rel(st.cpu().numpy(), ref["state"]) <= 1e-5


# --------------------------------------------------------------------------- multi-token decode
@pytest.mark.parametrize("d,bf16,T,extras", [(128, False, 1, False), (128, False, 7, True), (128, True, 16, False),
                                              (64, False, 5, True), (64, True, 3, False), (128, True, 4, True),
                                              (32, False, 1, False), (32, True, 6, True), (16, False, 9, True), (16, True, 1, False)])
def test_decode_tokens_matches_the_token_recurrence(d, bf16, T, extras):
    """T tokens in one call continue a prefix state exactly like the token-by-token recurrence (eq. (CH)):
    outputs and final state against the oracle run on prefix + T tokens, and against T single-token calls."""
    P = 64
    cfg = synth.shrink(synth.CONFIGS[0], B=3, heads=2, T=P + T, d=d, n_iter=7)
    inp = synth.make_inputs(cfg)
    if bf16:
        inp = {n: (synth.round_bf16(a) if n in ("q", "k", "v") else a) for n, a in inp.items()}
    alpha = _beta_for(inp, 3) if extras else None
    beta = _beta_for(inp, 4) if extras else None
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 7, alpha=alpha, beta=beta)
    pre = oracle.fwd(inp["q"][:, :P], inp["k"][:, :P], inp["v"][:, :P], inp["gate"][:, :P], inp["lam"][:, :P], 0,
                     beta=None if beta is None else beta[:, :P])
    state0 = pre["state"].astype(np.float32)
    tail = lambda a, b16=False: to_dev(np.ascontiguousarray(a[:, P:]), b16)
    opt = lambda a: None if a is None else tail(a)
    st = to_dev(state0)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = gka.gka_decode_tokens(st, tail(inp["q"], bf16), tail(inp["k"], bf16), tail(inp["v"], bf16),
                                tail(inp["gate"]), tail(inp["lam"]), 7, alpha=opt(alpha), beta=opt(beta),
                                device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert rel(out.float().cpu().numpy(), ref["out"][:, P:]) <= (TOL_BF16 if bf16 else TOL_F32)
    assert rel(st.cpu().numpy(), ref["state"]) <= 1e-5
    # the same tokens one call at a time
    st1 = to_dev(state0)
    outs = []
    for t in range(P, P + T):
        one = lambda a, b16=False: to_dev(np.ascontiguousarray(a[:, t]), b16)
        o = gka.gka_decode_step(st1, one(inp["q"], bf16), one(inp["k"], bf16), one(inp["v"], bf16),
                                one(inp["gate"]), one(inp["lam"]), 7,
                                alpha=None if alpha is None else one(alpha),
                                beta=None if beta is None else one(beta))
        outs.append(o.float().cpu().numpy())
    torch.cuda.synchronize()
    assert rel(out.float().cpu().numpy(), np.stack(outs, axis=1)) <= (1e-2 if bf16 else 1e-6)
    assert rel(st.cpu().numpy(), st1.cpu().numpy()) <= 1e-6


# --------------------------------------------------------------------------- tile shapes of the tensor-core path
@pytest.mark.parametrize("d", [128, 64])
@pytest.mark.parametrize("B,heads,T", [(1, 1, 64), (1, 1, 64 * 5), (1, 2, 64 * 7), (3, 1, 64 * 3), (1, 1, 64 * 300)])
def test_fwd_bf16_native_tile_shapes(B, heads, T, d):
    """One-chunk sequences, odd chunk counts (half-filled 128-token tiles at run ends), one chunk per work item
    (every start state comes through a chain of summaries), one long sequence over all work items; with a
    caller-supplied initial state.  Head dimension 64 runs on the same kernels, zero-extended on chip."""
    cfg = synth.shrink(synth.CONFIGS[1], B=B, heads=heads, T=T, n_iter=3, d=d)
    inp = synth.make_inputs(cfg)
    rng = np.random.default_rng(21)
    d = cfg.d
    s_in = np.zeros((B, heads, 2 * d * d), np.float32)
    for b in range(B):
        for h in range(heads):
            A = rng.standard_normal((d, 6)) * 0.3
            s_in[b, h, :d * d] = (A @ A.T).astype(np.float32).ravel()
            s_in[b, h, d * d:] = (0.1 * rng.standard_normal(d * d)).astype(np.float32)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], 3, state_in=s_in)
    out, st, _ = run_fwd(inp, 3, True, state_in=s_in, want_fro=False)
    assert np.all(np.isfinite(out))
    assert rel(out, ref["out"]) <= TOL_BF16
    assert rel(st, ref["state"]) <= 5e-3


# --------------------------------------------------------------------------- host-buffer entry point
@pytest.mark.parametrize("bf16,B,T", [(False, 3, 64 * 6), (True, 5, 64 * 6), (True, 11, 64 * 6), (True, 5, 64 * 6 + 21),
                                      (False, 2, 64 + 9), (True, 3, 64 * 20 + 5), (False, 1, 64 * 9), (True, 10, 64 * 8)])
def test_fwd_host_buffers_match_device_call_and_oracle(bf16, B, T):
    """gka_fwd_chunked_host (pinned host buffers in, pinned host buffers out; the batch moves through the copy
    and kernel stages in slices, the last batch entries also in pieces along the sequence whose state is carried on
    the device) against the oracle and against the device-pointer call."""
    cfg = synth.shrink(synth.CONFIGS[1 if bf16 else 0], B=B, heads=2, T=T, d=128, n_iter=4)
    inp = synth.make_inputs(cfg)
    ref = oracle.fwd(inp["q"], inp["k"], inp["v"], inp["gate"], inp["lam"], cfg.n_iter)
    tdt = torch.bfloat16 if bf16 else torch.float32
    pin = {n: torch.from_numpy(np.ascontiguousarray(inp[n])).to(tdt if n in ("q", "k", "v") else torch.float32).pin_memory()
           for n in ("q", "k", "v", "gate", "lam")}
    out_pin = torch.empty_like(pin["v"]).pin_memory()
    st_pin = torch.empty(B, cfg.heads, 2 * cfg.d * cfg.d, dtype=torch.float32).pin_memory()
    staging = torch.empty(gka.gka_fwd_host_staging_bytes(B, cfg.T, cfg.heads, cfg.d, gka.GKA_BF16 if bf16 else gka.GKA_F32),
                          dtype=torch.uint8, device=DEV)
    ws = gka.alloc_workspace(B, cfg.T, cfg.heads, cfg.d, DEV, io_dtype=gka.GKA_BF16 if bf16 else gka.GKA_F32)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for _ in range(2):      # the second call reuses staging and helper streams while the first is still in flight
        gka.gka_fwd_chunked_host(pin["q"], pin["k"], pin["v"], pin["gate"], pin["lam"], cfg.n_iter, 64, out_pin, st_pin,
                                 staging=staging, workspace=ws, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    out, st = out_pin.float().numpy(), st_pin.numpy()
    assert rel(out, ref["out"]) <= (TOL_BF16 if bf16 else TOL_F32)
    assert rel(st, ref["state"]) <= (5e-3 if bf16 else 1e-5)
    dev_out, dev_st, _ = run_fwd(inp, cfg.n_iter, bf16, want_fro=False)
    assert rel(out, dev_out) <= (1e-2 if bf16 else 1e-5)
    assert rel(st, dev_st) <= (5e-3 if bf16 else 1e-5)


# ------------------------------------------------------------------------------- failure detection on the device
def test_bounded_wait_runs_out_and_the_library_stays_usable():
    """A bounded device-side wait that nothing satisfies gives up after its poll limit, reports GKA_ERR_TIMEOUT
    through device_status and returns; the next ordinary call works (nothing was in flight, nothing hangs)."""
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    gka.gka_selftest_bounded_wait(status, polls=2000)
    torch.cuda.synchronize()
    assert int(status.item()) == gka.GKA_ERR_TIMEOUT
    check_fwd(synth.shrink(synth.CONFIGS[1], B=1, heads=2, T=256))


def test_validate_flag_reports_inputs_outside_their_domain():
    """GKA_FLAG_VALIDATE: gamma in (0, 1] and lambda > 0 (L >= mu > 0, the input condition of Algorithm 1) are checked in
    one pass on the device; a violation stores GKA_ERR_DOMAIN, valid inputs leave the status at 0."""
    cfg = synth.shrink(synth.CONFIGS[1], B=1, heads=2, T=128)
    inp = synth.make_inputs(cfg)
    q, k, v = (to_dev(inp[n], True) for n in ("q", "k", "v"))
    gate, lam = to_dev(inp["gate"]), to_dev(inp["lam"])
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    gka.gka_fwd_chunked(q, k, v, gate, lam, 2, flags=gka.GKA_FLAG_VALIDATE, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for bad_gate, bad_lam in ((1.5, None), (0.0, None), (None, 0.0), (None, float("nan"))):
        g2, l2 = gate.clone(), lam.clone()
        if bad_gate is not None:
            g2[0, 77, 1] = bad_gate
        if bad_lam is not None:
            l2[0, 5, 0] = bad_lam
        status.zero_()
        gka.gka_fwd_chunked(q, k, v, g2, l2, 2, flags=gka.GKA_FLAG_VALIDATE, device_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 6, (bad_gate, bad_lam)
    # the decode step checks its scalars the same way
    st = torch.zeros(1, 2, 2 * 128 * 128, device=DEV)
    gd = torch.full((1, 2), 2.0, device=DEV)
    status.zero_()
    gka.gka_decode_step(st, q[:, 0], k[:, 0], v[:, 0], gd, lam[:, 0].contiguous(), 1, flags=gka.GKA_FLAG_VALIDATE,
                        device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 6

