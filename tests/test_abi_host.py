"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, validates arguments before any launch, and splits work as documented."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2511_21016_b200 import build, gka, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return gka.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gka.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gka_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"gka_fwd_chunked", "gka_decode_step", "gka_fwd_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/gka.h but not exported"
    assert set(gka.EXPORTS) <= set(names)


def test_status_strings(lib):
    assert gka.status_string(0) == "GKA_OK"
    seen = {gka.status_string(i) for i in range(10)}
    assert len(seen) == 10
    assert "unknown" in gka.status_string(99)


def test_workspace_bytes_arithmetic(lib):
    st = 2 * 128 * 128
    up = lambda n: (n + 255) // 256 * 256
    # fp32 path: 64 sequences x 64 chunks = 4096 chunks -> capped at 296 work items
    n = gka.gka_fwd_workspace_bytes(4, 4096, 16, 128, io_dtype=gka.GKA_F32)
    assert n == ((3 * 296 * st + 296) * 4 + 255) // 256 * 256
    # tensor-core path (bf16, d = 128): 2048 tiles of 128 tokens, each with bf16 copies of H_0 and U_0 and a norm
    n = gka.gka_fwd_workspace_bytes(4, 4096, 16, 128)
    assert n == 2 * up(296 * st * 4) + up(296 * 4) + up(2048 * 4) + 2048 * 65536
    # tiny problem: 2 sequences x 4 chunks = 8 items
    n = gka.gka_fwd_workspace_bytes(1, 256, 2, 64, io_dtype=gka.GKA_F32)
    assert n == ((3 * 8 * 2 * 64 * 64 + 8) * 4 + 255) // 256 * 256
    # T need not be a multiple of the chunk: 100 tokens are two chunks, the second one short
    assert gka.gka_fwd_workspace_bytes(1, 100, 2, 64) == gka.gka_fwd_workspace_bytes(1, 128, 2, 64)
    assert gka.gka_fwd_workspace_bytes(1, 0, 2, 64) == 0
    assert gka.gka_fwd_workspace_bytes(1, 128, 2, 96) == 0       # unsupported head dim


def _call_fwd(lib, desc, ptrs, n_iter=1, chunk=64):
    return lib.gka_fwd_chunked(ctypes.byref(desc), *ptrs[:5], n_iter, chunk, *ptrs[5:])


def test_argument_errors_are_reported_before_any_launch(lib):
    """None of these reaches a CUDA call, so they run without a GPU."""
    ok = 256  # fake, aligned, non-null "device pointers": never dereferenced on these paths
    ptrs = [ok] * 7
    d = gka.make_desc(1, 128, 2, 64, 64, gka.GKA_F32)
    assert _call_fwd(lib, d, [None] + ptrs[1:]) == 1                       # NULL
    assert _call_fwd(lib, d, ptrs, n_iter=-1) == 2                         # negative n_iter
    assert _call_fwd(lib, d, ptrs, chunk=32) == 4                          # unsupported chunk
    assert _call_fwd(lib, d, ptrs, chunk=0) == 2
    assert _call_fwd(lib, d, [ok + 4] + ptrs[1:]) == 9                     # misaligned q
    assert _call_fwd(lib, d, ptrs) == 5                                    # no workspace
    d.workspace, d.workspace_bytes = 256, 16
    assert _call_fwd(lib, d, ptrs) == 5                                    # workspace too small
    d2 = gka.make_desc(1, 0, 2, 64, 64, gka.GKA_F32)
    assert _call_fwd(lib, d2, ptrs) == 2                                   # no token
    d2 = gka.make_desc(1, 100, 2, 64, 64, gka.GKA_F32)
    assert _call_fwd(lib, d2, ptrs) == 5                                   # a ragged T passes the shape check
    d3 = gka.make_desc(1, 128, 2, 64, 128, gka.GKA_F32)
    assert _call_fwd(lib, d3, ptrs) == 2                                   # d_k != d_v
    d4 = gka.make_desc(1, 128, 2, 64, 64, 7)
    assert _call_fwd(lib, d4, ptrs) == 3                                   # bad dtype
    d5 = gka.make_desc(1, 128, 2, 64, 64, gka.GKA_F32, flags=0x10)
    assert _call_fwd(lib, d5, ptrs) == 4                                   # unknown flag
    dd = gka.make_desc(4, 1, 2, 128, 128, gka.GKA_BF16)
    rc = lib.gka_decode_step(ctypes.byref(dd), None, ok, ok, ok, ok, ok, 3, ok)
    assert rc == 1
    rc = lib.gka_decode_step(ctypes.byref(dd), ok, ok, ok + 2, ok, ok, ok, 3, ok)
    assert rc == 9
    rc = lib.gka_decode_step(None, ok, ok, ok, ok, ok, ok, 3, ok)
    assert rc == 1
    d0 = gka.make_desc(4, 0, 2, 128, 128, gka.GKA_BF16)
    assert lib.gka_decode_tokens(ctypes.byref(d0), ok, ok, ok, ok, ok, ok, 3, ok) == 2   # no token
    assert lib.gka_decode_tokens(ctypes.byref(dd), ok, None, ok, ok, ok, ok, 3, ok) == 1
    assert lib.gka_decode_tokens(ctypes.byref(dd), ok + 4, ok, ok, ok, ok, ok, 3, ok) == 9


@pytest.mark.parametrize("B,T,heads,G", [(4, 4096, 16, 148), (1, 131072, 32, 148), (1, 256, 2, 4),
                                         (1, 6400, 3, 148), (3, 192, 5, 7), (1, 64, 1, 1)])
@pytest.mark.parametrize("io", ["bf16", "f32"])
def test_work_ranges_partition_the_chunk_list(lib, B, T, heads, G, io):
    """bf16 I/O with head dimension 128 is planned in 128-token tiles (pairs of chunks, the last tile of a
    sequence with an odd number of chunks holding one), everything else in chunks."""
    N = T // 64
    NC = B * heads * N
    tiles = io == "bf16"
    prev_hi = 0
    sizes = []
    for i in range(G):
        lo, hi, cin, cout = gka.gka_fwd_work_range(B, T, heads, 128, G, i,
                                                   io_dtype=gka.GKA_BF16 if tiles else gka.GKA_F32)
        assert lo == prev_hi and hi > lo
        assert cin == (lo % N != 0) and cout == (hi % N != 0)
        if tiles:
            assert (lo % N) % 2 == 0          # boundaries between tiles
        sizes.append(hi - lo)
        prev_hi = hi
    assert prev_hi == NC
    if tiles:
        assert max(sizes) - min(sizes) <= 2 + (N % 2)   # one tile, and a short last tile counts one chunk
    else:
        unit = 2 if (N % 2 == 0 and 2 * G <= NC) else 1    # even boundaries where pairs of chunks can be kept whole
        assert max(sizes) - min(sizes) <= unit       # balanced to within one unit
        if unit == 2:
            assert all(sz % 2 == 0 for sz in sizes)
    with pytest.raises(gka.GkaError):
        gka.gka_fwd_work_range(B, T, heads, 128, G, G)


@pytest.mark.parametrize("B,T,heads", [(4, 4096, 16), (2, 640, 5), (1, 2000, 40), (3, 100, 7)])
def test_whole_sequences_as_work_items_cut_nothing(lib, B, T, heads):
    """With as many work items as (sequence, head) pairs (the decomposition the tensor-core path takes when carrying
    whole sequences is cheaper than cutting them) every range is one sequence: no range starts or ends inside one."""
    N = (T + 63) // 64
    pairs = B * heads
    for i in range(pairs):
        lo, hi, cin, cout = gka.gka_fwd_work_range(B, T, heads, 128, pairs, i, io_dtype=gka.GKA_BF16)
        assert (lo, hi) == (i * N, (i + 1) * N)
        assert not cin and not cout


def test_missing_library_is_an_error(monkeypatch, tmp_path):
    monkeypatch.setattr(gka, "_lib", None)
    monkeypatch.setattr(gka, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        gka.load_library()


def test_cpu_tensors_are_rejected():
    import torch
    t = torch.zeros(1, 64, 1, 64)
    g = torch.ones(1, 64, 1)
    with pytest.raises(ValueError):
        gka.gka_fwd_chunked(t, t, t, g, g, 1)


def test_binding_rejects_mismatched_tensors():
    """The kernels trust the descriptor, so the binding compares every tensor's dtype and shape with q before it
    calls the library: a mismatch is a ValueError, never a launch (CPU tensors suffice to show it)."""
    import torch
    B, T, H, d = 2, 64, 3, 64
    q = torch.zeros(B, T, H, d)
    g = torch.ones(B, T, H)
    st = torch.zeros(B, H, 2 * d * d)
    cases = [
        dict(k=q.double()), dict(k=q[:, :32]), dict(v=q.bfloat16()), dict(gate=g.double()), dict(lam=g[:, :, :2]),
        dict(gate=g.bfloat16()), dict(out=q.bfloat16()), dict(state_out=st[:, :, :-4]), dict(state_out=st.double()),
        dict(state_in=st[:1]), dict(fro_out=g.double()), dict(beta=g[:, :10]), dict(alpha=g.half()),
        dict(device_status=torch.zeros(1, dtype=torch.int64)),
    ]
    for bad in cases:
        kw = dict(k=q, v=q, gate=g, lam=g)
        kw.update(bad)
        k, v, gate, lam = (kw.pop(n) for n in ("k", "v", "gate", "lam"))
        with pytest.raises(ValueError, match="dtype|shape"):
            gka.gka_fwd_chunked(q, k, v, gate, lam, 1, **kw)
    with pytest.raises(ValueError, match="dtype|shape"):
        gka.gka_solve_chunked(q, q.double(), g, g, 1)
    with pytest.raises(TypeError):
        gka.gka_fwd_chunked(q.double(), q.double(), q.double(), g, g, 1)          # unsupported I/O dtype
    # decode: state of the wrong size, per-head scalars of the wrong shape
    qd, gd = torch.zeros(4, H, d), torch.ones(4, H)
    with pytest.raises(ValueError, match="shape"):
        gka.gka_decode_step(torch.zeros(4, H, d * d), qd, qd, qd, gd, gd, 1)
    with pytest.raises(ValueError, match="shape"):
        gka.gka_decode_step(torch.zeros(4, H, 2 * d * d), qd, qd, qd, gd[:, :2], gd, 1)
    with pytest.raises(ValueError, match="dtype"):
        gka.gka_decode_tokens(torch.zeros(4, H, 2 * d * d).double(), q[:, :4].transpose(0, 1).contiguous(),
                              q[:, :4].transpose(0, 1).contiguous(), q[:, :4].transpose(0, 1).contiguous(),
                              torch.ones(4, 2, H), torch.ones(4, 2, H), 1)
    with pytest.raises(ValueError, match="dtype|shape"):
        gka.gka_fwd_chunked_noalloc(q, q, q, g, g.double(), 1)


def test_synth_substreams_and_distributions():
    cfg = synth.shrink(synth.CONFIGS[1], B=2, heads=3, T=128)
    full = synth.make_inputs(cfg)
    part = synth.make_inputs(cfg, pairs=[(1, 2)])
    for key in full:
        assert np.array_equal(full[key][1, :, 2], part[key][1, :, 2])
    assert full["q"].shape == (2, 128, 3, 128) and full["gate"].shape == (2, 128, 3)
    # bf16-representable, unit-norm up to bf16 rounding
    assert np.array_equal(synth.round_bf16(full["k"]), full["k"])
    assert np.allclose(np.linalg.norm(full["k"], axis=-1), 1.0, atol=2e-2)
    assert np.all((full["gate"] > 0) & (full["gate"] <= 1)) and np.all(full["lam"] >= 1e-2)
    # stress recipe: keys close to a rank-8 subspace, tiny lambda
    c4 = synth.shrink(synth.CONFIGS[4], B=1, heads=1, T=512)
    x = synth.make_inputs(c4)
    sv = np.linalg.svd(x["k"][0, :, 0].astype(np.float64), compute_uv=False)
    assert sv[8] < 0.05 * sv[7]
    assert x["lam"].max() < 1e-3
    # bf16 rounding helper: ties to even
    assert synth.to_bf16_bits(np.array([1.0, 1.00390625, 1.01171875], np.float32)).tolist() == \
        [0x3F80, 0x3F80, 0x3F82]
