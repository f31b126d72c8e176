"""hils_decode_noalloc, the decode entry point for embedders that cannot allocate device memory
(an engine whose KV-cache pool already owns all free HBM, a plugin without an allocator handle, a
loop that must not call cudaMalloc): it must give the same results as hils_decode while using only
the library's own fixed scratch array.  Collected last on purpose (file name), so that a run that
stops at the first failure has already run every other test.  The two calls in a row check that
what the first call leaves in the shared array does not leak into the second."""
import pytest
import torch

import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl
from parity import check_decode

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL_OUT, TOL_LSE = 2e-2, 1e-3          # the bf16 tolerances of the parity tests


def _run_pair(cfg, seq, query_set):
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32), query_set=query_set)
    g = {k: v.to(DEV) for k, v in inp.items()}
    ref_out, ref_lse, ref_sel = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K)
    out = torch.full_like(g["q"], float("nan"))
    lse = torch.full((cfg.B, cfg.Hq), float("nan"), dtype=torch.float32, device=DEV)
    sel = torch.full((cfg.B, cfg.Hkv, cfg.K), -7, dtype=torch.int32, device=DEV)
    status = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    hils.hils_decode_noalloc(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K, out, lse, sel,
                             device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert hils.last_launch_count() >= 1
    assert torch.equal(sel, ref_sel)
    assert (out.float() - ref_out.float()).abs().max().item() <= TOL_OUT
    assert (lse - ref_lse).abs().max().item() <= TOL_LSE
    return inp, out, lse, sel


def test_noalloc_matches_hils_decode_on_two_calls_in_a_row():
    # first call: many pairs, ragged lengths (also leaves partial sums and counters behind)
    _run_pair(wl.CONFIGS[3].scaled(B=16, L=4096, K=16, seed=71), [4096 - 97 * i for i in range(16)], 0)
    # second call: another shape and other queries over the same static scratch; this one also against the CPU oracle
    cfg = wl.CONFIGS[4].scaled(B=2, L=16384, K=64, seed=72)
    inp, out, lse, sel = _run_pair(cfg, [16384, 9001], 1)
    check_decode(cfg, inp, out, lse, sel)


def test_noalloc_clears_the_status_word_a_failed_call_left_in_the_shared_array():
    """A call with an impossible sequence length reports it through device_status (the bounds check skips the
    sequence, nothing faults); the word it leaves in the static array must not show up in the next call's status."""
    cfg = wl.CONFIGS[3].scaled(B=2, L=1024, K=4, seed=74)
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([1024, 512], dtype=torch.int32))
    g = {k: v.to(DEV) for k, v in inp.items()}
    out = torch.empty_like(g["q"])
    lse = torch.empty((cfg.B, cfg.Hq), dtype=torch.float32, device=DEV)
    sel = torch.empty((cfg.B, cfg.Hkv, cfg.K), dtype=torch.int32, device=DEV)
    status = torch.zeros((1,), dtype=torch.int32, device=DEV)
    bad = torch.tensor([1024, 0], dtype=torch.int32, device=DEV)
    hils.hils_decode_noalloc(g["q"], g["k"], g["v"], g["landmarks"], bad, cfg.S, cfg.K, out, lse, sel, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 2                  # bad index recorded, sequence skipped
    assert (sel[1] == -1).all()
    hils.hils_decode_noalloc(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K, out, lse, sel,
                             device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref_out, ref_lse, ref_sel = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K)
    assert torch.equal(sel, ref_sel)
    assert (out.float() - ref_out.float()).abs().max().item() <= TOL_OUT
    assert (lse - ref_lse).abs().max().item() <= TOL_LSE


def test_noalloc_rejects_shapes_beyond_its_fixed_scratch():
    cfg = wl.CONFIGS[3].scaled(B=1, L=1024, K=4, seed=73)
    inp = wl.make_decode_inputs(cfg, "cpu")
    g = {k: v.to(DEV) for k, v in inp.items()}
    out = torch.empty_like(g["q"])
    lse = torch.empty((1, cfg.Hq), dtype=torch.float32, device=DEV)
    sel = torch.empty((1, cfg.Hkv, cfg.K), dtype=torch.int32, device=DEV)
    # a cache far larger than 16 MiB of scratch allows: B*Hkv*C group scores alone exceed it
    import ctypes
    from paper_2607_02980_b200 import binding
    big = hils.make_params(B=128, Hq=32, Hkv=8, Hl=8, L=0, T_max=1 << 20, C=1 << 14, d=128, chunk_size=64,
                           top_k=64, dtype=binding.HILS_BF16)
    lib = hils.load_library()
    vp = ctypes.c_void_p
    lib.hils_decode_noalloc.restype = ctypes.c_int
    lib.hils_decode_noalloc.argtypes = [ctypes.POINTER(binding.HilsParams)] + [vp] * 11
    rc = lib.hils_decode_noalloc(ctypes.byref(big), vp(g["q"].data_ptr()), vp(g["k"].data_ptr()),
                                 vp(g["v"].data_ptr()), vp(g["landmarks"].data_ptr()), None,
                                 vp(g["seq_lens"].data_ptr()), vp(out.data_ptr()), vp(lse.data_ptr()),
                                 vp(sel.data_ptr()), None, None)
    assert rc == -4                       # HILS_ERR_WORKSPACE, nothing launched
    assert hils.last_launch_count() == 0
    # a shape outside the tuned decode kernels is refused, not silently routed elsewhere
    f32 = hils.make_params(B=1, Hq=32, Hkv=8, Hl=8, L=0, T_max=1024, C=16, d=128, chunk_size=64, top_k=4,
                           dtype=binding.HILS_F32)
    rc = lib.hils_decode_noalloc(ctypes.byref(f32), vp(g["q"].data_ptr()), vp(g["k"].data_ptr()),
                                 vp(g["v"].data_ptr()), vp(g["landmarks"].data_ptr()), None,
                                 vp(g["seq_lens"].data_ptr()), vp(out.data_ptr()), vp(lse.data_ptr()),
                                 vp(sel.data_ptr()), None, None)
    assert rc == -2
