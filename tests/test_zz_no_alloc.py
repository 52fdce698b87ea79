"""gptaq_quantize_static: the quantize step for callers that may not allocate device memory.

Some users of the library run where the CUDA allocator is out of reach -- a serving loop with a
fixed memory plan, a plug-in that is forbidden to allocate, a pool that is already full -- so
they cannot size a per-layer workspace for the lazy-batch update.  For them the library carries
a fixed scratch array of its own.  This file checks, through the C ABI, that the entry point
built on that array gives exactly what gptaq_quantize gives on the same factor, correction
matrix and weights, on two calls in a row (the second finds the first call's leftovers in the
shared array), that a layer wide enough for gptaq_quantize to switch to its tensor-core update
(which this entry point never uses) still matches the float64 oracle, and that sizes beyond the
array are refused on the host.

The file name sorts last on purpose: a run that stops at the first failure has then already
been through every other test.
"""
import numpy as np
import pytest
import torch

import paper_2504_02692_b200 as g
import workloads as wl
from oracle import gptaq_oracle as orc
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _factored_state(cfg):
    st = g.LayerState(cfg.n, cfg.m, cfg.batch_tokens, cfg.blocksize)
    for b in range(cfg.n_batches):
        X, Xfp = wl.make_batch(cfg, b)
        g.gptaq_accumulate(st.handle, X.cuda(), Xfp.cuda())
    g.gptaq_factor(st.handle, cfg.damp)
    g.gptaq_build_P(st.handle, cfg.alpha)
    assert g.gptaq_sync_status(st.handle)[0] == g.GPTAQ_OK
    return st


def _outputs(m, n, group):
    G = 1 if group <= 0 else (n + group - 1) // group
    return (torch.empty((m, n), dtype=torch.uint8, device="cuda"),
            torch.empty((m, G), dtype=torch.float32, device="cuda"),
            torch.empty((m, G), dtype=torch.float32, device="cuda"),
            torch.empty((m, n), dtype=torch.float32, device="cuda"))


def test_static_scratch_entry_point_matches_gptaq_quantize_twice_in_a_row():
    cfg = wl.scaled(wl.CONFIGS["cfg2"], name="static", n=384, m=200, batch_tokens=1536, n_batches=2,
                    outlier_channels=4, group=64, blocksize=128)
    st = _factored_state(cfg)
    U, P = st.H().clone(), st.D().clone()
    W_all = wl.make_weight(cfg).cuda()
    status = torch.full((2,), -1, dtype=torch.int64, device="cuda")
    # two different weight matrices, the second one smaller: its rows land on scratch that still
    # holds the first call's errors and pre-quantization columns
    for W in (W_all, W_all[37:150].contiguous() * 1.5):
        m = W.shape[0]
        codes, scales, zeros, Wq = _outputs(m, cfg.n, cfg.group)
        g.gptaq_quantize(st.handle, W, cfg.bits, cfg.group, cfg.sym, cfg.blocksize, codes, scales, zeros, Wq)
        assert g.gptaq_sync_status(st.handle)[0] == g.GPTAQ_OK
        codes2, scales2, zeros2, Wq2 = _outputs(m, cfg.n, cfg.group)
        g.gptaq_quantize_static(U, P, W, cfg.bits, cfg.group, cfg.sym, cfg.blocksize, codes2, scales2, zeros2,
                                Wq2, status)
        torch.cuda.synchronize()
        assert status.tolist() == [g.GPTAQ_OK, 0]
        # integer codes bit for bit; grids and dequantized weights are the same float32 arithmetic
        assert np.array_equal(codes2.cpu().numpy(), codes.cpu().numpy())
        assert np.array_equal(zeros2.cpu().numpy(), zeros.cpu().numpy())
        assert np.array_equal(scales2.cpu().numpy(), scales.cpu().numpy())
        assert np.array_equal(Wq2.cpu().numpy(), Wq.cpu().numpy())
    st.close()


def test_static_scratch_entry_point_against_the_oracle_on_a_wide_layer():
    """n = 640: gptaq_quantize takes the split-fp16 tensor-core update from this width on, the entry
    point without a workspace keeps the float32 FMA update, so the two no longer agree bit for bit.
    Both have to match the oracle: codes in follow mode, objective, and never worse than plain
    rounding -- on two calls in a row, the second on fewer rows."""
    cfg = wl.scaled(wl.CONFIGS["cfg2"], name="static_wide", n=640, m=104, batch_tokens=2560, n_batches=2,
                    outlier_channels=6, group=128, blocksize=128)
    batches = [wl.make_batch(cfg, b) for b in range(cfg.n_batches)]
    st = _factored_state(cfg)
    Ud, Pd = st.H().clone(), st.D().clone()
    ost = hp.oracle_stats(cfg, batches)
    U, dead = orc.factor(ost.H, ost.tokens, cfg.damp)
    P = orc.build_P(ost.D, ost.tokens, U, cfg.alpha)
    assert not dead.any()
    assert hp.rel_fro(np.triu(Ud.cpu().numpy().astype(np.float64)), U) <= hp.TOL_FACTOR
    W_all = wl.make_weight(cfg)
    status = torch.full((2,), -1, dtype=torch.int64, device="cuda")
    for W in (W_all, W_all[11:80].contiguous() * 0.7):
        m = W.shape[0]
        Wn = W.numpy().astype(np.float64)
        codes, scales, zeros, Wq = _outputs(m, cfg.n, cfg.group)
        g.gptaq_quantize_static(Ud, Pd, W.cuda(), cfg.bits, cfg.group, cfg.sym, cfg.blocksize, codes, scales, zeros,
                                Wq, status)
        torch.cuda.synchronize()
        assert status.tolist() == [g.GPTAQ_OK, 0]
        rep = orc.follow(Wn, U, P, dead, cfg.bits, cfg.group, cfg.sym, codes.cpu().numpy(),
                         scales.cpu().numpy().astype(np.float64), zeros.cpu().numpy().astype(np.float64),
                         band=hp.TOL_FLIP_BAND)
        assert rep.disallowed == 0 and rep.allowed <= hp.TOL_FLIP_RATE * rep.total, rep
        assert rep.grid_rel_err <= hp.TOL_GRID and rep.zero_mismatch == 0, rep
        res = orc.quantize(Wn, U, P, dead, cfg.bits, cfg.group, cfg.sym)
        rtn = orc.quantize(Wn, U, None, dead, cfg.bits, cfg.group, cfg.sym, update=False)
        J_gpu = orc.objective(Wn, Wq.cpu().numpy().astype(np.float64), ost)
        J_orc, J_rtn = orc.objective(Wn, res.Wq, ost), orc.objective(Wn, rtn.Wq, ost)
        assert abs(J_gpu - J_orc) <= hp.TOL_OBJECTIVE * J_orc, (J_gpu, J_orc)
        assert J_gpu <= J_rtn, (J_gpu, J_rtn)
    st.close()


def test_static_scratch_entry_point_refuses_sizes_beyond_its_array():
    n = 64
    U = torch.eye(n, device="cuda")
    P = torch.zeros((n, n), device="cuda")
    m = g.GPTAQ_STATIC_SCRATCH_FLOATS // (2 * 128) + 1          # one row too many at B = 128
    W = torch.zeros((m, n), device="cuda")
    codes, scales, zeros, _ = _outputs(m, n, 0)
    with pytest.raises(g.GptaqError) as e:
        g.gptaq_quantize_static(U, P, W, 4, 0, False, 128, codes, scales, zeros)
    assert e.value.status == g.GPTAQ_ERR_WORKSPACE and "built-in scratch" in str(e.value)
    # the same rows fit with a smaller lazy-batch block
    g.gptaq_quantize_static(U, P, W, 4, 0, False, 32, codes, scales, zeros)
    torch.cuda.synchronize()
    assert int(codes.max()) == 0 and float(scales.min()) == 1.0    # all-zero rows: grid (1, 0)
