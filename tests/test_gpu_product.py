"""Parity of csb_spmv / csb_spmm (CUDA, through the C ABI) with the float64 oracle."""
import numpy as np
import pytest
import torch

import workloads
from oracle import csb_oracle as O
from paper_2005_05758_b200 import binding

pytestmark = pytest.mark.gpu

RTOL = {"f16": 2e-3, "f32": 1e-5}   # max relative error per output allowed for each storage type


@pytest.fixture(autouse=True, params=["panel", "stream"])
def spmv_path(request, monkeypatch):
    """Batch-1 products of fp16 matrices have two kernels: the panel kernel (default) and the
    per-warp stream kernel that also serves fp32 values and small batches.  Every case runs on both;
    the choice is made when the matrix is encoded."""
    if request.param == "stream":
        monkeypatch.setenv("CSB_NO_PANEL", "1")
    else:
        monkeypatch.delenv("CSB_NO_PANEL", raising=False)
    return request.param


def check_product(got, want, scale, vd):
    """|got - want| <= rtol * max(|want|, 1e-2 * sum|w||x|): relative error per output, with
    the forward-error scale of the row as the floor where the exact output is near zero."""
    got = got.astype(np.float64)
    tol = RTOL[vd] * np.maximum(np.abs(want), 1e-2 * scale)
    bad = np.abs(got - want) > tol
    assert not bad.any(), "max excess %g at %s" % (np.max(np.abs(got - want) / np.maximum(tol, 1e-300)),
                                                   np.argwhere(bad)[:4].tolist())
    assert np.all(got[scale == 0] == 0.0)      # rows kept nowhere (or meeting only zeros) are exact zeros


def run_case(mat, X, opts=None, repeat=2):
    A = binding.csb_encode(mat.dense, mat.block_r, mat.block_c, mat.row_keep, mat.col_keep, mat.val_dtype, 0, opts)
    Xd = torch.from_numpy(X).cuda()
    B = X.shape[0]
    outs = []
    for _ in range(repeat):
        Y = torch.full((B, mat.rows), float("nan"), device="cuda")
        if B == 1:
            binding.csb_spmv(A, Xd[0], Y[0])
        else:
            binding.csb_spmm(A, Xd, Y)
        torch.cuda.synchronize()
        outs.append(Y.cpu().numpy())
    assert all(np.array_equal(outs[0], o) for o in outs[1:]), "two runs differ bitwise: summation order is not fixed"
    args = (mat.dense, mat.block_r, mat.block_c, mat.row_keep, mat.col_keep, mat.val_dtype)
    check_product(outs[0], O.spmm(*args, X), O.abs_scale(*args, X), mat.val_dtype)
    info = A.info()
    A.free()
    return info


@pytest.mark.parametrize("vd", ["f16", "f32"])
@pytest.mark.parametrize("shape", [(4, 4, 2, 2, 1), (64, 64, 16, 16, 1), (50, 39, 16, 8, 3), (512, 192, 16, 16, 1),
                                   (300, 1177, 32, 32, 1), (1024, 768, 64, 64, 8), (257, 513, 256, 256, 5),
                                   (2048, 2048, 64, 64, 13), (96, 4096, 32, 128, 2)])
def test_random_masks(shape, vd):
    R, C, br, bc, B = shape
    rng = np.random.default_rng(R + 7 * C + B)
    nblk = -(-R // br) * -(-C // bc)
    mat = workloads.MatrixSpec((rng.standard_normal((R, C)) * 0.1).astype(np.float32), br, bc,
                               (rng.random(nblk * br) < 0.45).astype(np.uint8),
                               (rng.random(nblk * bc) < 0.35).astype(np.uint8), vd)
    run_case(mat, rng.standard_normal((B, C)).astype(np.float32))


@pytest.mark.parametrize("law,kw", [("lognormal", dict(rate=16.0)), ("lognormal", dict(rate=4.0, diag_boost=4.0)),
                                    ("uniform", dict(lo=0.0, hi=1.0)), ("exact", dict(count=64)),
                                    ("exact", dict(count=0)), ("exact", dict(count=1))])
def test_keep_laws_and_degenerate_blocks(law, kw):
    w = workloads.make_spmv_workload(3, 1024, 1536, 64, 64, law, batch=1, w_std=0.05, **kw)
    run_case(w.matrix, w.X)


def test_rows_kept_nowhere_and_empty_block_rows():
    rng = np.random.default_rng(9)
    R, C, br, bc = 256, 256, 32, 32
    rk = (rng.random(64 * br) < 0.5).astype(np.uint8).reshape(8, 8, br)
    ck = (rng.random(64 * bc) < 0.5).astype(np.uint8).reshape(8, 8, bc)
    rk[2] = 0                # a whole block-row without kept rows
    ck[5] = 0                # a whole block-row without kept columns
    rk[:, :, 3] = 0          # in-block row 3 kept nowhere
    mat = workloads.MatrixSpec(rng.standard_normal((R, C)).astype(np.float32), br, bc, rk.reshape(-1), ck.reshape(-1), "f16")
    run_case(mat, rng.standard_normal((4, C)).astype(np.float32))


@pytest.mark.parametrize("B", [1, 3])
def test_heavy_block_row_is_divided_between_ctas(B):
    # one block-row keeps everything, the others about a tenth: the planner divides the heavy one
    # into pieces for several CTAs, which meet through partial sums; result and bit-reproducibility
    # as everywhere else
    w = workloads.make_spmv_workload(11, 8192, 4096, 64, 64, "lognormal", rate=10.0, batch=B, w_std=0.05)
    m = w.matrix
    m.row_keep.reshape(128, 64, 64)[5] = 1
    m.col_keep.reshape(128, 64, 64)[5] = 1
    info = run_case(m, w.X)
    A = binding.csb_encode(m.dense, 64, 64, m.row_keep, m.col_keep, "f16", device=-1)
    plan = binding.csb_plan_dump(A, info["plan_ctas"], 16, 4096)
    A.free()
    assert info["plan_ctas"] > 128 and plan["row_owned"] and plan["slots"] >= 2, "the case must exercise divided block-rows"


@pytest.mark.parametrize("opts", [dict(ctas=1, warps_per_cta=1), dict(ctas=3, warps_per_cta=5, stages=1),
                                  dict(ctas=148, warps_per_cta=16, stage_bytes=1024, stages=2), dict(ctas=500)])
def test_schedules_agree(opts):
    w = workloads.make_spmv_workload(4, 768, 1024, 32, 32, "lognormal", rate=8.0, batch=2, w_std=0.05)
    full = dict(ctas=0, warps_per_cta=0, stage_bytes=0, stages=0)
    full.update(opts)
    run_case(w.matrix, w.X, full)


def test_ring_too_large_for_16_warps_is_planned_with_fewer(spmv_path):
    # 128 block-rows make the plan row-owned (the CTA shape is then part of the plan); eight stages
    # of 8 KB per warp do not fit 16 warps, so the planner has to settle for fewer warps per CTA
    # instead of producing a plan that can never be launched
    if spmv_path != "stream":
        pytest.skip("csb_plan_opts belong to the stream kernel")
    rng = np.random.default_rng(17)
    R, C, br, bc = 8192, 512, 64, 64
    nblk = (R // br) * (C // bc)
    mat = workloads.MatrixSpec((rng.standard_normal((R, C)) * 0.1).astype(np.float32), br, bc,
                               (rng.random(nblk * br) < 0.4).astype(np.uint8), (rng.random(nblk * bc) < 0.4).astype(np.uint8), "f32")
    for B in (1, 5):
        info = run_case(mat, rng.standard_normal((B, C)).astype(np.float32), dict(ctas=0, warps_per_cta=0, stage_bytes=8192, stages=8))
        assert info["plan_warps"] < 16


@pytest.mark.parametrize("ctas,stage,ring", [(4, 8192, 14), (16, 8192, 15), (148, 16384, 15)])
def test_panel_ring_is_refilled_many_times(monkeypatch, spmv_path, ctas, stage, ring):
    # few CTAs and a ring of two or four small stages: every slot is refilled dozens of times and
    # warps run far ahead of each other, which is what the refill protocol has to survive
    if spmv_path != "panel":
        pytest.skip("the ring belongs to the panel kernel")
    monkeypatch.setenv("CSB_PANEL_STAGE", str(stage))
    monkeypatch.setenv("CSB_PANEL_RING_LOG2", str(ring))
    w = workloads.make_spmv_workload(21, 2048, 4096, 64, 64, "lognormal", rate=5.0, batch=1, w_std=0.05)
    run_case(w.matrix, w.X, dict(ctas=ctas, warps_per_cta=0, stage_bytes=0, stages=0), repeat=3)


@pytest.mark.parametrize("rate", [4.0, 8.0, 16.0, 25.0])
def test_cfg4_full_size_every_rate_and_batch(rate, spmv_path):
    # the benchmarked matrices themselves (8192 x 8192, 64 x 64 blocks), every output compared with
    # the oracle at every benchmarked batch size; the batched cases do not depend on the SpMV kernel
    # choice and run once
    w = workloads.CONFIGS["cfg4"](rate=rate, B=64)
    m = w.matrix
    args = (m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)
    want, scale = O.spmm(*args, w.X), O.abs_scale(*args, w.X)
    A = binding.csb_encode(*args[:5], m.val_dtype, 0)
    Xd = torch.from_numpy(w.X).cuda()
    for B in ((1,) if spmv_path == "stream" else (1, 8, 64)):
        outs = []
        for _ in range(2):
            Y = torch.full((B, m.rows), float("nan"), device="cuda")
            if B == 1:
                binding.csb_spmv(A, Xd[0], Y[0])
            else:
                binding.csb_spmm(A, Xd[:B], Y)
            torch.cuda.synchronize()
            outs.append(Y.cpu().numpy())
        assert np.array_equal(outs[0], outs[1]), "two runs differ bitwise at batch %d" % B
        check_product(outs[0], want[:B], scale[:B], m.val_dtype)
        big = np.abs(want[:B]) > 1e-2 * scale[:B]
        print("cfg4 %gx batch %d: max relative error %.3g over %d outputs above the floor"
              % (rate, B, float(np.max(np.abs(outs[0] - want[:B])[big] / np.abs(want[:B])[big])), int(big.sum())))
    assert A.info()["balance"] > 0.5
    A.free()
