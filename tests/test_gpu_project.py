"""Parity of csb_project (CUDA, through the C ABI) with the oracle of Algorithm 1's RowPrune /
ColumnPrune: the keep masks are integer work and must match bit for bit.  Norms are fp64 sums on
both sides; random fp32 data has no ties closer than the last bits of a double, coarse-valued data
has exact ties, which the index rule decides the same way on both sides."""
import numpy as np
import pytest
import torch

from oracle import csb_oracle as O
from oracle import project_oracle as P
from paper_2005_05758_b200 import binding

pytestmark = pytest.mark.gpu


def run(W, br, bc, pr):
    Wd = torch.from_numpy(W).cuda()
    rk, ck, _ = binding.csb_project(Wd, br, bc, pr)
    torch.cuda.synchronize()
    return rk.cpu().numpy(), ck.cpu().numpy()


@pytest.mark.parametrize("R,C,br,bc,pr", [(4, 4, 2, 2, 0.75), (64, 96, 16, 32, 0.84), (300, 1177, 32, 32, 0.875), (512, 192, 16, 16, 0.75),
                                         (257, 513, 64, 64, 0.5), (96, 640, 32, 128, 0.96), (33, 70, 256, 7, 0.3)])
def test_masks_match_the_oracle(R, C, br, bc, pr):
    rng = np.random.default_rng(R + C)
    W = rng.standard_normal((R, C)).astype(np.float32)
    rk, ck = run(W, br, bc, pr)
    wrk, wck, Z = P.project(W, br, bc, pr)
    assert np.array_equal(rk, wrk) and np.array_equal(ck, wck)
    # and the masks feed the encoder: its masked matrix is the projected one
    A = binding.csb_encode(W, br, bc, rk, ck, "f32", device=-1)
    assert A.info()["nnz"] == int((O.block_mask(R, C, br, bc, rk, ck)).sum())
    A.free()


def test_ties_limits_and_strided_input():
    W = (np.round(np.random.default_rng(2).standard_normal((128, 160)) * 2) / 2).astype(np.float32)   # many exact ties, zero rows
    W[5] = 0
    W[:, 9] = 0
    for pr in (0.0, 0.6, 1.0):
        rk, ck = run(W, 32, 32, pr)
        wrk, wck, _ = P.project(W, 32, 32, pr)
        assert np.array_equal(rk, wrk) and np.array_equal(ck, wck), pr
    big = torch.from_numpy(np.pad(W, ((0, 0), (0, 37)))).cuda()          # row stride larger than cols
    rk, ck, _ = binding.csb_project(big[:, :160], 32, 32, 0.6)
    wrk, wck, _ = P.project(W, 32, 32, 0.6)
    assert np.array_equal(rk.cpu().numpy(), wrk) and np.array_equal(ck.cpu().numpy(), wck)


def test_hand_worked_example_and_errors():
    import json, os
    with open(os.path.join(os.path.dirname(__file__), "golden", "project_4x4.json")) as f:
        g = json.load(f)
    rk, ck = run(np.array(g["W"], np.float32), 2, 2, g["PR"])
    assert rk.tolist() == g["row_keep"] and ck.tolist() == g["col_keep"]
    W = torch.zeros((8, 8), device="cuda")
    with pytest.raises(binding.CsbError) as e:
        binding.csb_project(W, 4, 4, 1.5)
    assert e.value.status == -1
    with pytest.raises(binding.CsbError) as e:
        binding.csb_project(W, 4, 4, 0.5, workspace=torch.empty(8, dtype=torch.uint8, device="cuda"))
    assert e.value.status == -1 and "workspace" in str(e.value)


def test_cfg4_shape_sampled_block_columns():
    # the benchmark's shape; the oracle's loops take a few seconds on it
    rng = np.random.default_rng(0)
    W = (rng.standard_normal((2048, 8192)) * 0.05).astype(np.float32)
    rk, ck = run(W, 64, 64, 0.75)
    wrk, wck, _ = P.project(W, 64, 64, 0.75)
    assert np.array_equal(rk, wrk) and np.array_equal(ck, wck)
