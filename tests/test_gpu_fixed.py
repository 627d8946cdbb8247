"""Parity of the 16-bit fixed-point CSB product (CUDA, through the C ABI) with the integer oracle:
integer work, so every accumulator must match exactly."""
import numpy as np
import pytest
import torch

import workloads
from oracle import fixed_oracle as F
from paper_2005_05758_b200 import binding

pytestmark = pytest.mark.gpu


def run(mat, X, fw, fx):
    A = binding.csb_encode_q16(mat.dense, mat.block_r, mat.block_c, mat.row_keep, mat.col_keep, fw, 0)
    Xq = F.quantize(X, fx)
    xd = torch.from_numpy(Xq.astype(np.int16)).cuda()
    outs = []
    for _ in range(2):
        acc = torch.full((X.shape[0], mat.rows), -7, dtype=torch.int64, device="cuda")
        binding.csb_spmm_q16(A, xd, acc)
        torch.cuda.synchronize()
        outs.append(acc.cpu().numpy())
    view = A.view()
    A.free()
    want = F.spmm_q16(mat.dense, mat.block_r, mat.block_c, mat.row_keep, mat.col_keep, fw, Xq)
    assert np.array_equal(outs[0], want) and np.array_equal(outs[1], want)
    assert view["val_dtype"] == "q16"
    assert np.array_equal(view["val"], F.encode_values(mat.dense, mat.block_r, mat.block_c, mat.row_keep, mat.col_keep, fw))
    return want


@pytest.mark.parametrize("shape", [(4, 4, 2, 2, 1), (64, 64, 16, 16, 1), (50, 39, 16, 8, 3), (300, 1177, 32, 32, 1), (1024, 768, 64, 64, 8),
                                   (257, 513, 128, 128, 5), (96, 4096, 32, 128, 2)])
def test_random_masks_exact(shape):
    R, C, br, bc, B = shape
    rng = np.random.default_rng(R + 7 * C + B)
    nblk = -(-R // br) * -(-C // bc)
    mat = workloads.MatrixSpec((rng.standard_normal((R, C)) * 0.1).astype(np.float32), br, bc, (rng.random(nblk * br) < 0.45).astype(np.uint8),
                               (rng.random(nblk * bc) < 0.35).astype(np.uint8), "f16")
    run(mat, rng.standard_normal((B, C)).astype(np.float32), 16, 12)


def test_saturating_values_and_full_range_inputs():
    rng = np.random.default_rng(3)
    R, C = 128, 256
    mat = workloads.MatrixSpec((rng.standard_normal((R, C)) * 4.0).astype(np.float32), 64, 64, np.ones(2 * 4 * 64, np.uint8), np.ones(2 * 4 * 64, np.uint8), "f16")
    mat.dense[0, :] = 1e9                      # saturates to 32767
    mat.dense[1, :] = -1e9                     # saturates to -32768
    X = np.full((2, C), -1e9, np.float32)      # every input -32768: the largest products there are
    want = run(mat, X, 13, 0)
    assert want[0, 1] == 256 * 32768 * 32768 and want[0, 0] == -256 * 32767 * 32768


def test_cfg4_full_size_exact_and_close_to_the_float_product():
    w = workloads.CONFIGS["cfg4"](rate=8.0, B=4)
    m = w.matrix
    fw, fx = 16, 12                            # |w| < 0.5 and |x| < 8 fit without saturating
    assert np.abs(m.dense).max() < 0.5 and np.abs(w.X).max() < 8
    acc = run(m, w.X, fw, fx)
    from oracle import csb_oracle as O
    want = O.spmm(m.dense, 64, 64, m.row_keep, m.col_keep, "f32", w.X)
    err = np.abs(F.dequantize(acc, fw + fx) - want)
    assert err.max() < 5e-3                    # about a thousand terms per output, each off by at most |w| 2^-13 + |x| 2^-17


def test_refusals():
    W = np.ones((8, 8), np.float32)
    ones = np.ones(16, np.uint8)
    with pytest.raises(binding.CsbError) as e:
        binding.csb_encode(W, 4, 4, ones, ones, 2, 0)                       # CSB_Q16 needs csb_encode_q16
    assert e.value.status == -3
    with pytest.raises(binding.CsbError) as e:
        binding.csb_encode_q16(W, 4, 4, ones, ones, 31, 0)
    assert e.value.status == -1
    A = binding.csb_encode_q16(W, 4, 4, ones, ones, 8, 0)
    x = torch.ones(8, device="cuda")
    y = torch.empty(8, device="cuda")
    with pytest.raises(binding.CsbError) as e:
        binding.csb_spmv(A, x, y)
    assert e.value.status == -8
    with pytest.raises(binding.CsbError) as e:
        binding.csb_lstm_forward([A], None, torch.zeros(1, 1, 6, device="cuda"), None, None, None, None, None)
    assert e.value.status == -8
    B = binding.csb_encode(W, 4, 4, ones, ones, "f16", 0)
    with pytest.raises(binding.CsbError) as e:
        binding.csb_spmm_q16(B, torch.ones(1, 8, dtype=torch.int16, device="cuda"), torch.zeros(1, 8, dtype=torch.int64, device="cuda"))
    assert e.value.status == -8
    A.free()
    B.free()
