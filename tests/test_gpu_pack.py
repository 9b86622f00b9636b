"""Bit-packed integer weights on the GPU against the oracle's reference packer: byte-exact packed
words, exact round trip, and the fused unpack + dequantize + compare."""
import numpy as np
import pytest

import oracle
from parity_util import make_problem, run_gpu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("shape", [(3, 32), (37, 416), (128, 4096)])
def test_pack_matches_the_reference_packer_and_round_trips(bits, shape):
    import torch
    import paper_2602_04929_b200 as tb
    g = np.random.default_rng(bits * 100 + shape[0])
    codes = g.integers(0, 1 << bits, size=shape).astype(np.uint8)
    d_out, d_in = shape
    ng = d_in // 32
    scales = (0.01 + g.random((d_out, ng))).astype(np.float32)
    zeros = g.integers(0, 1 << bits, size=(d_out, ng)).astype(np.int32)
    cd = torch.from_numpy(codes).cuda()
    packed = tb.tb_pack_codes(cd, bits)
    assert tb.load().tb_packed_bytes(d_out, d_in, bits) == d_out * d_in * bits // 8
    want = oracle.pack_codes(codes, bits)
    assert np.array_equal(packed.cpu().numpy().view(np.uint32), want)
    back, w_hat, mism = tb.tb_unpack_dequant(packed, torch.from_numpy(scales).cuda(), torch.from_numpy(zeros).cuda(),
                                             d_in, bits, 32, codes_ref=cd)
    assert torch.equal(back, cd) and mism.tolist() == [0, 0]
    ref = oracle.dequantize(codes, scales, zeros, 32)
    assert np.array_equal(w_hat.cpu().numpy(), (scales.repeat(32, axis=1) * (codes.astype(np.int32) - zeros.repeat(32, axis=1)).astype(np.float32)))
    assert np.max(np.abs(w_hat.cpu().numpy() - ref)) <= 2.0 ** -23 * np.max(np.abs(ref))
    # a planted difference is found and counted: one code and the value it gives
    bad = cd.clone()
    bad[d_out // 2, 5] ^= 1
    wrong_ref = w_hat.clone()
    wrong_ref[0, 0] += 1.0
    _, _, mism = tb.tb_unpack_dequant(packed, torch.from_numpy(scales).cuda(), torch.from_numpy(zeros).cuda(), d_in,
                                      bits, 32, want_codes=False, want_w_hat=False, codes_ref=bad, w_hat_ref=wrong_ref,
                                      tol=0.0)
    assert mism.tolist() == [1, 1]


@pytest.mark.parametrize("bits,gq", [(2, 128), (3, 0), (4, 64)])
def test_packed_output_of_a_quantized_layer_dequantizes_to_w_hat(bits, gq):
    """The deployment triple (packed codes, float scales, integer zero-points) of a quantized layer gives
    back its W_hat: within one float rounding of the library's own W_hat (formed from the scales in
    double), and within 1e-6 of the oracle's dequantization of the same triple."""
    import torch
    import paper_2602_04929_b200 as tb
    prob = make_problem(50, 256, 2, 64, 1024)
    gpu = run_gpu(prob, bits, gq, 16, 3)
    codes = torch.from_numpy(gpu["codes"]).cuda()
    packed = tb.tb_pack_codes(codes, bits)
    assert packed.numel() * 4 == gpu["codes"].size * bits // 8
    back, w_hat, mism = tb.tb_unpack_dequant(packed, torch.from_numpy(gpu["scales"]).cuda(),
                                             torch.from_numpy(gpu["zeros"]).cuda(), 256, bits, gq, codes_ref=codes,
                                             w_hat_ref=torch.from_numpy(gpu["w_hat"]).cuda(), tol=2.0 ** -22)
    assert mism.tolist() == [0, 0]
    ref = oracle.dequantize(oracle.unpack_codes(packed.cpu().numpy().view(np.uint32), bits, 256), gpu["scales"], gpu["zeros"], gq)
    assert np.linalg.norm(w_hat.cpu().numpy() - ref) <= 1e-6 * np.linalg.norm(ref)


def test_pack_rejects_bad_shapes():
    import paper_2602_04929_b200 as tb
    import ctypes
    lib = tb.load()
    one = ctypes.c_void_p(256)
    assert lib.tb_packed_bytes(4, 48, 3) == 0 and lib.tb_packed_bytes(4, 64, 9) == 0
    assert lib.tb_pack_codes(one, 4, 48, 3, one, None) == 2
    assert lib.tb_pack_codes(one, 4, 64, 1, one, None) == 1
    assert lib.tb_pack_codes(None, 4, 64, 2, one, None) == 1
    assert lib.tb_unpack_dequant(one, one, one, 4, 64, 2, 48, None, None, None, None, 0.0, None, None) == 1
    assert lib.tb_unpack_dequant(one, one, one, 4, 64, 2, 32, None, None, one, None, 0.0, None, None) == 1
