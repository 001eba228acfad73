"""Pins of the oracle's projection step: its single rounding to fp16 / bf16 against the library
conversions, and the product against a library matmul."""
import numpy as np
import torch

from oracle import moqae_oracle as O

RS = np.random.RandomState


def test_round_to_16bit_equals_library_conversion_on_float32_inputs():
    # for inputs that are float32 numbers a single rounding is what torch / numpy do
    rs = RS(1)
    x = np.concatenate([rs.randn(20000) * np.exp(rs.randn(20000) * 3), [0.0, -0.0, 1.0, -1.0, 65504.0, 1e-7, -3e-8]])
    x = x.astype(np.float32)
    got16 = O.round_to_16bit(x.astype(np.float64), 0)
    keep = np.abs(x) < 65504
    assert (got16[keep] == x[keep].astype(np.float16).view(np.uint16)).all()
    gotb = O.round_to_16bit(x.astype(np.float64), 1)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (gotb == want).all()


def test_round_to_16bit_ties_go_to_even_and_is_a_single_rounding():
    # bf16 keeps 8 significant bits: 1 + 2^-8 is exactly halfway between 1 and 1 + 2^-7
    assert O.round_to_16bit(np.array([1.0 + 2.0 ** -8]), 1)[0] == 0x3F80           # down to even
    assert O.round_to_16bit(np.array([1.0 + 3 * 2.0 ** -8]), 1)[0] == 0x3F82       # up to even
    # a float64 just above the tie must go up although float32 would first round it onto the tie
    assert O.round_to_16bit(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]), 1)[0] == 0x3F81
    assert O.round_to_16bit(np.array([1.0 + 2.0 ** -11 + 2.0 ** -40]), 0)[0] == 0x3C01
    assert O.round_to_16bit(np.array([2.0 ** -25]), 0)[0] == 0 and O.round_to_16bit(np.array([3 * 2.0 ** -25]), 0)[0] == 2


def test_project_kv_is_a_matmul_then_one_rounding():
    rs = RS(2)
    B, T, D, H = 2, 37, 96, 2
    hid = rs.randn(B, T, D).astype(np.float16)
    Wk = (rs.randn(H * 128, D) / np.sqrt(D)).astype(np.float16)
    Wv = (rs.randn(H * 128, D) / np.sqrt(D)).astype(np.float16)
    K16, V16, K64, V64 = O.project_kv(hid.view(np.uint16), Wk.view(np.uint16), Wv.view(np.uint16), 0, H)
    ref = torch.from_numpy(hid.astype(np.float64)) @ torch.from_numpy(Wk.astype(np.float64)).T
    assert np.abs(K64.reshape(B, T, -1) - ref.numpy()).max() < 1e-12
    assert K16.shape == (B, T, H, 128)
    back = K16.view(np.float16).astype(np.float64)
    assert (np.abs(back - K64) <= np.abs(K64) * 2.0 ** -11 + 2.0 ** -25).all()      # half an ulp
    # head h of V uses rows 128 h .. 128 h + 127 of Wv
    v_h1 = hid.astype(np.float64)[0, 5] @ Wv.astype(np.float64)[128:256].T
    assert np.abs(V64[0, 5, 1] - v_h1).max() < 1e-12
