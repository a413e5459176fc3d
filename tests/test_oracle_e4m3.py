"""Pins for the 8-bit (E4M3) index-key functions of the oracle."""
import numpy as np
import pytest
import torch

from oracle import rtp_oracle as orc


def _torch_decode(codes: np.ndarray) -> np.ndarray:
    return torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def _torch_encode(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()


def test_decode_every_code_against_the_library_type():
    codes = np.arange(256, dtype=np.uint8)
    got, want = orc.e4m3_decode(codes), _torch_decode(codes)
    assert np.array_equal(np.isnan(got), np.isnan(want)) and int(np.isnan(got).sum()) == 2
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])
    assert np.array_equal(np.signbit(got[ok]), np.signbit(want[ok]))
    assert got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x08] == 2.0 ** -6 and got[0x38] == 1.0


def test_encode_against_the_library_type_below_saturation():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000) * 3.0, rng.standard_normal(20000) * 100.0,
                        rng.standard_normal(20000) * 0.01, np.linspace(-464.0, 464.0, 20001)])
    x = x[np.abs(x) <= 464.0].astype(np.float32)          # the library type has no saturation beyond this point
    assert np.array_equal(orc.e4m3_encode(x), _torch_encode(x))


def test_round_trip_ties_saturation_and_order():
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    vals = orc.e4m3_decode(codes)
    assert np.array_equal(orc.e4m3_encode(vals), codes)                    # every finite code is a fixed point
    pos = orc.e4m3_decode(np.arange(0, 127, dtype=np.uint8))
    mid = (pos[:-1] + pos[1:]) / 2.0                                        # exact midpoints: ties
    enc = orc.e4m3_encode(mid)
    assert np.all(enc % 2 == 0) and np.all((enc == np.arange(0, 126)) | (enc == np.arange(1, 127)))
    assert np.array_equal(orc.e4m3_encode(np.nextafter(mid, np.inf)), np.arange(1, 127))
    assert np.array_equal(orc.e4m3_encode(np.nextafter(mid, -np.inf)), np.arange(0, 126))
    assert orc.e4m3_encode(np.array([449.0, 1e9, -1e9, 464.1])).tolist() == [0x7E, 0x7E, 0xFE, 0x7E]
    assert orc.e4m3_encode(np.array([0.0, -0.0, -1e-12, 1e-12])).tolist() == [0x00, 0x80, 0x80, 0x00]
    x = np.sort(np.random.default_rng(2).standard_normal(5000) * 50.0)
    assert np.all(np.diff(orc.e4m3_decode(orc.e4m3_encode(x))) >= 0)       # monotone
    rel = np.abs(orc.e4m3_decode(orc.e4m3_encode(x)) - x)
    assert np.all(rel <= np.maximum(np.abs(x) * 2.0 ** -4, 2.0 ** -10))    # half a step of a 3-bit mantissa


def test_scores_on_exactly_representable_inputs_equal_the_bf16_scores():
    # keys whose projections are E4M3 values: the 8-bit cache loses nothing and both score routines agree
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 127, size=(200, 16)).astype(np.uint8) | (rng.integers(0, 2, size=(200, 16)).astype(np.uint8) << 7)
    k = orc.e4m3_decode(codes)
    k_bf16 = orc.f32_to_bf16(k.astype(np.float32))
    assert np.array_equal(orc.bf16_to_f64(k_bf16), k)                        # 3 mantissa bits fit into bf16
    qt = orc.f32_to_bf16(rng.standard_normal(16).astype(np.float32))
    assert np.array_equal(orc.index_scores_e4m3(qt, codes, 0.37), orc.index_scores(qt, k_bf16, 0.37))


def test_projection_is_the_encoded_fp32_projection():
    rng = np.random.default_rng(4)
    x = orc.f32_to_bf16(rng.standard_normal((50, 128)).astype(np.float32))
    w = orc.f32_to_bf16((rng.standard_normal((128, 16)) / np.sqrt(128)).astype(np.float32))
    got = orc.index_project_e4m3(x, w)
    y = orc.bf16_to_f64(x) @ orc.bf16_to_f64(w)
    assert got.shape == (50, 16) and got.dtype == np.uint8
    err = np.abs(orc.e4m3_decode(got) - y)
    assert np.all(err <= np.maximum(np.abs(y) * 2.0 ** -4, 2.0 ** -10) * (1 + 1e-6))
    # against the bf16 projection: the same value before rounding, so the two caches agree to the coarser step
    yb = orc.bf16_to_f64(orc.index_project(x, w))
    assert np.all(np.abs(orc.e4m3_decode(got) - yb) <= np.maximum(np.abs(y) * (2.0 ** -4 + 2.0 ** -8), 2.0 ** -9))


def test_scores_by_hand_on_a_tiny_case():
    # one query, three keys, written out term by term with exact binary fractions
    q = orc.f32_to_bf16(np.array([1.0, -0.5, 2.0, 0.25] + [0.0] * 12, dtype=np.float32))
    keys = np.zeros((3, 16), dtype=np.float64)
    keys[0, :4] = [1.0, 1.0, 1.0, 1.0]          # 1 - 0.5 + 2 + 0.25 = 2.75
    keys[1, :4] = [448.0, 0.0, -448.0, 0.0]     # 448 - 896 = -448
    keys[2, :4] = [2.0 ** -9, 0.0, 0.0, 2.0 ** -6]   # subnormal and smallest normal: 2^-9 + 2^-8
    codes = orc.e4m3_encode(keys)
    assert np.array_equal(orc.e4m3_decode(codes), keys)
    got = orc.index_scores_e4m3(q, codes, 0.5)
    assert got.dtype == np.float32
    assert got.tolist() == [1.375, -224.0, 0.5 * (2.0 ** -9 + 2.0 ** -8)]
