"""Pins for the deployment-matched weight-side options of the oracle (App. E.5): one FP32 scale per
128 x 128 tile of each encoded weight combination, and the bf16 rounding of that combination."""
import numpy as np
import torch

from oracle import oracle as O
from oracle import realizations as R


def _strassen():
    return [np.array(R.to_float(x), np.float32) for x in R.strassen()]


def test_bf16_round_matches_torch_and_ties_go_to_even():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4000).astype(np.float32) * 10.0 ** rng.integers(-20, 20, 4000),
                        np.array([0.0, -0.0, 1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 3.3895314e38], np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = O.bf16_round(x)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # exact ties: 1 + 2^-8 lies halfway between 1 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert O.bf16_round(np.float32(1.0 + 2.0 ** -8))[0] == 1.0
    assert O.bf16_round(np.float32(1.0 + 3 * 2.0 ** -8))[0] == np.float32(1.0 + 2.0 ** -6)


def test_tile_quantizer_scale_is_the_maximum_of_the_column_scales():
    # a tile's amax is the maximum of its columns' amaxes, and amax -> amax/448 is monotone, so the tile scale
    # equals the largest per-column scale of the 1 x blk grouping; every column of the tile carries it
    rng = np.random.default_rng(1)
    X = (rng.standard_normal((256, 384)) * np.exp(rng.standard_normal((1, 384)))).astype(np.float32)
    _, s_col, _ = O.quant_cols(X, 128)
    codes, s_tile = O.quant_tiles(X, 128, 128)
    want = s_col.reshape(2, 3, 128).max(axis=2)
    assert np.array_equal(s_tile.reshape(2, 3, 128), np.broadcast_to(want[:, :, None], (2, 3, 128)))
    # where a column's own scale already equals the tile scale, its codes are those of the column quantizer
    c_col, _, _ = O.quant_cols(X, 128)
    same = (s_col == s_tile)
    assert same.any() and not same.all()
    mask = np.repeat(same, 128, axis=0)
    assert np.array_equal(codes[mask], c_col[mask])


def test_tile_quantizer_brute_force_on_one_tile():
    rng = np.random.default_rng(2)
    X = rng.standard_normal((128, 128)).astype(np.float32) * np.float32(3.0)
    codes, s = O.quant_tiles(X, 128, 128)
    amax = np.float32(np.abs(X).max())
    assert np.all(s == np.float32(amax / np.float32(448.0)))
    inv = np.float32(np.float32(448.0) / amax)
    y = (X * inv).astype(np.float32)
    want = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(codes, want)
    # the element holding the maximum maps to +-448 (code 0x7e / 0xfe)
    i, j = np.unravel_index(np.abs(X).argmax(), X.shape)
    assert codes[i, j] & 0x7f == 0x7e


def test_homogeneous_tiles_give_nearly_the_column_quantizer_error_and_heterogeneous_ones_more():
    # App. E.5: on iid Gaussian operands the two groupings are nearly the same quantizer.  e4m3 keeps its
    # relative precision over ~15 binades, so only columns far below their tile's maximum lose accuracy:
    # with column magnitudes spread by exp(4 g) the typical (median) column error rises sharply.
    rng = np.random.default_rng(3)
    U, V, W = _strassen()
    A = rng.standard_normal((256, 256)).astype(np.float32)
    for sigma in (0.0, 4.0):
        B = rng.standard_normal((256, 256)).astype(np.float32)
        B *= np.exp(sigma * rng.standard_normal((1, 256))).astype(np.float32)
        ref = O.ref_gemm(A, B)
        c_col = O.fused_fmm(A, B, U, V, W, levels=1, blk=128)
        c_tile = O.fused_fmm(A, B, U, V, W, levels=1, blk=128, b_tile=128)
        e_col, e_tile = O.rel_frobenius(c_col, ref), O.rel_frobenius(c_tile, ref)
        per_col = lambda X: np.median(np.linalg.norm(X - ref, axis=0) / np.linalg.norm(ref, axis=0))
        if sigma == 0.0:
            assert abs(e_tile / e_col - 1.0) < 0.05
            assert abs(per_col(c_tile) / per_col(c_col) - 1.0) < 0.05
        else:
            assert e_tile > e_col
            assert per_col(c_tile) > 2.0 * per_col(c_col)


def test_bf16_preround_is_a_no_op_on_bf16_representable_weights_and_small_otherwise():
    rng = np.random.default_rng(4)
    A = rng.standard_normal((128, 256)).astype(np.float32)
    B = rng.standard_normal((256, 128)).astype(np.float32)
    Bb = O.bf16_round(B)
    # cubic product: the encoded weight is the weight itself
    c0 = O.fused_fmm(A, Bb, levels=0, blk=128, b_tile=128)
    c1 = O.fused_fmm(A, Bb, levels=0, blk=128, b_tile=128, b_bf16=True)
    assert np.array_equal(c0, c1)
    c2 = O.fused_fmm(A, B, levels=0, blk=128, b_tile=128, b_bf16=True)
    assert np.array_equal(c2, O.fused_fmm(A, Bb, levels=0, blk=128, b_tile=128))
    # encode() exposes the same leaf operands that fused_fmm multiplies
    U, V, W = _strassen()
    B2 = rng.standard_normal((256, 256)).astype(np.float32)
    codes, scales, _ = O.encode(B2, "B", U, V, 1, blk=128, b_tile=128, b_bf16=True)
    T3 = O.bf16_round(B2[:128, 128:] - B2[128:, 128:])        # Strassen's third weight combination B12 - B22
    want_c, want_s = O.quant_tiles(T3, 128, 128)
    assert np.array_equal(codes[2], want_c) and np.array_equal(scales[2], want_s)
