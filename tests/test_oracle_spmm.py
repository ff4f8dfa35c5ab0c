"""Pins for the CPU oracle's SpMM and its fp16 conversions (no GPU)."""
import numpy as np
import pytest

from paper_2607_08786_b200 import workloads as wl


def test_half_conversions_match_numpy(oracle_mod):
    # every fp16 bit pattern -> float
    for h in list(range(0, 65536, 7)) + [0x0001, 0x03FF, 0x0400, 0x7BFF, 0x7C00, 0xFC00, 0x8000]:
        want = np.array([h], dtype=np.uint16).view(np.float16).astype(np.float32)[0]
        got = np.float32(oracle_mod.half_to_float(h))
        assert (np.isnan(want) and np.isnan(got)) or want == got, hex(h)
    # float -> half, round to nearest even, including ties, subnormals and overflow
    rng = np.random.default_rng(3)
    samples = np.concatenate([
        rng.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** rng.integers(-8, 5, 4000).astype(np.float32),
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, -1e9, 2.0**-24, 2.0**-25, 2.0**-25 * 1.0001,
                  2.0**-14, 2.0**-14 - 2.0**-25, 1.0 + 2.0**-11, 1.0 + 3 * 2.0**-11, 1.0 + 2.0**-11 + 2.0**-20,
                  0.1, 1 / 3, 2047.5, 2048.5, 2049.5], dtype=np.float32)])
    for f in samples:
        with np.errstate(over="ignore"):
            want = int(np.array([f], dtype=np.float32).astype(np.float16).view(np.uint16)[0])
        assert oracle_mod.float_to_half(float(f)) == want, float(f)


@pytest.mark.parametrize("shape,N,tile", [((4, 8), 3, (4, 8)), ((96, 200), 5, (32, 64)), ((256, 384), 8, (128, 128)),
                                          ((130, 260), 16, (128, 128))])
def test_matches_dense_fp64_on_small_inputs(oracle_mod, shape, N, tile):
    rng = np.random.default_rng(shape[1] + N)
    W = np.where(rng.random(shape) < 0.55, rng.standard_normal(shape).astype(np.float16), np.float16(0))
    X = rng.standard_normal((shape[1], N)).astype(np.float16)
    c = oracle_mod.encode(W, *tile)
    Y = oracle_mod.spmm(c, X).view(np.float16).astype(np.float64)
    Yref, bound = oracle_mod.dense_fp64(W, X)
    # independent of oracle.dense_fp64's blocking: a direct einsum on the decoded matrix
    Wd = oracle_mod.decode(c).view(np.float16).astype(np.float64)
    assert np.allclose(Yref, np.einsum("ik,kj->ij", Wd, X.astype(np.float64)), rtol=1e-12, atol=1e-12)
    assert np.all(np.abs(Y - Yref) <= oracle_mod.tolerance(bound))
    # fp32 accumulation + one fp16 rounding: much tighter than the task tolerance
    assert np.all(np.abs(Y - Yref) <= 2.0**-10 * np.abs(Yref) + 1e-4 * bound + 1e-7)


def test_identity_activation_reproduces_W_exactly(oracle_mod):
    """X = I: every y_ij is a single product w_ij * 1, so Y must equal W bit for bit."""
    case = wl.Case(0, "id", 256, 128, 128, 31, 0.5, "magnitude")
    W = case.make_W()
    c = oracle_mod.encode(W)
    Y = oracle_mod.spmm(c, np.eye(128, dtype=np.float16))
    assert np.array_equal(Y, W.view(np.uint16))


def test_integer_valued_inputs_are_exact(oracle_mod):
    """Small integers: all partial sums are exact in fp32, so Y equals the integer product."""
    rng = np.random.default_rng(9)
    W = np.where(rng.random((128, 256)) < 0.5, rng.integers(-4, 5, (128, 256)), 0).astype(np.float16)
    X = rng.integers(-3, 4, (256, 8)).astype(np.float16)
    c = oracle_mod.encode(W)
    Y = oracle_mod.spmm(c, X).view(np.float16).astype(np.int64)
    assert np.array_equal(Y, W.astype(np.int64) @ X.astype(np.int64))


def test_exact_two_four_matrix_is_a_plain_sparse_gemm(oracle_mod):
    rng = np.random.default_rng(4)
    W = rng.integers(1, 5, (128, 128)).astype(np.float16)
    W[:, 1::4] = 0
    W[:, 2::4] = 0                                         # keeps positions 0 and 3 of every window
    X = rng.integers(-3, 4, (128, 4)).astype(np.float16)
    c = oracle_mod.encode(W)
    assert c.stats["n_sf"] == 0 and c.stats["n_res"] == 0
    vals = c.tc_vals.view(np.float16).reshape(128, 64).astype(np.int64)
    # compressed product: slot 2q ↔ column 4q, slot 2q+1 ↔ column 4q+3
    Xc = np.empty((64, 4), dtype=np.int64)
    Xc[0::2] = X[0::4]
    Xc[1::2] = X[3::4]
    assert np.array_equal(oracle_mod.spmm(c, X).view(np.float16).astype(np.int64), vals @ Xc)


def test_columns_of_X_are_independent(oracle_mod):
    case = wl.Case(0, "cols", 256, 384, 8, 17, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    c = oracle_mod.encode(W)
    Y = oracle_mod.spmm(c, X)
    for j in (0, 5):
        assert np.array_equal(oracle_mod.spmm(c, X[:, j:j + 1].copy())[:, 0], Y[:, j])


def test_tile_shape_does_not_change_Y_beyond_rounding(oracle_mod):
    case = wl.Case(0, "tiles", 256, 512, 4, 23, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    Yref, bound = oracle_mod.dense_fp64(W, X)
    for tile in ((128, 128), (64, 128), (128, 256), (32, 64)):
        Y = oracle_mod.spmm(oracle_mod.encode(W, *tile), X).view(np.float16).astype(np.float64)
        assert np.all(np.abs(Y - Yref) <= oracle_mod.tolerance(bound))


def test_config1_against_dense_fp64(oracle_mod):
    case = next(wl.config_cases(1))
    W, X = case.make_W(), case.make_X()
    c = oracle_mod.encode(W)
    Y = oracle_mod.spmm(c, X).view(np.float16).astype(np.float64)
    Yref, bound = oracle_mod.dense_fp64(W, X)
    assert np.all(np.abs(Y - Yref) <= oracle_mod.tolerance(bound))
