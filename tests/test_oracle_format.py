"""Pins for the CPU oracle's encoder and decoder (no GPU).

The oracle is checked against things other than itself: hand-worked examples (tests/golden),
the table of all 16 window patterns, structural invariants of the format, closed-form layer
shares for an i.i.d. mask, the paper's printed layer shares, and bit-exact round trips.
"""
import json
import os

import numpy as np
import pytest

from paper_2607_08786_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f16(x):
    return np.asarray(x, dtype=np.float16)


def load(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return json.load(f)


def nibbles(c):
    """tc_meta as one nibble per window, shape (M_pad, K_pad/4)."""
    m = c.tc_meta.reshape(c.M_pad, c.K_pad // 8)
    out = np.empty((c.M_pad, c.K_pad // 4), dtype=np.uint8)
    out[:, 0::2] = m & 0xF
    out[:, 1::2] = m >> 4
    return out


@pytest.mark.parametrize("name", ["example_1.json", "example_2.json", "example_3.json"])
def test_worked_examples_encode(oracle_mod, name):
    g = load(name)
    W = f16(g["W"])
    c = oracle_mod.encode(W, g["tile_m"], g["tile_k"])
    assert np.array_equal(c.tc_vals.view(np.float16).reshape(c.M_pad, -1), f16(g["tc_vals"]))
    assert np.array_equal(nibbles(c), np.asarray(g["tc_meta_nibbles"], dtype=np.uint8))
    assert c.chain_tau0.tolist() == g["chain_tau0"]
    assert c.chain_rho0.tolist() == g["chain_rho0"]
    assert c.chain_len.tolist() == g["chain_len"]
    assert c.pdd_bytes.tolist() == g["pdd_bytes"]
    assert c.tile_dir.tolist() == g["tile_dir"]
    assert c.res_rho.tolist() == g["res_rho"]
    assert c.res_val.view(np.float16).tolist() == [float(v) for v in g["res_val"]]


@pytest.mark.parametrize("name", ["example_1.json", "example_2.json", "example_3.json"])
def test_worked_examples_decode_from_hand_built_container(oracle_mod, name):
    """The decoder alone, fed a container typed in by hand (not produced by the encoder)."""
    g = load(name)
    W = f16(g["W"])
    M, K = W.shape
    nib = np.asarray(g["tc_meta_nibbles"], dtype=np.uint8)
    meta = (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)
    c = oracle_mod.Container(
        M, K, g["tile_m"], g["tile_k"], 15,
        tc_vals=f16(g["tc_vals"]).view(np.uint16).ravel(), tc_meta=meta.ravel(),
        chain_tau0=np.asarray(g["chain_tau0"], dtype=np.uint16),
        chain_rho0=np.asarray(g["chain_rho0"], dtype=np.uint16),
        chain_len=np.asarray(g["chain_len"], dtype=np.uint8),
        pdd_bytes=np.asarray(g["pdd_bytes"], dtype=np.uint8),
        tile_dir=np.asarray(g["tile_dir"], dtype=np.uint32),
        res_rho=np.asarray(g["res_rho"], dtype=np.uint16),
        res_val=f16(g["res_val"]).view(np.uint16))
    assert np.array_equal(oracle_mod.decode(c).view(np.float16), W)


def test_all_sixteen_window_patterns(oracle_mod):
    """1 x 8 tiles (second window holds exactly two weights, so it neither offers a hole nor
    adds surplus): every zero/non-zero pattern of a window against the hand-written table."""
    tbl = load("window_table.json")["rows"]
    for row in tbl:
        p = row["pattern"]
        w = f16([[(i + 1) if (p >> i) & 1 else 0 for i in range(4)] + [8, 9, 0, 0]])
        c = oracle_mod.encode(w, 1, 8)
        nib = int(c.tc_meta[0]) & 0xF
        assert [nib & 3, nib >> 2] == row["idx"], p
        vals = c.tc_vals.view(np.float16)
        for s in range(2):
            if row["slot_kept"][s]:
                assert vals[s] == row["idx"][s] + 1, p
            else:
                assert vals[s] == 0, p           # this tile has nowhere to park a surplus weight
        # surplus weights of a 1x4 tile have no empty slot to go to only if the window is full
        n_sur = len(row["surplus"])
        n_empty = 2 - sum(row["slot_kept"])
        assert c.stats["n_sf"] == min(n_sur, n_empty) == 0
        assert c.res_rho.tolist() == [i - 2 for i in row["surplus"]], p
        assert c.res_val.view(np.float16).tolist() == [float(i + 1) for i in row["surplus"]], p
        assert np.array_equal(oracle_mod.decode(c).view(np.float16), w)


def test_legal_metadata_nibbles_only(oracle_mod):
    W = wl.Case(1, "t", 256, 512, 8, 7, 0.5, "bernoulli").make_W()
    c = oracle_mod.encode(W)
    assert set(np.unique(nibbles(c)).tolist()) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}


def pair_lists(c, tile):
    """Replays the PDD chains of one tile -> list of (tau, rho) of real entries, n dummies."""
    tm = c.tile_m
    off = int(c.tile_dir[tile, 0])
    pairs, dummies = [], 0
    for r in range(tm):
        ch = tile * tm + r
        ln = int(c.chain_len[ch])
        if c.chain_tau0[ch] == 0xFFFF and ln == 0:
            continue
        t, rho = int(c.chain_tau0[ch]), int(c.chain_rho0[ch])
        pairs.append((t, rho))
        for b in c.pdd_bytes[off:off + ln]:
            dt, dr = int(b) & 15, int(b) >> 4
            t += dt
            rho += dr
            if dt and dr:
                pairs.append((t, rho))
            else:
                dummies += 1
        off += ln
    assert off == int(c.tile_dir[tile, 0]) + int(c.tile_dir[tile, 1])
    return pairs, dummies


@pytest.mark.parametrize("kind,sparsity", [("bernoulli", 0.5), ("magnitude", 0.4), ("magnitude", 0.5),
                                           ("magnitude", 0.7), ("wanda", 0.5)])
def test_invariants(oracle_mod, kind, sparsity):
    case = wl.Case(0, "inv", 384, 640, 8, 11, sparsity, kind)
    W = case.make_W()
    c = oracle_mod.encode(W)
    s = c.stats
    assert s["nnz"] == int((W != 0).sum()) == s["n_tc"] + s["n_sf"] + s["n_res"]
    H = c.tile_k // 2
    tiles_k = c.K_pad // c.tile_k
    Wp = np.zeros((c.M_pad, c.K_pad), dtype=np.float16)
    Wp[:c.M, :c.K] = W
    nib = nibbles(c)
    vals = c.tc_vals.view(np.float16).reshape(c.M_pad, c.K_pad // 2)
    n_pairs = n_dummy = 0
    for tile in range(c.tile_dir.shape[0]):
        tm_i, tk_i = divmod(tile, tiles_k)
        pairs, d = pair_lists(c, tile)
        n_pairs += len(pairs)
        n_dummy += d
        taus = [p[0] for p in pairs]
        rhos = [p[1] for p in pairs]
        assert all(a < b for a, b in zip(taus, taus[1:]))      # both streams strictly increase
        assert all(a < b for a, b in zip(rhos, rhos[1:]))
        for t, rho in pairs:
            r, sl = divmod(t, H)
            q, s_ = divmod(sl, 2)
            row, gq = tm_i * c.tile_m + r, tk_i * (c.tile_k // 4) + q
            idx = (int(nib[row, gq]) & 3, int(nib[row, gq]) >> 2)[s_]
            assert Wp[row, 4 * gq + idx] == 0                  # tau is a hole of the Sparse-TC layer
            rr, rs = divmod(rho, H)
            col = tk_i * c.tile_k + 4 * (rs // 2) + 2 + (rs & 1)
            v = vals[row, tk_i * H + sl]
            assert v != 0 and v == Wp[tm_i * c.tile_m + rr, col]   # the parked value is the surplus weight
        r0, rn = int(c.tile_dir[tile, 2]), int(c.tile_dir[tile, 3])
        rr = c.res_rho[r0:r0 + rn].astype(int)
        assert np.all(np.diff(rr) > 0)
        for rho, v in zip(rr, c.res_val[r0:r0 + rn].view(np.float16)):
            r_, rs = divmod(int(rho), H)
            assert v == Wp[tm_i * c.tile_m + r_, tk_i * c.tile_k + 4 * (rs // 2) + 2 + (rs & 1)]
    assert n_pairs == s["n_sf"] and n_dummy == s["n_dummy"]
    assert np.array_equal(oracle_mod.decode(c), W.view(np.uint16))


def test_special_matrices(oracle_mod):
    rng = np.random.default_rng(5)
    # exact 2:4: nothing leaves the Sparse-TC layer
    W = (rng.standard_normal((128, 256)) + 3).astype(np.float16)
    keep = np.zeros((128, 64, 4), dtype=bool)
    for i in range(128):
        for q in range(64):
            keep[i, q, rng.choice(4, 2, replace=False)] = True
    W24 = np.where(keep.reshape(128, 256), W, np.float16(0))
    c = oracle_mod.encode(W24)
    assert c.stats["n_sf"] == 0 and c.stats["n_res"] == 0 and c.stats["n_tc"] == 128 * 128
    assert c.pdd_bytes.size == 0 and np.all(c.chain_tau0 == 0xFFFF)
    assert np.array_equal(oracle_mod.decode(c), W24.view(np.uint16))
    # all zero
    Z = np.zeros((128, 128), dtype=np.float16)
    c = oracle_mod.encode(Z)
    assert c.stats["nnz"] == 0 and not c.tc_vals.any() and np.all(nibbles(c) == 4)
    assert np.array_equal(oracle_mod.decode(c), Z.view(np.uint16))
    # fully dense: every window keeps 2 and has 2 surplus, no holes -> half of nnz is Residual
    c = oracle_mod.encode(W)
    assert c.stats["n_tc"] == c.stats["n_res"] == W.size // 2 and c.stats["n_sf"] == 0
    assert np.array_equal(oracle_mod.decode(c), W.view(np.uint16))
    # dense top half / zero bottom half of one tile: every surplus parked in another row,
    # consecutive pairs are (1,1) apart
    T = np.zeros((128, 128), dtype=np.float16)
    T[:64] = W[:64, :128]
    c = oracle_mod.encode(T)
    assert c.stats["n_sf"] == 64 * 64 and c.stats["n_res"] == 0 and c.stats["n_dummy"] == 0
    assert np.all(c.pdd_bytes == 0x11)
    assert np.all(c.chain_len[:64] == 63) and np.all(c.chain_len[64:] == 0)
    assert c.chain_tau0[0] == 64 * 64 and c.chain_rho0[0] == 0
    assert np.array_equal(oracle_mod.decode(c), T.view(np.uint16))


def test_dummy_points_for_long_spans(oracle_mod):
    """One row whose two surplus weights are 40 slots apart and whose holes are 33 apart."""
    W = np.zeros((1, 256), dtype=np.float16)
    W[0, 0:4] = [1, 2, 3, 0]            # surplus at rho = 0
    W[0, 80:84] = [4, 5, 0, 6]          # surplus at rho = 2*20 + 1 = 41
    for q in range(1, 64):               # fill every other window with exactly two weights ...
        if q not in (20, 2, 35):
            W[0, 4 * q:4 * q + 2] = [7, 8]
    # ... so the only holes are windows 2 (tau 4,5) and 35 (tau 70,71)
    W[0, 8:12] = [0, 0, 0, 0]
    W[0, 140:144] = [9, 0, 0, 0]         # window 35: slot 0 kept, slot 1 (tau 71) empty
    c = oracle_mod.encode(W, 1, 256)
    # holes: tau 4, 5, 71 ; surplus rho 0, 41 -> pairs (4,0), (5,41): gaps (1, 41)
    assert c.chain_tau0.tolist() == [4] and c.chain_rho0.tolist() == [0]
    assert c.pdd_bytes.tolist() == [0xF0, 0xF0, 0x11 | (41 - 30 - 1) << 4]
    assert c.stats["n_dummy"] == 2
    assert np.array_equal(oracle_mod.decode(c), W.view(np.uint16))


def test_chain_overflow_goes_to_residual(oracle_mod):
    """A chain may hold at most 255 delta bytes; what does not fit becomes Residual."""
    # tile 2 x 2048 (H = 1024 slots per row): row 0 fully dense -> 1024 surplus in one row,
    # row 1 all zero -> 1024 holes.  Chain 0 takes 1 + 255 pairs, the other 768 go to Residual.
    W = np.zeros((2, 2048), dtype=np.float16)
    W[0] = (np.arange(2048) % 200 + 1).astype(np.float16)
    c = oracle_mod.encode(W, 2, 2048)
    assert c.chain_len.tolist() == [255, 0]
    assert c.stats["n_sf"] == 256 and c.stats["n_res"] == 768
    assert np.array_equal(oracle_mod.decode(c), W.view(np.uint16))


def test_negative_zero_and_specials(oracle_mod):
    W = np.zeros((4, 8), dtype=np.float16)
    W[0, :4] = [-0.0, 1.0, np.inf, np.nan]
    W[1, :4] = [6e-8, -6e-8, 65504, -65504]       # subnormals and extremes are non-zero
    c = oracle_mod.encode(W, 4, 8)
    back = oracle_mod.decode(c)
    expect = W.view(np.uint16).copy()
    expect[0, 0] = 0                                  # -0.0 is a zero and decodes as +0.0
    assert np.array_equal(back, expect)
    assert c.stats["nnz"] == 7


@pytest.mark.parametrize("p", [0.3, 0.5, 0.7])
def test_closed_form_layer_shares_iid_mask(oracle_mod, p):
    """For an i.i.d. Bernoulli(p) mask: E[surplus per window] = 4p^3(1-p) + 2p^4 and
    E[holes per window] = 2(1-p)^4 + 4p(1-p)^3 (binomial counts of a 4-window)."""
    M, K = 512, 2048
    rng = np.random.default_rng(123)
    W = np.where(rng.random((M, K)) < p, np.float16(1.5), np.float16(0))
    c = oracle_mod.encode(W)
    windows = M * K // 4
    surplus = 4 * p**3 * (1 - p) + 2 * p**4
    holes = 2 * (1 - p)**4 + 4 * p * (1 - p)**3
    s = c.stats
    got_surplus = (s["n_sf"] + s["n_res"]) / windows
    got_holes = (s["n_sf"] + s["n_slots_unused"]) / windows
    sd = 1.0 / np.sqrt(windows)                       # per-window variance is < 1
    assert abs(got_surplus - surplus) < 5 * sd
    assert abs(got_holes - holes) < 5 * sd
    assert abs(s["n_tc"] / windows - (4 * p - surplus)) < 5 * sd
    if p == 0.5:
        assert abs(got_surplus / (4 * p) - 0.1875) < 0.002     # 18.75 % of non-zeros


@pytest.mark.parametrize("kind", ["magnitude", "wanda"])
def test_paper_layer_shares_at_half_sparsity(oracle_mod, kind):
    """Sec. 3.2 prints ~17.7 % Slot-Filling, 2.13 % dummy points, < 1 % Residual for pruned LLM
    weights; synthetic 50 % masks must land in a band around that."""
    W = wl.Case(0, "band", 1024, 2048, 8, 21, 0.5, kind).make_W()
    s = oracle_mod.encode(W).stats
    nnz = s["nnz"]
    assert 0.17 <= s["n_sf"] / nnz <= 0.195
    # "typically less than 1 %": holds for the row-wise mask; the column-correlated stand-in for a
    # Wanda mask (outlier channels drawn at random) clusters more and may sit a little above it
    assert s["n_res"] / nnz < (0.01 if kind == "magnitude" else 0.02)
    assert 0.01 <= s["n_dummy"] / nnz <= 0.03
    assert abs(s["n_tc"] / nnz - 0.8125) < 0.01


@pytest.mark.parametrize("shape,tile", [((1, 4), (128, 128)), ((130, 260), (128, 128)), ((64, 128), (64, 128)),
                                        ((257, 131), (128, 256)), ((3, 1000), (32, 64))])
def test_round_trip_ragged_shapes_and_tiles(oracle_mod, shape, tile):
    rng = np.random.default_rng(shape[0] * 1000 + shape[1])
    W = np.where(rng.random(shape) < 0.5, (rng.standard_normal(shape) * 0.02).astype(np.float16), np.float16(0))
    c = oracle_mod.encode(W, *tile)
    assert c.M_pad % tile[0] == 0 and c.K_pad % tile[1] == 0
    assert np.array_equal(oracle_mod.decode(c), W.view(np.uint16))


def test_round_trip_config1(oracle_mod):
    case = next(wl.config_cases(1))
    W = case.make_W()
    c = oracle_mod.encode(W)
    assert np.array_equal(oracle_mod.decode(c), W.view(np.uint16))
    assert 0.62 < c.nbytes() / W.nbytes < 0.64          # ~0.631 x dense at 50 %


def test_rejects_bad_parameters(oracle_mod):
    W = np.zeros((4, 8), dtype=np.float16)
    with pytest.raises(ValueError):
        oracle_mod.encode(W, 4, 12)                     # tile_k not a multiple of 8
    with pytest.raises(ValueError):
        oracle_mod.encode(W, 1024, 256)                 # more than 65535 slots per tile


# ---- compact Residual layer ---------------------------------------------------------------------
def _bare_container(oracle_mod, tile_m, tile_k, tile_dir, res_rho):
    z8, z16 = np.zeros(0, np.uint8), np.zeros(0, np.uint16)
    return oracle_mod.Container(1, 1, tile_m, tile_k, 15, z16, z8, z16, z16, z8, z8, np.asarray(tile_dir, np.uint32).reshape(-1, 4),
                                np.asarray(res_rho, np.uint16), np.zeros(len(res_rho), np.uint16))


def test_compact_residual_golden(oracle_mod):
    import json, os
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "residual_compact.json")))
    c = _bare_container(oracle_mod, g["tile_m"], g["tile_k"], g["tile_dir"], g["res_rho"])
    res_dir, res_list, res_mask = oracle_mod.residual_compact(c)
    assert res_dir.tolist() == g["res_dir"]
    assert res_list.tolist() == g["res_list"]
    assert res_mask.tolist() == g["res_mask"]
    assert oracle_mod.residual_expand(c, res_dir, res_list, res_mask).tolist() == g["res_rho"]


def test_compact_residual_round_trip_and_size_rule(oracle_mod):
    """Brute force on random position sets: expanding the compact form gives the positions back,
    every tile took the smaller of its two codings, and bit b of a bitmap stands for position b."""
    rng = np.random.default_rng(5)
    for tile_m, tile_k in ((128, 128), (4, 32), (1, 8)):
        slots = tile_m * tile_k // 2
        B = (slots + 7) // 8
        counts = [0, 1, B // 2, B // 2 + 1, slots // 3, slots]
        tile_dir, rho = [], []
        for n in counts:
            tile_dir.append([0, 0, len(rho), n])
            rho += sorted(rng.choice(slots, size=n, replace=False).tolist())
        c = _bare_container(oracle_mod, tile_m, tile_k, tile_dir, rho)
        res_dir, res_list, res_mask = oracle_mod.residual_compact(c)
        assert oracle_mod.residual_expand(c, res_dir, res_list, res_mask).tolist() == rho
        for t, n in enumerate(counts):
            assert int(res_dir[t, 0]) == (1 if B < 2 * n else 0)
        assert len(res_list) == sum(n for n in counts if not B < 2 * n)
        assert len(res_mask) == B * sum(1 for n in counts if B < 2 * n)
        # the full tile: every bit of its bitmap is set
        t = len(counts) - 1
        if res_dir[t, 0] == 1:
            m = res_mask[int(res_dir[t, 1]):int(res_dir[t, 1]) + B]
            assert int(np.unpackbits(m, bitorder="little")[:slots].sum()) == slots


def test_compact_residual_shrinks_a_40_percent_matrix(oracle_mod):
    """At 40 % sparsity a sixth of the non-zeros lands in the Residual layer (no tile can hold more
    than half of its weights in value slots): the compact form must bring the container from about
    0.81 to under 0.78 of the dense size, and leave a 50 % matrix as it is."""
    from paper_2607_08786_b200 import workloads as wl
    case = wl.Case(0, "s40", 512, 1024, 8, 3, 0.4, "magnitude")
    c = oracle_mod.encode(case.make_W())
    dense = 2 * case.M * case.K
    assert 0.15 < c.stats["n_res"] / c.stats["nnz"] < 0.18
    assert c.nbytes() / dense > 0.80 and oracle_mod.compact_nbytes(c) / dense < 0.78
    assert np.array_equal(oracle_mod.residual_expand(c, *oracle_mod.residual_compact(c)), c.res_rho)
    c50 = oracle_mod.encode(wl.Case(0, "s50", 512, 1024, 8, 3, 0.5, "magnitude").make_W())
    assert abs(oracle_mod.compact_nbytes(c50) - c50.nbytes()) <= 8 * c50.tile_dir.shape[0]


def _values_container(oracle_mod, M, K, tile_m, tile_k, tc_vals):
    """A container of which only the value array matters."""
    z16, z8 = np.zeros(0, np.uint16), np.zeros(0, np.uint8)
    return oracle_mod.Container(M, K, tile_m, tile_k, 15, np.asarray(tc_vals, np.uint16).reshape(-1), z8, z16, z16, z8, z8,
                                np.zeros((0, 4), np.uint32), z16, z16)


def test_compact_values_golden(oracle_mod):
    import json, os
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "values_compact.json")))
    c = _values_container(oracle_mod, g["M"], g["K"], g["tile_m"], g["tile_k"], g["tc_vals"])
    val_dir, val_pack, val_mask = oracle_mod.values_compact(c)
    assert val_dir.tolist() == g["val_dir"]
    assert val_pack.tolist() == g["val_pack"]
    assert val_mask.tolist() == g["val_mask"]
    assert oracle_mod.values_expand(c, val_dir, val_pack, val_mask).tolist() == np.asarray(g["tc_vals"]).reshape(-1).tolist()


def test_compact_values_round_trip_and_size_rule(oracle_mod):
    """Brute force on random occupancies, tile by tile: the expansion gives every value back in its
    slot, a tile took the bitmap exactly when that is smaller, bit b of a bitmap stands for slot b,
    and the packed values of a tile follow the previous tile's."""
    rng = np.random.default_rng(11)
    for tile_m, tile_k, tiles_m, tiles_k in ((128, 128, 1, 3), (4, 32, 3, 2), (1, 8, 2, 5)):
        H = tile_k // 2
        S = tile_m * H
        B = (S + 7) // 8
        M, K = tile_m * tiles_m, tile_k * tiles_k
        vals = np.zeros((M, K // 2), dtype=np.uint16)
        occ = []
        for t in range(tiles_m * tiles_k):
            n = [0, S, S - B // 2, S - B // 2 - 1, S // 3, S - 1][t % 6]
            n = max(0, min(S, n))
            tile = np.zeros(S, dtype=np.uint16)
            at = np.sort(rng.choice(S, size=n, replace=False))
            tile[at] = rng.integers(1, 0x7C00, size=n).astype(np.uint16) | (rng.integers(0, 2, size=n).astype(np.uint16) << 15)
            tm, tk = divmod(t, tiles_k)
            vals[tm * tile_m:(tm + 1) * tile_m, tk * H:(tk + 1) * H] = tile.reshape(tile_m, H)
            occ.append(at)
        c = _values_container(oracle_mod, M, K, tile_m, tile_k, vals)
        val_dir, val_pack, val_mask = oracle_mod.values_compact(c)
        assert np.array_equal(oracle_mod.values_expand(c, val_dir, val_pack, val_mask), vals.reshape(-1))
        # a slot that holds -0.0 is a bit pattern to keep: the form is lossless for every container
        v2 = vals.copy()
        v2[0, 0] = 0x8000
        c2 = _values_container(oracle_mod, M, K, tile_m, tile_k, v2)
        assert np.array_equal(oracle_mod.values_expand(c2, *oracle_mod.values_compact(c2)), v2.reshape(-1))
        at_pack = at_mask = 0
        for t, at in enumerate(occ):
            bitmap = B < 2 * (S - len(at))
            assert val_dir[t].tolist() == [1 if bitmap else 0, at_pack]
            if bitmap:
                bits = np.unpackbits(val_mask[at_mask:at_mask + B], bitorder="little")[:S]
                assert np.flatnonzero(bits).tolist() == at.tolist()
                at_mask += B
                at_pack += len(at)
            else:
                at_pack += S
        assert len(val_pack) == at_pack and len(val_mask) == at_mask


def test_compact_values_shrink_matrices_above_50_percent(oracle_mod):
    """At 60 / 70 % sparsity a fifth / two fifths of the value slots stay empty: with the value array
    in its compact form the container must fall from about 0.61 / 0.59 of the dense size to under
    0.56 / 0.45, the round trip must be exact on an encoder's output, and a 50 % matrix (no tile with
    more than a few empty slots) must keep its size up to the directory."""
    from paper_2607_08786_b200 import workloads as wl
    for sparsity, before, after in ((0.6, 0.60, 0.56), (0.7, 0.58, 0.45)):
        case = wl.Case(0, "hc", 512, 1024, 8, 4, sparsity, "magnitude")
        c = oracle_mod.encode(case.make_W())
        dense = 2 * case.M * case.K
        assert c.nbytes() / dense > before and oracle_mod.compact_nbytes_all(c) / dense < after
        assert abs(c.stats["n_slots_unused"] / (case.M * case.K / 2) - (2 * sparsity - 1)) < 0.02
        assert np.array_equal(oracle_mod.values_expand(c, *oracle_mod.values_compact(c)), np.asarray(c.tc_vals, np.uint16).reshape(-1))
    c50 = oracle_mod.encode(wl.Case(0, "s50", 512, 1024, 8, 3, 0.5, "magnitude").make_W())
    assert 0 <= oracle_mod.compact_nbytes_all(c50) - oracle_mod.compact_nbytes(c50) <= 8 * c50.tile_dir.shape[0]
