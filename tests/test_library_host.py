"""Host side of the C-ABI library (no GPU): symbols, encoder parity with the oracle, decoder,
persistence, device packing and error codes."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2607_08786_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tl3():
    from paper_2607_08786_b200 import build, tl3 as mod
    build.build_library()
    return mod


def test_library_exports_every_declared_symbol(tl3):
    header = open(os.path.join(ROOT, "include", "tl3.h")).read()
    declared = sorted(set(re.findall(r"\b(tl3_[a-z_0-9]+)\s*\(", header)))
    assert declared, "no declarations found"
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2607_08786_b200", "libtl3.so"))
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in tl3.h but not exported"
    assert sorted(tl3.SYMBOLS) == declared


CASES = [
    wl.Case(0, "bern", 256, 384, 8, 1, 0.5, "bernoulli"),
    wl.Case(0, "mag40", 300, 520, 8, 2, 0.4, "magnitude"),
    wl.Case(0, "mag50", 1024, 1024, 8, 3, 0.5, "magnitude"),
    wl.Case(0, "mag70", 129, 1000, 8, 4, 0.7, "magnitude"),
    wl.Case(0, "wanda", 512, 768, 8, 5, 0.5, "wanda"),
    wl.Case(0, "rows", 384, 256, 8, 6, 0.5, "row_scaled"),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: c.name)
def test_encoder_is_byte_identical_to_the_oracle(tl3, oracle_mod, case):
    W = case.make_W()
    m = tl3.encode(W)
    c = oracle_mod.encode(W)
    for name in tl3.CANONICAL:
        got, want = m.canonical(name), getattr(c, name).ravel()
        assert got.dtype == want.dtype and np.array_equal(got, want), name
    st = m.stats()
    for k, v in c.stats.items():
        assert st[k] == v, k
    assert st["canonical_bytes"] == c.nbytes()
    assert np.array_equal(m.decode(), W.view(np.uint16))
    assert np.array_equal(oracle_mod.decode(c), m.decode())


@pytest.mark.parametrize("tile", [(64, 128), (128, 256), (32, 64), (2, 2048)])
def test_other_tile_shapes_match_the_oracle(tl3, oracle_mod, tile):
    rng = np.random.default_rng(tile[0])
    W = np.where(rng.random((130, 2100)) < 0.55, rng.standard_normal((130, 2100)).astype(np.float16), np.float16(0))
    m = tl3.encode(W, tile_m=tile[0], tile_k=tile[1])
    c = oracle_mod.encode(W, *tile)
    for name in tl3.CANONICAL:
        assert np.array_equal(m.canonical(name), getattr(c, name).ravel()), name
    assert np.array_equal(m.decode(), W.view(np.uint16))


def test_golden_examples_through_the_library(tl3):
    import json
    for i in (1, 2, 3):
        g = json.load(open(os.path.join(ROOT, "tests", "golden", f"example_{i}.json")))
        W = np.asarray(g["W"], dtype=np.float16)
        m = tl3.encode(W, tile_m=g["tile_m"], tile_k=g["tile_k"])
        assert m.canonical("pdd_bytes").tolist() == g["pdd_bytes"]
        assert m.canonical("chain_tau0").tolist() == g["chain_tau0"]
        assert m.canonical("chain_rho0").tolist() == g["chain_rho0"]
        assert m.canonical("res_rho").tolist() == g["res_rho"]
        assert np.array_equal(m.canonical("tc_vals").view(np.float16), np.asarray(g["tc_vals"], dtype=np.float16).ravel())
        assert np.array_equal(m.decode().view(np.float16), W)


def test_serialize_round_trip_is_bit_exact(tl3):
    W = CASES[1].make_W()
    m = tl3.encode(W)
    blob = m.serialize()
    m2 = tl3.Matrix.deserialize(blob)
    assert m2.serialize() == blob
    for name in tl3.CANONICAL:
        assert np.array_equal(m.canonical(name), m2.canonical(name))
    assert m2.stats() == m.stats()
    assert np.array_equal(m2.decode(), W.view(np.uint16))


def test_corrupted_containers_are_rejected(tl3):
    W = CASES[0].make_W()
    blob = bytearray(tl3.encode(W).serialize())
    with pytest.raises(tl3.Tl3Error) as e:
        tl3.Matrix.deserialize(bytes(blob[:100]))                 # truncated
    assert e.value.code == tl3.ERR_BAD_CONTAINER
    bad = bytearray(blob)
    bad[0] ^= 0xFF                                                # wrong magic
    with pytest.raises(tl3.Tl3Error):
        tl3.Matrix.deserialize(bytes(bad))
    bad = bytearray(blob)
    bad[8:16] = (10**12).to_bytes(8, "little")                   # absurd M
    with pytest.raises(tl3.Tl3Error):
        tl3.Matrix.deserialize(bytes(bad))
    with pytest.raises(tl3.Tl3Error):
        tl3.Matrix.deserialize(bytes(blob) + b"\0" * 8)           # trailing bytes
    # a residual position outside the tile
    m = tl3.encode(np.full((128, 128), 1.0, dtype=np.float16))    # dense: half of it is Residual
    blob = bytearray(m.serialize())
    rho = m.canonical("res_rho")
    assert rho.size == 128 * 64
    needle = rho.tobytes()
    at = bytes(blob).rfind(needle)
    assert at > 0
    blob[at:at + 2] = (0xFFFF).to_bytes(2, "little")
    with pytest.raises(tl3.Tl3Error):
        tl3.Matrix.deserialize(bytes(blob))
    # a chain that runs out of its tile: a start beyond the last slot, and a delta byte that pushes it over
    m = tl3.encode(CASES[0].make_W())
    good = bytes(m.serialize())
    tau0 = m.canonical("chain_tau0")
    at = good.find(tau0.tobytes())
    assert at > 0 and tau0[0] != 0xFFFF
    bad = bytearray(good)
    bad[at:at + 2] = (8192).to_bytes(2, "little")
    with pytest.raises(tl3.Tl3Error) as e:
        tl3.Matrix.deserialize(bytes(bad))
    assert e.value.code == tl3.ERR_BAD_CONTAINER
    pdd = m.canonical("pdd_bytes")
    at = good.find(pdd.tobytes())
    assert at > 0
    bad = bytearray(good)
    last_chain = int(np.flatnonzero(m.canonical("chain_len"))[-1])          # a chain near the end of a tile
    bad[at:at + pdd.size] = b"\xFF" * pdd.size                              # every delta 15 + 15
    with pytest.raises(tl3.Tl3Error):
        tl3.Matrix.deserialize(bytes(bad))
    assert last_chain >= 0


def test_error_codes(tl3):
    L = tl3.lib()
    h = ctypes.c_void_p()
    W = np.zeros((4, 8), dtype=np.uint16)
    assert L.tl3_encode(None, 4, 8, None, ctypes.byref(h)) == tl3.ERR_INVALID_ARG
    assert L.tl3_encode(W.ctypes.data, 0, 8, None, ctypes.byref(h)) == tl3.ERR_INVALID_ARG
    p = tl3.Params(4, 12, 15)
    assert L.tl3_encode(W.ctypes.data, 4, 8, ctypes.byref(p), ctypes.byref(h)) == tl3.ERR_INVALID_ARG
    p = tl3.Params(1024, 256, 15)
    assert L.tl3_encode(W.ctypes.data, 4, 8, ctypes.byref(p), ctypes.byref(h)) == tl3.ERR_INVALID_ARG
    assert L.tl3_decode(None, None) == tl3.ERR_INVALID_ARG
    m = tl3.encode(np.zeros((8, 16), dtype=np.float16), tile_m=8, tile_k=16)
    # kernels exist for the 128 x 128 tile only; spmm before upload is refused
    assert L.tl3_pack(m._h, W.ctypes.data, 1 << 20) == tl3.ERR_UNSUPPORTED
    assert L.tl3_spmm(m._h, 16, 8, 16, 8, 8, 256, None) == tl3.ERR_NOT_UPLOADED
    assert L.tl3_spmm(None, None, 8, None, 8, 8, None, None) == tl3.ERR_INVALID_ARG
    assert L.tl3_workspace_bytes(m._h, 4097) == 0 and L.tl3_workspace_bytes(m._h, 0) == 0
    # argument checks of the entry points that need a device come before any CUDA call
    hd = ctypes.c_void_p()
    assert L.tl3_encode_device(None, 8, 8, 8, None, ctypes.byref(hd)) == tl3.ERR_INVALID_ARG
    assert L.tl3_encode_device(256, 8, 16, 8, None, ctypes.byref(hd)) == tl3.ERR_INVALID_ARG      # ldw < K
    assert L.tl3_bind(None, 256) == tl3.ERR_INVALID_ARG
    assert L.tl3_bind(m._h, 256) == tl3.ERR_UNSUPPORTED                                            # 8 x 16 tiles
    m128 = tl3.encode(np.zeros((8, 16), dtype=np.float16))
    assert L.tl3_bind(m128._h, 260) == tl3.ERR_INVALID_ARG                                         # not 256-byte aligned
    assert b"invalid" in L.tl3_strerror(tl3.ERR_INVALID_ARG)
    assert L.tl3_strerror(-99) == b"unknown error"


@pytest.mark.parametrize("sparsity", [0.3, 0.4, 0.5])
def test_compact_residual_matches_the_oracle(tl3, oracle_mod, sparsity):
    """The library's compact form of the Residual layer (list or bitmap per tile) byte for byte
    against the oracle's, and the sizes tl3_stats reports against the arrays themselves."""
    W = wl.Case(0, "cr", 300, 520, 8, 12, sparsity, "magnitude").make_W()
    m = tl3.encode(W)
    cont = oracle_mod.encode(W)
    res_dir, res_list, res_mask = oracle_mod.residual_compact(cont)
    assert np.array_equal(m.canonical("res_dir").reshape(-1, 2), res_dir)
    assert np.array_equal(m.canonical("res_list"), res_list)
    assert np.array_equal(m.canonical("res_mask"), res_mask)
    st = m.stats()
    assert st["canonical_bytes"] == cont.nbytes()
    assert st["canonical_bytes_compact"] == oracle_mod.compact_nbytes(cont)
    if sparsity < 0.5:
        assert (res_dir[:, 0] == 1).any()
    # the device image's own layer counts add up to the surplus elements of the matrix; its
    # Residual list also takes what the three code words of a chain cannot hold
    assert st["dev_n_sf"] + st["dev_n_res"] == st["n_sf"] + st["n_res"]
    assert st["dev_n_res"] >= st["n_res"] and 0 <= st["dev_n_dummy"] <= st["dev_pdd_bytes"]


@pytest.mark.parametrize("sparsity,tiles", [(0.5, (128, 128)), (0.6, (128, 128)), (0.7, (128, 128)), (0.7, (4, 32))])
def test_compact_values_match_the_oracle(tl3, oracle_mod, sparsity, tiles):
    """The library's compact form of the Sparse-TC value array (all values, or a bitmap of the
    occupied slots and their values, per tile) byte for byte against the oracle's, on a ragged
    shape, and the size tl3_stats reports against the oracle's."""
    W = wl.Case(0, "cv", 300, 520, 8, 21, sparsity, "magnitude").make_W()
    m = tl3.encode(W, tile_m=tiles[0], tile_k=tiles[1])
    cont = oracle_mod.encode(W, *tiles)
    val_dir, val_pack, val_mask = oracle_mod.values_compact(cont)
    assert np.array_equal(m.canonical("val_dir").reshape(-1, 2), val_dir)
    assert np.array_equal(m.canonical("val_pack"), val_pack)
    assert np.array_equal(m.canonical("val_mask"), val_mask)
    assert m.stats()["canonical_bytes_compact_all"] == oracle_mod.compact_nbytes_all(cont)
    # above 50 % every tile takes the bitmap; at 50 % an interior tile does not (the ragged edge's
    # padded tiles, mostly empty, do)
    assert (val_dir[:, 0] == 1).all() if sparsity > 0.5 else val_dir[0, 0] == 0
    assert np.array_equal(oracle_mod.values_expand(cont, m.canonical("val_dir").reshape(-1, 2), m.canonical("val_pack"),
                                                   m.canonical("val_mask")), m.canonical("tc_vals"))


def test_launch_tuning_round_trip(tl3):
    L = tl3.lib()
    assert tl3.get_tuning() == {"decode_before_x": 4}
    try:
        tl3.set_tuning(decode_before_x=-1)
        assert tl3.get_tuning()["decode_before_x"] == -1
        bad = tl3.Tuning(-2)
        assert L.tl3_set_tuning(ctypes.byref(bad)) == tl3.ERR_INVALID_ARG
        assert tl3.get_tuning()["decode_before_x"] == -1          # a refused setting changes nothing
        assert L.tl3_get_tuning(None) == tl3.ERR_INVALID_ARG
    finally:
        tl3.set_tuning()
    assert tl3.get_tuning() == {"decode_before_x": 4}


def test_const_calls_on_one_handle_from_several_threads(tl3):
    """tl3_device_bytes / tl3_stats / tl3_pack take a const handle and compute the layout of the
    device image on first use: four threads that make that first use together must all see the same,
    complete layout (the blob of each equals the blob packed afterwards by one thread)."""
    import threading
    case = wl.Case(0, "thr", 1024, 1536, 8, 31, 0.5, "magnitude")
    m = tl3.encode(case.make_W())
    out, errs = [None] * 4, []

    def work(i):
        try:
            n = m.device_bytes()
            st = m.stats()
            assert st["device_bytes"] == n
            out[i] = m.pack()
        except Exception as e:                                   # pragma: no cover
            errs.append(e)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errs
    ref = m.pack()
    for o in out:
        assert o is not None and np.array_equal(o, ref)


def _image_offset(u):
    """Byte offset of bank-major slot u = bank << 8 | slot-in-window << 7 | row in the value image."""
    return ((u & 127) << 7) | ((u >> 6) & 0x7E)


def _decode_device_blob(blob, M_pad, K_pad):
    """Algorithm 1 run in numpy over every tile block of a packed blob, as the kernel runs it:
    parked values move from W_t[tau] to W_r[rho], Residual entries go to W_r, then both sparse
    operands are expanded with their metadata.  Returns the dense fp16 bit patterns and checks the
    structure of each block on the way."""
    tiles_m, tiles_k = M_pad // 128, K_pad // 128
    n_tiles = tiles_m * tiles_k
    directory = blob[256:256 + 16 * n_tiles].view(np.uint32).reshape(n_tiles, 4)
    W = np.zeros((M_pad, K_pad), dtype=np.uint16)
    seen_end = 256 + 16 * n_tiles
    for t in range(n_tiles):
        tm, tk = divmod(t, tiles_k)
        off16, nbytes, pdd_len, res_cnt = (int(x) for x in directory[t])
        assert (off16 * 16) % 128 == 0 and off16 * 16 >= seen_end             # aligned, no overlap
        assert nbytes == (18960 + pdd_len + 4 * res_cnt + 15) // 16 * 16
        seen_end = off16 * 16 + nbytes
        blk = blob[off16 * 16: off16 * 16 + nbytes]
        img = blk[:16384].view(np.uint16).copy()                              # W_t image, halfword = byte offset / 2
        meta = blk[16384:18432].view(np.uint32).reshape(128, 4)
        info = blk[18432:18448].view(np.uint32)
        assert (int(info[0]), int(info[1])) == (pdd_len, res_cnt)
        hdr = blk[18448:18960].view(np.uint32)
        n_words = int(info[2])                                                 # code words per chain, transposed
        assert n_words <= 3 and pdd_len == 512 * n_words
        words = blk[18960:18960 + pdd_len].view(np.uint32).reshape(n_words, 128)
        res = blk[18960 + pdd_len:][:4 * res_cnt].view(np.uint32)
        wr = np.zeros(8192, dtype=np.uint16)                                   # W_r image
        for j in range(128):
            h = int(hdr[j])
            code = np.ascontiguousarray(words[:, j]).view(np.uint8)            # 4 * n_words delta bytes, zero padded
            if h == 0xFFFFFFFF:
                assert not code.any()
                continue
            pt, pr = h & 0xFFFF, h >> 16
            assert pt < 8192 and pr < 8192 and (pt >> 8) == (j & 31)           # slot j: a chain of bank j % 32
            bank = pt >> 8

            def move(pt, pr):
                assert (pt >> 8) == bank                                       # a chain stays in the bank of its lane
                v = img[_image_offset(pt) // 2]
                assert v & 0x7FFF and wr[_image_offset(pr) // 2] == 0
                img[_image_offset(pt) // 2] = 0
                wr[_image_offset(pr) // 2] = v

            move(pt, pr)
            for b in code:
                dt, dr = int(b) & 15, int(b) >> 4
                pt += dt
                pr += dr
                if dt and dr:
                    move(pt, pr)
        for e in res:
            u, v = int(e) & 0xFFFF, int(e) >> 16
            assert u < 8192 and wr[_image_offset(u) // 2] == 0
            wr[_image_offset(u) // 2] = v
        nib = np.zeros((128, 32), dtype=np.uint8)                              # metadata nibble of (row, window)
        for lane in range(128):
            row, half = (lane & 7) + 16 * (lane >> 4), (lane >> 3) & 1
            for kb in range(4):
                w = int(meta[lane, kb])
                for i in range(4):
                    nib[row, 8 * kb + 4 * half + i] = (w >> (4 * i)) & 15
                    nib[row + 8, 8 * kb + 4 * half + i] = (w >> (16 + 4 * i)) & 15
        for r in range(128):
            for q in range(32):
                base = r * 128 + (((q >> 2) ^ (r & 7)) << 4) + (q & 3) * 4    # 128-byte swizzle
                idx = (int(nib[r, q]) & 3, int(nib[r, q]) >> 2)
                assert idx[0] < idx[1]
                for s in range(2):
                    v = img[(base + 2 * s) // 2]
                    if v & 0x7FFF:
                        W[tm * 128 + r, tk * 128 + 4 * q + idx[s]] = v
                    v = wr[(base + 2 * s) // 2]
                    if v & 0x7FFF:
                        assert W[tm * 128 + r, tk * 128 + 4 * q + 2 + s] == 0
                        W[tm * 128 + r, tk * 128 + 4 * q + 2 + s] = v
    assert seen_end <= blob.size
    return W


@pytest.mark.parametrize("shape,sparsity,mask", [((200, 300), 0.45, "magnitude"), ((256, 384), 0.5, "bernoulli"),
                                                 ((256, 256), 0.7, "magnitude"), ((128, 256), 0.3, "magnitude"),
                                                 ((128, 128), 1.0, "bernoulli"), ((128, 128), 0.0, "bernoulli")])
def test_device_blob_decodes_to_the_matrix(tl3, shape, sparsity, mask):
    """The packed device image (bank-major re-pairing of the Slot-Filling layer) holds the same
    matrix: an independent numpy decoder of the blob reproduces W bit for bit, every chain lies in
    the bank of its lane, and the blob is hardly larger than the canonical container."""
    M, K = shape
    W = wl.Case(0, "pack", M, K, 8, 9, sparsity, mask).make_W()
    m = tl3.encode(W)
    blob = m.pack()
    st = m.stats()
    assert blob.size == m.device_bytes() and blob.size % 256 == 0
    ref = np.zeros((st["M_pad"], st["K_pad"]), dtype=np.uint16)
    ref[:M, :K] = W.view(np.uint16)
    ref[ref == 0x8000] = 0
    assert np.array_equal(_decode_device_blob(blob, st["M_pad"], st["K_pad"]), ref)


@pytest.mark.parametrize("seed", range(12))
def test_device_blob_on_adversarial_patterns(tl3, seed):
    """Tiles whose density changes abruptly by row band and by column band (empty bands, dense
    bands, bands with only surplus or only empty slots): the packer's proportional selection of
    empty slots, its equal-count chains and its cut after three code words must still give a blob
    that decodes to the matrix."""
    rng = np.random.default_rng([77, seed])
    M, K = 256, 384
    dens_r = rng.choice([0.0, 0.1, 0.5, 0.9, 1.0], size=M // 32).repeat(32)
    dens_c = rng.choice([0.0, 0.25, 0.5, 0.75, 1.0], size=K // 64).repeat(64)
    p = np.clip(0.5 * (dens_r[:, None] + dens_c[None, :]) + rng.choice([-0.3, 0.0, 0.3]), 0, 1)
    W = np.where(rng.random((M, K)) < p, (rng.standard_normal((M, K)) * 0.05).astype(np.float16), np.float16(0))
    W[(W.view(np.uint16) & 0x7FFF) == 0] = 0
    m = tl3.encode(W)
    st = m.stats()
    blob = m.pack()
    assert np.array_equal(_decode_device_blob(blob, st["M_pad"], st["K_pad"]), W.view(np.uint16))
    assert np.array_equal(m.decode(), W.view(np.uint16))


def test_device_chain_overflow_goes_to_the_residual_list(tl3):
    """A chain of the device image is cut when it is full (here: because two consecutive pairs lie
    thousands of positions apart); what is cut off travels in the Residual list, and the blob
    still decodes to the matrix."""
    from special_cases import clustered_surplus_tile
    W = clustered_surplus_tile()
    m = tl3.encode(W)
    assert m.stats()["n_res"] == 0                                   # nothing in the canonical Residual layer
    blob = m.pack()
    directory = blob[256:272].view(np.uint32)
    assert int(directory[3]) > 0                                       # but the device image has Residual entries
    assert np.array_equal(_decode_device_blob(blob, 128, 128), W.view(np.uint16))


def test_device_blob_size_stays_close_to_canonical(tl3):
    for sparsity in (0.4, 0.5, 0.6, 0.7):
        m = tl3.encode(wl.Case(0, "pack", 512, 1024, 8, 9, sparsity, "magnitude").make_W())
        st = m.stats()
        assert st["device_bytes"] <= 1.035 * st["canonical_bytes"] + 4096


def test_two_rank_plumbing_on_cpu():
    """world_size 2 over gloo: the barrier / max-over-ranks timing and the per-rank seeds."""
    import subprocess
    import sys
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    code = r"""
import os, sys
sys.path.insert(0, %r)
import numpy as np
from paper_2607_08786_b200 import dist, workloads as wl
rank, local_rank, world = dist.init_process_group("gloo")
assert world == 2 and rank == local_rank
dist.barrier()
t = dist.max_over_ranks(1.0 + rank)
n = dist.sum_over_ranks(10.0)
assert t == 2.0 and n == 20.0, (t, n)
case = wl.Case(2, "x", 128, 128, 8, 2000 + dist.rank_seed_offset(rank))
h = int(case.make_W().view(np.uint16).astype(np.uint64).sum())
both = dist.sum_over_ranks(float(h)) - h
assert both != h                      # the other rank drew a different matrix
assert dist.shard_round_robin(list(range(5)), rank, world) == ([0, 2, 4] if rank == 0 else [1, 3])
dist.barrier()
print("rank", rank, "ok")
""" % ROOT
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_row_shard_ranges():
    from paper_2607_08786_b200 import dist
    for M, world in ((1000, 2), (128, 4), (36864, 8), (130, 3)):
        ranges = [dist.row_shard(M, r, world) for r in range(world)]
        assert ranges[0][0] == 0 and ranges[-1][1] == M
        for (a, b), (c, d) in zip(ranges[:-1], ranges[1:]):
            assert b == c and a % 128 == 0 and c % 128 == 0      # contiguous, cut between row-tiles
        sizes = [(b - a + 127) // 128 for a, b in ranges]
        assert max(sizes) - min(sizes) <= 1


def test_row_split_over_two_ranks_on_cpu():
    """world_size 2 over gloo: one W split by rows (the 2-GPU arrangement of Sec. 5.3), X replicated,
    all-gather of Y.  The per-rank product is a CPU stand-in (the library's own encoder and decoder
    around a float32 matmul), so this covers the partitioning, the padding of unequal slabs and the
    collective; the kernel itself is covered by the GPU tests."""
    import subprocess
    import sys
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    code = r"""
import os, sys
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2607_08786_b200 import dist, tl3, workloads as wl
rank, local_rank, world = dist.init_process_group("gloo")
case = wl.Case(0, "split", 1000, 512, 8, 99, 0.5, "magnitude")      # 8 row-tiles, the last one ragged
W, X = case.make_W(), case.make_X()
def stand_in(slab):
    m = tl3.encode(slab)                                              # each rank encodes only its slab
    Wd = torch.from_numpy(m.decode().view(np.float16).astype(np.float32))
    return lambda Xt: (Wd @ Xt.float()).half()
sh = dist.RowShardedMatrix(W, local_product=stand_in)
assert sh.ranges == [(0, 512), (512, 1000)], sh.ranges
Y = sh.matmul(torch.from_numpy(X))
ref = (torch.from_numpy(W.astype(np.float32)) @ torch.from_numpy(X.astype(np.float32))).half()
assert Y.shape == (1000, 8) and torch.allclose(Y.float(), ref.float(), atol=2e-3, rtol=2e-3)
dist.barrier()
print("rank", rank, "ok")
""" % ROOT
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


@pytest.mark.parametrize("sparsity,tiles", [(0.3, (128, 128)), (0.5, (128, 128)), (0.7, (128, 128)), (0.6, (4, 32)), (0.95, (128, 128))])
def test_compact_persistence_round_trip(tl3, sparsity, tiles):
    """tl3_serialize_compact -> tl3_deserialize gives the same container: re-serialised in the plain
    form it is the original's plain bytes.  Its size is the header, thirteen lengths and what
    tl3_stats announces; above and below 50 % it is smaller than the plain form."""
    W = wl.Case(0, "cp", 300, 520, 8, 33, sparsity, "magnitude").make_W()
    W[5, 7] = np.float16(-0.0)                                     # a zero as far as the format is concerned
    m = tl3.encode(W, tile_m=tiles[0], tile_k=tiles[1])
    plain, compact = m.serialize(), m.serialize(compact=True)
    back = tl3.Matrix.deserialize(compact)
    assert back.serialize() == plain
    assert back.serialize(compact=True) == compact
    assert np.array_equal(back.decode(), m.decode())
    header = len(plain) - 9 * 8 - m.stats()["canonical_bytes"]
    assert len(compact) == header + 13 * 8 + m.stats()["canonical_bytes_compact_all"]
    if sparsity != 0.5:
        assert len(compact) < len(plain)


def test_corrupted_compact_containers_are_rejected_or_valid(tl3):
    """Nothing in a compact container is trusted: truncations, and single bytes overwritten anywhere
    in the directories, bitmaps, lists and values, either fail with BAD_CONTAINER or give a container
    that serialises again and decodes or is refused by the decoder; none may crash or read out of
    bounds."""
    rng = np.random.default_rng(17)
    W = wl.Case(0, "cc", 260, 300, 8, 5, 0.4, "magnitude").make_W()
    W[128:, :] = np.where(rng.random((132, 300)) < 0.25, W[128:, :], np.float16(0))      # sparse lower half: bitmap tiles
    m = tl3.encode(W)
    good = m.serialize(compact=True)
    assert tl3.Matrix.deserialize(good).serialize() == m.serialize()
    modes_v, modes_r = m.canonical("val_dir").reshape(-1, 2)[:, 0], m.canonical("res_dir").reshape(-1, 2)[:, 0]
    assert set(modes_v.tolist()) == {0, 1} and set(modes_r.tolist()) == {0, 1}           # both forms of both layers occur
    for cut in (0, 50, 79, 80, 200, len(good) // 2, len(good) - 1):
        with pytest.raises(tl3.Tl3Error):
            tl3.Matrix.deserialize(good[:cut])
    with pytest.raises(tl3.Tl3Error):
        tl3.Matrix.deserialize(good + b"\0")
    rejected = accepted = 0
    # the first kilobyte holds the header and the value directory; then spread over the whole blob
    places = list(range(40, 400)) + rng.integers(0, len(good), size=600).tolist()
    for at in places:
        bad = bytearray(good)
        bad[at] ^= int(rng.integers(1, 256))
        try:
            back = tl3.Matrix.deserialize(bytes(bad))
        except tl3.Tl3Error as e:
            assert e.code == tl3.ERR_BAD_CONTAINER
            rejected += 1
            continue
        accepted += 1                                             # e.g. a changed value: still a container
        assert len(back.serialize()) > 0
        try:
            assert back.decode().shape == W.shape
        except tl3.Tl3Error as e:                                 # the decoder walks the chains and may still refuse
            assert e.code == tl3.ERR_BAD_CONTAINER
        back.close()
    assert rejected > 100 and accepted > 100
