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
    assert b"invalid" in L.tl3_strerror(tl3.ERR_INVALID_ARG)
    assert L.tl3_strerror(-99) == b"unknown error"


def _expected_blob_blocks(c, M_pad, K_pad):
    """The device layout re-derived in numpy from the oracle's container, tile by tile."""
    H = 64
    tiles_m, tiles_k = M_pad // 128, K_pad // 128
    vals = c.tc_vals.reshape(M_pad, K_pad // 2)
    meta = c.tc_meta.reshape(M_pad, K_pad // 8)
    for tm in range(tiles_m):
        for tk in range(tiles_k):
            t = tm * tiles_k + tk
            pdd_off, pdd_len, res_off, res_cnt = (int(x) for x in c.tile_dir[t])
            v = vals[tm * 128:(tm + 1) * 128, tk * H:(tk + 1) * H].reshape(128, 8, 8)     # row, chunk, 8 values
            img = np.zeros((128, 8, 8), dtype=np.uint16)
            for r in range(128):
                for j in range(8):
                    img[r, j ^ (r & 7)] = v[r, j]
            mt = meta[tm * 128:(tm + 1) * 128, tk * 16:(tk + 1) * 16]                         # 16 bytes per row
            words = np.zeros((128, 4), dtype=np.uint32)
            for L in range(128):
                row, half = (L & 7) + 16 * (L >> 4), (L >> 3) & 1
                for kb in range(4):
                    lo = mt[row, 4 * kb + 2 * half: 4 * kb + 2 * half + 2].astype(np.uint32)
                    hi = mt[row + 8, 4 * kb + 2 * half: 4 * kb + 2 * half + 2].astype(np.uint32)
                    words[L, kb] = lo[0] | lo[1] << 8 | hi[0] << 16 | hi[1] << 24
            info = np.array([pdd_len, res_cnt, 0, 0], dtype=np.uint32)
            hdr = (c.chain_tau0[t * 128:(t + 1) * 128].astype(np.uint32) |
                   c.chain_rho0[t * 128:(t + 1) * 128].astype(np.uint32) << 16)
            lens = c.chain_len[t * 128:(t + 1) * 128]
            # chains longest first, ties by row
            order = sorted(range(128), key=lambda r: (-int(lens[r]), r))
            starts = np.concatenate([[0], np.cumsum(lens.astype(np.int64))])
            codes = c.pdd_bytes[pdd_off:pdd_off + pdd_len]
            pdd = np.concatenate([codes[starts[r]:starts[r + 1]] for r in order]) if pdd_len else codes
            hdr, lens = hdr[order], lens[order]
            pad = (-pdd_len) % 4
            res = (c.res_rho[res_off:res_off + res_cnt].astype(np.uint32) |
                   c.res_val[res_off:res_off + res_cnt].astype(np.uint32) << 16)
            block = b"".join([img.tobytes(), words.tobytes(), info.tobytes(), hdr.tobytes(), lens.tobytes(),
                              pdd.tobytes(), b"\0" * pad, res.tobytes()])
            block += b"\0" * ((-len(block)) % 16)
            yield t, block, pdd_len, res_cnt


def test_device_blob_layout(tl3, oracle_mod):
    """Every tile block of the packed blob against an independent numpy construction."""
    W = wl.Case(0, "pack", 200, 300, 8, 9, 0.45, "magnitude").make_W()     # ragged, some Residual
    m = tl3.encode(W)
    c = oracle_mod.encode(W)
    blob = m.pack()
    assert blob.size == m.device_bytes() and blob.size % 256 == 0
    st = m.stats()
    n_tiles = st["n_tiles"]
    directory = blob[256:256 + 16 * n_tiles].view(np.uint32).reshape(n_tiles, 4)
    seen_end = 0
    for t, block, pdd_len, res_cnt in _expected_blob_blocks(c, st["M_pad"], st["K_pad"]):
        off16, nbytes, d_pdd, d_res = (int(x) for x in directory[t])
        assert (off16 * 16) % 128 == 0 and nbytes % 16 == 0
        assert (nbytes, d_pdd, d_res) == (len(block), pdd_len, res_cnt)
        assert off16 * 16 >= seen_end                                   # blocks do not overlap
        seen_end = off16 * 16 + nbytes
        assert blob[off16 * 16: off16 * 16 + nbytes].tobytes() == block, f"tile {t}"
    assert seen_end <= blob.size


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
