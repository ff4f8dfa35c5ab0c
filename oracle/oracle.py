"""ctypes front end of ``tl3_oracle.c`` plus the dense fp64 definition of the product.

TEST INFRASTRUCTURE ONLY (see ``tl3_oracle.c``).  ``encode`` / ``decode`` / ``spmm`` follow the
paper's storage format (Sec. 3.2) and Algorithm 1 step by step in plain C; ``dense_fp64`` is the
problem statement of Sec. 5.1 written out (``Y = W X``) with a library matmul in float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tl3_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

FIELDS = ("tc_vals", "tc_meta", "chain_tau0", "chain_rho0", "chain_len", "pdd_bytes", "tile_dir",
          "res_rho", "res_val")
_DTYPES = (np.uint16, np.uint8, np.uint16, np.uint16, np.uint8, np.uint8, np.uint32, np.uint16,
           np.uint16)


def build(force: bool = False) -> str:
    """Compile the oracle's C file with gcc (OpenMP if available) and return the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True, capture_output=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_encode.restype = ctypes.c_int
        lib.oracle_encode.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
                                      ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_void_p)]
        lib.oracle_get.restype = ctypes.c_int
        lib.oracle_get.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_void_p),
                                   ctypes.POINTER(ctypes.c_int64)]
        lib.oracle_stats.restype = None
        lib.oracle_stats.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        lib.oracle_free.restype = None
        lib.oracle_free.argtypes = [ctypes.c_void_p]
        arrays = [ctypes.c_void_p] * 9
        lib.oracle_decode.restype = ctypes.c_int
        lib.oracle_decode.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                      *arrays, ctypes.c_void_p]
        lib.oracle_spmm.restype = ctypes.c_int
        lib.oracle_spmm.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                    *arrays, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                    ctypes.c_int64, ctypes.c_int]
        lib.oracle_threads.restype = ctypes.c_int
        lib.oracle_half_to_float.restype = ctypes.c_float
        lib.oracle_half_to_float.argtypes = [ctypes.c_uint16]
        lib.oracle_float_to_half.restype = ctypes.c_uint16
        lib.oracle_float_to_half.argtypes = [ctypes.c_float]
        _lib = lib
    return _lib


@dataclass
class Container:
    """The canonical container: nine flat arrays plus the shape and tile parameters."""
    M: int
    K: int
    tile_m: int
    tile_k: int
    maxd: int
    tc_vals: np.ndarray
    tc_meta: np.ndarray
    chain_tau0: np.ndarray
    chain_rho0: np.ndarray
    chain_len: np.ndarray
    pdd_bytes: np.ndarray
    tile_dir: np.ndarray
    res_rho: np.ndarray
    res_val: np.ndarray
    stats: dict = field(default_factory=dict)

    @property
    def M_pad(self) -> int:
        return -(-self.M // self.tile_m) * self.tile_m

    @property
    def K_pad(self) -> int:
        return -(-self.K // self.tile_k) * self.tile_k

    def arrays(self):
        return [np.ascontiguousarray(getattr(self, f), dtype=d) for f, d in zip(FIELDS, _DTYPES)]

    def nbytes(self) -> int:
        return sum(a.nbytes for a in self.arrays())


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _as_u16(a) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("expected float16 or uint16 (fp16 bit patterns)")
    return np.ascontiguousarray(a)


def encode(W, tile_m: int = 128, tile_k: int = 128, maxd: int = 15) -> Container:
    """Dense masked fp16 ``W`` (M x K) -> container (Sec. 3.2)."""
    W = _as_u16(W)
    M, K = W.shape
    lib = _load()
    h = ctypes.c_void_p()
    rc = lib.oracle_encode(_ptr(W), M, K, tile_m, tile_k, maxd, ctypes.byref(h))
    if rc != 0:
        raise ValueError(f"oracle_encode failed ({rc})")
    try:
        out = {}
        for i, (name, dt) in enumerate(zip(FIELDS, _DTYPES)):
            p = ctypes.c_void_p()
            n = ctypes.c_int64()
            lib.oracle_get(h, i, ctypes.byref(p), ctypes.byref(n))
            if n.value:
                buf = (ctypes.c_uint8 * n.value).from_address(p.value)
                out[name] = np.frombuffer(buf, dtype=dt).copy()
            else:
                out[name] = np.zeros(0, dtype=dt)
        st = np.zeros(6, dtype=np.int64)
        lib.oracle_stats(h, _ptr(st))
    finally:
        lib.oracle_free(h)
    out["tile_dir"] = out["tile_dir"].reshape(-1, 4)
    stats = dict(zip(("nnz", "n_tc", "n_sf", "n_res", "n_dummy", "n_slots_unused"), map(int, st)))
    return Container(M, K, tile_m, tile_k, maxd, stats=stats, **out)


def decode(c: Container) -> np.ndarray:
    """Container -> dense fp16 bit patterns (Algorithm 1 on the CPU, then the 2:4 expansion)."""
    W = np.zeros((c.M, c.K), dtype=np.uint16)
    arrs = c.arrays()
    rc = _load().oracle_decode(c.M, c.K, c.tile_m, c.tile_k, *[_ptr(a) for a in arrs], _ptr(W))
    if rc != 0:
        raise ValueError(f"oracle_decode failed ({rc})")
    return W


def spmm(c: Container, X) -> np.ndarray:
    """``Y = W X`` over the container, fp32 accumulation, fp16 output (bit patterns)."""
    X = _as_u16(X)
    K, N = X.shape
    if K != c.K:
        raise ValueError("X has the wrong number of rows")
    Y = np.zeros((c.M, N), dtype=np.uint16)
    arrs = c.arrays()
    rc = _load().oracle_spmm(c.M, c.K, c.tile_m, c.tile_k, *[_ptr(a) for a in arrs], _ptr(X), N,
                             _ptr(Y), N, N)
    if rc != 0:
        raise ValueError(f"oracle_spmm failed ({rc})")
    return Y


def dense_fp64(W, X, row_block: int = 2048):
    """The definition ``y_ij = sum_k w_ik x_kj`` in float64, and ``sum_k |w_ik x_kj|`` beside it.

    Products of two fp16 numbers are exact in float64, so only the summation order rounds.
    """
    W = _as_u16(W).view(np.float16)
    X64 = _as_u16(X).view(np.float16).astype(np.float64)
    M = W.shape[0]
    Y = np.empty((M, X64.shape[1]), dtype=np.float64)
    B = np.empty_like(Y)
    absX = np.abs(X64)
    for r in range(0, M, row_block):
        w = W[r:r + row_block].astype(np.float64)
        Y[r:r + row_block] = w @ X64
        B[r:r + row_block] = np.abs(w) @ absX
    return Y, B


def tolerance(bound: np.ndarray) -> np.ndarray:
    """Per-element tolerance of the benchmark spec: 2e-3 * sum_k |w_ik x_kj| + 1e-3."""
    return 2e-3 * bound + 1e-3


def threads() -> int:
    return int(_load().oracle_threads())


def half_to_float(h: int) -> float:
    return float(_load().oracle_half_to_float(int(h)))


def float_to_half(f: float) -> int:
    return int(_load().oracle_float_to_half(float(f)))


# ---- compact form of the Residual layer ---------------------------------------------------------
# Sec. 3.2 leaves the Residual format open ("a classic format such as CSR") because at 50 % it
# holds under 1 % of the non-zeros.  Below 50 % sparsity it does not stay small (no tile has room
# for more than half of its weights in the value slots), and two bytes of position per entry add
# up.  The compact form keeps, per tile, whichever is smaller: the position list, or a bitmap over
# the tile's tile_m * H positions of W_r (bit rho % 8 of byte rho // 8) with the values in
# ascending position order as before.
def residual_compact(c: Container):
    """(res_dir, res_list, res_mask) of a container's Residual layer.

    res_dir  u32[tiles][2]  {mode, off}: mode 0 = position list, off = index of the tile's first
                            position in res_list; mode 1 = bitmap, off = byte offset of the tile's
                            bitmap in res_mask
    res_list u16[]          positions of the list-mode tiles, tile after tile
    res_mask u8[]           ceil(tile_m * H / 8) bytes per bitmap-mode tile
    A tile takes the bitmap iff it is strictly smaller than the tile's two-byte positions."""
    H = c.tile_k // 2
    B = (c.tile_m * H + 7) // 8
    n_tiles = c.tile_dir.shape[0]
    res_dir = np.zeros((n_tiles, 2), dtype=np.uint32)
    lists, masks = [], []
    n_list = n_mask = 0
    for t in range(n_tiles):
        off, cnt = int(c.tile_dir[t, 2]), int(c.tile_dir[t, 3])
        rho = c.res_rho[off:off + cnt].astype(np.int64)
        if B < 2 * cnt:
            bits = np.zeros(B * 8, dtype=np.uint8)
            bits[rho] = 1
            masks.append(np.packbits(bits, bitorder="little"))
            res_dir[t] = (1, n_mask)
            n_mask += B
        else:
            lists.append(rho.astype(np.uint16))
            res_dir[t] = (0, n_list)
            n_list += cnt
    res_list = np.concatenate(lists) if lists else np.zeros(0, dtype=np.uint16)
    res_mask = np.concatenate(masks) if masks else np.zeros(0, dtype=np.uint8)
    return res_dir, res_list.astype(np.uint16), res_mask.astype(np.uint8)


def residual_expand(c: Container, res_dir, res_list, res_mask) -> np.ndarray:
    """The inverse: the positions res_rho of every Residual entry, from the compact form."""
    H = c.tile_k // 2
    B = (c.tile_m * H + 7) // 8
    out = np.zeros(len(c.res_val), dtype=np.uint16)
    for t in range(c.tile_dir.shape[0]):
        off, cnt = int(c.tile_dir[t, 2]), int(c.tile_dir[t, 3])
        mode, at = int(res_dir[t, 0]), int(res_dir[t, 1])
        if mode == 1:
            bits = np.unpackbits(np.asarray(res_mask[at:at + B], dtype=np.uint8), bitorder="little")
            rho = np.flatnonzero(bits)
            if len(rho) != cnt:
                raise ValueError("bitmap and entry count disagree")
        else:
            rho = np.asarray(res_list[at:at + cnt])
        out[off:off + cnt] = rho
    return out


# --- Empty value slots above 50 % sparsity (the paper's Sec. 6: "most regions require zero padding").
# The paper stores every slot of the Sparse-TC value array; a slot that neither keeps a weight nor
# had one parked in it holds zero.  Compact form (a reading, like the Residual's): per tile either
# the tile's tile_m * H values as they are, or a bitmap of the occupied slots (bit pos % 8 of byte
# pos // 8, pos = row * H + slot, the coordinate of the PDD streams) followed by the occupied
# slots' values in ascending position order; the bitmap is taken iff it is strictly smaller, i.e.
# iff its bytes are fewer than two per empty slot.  "Occupied" = any non-zero bit pattern (the
# encoder writes +0.0 into an empty slot; a container that carries -0.0 there keeps it, so the
# compact form is lossless for every container).
def values_compact(c: Container):
    """(val_dir, val_pack, val_mask) of a container's Sparse-TC value array.

    val_dir  u32[tiles][2]  {mode, off}: mode 0 = all tile_m * H values of the tile, starting at
                            val_pack[off]; mode 1 = only the occupied slots' values, starting at
                            val_pack[off], and the tile's bitmap at val_mask[index * B] where index
                            counts the bitmap-mode tiles before this one
    val_pack u16[]          values, tile after tile, row-major inside a tile
    val_mask u8[]           B = ceil(tile_m * H / 8) bytes per bitmap-mode tile"""
    H = c.tile_k // 2
    S = c.tile_m * H
    B = (S + 7) // 8
    tiles_m, tiles_k = c.M_pad // c.tile_m, c.K_pad // c.tile_k
    vals = np.asarray(c.tc_vals, dtype=np.uint16).reshape(c.M_pad, c.K_pad // 2)
    val_dir = np.zeros((tiles_m * tiles_k, 2), dtype=np.uint32)
    packs, masks = [], []
    n_pack = 0
    for tm in range(tiles_m):
        for tk in range(tiles_k):
            t = tm * tiles_k + tk
            tile = vals[tm * c.tile_m:(tm + 1) * c.tile_m, tk * H:(tk + 1) * H].reshape(-1)
            occupied = tile != 0
            empties = S - int(occupied.sum())
            if B < 2 * empties:
                masks.append(np.packbits(occupied.astype(np.uint8), bitorder="little"))
                packs.append(tile[occupied])
                val_dir[t] = (1, n_pack)
                n_pack += int(occupied.sum())
            else:
                packs.append(tile.copy())
                val_dir[t] = (0, n_pack)
                n_pack += S
    val_pack = np.concatenate(packs) if packs else np.zeros(0, dtype=np.uint16)
    val_mask = np.concatenate(masks) if masks else np.zeros(0, dtype=np.uint8)
    return val_dir, val_pack.astype(np.uint16), val_mask.astype(np.uint8)


def values_expand(c: Container, val_dir, val_pack, val_mask) -> np.ndarray:
    """The inverse: the full value array tc_vals (u16, M_pad * K_pad / 2) from the compact form
    (an empty slot is the bit pattern 0)."""
    H = c.tile_k // 2
    S = c.tile_m * H
    B = (S + 7) // 8
    tiles_m, tiles_k = c.M_pad // c.tile_m, c.K_pad // c.tile_k
    out = np.zeros((c.M_pad, c.K_pad // 2), dtype=np.uint16)
    n_mask = 0
    for tm in range(tiles_m):
        for tk in range(tiles_k):
            t = tm * tiles_k + tk
            mode, at = int(val_dir[t, 0]), int(val_dir[t, 1])
            if mode == 1:
                bits = np.unpackbits(np.asarray(val_mask[n_mask * B:(n_mask + 1) * B], dtype=np.uint8), bitorder="little")[:S].astype(bool)
                n_mask += 1
                tile = np.zeros(S, dtype=np.uint16)
                tile[bits] = val_pack[at:at + int(bits.sum())]
            else:
                tile = np.asarray(val_pack[at:at + S], dtype=np.uint16)
            out[tm * c.tile_m:(tm + 1) * c.tile_m, tk * H:(tk + 1) * H] = tile.reshape(c.tile_m, H)
    return out.reshape(-1)


def compact_nbytes_all(c: Container) -> int:
    """Size of the container with the Residual layer and the value array in their compact forms."""
    val_dir, val_pack, val_mask = values_compact(c)
    return compact_nbytes(c) - np.asarray(c.tc_vals, dtype=np.uint16).nbytes + val_dir.nbytes + val_pack.nbytes + val_mask.nbytes


def compact_nbytes(c: Container) -> int:
    """Size of the container with the Residual layer in its compact form."""
    res_dir, res_list, res_mask = residual_compact(c)
    return c.nbytes() - c.res_rho.nbytes + res_dir.nbytes + res_list.nbytes + res_mask.nbytes
