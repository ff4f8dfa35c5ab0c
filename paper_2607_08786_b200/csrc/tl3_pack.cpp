// Device packer: lays the canonical container out as one blob of per-tile blocks, each ready for
// a single bulk copy into shared memory (layout described in tl3_internal.h).  The blob is a
// permutation of the canonical bytes plus alignment padding; nothing is re-encoded.
#include <algorithm>
#include <cstring>

#include "tl3_internal.h"

namespace tl3 {

static inline uint32_t align_up(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

static inline uint32_t block_bytes(uint32_t pdd_len, uint32_t res_cnt) {
  return align_up(kPddOff + align_up(pdd_len, 4) + 4 * res_cnt, 16);
}

size_t plan_device_layout(tl3_matrix* m) {
  if (m->device_bytes) return m->device_bytes;
  size_t off = 256;
  m->dir_offset = off;
  off += static_cast<size_t>(m->n_tiles) * sizeof(DirEntry);
  off = (off + 255) / 256 * 256;
  m->blocks_offset = off;
  uint32_t max_block = 0;
  for (int64_t t = 0; t < m->n_tiles; ++t) {
    const uint32_t b = block_bytes(m->tile_dir[t * 4 + 1], m->tile_dir[t * 4 + 3]);
    if (b > max_block) max_block = b;
    off += align_up(b, kBlockAlign);
  }
  m->max_block_bytes = max_block;
  m->device_bytes = (off + 255) / 256 * 256;
  return m->device_bytes;
}

void pack_device_blob(const tl3_matrix* m, uint8_t* out) {
  std::memset(out, 0, m->device_bytes);
  // header (informational; the kernel takes its geometry from its arguments)
  struct { uint32_t magic, version; int64_t M, K, M_pad, K_pad, n_tiles; uint64_t dir_off, blocks_off; uint32_t max_block; } hdr{
      0x33334C54u, 1, m->M, m->K, m->M_pad, m->K_pad, m->n_tiles, m->dir_offset, m->blocks_offset, m->max_block_bytes};
  std::memcpy(out, &hdr, sizeof(hdr));
  DirEntry* dir = reinterpret_cast<DirEntry*>(out + m->dir_offset);
  const int64_t half_ld = m->K_pad / 2, meta_ld = m->K_pad / 8;
  size_t off = m->blocks_offset;
  for (int64_t tm = 0; tm < m->tiles_m; ++tm) {
    for (int64_t tk = 0; tk < m->tiles_k; ++tk) {
      const int64_t t = tm * m->tiles_k + tk;
      const uint32_t pdd_off = m->tile_dir[t * 4], pdd_len = m->tile_dir[t * 4 + 1];
      const uint32_t res_off = m->tile_dir[t * 4 + 2], res_cnt = m->tile_dir[t * 4 + 3];
      const uint32_t bytes = block_bytes(pdd_len, res_cnt);
      uint8_t* blk = out + off;
      dir[t] = DirEntry{static_cast<uint32_t>(off / 16), bytes, pdd_len, res_cnt};
      // values: row r, 16-byte chunk j -> chunk j ^ (r & 7)
      for (int r = 0; r < kTileM; ++r) {
        const uint8_t* src = reinterpret_cast<const uint8_t*>(&m->tc_vals[(tm * kTileM + r) * half_ld + tk * kH]);
        for (int j = 0; j < 8; ++j) std::memcpy(blk + r * 128 + ((j ^ (r & 7)) << 4), src + j * 16, 16);
      }
      // metadata in tensor-memory lane order
      uint32_t* meta = reinterpret_cast<uint32_t*>(blk + kMetaOff);
      for (int L = 0; L < 128; ++L) {
        const int row = (L & 7) + 16 * (L >> 4), half = (L >> 3) & 1;
        for (int kb = 0; kb < 4; ++kb) {
          // canonical bytes: 2 windows per byte; k-block kb covers windows 8kb..8kb+7 = bytes 4kb..4kb+3
          const uint8_t* lo = &m->tc_meta[(tm * kTileM + row) * meta_ld + tk * (kTileK / 8) + 4 * kb + 2 * half];
          const uint8_t* hi = &m->tc_meta[(tm * kTileM + row + 8) * meta_ld + tk * (kTileK / 8) + 4 * kb + 2 * half];
          meta[L * 4 + kb] = static_cast<uint32_t>(lo[0]) | static_cast<uint32_t>(lo[1]) << 8 |
                             static_cast<uint32_t>(hi[0]) << 16 | static_cast<uint32_t>(hi[1]) << 24;
        }
      }
      uint32_t* info = reinterpret_cast<uint32_t*>(blk + kInfoOff);
      info[0] = pdd_len;
      info[1] = res_cnt;
      // Chains are stored longest first (ties: lower row first).  A decode thread takes the chain at
      // its own index, so the 32 lanes of a warp get chains of similar length and few lanes idle
      // while the longest one finishes.  Which row a chain belongs to is carried by its rho values.
      int order[kTileM];
      uint32_t start[kTileM];
      {
        uint32_t acc = 0;
        for (int r = 0; r < kTileM; ++r) { order[r] = r; start[r] = acc; acc += m->chain_len[t * kTileM + r]; }
        std::stable_sort(order, order + kTileM, [&](int a, int b) {
          return m->chain_len[t * kTileM + a] > m->chain_len[t * kTileM + b];
        });
      }
      uint32_t* hdrs = reinterpret_cast<uint32_t*>(blk + kHdrOff);
      uint8_t* code = blk + kPddOff;
      for (int j = 0; j < kTileM; ++j) {
        const int r = order[j];
        const uint32_t len = m->chain_len[t * kTileM + r];
        hdrs[j] = static_cast<uint32_t>(m->chain_tau0[t * kTileM + r]) | static_cast<uint32_t>(m->chain_rho0[t * kTileM + r]) << 16;
        blk[kLenOff + j] = static_cast<uint8_t>(len);
        if (len) std::memcpy(code, &m->pdd_bytes[pdd_off + start[r]], len);
        code += len;
      }
      uint32_t* res = reinterpret_cast<uint32_t*>(blk + kPddOff + align_up(pdd_len, 4));
      for (uint32_t j = 0; j < res_cnt; ++j)
        res[j] = static_cast<uint32_t>(m->res_rho[res_off + j]) | static_cast<uint32_t>(m->res_val[res_off + j]) << 16;
      off += align_up(bytes, kBlockAlign);
    }
  }
}

}  // namespace tl3
