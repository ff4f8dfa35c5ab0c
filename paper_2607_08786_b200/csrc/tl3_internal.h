// Internal definitions shared by the host-side and CUDA-side translation units of libtl3.
#pragma once
#include <atomic>
#include <cstdint>
#include <cstddef>
#include <mutex>
#include <vector>

#include "tl3.h"

struct tl3_matrix {
  int64_t M = 0, K = 0, M_pad = 0, K_pad = 0;
  int64_t tiles_m = 0, tiles_k = 0, n_tiles = 0;
  tl3_params p{128, 128, 15};

  // canonical container (Sec. 3.2)
  std::vector<uint16_t> tc_vals;
  std::vector<uint8_t> tc_meta;
  std::vector<uint16_t> chain_tau0, chain_rho0;
  std::vector<uint8_t> chain_len;
  std::vector<uint8_t> pdd_bytes;
  std::vector<uint32_t> tile_dir;      // 4 per tile: pdd_off, pdd_len, res_off, res_cnt
  std::vector<uint16_t> res_rho, res_val;

  // layer statistics
  int64_t nnz = 0, n_tc = 0, n_sf = 0, n_res = 0, n_dummy = 0, n_slots_unused = 0;

  // device binding (filled by tl3_upload)
  void* dptr = nullptr;
  // device copies of the canonical arrays between tl3_plan_device and tl3_upload_device (one
  // cudaMalloc, released by tl3_upload_device or tl3_free through `release_device_canon`)
  void* device_canon = nullptr;             // a tl3::DeviceCanon
  void (*release_device_canon)(void*) = nullptr;
  // false for a handle made by tl3_encode_device_only: the nine arrays above are empty, the
  // container lives on the device until tl3_upload_device has packed it, and `canon_bytes` keeps
  // the sizes the arrays would have
  bool host_arrays = true;
  int64_t canon_bytes = 0;
  // Layout of the device image, computed on first use (tl3_device_bytes, tl3_pack, tl3_upload,
  // tl3_stats) under `layout_mu`, so that calls that take a const handle may share it between
  // threads; `layout_ready` is set last.
  mutable std::mutex layout_mu;
  mutable std::atomic<bool> layout_ready{false};
  mutable size_t device_bytes = 0;
  mutable uint32_t max_block_bytes = 0;
  mutable std::vector<uint32_t> dev_sizes;   // per tile: PDD bytes and Residual entries of the device image
  mutable size_t dir_offset = 0, blocks_offset = 0;
  // layer counts of the device image (set with the layout)
  mutable int64_t dev_n_sf = 0, dev_n_res = 0, dev_n_dummy = 0, dev_pdd_bytes = 0;
  // compact form of the canonical Residual layer (computed on first use, under layout_mu)
  mutable std::atomic<bool> compact_ready{false};
  mutable std::vector<uint32_t> res_dir;
  mutable std::vector<uint16_t> res_list;
  mutable std::vector<uint8_t> res_mask;
  mutable std::atomic<bool> val_compact_ready{false};      // compact form of the value array (tl3_canonical 12-14)
  mutable std::vector<uint32_t> val_dir;
  mutable std::vector<uint16_t> val_pack;
  mutable std::vector<uint8_t> val_mask;

  // last launch geometry (reporting only)
  mutable std::atomic<int> last_ctas{0}, last_stages{0}, last_smem{0};
};

namespace tl3 {

// The canonical arrays on the device (between an encode or a copy there and tl3_upload_device).
struct DeviceCanon {
  const uint16_t* tc_vals; const uint8_t* tc_meta; const uint16_t* chain_tau0; const uint16_t* chain_rho0;
  const uint8_t* chain_len; const uint8_t* pdd_bytes; const uint32_t* tile_dir; const uint16_t* res_rho; const uint16_t* res_val;
  void* alloc[2];                            // what to cudaFree
};

// ---- device blob layout ------------------------------------------------------------------
// [0, 256)                 header (magic, shape; informational)
// [dir_offset, ...)        one DirEntry per tile
// [blocks_offset, ...)     tile blocks, each 128-byte aligned, row-tile-major
//
// Tile block (tile 128 x 128, H = 64 value slots per row):
//   +0      values   128 rows x 128 B, the K-major 128-byte-swizzled image the MMA descriptor
//                    reads: 16-byte chunk j of row r sits at chunk (j ^ (r & 7)).  Kept values are
//                    those of the canonical container; parked values are re-parked bank-major
//                    (see tl3_pack.cpp)
//   +16384  metadata 128 x 16 B: word kb of entry L is the TMEM word of lane L for k-block kb:
//                    bits 0-15 = nibbles of windows 8kb+4h .. 8kb+4h+3 of row (L&7)+16(L>>4),
//                    bits 16-31 = the same windows of that row + 8, with h = (L>>3)&1
//   +18432  u32[4]: pdd_len, res_cnt, n_words, 0
//   +18448  chain starts u32[128]: tau0 | rho0 << 16 (0xFFFFFFFF = empty chain) in the bank-major
//           slot coordinate u = bank << 8 | slot-in-window << 7 | row; chain slot w * 32 + l holds
//           the w-th longest of the four chains whose empty slots lie in bank l
//   +18960  PDD code words, transposed: word k (delta bytes 4k..4k+3) of chain slot j at byte
//           (k * 128 + j) * 4; every chain of the tile has n_words <= 3 of them, padded with zero
//           bytes (dummy points); pdd_len = 512 * n_words
//   +...    Residual entries u32[res_cnt]: u of the element | value << 16, padded to 16 bytes
constexpr int kTileM = 128, kTileK = 128, kH = 64;
constexpr uint32_t kValsBytes = 16384, kMetaOff = 16384, kMetaBytes = 2048;
constexpr uint32_t kInfoOff = 18432, kHdrOff = 18448, kPddOff = 18960;
constexpr uint32_t kBlockAlign = 128;

struct DirEntry {
  uint32_t off16;     // block offset from the blob base, in 16-byte units
  uint32_t bytes;     // block size (multiple of 16)
  uint32_t pdd_len;
  uint32_t res_cnt;
};

size_t plan_device_layout(const tl3_matrix* m);           // fills device_bytes, offsets, max block (once, thread-safe)
void pack_device_blob(const tl3_matrix* m, uint8_t* out); // out: device_bytes bytes, host
void set_device_layout(const tl3_matrix* m, const uint32_t* sizes);   // layout from per-tile sizes computed on the GPU
void blob_header_and_offsets(const tl3_matrix* m, uint8_t* header256, std::vector<unsigned long long>* block_off);

void set_cuda_error(int e);

}  // namespace tl3
