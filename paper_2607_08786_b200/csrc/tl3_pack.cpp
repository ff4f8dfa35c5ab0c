// Device packer: turns the canonical container into one blob of per-tile blocks, each ready for a
// single bulk copy into shared memory (layout described in tl3_internal.h).
//
// Values and metadata are carried over unchanged (permuted into the image the MMA reads).  The
// Slot-Filling layer is re-paired and its PDD chains re-cut for the 32 banks of shared memory:
// the canonical container pairs the i-th surplus element with the i-th empty slot in row-major
// order and cuts one chain per tile row, which makes the 32 lanes of a decode warp touch random
// banks.  Here both streams are ordered bank-major -- a slot's coordinate is
//     u = bank << 8 | slot-in-window << 7 | row,      bank = word of the 128-byte swizzled row
// -- the i-th surplus element in that order is parked in the i-th selected empty slot in that
// order, and the pairs whose empty slot lies in bank b are cut into four chains of equal count.
// Lane l of a decode warp
// takes a chain of bank l, so its loads and stores in W_t never collide with another lane's, and
// its stores in W_r land in bank l or a neighbour.  It is the same format (Sec. 3.2: values parked
// in empty slots, 16-bit absolute starts, 4-bit delta pairs, dummy points, Residual list) over a
// different enumeration of the tile's slots.  Kept values, metadata and the canonical Residual
// elements are carried over as they are; of the canonical parked elements, those that do not fit
// the code words of their chain (at most three) become Residual entries of the device image.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <thread>
#include <vector>

#include "tl3_internal.h"

namespace tl3 {

static inline uint32_t align_up(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

static inline uint32_t block_bytes(uint32_t pdd_len, uint32_t res_cnt) {
  return align_up(kPddOff + align_up(pdd_len, 4) + 4 * res_cnt, 16);
}

// slot position pos = row * 64 + 2 * window + slot-in-window  <->  bank-major coordinate u
static inline uint32_t u_of_pos(uint32_t pos) {
  const uint32_t r = pos >> 6, q = (pos >> 1) & 31u, s = pos & 1u;
  const uint32_t bank = (((q >> 2) ^ (r & 7u)) << 2) | (q & 3u);
  return (bank << 8) | (s << 7) | r;
}
static inline uint32_t pos_of_u(uint32_t u) {
  const uint32_t r = u & 127u, s = (u >> 7) & 1u, bank = u >> 8;
  const uint32_t q = (((bank >> 2) ^ (r & 7u)) << 2) | (bank & 3u);
  return r * 64u + 2u * q + s;
}
// byte offset of slot u in the 128-byte-swizzled K-major image (row pitch 128 B)
static inline uint32_t image_offset(uint32_t u) { return ((u & 127u) << 7) | ((u >> 6) & 0x7Eu); }

namespace {

constexpr int kSlots = kTileM * kH;      // 8192
constexpr int kChains = 128;             // four per bank
// (How long a chain may get is decided per tile in build_tile.  Measured on 20480 x 5120, N = 16,
// with chains of any length 32.2 us, cut after 16 / 14 / 12 / 10 / 8 delta bytes 31.4 / 31.5 /
// 30.1 / 30.9 / 31.5 us: the MMA of a tile waits for its slowest chain, while Residual entries are
// scattered by whichever lane is free.)

struct TileCode {
  uint32_t pdd_len = 0, res_cnt = 0, real_bytes = 0;        // real_bytes: delta bytes that move a value
  uint16_t vals[kSlots];                 // by pos; parked values removed, then re-parked
  uint32_t hdr[kChains];                 // by chain c (u order): u_tau0 | u_rho0 << 16
  uint8_t len[kChains];
  uint32_t code_off[kChains];
  std::vector<uint8_t> code;             // chain after chain in u order
  std::vector<uint32_t> res;             // u_rho | value << 16
};

// Re-pairs and re-chains tile (tm, tk).
void build_tile(const tl3_matrix* m, int64_t tm, int64_t tk, TileCode& tc) {
  const int64_t t = tm * m->tiles_k + tk;
  const int64_t half_ld = m->K_pad / 2;
  for (int r = 0; r < kTileM; ++r)
    std::memcpy(&tc.vals[r * kH], &m->tc_vals[(tm * kTileM + r) * half_ld + tk * kH], kH * sizeof(uint16_t));
  // the parked elements of the canonical chains: value, and where it belongs (by u)
  static thread_local std::vector<uint16_t> sval(kSlots);
  static thread_local std::vector<uint8_t> sflag(kSlots);
  std::fill(sflag.begin(), sflag.end(), 0);
  uint32_t n_pairs = 0;
  const uint32_t pdd_off = m->tile_dir[t * 4];
  uint32_t byte_at = pdd_off;
  auto take = [&](uint32_t tau, uint32_t rho) {
    const uint32_t ur = u_of_pos(rho);
    sval[ur] = tc.vals[tau];
    sflag[ur] = 1;
    tc.vals[tau] = 0;
    ++n_pairs;
  };
  for (int r = 0; r < kTileM; ++r) {
    const uint32_t len = m->chain_len[t * kTileM + r];
    uint32_t tau = m->chain_tau0[t * kTileM + r], rho = m->chain_rho0[t * kTileM + r];
    if (tau != 0xFFFFu) {
      take(tau, rho);
      for (uint32_t k = 0; k < len; ++k) {
        const uint32_t b = m->pdd_bytes[byte_at + k], dt = b & 15u, dr = b >> 4;
        tau += dt;
        rho += dr;
        if (dt && dr) take(tau, rho);
      }
    }
    byte_at += len;
  }
  // Empty slots in u order (every slot whose value is zero: kept values are non-zero), counted per
  // bank.  n_pairs <= their number (the canonical encoder parked each element in an empty slot).
  // Bank b gets a share of the parked elements proportional to its empty slots; its empty slots
  // are cut into four runs of equal count, and run q uses its first quota(b)/4 slots.  So the
  // parked elements spread evenly over the tile however many empty slots stay unused, every
  // chain is a dense run of empty slots (small deltas), and the four chains of a bank are equally
  // long.
  uint32_t cand_in_bank[32];
  uint32_t n_cand = 0;
  static thread_local std::vector<uint16_t> cand;         // empty slots, in u order
  cand.clear();
  for (int b = 0; b < 32; ++b) {
    uint32_t n = 0;
    for (uint32_t u = 256u * b; u < 256u * b + 256u; ++u)
      if ((tc.vals[pos_of_u(u)] & 0x7FFFu) == 0) { cand.push_back(static_cast<uint16_t>(u)); ++n; }
    cand_in_bank[b] = n;
    n_cand += n;
  }
  n_pairs = 0;
  for (int u = 0; u < kSlots; ++u) n_pairs += sflag[u];
  static thread_local std::vector<uint16_t> sel;          // selected empty slots, in u order
  sel.clear();
  uint32_t sel_in_chain[kChains];
  {
    uint64_t cum = 0;
    size_t base = 0;                      // first candidate of the bank
    uint32_t carry = 0;
    for (int b = 0; b < 32; ++b) {
      const uint64_t lo = n_cand ? cum * n_pairs / n_cand : 0;
      cum += cand_in_bank[b];
      const uint64_t hi = n_cand ? cum * n_pairs / n_cand : 0;
      const uint32_t n_b = static_cast<uint32_t>(hi - lo), N_b = cand_in_bank[b];
      for (uint32_t q = 0; q < 4; ++q) {
        const uint32_t first = N_b * q / 4, size = N_b * (q + 1) / 4 - first;
        const uint32_t want = n_b * (q + 1) / 4 - n_b * q / 4 + carry;
        const uint32_t take = want < size ? want : size;
        carry = want - take;
        for (uint32_t i = 0; i < take; ++i) sel.push_back(cand[base + first + i]);
        sel_in_chain[4 * b + q] = take;
      }
      base += N_b;
    }
  }
  // Pairs: the i-th selected empty slot takes the i-th surplus element (both in u order).
  static thread_local std::vector<uint16_t> sur;          // surplus elements, in u order
  sur.clear();
  for (uint32_t u = 0; u < static_cast<uint32_t>(kSlots); ++u)
    if (sflag[u]) sur.push_back(static_cast<uint16_t>(u));
  const size_t n_use = sel.size() < sur.size() ? sel.size() : sur.size();
  // Chains: one per run, so the four warps of a decode group finish a tile at about the same
  // time.  Every chain of a tile gets the same number of code words, n_words <= 3 (zero bytes pad
  // the shorter ones); what a run holds beyond 4 * n_words delta bytes travels as Residual
  // entries.  n_words is the count that makes the block smallest (512 bytes per code word against
  // 4 bytes per Residual entry): three at 50 % sparsity, one or two where few elements are parked.
  auto delta_bytes = [](uint32_t gt, uint32_t gr) { return (gt - 1) / 15 + (gr - 1) / 15 + 1; };
  uint32_t beyond[4] = {0, 0, 0, 0};      // entries whose last delta byte lies beyond 0, 4, 8, 12 bytes
  {
    size_t i = 0;
    for (int c = 0; c < kChains; ++c) {
      uint32_t end = 0;
      for (uint32_t k = 0; k < sel_in_chain[c] && i < n_use; ++k, ++i) {
        if (k == 0) continue;             // the first pair of a chain sits in its header
        end += delta_bytes(static_cast<uint32_t>(sel[i] - sel[i - 1]), static_cast<uint32_t>(sur[i] - sur[i - 1]));
        for (int w = 0; w < 4; ++w) beyond[w] += end > 4u * w;
      }
    }
  }
  uint32_t n_words = 0;
  for (uint32_t w = 1; w < 4; ++w)
    if (512u * w + 4u * beyond[w] < 512u * n_words + 4u * beyond[n_words]) n_words = w;
  const uint32_t cap = 4u * n_words;
  tc.code.clear();
  tc.res.clear();
  tc.real_bytes = 0;
  {
    size_t i = 0;
    for (int c = 0; c < kChains; ++c) {
      tc.hdr[c] = 0xFFFFFFFFu;
      tc.len[c] = 0;
      tc.code_off[c] = static_cast<uint32_t>(tc.code.size());
      uint32_t n_bytes = 0;
      bool cut = false;
      for (uint32_t k = 0; k < sel_in_chain[c] && i < n_use; ++k, ++i) {
        const uint32_t u = sel[i], r_u = sur[i];
        const uint16_t v = sval[r_u];
        if (k == 0) {
          tc.hdr[c] = u | r_u << 16;
        } else {
          uint32_t gt = u - sel[i - 1], gr = r_u - sur[i - 1];
          const uint32_t need = delta_bytes(gt, gr);
          if (cut || n_bytes + need > cap) {            // the chain is full: the rest of its run goes to the Residual list
            cut = true;
            tc.res.push_back(r_u | static_cast<uint32_t>(v) << 16);
            continue;
          }
          while (gt > 15) { tc.code.push_back(0x0F); gt -= 15; }     // dummy points (a zero nibble moves nothing)
          while (gr > 15) { tc.code.push_back(0xF0); gr -= 15; }
          tc.code.push_back(static_cast<uint8_t>(gt | gr << 4));
          ++tc.real_bytes;
          n_bytes += need;
        }
        tc.vals[pos_of_u(u)] = v;
      }
      tc.len[c] = static_cast<uint8_t>(n_bytes);
    }
  }
  for (size_t i = n_use; i < sur.size(); ++i)               // none left unless the container had more parked elements than empty slots
    tc.res.push_back(sur[i] | static_cast<uint32_t>(sval[sur[i]]) << 16);
  // canonical Residual entries, in the same coordinate
  const uint32_t res_off = m->tile_dir[t * 4 + 2], res_cnt = m->tile_dir[t * 4 + 3];
  for (uint32_t j = 0; j < res_cnt; ++j)
    tc.res.push_back(u_of_pos(m->res_rho[res_off + j]) | static_cast<uint32_t>(m->res_val[res_off + j]) << 16);
  tc.pdd_len = n_words * 4u * kChains;                      // every chain takes the same number of code words
  tc.res_cnt = static_cast<uint32_t>(tc.res.size());
}

template <class F>
void for_each_tile(const tl3_matrix* m, F&& f) {
  unsigned hw = std::thread::hardware_concurrency();
  const int n_threads = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(hw ? hw : 1, m->n_tiles / 64 + 1)));
  std::atomic<int64_t> next{0};
  auto worker = [&]() {
    std::vector<TileCode> tc(1);
    for (;;) {
      const int64_t t0 = next.fetch_add(16);
      if (t0 >= m->n_tiles) break;
      for (int64_t t = t0; t < std::min<int64_t>(t0 + 16, m->n_tiles); ++t) {
        build_tile(m, t / m->tiles_k, t % m->tiles_k, tc[0]);
        f(t, tc[0]);
      }
    }
  };
  std::vector<std::thread> pool;
  for (int i = 1; i < n_threads; ++i) pool.emplace_back(worker);
  worker();
  for (auto& th : pool) th.join();
}

}  // namespace

// From the per-tile sizes to the layout of the blob and the layer counts of the device image.
// Caller holds layout_mu.
static void finish_device_layout(const tl3_matrix* m, const std::vector<uint32_t>& real_bytes) {
  // layer shares of the device image (what actually streams): elements whose position is PDD-coded,
  // elements that travel as Residual entries, and delta bytes that move nothing (dummy points and
  // the zero bytes that pad every chain of a tile to the same number of code words)
  m->dev_n_res = m->dev_pdd_bytes = 0;
  int64_t real = 0;
  for (int64_t t = 0; t < m->n_tiles; ++t) {
    m->dev_n_res += m->dev_sizes[2 * t + 1];
    m->dev_pdd_bytes += m->dev_sizes[2 * t];
    real += real_bytes[t];
  }
  m->dev_n_sf = m->n_sf + m->n_res - m->dev_n_res;
  m->dev_n_dummy = m->dev_pdd_bytes - real;
  size_t off = 256;
  m->dir_offset = off;
  off += static_cast<size_t>(m->n_tiles) * sizeof(DirEntry);
  off = (off + 255) / 256 * 256;
  m->blocks_offset = off;
  uint32_t max_block = 0;
  for (int64_t t = 0; t < m->n_tiles; ++t) {
    const uint32_t b = block_bytes(m->dev_sizes[2 * t], m->dev_sizes[2 * t + 1]);
    if (b > max_block) max_block = b;
    off += align_up(b, kBlockAlign);
  }
  m->max_block_bytes = max_block;
  m->device_bytes = (off + 255) / 256 * 256;
  m->layout_ready.store(true, std::memory_order_release);
}

size_t plan_device_layout(const tl3_matrix* m) {
  if (m->p.tile_m != kTileM || m->p.tile_k != kTileK) return 0;   // the device image exists for 128 x 128 tiles only
  if (m->layout_ready.load(std::memory_order_acquire)) return m->device_bytes;
  std::lock_guard<std::mutex> lock(m->layout_mu);
  if (m->layout_ready.load(std::memory_order_relaxed)) return m->device_bytes;
  m->dev_sizes.assign(static_cast<size_t>(m->n_tiles) * 2, 0);
  std::vector<uint32_t> real_bytes(static_cast<size_t>(m->n_tiles), 0);
  for_each_tile(m, [&](int64_t t, const TileCode& tc) {
    m->dev_sizes[2 * t] = tc.pdd_len;
    m->dev_sizes[2 * t + 1] = tc.res_cnt;
    real_bytes[t] = tc.real_bytes;
  });
  finish_device_layout(m, real_bytes);
  return m->device_bytes;
}

// The same layout from sizes that were computed elsewhere (the pack kernel's count pass):
// sizes[3 t] = PDD bytes, [3 t + 1] = Residual entries, [3 t + 2] = delta bytes that move a value.
void set_device_layout(const tl3_matrix* m, const uint32_t* sizes) {
  std::lock_guard<std::mutex> lock(m->layout_mu);
  if (m->layout_ready.load(std::memory_order_relaxed)) return;
  m->dev_sizes.assign(static_cast<size_t>(m->n_tiles) * 2, 0);
  std::vector<uint32_t> real_bytes(static_cast<size_t>(m->n_tiles), 0);
  for (int64_t t = 0; t < m->n_tiles; ++t) {
    m->dev_sizes[2 * t] = sizes[3 * t];
    m->dev_sizes[2 * t + 1] = sizes[3 * t + 1];
    real_bytes[t] = sizes[3 * t + 2];
  }
  finish_device_layout(m, real_bytes);
}

// Offsets of the tile blocks and the 256-byte header of a blob (what pack_device_blob writes first).
void blob_header_and_offsets(const tl3_matrix* m, uint8_t* header256, std::vector<unsigned long long>* block_off) {
  std::memset(header256, 0, 256);
  struct { uint32_t magic, version; int64_t M, K, M_pad, K_pad, n_tiles; uint64_t dir_off, blocks_off; uint32_t max_block; } hdr{
      0x33334C54u, 2, m->M, m->K, m->M_pad, m->K_pad, m->n_tiles, m->dir_offset, m->blocks_offset, m->max_block_bytes};
  std::memcpy(header256, &hdr, sizeof(hdr));
  block_off->resize(static_cast<size_t>(m->n_tiles));
  size_t off = m->blocks_offset;
  for (int64_t t = 0; t < m->n_tiles; ++t) {
    (*block_off)[t] = off;
    off += align_up(block_bytes(m->dev_sizes[2 * t], m->dev_sizes[2 * t + 1]), kBlockAlign);
  }
}

void pack_device_blob(const tl3_matrix* m, uint8_t* out) {
  std::memset(out, 0, m->device_bytes);
  // header (informational; the kernel takes its geometry from its arguments)
  struct { uint32_t magic, version; int64_t M, K, M_pad, K_pad, n_tiles; uint64_t dir_off, blocks_off; uint32_t max_block; } hdr{
      0x33334C54u, 2, m->M, m->K, m->M_pad, m->K_pad, m->n_tiles, m->dir_offset, m->blocks_offset, m->max_block_bytes};
  std::memcpy(out, &hdr, sizeof(hdr));
  DirEntry* dir = reinterpret_cast<DirEntry*>(out + m->dir_offset);
  std::vector<size_t> block_off(static_cast<size_t>(m->n_tiles));
  {
    size_t off = m->blocks_offset;
    for (int64_t t = 0; t < m->n_tiles; ++t) {
      block_off[t] = off;
      off += align_up(block_bytes(m->dev_sizes[2 * t], m->dev_sizes[2 * t + 1]), kBlockAlign);
    }
  }
  const int64_t meta_ld = m->K_pad / 8;
  for_each_tile(m, [&](int64_t t, const TileCode& tc) {
    const int64_t tm = t / m->tiles_k, tk = t % m->tiles_k;
    uint8_t* blk = out + block_off[t];
    dir[t] = DirEntry{static_cast<uint32_t>(block_off[t] / 16), block_bytes(tc.pdd_len, tc.res_cnt), tc.pdd_len, tc.res_cnt};
    // values: slot u of the tile at image_offset(u) (row r, 16-byte chunk j -> chunk j ^ (r & 7))
    for (uint32_t pos = 0; pos < static_cast<uint32_t>(kSlots); ++pos)
      std::memcpy(blk + image_offset(u_of_pos(pos)), &tc.vals[pos], 2);
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
    info[0] = tc.pdd_len;
    info[1] = tc.res_cnt;
    // Chain slot w * 32 + l holds the w-th longest of the four chains of bank l (ties: lower u
    // first).  Decode thread j takes slot j (rotated by 32 from tile to tile), so the lanes of a
    // warp sit in 32 different banks and get chains of similar length.
    uint32_t* hdrs = reinterpret_cast<uint32_t*>(blk + kHdrOff);
    int chain_at[kChains];
    for (int bank = 0; bank < 32; ++bank) {
      int cs[4] = {4 * bank, 4 * bank + 1, 4 * bank + 2, 4 * bank + 3};
      std::stable_sort(cs, cs + 4, [&](int a, int b) { return tc.len[a] > tc.len[b]; });
      for (int w = 0; w < 4; ++w) chain_at[w * 32 + bank] = cs[w];
    }
    // code words, transposed: word k of chain slot j at byte (k * 128 + j) * 4, every chain padded
    // with zero bytes (dummy points that move nothing) to the tile's code-word count
    const uint32_t n_words = tc.pdd_len / (4u * kChains);
    uint8_t* code = blk + kPddOff;
    for (int j = 0; j < kChains; ++j) {
      const int c = chain_at[j];
      hdrs[j] = tc.hdr[c];
      for (uint32_t k = 0; k < tc.len[c]; ++k)
        code[((k >> 2) * kChains + static_cast<uint32_t>(j)) * 4u + (k & 3u)] = tc.code[tc.code_off[c] + k];
    }
    info[2] = n_words;
    if (tc.res_cnt) std::memcpy(blk + kPddOff + align_up(tc.pdd_len, 4), tc.res.data(), 4 * static_cast<size_t>(tc.res_cnt));
  });
}

}  // namespace tl3
