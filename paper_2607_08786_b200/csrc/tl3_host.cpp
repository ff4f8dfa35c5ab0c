// Host side of libtl3: encoder, decoder, container access, persistence.
//
// The encoder builds the three layers of Sec. 3.2 tile by tile.  Row-tiles are independent, so
// they are encoded by a pool of threads and stitched together in order afterwards.
#include <algorithm>
#include <array>
#include <atomic>
#include <cstring>
#include <new>
#include <thread>

#include "tl3_internal.h"

namespace {

// Classification of one window of four consecutive weights by its non-zero pattern
// (bit i set = weight i non-zero).  Sec. 3.2, Sparse-TC layer: two weights stay, each with a
// 2-bit in-window index; a window short of two weights leaves empty slots, a window with more
// than two has surplus weights.
struct WindowClass {
  uint8_t idx[2];       // in-window index carried by slot 0 and slot 1 (idx[0] < idx[1])
  uint8_t kept_mask;    // bit s set: slot s holds a weight of this window
  uint8_t n_surplus;
  uint8_t surplus[2];   // in-window indices (2 or 3) of the surplus weights
};

constexpr WindowClass classify(unsigned pattern) {
  WindowClass w{};
  int pos[4] = {0, 0, 0, 0};
  int n = 0;
  for (int i = 0; i < 4; ++i)
    if (pattern >> i & 1u) pos[n++] = i;
  const int kept = n < 2 ? n : 2;
  // slots carry the kept positions plus, if fewer than two are kept, the lowest unused ones
  bool used[4] = {false, false, false, false};
  for (int j = 0; j < kept; ++j) used[pos[j]] = true;
  int chosen[2] = {0, 0};
  int c = 0;
  for (int j = 0; j < kept; ++j) chosen[c++] = pos[j];
  for (int i = 0; i < 4 && c < 2; ++i)
    if (!used[i]) { chosen[c++] = i; }
  const int lo = chosen[0] < chosen[1] ? chosen[0] : chosen[1];
  const int hi = chosen[0] < chosen[1] ? chosen[1] : chosen[0];
  w.idx[0] = static_cast<uint8_t>(lo);
  w.idx[1] = static_cast<uint8_t>(hi);
  w.kept_mask = static_cast<uint8_t>((used[lo] ? 1 : 0) | (used[hi] ? 2 : 0));
  w.n_surplus = static_cast<uint8_t>(n - kept);
  for (int j = kept; j < n; ++j) w.surplus[j - kept] = static_cast<uint8_t>(pos[j]);
  return w;
}

constexpr std::array<WindowClass, 16> make_table() {
  std::array<WindowClass, 16> t{};
  for (unsigned p = 0; p < 16; ++p) t[p] = classify(p);
  return t;
}
constexpr std::array<WindowClass, 16> kWindow = make_table();

inline bool nonzero(uint16_t h) { return (h & 0x7FFFu) != 0; }

struct RowTileOut {
  std::vector<uint8_t> pdd;
  std::vector<uint32_t> res;                 // rho | value << 16
  std::vector<uint32_t> dir;                 // per tile: pdd_off (local), pdd_len, res_off (local), res_cnt
  int64_t nnz = 0, n_tc = 0, n_sf = 0, n_res = 0, n_dummy = 0, n_unused = 0;
};

void encode_row_tile(const uint16_t* W, tl3_matrix& m, int64_t tm, RowTileOut& out) {
  const int TM = m.p.tile_m, TK = m.p.tile_k, H = TK / 2, QW = TK / 4, maxd = m.p.maxd;
  const int64_t half_ld = m.K_pad / 2, meta_ld = m.K_pad / 8;
  std::vector<uint32_t> surplus;             // rho | value << 16, ascending rho
  std::vector<uint16_t> holes;               // tau, ascending
  std::vector<uint32_t> residual;
  surplus.reserve(static_cast<size_t>(TM) * H);
  holes.reserve(static_cast<size_t>(TM) * H);
  out.dir.assign(static_cast<size_t>(m.tiles_k) * 4, 0);

  for (int64_t tk = 0; tk < m.tiles_k; ++tk) {
    surplus.clear();
    holes.clear();
    residual.clear();
    // pass 1: Sparse-TC split, collect surplus weights and empty slots
    for (int r = 0; r < TM; ++r) {
      const int64_t row = tm * TM + r;
      if (row >= m.M) {                       // padding rows: all windows empty
        for (int q = 0; q < QW; ++q) {
          const int64_t gq = tk * QW + q;
          m.tc_meta[row * meta_ld + gq / 2] |= static_cast<uint8_t>((gq & 1) ? 0x40 : 0x04);
          holes.push_back(static_cast<uint16_t>(r * H + 2 * q));
          holes.push_back(static_cast<uint16_t>(r * H + 2 * q + 1));
        }
        continue;
      }
      const uint16_t* wrow = W + row * m.K;
      for (int q = 0; q < QW; ++q) {
        const int64_t gq = tk * QW + q, col0 = tk * TK + 4 * q;
        uint16_t w[4];
        unsigned pattern = 0;
        for (int i = 0; i < 4; ++i) {
          w[i] = (col0 + i < m.K) ? wrow[col0 + i] : uint16_t{0};
          pattern |= static_cast<unsigned>(nonzero(w[i])) << i;
        }
        const WindowClass& wc = kWindow[pattern];
        const uint8_t nib = static_cast<uint8_t>(wc.idx[0] | wc.idx[1] << 2);
        m.tc_meta[row * meta_ld + gq / 2] |= static_cast<uint8_t>((gq & 1) ? nib << 4 : nib);
        for (int s = 0; s < 2; ++s) {
          if (wc.kept_mask >> s & 1) {
            m.tc_vals[row * half_ld + 2 * gq + s] = w[wc.idx[s]];
            ++out.n_tc;
          } else {
            holes.push_back(static_cast<uint16_t>(r * H + 2 * q + s));
          }
        }
        for (int j = 0; j < wc.n_surplus; ++j) {
          const uint32_t rho = static_cast<uint32_t>(r * H + 2 * q + (wc.surplus[j] - 2));
          surplus.push_back(rho | static_cast<uint32_t>(w[wc.surplus[j]]) << 16);
        }
        out.nnz += __builtin_popcount(pattern);
      }
    }
    // pass 2: i-th surplus weight <-> i-th empty slot, coded as one PDD chain per tile row
    const size_t P = std::min(surplus.size(), holes.size());
    for (size_t i = P; i < surplus.size(); ++i) residual.push_back(surplus[i]);
    out.n_unused += static_cast<int64_t>(holes.size() - P);
    const int64_t tile = tm * m.tiles_k + tk;
    const size_t pdd_begin = out.pdd.size();
    auto park = [&](uint32_t tau, uint32_t sv) {
      m.tc_vals[(tm * TM + tau / H) * half_ld + tk * H + tau % H] = static_cast<uint16_t>(sv >> 16);
      ++out.n_sf;
    };
    size_t i = 0;
    for (int r = 0; r < TM; ++r) {
      const int64_t ch = tile * TM + r;
      m.chain_tau0[ch] = 0xFFFF;
      m.chain_rho0[ch] = 0xFFFF;
      m.chain_len[ch] = 0;
      const uint32_t row_end = static_cast<uint32_t>((r + 1) * H);
      if (i >= P || (surplus[i] & 0xFFFFu) >= row_end) continue;
      uint32_t tau = holes[i], rho = surplus[i] & 0xFFFFu;
      m.chain_tau0[ch] = static_cast<uint16_t>(tau);
      m.chain_rho0[ch] = static_cast<uint16_t>(rho);
      park(tau, surplus[i]);
      ++i;
      int len = 0;
      bool full = false;
      for (; i < P && (surplus[i] & 0xFFFFu) < row_end; ++i) {
        const uint32_t ntau = holes[i], nrho = surplus[i] & 0xFFFFu;
        if (!full) {
          const uint32_t dt = ntau - tau, dr = nrho - rho;
          const int dummies_t = static_cast<int>((dt - 1) / maxd), dummies_r = static_cast<int>((dr - 1) / maxd);
          if (len + dummies_t + dummies_r + 1 > 255) {
            full = true;
          } else {
            out.pdd.insert(out.pdd.end(), dummies_t, static_cast<uint8_t>(maxd));
            out.pdd.insert(out.pdd.end(), dummies_r, static_cast<uint8_t>(maxd << 4));
            out.pdd.push_back(static_cast<uint8_t>((dt - dummies_t * maxd) | (dr - dummies_r * maxd) << 4));
            out.n_dummy += dummies_t + dummies_r;
            len += dummies_t + dummies_r + 1;
            tau = ntau;
            rho = nrho;
            park(tau, surplus[i]);
            continue;
          }
        }
        residual.push_back(surplus[i]);       // the chain is full: rest of this row -> Residual
        ++out.n_unused;
      }
      m.chain_len[ch] = static_cast<uint8_t>(len);
    }
    std::sort(residual.begin(), residual.end(),
              [](uint32_t a, uint32_t b) { return (a & 0xFFFFu) < (b & 0xFFFFu); });
    out.dir[tk * 4 + 0] = static_cast<uint32_t>(pdd_begin);
    out.dir[tk * 4 + 1] = static_cast<uint32_t>(out.pdd.size() - pdd_begin);
    out.dir[tk * 4 + 2] = static_cast<uint32_t>(out.res.size());
    out.dir[tk * 4 + 3] = static_cast<uint32_t>(residual.size());
    out.res.insert(out.res.end(), residual.begin(), residual.end());
    out.n_res += static_cast<int64_t>(residual.size());
  }
}

bool valid_params(const tl3_params& p) {
  return p.tile_m > 0 && p.tile_k > 0 && p.tile_k % 8 == 0 &&
         static_cast<int64_t>(p.tile_m) * p.tile_k / 2 <= 65535 && p.maxd >= 1 && p.maxd <= 15;
}

void set_shape(tl3_matrix& m, int64_t M, int64_t K, const tl3_params& p) {
  m.M = M; m.K = K; m.p = p;
  m.tiles_m = (M + p.tile_m - 1) / p.tile_m;
  m.tiles_k = (K + p.tile_k - 1) / p.tile_k;
  m.M_pad = m.tiles_m * p.tile_m;
  m.K_pad = m.tiles_k * p.tile_k;
  m.n_tiles = m.tiles_m * m.tiles_k;
}

// Structural check of a container (sizes and ranges) so that decode and pack never read out of
// bounds whatever deserialize was given.
bool consistent(const tl3_matrix& m) {
  if (!valid_params(m.p) || m.M <= 0 || m.K <= 0) return false;
  const size_t slots = static_cast<size_t>(m.M_pad) * static_cast<size_t>(m.K_pad) / 2;
  if (m.tc_vals.size() != slots || m.tc_meta.size() != slots / 4) return false;
  const size_t chains = static_cast<size_t>(m.n_tiles) * m.p.tile_m;
  if (m.chain_tau0.size() != chains || m.chain_rho0.size() != chains || m.chain_len.size() != chains) return false;
  if (m.tile_dir.size() != static_cast<size_t>(m.n_tiles) * 4 || m.res_rho.size() != m.res_val.size()) return false;
  const uint32_t tile_slots = static_cast<uint32_t>(m.p.tile_m * (m.p.tile_k / 2));
  for (int64_t t = 0; t < m.n_tiles; ++t) {
    const uint32_t* d = &m.tile_dir[t * 4];
    if (static_cast<uint64_t>(d[0]) + d[1] > m.pdd_bytes.size()) return false;
    if (static_cast<uint64_t>(d[2]) + d[3] > m.res_rho.size()) return false;
    uint64_t len_sum = 0;
    for (int r = 0; r < m.p.tile_m; ++r) len_sum += m.chain_len[t * m.p.tile_m + r];
    if (len_sum != d[1]) return false;
    // every position a chain reaches lies inside the tile (the device packer and the decoders
    // index with them)
    uint64_t at = d[0];
    for (int r = 0; r < m.p.tile_m; ++r) {
      const size_t c = static_cast<size_t>(t) * m.p.tile_m + r;
      uint32_t tau = m.chain_tau0[c], rho = m.chain_rho0[c];
      const uint32_t len = m.chain_len[c];
      if (tau == 0xFFFFu || rho == 0xFFFFu) {
        if (tau != rho || len != 0) return false;
        continue;
      }
      if (tau >= tile_slots || rho >= tile_slots) return false;
      for (uint32_t k = 0; k < len; ++k) {
        const uint32_t b = m.pdd_bytes[at + k];
        tau += b & 15u;
        rho += b >> 4;
        if (tau >= tile_slots || rho >= tile_slots) return false;
      }
      at += len;
    }
    for (uint32_t j = d[2]; j < d[2] + d[3]; ++j)
      if (m.res_rho[j] >= tile_slots) return false;
  }
  return true;
}

}  // namespace

extern "C" {

int tl3_encode(const uint16_t* W, int64_t M, int64_t K, const tl3_params* params, tl3_matrix** out) {
  if (!W || !out || M <= 0 || K <= 0) return TL3_ERR_INVALID_ARG;
  const tl3_params p = params ? *params : tl3_params{128, 128, 15};
  if (!valid_params(p)) return TL3_ERR_INVALID_ARG;
  tl3_matrix* m = new (std::nothrow) tl3_matrix();
  if (!m) return TL3_ERR_NO_MEMORY;
  try {
    set_shape(*m, M, K, p);
    m->tc_vals.assign(static_cast<size_t>(m->M_pad) * m->K_pad / 2, 0);
    m->tc_meta.assign(static_cast<size_t>(m->M_pad) * m->K_pad / 8, 0);
    const size_t chains = static_cast<size_t>(m->n_tiles) * p.tile_m;
    m->chain_tau0.resize(chains);
    m->chain_rho0.resize(chains);
    m->chain_len.resize(chains);
    m->tile_dir.resize(static_cast<size_t>(m->n_tiles) * 4);

    std::vector<RowTileOut> parts(static_cast<size_t>(m->tiles_m));
    unsigned hw = std::thread::hardware_concurrency();
    const int n_threads = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(hw ? hw : 1, m->tiles_m)));
    std::atomic<int64_t> next{0};
    auto worker = [&]() {
      for (int64_t tm = next.fetch_add(1); tm < m->tiles_m; tm = next.fetch_add(1))
        encode_row_tile(W, *m, tm, parts[static_cast<size_t>(tm)]);
    };
    std::vector<std::thread> pool;
    for (int t = 1; t < n_threads; ++t) pool.emplace_back(worker);
    worker();
    for (auto& th : pool) th.join();

    // stitch the per-row-tile pieces in order
    size_t pdd_total = 0, res_total = 0;
    for (const auto& pt : parts) { pdd_total += pt.pdd.size(); res_total += pt.res.size(); }
    m->pdd_bytes.reserve(pdd_total);
    m->res_rho.reserve(res_total);
    m->res_val.reserve(res_total);
    for (int64_t tm = 0; tm < m->tiles_m; ++tm) {
      const RowTileOut& pt = parts[static_cast<size_t>(tm)];
      const uint32_t pdd_base = static_cast<uint32_t>(m->pdd_bytes.size());
      const uint32_t res_base = static_cast<uint32_t>(m->res_rho.size());
      for (int64_t tk = 0; tk < m->tiles_k; ++tk) {
        uint32_t* d = &m->tile_dir[(tm * m->tiles_k + tk) * 4];
        d[0] = pdd_base + pt.dir[tk * 4 + 0];
        d[1] = pt.dir[tk * 4 + 1];
        d[2] = res_base + pt.dir[tk * 4 + 2];
        d[3] = pt.dir[tk * 4 + 3];
      }
      m->pdd_bytes.insert(m->pdd_bytes.end(), pt.pdd.begin(), pt.pdd.end());
      for (uint32_t e : pt.res) {
        m->res_rho.push_back(static_cast<uint16_t>(e & 0xFFFFu));
        m->res_val.push_back(static_cast<uint16_t>(e >> 16));
      }
      m->nnz += pt.nnz; m->n_tc += pt.n_tc; m->n_sf += pt.n_sf; m->n_res += pt.n_res;
      m->n_dummy += pt.n_dummy; m->n_slots_unused += pt.n_unused;
    }
  } catch (const std::bad_alloc&) {
    delete m;
    return TL3_ERR_NO_MEMORY;
  }
  *out = m;
  return TL3_OK;
}

int tl3_decode(const tl3_matrix* m, uint16_t* W_out) {
  if (!m || !W_out) return TL3_ERR_INVALID_ARG;
  if (!m->host_arrays) return TL3_ERR_UNSUPPORTED;               // tl3_encode_device_only: the container is not on the host
  if (!consistent(*m)) return TL3_ERR_BAD_CONTAINER;
  const int TM = m->p.tile_m, TK = m->p.tile_k, H = TK / 2;
  const int64_t half_ld = m->K_pad / 2, meta_ld = m->K_pad / 8;
  const uint32_t tile_slots = static_cast<uint32_t>(TM * H);
  std::memset(W_out, 0, static_cast<size_t>(m->M) * m->K * sizeof(uint16_t));
  std::vector<uint16_t> Wt(tile_slots);
  bool bad = false;
  auto place = [&](int64_t tm, int64_t tk, uint32_t rho, uint16_t v) {
    // offset_r names a slot of W_r: row rho / H, column 4 * (window) + 2 + parity
    const int64_t row = tm * TM + rho / H, col = tk * TK + 4 * ((rho % H) / 2) + 2 + (rho & 1);
    if (!nonzero(v)) return;
    if (row >= m->M || col >= m->K || W_out[row * m->K + col] != 0) { bad = true; return; }
    W_out[row * m->K + col] = v;
  };
  for (int64_t tm = 0; tm < m->tiles_m; ++tm) {
    for (int64_t tk = 0; tk < m->tiles_k; ++tk) {
      const int64_t tile = tm * m->tiles_k + tk;
      for (int r = 0; r < TM; ++r)
        std::memcpy(&Wt[static_cast<size_t>(r) * H], &m->tc_vals[(tm * TM + r) * half_ld + tk * H], H * sizeof(uint16_t));
      // Algorithm 1, chain by chain
      const uint8_t* code = m->pdd_bytes.data() + m->tile_dir[tile * 4];
      for (int t = 0; t < TM; ++t) {
        const int64_t ch = tile * TM + t;
        const int len = m->chain_len[ch];
        uint32_t off_t = m->chain_tau0[ch], off_r = m->chain_rho0[ch];
        if (off_t == 0xFFFF && off_r == 0xFFFF && len == 0) continue;
        if (off_t >= tile_slots || off_r >= tile_slots) return TL3_ERR_BAD_CONTAINER;
        place(tm, tk, off_r, Wt[off_t]);
        Wt[off_t] = 0;
        for (int i = 0; i < len; ++i) {
          const uint32_t dt = code[i] & 0xFu, dr = code[i] >> 4;
          off_t += dt;
          off_r += dr;
          if (dt == 0 || dr == 0) continue;                 // dummy point
          if (off_t >= tile_slots || off_r >= tile_slots) return TL3_ERR_BAD_CONTAINER;
          place(tm, tk, off_r, Wt[off_t]);
          Wt[off_t] = 0;
        }
        code += len;
      }
      const uint32_t r0 = m->tile_dir[tile * 4 + 2], rn = m->tile_dir[tile * 4 + 3];
      for (uint32_t j = r0; j < r0 + rn; ++j) place(tm, tk, m->res_rho[j], m->res_val[j]);
      // what is left in W_t is the Sparse-TC layer
      for (int r = 0; r < TM; ++r) {
        const int64_t row = tm * TM + r;
        for (int s = 0; s < H; ++s) {
          const uint16_t v = Wt[static_cast<size_t>(r) * H + s];
          if (!nonzero(v)) continue;
          const int64_t gq = tk * (TK / 4) + s / 2;
          const uint8_t byte = m->tc_meta[row * meta_ld + gq / 2];
          const unsigned nib = (gq & 1) ? byte >> 4 : byte & 0xFu;
          const unsigned idx = (s & 1) ? nib >> 2 : nib & 3u;
          const int64_t col = 4 * gq + idx;
          if (row >= m->M || col >= m->K || W_out[row * m->K + col] != 0) { bad = true; continue; }
          W_out[row * m->K + col] = v;
        }
      }
    }
  }
  return bad ? TL3_ERR_BAD_CONTAINER : TL3_OK;
}

// Compact form of the Residual layer: per tile the smaller of the two-byte position list and a
// bitmap over the tile's tile_m * H positions of W_r (bit rho % 8 of byte rho / 8).  Derived from
// res_rho on first use.
static void ensure_compact(const tl3_matrix* m) {
  if (m->compact_ready.load(std::memory_order_acquire)) return;
  std::lock_guard<std::mutex> lock(m->layout_mu);
  if (m->compact_ready.load(std::memory_order_relaxed)) return;
  const size_t mask_bytes = (static_cast<size_t>(m->p.tile_m) * (m->p.tile_k / 2) + 7) / 8;
  m->res_dir.assign(static_cast<size_t>(m->n_tiles) * 2, 0);
  m->res_list.clear();
  m->res_mask.clear();
  for (int64_t t = 0; t < m->n_tiles; ++t) {
    const uint32_t off = m->tile_dir[t * 4 + 2], cnt = m->tile_dir[t * 4 + 3];
    if (mask_bytes < 2u * static_cast<size_t>(cnt)) {
      m->res_dir[2 * t] = 1;
      m->res_dir[2 * t + 1] = static_cast<uint32_t>(m->res_mask.size());
      m->res_mask.resize(m->res_mask.size() + mask_bytes, 0);
      uint8_t* bits = m->res_mask.data() + m->res_dir[2 * t + 1];
      for (uint32_t j = off; j < off + cnt; ++j) bits[m->res_rho[j] >> 3] |= static_cast<uint8_t>(1u << (m->res_rho[j] & 7u));
    } else {
      m->res_dir[2 * t] = 0;
      m->res_dir[2 * t + 1] = static_cast<uint32_t>(m->res_list.size());
      m->res_list.insert(m->res_list.end(), m->res_rho.begin() + off, m->res_rho.begin() + off + cnt);
    }
  }
  m->compact_ready.store(true, std::memory_order_release);
}

// Compact form of the value array (Sec. 3.2 stores every slot; Sec. 6 names the empty ones above
// 50 % sparsity): per tile all values, or a bitmap of the occupied slots and their values,
// whichever is smaller.
static void ensure_val_compact(const tl3_matrix* m) {
  if (m->val_compact_ready.load(std::memory_order_acquire)) return;
  std::lock_guard<std::mutex> lock(m->layout_mu);
  if (m->val_compact_ready.load(std::memory_order_relaxed)) return;
  const int64_t H = m->p.tile_k / 2, slots = static_cast<int64_t>(m->p.tile_m) * H, half_ld = m->K_pad / 2;
  const size_t mask_bytes = (static_cast<size_t>(slots) + 7) / 8;
  const int64_t tiles_k = m->K_pad / m->p.tile_k;
  m->val_dir.assign(static_cast<size_t>(m->n_tiles) * 2, 0);
  m->val_pack.clear();
  m->val_mask.clear();
  for (int64_t t = 0; t < m->n_tiles; ++t) {
    const int64_t tm = t / tiles_k, tk = t % tiles_k;
    const uint16_t* base = m->tc_vals.data() + tm * m->p.tile_m * half_ld + tk * H;
    int64_t occupied = 0;
    for (int64_t r = 0; r < m->p.tile_m; ++r)
      for (int64_t h = 0; h < H; ++h) occupied += base[r * half_ld + h] != 0;
    const bool bitmap = mask_bytes < 2u * static_cast<size_t>(slots - occupied);
    m->val_dir[2 * t] = bitmap ? 1u : 0u;
    m->val_dir[2 * t + 1] = static_cast<uint32_t>(m->val_pack.size());
    uint8_t* bits = nullptr;
    if (bitmap) {
      m->val_mask.resize(m->val_mask.size() + mask_bytes, 0);
      bits = m->val_mask.data() + m->val_mask.size() - mask_bytes;
    }
    for (int64_t r = 0; r < m->p.tile_m; ++r)
      for (int64_t h = 0; h < H; ++h) {
        const uint16_t v = base[r * half_ld + h];
        if (!bitmap) { m->val_pack.push_back(v); continue; }
        if (v != 0) {
          const int64_t pos = r * H + h;
          bits[pos >> 3] |= static_cast<uint8_t>(1u << (pos & 7));
          m->val_pack.push_back(v);
        }
      }
  }
  m->val_compact_ready.store(true, std::memory_order_release);
}

int tl3_canonical(const tl3_matrix* m, int which, const void** ptr, size_t* bytes) {
  if (!m || !ptr || !bytes) return TL3_ERR_INVALID_ARG;
  if (!m->host_arrays) return TL3_ERR_UNSUPPORTED;
  if (which >= TL3_RES_DIR && which <= TL3_RES_MASK) ensure_compact(m);
  if (which >= TL3_VAL_DIR && which <= TL3_VAL_MASK) ensure_val_compact(m);
  switch (which) {
    case TL3_VAL_DIR:    *ptr = m->val_dir.data();    *bytes = m->val_dir.size() * 4; break;
    case TL3_VAL_PACK:   *ptr = m->val_pack.data();   *bytes = m->val_pack.size() * 2; break;
    case TL3_VAL_MASK:   *ptr = m->val_mask.data();   *bytes = m->val_mask.size(); break;
    case TL3_RES_DIR:    *ptr = m->res_dir.data();    *bytes = m->res_dir.size() * 4; break;
    case TL3_RES_LIST:   *ptr = m->res_list.data();   *bytes = m->res_list.size() * 2; break;
    case TL3_RES_MASK:   *ptr = m->res_mask.data();   *bytes = m->res_mask.size(); break;
    case TL3_TC_VALS:    *ptr = m->tc_vals.data();    *bytes = m->tc_vals.size() * 2; break;
    case TL3_TC_META:    *ptr = m->tc_meta.data();    *bytes = m->tc_meta.size(); break;
    case TL3_CHAIN_TAU0: *ptr = m->chain_tau0.data(); *bytes = m->chain_tau0.size() * 2; break;
    case TL3_CHAIN_RHO0: *ptr = m->chain_rho0.data(); *bytes = m->chain_rho0.size() * 2; break;
    case TL3_CHAIN_LEN:  *ptr = m->chain_len.data();  *bytes = m->chain_len.size(); break;
    case TL3_PDD_BYTES:  *ptr = m->pdd_bytes.data();  *bytes = m->pdd_bytes.size(); break;
    case TL3_TILE_DIR:   *ptr = m->tile_dir.data();   *bytes = m->tile_dir.size() * 4; break;
    case TL3_RES_RHO:    *ptr = m->res_rho.data();    *bytes = m->res_rho.size() * 2; break;
    case TL3_RES_VAL:    *ptr = m->res_val.data();    *bytes = m->res_val.size() * 2; break;
    default: return TL3_ERR_INVALID_ARG;
  }
  return TL3_OK;
}

static int64_t canonical_bytes(const tl3_matrix* m) {
  return static_cast<int64_t>(m->tc_vals.size() * 2 + m->tc_meta.size() + m->chain_tau0.size() * 2 +
                              m->chain_rho0.size() * 2 + m->chain_len.size() + m->pdd_bytes.size() +
                              m->tile_dir.size() * 4 + m->res_rho.size() * 2 + m->res_val.size() * 2);
}

int tl3_stats(const tl3_matrix* m, tl3_stats_t* out) {
  if (!m || !out) return TL3_ERR_INVALID_ARG;
  out->M = m->M; out->K = m->K; out->M_pad = m->M_pad; out->K_pad = m->K_pad; out->n_tiles = m->n_tiles;
  out->nnz = m->nnz; out->n_tc = m->n_tc; out->n_sf = m->n_sf; out->n_res = m->n_res;
  out->n_dummy = m->n_dummy; out->n_slots_unused = m->n_slots_unused;
  out->device_bytes = static_cast<int64_t>(tl3_device_bytes(m));
  out->dev_n_sf = m->dev_n_sf; out->dev_n_res = m->dev_n_res; out->dev_n_dummy = m->dev_n_dummy;
  out->dev_pdd_bytes = m->dev_pdd_bytes;
  if (!m->host_arrays) {                                           // the sizes of the compact forms need the arrays
    out->canonical_bytes = m->canon_bytes;
    out->canonical_bytes_compact = out->canonical_bytes_compact_all = -1;
    return TL3_OK;
  }
  out->canonical_bytes = canonical_bytes(m);
  ensure_compact(m);
  out->canonical_bytes_compact = out->canonical_bytes - static_cast<int64_t>(m->res_rho.size() * 2) +
                                 static_cast<int64_t>(m->res_dir.size() * 4 + m->res_list.size() * 2 + m->res_mask.size());
  out->dev_n_sf = m->dev_n_sf; out->dev_n_res = m->dev_n_res; out->dev_n_dummy = m->dev_n_dummy;
  out->dev_pdd_bytes = m->dev_pdd_bytes;
  ensure_val_compact(m);
  out->canonical_bytes_compact_all = out->canonical_bytes_compact - static_cast<int64_t>(m->tc_vals.size() * 2) +
                                     static_cast<int64_t>(m->val_dir.size() * 4 + m->val_pack.size() * 2 + m->val_mask.size());
  return TL3_OK;
}

// ---- persistence: header + the nine arrays, each preceded by its byte count ----------------
namespace {
constexpr uint64_t kMagic = 0x31304C33544C33ULL;   // container tag
struct FileHeader {
  uint64_t magic;
  int64_t M, K;
  int32_t tile_m, tile_k, maxd, reserved;
  int64_t stats[6];
};
}  // namespace

int tl3_serialize(const tl3_matrix* m, void* buf, size_t* bytes) {
  if (!m || !bytes) return TL3_ERR_INVALID_ARG;
  if (!m->host_arrays) return TL3_ERR_UNSUPPORTED;
  size_t need = sizeof(FileHeader);
  for (int w = 0; w < 9; ++w) {
    const void* p; size_t n;
    tl3_canonical(m, w, &p, &n);
    need += sizeof(uint64_t) + n;
  }
  if (!buf) { *bytes = need; return TL3_OK; }
  if (*bytes < need) { *bytes = need; return TL3_ERR_INVALID_ARG; }
  uint8_t* o = static_cast<uint8_t*>(buf);
  FileHeader h{kMagic, m->M, m->K, m->p.tile_m, m->p.tile_k, m->p.maxd, 0,
               {m->nnz, m->n_tc, m->n_sf, m->n_res, m->n_dummy, m->n_slots_unused}};
  std::memcpy(o, &h, sizeof(h));
  o += sizeof(h);
  for (int w = 0; w < 9; ++w) {
    const void* p; size_t n;
    tl3_canonical(m, w, &p, &n);
    const uint64_t n64 = n;
    std::memcpy(o, &n64, 8);
    o += 8;
    if (n) std::memcpy(o, p, n);
    o += n;
  }
  *bytes = need;
  return TL3_OK;
}

// The compact form on disk: header (reserved = 1) and thirteen arrays.
static const int kCompactOrder[13] = {TL3_VAL_DIR, TL3_VAL_PACK, TL3_VAL_MASK, TL3_TC_META, TL3_CHAIN_TAU0, TL3_CHAIN_RHO0, TL3_CHAIN_LEN,
                                      TL3_PDD_BYTES, TL3_TILE_DIR, TL3_RES_DIR, TL3_RES_LIST, TL3_RES_MASK, TL3_RES_VAL};

int tl3_serialize_compact(const tl3_matrix* m, void* buf, size_t* bytes) {
  if (!m || !bytes) return TL3_ERR_INVALID_ARG;
  if (!m->host_arrays) return TL3_ERR_UNSUPPORTED;
  size_t need = sizeof(FileHeader);
  for (int w : kCompactOrder) {
    const void* p; size_t n;
    tl3_canonical(m, w, &p, &n);
    need += sizeof(uint64_t) + n;
  }
  if (!buf) { *bytes = need; return TL3_OK; }
  if (*bytes < need) { *bytes = need; return TL3_ERR_INVALID_ARG; }
  uint8_t* o = static_cast<uint8_t*>(buf);
  FileHeader h{kMagic, m->M, m->K, m->p.tile_m, m->p.tile_k, m->p.maxd, 1,
               {m->nnz, m->n_tc, m->n_sf, m->n_res, m->n_dummy, m->n_slots_unused}};
  std::memcpy(o, &h, sizeof(h));
  o += sizeof(h);
  for (int w : kCompactOrder) {
    const void* p; size_t n;
    tl3_canonical(m, w, &p, &n);
    const uint64_t n64 = n;
    std::memcpy(o, &n64, 8);
    o += 8;
    if (n) std::memcpy(o, p, n);
    o += n;
  }
  *bytes = need;
  return TL3_OK;
}

// Expands the compact arrays of a container that was just read; false if anything is out of range.
static bool expand_compact(tl3_matrix& m, const std::vector<uint32_t>& val_dir, const std::vector<uint16_t>& val_pack,
                           const std::vector<uint8_t>& val_mask, const std::vector<uint32_t>& res_dir,
                           const std::vector<uint16_t>& res_list, const std::vector<uint8_t>& res_mask) {
  const int64_t H = m.p.tile_k / 2, slots = static_cast<int64_t>(m.p.tile_m) * H, half_ld = m.K_pad / 2;
  const size_t mask_bytes = (static_cast<size_t>(slots) + 7) / 8;
  const int64_t tiles_k = m.K_pad / m.p.tile_k;
  const size_t nt = static_cast<size_t>(m.n_tiles);
  if (val_dir.size() != 2 * nt || res_dir.size() != 2 * nt || m.tile_dir.size() != 4 * nt) return false;
  m.tc_vals.assign(static_cast<size_t>(m.M_pad) * static_cast<size_t>(half_ld), 0);
  size_t n_mask = 0, expect_pack = 0;
  for (size_t t = 0; t < nt; ++t) {
    const uint32_t mode = val_dir[2 * t], off = val_dir[2 * t + 1];
    if (mode > 1 || off != expect_pack) return false;               // tiles follow each other in val_pack
    const int64_t tm = static_cast<int64_t>(t) / tiles_k, tk = static_cast<int64_t>(t) % tiles_k;
    uint16_t* base = m.tc_vals.data() + tm * m.p.tile_m * half_ld + tk * H;
    if (mode == 0) {
      if (val_pack.size() - off < static_cast<size_t>(slots)) return false;
      for (int64_t r = 0; r < m.p.tile_m; ++r) std::memcpy(base + r * half_ld, val_pack.data() + off + r * H, static_cast<size_t>(H) * 2);
      expect_pack += static_cast<size_t>(slots);
    } else {
      if (val_mask.size() / mask_bytes <= n_mask) return false;
      const uint8_t* bits = val_mask.data() + n_mask * mask_bytes;
      ++n_mask;
      size_t at = off;
      for (int64_t pos = 0; pos < slots; ++pos) {
        if (!((bits[pos >> 3] >> (pos & 7)) & 1u)) continue;
        if (at >= val_pack.size() || val_pack[at] == 0) return false;  // an occupied slot holds a non-zero pattern
        base[(pos / H) * half_ld + pos % H] = val_pack[at++];
      }
      for (int64_t pos = slots; pos < static_cast<int64_t>(mask_bytes) * 8; ++pos)
        if ((bits[pos >> 3] >> (pos & 7)) & 1u) return false;          // bits beyond the tile
      expect_pack = at;
    }
  }
  if (expect_pack != val_pack.size() || n_mask * mask_bytes != val_mask.size()) return false;
  m.res_rho.assign(m.res_val.size(), 0);
  size_t expect_list = 0, expect_mask = 0;
  for (size_t t = 0; t < nt; ++t) {
    const uint32_t off = m.tile_dir[4 * t + 2], cnt = m.tile_dir[4 * t + 3];
    const uint32_t mode = res_dir[2 * t], at = res_dir[2 * t + 1];
    if (mode > 1 || static_cast<size_t>(off) + cnt > m.res_rho.size()) return false;
    if (mode == 0) {
      if (at != expect_list || res_list.size() - at < cnt) return false;
      std::memcpy(m.res_rho.data() + off, res_list.data() + at, static_cast<size_t>(cnt) * 2);
      expect_list += cnt;
    } else {
      if (at != expect_mask || res_mask.size() - at < mask_bytes) return false;
      const uint8_t* bits = res_mask.data() + at;
      uint32_t k = 0;
      for (int64_t pos = 0; pos < static_cast<int64_t>(mask_bytes) * 8; ++pos) {
        if (!((bits[pos >> 3] >> (pos & 7)) & 1u)) continue;
        if (pos >= slots || k >= cnt) return false;
        m.res_rho[off + k++] = static_cast<uint16_t>(pos);
      }
      if (k != cnt) return false;
      expect_mask += mask_bytes;
    }
  }
  return expect_list == res_list.size() && expect_mask == res_mask.size();
}

int tl3_deserialize(const void* buf, size_t bytes, tl3_matrix** out) {
  if (!buf || !out) return TL3_ERR_INVALID_ARG;
  if (bytes < sizeof(FileHeader)) return TL3_ERR_BAD_CONTAINER;
  const uint8_t* p = static_cast<const uint8_t*>(buf);
  const uint8_t* end = p + bytes;
  FileHeader h;
  std::memcpy(&h, p, sizeof(h));
  p += sizeof(h);
  const tl3_params prm{h.tile_m, h.tile_k, h.maxd};
  if (h.magic != kMagic || h.M <= 0 || h.K <= 0 || !valid_params(prm)) return TL3_ERR_BAD_CONTAINER;
  if (h.M > (int64_t{1} << 31) || h.K > (int64_t{1} << 31)) return TL3_ERR_BAD_CONTAINER;
  tl3_matrix* m = new (std::nothrow) tl3_matrix();
  if (!m) return TL3_ERR_NO_MEMORY;
  set_shape(*m, h.M, h.K, prm);
  m->nnz = h.stats[0]; m->n_tc = h.stats[1]; m->n_sf = h.stats[2]; m->n_res = h.stats[3];
  m->n_dummy = h.stats[4]; m->n_slots_unused = h.stats[5];
  auto read = [&](auto& vec) -> bool {
    using T = typename std::remove_reference<decltype(vec)>::type::value_type;
    if (end - p < 8) return false;
    uint64_t n;
    std::memcpy(&n, p, 8);
    p += 8;
    if (n > static_cast<uint64_t>(end - p) || n % sizeof(T) != 0) return false;
    vec.resize(n / sizeof(T));
    if (n) std::memcpy(vec.data(), p, n);
    p += n;
    return true;
  };
  bool ok = false;
  try {
    if (h.reserved == 0) {
      ok = read(m->tc_vals) && read(m->tc_meta) && read(m->chain_tau0) && read(m->chain_rho0) &&
           read(m->chain_len) && read(m->pdd_bytes) && read(m->tile_dir) && read(m->res_rho) && read(m->res_val);
    } else if (h.reserved == 1) {                                   // compact form (tl3_serialize_compact)
      std::vector<uint32_t> val_dir, res_dir;
      std::vector<uint16_t> val_pack, res_list;
      std::vector<uint8_t> val_mask, res_mask;
      ok = read(val_dir) && read(val_pack) && read(val_mask) && read(m->tc_meta) && read(m->chain_tau0) && read(m->chain_rho0) &&
           read(m->chain_len) && read(m->pdd_bytes) && read(m->tile_dir) && read(res_dir) && read(res_list) && read(res_mask) &&
           read(m->res_val) && expand_compact(*m, val_dir, val_pack, val_mask, res_dir, res_list, res_mask);
    }
  } catch (const std::bad_alloc&) {
    delete m;
    return TL3_ERR_NO_MEMORY;
  }
  if (!ok || p != end || !consistent(*m)) { delete m; return TL3_ERR_BAD_CONTAINER; }
  *out = m;
  return TL3_OK;
}

void tl3_free(tl3_matrix* m) {
  if (m && m->device_canon && m->release_device_canon) m->release_device_canon(m->device_canon);
  delete m;
}

const char* tl3_strerror(int code) {
  switch (code) {
    case TL3_OK: return "ok";
    case TL3_ERR_INVALID_ARG: return "invalid argument";
    case TL3_ERR_UNSUPPORTED: return "unsupported N, tile shape or device";
    case TL3_ERR_NOT_UPLOADED: return "matrix has not been uploaded to the device";
    case TL3_ERR_BAD_CONTAINER: return "inconsistent container";
    case TL3_ERR_CUDA: return "CUDA runtime error";
    case TL3_ERR_DEVICE_TIMEOUT: return "a bounded wait inside the kernel expired";
    case TL3_ERR_NO_MEMORY: return "out of host memory";
    case TL3_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the library's built-in array holds";
    default: return "unknown error";
  }
}

}  // extern "C"
