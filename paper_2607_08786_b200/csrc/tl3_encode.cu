// Format conversion on the GPU: dense masked fp16 W (device) -> the canonical three-layer container
// of Sec. 3.2, byte for byte what tl3_encode() builds on the host.  (The paper converts on the CPU,
// 41-93 s per model, Sec. 5.3 "Storage Format Conversion".)
//
// Tiles are independent, so one CTA of 128 threads takes one 128 x 128 tile; thread r owns row r of
// the tile -- its 32 windows, and later the PDD chain of the surplus weights of that row.
//   pass A   every thread classifies its 32 windows (which two weights stay, which slots are
//            empty, which weights are surplus) and counts its surplus weights and empty slots;
//   scan     a block-wide exclusive scan of both counts gives every row the index of its first
//            surplus weight and of its first empty slot in the tile's row-major order;
//   pass B   the same classification again, this time writing the kept values and the metadata to
//            the container and the surplus list (position, value) and the empty-slot list into
//            shared memory at their scanned positions -- both lists come out sorted;
//   chains   the i-th surplus weight is parked in the i-th empty slot; thread r walks the pairs
//            whose surplus weight lies in row r, writes the parked values into the value array,
//            and forms the chain: 16-bit starts, 4-bit delta pairs, dummy points for spans above
//            the 4-bit range, cut after 255 bytes;
//   residual what found no empty slot (and what a cut chain left over) goes to the Residual list.
// The kernel runs twice: first it only counts the PDD bytes and Residual entries of every tile,
// a one-block scan turns the counts into the offsets of the tile directory, then it runs again
// and writes the bytes where they belong.
#include <cuda_runtime.h>

#include <cstdint>
#include <new>
#include <vector>

#include "tl3_internal.h"

namespace tl3 {

void set_cuda_error(int e);

#define TL3_ENC_CUDA(expr)                                    \
  do {                                                        \
    cudaError_t e_ = (expr);                                  \
    if (e_ != cudaSuccess) {                                  \
      tl3::set_cuda_error(static_cast<int>(e_));              \
      rc = TL3_ERR_CUDA;                                      \
      goto done;                                              \
    }                                                         \
  } while (0)

namespace {

constexpr int kEncThreads = 128;
constexpr int kMaxd = 15;
constexpr int kChainCap = 255;

struct EncodeArgs {
  const uint16_t* W;            // device, row-major, leading dimension ldw
  long long M, K, ldw;
  long long K_pad;
  int tiles_k;
  uint16_t* tc_vals;            // [M_pad][K_pad / 2]
  uint8_t* tc_meta;             // [M_pad][K_pad / 8]
  uint16_t* chain_tau0;         // [tiles][128]
  uint16_t* chain_rho0;
  uint8_t* chain_len;
  uint32_t* tile_dir;           // [tiles][4]: pdd_off, pdd_len, res_off, res_cnt
  uint8_t* pdd_bytes;           // emit pass only
  uint16_t* res_rho;
  uint16_t* res_val;
  unsigned long long* stats;    // nnz, n_tc, n_sf, n_res, n_dummy, n_slots_unused
  int emit;                     // 0: count pass (fills pdd_len and res_cnt of the directory), 1: write everything
};

__device__ __forceinline__ bool nonzero(uint16_t h) { return (h & 0x7FFFu) != 0; }

// One window of four consecutive weights (Sec. 3.2, Sparse-TC layer): the first two non-zeros stay;
// a window short of two completes its index pair with the lowest unused positions (those slots are
// empty); the third and fourth non-zero are surplus and always sit at in-window index 2 or 3.
struct Window {
  int idx0, idx1;               // in-window index carried by slot 0 / slot 1
  bool kept0, kept1;
  int n_surplus;
  int sur[2];                   // in-window indices of the surplus weights
};

__device__ __forceinline__ Window classify(const uint16_t w[4]) {
  Window c;
  int nz[4], n = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (nonzero(w[i])) nz[n++] = i;
  if (n >= 2) { c.idx0 = nz[0]; c.idx1 = nz[1]; c.kept0 = true; c.kept1 = true; }
  else if (n == 1) {
    if (nz[0] == 0) { c.idx0 = 0; c.idx1 = 1; c.kept0 = true; c.kept1 = false; }
    else { c.idx0 = 0; c.idx1 = nz[0]; c.kept0 = false; c.kept1 = true; }
  } else { c.idx0 = 0; c.idx1 = 1; c.kept0 = false; c.kept1 = false; }
  c.n_surplus = n > 2 ? n - 2 : 0;
  c.sur[0] = n > 2 ? nz[2] : 0;
  c.sur[1] = n > 3 ? nz[3] : 0;
  return c;
}

// exclusive scan of one int per thread over the 128 threads of the CTA; *total gets the sum
__device__ __forceinline__ int block_exclusive_scan(int v, int* s_warp, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int x = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int y = __shfl_up_sync(0xFFFFFFFFu, x, d);
    if (lane >= d) x += y;
  }
  if (lane == 31) s_warp[warp] = x;
  __syncthreads();
  int base = 0;
  for (int w = 0; w < warp; ++w) base += s_warp[w];
  *total = s_warp[0] + s_warp[1] + s_warp[2] + s_warp[3];
  __syncthreads();
  return base + x - v;
}

__global__ void __launch_bounds__(kEncThreads)
tl3_encode_kernel(const EncodeArgs a) {
  __shared__ uint16_t s_rho[kTileM * kH];      // surplus weights of the tile, ascending position in W_r
  __shared__ uint16_t s_tau[kTileM * kH];      // empty slots of the tile, ascending position in W_t
  __shared__ int s_warp[4];
  const int r = threadIdx.x;
  const long long tile = blockIdx.x;
  const long long tm = tile / a.tiles_k, tk = tile % a.tiles_k;
  const long long row = tm * kTileM + r;
  const long long half_ld = a.K_pad / 2, meta_ld = a.K_pad / 8;
  const bool row_in = row < a.M;
  const uint16_t* wrow = a.W + row * a.ldw + tk * kTileK;
  auto load_window = [&](int q, uint16_t w[4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const long long col = tk * kTileK + 4 * q + i;
      w[i] = (row_in && col < a.K) ? wrow[4 * q + i] : uint16_t{0};
    }
  };

  // ---- pass A: count the surplus weights and the empty slots of this row
  int nS = 0, nE = 0, nnz = 0;
  for (int q = 0; q < kTileK / 4; ++q) {
    uint16_t w[4];
    load_window(q, w);
    const Window c = classify(w);
    nS += c.n_surplus;
    nE += (c.kept0 ? 0 : 1) + (c.kept1 ? 0 : 1);
    nnz += (c.kept0 ? 1 : 0) + (c.kept1 ? 1 : 0) + c.n_surplus;
  }
  int totS = 0, totE = 0;
  const int offS = block_exclusive_scan(nS, s_warp, &totS);
  const int offE = block_exclusive_scan(nE, s_warp, &totE);
  const int P = totS < totE ? totS : totE;     // pairs: the i-th surplus weight goes to the i-th empty slot

  // ---- pass B: kept values and metadata to the container, both lists to shared memory
  {
    int iS = offS, iE = offE;
    uint32_t* mrow = reinterpret_cast<uint32_t*>(a.tc_meta + row * meta_ld + tk * (kTileK / 8));   // 16 bytes of this row, 4-byte aligned
    uint32_t word = 0;                         // eight nibbles: windows 8k .. 8k + 7, even window in the low nibble of its byte
    for (int q = 0; q < kTileK / 4; ++q) {
      uint16_t w[4];
      load_window(q, w);
      const Window c = classify(w);
      word |= static_cast<uint32_t>(c.idx0 | (c.idx1 << 2)) << (4 * (q & 7));
      if (a.emit) {
        uint16_t* v = a.tc_vals + row * half_ld + tk * kH + 2 * q;
        v[0] = c.kept0 ? w[c.idx0] : uint16_t{0};
        v[1] = c.kept1 ? w[c.idx1] : uint16_t{0};
        if ((q & 7) == 7) mrow[q >> 3] = word;
      }
      if ((q & 7) == 7) word = 0;
      if (!c.kept0) s_tau[iE++] = static_cast<uint16_t>(r * kH + 2 * q);
      if (!c.kept1) s_tau[iE++] = static_cast<uint16_t>(r * kH + 2 * q + 1);
      for (int j = 0; j < c.n_surplus; ++j) s_rho[iS++] = static_cast<uint16_t>(r * kH + 2 * q + (c.sur[j] - 2));
    }
  }
  __syncthreads();

  // value of the surplus weight at position rho of W_r (it lies in this thread's row)
  auto surplus_value = [&](int rho) -> uint16_t {
    const int s = rho - r * kH;                // slot of W_r in this row: window s / 2, in-window index 2 + (s & 1)
    return wrow[4 * (s >> 1) + 2 + (s & 1)];
  };
  auto park = [&](int tau, uint16_t v) {       // the value goes into empty slot tau of the tile's value array
    a.tc_vals[(tm * kTileM + tau / kH) * half_ld + tk * kH + tau % kH] = v;
  };

  // ---- chains, first walk: length of this row's chain, what a cut leaves over
  const int i0 = offS, i1 = (offS + nS) < P ? (offS + nS) : (P > offS ? P : offS);   // pairs [i0, i1) of this row
  int len = 0, n_cut = 0, n_sf = 0, n_dummy = 0;
  if (i1 > i0) {
    int tau = s_tau[i0], rho = s_rho[i0];
    n_sf = 1;
    bool cut = false;
    for (int i = i0 + 1; i < i1; ++i) {
      if (!cut) {
        const int gt = s_tau[i] - tau, gr = s_rho[i] - rho;
        const int need = 1 + (gt - 1) / kMaxd + (gr - 1) / kMaxd;
        if (len + need > kChainCap) cut = true;
        else { len += need; n_dummy += need - 1; tau = s_tau[i]; rho = s_rho[i]; ++n_sf; }
      }
      if (cut) ++n_cut;
    }
  }
  int tot_len = 0, tot_cut = 0;
  const int off_len = block_exclusive_scan(len, s_warp, &tot_len);
  const int off_cut = block_exclusive_scan(n_cut, s_warp, &tot_cut);
  const int n_beyond = totS - P;               // surplus weights that found no empty slot
  if (!a.emit) {
    if (r == 0) {
      a.tile_dir[tile * 4 + 1] = static_cast<uint32_t>(tot_len);
      a.tile_dir[tile * 4 + 3] = static_cast<uint32_t>(tot_cut + n_beyond);
    }
    return;
  }

  // ---- second walk: write the chain, park the values, list the Residual entries
  const uint32_t pdd_off = a.tile_dir[tile * 4 + 0], res_off = a.tile_dir[tile * 4 + 2];
  const long long ch = tile * kTileM + r;
  if (i1 > i0) {
    int tau = s_tau[i0], rho = s_rho[i0];
    a.chain_tau0[ch] = static_cast<uint16_t>(tau);
    a.chain_rho0[ch] = static_cast<uint16_t>(rho);
    park(tau, surplus_value(rho));
    uint8_t* code = a.pdd_bytes + pdd_off + off_len;
    uint32_t res_at = res_off + off_cut;
    int at = 0;
    bool cut = false;
    for (int i = i0 + 1; i < i1; ++i) {
      if (!cut) {
        int gt = s_tau[i] - tau, gr = s_rho[i] - rho;
        const int need = 1 + (gt - 1) / kMaxd + (gr - 1) / kMaxd;
        if (at + need > kChainCap) cut = true;
        else {
          while (gt > kMaxd) { code[at++] = static_cast<uint8_t>(kMaxd); gt -= kMaxd; }        // dummy points: a zero nibble moves nothing
          while (gr > kMaxd) { code[at++] = static_cast<uint8_t>(kMaxd << 4); gr -= kMaxd; }
          code[at++] = static_cast<uint8_t>(gt | gr << 4);
          tau = s_tau[i];
          rho = s_rho[i];
          park(tau, surplus_value(rho));
        }
      }
      if (cut) {                               // the chain is full: the rest of the row goes to the Residual layer
        a.res_rho[res_at] = s_rho[i];
        a.res_val[res_at] = surplus_value(s_rho[i]);
        ++res_at;
      }
    }
    a.chain_len[ch] = static_cast<uint8_t>(at);
  } else {
    a.chain_tau0[ch] = 0xFFFFu;
    a.chain_rho0[ch] = 0xFFFFu;
    a.chain_len[ch] = 0;
  }
  // surplus weights beyond the number of empty slots: Residual entries after the cut leftovers
  {
    const int b0 = offS > P ? offS : P, b1 = offS + nS;
    for (int i = b0; i < b1; ++i) {
      const uint32_t at = res_off + tot_cut + (i - P);
      a.res_rho[at] = s_rho[i];
      a.res_val[at] = surplus_value(s_rho[i]);
    }
  }
  // layer statistics (Sec. 3.2 quotes their shares)
  const int n_tc = nnz - nS;
  atomicAdd(a.stats + 0, static_cast<unsigned long long>(nnz));
  atomicAdd(a.stats + 1, static_cast<unsigned long long>(n_tc));
  atomicAdd(a.stats + 2, static_cast<unsigned long long>(n_sf));
  atomicAdd(a.stats + 4, static_cast<unsigned long long>(n_dummy));
  if (r == 0) {
    atomicAdd(a.stats + 3, static_cast<unsigned long long>(tot_cut + n_beyond));
    atomicAdd(a.stats + 5, static_cast<unsigned long long>(totE - P + tot_cut));
  }
}

// Exclusive scan of the per-tile byte and entry counts into the offsets of the tile directory
// (one CTA; the directory has a few thousand to a hundred thousand tiles).
__global__ void __launch_bounds__(1024)
tl3_encode_scan_kernel(uint32_t* tile_dir, long long n_tiles, unsigned long long* totals) {
  __shared__ unsigned long long s_part[2][32];
  __shared__ unsigned long long s_carry[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { s_carry[0] = 0; s_carry[1] = 0; }
  __syncthreads();
  for (long long base = 0; base < n_tiles; base += 1024) {
    const long long t = base + tid;
    unsigned long long v[2] = {0, 0};
    if (t < n_tiles) { v[0] = tile_dir[t * 4 + 1]; v[1] = tile_dir[t * 4 + 3]; }
    unsigned long long x[2] = {v[0], v[1]};
#pragma unroll
    for (int k = 0; k < 2; ++k) {
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x[k], d);
        if (lane >= d) x[k] += y;
      }
      if (lane == 31) s_part[k][warp] = x[k];
    }
    __syncthreads();
    unsigned long long pre[2] = {s_carry[0], s_carry[1]};
    for (int w = 0; w < warp; ++w) { pre[0] += s_part[0][w]; pre[1] += s_part[1][w]; }
    if (t < n_tiles) {
      tile_dir[t * 4 + 0] = static_cast<uint32_t>(pre[0] + x[0] - v[0]);
      tile_dir[t * 4 + 2] = static_cast<uint32_t>(pre[1] + x[1] - v[1]);
    }
    __syncthreads();
    if (tid == 1023) { s_carry[0] = pre[0] + x[0]; s_carry[1] = pre[1] + x[1]; }
    __syncthreads();
  }
  if (tid == 0) { totals[0] = s_carry[0]; totals[1] = s_carry[1]; }
}

}  // namespace
}  // namespace tl3

namespace tl3 {
namespace {
void release_encoded(void* p) {
  DeviceCanon* c = static_cast<DeviceCanon*>(p);
  if (!c) return;
  for (void* a : c->alloc) if (a) cudaFree(a);
  delete c;
}
}  // namespace
}  // namespace tl3

extern "C" int tl3_plan_device(tl3_matrix* m, void* stream);

// keep_on_device: leave the container where the kernels wrote it (for tl3_upload_device) and make
// no host copies of it.
static int encode_device_impl(const void* dW, int64_t M, int64_t K, int64_t ldw, void* stream, bool keep_on_device, tl3_matrix** out) {
  using namespace tl3;
  if (!dW || !out || M <= 0 || K <= 0 || ldw < K || M > (int64_t{1} << 31) || K > (int64_t{1} << 31)) return TL3_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  tl3_matrix* m = new (std::nothrow) tl3_matrix();
  if (!m) return TL3_ERR_NO_MEMORY;
  m->M = M; m->K = K; m->p = tl3_params{kTileM, kTileK, kMaxd};
  m->tiles_m = (M + kTileM - 1) / kTileM;
  m->tiles_k = (K + kTileK - 1) / kTileK;
  m->M_pad = m->tiles_m * kTileM;
  m->K_pad = m->tiles_k * kTileK;
  m->n_tiles = m->tiles_m * m->tiles_k;
  if (m->n_tiles > 0x7FFFFFFF) { delete m; return TL3_ERR_UNSUPPORTED; }
  const size_t n_vals = static_cast<size_t>(m->M_pad) * m->K_pad / 2, n_meta = n_vals / 4;
  const size_t n_chain = static_cast<size_t>(m->n_tiles) * kTileM, n_dir = static_cast<size_t>(m->n_tiles) * 4;

  int rc = TL3_OK;
  uint8_t* scratch = nullptr;               // everything the kernels write, in one allocation
  uint8_t* var = nullptr;                   // PDD bytes and Residual entries (sized after the count pass)
  unsigned long long totals[2] = {0, 0}, stats[6] = {0, 0, 0, 0, 0, 0};
  // layout of `scratch` (every part 256-byte aligned)
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const size_t o_vals = 0, o_meta = o_vals + up(n_vals * 2), o_tau = o_meta + up(n_meta), o_rho = o_tau + up(n_chain * 2),
               o_len = o_rho + up(n_chain * 2), o_dir = o_len + up(n_chain), o_stats = o_dir + up(n_dir * 4), total = o_stats + 256;
  EncodeArgs a{};
  {
    TL3_ENC_CUDA(cudaMalloc(reinterpret_cast<void**>(&scratch), total));
    TL3_ENC_CUDA(cudaMemsetAsync(scratch + o_stats, 0, 256, st));
    a.W = static_cast<const uint16_t*>(dW);
    a.M = M; a.K = K; a.ldw = ldw; a.K_pad = m->K_pad; a.tiles_k = static_cast<int>(m->tiles_k);
    a.tc_vals = reinterpret_cast<uint16_t*>(scratch + o_vals);
    a.tc_meta = scratch + o_meta;
    a.chain_tau0 = reinterpret_cast<uint16_t*>(scratch + o_tau);
    a.chain_rho0 = reinterpret_cast<uint16_t*>(scratch + o_rho);
    a.chain_len = scratch + o_len;
    a.tile_dir = reinterpret_cast<uint32_t*>(scratch + o_dir);
    a.stats = reinterpret_cast<unsigned long long*>(scratch + o_stats);
    a.emit = 0;
    tl3_encode_kernel<<<static_cast<unsigned>(m->n_tiles), kEncThreads, 0, st>>>(a);
    tl3_encode_scan_kernel<<<1, 1024, 0, st>>>(a.tile_dir, m->n_tiles, a.stats + 8);
    TL3_ENC_CUDA(cudaGetLastError());
    TL3_ENC_CUDA(cudaMemcpyAsync(totals, a.stats + 8, sizeof(totals), cudaMemcpyDeviceToHost, st));
    TL3_ENC_CUDA(cudaStreamSynchronize(st));
    if (totals[0] > 0xFFFFFFFFull || totals[1] > 0xFFFFFFFFull) { rc = TL3_ERR_UNSUPPORTED; goto done; }   // 32-bit directory offsets
    const size_t o_res_rho = up(totals[0]), o_res_val = o_res_rho + up(totals[1] * 2), var_total = o_res_val + up(totals[1] * 2) + 256;
    TL3_ENC_CUDA(cudaMalloc(reinterpret_cast<void**>(&var), var_total));
    a.pdd_bytes = var;
    a.res_rho = reinterpret_cast<uint16_t*>(var + o_res_rho);
    a.res_val = reinterpret_cast<uint16_t*>(var + o_res_val);
    a.emit = 1;
    tl3_encode_kernel<<<static_cast<unsigned>(m->n_tiles), kEncThreads, 0, st>>>(a);
    TL3_ENC_CUDA(cudaGetLastError());
    if (keep_on_device) {
      TL3_ENC_CUDA(cudaMemcpyAsync(stats, a.stats, sizeof(stats), cudaMemcpyDeviceToHost, st));
      TL3_ENC_CUDA(cudaStreamSynchronize(st));
      m->nnz = static_cast<int64_t>(stats[0]); m->n_tc = static_cast<int64_t>(stats[1]); m->n_sf = static_cast<int64_t>(stats[2]);
      m->n_res = static_cast<int64_t>(stats[3]); m->n_dummy = static_cast<int64_t>(stats[4]); m->n_slots_unused = static_cast<int64_t>(stats[5]);
      DeviceCanon* c = new (std::nothrow) DeviceCanon();
      if (!c) { rc = TL3_ERR_NO_MEMORY; goto done; }
      *c = DeviceCanon{a.tc_vals, a.tc_meta, a.chain_tau0, a.chain_rho0, a.chain_len, a.pdd_bytes, a.tile_dir, a.res_rho, a.res_val, {scratch, var}};
      m->device_canon = c;
      m->release_device_canon = release_encoded;
      m->host_arrays = false;
      m->canon_bytes = static_cast<int64_t>(n_vals * 2 + n_meta + n_chain * 5 + n_dir * 4 + totals[0] + totals[1] * 4);
      scratch = nullptr;                                            // owned by the handle from here on
      var = nullptr;
      goto done;
    }
    try {
      m->tc_vals.resize(n_vals); m->tc_meta.resize(n_meta);
      m->chain_tau0.resize(n_chain); m->chain_rho0.resize(n_chain); m->chain_len.resize(n_chain);
      m->tile_dir.resize(n_dir);
      m->pdd_bytes.resize(totals[0]); m->res_rho.resize(totals[1]); m->res_val.resize(totals[1]);
    } catch (const std::bad_alloc&) { rc = TL3_ERR_NO_MEMORY; goto done; }
    TL3_ENC_CUDA(cudaMemcpyAsync(m->tc_vals.data(), a.tc_vals, n_vals * 2, cudaMemcpyDeviceToHost, st));
    TL3_ENC_CUDA(cudaMemcpyAsync(m->tc_meta.data(), a.tc_meta, n_meta, cudaMemcpyDeviceToHost, st));
    TL3_ENC_CUDA(cudaMemcpyAsync(m->chain_tau0.data(), a.chain_tau0, n_chain * 2, cudaMemcpyDeviceToHost, st));
    TL3_ENC_CUDA(cudaMemcpyAsync(m->chain_rho0.data(), a.chain_rho0, n_chain * 2, cudaMemcpyDeviceToHost, st));
    TL3_ENC_CUDA(cudaMemcpyAsync(m->chain_len.data(), a.chain_len, n_chain, cudaMemcpyDeviceToHost, st));
    TL3_ENC_CUDA(cudaMemcpyAsync(m->tile_dir.data(), a.tile_dir, n_dir * 4, cudaMemcpyDeviceToHost, st));
    if (totals[0]) TL3_ENC_CUDA(cudaMemcpyAsync(m->pdd_bytes.data(), a.pdd_bytes, totals[0], cudaMemcpyDeviceToHost, st));
    if (totals[1]) {
      TL3_ENC_CUDA(cudaMemcpyAsync(m->res_rho.data(), a.res_rho, totals[1] * 2, cudaMemcpyDeviceToHost, st));
      TL3_ENC_CUDA(cudaMemcpyAsync(m->res_val.data(), a.res_val, totals[1] * 2, cudaMemcpyDeviceToHost, st));
    }
    TL3_ENC_CUDA(cudaMemcpyAsync(stats, a.stats, sizeof(stats), cudaMemcpyDeviceToHost, st));
    TL3_ENC_CUDA(cudaStreamSynchronize(st));
    m->nnz = static_cast<int64_t>(stats[0]); m->n_tc = static_cast<int64_t>(stats[1]); m->n_sf = static_cast<int64_t>(stats[2]);
    m->n_res = static_cast<int64_t>(stats[3]); m->n_dummy = static_cast<int64_t>(stats[4]); m->n_slots_unused = static_cast<int64_t>(stats[5]);
  }
done:
  if (scratch) cudaFree(scratch);
  if (var) cudaFree(var);
  if (rc == TL3_OK && keep_on_device) rc = tl3_plan_device(m, stream);   // sizes of the packed blocks: tl3_device_bytes() is valid on return
  if (rc != TL3_OK) { tl3_free(m); return rc; }
  *out = m;
  return TL3_OK;
}

extern "C" int tl3_encode_device(const void* dW, int64_t M, int64_t K, int64_t ldw, void* stream, tl3_matrix** out) {
  return encode_device_impl(dW, M, K, ldw, stream, false, out);
}

extern "C" int tl3_encode_device_only(const void* dW, int64_t M, int64_t K, int64_t ldw, void* stream, tl3_matrix** out) {
  return encode_device_impl(dW, M, K, ldw, stream, true, out);
}
