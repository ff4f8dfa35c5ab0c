// The device packer on the GPU: canonical container -> the blob of per-tile blocks that the SpMM
// kernel streams, byte for byte what tl3_pack() / tl3_upload() build on the host (tl3_pack.cpp has
// the reasoning behind the layout: bank-major re-pairing of the Slot-Filling layer, four equal
// chains per bank, the same number of transposed code words for every chain of a tile, the tails
// as Residual entries).
//
// One CTA of 128 threads per 128 x 128 tile.  In turn a thread is the owner of canonical chain r
// (to lift the parked values out of the value array), of 64 consecutive bank-major slot
// coordinates (to list the empty slots and the surplus weights in that order), and of device
// chain c (bank c / 4, run c % 4).  The kernel runs twice: a count pass that yields every tile's
// number of code words and Residual entries, from which the host lays the blocks out exactly as
// plan_device_layout() does, and an emit pass that writes the blocks.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include "tl3_internal.h"

namespace tl3 {

void set_cuda_error(int e);

namespace {

constexpr int kSlots = kTileM * kH;        // 8192
constexpr int kChains = 128;

struct PackArgs {
  // canonical container (device copies)
  const uint16_t* tc_vals;
  const uint8_t* tc_meta;
  const uint16_t* chain_tau0;
  const uint16_t* chain_rho0;
  const uint8_t* chain_len;
  const uint8_t* pdd_bytes;
  const uint32_t* tile_dir;
  const uint16_t* res_rho;
  const uint16_t* res_val;
  long long K_pad;
  int tiles_k;
  // count pass: per tile {pdd_len, res_cnt, real delta bytes}
  uint32_t* sizes;
  // emit pass
  uint8_t* blob;
  const unsigned long long* block_off;     // byte offset of every tile's block in the blob
  unsigned long long dir_offset;
  int emit;
};

__device__ __forceinline__ uint32_t u_of_pos(uint32_t pos) {
  const uint32_t r = pos >> 6, q = (pos >> 1) & 31u, s = pos & 1u;
  const uint32_t bank = (((q >> 2) ^ (r & 7u)) << 2) | (q & 3u);
  return (bank << 8) | (s << 7) | r;
}
__device__ __forceinline__ uint32_t pos_of_u(uint32_t u) {
  const uint32_t r = u & 127u, s = (u >> 7) & 1u, bank = u >> 8;
  const uint32_t q = (((bank >> 2) ^ (r & 7u)) << 2) | (bank & 3u);
  return r * 64u + 2u * q + s;
}
__device__ __forceinline__ uint32_t delta_bytes(uint32_t gt, uint32_t gr) { return (gt - 1) / 15 + (gr - 1) / 15 + 1; }
__device__ __forceinline__ uint32_t align_up_d(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

// exclusive scan over the 128 threads of the CTA
__device__ __forceinline__ int scan128(int v, int* s_warp, int* total) {
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

// dynamic shared memory of the pack kernel
struct PackSmem {
  uint16_t vals[kSlots];       // value slots of the tile by row-major position; parked values lifted out, later re-parked
  uint16_t sval[kSlots];       // value of the surplus weight at bank-major coordinate u
  uint16_t cand[kSlots];       // empty slots, ascending u
  uint16_t sur[kSlots];        // surplus weights, ascending u
  uint16_t sel[kSlots];        // selected empty slots, ascending u
  uint32_t flag[kSlots / 32];  // bit u set: a surplus weight sits at u
  int off_cand[kChains + 1];   // first candidate of the thread that owns u in [64 t, 64 t + 64)
  int take[kChains], src[kChains], off_sel[kChains + 1];
  int len[kChains];            // delta bytes of device chain c
  int beyond[4];
  int real_bytes;
  int warp_tmp[4];
};

__global__ void __launch_bounds__(128)
tl3_pack_kernel(const PackArgs a) {
  extern __shared__ __align__(16) uint8_t pack_smem_raw[];
  PackSmem& sm = *reinterpret_cast<PackSmem*>(pack_smem_raw);
  const int tid = threadIdx.x;
  const long long t = blockIdx.x;
  const long long tm = t / a.tiles_k, tk = t % a.tiles_k;
  const long long half_ld = a.K_pad / 2, meta_ld = a.K_pad / 8;

  // (1) the tile's value slots; thread r copies row r
  {
    const uint16_t* src = a.tc_vals + (tm * kTileM + tid) * half_ld + tk * kH;
    for (int s = 0; s < kH; ++s) sm.vals[tid * kH + s] = src[s];
    sm.flag[tid] = 0u;
    sm.flag[tid + 128] = 0u;
    if (tid < 4) sm.beyond[tid] = 0;
    if (tid == 0) sm.real_bytes = 0;
  }
  __syncthreads();

  // (2) Algorithm 1 over the canonical chains (one per tile row): lift every parked value out of
  //     its slot and note it at the bank-major coordinate of the position it belongs to
  {
    const int len = a.chain_len[t * kTileM + tid];
    int tot = 0;
    const int at0 = scan128(len, sm.warp_tmp, &tot);
    const uint8_t* code = a.pdd_bytes + a.tile_dir[t * 4] + at0;
    uint32_t tau = a.chain_tau0[t * kTileM + tid], rho = a.chain_rho0[t * kTileM + tid];
    auto lift = [&](uint32_t ta, uint32_t rh) {
      const uint32_t ur = u_of_pos(rh);
      sm.sval[ur] = sm.vals[ta];
      atomicOr(&sm.flag[ur >> 5], 1u << (ur & 31u));
      sm.vals[ta] = 0;
    };
    if (tau != 0xFFFFu) {
      lift(tau, rho);
      for (int k = 0; k < len; ++k) {
        const uint32_t b = code[k], dt = b & 15u, dr = b >> 4;
        tau += dt;
        rho += dr;
        if (dt && dr) lift(tau, rho);
      }
    }
  }
  __syncthreads();

  // (3) empty slots and surplus weights in bank-major order; thread t owns u in [64 t, 64 t + 64)
  int n_cand = 0, n_pairs = 0;
  {
    int nc = 0, ns = 0;
    for (uint32_t u = 64u * tid; u < 64u * tid + 64u; ++u) {
      nc += (sm.vals[pos_of_u(u)] & 0x7FFFu) == 0 ? 1 : 0;
      ns += (sm.flag[u >> 5] >> (u & 31u)) & 1u;
    }
    int oc = scan128(nc, sm.warp_tmp, &n_cand);
    int os = scan128(ns, sm.warp_tmp, &n_pairs);
    sm.off_cand[tid] = oc;
    if (tid == 0) sm.off_cand[kChains] = n_cand;
    for (uint32_t u = 64u * tid; u < 64u * tid + 64u; ++u) {
      if ((sm.vals[pos_of_u(u)] & 0x7FFFu) == 0) sm.cand[oc++] = static_cast<uint16_t>(u);
      if ((sm.flag[u >> 5] >> (u & 31u)) & 1u) sm.sur[os++] = static_cast<uint16_t>(u);
    }
  }
  __syncthreads();

  // (4) every bank gets a share of the parked elements proportional to its empty slots; its empty
  //     slots are cut into four runs of equal count and run q uses its first slots (one thread:
  //     what a run cannot take is carried to the next)
  if (tid == 0) {
    uint32_t cum = 0, carry = 0;
    int base = 0;
    for (int b = 0; b < 32; ++b) {
      const uint32_t N_b = static_cast<uint32_t>(sm.off_cand[4 * b + 4] - sm.off_cand[4 * b]);
      const uint32_t lo = n_cand ? static_cast<uint32_t>(static_cast<unsigned long long>(cum) * n_pairs / n_cand) : 0u;
      cum += N_b;
      const uint32_t hi = n_cand ? static_cast<uint32_t>(static_cast<unsigned long long>(cum) * n_pairs / n_cand) : 0u;
      const uint32_t n_b = hi - lo;
      for (uint32_t q = 0; q < 4; ++q) {
        const uint32_t first = N_b * q / 4, size = N_b * (q + 1) / 4 - first;
        const uint32_t want = n_b * (q + 1) / 4 - n_b * q / 4 + carry;
        const uint32_t tk_ = want < size ? want : size;
        carry = want - tk_;
        sm.take[4 * b + q] = static_cast<int>(tk_);
        sm.src[4 * b + q] = base + static_cast<int>(first);
      }
      base += static_cast<int>(N_b);
    }
  }
  __syncthreads();
  int n_sel = 0;
  const int my_take = sm.take[tid];
  const int my_off = scan128(my_take, sm.warp_tmp, &n_sel);
  sm.off_sel[tid] = my_off;
  for (int i = 0; i < my_take; ++i) sm.sel[my_off + i] = sm.cand[sm.src[tid] + i];
  __syncthreads();

  // (5) device chain c = the pairs [off, off + take) of run c; how many entries end beyond 0, 4, 8, 12 delta bytes
  const int n_use = n_sel < n_pairs ? n_sel : n_pairs;
  const int i0 = my_off, i1 = (my_off + my_take) < n_use ? (my_off + my_take) : (n_use > my_off ? n_use : my_off);
  {
    uint32_t end = 0;
    int by[4] = {0, 0, 0, 0};
    for (int i = i0 + 1; i < i1; ++i) {
      end += delta_bytes(static_cast<uint32_t>(sm.sel[i] - sm.sel[i - 1]), static_cast<uint32_t>(sm.sur[i] - sm.sur[i - 1]));
#pragma unroll
      for (int w = 0; w < 4; ++w) by[w] += end > 4u * w ? 1 : 0;
    }
#pragma unroll
    for (int w = 0; w < 4; ++w)
      if (by[w]) atomicAdd(&sm.beyond[w], by[w]);
  }
  __syncthreads();
  uint32_t n_words = 0;
  for (uint32_t w = 1; w < 4; ++w)
    if (512u * w + 4u * sm.beyond[w] < 512u * n_words + 4u * sm.beyond[n_words]) n_words = w;
  const uint32_t cap = 4u * n_words;

  // (6) first walk of the device chain: its delta bytes within the cap, what the cut leaves over
  int n_bytes = 0, n_tail = 0, n_real = 0;
  {
    bool cut = false;
    for (int i = i0 + 1; i < i1; ++i) {
      const uint32_t need = delta_bytes(static_cast<uint32_t>(sm.sel[i] - sm.sel[i - 1]), static_cast<uint32_t>(sm.sur[i] - sm.sur[i - 1]));
      if (cut || n_bytes + need > cap) { cut = true; ++n_tail; }
      else { n_bytes += need; ++n_real; }
    }
  }
  sm.len[tid] = n_bytes;
  if (n_real) atomicAdd(&sm.real_bytes, n_real);
  int tot_tail = 0;
  const int off_tail = scan128(n_tail, sm.warp_tmp, &tot_tail);
  const uint32_t canon_res_off = a.tile_dir[t * 4 + 2], canon_res_cnt = a.tile_dir[t * 4 + 3];
  const uint32_t pdd_len = n_words * 4u * kChains;
  const uint32_t res_cnt = static_cast<uint32_t>(tot_tail + (n_pairs - n_use)) + canon_res_cnt;
  __syncthreads();
  if (!a.emit) {
    if (tid == 0) {
      a.sizes[t * 3 + 0] = pdd_len;
      a.sizes[t * 3 + 1] = res_cnt;
      a.sizes[t * 3 + 2] = static_cast<uint32_t>(sm.real_bytes);
    }
    return;
  }

  // (7) the block
  uint8_t* blk = a.blob + a.block_off[t];
  const uint32_t block_bytes = align_up_d(kPddOff + align_up_d(pdd_len, 4) + 4u * res_cnt, 16);
  {
    // everything behind the metadata starts from zero (padding of short chains, alignment)
    uint32_t* z = reinterpret_cast<uint32_t*>(blk + kInfoOff);
    const uint32_t n = (align_up_d(block_bytes, kBlockAlign) - kInfoOff) / 4;
    for (uint32_t i = tid; i < n; i += 128) z[i] = 0u;
  }
  __syncthreads();
  // chain slot w * 32 + l holds the w-th longest of the four chains of bank l (ties: lower chain first)
  int slot;
  {
    const int b = tid >> 2;
    int w = 0;
    for (int c = 4 * b; c < 4 * b + 4; ++c)
      if (sm.len[c] > n_bytes || (sm.len[c] == n_bytes && c < tid)) ++w;
    slot = w * 32 + b;
  }
  uint32_t* res = reinterpret_cast<uint32_t*>(blk + kPddOff + align_up_d(pdd_len, 4));
  {
    uint32_t hdr = 0xFFFFFFFFu;
    uint8_t* code = blk + kPddOff;
    uint32_t at = 0, res_at = static_cast<uint32_t>(off_tail);
    bool cut = false;
    for (int i = i0; i < i1; ++i) {
      const uint32_t u = sm.sel[i], r_u = sm.sur[i];
      const uint16_t v = sm.sval[r_u];
      if (i == i0) {
        hdr = u | r_u << 16;
      } else {
        uint32_t gt = u - sm.sel[i - 1], gr = r_u - sm.sur[i - 1];
        const uint32_t need = delta_bytes(gt, gr);
        if (cut || at + need > cap) {          // the chain is full: the rest of its run goes to the Residual list
          cut = true;
          res[res_at++] = r_u | static_cast<uint32_t>(v) << 16;
          continue;
        }
        auto put = [&](uint8_t b) { code[((at >> 2) * kChains + static_cast<uint32_t>(slot)) * 4u + (at & 3u)] = b; ++at; };
        while (gt > 15) { put(0x0F); gt -= 15; }           // dummy points (a zero nibble moves nothing)
        while (gr > 15) { put(0xF0); gr -= 15; }
        put(static_cast<uint8_t>(gt | gr << 4));
      }
      sm.vals[pos_of_u(u)] = v;                // the value is parked in its new slot
    }
    reinterpret_cast<uint32_t*>(blk + kHdrOff)[slot] = hdr;
  }
  // surplus weights beyond the selected empty slots, then the canonical Residual entries
  for (int i = n_use + tid; i < n_pairs; i += 128)
    res[tot_tail + (i - n_use)] = sm.sur[i] | static_cast<uint32_t>(sm.sval[sm.sur[i]]) << 16;
  for (uint32_t j = tid; j < canon_res_cnt; j += 128)
    res[tot_tail + (n_pairs - n_use) + j] = u_of_pos(a.res_rho[canon_res_off + j]) | static_cast<uint32_t>(a.res_val[canon_res_off + j]) << 16;
  __syncthreads();
  // values: row r of the K-major 128-byte-swizzled image; word `bank` of the row holds both slots of one window
  {
    uint32_t* row = reinterpret_cast<uint32_t*>(blk + tid * 128);
    for (uint32_t bank = 0; bank < 32; ++bank) {
      const uint32_t p0 = pos_of_u(bank << 8 | static_cast<uint32_t>(tid));
      row[bank] = static_cast<uint32_t>(sm.vals[p0]) | static_cast<uint32_t>(sm.vals[p0 + 1]) << 16;
    }
  }
  // metadata in tensor-memory lane order
  {
    const int L = tid, mrow = (L & 7) + 16 * (L >> 4), half = (L >> 3) & 1;
    uint32_t* meta = reinterpret_cast<uint32_t*>(blk + kMetaOff);
    for (int kb = 0; kb < 4; ++kb) {
      const uint8_t* lo = a.tc_meta + (tm * kTileM + mrow) * meta_ld + tk * (kTileK / 8) + 4 * kb + 2 * half;
      const uint8_t* hi = a.tc_meta + (tm * kTileM + mrow + 8) * meta_ld + tk * (kTileK / 8) + 4 * kb + 2 * half;
      meta[L * 4 + kb] = static_cast<uint32_t>(lo[0]) | static_cast<uint32_t>(lo[1]) << 8 |
                         static_cast<uint32_t>(hi[0]) << 16 | static_cast<uint32_t>(hi[1]) << 24;
    }
  }
  if (tid == 0) {
    uint32_t* info = reinterpret_cast<uint32_t*>(blk + kInfoOff);
    info[0] = pdd_len;
    info[1] = res_cnt;
    info[2] = n_words;
    DirEntry* dir = reinterpret_cast<DirEntry*>(a.blob + a.dir_offset);
    dir[t] = DirEntry{static_cast<uint32_t>(a.block_off[t] / 16), block_bytes, pdd_len, res_cnt};
  }
}

}  // namespace
}  // namespace tl3

namespace tl3 {
namespace {

struct CanonOnDevice {
  uint8_t* base = nullptr;
  PackArgs args{};
};

void release_canon(void* p) {
  DeviceCanon* c = static_cast<DeviceCanon*>(p);
  if (!c) return;
  for (void* a : c->alloc) if (a) cudaFree(a);
  delete c;
}

#define TL3_PK_CUDA(expr)                                     \
  do {                                                        \
    cudaError_t e_ = (expr);                                  \
    if (e_ != cudaSuccess) {                                  \
      tl3::set_cuda_error(static_cast<int>(e_));              \
      return TL3_ERR_CUDA;                                    \
    }                                                         \
  } while (0)

// Copies the canonical arrays of the handle to the device (one allocation, kept in the handle) and
// fills the kernel arguments that point into it.
int canon_to_device(tl3_matrix* m, cudaStream_t st, PackArgs* out) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const size_t sz[9] = {m->tc_vals.size() * 2, m->tc_meta.size(), m->chain_tau0.size() * 2, m->chain_rho0.size() * 2, m->chain_len.size(),
                        m->pdd_bytes.size(), m->tile_dir.size() * 4, m->res_rho.size() * 2, m->res_val.size() * 2};
  const void* src[9] = {m->tc_vals.data(), m->tc_meta.data(), m->chain_tau0.data(), m->chain_rho0.data(), m->chain_len.data(),
                        m->pdd_bytes.data(), m->tile_dir.data(), m->res_rho.data(), m->res_val.data()};
  size_t off[10];
  off[0] = 0;
  for (int i = 0; i < 9; ++i) off[i + 1] = off[i] + up(sz[i] + 16);
  if (!m->device_canon) {
    if (!m->host_arrays) return TL3_ERR_UNSUPPORTED;           // a device-only handle whose container has been packed and released
    void* p = nullptr;
    TL3_PK_CUDA(cudaMalloc(&p, off[9]));
    DeviceCanon* c = new (std::nothrow) DeviceCanon();
    if (!c) { cudaFree(p); return TL3_ERR_NO_MEMORY; }
    uint8_t* b = static_cast<uint8_t*>(p);
    *c = DeviceCanon{reinterpret_cast<const uint16_t*>(b + off[0]), b + off[1], reinterpret_cast<const uint16_t*>(b + off[2]),
                     reinterpret_cast<const uint16_t*>(b + off[3]), b + off[4], b + off[5], reinterpret_cast<const uint32_t*>(b + off[6]),
                     reinterpret_cast<const uint16_t*>(b + off[7]), reinterpret_cast<const uint16_t*>(b + off[8]), {p, nullptr}};
    m->device_canon = c;
    m->release_device_canon = release_canon;
    for (int i = 0; i < 9; ++i)
      if (sz[i]) TL3_PK_CUDA(cudaMemcpyAsync(b + off[i], src[i], sz[i], cudaMemcpyHostToDevice, st));
  }
  const DeviceCanon* c = static_cast<const DeviceCanon*>(m->device_canon);
  PackArgs a{};
  a.tc_vals = c->tc_vals;
  a.tc_meta = c->tc_meta;
  a.chain_tau0 = c->chain_tau0;
  a.chain_rho0 = c->chain_rho0;
  a.chain_len = c->chain_len;
  a.pdd_bytes = c->pdd_bytes;
  a.tile_dir = c->tile_dir;
  a.res_rho = c->res_rho;
  a.res_val = c->res_val;
  a.K_pad = m->K_pad;
  a.tiles_k = static_cast<int>(m->tiles_k);
  *out = a;
  return TL3_OK;
}

int configure_pack_kernel() {
  static bool done[64] = {};
  int dev = 0;
  TL3_PK_CUDA(cudaGetDevice(&dev));
  if (dev < 64 && done[dev]) return TL3_OK;
  TL3_PK_CUDA(cudaFuncSetAttribute(tl3_pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(PackSmem))));
  if (dev < 64) done[dev] = true;
  return TL3_OK;
}

}  // namespace
}  // namespace tl3

extern "C" int tl3_plan_device(tl3_matrix* m, void* stream) {
  using namespace tl3;
  if (!m) return TL3_ERR_INVALID_ARG;
  if (m->p.tile_m != kTileM || m->p.tile_k != kTileK) return TL3_ERR_UNSUPPORTED;
  if (m->layout_ready.load(std::memory_order_acquire)) return TL3_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (int rc = configure_pack_kernel()) return rc;
  PackArgs a{};
  if (int rc = canon_to_device(m, st, &a)) return rc;
  uint32_t* d_sizes = nullptr;
  TL3_PK_CUDA(cudaMalloc(reinterpret_cast<void**>(&d_sizes), static_cast<size_t>(m->n_tiles) * 12));
  a.sizes = d_sizes;
  a.emit = 0;
  tl3_pack_kernel<<<static_cast<unsigned>(m->n_tiles), 128, sizeof(PackSmem), st>>>(a);
  std::vector<uint32_t> sizes;
  int rc = TL3_OK;
  try { sizes.resize(static_cast<size_t>(m->n_tiles) * 3); } catch (const std::bad_alloc&) { rc = TL3_ERR_NO_MEMORY; }
  cudaError_t e = cudaGetLastError();
  if (rc == TL3_OK && e == cudaSuccess) e = cudaMemcpyAsync(sizes.data(), d_sizes, sizes.size() * 4, cudaMemcpyDeviceToHost, st);
  if (rc == TL3_OK && e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFree(d_sizes);
  if (rc != TL3_OK) return rc;
  if (e != cudaSuccess) { set_cuda_error(static_cast<int>(e)); return TL3_ERR_CUDA; }
  set_device_layout(m, sizes.data());
  return TL3_OK;
}

extern "C" int tl3_upload_device(tl3_matrix* m, void* dptr, void* stream) {
  using namespace tl3;
  if (!m || !dptr || (reinterpret_cast<uintptr_t>(dptr) & 255) != 0) return TL3_ERR_INVALID_ARG;
  if (m->p.tile_m != kTileM || m->p.tile_k != kTileK) return TL3_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (int rc = tl3_plan_device(m, stream)) return rc;          // no-op when the layout is known already
  if (int rc = configure_pack_kernel()) return rc;
  PackArgs a{};
  if (int rc = canon_to_device(m, st, &a)) return rc;
  uint8_t header[256];
  std::vector<unsigned long long> block_off;
  try { blob_header_and_offsets(m, header, &block_off); } catch (const std::bad_alloc&) { return TL3_ERR_NO_MEMORY; }
  unsigned long long* d_off = nullptr;
  TL3_PK_CUDA(cudaMalloc(reinterpret_cast<void**>(&d_off), block_off.size() * 8));
  cudaError_t e = cudaMemcpyAsync(d_off, block_off.data(), block_off.size() * 8, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(dptr, 0, m->device_bytes, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dptr, header, 256, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) {
    a.blob = static_cast<uint8_t*>(dptr);
    a.block_off = d_off;
    a.dir_offset = m->dir_offset;
    a.emit = 1;
    tl3_pack_kernel<<<static_cast<unsigned>(m->n_tiles), 128, sizeof(PackSmem), st>>>(a);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);          // header, offsets and the canonical copies are released below
  cudaFree(d_off);
  if (m->device_canon) { release_canon(m->device_canon); m->device_canon = nullptr; }
  if (e != cudaSuccess) { set_cuda_error(static_cast<int>(e)); return TL3_ERR_CUDA; }
  m->dptr = dptr;
  return TL3_OK;
}
