// Device side of libtl3: upload, workspace, and the SpMM kernel for sm_100a.
//
// Kernel design (what the paper's Sec. 4 pipeline becomes on B200):
//   * one persistent CTA per SM owns a contiguous range of 128 x 128 tiles in row-tile-major
//     order (split-K: a row-tile may be shared by several CTAs);
//   * a producer warp streams each tile's packed block (values + metadata + PDD codes + Residual)
//     with ONE bulk copy and the matching 128 x N block of X with one TMA tensor copy into a ring
//     of shared-memory stages (Sec. 4.2 "Efficient Matrix Loading": W streamed tile by tile, X
//     small enough to live in L2);
//   * four groups of four decode warps take the tiles in turn: copy the 2-bit metadata to tensor
//     memory, run Algorithm 1 (one PDD chain per thread, lane l on a chain whose empty slots lie
//     in shared-memory bank l) moving each parked value from W_t to a second 2:4 operand
//     W_r and zeroing its slot, and scatter the Residual entries into W_r as well
//     (Sec. 4.3; surplus weights always sit at in-window index 2 or 3, so W_r's metadata is the
//     constant pattern {2,3}); two more warps clear each W_r buffer as soon as its MMAs are done;
//   * one thread issues tcgen05.mma.sp (kind::f16, M = 128, K = 32) on W_t and on W_r into the
//     same fp32 accumulator in tensor memory (Sec. 4.3 "Sparse TC Computation");
//   * four epilogue warps read the accumulator; a row-tile owned by one CTA is written to Y
//     directly, otherwise the CTAs that share it store partial sums in the workspace and raise a
//     flag each, and the CTA that owns the row-tile's first tile collects them as the flags come
//     up and adds them in a fixed order (Sec. 4.4: a single reduction at the end of the pipeline).
// Every wait is bounded: on expiry the CTA records a code in the workspace status word, stops
// issuing work, waits for its copies in flight, frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_fp16.h>

#include <atomic>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <vector>

#include "tl3_internal.h"

namespace tl3 {

static thread_local int g_last_cuda_error = 0;
void set_cuda_error(int e) { g_last_cuda_error = e; }

#define TL3_CUDA(expr)                                        \
  do {                                                        \
    cudaError_t e_ = (expr);                                  \
    if (e_ != cudaSuccess) {                                  \
      tl3::set_cuda_error(static_cast<int>(e_));              \
      return TL3_ERR_CUDA;                                    \
    }                                                         \
  } while (0)

// ---------------------------------------------------------------------------------------------
// Kernel configuration
// ---------------------------------------------------------------------------------------------
constexpr int kGroups = 4;                // decode groups of four warps; tile i goes to group i % 4
constexpr int kProducerWarp = 0;
constexpr int kMmaWarp = 1;
constexpr int kAllocWarp = 2;
constexpr int kClearWarp0 = 2;            // warps 2 and 3 clear the W_r buffers (warp 2 also owns the TMEM allocation)
                                          // decode groups start at a multiple of four warps because a
                                          // warp reaches tensor-memory lanes 32*(warp%4)..+31
constexpr int kDecodeWarp0 = 4;           // warps 4-7: decode group 0, 8-11: group 1, ...
constexpr int kEpilogueWarp0 = kDecodeWarp0 + 4 * kGroups;
constexpr int kThreads = (kEpilogueWarp0 + 4) * 32;
constexpr int kSetupBarrier = 2 + kGroups;   // named barriers: 0 = whole CTA, 1 + kGroups = epilogue warps, 2 + kGroups = set-up
constexpr int kMaxStages = 8;
constexpr uint32_t kWrBytes = 16384;
constexpr int kMaxWrBuffers = 5;          // W_r ring: tile i uses buffer i % num_wr (4 or 5, see the launcher)
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColMetaT = 128;       // + 4 * (W_r buffer): metadata of W_t, four columns per tile in flight
constexpr uint32_t kColMetaR = 152;       // two columns of 0xEEEEEEEE
constexpr uint32_t kSmemLimit = 232448;   // 227 KB
constexpr uint32_t kBarrierBytes = 1024;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s without progress, per wait
#ifndef TL3_TRYWAIT_HINT_NS
#define TL3_TRYWAIT_HINT_NS 20000u
#endif
constexpr uint32_t kTryWaitHintNs = TL3_TRYWAIT_HINT_NS;     // how long one barrier probe may park the thread

// status codes written to the workspace status word (0 = ok)
enum : uint32_t {
  kStProducer = 1, kStDecodeFull = 2, kStDecodeWrFree = 3, kStMmaDecoded = 4, kStMmaAccEmpty = 5,
  kStEpilogueAccFull = 6, kStDrain = 7, kStClearWrFree = 8, kStDecodeWrReady = 9, kStEpilogueTail = 10, kStEpilogueFlags = 11, kStMmaX = 12,
  kStBadBlock = 16           // a block's lengths or a decoded position were out of range (+ detail in bits 8..)
};

struct KernelArgs {
  const uint8_t* blob;       // base of the packed blob (device)
  const DirEntry* dir;       // tile directory (device)
  long long total_tiles;
  int tiles_m, tiles_k;
  int M, N;
  long long ldy;
  __half* Y;
  const __half* bias;        // per output row, added before the activation (null: none)
  int act;                   // TL3_ACT_*
  float* partials;           // [2 * gridDim.x][n_pad][128]
  unsigned int* flags;       // [2 * gridDim.x] one per partial-sum slot: 1 = written and not yet collected
  unsigned int* status;      // status word
  uint32_t stage_stride;     // bytes per stage (block area + X tile), multiple of 1024
  uint32_t x_offset;         // offset of the X tile inside a stage, multiple of 1024
  int num_stages;
  int num_wr;                // W_r buffers (4 or 5)
  uint32_t opts;             // kOpt* bits
  long long* timing;         // time-stamp records (debug builds), else null
};

// Launch options (chosen by the launcher, see tl3_tuning):
//   kOptSplitX  the X tile of a stage completes on a barrier of its own, so that the decode of a
//               block starts when the block is there, whether or not the kernel before this one
//               (which may still be producing X) has finished; the MMA warp waits for both
enum : uint32_t { kOptSplitX = 1u };

// Optional per-CTA time stamps (build with -DTL3_CTA_STAMPS): one thread of a role writes the
// SM's cycle counter into record `blockIdx.x` of the buffer set with tl3_debug_set_timing_buffer()
// (plus the global timer once, at entry, read by a warp that idles then -- the read takes
// microseconds -- to line the CTAs of different SMs up).  Compiled out of the product.
#ifdef TL3_CTA_STAMPS
static long long* g_timing_buffer = nullptr;
static int g_timing_launch = 0;
__device__ __forceinline__ long long clock_now() { long long c; asm volatile("mov.u64 %0, %%clock64;" : "=l"(c) :: "memory"); return c; }
#define TL3_GT(k) { if (a.timing) a.timing[blockIdx.x * 32 + (k)] = clock_now(); }
#define TL3_GV(k, v) { if (a.timing) a.timing[blockIdx.x * 32 + (k)] = static_cast<long long>(v); }
#else
#define TL3_GT(k) {}
#define TL3_GV(k, v) {}
#endif

// ---------------------------------------------------------------------------------------------
// PTX helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ unsigned long long global_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {   // more bytes to come, no arrival
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One probe of the barrier phase.  The hint lets the hardware park the thread (up to that many
// nanoseconds, or until the phase completes) instead of spinning, so waiting warps do not take
// issue slots from the warps that have work.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred q;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(done) : "r"(bar), "r"(parity), "r"(kTryWaitHintNs) : "memory");
  return done != 0;
}

// Shared state every wait looks at: the abort flag (set by whoever gives up first) and the
// status word in global memory.
struct WaitCtx {
  volatile int* abort_flag;
  unsigned int* status;
};

// Bounded wait.  Returns false if the CTA is aborting (this or another waiter ran out of time).
// The limit runs from the moment THIS wait began to look slow (its sixteenth unsuccessful probe), not
// from the start of the kernel: a wait that completes is progress, so a long launch, or one whose
// context was switched out for a while earlier on, does not use up the allowance of later waits.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& w, uint32_t code) {
  unsigned long long t_slow = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 15u) == 15u) {
      if (*w.abort_flag) return false;
      const unsigned long long now = global_timer();
      if (t_slow == 0) t_slow = now;
      if (now - t_slow > kWaitLimitNs) {
        atomicCAS(w.status, 0u, code);
        *w.abort_flag = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// barrier + AND-reduction of a predicate over the `threads` threads that use barrier `id`
__device__ __forceinline__ bool named_bar_all(int id, int threads, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %3, 0;\n\t"
      "bar.red.and.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out) : "r"(id), "r"(threads), "r"(static_cast<uint32_t>(pred)) : "memory");
  return out != 0;
}

// The weight blocks are read once: they are marked evict-first in L2 so that what is read again
// (X, the kernel's own code, partial sums) is not pushed out by the stream.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// Programmatic dependent launch: the next kernel on the stream may be scheduled as soon as every
// CTA of this one has said so (it still cannot take an SM before a CTA here exits), and a kernel
// must call pdl_wait() before it reads what its predecessor wrote or writes what its
// predecessor may still read.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// One lane of a converged warp; the caller keeps every operand warp-uniform so that the
// single-thread instructions (bulk copies, MMAs, commits) take uniform registers directly.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xFFFFFFFF;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}

// D[tmem] (+)= A_sparse[smem] * B[smem] with the 2-bit metadata at e_tmem.  The shared-memory
// descriptors are passed as their low words (start address field) and one common high word each.
__device__ __forceinline__ void umma_sp_f16(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                            uint32_t e_tmem, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %7, 0;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], da, db, [%5], %6, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Positions in a block are bank-major slot coordinates u = bank << 8 | slot-in-window << 7 | row,
// where bank is the 32-bit word of the 128-byte (swizzled) row that holds the slot's window.  The
// byte offset of slot u inside the 128 x 128-byte K-major image is therefore a bit-field move:
// row * 128 + bank * 4 + slot-in-window * 2.  The packer orders both PDD streams by u and gives
// lane l of a decode warp a chain whose empty slots all lie in bank l.
__device__ __forceinline__ uint32_t swizzled_offset(uint32_t u) { return ((u & 0x7Fu) << 7) | ((u >> 6) & 0x7Eu); }

// Epilogue of tl3_spmm_ex: y = act(sum + bias), in fp32, before the rounding to fp16.  A real
// call, not inlined: it is used from many unrolled places, and a kernel image that grows by tens of
// kilobytes costs every launch time at its start.
__device__ __noinline__ float finish(float v, float bias, int act) {
  v += bias;
  if (act == TL3_ACT_RELU) return fmaxf(v, 0.f);
  if (act == TL3_ACT_SILU) return v / (1.f + __expf(-v));
  if (act == TL3_ACT_GELU_TANH) return 0.5f * v * (1.f + tanhf(0.7978845608f * (v + 0.044715f * v * v * v)));
  return v;
}

template <int NPAD> struct TmemLd;
template <> struct TmemLd<16> {
  static __device__ __forceinline__ void ld(uint32_t taddr, uint32_t* v) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr) : "memory");
  }
};
template <> struct TmemLd<32> {
  static __device__ __forceinline__ void ld(uint32_t taddr, uint32_t* v) {
    TmemLd<16>::ld(taddr, v);
    TmemLd<16>::ld(taddr + 16, v + 16);
  }
};
template <> struct TmemLd<64> {
  static __device__ __forceinline__ void ld(uint32_t taddr, uint32_t* v) {
    TmemLd<32>::ld(taddr, v);
    TmemLd<32>::ld(taddr + 32, v + 32);
  }
};

// CTA c of G owns tiles [c*T/G, (c+1)*T/G); the CTA that owns tile t.  In 32 bits: the launcher
// refuses matrices with (G + 1) * T >= 2^32 (hundreds of gigabytes), and a 64-bit division costs a
// CTA 0.15 us each at its cold start, where there are three of them.
__device__ __forceinline__ uint32_t range_begin(uint32_t c, uint32_t T, uint32_t G) { return c * T / G; }
__device__ __forceinline__ int owner_of(uint32_t t, uint32_t T, uint32_t G) { return static_cast<int>(((t + 1u) * G - 1u) / T); }

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts_u16(uint32_t addr, uint32_t v) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(static_cast<uint16_t>(v)) : "memory");
}
__device__ __forceinline__ void sts_zero16B(uint32_t addr) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
}

// Algorithm 1 for one chain, one code word (four delta bytes) at a time.  `pos` carries offset_t in
// its low and offset_r in its high 16 bits (both as bank-major coordinates u), so one add advances
// both cursors and two shift/mask pairs form both byte offsets.  Within a round all positions are
// formed first, then all W_t loads are issued, then all stores, so that the shared-memory round
// trips of different entries overlap.  (Rounds of two code words, and a software-pipelined loop
// that issues the next round's loads before this round's stores, both measured slower.)

// packed byte offsets (W_t offset low, W_r offset high) of the packed positions `pos`
__device__ __forceinline__ uint32_t swizzled_offset2(uint32_t pos) { return ((pos & 0x007F007Fu) << 7) | ((pos >> 6) & 0x007E007Eu); }

// Positions are checked (< 8192 slots per tile) before they become addresses; a violation is
// reported in *bad and the entry is skipped.  The code words of a tile are stored transposed
// (word k of chain slot j at (k * 128 + j) * 4) and every chain has `n_words` of them (<= 3, padded
// with zero bytes = dummy points), so the loads are conflict free and the loop is warp-uniform.
__device__ __forceinline__ void decode_chain(uint32_t stage, uint32_t wr, uint32_t hdr, uint32_t code_addr, uint32_t n_words, uint32_t* bad) {
  if (hdr == 0xFFFFFFFFu) return;                       // empty chain
  if (hdr & 0xE000E000u) { *bad = 1u; return; }
  uint32_t pos = hdr;
  uint32_t w[3] = {0u, 0u, 0u};
#pragma unroll
  for (int k = 0; k < 3; ++k)
    if (static_cast<uint32_t>(k) < n_words) w[k] = lds_u32(code_addr + k * 512);
  {                                                     // first pair: absolute 16-bit positions
    const uint32_t off2 = swizzled_offset2(pos);
    const uint32_t at = stage + (off2 & 0xFFFFu);
    const uint32_t v = lds_u16(at);
    sts_u16(at, 0);                                     // the slot it was parked in is empty again
    sts_u16(wr + (off2 >> 16), v);                      // the value goes to its own position in W_r
  }
#pragma unroll
  for (int k = 0; k < 3; ++k) {                         // one code word = four delta bytes
    if (static_cast<uint32_t>(k) >= n_words) break;
    const uint32_t bytes = w[k];
    uint32_t off2[4], val[4];
    bool real[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint32_t bt = __byte_perm(bytes, 0u, 0x4440u + q);    // delta byte q
      const uint32_t delta = (bt * 0x1001u) & 0x000F000Fu;        // t delta | r delta << 16
      pos += delta;
      real[q] = ((delta - 0x00010001u) & 0x80008000u) == 0u;      // both nibbles non-zero (else a dummy point)
      off2[q] = swizzled_offset2(pos);
    }
    // both cursors only grow, so the last position of the round bounds them all
    if (pos & 0xE000E000u) {
      *bad = 2u;
#pragma unroll
      for (int q = 0; q < 4; ++q) real[q] = false;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (real[q]) val[q] = lds_u16(stage + (off2[q] & 0xFFFFu));
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (real[q]) { sts_u16(stage + (off2[q] & 0xFFFFu), 0); sts_u16(wr + (off2[q] >> 16), val[q]); }
  }
}

// XT: the activations are given as X^T (N x K row-major, the [batch, hidden] layout of an inference
// stack, Sec. 2.1) and the result is written as Y^T (N x M row-major).  The X tile then arrives as
// two boxes of 64 k-values (128 bytes per row, 128-byte swizzle) and is a K-major B operand.
template <int NPAD, bool XT>
__global__ void __launch_bounds__(kThreads, 1)
tl3_spmm_kernel(const __grid_constant__ CUtensorMap x_map, const KernelArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int S = a.num_stages;
  const int NW = a.num_wr;
  uint8_t* wr_base = smem + static_cast<size_t>(S) * a.stage_stride;           // NW x 16 KB
  uint8_t* bar_base = wr_base + NW * kWrBytes;
  // barrier block: full[8] mma_done[8] decoded[8] acc_full[2] acc_empty[2] | tmem slot | flags | tail | wr_ready[5] wr_free[5] | x_full[8]
  uint64_t* bars = reinterpret_cast<uint64_t*>(bar_base);
  const uint32_t bar_full = smem_u32(bars), bar_mma = smem_u32(bars + 8), bar_dec = smem_u32(bars + 16);
  const uint32_t bar_accfull = smem_u32(bars + 24), bar_accempty = smem_u32(bars + 26), bar_wrready = smem_u32(bars + 44), bar_wrfree = smem_u32(bars + 49);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 33);
  const uint32_t bar_tail = smem_u32(bars + 36);               // partial sums fetched into the idle stages at the very end
  const uint32_t bar_xfull = smem_u32(bars + 56);              // [8] X tile of a stage (kOptSplitX)
  const bool split_x = (a.opts & kOptSplitX) != 0u;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) { TL3_GT(0) }
  if (tid == kEpilogueWarp0 * 32) { TL3_GT(1) TL3_GV(14, global_timer()) }
  const uint32_t T = static_cast<uint32_t>(a.total_tiles), G = gridDim.x;
  const uint32_t t_begin = range_begin(blockIdx.x, T, G), t_end = range_begin(blockIdx.x + 1, T, G);
  const int n_tiles = static_cast<int>(t_end - t_begin);
  const int kt_begin = static_cast<int>(t_begin % a.tiles_k);
  // Decode groups in use: a group may wait for its next tile only once the stage's previous
  // phase has completed (a parity wait cannot tell phases two apart), which holds as long as
  // there are no more groups than stages.  Tile i goes to group i % AG and W_r buffer i % NW.
  const int AG = S < kGroups ? S : kGroups;
  const uint32_t smem_base = smem_u32(smem);

  // Set-up.  The producer warp starts the (cold) global fetches of its first directory entries and
  // of the X tensor map, initialises the barriers -- lane l words l and l + 32 of the block, two
  // instructions instead of 57 in a row -- and goes on to request its first blocks without waiting
  // for the tensor-memory allocation, which it does not use: it only arrives at the set-up barrier,
  // the other warps wait there for it and for the allocating warp.
  uint4 dir_first = make_uint4(0, 0, 0, 0);
  if (tid == 0) { TL3_GT(28) }                                   // (ranges known)
  if (warp == kProducerWarp) {
    if (lane < n_tiles) dir_first = __ldg(reinterpret_cast<const uint4*>(a.dir + t_begin + lane));
    if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&x_map) : "memory");
    if (lane == 0) { TL3_GT(30) }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int i = lane + 32 * h;                                // word of the barrier block (layout above)
      const uint32_t count = i < 16 ? 1u : i < 24 ? 128u : i < 26 ? 1u : i < 28 ? 128u : i == 36 ? 1u
                           : (i >= 44 && i < 44 + kMaxWrBuffers) ? 64u : (i >= 49 && i < 49 + kMaxWrBuffers) ? 1u : i >= 56 ? 1u : 0u;
      if (count) mbar_init(smem_u32(bars + i), count);
    }
    if (lane == 0) *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    if (lane == 0) { TL3_GT(16) }
  }
  if (warp == kAllocWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    if (lane == 0) { TL3_GT(19) }
  }
  tc_fence_before();
  if (warp == kProducerWarp) asm volatile("bar.arrive %0, %1;" ::"r"(kSetupBarrier), "r"(kThreads) : "memory");
  else named_bar_sync(kSetupBarrier, kThreads);
  tc_fence_after();
  if (tid == 0) { TL3_GT(17) }
  const uint32_t tmem_base = warp == kProducerWarp ? 0u : *tmem_slot;   // (written by the allocating warp before it arrives)
  const WaitCtx wctx{abort_flag, a.status};
  pdl_launch_dependents();

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ producer
    // The whole warp runs the loop with warp-uniform state; one elected lane issues the copies.
    // Directory entries are read 32 at a time (one per lane) and broadcast with shuffles.
    // The weight blocks never depend on the kernel that ran before this one, X may: the blocks of
    // the first S tiles are requested at once, then the warp waits for the predecessor, then X.
    constexpr uint32_t kXBytes = 128u * NPAD * 2u;
    int issued = 0, s = 0, kt = kt_begin;
    uint32_t ph = 0;                                            // phase of the stage's current use
    uint32_t stage = smem_base;
    bool alive = true;
    const int pre = n_tiles < S ? n_tiles : S;                  // tiles whose stages are free at the start
    for (int base = 0; base < n_tiles && alive; base += 32) {
      uint4 mine = dir_first;
      if (base > 0) {
        mine = make_uint4(0, 0, 0, 0);
        if (base + lane < n_tiles) mine = __ldg(reinterpret_cast<const uint4*>(a.dir + t_begin + base + lane));
      }
      const int cnt = n_tiles - base < 32 ? n_tiles - base : 32;
      if (base == 0) {
        // S <= 8 < 32: all in this batch, and lane j holds the entry of tile j -- the lanes request
        // their blocks side by side (one after the other took 0.09 us per request)
        if (lane == 0 && mine.x != 0xFFFFFFFFu) { TL3_GT(18) }
        if (lane < pre) {
          const uint32_t full = bar_full + 8 * lane;
          mbar_arrive_expect_tx(full, split_x ? mine.y : mine.y + kXBytes);
          bulk_copy_g2s(smem_base + static_cast<uint32_t>(lane) * a.stage_stride, a.blob + static_cast<size_t>(mine.x) * 16, mine.y, full);
        }
        __syncwarp();
        if (lane == 0) { TL3_GT(2) }
        pdl_wait();
        if (lane == 0) { TL3_GT(3) }
      }
      for (int j = 0; j < cnt; ++j) {
        const uint32_t off16 = __shfl_sync(0xFFFFFFFFu, mine.x, j), bytes = __shfl_sync(0xFFFFFFFFu, mine.y, j);
        const int i = base + j;
        if (i >= S) alive = __all_sync(0xFFFFFFFFu, mbar_wait(bar_mma + 8 * s, ph ^ 1u, wctx, kStProducer));
        if (!alive) break;
        const uint32_t full = bar_full + 8 * s;
        const uint32_t xbar = split_x ? bar_xfull + 8 * s : full;
        const uint8_t* src = a.blob + static_cast<size_t>(off16) * 16;
        if (elect_one()) {
          if (i >= pre) {
            mbar_arrive_expect_tx(full, split_x ? bytes : bytes + kXBytes);
            bulk_copy_g2s(stage, src, bytes, full);
          }
          if (split_x) mbar_arrive_expect_tx(xbar, kXBytes);
          if (XT) {
            tma_load_2d(stage + a.x_offset, &x_map, kt * kTileK, 0, xbar);
            tma_load_2d(stage + a.x_offset + NPAD * 128u, &x_map, kt * kTileK + 64, 0, xbar);
          } else {
            tma_load_2d(stage + a.x_offset, &x_map, 0, kt * kTileK, xbar);
          }
        }
        __syncwarp();
        if (lane == 0) { if (i == 0) { TL3_GT(4) } if (i == n_tiles - 1) { TL3_GT(8) } }
        issued = i + 1;
        stage += a.stage_stride;
        if (++s == S) { s = 0; ph ^= 1u; stage = smem_base; }
        if (++kt == a.tiles_k) kt = 0;
      }
    }
    if (lane == 0 && *abort_flag) {
      // let the copies still in flight land before the CTA goes away
      const int first = issued > S ? issued - S : 0;
      for (int i = first; i < issued; ++i) {
        const unsigned long long t1 = global_timer();
        for (int which = 0; which < (split_x ? 2 : 1); ++which) {
          const uint32_t bar = (which ? bar_xfull : bar_full) + 8 * (i % S);
          while (!mbar_try_wait(bar, (i / S) & 1)) {
            if (global_timer() - t1 > kWaitLimitNs / 4) { atomicCAS(a.status, 0u, (uint32_t)kStDrain); break; }
          }
        }
      }
    }
  } else if (warp == kClearWarp0 || warp == kClearWarp0 + 1) {
    // ------------------------------------------------------------------ W_r clearing
    // Tile i scatters into W_r buffer i % NW.  These two warps zero a buffer as soon as the MMAs
    // of tile i - NW (its previous user) are done (the MMA warp commits to the buffer's own
    // barrier) and then open it for the decode warps, so the decode path neither clears nor needs
    // a group-wide barrier.
    const int ct = tid - kClearWarp0 * 32;                       // 0..63
    const uint32_t wr0 = smem_u32(wr_base);
    int wb = 0, use = 0;                                         // buffer of tile i, and how often it was filled before
    for (int i = 0; i < n_tiles; ++i) {
      bool ok = true;
      if (use >= 1) ok = mbar_wait(bar_wrfree + 8 * wb, (use - 1) & 1, wctx, kStClearWrFree);
      if (!__all_sync(0xFFFFFFFFu, ok)) break;
      const uint32_t wr = wr0 + wb * kWrBytes;
#pragma unroll
      for (int c = 0; c < 16; ++c) sts_zero16B(wr + (c * 64 + ct) * 16);
      fence_proxy_async_smem();                                  // the MMA reads what stays zero
      mbar_arrive(bar_wrready + 8 * wb);
      if (++wb == NW) { wb = 0; ++use; }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    // Warp-uniform loop; one elected lane issues the eight MMAs of a tile and the commits.
    // instruction descriptor: sparse, D = f32, A = B = f16, A K-major, B MN-major, N = NPAD, M = 128
    const uint32_t idesc = (1u << 2) | (1u << 4) | (XT ? 0u : (1u << 16)) | (static_cast<uint32_t>(NPAD >> 3) << 17) | (8u << 24);
    // Shared-memory descriptors: low word = start address >> 4 (+ an unused leading-offset field),
    // high word = stride between 8-row groups, descriptor version, swizzle mode.
    // A: K-major, 128-byte swizzle, 8-row groups 1024 B apart; a 32-wide k-block is 32 bytes of a row.
    // B: X block, k rows of NPAD*2 bytes, swizzle span = row pitch, 8-row groups 8*pitch apart;
    //    a k-block is 32 rows.
    constexpr uint32_t kAHi = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t kBLayout = NPAD == 16 ? 6u : NPAD == 32 ? 4u : 2u;
    //    With XT: two sub-tiles of NPAD rows x 128 bytes (64 k-values each), K-major, 128-byte swizzle,
    //    8-row groups 1024 B apart; a k-block is 64 bytes of a row.
    constexpr uint32_t kBHi = XT ? ((1024u >> 4) | (1u << 14) | (2u << 29)) : (((8u * NPAD * 2u) >> 4) | (1u << 14) | (kBLayout << 29));
    constexpr uint32_t kLboOne = 1u << 16;
    constexpr uint32_t kAStep = 32u >> 4;
    auto b_step = [](int kb) -> uint32_t {                       // descriptor offset of k-block kb inside the X tile
      return XT ? ((static_cast<uint32_t>(kb >> 1) * (NPAD * 128u) + static_cast<uint32_t>(kb & 1) * 64u) >> 4)
                : (static_cast<uint32_t>(kb) * ((32u * NPAD * 2u) >> 4));
    };
    const uint32_t a_lo0 = (smem_base >> 4) | kLboOne, stride16 = a.stage_stride >> 4, x16 = a.x_offset >> 4;
    const uint32_t w_lo0 = (smem_u32(wr_base) >> 4) | kLboOne;
    int seg = 0, s = 0, kt = kt_begin, wb = 0;
    uint32_t ph = 0, a_lo = a_lo0;
    for (int i = 0; i < n_tiles; ++i) {
      const bool first_of_seg = (i == 0) || (kt == 0);
      const bool last_of_seg = (i == n_tiles - 1) || (kt == a.tiles_k - 1);
      const int b = seg & 1;
      bool ok = true;
      if (first_of_seg && (seg >> 1) >= 1) ok = mbar_wait(bar_accempty + 8 * b, ((seg >> 1) - 1) & 1, wctx, kStMmaAccEmpty);
      ok = ok && mbar_wait(bar_dec + 8 * s, ph, wctx, kStMmaDecoded);
      if (split_x) ok = ok && mbar_wait(bar_xfull + 8 * s, ph, wctx, kStMmaX);
      if (!__all_sync(0xFFFFFFFFu, ok)) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(b * NPAD);
      const uint32_t e_t = tmem_base + kColMetaT + 4 * wb, e_r = tmem_base + kColMetaR;
      const uint32_t b_lo = a_lo + x16, w_lo = w_lo0 + wb * (kWrBytes >> 4);
      const uint32_t mma_bar = bar_mma + 8 * s, acc_bar = bar_accfull + 8 * b, wrfree_bar = bar_wrfree + 8 * wb;
      if (elect_one()) {
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
          const uint32_t id = idesc | static_cast<uint32_t>(kb & 1);
          umma_sp_f16(d_tmem, a_lo + kb * kAStep, kAHi, b_lo + b_step(kb), kBHi, e_t + (kb & ~1), id,
                      (first_of_seg && kb == 0) ? 0u : 1u);
          umma_sp_f16(d_tmem, w_lo + kb * kAStep, kAHi, b_lo + b_step(kb), kBHi, e_r, id, 1u);
        }
        umma_commit(mma_bar);         // frees the stage
        umma_commit(wrfree_bar);      // frees this tile's W_r buffer and metadata columns
        if (last_of_seg) umma_commit(acc_bar);
      }
      __syncwarp();
      if (lane == 0) { if (i == 0) { TL3_GT(7) } if (i == n_tiles - 1) { TL3_GT(9) } }
      if (last_of_seg) ++seg;
      a_lo += stride16;
      if (++s == S) { s = 0; ph ^= 1u; a_lo = a_lo0; }
      if (++kt == a.tiles_k) kt = 0;
      if (++wb == NW) wb = 0;
    }
  } else if (warp >= kDecodeWarp0 && warp < kEpilogueWarp0) {
    // ------------------------------------------------------------------ decode (Algorithm 1)
    const int g = (warp - kDecodeWarp0) >> 2;
    const int r = tid - (kDecodeWarp0 + 4 * g) * 32;            // chain / row / tensor-memory lane 0..127
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t wr0 = smem_u32(wr_base);
    if (g == 0) {   // constant metadata of W_r: every window selects in-window positions {2, 3}
      asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};"
                   ::"r"(tmem_base + lane_base + kColMetaR), "r"(0xEEEEEEEEu), "r"(0xEEEEEEEEu) : "memory");
    }
    int wb = g % NW, use = g / NW;                              // W_r buffer of tile i and how often it was filled before
    int s = g;                                                  // g < AG <= S
    uint32_t ph = 0;
    for (int i = g, j = 0; g < AG && i < n_tiles; i += AG, ++j) {
      // Warps of a group do not wait for each other.  The packed block lists chains longest
      // first, so the four warps get blocks of different length; the block a warp takes rotates
      // from tile to tile to even the load out.
      const int cr = (r + 32 * (j & 3)) & 127;                  // chain handled by this thread
      const uint32_t wr = wr0 + wb * kWrBytes;
      // Order matters.  The W_r buffer is ready once the MMAs of tile i - AG are done, and MMAs
      // are issued in tile order, so by then every tile up to i - AG -- in particular the previous
      // user of this stage, tile i - S -- has been loaded and consumed.  Only then is the parity
      // wait on the stage's `full` barrier unambiguous (loads may complete out of order, and a
      // parity wait cannot tell "two phases back" from "done").
      bool ok = mbar_wait(bar_wrready + 8 * wb, use & 1, wctx, kStDecodeWrReady);
      ok = ok && mbar_wait(bar_full + 8 * s, ph, wctx, kStDecodeFull);
      if (r == 0 && i == 0) { TL3_GT(5) }
      const uint32_t stage = smem_base + static_cast<uint32_t>(s) * a.stage_stride;
      uint32_t m0 = 0, m1 = 0, m2 = 0, m3 = 0, span = 0, hdr = 0xFFFFFFFFu, pdd_len = 0, res_cnt = 0;
      if (ok) {
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(m0), "=r"(m1), "=r"(m2), "=r"(m3) : "r"(stage + kMetaOff + r * 16));
        span = lds_u32(stage + kInfoOff + 8);                      // code words per chain
        hdr = lds_u32(stage + kHdrOff + cr * 4);
        pdd_len = lds_u32(stage + kInfoOff);
        res_cnt = lds_u32(stage + kInfoOff + 4);
      }
      if (!__all_sync(0xFFFFFFFFu, ok)) break;
      // metadata -> tensor memory (4 columns of this group)
      {
        asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(tmem_base + lane_base + kColMetaT + 4 * wb), "r"(m0), "r"(m1), "r"(m2), "r"(m3) : "memory");
      }
      const uint32_t n_words = span;
      uint32_t bad = 0;
      const uint32_t room = a.x_offset - kPddOff;               // bytes a block may use after its fixed part
      const bool lens_ok = pdd_len <= room && res_cnt <= room / 4 && ((pdd_len + 3u) & ~3u) + 4u * res_cnt <= room &&
                           n_words <= 3u && pdd_len == n_words * 512u;
      if (lens_ok) decode_chain(stage, wr, hdr, stage + kPddOff + cr * 4, n_words, &bad);
      else bad = 3u;
      __syncwarp();
      // Residual layer: (position, value) entries go to W_r too
      if (lens_ok) {
        const uint32_t res = stage + kPddOff + ((pdd_len + 3u) & ~3u);
        for (uint32_t k = r; k < res_cnt; k += 128) {
          const uint32_t rv = lds_u32(res + 4 * k);
          if ((rv & 0xFFFFu) < 8192u) sts_u16(wr + swizzled_offset(rv & 0xFFFFu), rv >> 16);
          else bad = 4u;
        }
      }
      if (bad) atomicCAS(a.status, 0u, kStBadBlock | (bad << 8) | (static_cast<uint32_t>(i) << 12));
      fence_proxy_async_smem();                                   // generic-proxy writes -> MMA reads
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      tc_fence_before();
      mbar_arrive(bar_dec + 8 * s);
      if (r == 0 && i == 0) { TL3_GT(6) }
      if (r == 0 && i == n_tiles - 1) { TL3_GT(15) }
      s += AG;
      while (s >= S) { s -= S; ph ^= 1u; }
      wb += AG;
      while (wb >= NW) { wb -= NW; ++use; }
    }
  } else if (warp >= kEpilogueWarp0) {
    // ------------------------------------------------------------------ epilogue
    const int et = tid - kEpilogueWarp0 * 32;                    // 0..127 = row of the tile = tensor-memory lane
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    int seg = 0;
    uint32_t t = t_begin;
    pdl_wait();   // Y, the partial sums and their flags may still be in use by the previous kernel
    while (t < t_end) {
      const int mt = static_cast<int>(t / a.tiles_k);
      const uint32_t row_tile_begin = static_cast<uint32_t>(mt) * static_cast<uint32_t>(a.tiles_k), row_tile_end = row_tile_begin + static_cast<uint32_t>(a.tiles_k);
      const uint32_t seg_end = row_tile_end < t_end ? row_tile_end : t_end;
      const bool complete = (t == row_tile_begin) && (seg_end == row_tile_end);
      const int b = seg & 1;
      const int c_first = owner_of(row_tile_begin, T, G), c_last = owner_of(row_tile_end - 1, T, G);
      const int row = mt * kTileM + et;
      float bias_v = 0.f;                                         // fetched before the wait: off the tail of the segment
      if (a.bias != nullptr && row < a.M) bias_v = __half2float(__ldg(a.bias + row));
      // A row-tile shared with other CTAs is finished by the CTA that owns its first tile.  That
      // CTA's range ends inside the row-tile (else the row-tile would not be shared), so this is
      // always the last segment it works on: nothing of its own is held up while it collects.
      const bool reducer = !complete && static_cast<int>(blockIdx.x) == c_first;
      const int n_others = c_last - c_first;
      if (!named_bar_all(1 + kGroups, 128, mbar_wait(bar_accfull + 8 * b, (seg >> 1) & 1, wctx, kStEpilogueAccFull))) break;
      if (et == 0 && seg_end == t_end) { TL3_GT(10) TL3_GV(13, reducer ? n_others : (complete ? 0 : -1)) }
      tc_fence_after();
      constexpr int CH = NPAD < 32 ? NPAD : 32;                 // columns handled per round (register budget)
      __half* y = XT ? a.Y + row : a.Y + static_cast<long long>(row) * a.ldy;   // XT: element (row, c) at y[c * ldy]
      // 16-byte stores when the columns fill them (N = 8 runs in the 16-column kernel)
      const bool vec_ok = !XT && (NPAD == 16 ? (a.N & 7) == 0 : a.N == NPAD) && (a.ldy & 7) == 0 && (reinterpret_cast<uintptr_t>(a.Y) & 15) == 0;
      const bool plain = a.bias == nullptr && a.act == TL3_ACT_NONE;
      auto fin = [](uint32_t bits) { return __uint_as_float(bits); };
      auto store_y = [&](uint32_t* v, int c0) {                 // (bias, activation,) fp32 -> fp16 (round to nearest even) -> Y
        if (row >= a.M) return;
        if (!plain) {                                             // one test per call, not one per element
#pragma unroll
          for (int c = 0; c < CH; ++c) v[c] = __float_as_uint(finish(__uint_as_float(v[c]), bias_v, a.act));
        }
        if (vec_ok) {
#pragma unroll
          for (int c = 0; c < CH; c += 8) {
            if (NPAD == 16 && c0 + c >= a.N) break;
            uint4 o;
            __half2 h0 = __floats2half2_rn(fin(v[c + 0]), fin(v[c + 1]));
            __half2 h1 = __floats2half2_rn(fin(v[c + 2]), fin(v[c + 3]));
            __half2 h2 = __floats2half2_rn(fin(v[c + 4]), fin(v[c + 5]));
            __half2 h3 = __floats2half2_rn(fin(v[c + 6]), fin(v[c + 7]));
            o.x = *reinterpret_cast<uint32_t*>(&h0); o.y = *reinterpret_cast<uint32_t*>(&h1);
            o.z = *reinterpret_cast<uint32_t*>(&h2); o.w = *reinterpret_cast<uint32_t*>(&h3);
            *reinterpret_cast<uint4*>(y + c0 + c) = o;
          }
        } else {
          if (XT) {
            __half* yc = y + static_cast<long long>(c0) * a.ldy;          // column c0 of this row: Yt[c0][row]
#pragma unroll
            for (int c = 0; c < CH; ++c, yc += a.ldy)
              if (c0 + c < a.N) *yc = __float2half_rn(fin(v[c]));
          } else {
#pragma unroll
            for (int c = 0; c < CH; ++c)
              if (c0 + c < a.N) y[c0 + c] = __float2half_rn(fin(v[c]));
          }
        }
      };
      const uint32_t acc_tmem = tmem_base + lane_base + static_cast<uint32_t>(b * NPAD);
      // partial sums of a shared row-tile: slot 2*cta + (this row-tile is not the first one of my range)
      const int slot = 2 * blockIdx.x + (t_begin < row_tile_begin ? 1 : 0);
      float* mine = a.partials + static_cast<size_t>(slot) * NPAD * 128 + et;
      if (reducer) {
        // The other contributors store their partial sums and then raise the flag of their slot.
        // One warp watches the flags and requests a slot the moment its flag is up (bulk copy into
        // the stages, idle by now), so that when the last contributor arrives only its slot is
        // still to come.  The sum runs in ascending CTA order whatever the order of arrival: the
        // result does not depend on timing.
        // Progress: a contributor waits for nobody, so it finishes once it holds an SM; the reducer
        // waits only for CTAs with a higher index, and blocks are dispatched in index order, so only
        // the reducers just below a launch's dispatch front can be waiting for a CTA that is not
        // resident yet.  The wait is bounded all the same (status code kStEpilogueFlags).
        constexpr uint32_t kSlotBytes = NPAD * 128u * 4u;
        const bool staged = seg_end == t_end && static_cast<uint32_t>(n_others) * kSlotBytes <= static_cast<uint32_t>(S) * a.stage_stride;
        bool ok = true;
        if (et < 32) {
          for (int base = 0; base < n_others && ok; base += 32) {
            const int k = base + et;                              // this lane watches contributor c_first + 1 + k
            bool pending = k < n_others;
            int sl = 0;
            if (pending) {
              const int c_id = c_first + 1 + k;
              sl = 2 * c_id + (range_begin(c_id, T, G) < row_tile_begin ? 1 : 0);
            }
            unsigned long long t_slow = 0;                        // limit counted from when this poll began to look slow
            for (uint32_t it = 0; __any_sync(0xFFFFFFFFu, pending); ++it) {
              if (pending) {
                unsigned int up;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(up) : "l"(a.flags + sl) : "memory");
                if (up != 0u) {
                  pending = false;
                  a.flags[sl] = 0u;                               // leave the workspace cleared
                  if (staged) {
                    fence_proxy_async_all();
                    mbar_expect_tx(bar_tail, kSlotBytes);
                    bulk_copy_g2s(smem_base + static_cast<uint32_t>(k) * kSlotBytes, a.partials + static_cast<size_t>(sl) * NPAD * 128, kSlotBytes, bar_tail);
                  }
                }
              }
              if ((it & 15u) == 15u) {
                const unsigned long long now = global_timer();
                if (t_slow == 0) t_slow = now;
                const bool out = *abort_flag != 0 || now - t_slow > kWaitLimitNs;
                if (__any_sync(0xFFFFFFFFu, out)) {
                  if (et == 0) { atomicCAS(a.status, 0u, static_cast<uint32_t>(kStEpilogueFlags)); *abort_flag = 1; }
                  ok = false;
                  break;
                }
              }
            }
          }
          __syncwarp();
          if (et == 0) { TL3_GT(20) }
          if (staged && et == 0) mbar_arrive(bar_tail);           // the phase ends when every requested slot has landed
        }
        bool fetched = named_bar_all(1 + kGroups, 128, ok);
        if (staged) {
          if (fetched) {
            fetched = mbar_wait(bar_tail, 0, wctx, kStEpilogueTail);
            if (et == 0) { TL3_GT(21) }
          } else if (et == 0) {                                   // giving up: still no exit with copies in flight
            for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(bar_tail, 0); ++it) {}
          }
        }
        if (fetched) {
          if (!staged) __threadfence();                           // the others' partial sums, after their flags
#pragma unroll 1
          for (int c0 = 0; c0 < NPAD; c0 += CH) {
            uint32_t v[CH];
            TmemLd<CH>::ld(acc_tmem + c0, v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            // own part first (lowest CTA), then the others in ascending order.  Two loops: in one
            // loop the slot arithmetic of the unstaged case (a 64-bit division per contributor)
            // was computed on the staged path too, 0.25 us on a reducer's way out.
            if (staged) {
              uint32_t p = smem_base + static_cast<uint32_t>(et) * 4u + static_cast<uint32_t>(c0) * 512u;
              for (int k = 0; k < n_others; ++k, p += NPAD * 512u) {
                uint32_t w[CH];
#pragma unroll
                for (int c = 0; c < CH; ++c) w[c] = lds_u32(p + static_cast<uint32_t>(c) * 512u);
#pragma unroll
                for (int c = 0; c < CH; ++c) v[c] = __float_as_uint(__uint_as_float(v[c]) + __uint_as_float(w[c]));
              }
            } else {
              for (int k = 0; k < n_others; ++k) {
                const int c_id = c_first + 1 + k;
                const int sl = 2 * c_id + (range_begin(c_id, T, G) < row_tile_begin ? 1 : 0);
                const float* p = a.partials + static_cast<size_t>(sl) * NPAD * 128 + et;
#pragma unroll
                for (int c = 0; c < CH; ++c) v[c] = __float_as_uint(__uint_as_float(v[c]) + __ldcg(p + (c0 + c) * 128));
              }
            }
            store_y(v, c0);
          }
        }
        tc_fence_before();
        mbar_arrive(bar_accempty + 8 * b);
        ++seg;
        t = seg_end;
        continue;
      }
#pragma unroll 1
      for (int c0 = 0; c0 < NPAD; c0 += CH) {
        uint32_t v[CH];
        TmemLd<CH>::ld(acc_tmem + c0, v);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (complete) {
          store_y(v, c0);
        } else {
#pragma unroll
          for (int c = 0; c < CH; ++c) __stcg(mine + (c0 + c) * 128, __uint_as_float(v[c]));
        }
      }
      tc_fence_before();
      mbar_arrive(bar_accempty + 8 * b);
      if (!complete) {
        __threadfence();                                          // the partial sums, before the flag
        named_bar_sync(1 + kGroups, 128);
        if (et == 0) asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(a.flags + slot), "r"(1u) : "memory");
        if (et == 0 && seg_end == t_end) { TL3_GT(22) }
      }
      ++seg;
      t = seg_end;
    }
  }

  // ------------------------------------------------------------------ teardown
  if (tid == kEpilogueWarp0 * 32) { TL3_GT(11) }
  tc_fence_before();
  __syncthreads();
  if (tid == kEpilogueWarp0 * 32) { TL3_GT(12) }
  if (warp == kAllocWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// Self-test of the bounded wait: one CTA waits on a barrier that nothing ever arrives at.  The
// wait gives up after its limit, records its code in the status word and the kernel returns; the
// context stays usable.
__global__ void bounded_wait_probe_kernel(unsigned int* status, unsigned int* outcome) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const WaitCtx w{&abort_flag, status};
  const bool completed = mbar_wait(smem_u32(&bar), 0, w, kStProducer);
  if (threadIdx.x == 0) *outcome = completed ? 1u : 2u;
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
struct DeviceInfo {
  int sm_count = 0;
  int cc_major = 0;
  bool ok = false;
};

static int device_info(DeviceInfo* out) {
  int dev = 0;
  TL3_CUDA(cudaGetDevice(&dev));
  static std::mutex mu;
  static std::vector<DeviceInfo> cache;
  std::lock_guard<std::mutex> lock(mu);
  if (static_cast<size_t>(dev) >= cache.size()) cache.resize(dev + 1);
  DeviceInfo& d = cache[dev];
  if (!d.ok) {
    TL3_CUDA(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
    TL3_CUDA(cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    d.ok = true;
  }
  *out = d;
  return TL3_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

static inline int n_pad_of(int N) { return N <= 16 ? 16 : N <= 32 ? 32 : 64; }

struct WorkspaceLayout {
  size_t status_off = 0, flags_off = 256, partials_off = 0, total = 0;
};

static WorkspaceLayout workspace_layout(const tl3_matrix* m, int n_pad, int sm_count) {
  WorkspaceLayout w;
  (void)m;
  w.partials_off = (256 + static_cast<size_t>(2) * sm_count * 4 + 4095) / 4096 * 4096;
  w.total = w.partials_off + static_cast<size_t>(2) * sm_count * n_pad * 128 * sizeof(float);
  return w;
}

// Process-wide launch tuning (tl3_set_tuning); the default is what measured best on B200.
static std::atomic<int> g_decode_before_x{TL3_DEFAULT_DECODE_BEFORE_X};

template <int NPAD, bool XT>
static int launch(const CUtensorMap& map, const KernelArgs& args, int grid, uint32_t smem_bytes, cudaStream_t stream) {
  // The opt-in to more than 48 KB of dynamic shared memory is a property of the function on ONE
  // device: it is set once per device and template instance.
  {
    int dev = 0;
    TL3_CUDA(cudaGetDevice(&dev));
    static std::mutex mu;
    static std::vector<char> configured;
    std::lock_guard<std::mutex> lock(mu);
    if (static_cast<size_t>(dev) >= configured.size()) configured.resize(dev + 1, 0);
    if (!configured[dev]) {
      TL3_CUDA(cudaFuncSetAttribute(tl3_spmm_kernel<NPAD, XT>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemLimit)));
      configured[dev] = 1;
    }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see pdl_wait() in the kernel
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  TL3_CUDA(cudaLaunchKernelEx(&cfg, tl3_spmm_kernel<NPAD, XT>, map, args));
  TL3_CUDA(cudaGetLastError());
  return TL3_OK;
}

}  // namespace tl3

extern "C" {

size_t tl3_device_bytes(const tl3_matrix* m) {
  if (!m) return 0;
  return tl3::plan_device_layout(m);
}

int tl3_pack(const tl3_matrix* m, void* host_buf, size_t bytes) {
  if (!m || !host_buf) return TL3_ERR_INVALID_ARG;
  if (!m->host_arrays) return TL3_ERR_UNSUPPORTED;               // tl3_encode_device_only: pack with tl3_upload_device
  if (m->p.tile_m != tl3::kTileM || m->p.tile_k != tl3::kTileK) return TL3_ERR_UNSUPPORTED;
  if (bytes < tl3::plan_device_layout(m)) return TL3_ERR_INVALID_ARG;
  tl3::pack_device_blob(m, static_cast<uint8_t*>(host_buf));
  return TL3_OK;
}

int tl3_upload(tl3_matrix* m, void* dptr, void* stream) {
  if (!m || !dptr || (reinterpret_cast<uintptr_t>(dptr) & 255) != 0) return TL3_ERR_INVALID_ARG;
  if (m->p.tile_m != tl3::kTileM || m->p.tile_k != tl3::kTileK) return TL3_ERR_UNSUPPORTED;
  if (!m->host_arrays) return TL3_ERR_UNSUPPORTED;               // tl3_encode_device_only: pack with tl3_upload_device
  const size_t bytes = tl3::plan_device_layout(m);
  std::vector<uint8_t> staging;
  try {
    staging.resize(bytes);
  } catch (const std::bad_alloc&) {
    return TL3_ERR_NO_MEMORY;
  }
  tl3::pack_device_blob(m, staging.data());
  // pageable source: the runtime returns once the data sits in its own staging buffers
  TL3_CUDA(cudaMemcpyAsync(dptr, staging.data(), bytes, cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream)));
  m->dptr = dptr;
  return TL3_OK;
}

int tl3_bind(tl3_matrix* m, void* dptr) {
  if (!m || !dptr || (reinterpret_cast<uintptr_t>(dptr) & 255) != 0) return TL3_ERR_INVALID_ARG;
  if (m->p.tile_m != tl3::kTileM || m->p.tile_k != tl3::kTileK) return TL3_ERR_UNSUPPORTED;
  tl3::plan_device_layout(m);
  m->dptr = dptr;
  return TL3_OK;
}

size_t tl3_workspace_bytes(const tl3_matrix* m, int N) {
  if (!m || N < 1 || N > TL3_MAX_N) return 0;
  tl3::DeviceInfo di;
  if (tl3::device_info(&di) != TL3_OK) return 0;
  return tl3::workspace_layout(m, tl3::n_pad_of(N), di.sm_count).total;
}

int tl3_workspace_init(void* workspace, size_t bytes, void* stream) {
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return TL3_ERR_INVALID_ARG;
  TL3_CUDA(cudaMemsetAsync(workspace, 0, bytes, static_cast<cudaStream_t>(stream)));
  return TL3_OK;
}

// one launch: at most 64 columns
// (xt: X and Y are given transposed, N x K and N x M row-major)
static int spmm_block(const tl3_matrix* m, const void* X, int64_t ldx, void* Y, int64_t ldy, int N, const tl3_epilogue* ep, bool xt,
                      void* workspace, void* stream) {
  using namespace tl3;
  if (N < 1 || N > 64) return TL3_ERR_UNSUPPORTED;
  if (ldx < (xt ? m->K : N) || ldy < (xt ? m->M : N) || (ldx & 7) != 0 || (reinterpret_cast<uintptr_t>(X) & 15) != 0 ||
      (reinterpret_cast<uintptr_t>(Y) & 1) != 0 || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0)
    return TL3_ERR_INVALID_ARG;
  DeviceInfo di;
  if (int rc = device_info(&di)) return rc;
  if (di.cc_major != 10) return TL3_ERR_UNSUPPORTED;
  const int n_pad = n_pad_of(N);

  // shared-memory plan
  const uint32_t block_area = (m->max_block_bytes + 1023u) / 1024u * 1024u;
  const uint32_t x_bytes = 128u * n_pad * 2u;
  const uint32_t stage_stride = block_area + x_bytes;
  // W_r ring of five buffers, or four if that makes room for one more stage (measured on
  // 20480 x 5120, N = 16: 5 buffers + 5 stages 28.7 us, 4 + 6 28.1 us, 3 + 7 slower); the rest of
  // the shared memory is stages
  int num_wr = kMaxWrBuffers, stages = 0;
  uint32_t fixed = 0;
  {
    auto plan = [&](int nw) {
      const uint32_t f = nw * kWrBytes + kBarrierBytes + 1024u;              // + alignment slack
      return f + stage_stride <= kSmemLimit ? static_cast<int>((kSmemLimit - f) / stage_stride) : 0;
    };
    const int s5 = plan(kMaxWrBuffers), s4 = plan(4);
    if (s4 > s5 && s5 < kMaxStages) num_wr = 4;
    stages = num_wr == 4 ? s4 : s5;
    fixed = num_wr * kWrBytes + kBarrierBytes + 1024u;
  }
  if (stages < 2) return TL3_ERR_UNSUPPORTED;
  if (stages > kMaxStages) stages = kMaxStages;
  const uint32_t smem_bytes = fixed + static_cast<uint32_t>(stages) * stage_stride;

  // tensor map of X: dims {N, K}, box {n_pad, 128}; columns >= N and rows >= K read as zero
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return TL3_ERR_UNSUPPORTED;
  CUtensorMap map;
  // (transposed: dims {K, N}, box {64, n_pad}, two boxes per tile)
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(xt ? m->K : N), static_cast<cuuint64_t>(xt ? N : m->K)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldx) * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(xt ? 64 : n_pad), static_cast<cuuint32_t>(xt ? n_pad : 128)};
  const cuuint32_t elem_strides[2] = {1, 1};
  const CUtensorMapSwizzle swz = xt ? CU_TENSOR_MAP_SWIZZLE_128B
                               : n_pad == 16 ? CU_TENSOR_MAP_SWIZZLE_32B : n_pad == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
  const CUresult cr = encode(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(X), dims, strides, box, elem_strides,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) { set_cuda_error(static_cast<int>(cr)); return TL3_ERR_CUDA; }

  const long long total = m->n_tiles;
  const int grid = static_cast<int>(total < di.sm_count ? total : di.sm_count);
  if (static_cast<unsigned long long>(total) * static_cast<unsigned long long>(grid + 1) >= (1ull << 32)) return TL3_ERR_UNSUPPORTED;   // the kernel splits the tiles in 32-bit arithmetic
  const WorkspaceLayout wl = workspace_layout(m, n_pad, di.sm_count);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  KernelArgs args;
  args.blob = static_cast<const uint8_t*>(m->dptr);
  args.dir = reinterpret_cast<const DirEntry*>(args.blob + m->dir_offset);
  args.total_tiles = total;
  args.tiles_m = static_cast<int>(m->tiles_m);
  args.tiles_k = static_cast<int>(m->tiles_k);
  args.M = static_cast<int>(m->M);
  args.N = N;
  args.ldy = ldy;
  args.Y = static_cast<__half*>(Y);
  args.bias = ep ? static_cast<const __half*>(ep->bias) : nullptr;
  args.act = ep ? ep->activation : TL3_ACT_NONE;
  args.partials = reinterpret_cast<float*>(ws + wl.partials_off);
  args.flags = reinterpret_cast<unsigned int*>(ws + wl.flags_off);
  args.status = reinterpret_cast<unsigned int*>(ws + wl.status_off);
  args.stage_stride = stage_stride;
  args.x_offset = block_area;
  args.num_stages = stages;
  args.num_wr = num_wr;
  // Decoding ahead of X pays where a launch is short (a tile or a few per CTA: most of its time is
  // the start) and measured level or slightly worse on longer ones.
  const int dbx = g_decode_before_x.load(std::memory_order_relaxed);
  const long long tiles_per_cta = (total + grid - 1) / grid;
  args.opts = (dbx < 0 || tiles_per_cta <= dbx) ? kOptSplitX : 0u;
#ifdef TL3_CTA_STAMPS
  args.timing = g_timing_buffer ? g_timing_buffer + static_cast<long long>(g_timing_launch++ % 64) * 148 * 32 : nullptr;
#else
  args.timing = nullptr;
#endif
  m->last_ctas = grid; m->last_stages = stages; m->last_smem = static_cast<int>(smem_bytes);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (xt) {
    switch (n_pad) {
      case 16: return launch<16, true>(map, args, grid, smem_bytes, st);
      case 32: return launch<32, true>(map, args, grid, smem_bytes, st);
      default: return launch<64, true>(map, args, grid, smem_bytes, st);
    }
  }
  switch (n_pad) {
    case 16: return launch<16, false>(map, args, grid, smem_bytes, st);
    case 32: return launch<32, false>(map, args, grid, smem_bytes, st);
    default: return launch<64, false>(map, args, grid, smem_bytes, st);
  }
}

int tl3_spmm(const tl3_matrix* m, const void* X, int64_t ldx, void* Y, int64_t ldy, int N, void* workspace, void* stream) {
  return tl3_spmm_ex(m, X, ldx, Y, ldy, N, nullptr, workspace, stream);
}

int tl3_spmm_ex(const tl3_matrix* m, const void* X, int64_t ldx, void* Y, int64_t ldy, int N, const tl3_epilogue* ep,
                void* workspace, void* stream) {
  if (!m || !X || !Y || !workspace) return TL3_ERR_INVALID_ARG;
  if (ep && (ep->activation < TL3_ACT_NONE || ep->activation > TL3_ACT_GELU_TANH ||
             (reinterpret_cast<uintptr_t>(ep->bias) & 1) != 0))
    return TL3_ERR_INVALID_ARG;
  if (!m->dptr) return TL3_ERR_NOT_UPLOADED;
  if (N < 1 || N > TL3_MAX_N) return TL3_ERR_UNSUPPORTED;
  if (ldx < N || ldy < N) return TL3_ERR_INVALID_ARG;
  // Wider activation blocks are processed 64 columns at a time; every block streams W again, so
  // beyond N = 64 the time grows in proportion to N (this kernel targets the decode phase; the
  // paper, too, loses to the dense GEMM at large N, Sec. 6).
  for (int n0 = 0; n0 < N; n0 += 64) {
    const int nb = N - n0 < 64 ? N - n0 : 64;
    const int rc = spmm_block(m, static_cast<const uint16_t*>(X) + n0, ldx, static_cast<uint16_t*>(Y) + n0, ldy, nb, ep, false, workspace, stream);
    if (rc != TL3_OK) return rc;
  }
  return TL3_OK;
}

int tl3_spmm_nt(const tl3_matrix* m, const void* Xt, int64_t ldxt, void* Yt, int64_t ldyt, int N, const tl3_epilogue* ep,
                void* workspace, void* stream) {
  if (!m || !Xt || !Yt || !workspace) return TL3_ERR_INVALID_ARG;
  if (ep && (ep->activation < TL3_ACT_NONE || ep->activation > TL3_ACT_GELU_TANH ||
             (reinterpret_cast<uintptr_t>(ep->bias) & 1) != 0))
    return TL3_ERR_INVALID_ARG;
  if (!m->dptr) return TL3_ERR_NOT_UPLOADED;
  if (N < 1 || N > TL3_MAX_N) return TL3_ERR_UNSUPPORTED;
  if (ldxt < m->K || ldyt < m->M) return TL3_ERR_INVALID_ARG;
  for (int n0 = 0; n0 < N; n0 += 64) {                           // 64 rows of X^T (= columns of X) per launch
    const int nb = N - n0 < 64 ? N - n0 : 64;
    const int rc = spmm_block(m, static_cast<const uint16_t*>(Xt) + static_cast<int64_t>(n0) * ldxt, ldxt,
                              static_cast<uint16_t*>(Yt) + static_cast<int64_t>(n0) * ldyt, ldyt, nb, ep, true, workspace, stream);
    if (rc != TL3_OK) return rc;
  }
  return TL3_OK;
}

int tl3_spmm_host_async(const tl3_matrix* m, const uint16_t* X, uint16_t* Y, int N, void* dX, void* dY, void* workspace, void* stream) {
  if (!m || !X || !Y || !dX || !dY) return TL3_ERR_INVALID_ARG;
  if (N < 1 || N > TL3_MAX_N) return TL3_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // device copy of X with a leading dimension that satisfies the 16-byte rule
  const int64_t ldx = (N + 7) / 8 * 8;
  if (ldx == N) {
    TL3_CUDA(cudaMemcpyAsync(dX, X, static_cast<size_t>(m->K) * N * 2, cudaMemcpyHostToDevice, st));
  } else {
    TL3_CUDA(cudaMemcpy2DAsync(dX, static_cast<size_t>(ldx) * 2, X, static_cast<size_t>(N) * 2, static_cast<size_t>(N) * 2,
                               static_cast<size_t>(m->K), cudaMemcpyHostToDevice, st));
  }
  if (int rc = tl3_spmm(m, dX, ldx, dY, N, N, workspace, stream)) return rc;
  TL3_CUDA(cudaMemcpyAsync(Y, dY, static_cast<size_t>(m->M) * N * 2, cudaMemcpyDeviceToHost, st));
  return TL3_OK;
}

int tl3_spmm_host(const tl3_matrix* m, const uint16_t* X, uint16_t* Y, int N, void* dX, void* dY, void* workspace, void* stream) {
  if (int rc = tl3_spmm_host_async(m, X, Y, N, dX, dY, workspace, stream)) return rc;
  TL3_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  return TL3_OK;
}

// ---- entry point that allocates nothing: scratch inside the library image -------------------
// Split-K partials, their arrival flags and the status word for callers that cannot supply a
// workspace.  The name below is a host-side handle of the symbol, not a device address: host code
// must go through cudaGetSymbolAddress (done once per device, with that device current).
static __device__ __align__(256) unsigned char g_static_scratch[TL3_STATIC_SCRATCH_BYTES];

namespace tl3 {
static int static_scratch_address(void** out) {
  int dev = 0;
  TL3_CUDA(cudaGetDevice(&dev));
  static std::mutex mu;
  static std::vector<void*> per_device;
  std::lock_guard<std::mutex> lock(mu);
  if (static_cast<size_t>(dev) >= per_device.size()) per_device.resize(dev + 1, nullptr);
  if (!per_device[dev]) {
    void* p = nullptr;
    TL3_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
    per_device[dev] = p;
  }
  *out = per_device[dev];
  return TL3_OK;
}
}  // namespace tl3

int tl3_spmm_static_scratch(const tl3_matrix* m, const void* X, int64_t ldx, void* Y, int64_t ldy, int N, void* stream) {
  if (!m || !X || !Y) return TL3_ERR_INVALID_ARG;
  if (!m->dptr) return TL3_ERR_NOT_UPLOADED;
  if (N < 1 || N > TL3_MAX_N) return TL3_ERR_UNSUPPORTED;
  tl3::DeviceInfo di;
  if (int rc = tl3::device_info(&di)) return rc;
  const tl3::WorkspaceLayout wl = tl3::workspace_layout(m, tl3::n_pad_of(N), di.sm_count);
  if (wl.total > TL3_STATIC_SCRATCH_BYTES) return TL3_ERR_SCRATCH_LIMIT;
  void* scratch = nullptr;
  if (int rc = tl3::static_scratch_address(&scratch)) return rc;
  // flags and status word must start at zero; the partial-sum slots are always written before
  // they are read, so the last call's contents there do not matter
  TL3_CUDA(cudaMemsetAsync(scratch, 0, wl.partials_off, static_cast<cudaStream_t>(stream)));
  return tl3_spmm(m, X, ldx, Y, ldy, N, scratch, stream);
}

int tl3_static_scratch_status(void* stream) {
  void* scratch = nullptr;
  if (int rc = tl3::static_scratch_address(&scratch)) return rc;
  return tl3_status(nullptr, scratch, stream);
}

int tl3_status_word(void* workspace, void* stream, uint32_t* word) {
  if (!workspace || !word) return TL3_ERR_INVALID_ARG;
  unsigned int st = 0;
  TL3_CUDA(cudaMemcpyAsync(&st, workspace, sizeof(st), cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream)));
  TL3_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  *word = st;
  return TL3_OK;
}

int tl3_status(const tl3_matrix* m, void* workspace, void* stream) {
  (void)m;
  uint32_t st = 0;
  if (int rc = tl3_status_word(workspace, stream, &st)) return rc;
  if (st == 0) return TL3_OK;
  return (st & 0xFFu) >= tl3::kStBadBlock ? TL3_ERR_BAD_CONTAINER : TL3_ERR_DEVICE_TIMEOUT;
}

int tl3_last_launch(const tl3_matrix* m, int* ctas, int* stages, int* smem_bytes) {
  if (!m) return TL3_ERR_INVALID_ARG;
  if (ctas) *ctas = m->last_ctas;
  if (stages) *stages = m->last_stages;
  if (smem_bytes) *smem_bytes = m->last_smem;
  return TL3_OK;
}

int tl3_last_cuda_error(void) { return tl3::g_last_cuda_error; }

int tl3_get_tuning(tl3_tuning* out) {
  if (!out) return TL3_ERR_INVALID_ARG;
  out->decode_before_x = tl3::g_decode_before_x.load();
  return TL3_OK;
}

int tl3_set_tuning(const tl3_tuning* t) {
  if (!t) {
    tl3::g_decode_before_x = TL3_DEFAULT_DECODE_BEFORE_X;
    return TL3_OK;
  }
  if (t->decode_before_x < -1) return TL3_ERR_INVALID_ARG;
  tl3::g_decode_before_x = t->decode_before_x;
  return TL3_OK;
}

int tl3_selftest_bounded_wait(void* workspace, void* stream) {
  if (!workspace) return TL3_ERR_INVALID_ARG;
  unsigned int* words = static_cast<unsigned int*>(workspace);
  tl3::bounded_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(words, words + 1);
  TL3_CUDA(cudaGetLastError());
  return TL3_OK;
}

#ifdef TL3_CTA_STAMPS
void tl3_debug_set_timing_buffer(long long* device_ptr) { tl3::g_timing_buffer = device_ptr; tl3::g_timing_launch = 0; }   // 64 x 148 x 32 int64
#endif

}  // extern "C"
