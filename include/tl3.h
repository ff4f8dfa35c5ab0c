/*
 * tl3 -- C ABI of the three-layer sparse-weight SpMM library for NVIDIA B200 (sm_100a).
 *
 * The library stores an fp16 weight matrix W (M x K, ~50 % unstructured sparsity) in the paper's
 * three-layer format (Sec. 3.2: Sparse-TC layer, Slot-Filling layer with parallel-differential-
 * distance position codes, Residual layer) and computes Y = W X for a small-N fp16 activation
 * block X (Sec. 5.1: W is M x K, X is K x N, Y is M x N) with hand-written CUDA kernels that run
 * the Sparse-TC layer on the sparse tensor cores and decode the other two layers on chip
 * (Sec. 4).  The format is built once, ahead of time, on the host (Sec. 2.1).
 *
 * Conventions
 *   - Every function returns TL3_OK (0) or a negative TL3_ERR_* code; nothing throws, exits or
 *     synchronises the device unless stated.
 *   - "host" / "device" in a comment says where the pointer must point.
 *   - fp16 values cross the ABI as their 16-bit patterns (uint16_t).
 *   - The handle owns its host copies of the format.  The caller owns ALL device memory (the
 *     packed weight blob, X, Y, the workspace) and keeps it alive while work is queued.
 *   - There is no CPU fallback: tl3_spmm fails if no sm_100 device is current.
 */
#ifndef TL3_H_
#define TL3_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tl3_matrix tl3_matrix;          /* opaque */

/* Tile of the format: pairing of surplus weights with empty slots and the 16-bit start
 * positions of Algorithm 1 are local to one tile (Sec. 4.2 loads the matrix tile by tile).
 * NULL means {128, 128, 15}; the GPU kernels accept only that default. */
typedef struct {
  int32_t tile_m;   /* rows per tile, > 0                                             */
  int32_t tile_k;   /* columns per tile, multiple of 8, tile_m*tile_k/2 <= 65535      */
  int32_t maxd;     /* largest 4-bit differential distance, 1..15 (0 marks a dummy)   */
} tl3_params;

/* Non-zero counts by layer (Sec. 3.2 quotes their shares) and sizes in bytes. */
typedef struct {
  int64_t M, K, M_pad, K_pad, n_tiles;
  int64_t nnz, n_tc, n_sf, n_res, n_dummy, n_slots_unused;
  int64_t canonical_bytes;    /* sum of the nine canonical arrays                     */
  int64_t device_bytes;       /* size of the packed device blob                       */
  int64_t canonical_bytes_compact;  /* the same with the Residual layer in its compact form        */
  /* Layer counts of the device image, i.e. of what the kernel streams (0 for tiles other than
   * 128 x 128).  The device image pairs and cuts the PDD chains for the banks of shared memory and
   * sends what does not fit three code words per chain to its Residual list, so its Residual share
   * is larger than the canonical one. */
  int64_t dev_n_sf;           /* elements whose position is PDD-coded                               */
  int64_t dev_n_res;          /* elements that travel as Residual entries                           */
  int64_t dev_n_dummy;        /* delta bytes that move nothing: dummy points and chain padding      */
  int64_t dev_pdd_bytes;      /* delta bytes in all                                                 */
  int64_t canonical_bytes_compact_all;  /* canonical_bytes_compact with the value array in its compact form too */
} tl3_stats_t;

enum {
  TL3_OK = 0,
  TL3_ERR_INVALID_ARG = -1,
  TL3_ERR_UNSUPPORTED = -2,      /* N, tile shape or device not supported by the kernels       */
  TL3_ERR_NOT_UPLOADED = -3,
  TL3_ERR_BAD_CONTAINER = -4,    /* inconsistent container (deserialize / decode)               */
  TL3_ERR_CUDA = -5,             /* a CUDA runtime call failed; see tl3_last_cuda_error()       */
  TL3_ERR_DEVICE_TIMEOUT = -6,   /* a bounded wait inside the kernel gave up (status word)      */
  TL3_ERR_NO_MEMORY = -7,
  TL3_ERR_SCRATCH_LIMIT = -8     /* tl3_spmm_static_scratch: the problem needs more than the built-in scratch */
};

/* Canonical arrays, in the order tl3_canonical() numbers them. */
enum {
  TL3_TC_VALS = 0,     /* u16 [M_pad][K_pad/2]  two value slots per window of four weights      */
  TL3_TC_META = 1,     /* u8  [M_pad][K_pad/8]  nibble idx0|idx1<<2 per window, even window low  */
  TL3_CHAIN_TAU0 = 2,  /* u16 [tiles][tile_m]   first offset_t of each chain (Algorithm 1 l.3)   */
  TL3_CHAIN_RHO0 = 3,  /* u16 [tiles][tile_m]   first offset_r of each chain (Algorithm 1 l.4)   */
  TL3_CHAIN_LEN = 4,   /* u8  [tiles][tile_m]   number of delta bytes of each chain              */
  TL3_PDD_BYTES = 5,   /* u8  []                t delta low nibble, r delta high nibble          */
  TL3_TILE_DIR = 6,    /* u32 [tiles][4]        pdd_off, pdd_len, res_off, res_cnt               */
  TL3_RES_RHO = 7,     /* u16 []                Residual positions                               */
  TL3_RES_VAL = 8,     /* u16 []                Residual values                                  */
  /* Compact form of the Residual layer (Sec. 3.2 leaves its format open: "such as CSR"), derived
   * from TL3_RES_RHO: per tile whichever is smaller, the position list or a bitmap over the tile's
   * tile_m * tile_k / 2 positions of W_r; values stay in TL3_RES_VAL, in ascending position order. */
  TL3_RES_DIR = 9,     /* u32 [tiles][2]        {mode, off}: 0 = list, off indexes TL3_RES_LIST;        */
                       /*                       1 = bitmap, off = byte offset into TL3_RES_MASK         */
  TL3_RES_LIST = 10,   /* u16 []                positions of the list-mode tiles                         */
  TL3_RES_MASK = 11,   /* u8  []                ceil(tile_m*tile_k/16) bytes per bitmap-mode tile, bit   */
                       /*                       rho % 8 of byte rho / 8                                  */
  /* Compact form of the Sparse-TC value array, derived from TL3_TC_VALS.  The paper stores every
   * slot (Sec. 3.2) and names the slots that stay empty above 50 % sparsity as a limitation
   * (Sec. 6).  Per tile whichever is smaller: all tile_m * tile_k / 2 values, or a bitmap of the
   * occupied slots (value bits != 0; bit pos % 8 of byte pos / 8, pos = row * tile_k / 2 +
   * slot) plus the occupied slots' values in ascending position order. */
  TL3_VAL_DIR = 12,    /* u32 [tiles][2]        {mode, off}: off indexes TL3_VAL_PACK; 0 = all values,  */
                       /*                       1 = occupied slots only, bitmaps in tile order           */
  TL3_VAL_PACK = 13,   /* u16 []                values, tile after tile                                  */
  TL3_VAL_MASK = 14    /* u8  []                ceil(tile_m*tile_k/16) bytes per bitmap-mode tile        */
};

/* ---- format: host side (Sec. 3.2) ------------------------------------------------------ */

/* Encode a dense, already masked matrix (pruned weights are zeros; -0.0 counts as zero).
 * W: host, fp16 bits, row-major M x K, leading dimension K.  *out receives a new handle that the
 * caller releases with tl3_free().  Errors: INVALID_ARG (NULL, M or K <= 0, bad params). */
int tl3_encode(const uint16_t* W, int64_t M, int64_t K, const tl3_params* params, tl3_matrix** out);

/* The same conversion on the GPU (the paper converts on the CPU and quotes 41-93 s per model,
 * Sec. 5.3): window classification, ordered lists of surplus weights and empty slots by prefix
 * scans, pairing and chain emission run as CUDA kernels, one CTA per 128 x 128 tile; the result is
 * the same canonical container, byte for byte, in a new handle with host copies of the arrays
 * (tl3_decode, tl3_upload, tl3_serialize ... work on it as on any other).
 *   dW: device, fp16 bits, row-major M x K, leading dimension ldw >= K, already masked.
 *   Tile 128 x 128, maxd 15 only.  The call allocates and frees device scratch of about the size
 *   of the container (cudaMalloc), runs on `stream` and waits for it.
 * Errors: INVALID_ARG, UNSUPPORTED (more than 4 GiB of PDD bytes), CUDA, NO_MEMORY. */
int tl3_encode_device(const void* dW, int64_t M, int64_t K, int64_t ldw, void* stream, tl3_matrix** out);
/* The same conversion for a matrix that is only going to be multiplied: the container stays on the
 * device, no host copy of it is made, and the handle comes back planned (tl3_device_bytes() is
 * valid).  tl3_upload_device() then packs it into the caller's blob and releases the device copy
 * of the container; tl3_spmm*, tl3_bind, tl3_stats (layer counts; the sizes of the compact forms
 * read -1), tl3_workspace_bytes and tl3_free work as on any handle.  The calls that need the
 * container on the host -- tl3_decode, tl3_canonical, tl3_serialize*, tl3_pack, tl3_upload --
 * return UNSUPPORTED.  dW, ldw, stream, errors: as for tl3_encode_device. */
int tl3_encode_device_only(const void* dW, int64_t M, int64_t K, int64_t ldw, void* stream, tl3_matrix** out);

/* Decode back to dense: Algorithm 1 run on the host, then the 2:4 expansion and the Residual
 * entries.  W_out: host, M*K uint16_t, caller-owned, fully overwritten.  The result equals the
 * encoder's input bit for bit (with -0.0 read as +0.0).  Errors: BAD_CONTAINER. */
int tl3_decode(const tl3_matrix* m, uint16_t* W_out);

/* Borrow one canonical array (TL3_TC_VALS ...).  *ptr stays valid until tl3_free(). */
int tl3_canonical(const tl3_matrix* m, int which, const void** ptr, size_t* bytes);

int tl3_stats(const tl3_matrix* m, tl3_stats_t* out);

/* Bit-exact persistence of the canonical container ("stored ahead of time", Sec. 2.1).
 * tl3_serialize: buf == NULL writes the needed size to *bytes; otherwise *bytes is the capacity
 * on entry and the size written on return.  buf: host. */
int tl3_serialize(const tl3_matrix* m, void* buf, size_t* bytes);
/* The same container with the Residual positions and the value array in their compact forms
 * (TL3_RES_DIR ... TL3_VAL_MASK): what to write to disk or send below 50 % and above 50 %
 * sparsity (0.81 -> 0.75 x dense at 40 %, 0.61 -> 0.54 at 60 %, 0.59 -> 0.43 at 70 %; the same
 * size as tl3_serialize plus two small directories at 50 %).  Same calling convention. */
int tl3_serialize_compact(const tl3_matrix* m, void* buf, size_t* bytes);
/* Reads either form (the header says which) into a new handle whose nine canonical arrays are
 * those of the container that was written, bit for bit.  Errors: INVALID_ARG, BAD_CONTAINER
 * (truncated, inconsistent or out-of-range contents; nothing is trusted), NO_MEMORY. */
int tl3_deserialize(const void* buf, size_t bytes, tl3_matrix** out);

void tl3_free(tl3_matrix* m);

/* ---- device side (Sec. 4) -------------------------------------------------------------- */

/* Size of the packed device blob (tile blocks ready for bulk copies); 0 for a container whose
 * tiles are not 128 x 128 (the device path exists for that tile only). */
size_t tl3_device_bytes(const tl3_matrix* m);

/* Pack the container into a HOST buffer of tl3_device_bytes() bytes: exactly the bytes tl3_upload()
 * sends to the device: per tile one contiguous block holding the value slots in the shared-memory
 * image the MMA reads, the metadata in tensor-memory word order, the chain starts, lengths and delta
 * bytes, and the Residual entries.  Values, metadata and the sets of parked and Residual elements
 * are those of the canonical container; which empty slot a parked element sits in and how the
 * PDD chains are cut follow the banks of shared memory (Sec. 3.2 leaves both open), so the PDD
 * bytes differ from the canonical ones.  For callers that stage the blob themselves.
 * Errors: UNSUPPORTED, INVALID_ARG. */
int tl3_pack(const tl3_matrix* m, void* host_buf, size_t bytes);

/* Pack the container and copy it to dptr (device, >= tl3_device_bytes(), 256-byte aligned) on
 * `stream` (a cudaStream_t passed as void*; NULL = default stream), then bind dptr to the handle.
 * The copy is asynchronous with respect to the device; host staging is released before return.
 * Errors: UNSUPPORTED (tile shape other than 128 x 128), INVALID_ARG, CUDA. */
int tl3_upload(tl3_matrix* m, void* dptr, void* stream);

/* The device packer on the GPU.  tl3_plan_device() computes the layout of the device image with a
 * CUDA kernel (afterwards tl3_device_bytes() returns at once instead of running the host packer's
 * first pass), tl3_upload_device() writes the blob into dptr with a second pass of the same
 * kernel: the same bytes as tl3_pack() / tl3_upload().  Both copy the canonical arrays to the
 * device first (one cudaMalloc of the container's size, shared between the two calls, released
 * by tl3_upload_device or tl3_free), run on `stream` and wait for it.
 *   dptr: device, >= tl3_device_bytes(), 256-byte aligned; bound to the handle on success.
 * Errors: INVALID_ARG, UNSUPPORTED (tile shape other than 128 x 128), CUDA, NO_MEMORY. */
int tl3_plan_device(tl3_matrix* m, void* stream);
int tl3_upload_device(tl3_matrix* m, void* dptr, void* stream);

/* Bind a device buffer that already holds the packed blob -- the bytes of tl3_pack() copied to the
 * device by the caller, or a device-side copy of a blob that tl3_upload() wrote -- to the handle:
 * later tl3_spmm* calls read the weights from there.  dptr: device, >= tl3_device_bytes(),
 * 256-byte aligned.  Nothing is copied or checked.  A launch reads the binding when it is enqueued
 * (or captured into a CUDA graph), so one handle may serve several device copies in turn.
 * Errors: INVALID_ARG, UNSUPPORTED (tile shape other than 128 x 128). */
int tl3_bind(tl3_matrix* m, void* dptr);

/* Scratch the kernel needs for N columns: split-K partial sums, one arrival flag per partial-sum
 * slot, a status word.  Depends on the current device's SM count.  The caller allocates it (device,
 * 256-byte aligned), clears it once with tl3_workspace_init(), and may then reuse it for any number
 * of calls that do not overlap on the GPU (the kernel leaves it cleared; after a call that ended
 * with a non-zero status, clear it again). */
size_t tl3_workspace_bytes(const tl3_matrix* m, int N);
int tl3_workspace_init(void* workspace, size_t bytes, void* stream);

/* Y = W X  (Sec. 5.1 problem statement; kernel design after Sec. 4: tile-wise streaming of the
 * compressed weights, on-chip PDD decoding per Algorithm 1, sparse tensor-core MMA, Residual
 * folded into the same accumulators, one final reduction).
 *   X: device, fp16, K x N row-major, leading dimension ldx >= N, ldx % 8 == 0, 16-byte aligned.
 *   Y: device, fp16, M x N row-major, leading dimension ldy >= N; fully overwritten.
 *   1 <= N <= TL3_MAX_N.  Up to 64 columns are one kernel launch (the decode-phase case the
 *   kernels are built for); wider blocks are processed 64 columns at a time, each streaming W
 *   again.  fp32 accumulation, fp16 round-to-nearest-even output.  W and X are assumed finite (an
 *   empty slot multiplies an exact zero with an element of X).
 * Asynchronous on `stream`; allocates nothing; does not synchronise.  Calls that share a
 * workspace must not overlap on the GPU; the workspace must hold tl3_workspace_bytes(m, N) bytes
 * for THIS N (it grows with N: 16, 32 or 64 columns of partial sums per slot), the call cannot
 * check that.  Calls on different streams, each with its own workspace, may be in flight together.
 * A row-tile shared by several CTAs is finished by the CTA that owns its first tile, which waits
 * (bounded, status code 11) for CTAs with a higher index; that those get to run while other
 * kernels hold SMs rests on the GPU dispatching the blocks of a grid in index order.
 * Threads: calls that take a const handle may share it; tl3_upload() and tl3_free() may not run
 * beside another call on the same handle.
 * Errors: NOT_UPLOADED, INVALID_ARG, UNSUPPORTED (N out of range, device is not sm_100, or a matrix of
 * 2^32 / (SMs + 1) tiles or more -- 28.8 million on B200, hundreds of gigabytes), CUDA. */
#define TL3_MAX_N 4096
int tl3_spmm(const tl3_matrix* m, const void* X, int64_t ldx, void* Y, int64_t ldy, int N,
             void* workspace, void* stream);

/* (No counterpart in the paper: the usual fused epilogue of a linear layer.)  Y = act(W X + b):
 * tl3_spmm with a per-row bias and an activation applied to the fp32 sums before they are rounded
 * to fp16.
 *   ep->bias: device, fp16[M], or NULL for none.  ep->activation: TL3_ACT_NONE, TL3_ACT_RELU,
 *   TL3_ACT_SILU (x / (1 + exp(-x))), TL3_ACT_GELU_TANH (0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))).
 *   ep == NULL is tl3_spmm.  Everything else as for tl3_spmm; INVALID_ARG for an unknown activation. */
enum { TL3_ACT_NONE = 0, TL3_ACT_RELU = 1, TL3_ACT_SILU = 2, TL3_ACT_GELU_TANH = 3 };
typedef struct {
  const void* bias;
  int activation;
} tl3_epilogue;
int tl3_spmm_ex(const tl3_matrix* m, const void* X, int64_t ldx, void* Y, int64_t ldy, int N,
                const tl3_epilogue* ep, void* workspace, void* stream);

/* The same product with both activations transposed, the [batch, hidden] layout of an inference
 * stack (Sec. 2.1): Yt = Xt W^T, i.e. Yt[n][m] = sum_k W[m][k] Xt[n][k] (+ bias[m], activation).
 *   Xt: device, fp16, N x K row-major, leading dimension ldxt >= K, ldxt % 8 == 0, 16-byte aligned.
 *   Yt: device, fp16, N x M row-major, leading dimension ldyt >= M; rows 0..N-1 fully overwritten.
 *   ep: as for tl3_spmm_ex, or NULL.  Everything else as for tl3_spmm. */
int tl3_spmm_nt(const tl3_matrix* m, const void* Xt, int64_t ldxt, void* Yt, int64_t ldyt, int N,
                const tl3_epilogue* ep, void* workspace, void* stream);

/* Same product with HOST buffers: copies X to dX, runs tl3_spmm, copies dY to Y and waits for the
 * stream.  X, Y: host (pinned memory makes the copies asynchronous), dense leading dimensions
 * ldx = ldy = N.  dX (>= K*N*2 bytes) and dY (>= M*N*2 bytes): device scratch owned by the caller. */
int tl3_spmm_host(const tl3_matrix* m, const uint16_t* X, uint16_t* Y, int N, void* dX, void* dY,
                  void* workspace, void* stream);

/* The same without the wait: the three steps are only enqueued on `stream`.  X must stay valid and
 * Y is defined once the stream has passed this point (cudaStreamSynchronize, an event).  Calls on
 * different streams may be in flight together as long as each has its own dX, dY and workspace:
 * the copies of one then overlap the kernel of another. */
int tl3_spmm_host_async(const tl3_matrix* m, const uint16_t* X, uint16_t* Y, int N, void* dX, void* dY,
                        void* workspace, void* stream);

/* (No counterpart in the paper.)  Y = W X exactly as tl3_spmm computes it, for callers that are
 * not allowed to obtain device memory themselves and so cannot provide a workspace: a driver-level
 * plug-in whose host application hands it only the input and output buffers and forbids allocation
 * calls inside its execute hook, or a process running under a fixed device-memory budget that was
 * spent before this library was loaded.  The split-K partial sums, the arrival flags and the
 * status word live in a fixed array that is part of the library image: TL3_STATIC_SCRATCH_BYTES
 * (3 MiB) of device memory on every GPU that loads the library, held until the process exits.
 *   - Problems whose scratch need (what tl3_workspace_bytes() reports; it depends on the SM count
 *     and on N, not on the matrix) exceeds that size are refused with TL3_ERR_SCRATCH_LIMIT and
 *     nothing is launched.  On a 148-SM device this admits N <= 16; N > 16 is refused there.
 *   - X, Y, ldx, ldy, N, stream: as for tl3_spmm.  The caller still owns X and Y.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current); make that first call outside any stream capture.  Later calls only enqueue work.
 *   - No call obtains device memory: no cudaMalloc / cudaFree, no allocating library routine.
 *     The first call per device does one-time host-side set-up (the address look-up, the kernel's
 *     shared-memory opt-in, the driver's lazy loading of the kernel image).
 *   - All calls on a device share the one array.  Each call clears the flags and the status word
 *     on `stream` before the kernel, so a call that was cut short does not poison the next one, but
 *     two calls that overlap on the GPU (different streams, no dependency) race on it: serialise
 *     them.  tl3_static_scratch_status() reads the status word of the current device. */
#define TL3_STATIC_SCRATCH_BYTES (3u << 20)
int tl3_spmm_static_scratch(const tl3_matrix* m, const void* X, int64_t ldx, void* Y, int64_t ldy, int N,
                            void* stream);
int tl3_static_scratch_status(void* stream);

/* Read the workspace's status word (synchronises `stream`).  TL3_OK; DEVICE_TIMEOUT if a bounded
 * wait inside a kernel expired since the last tl3_workspace_init(); BAD_CONTAINER if the decoder
 * met a block whose lengths or decoded positions were out of range (it skips such entries rather
 * than touching memory outside the tile).  tl3_status_word() also hands back the raw word:
 * bits 0-7 = code (1-11: which wait gave up, 16: bad block), higher bits = detail. */
int tl3_status(const tl3_matrix* m, void* workspace, void* stream);
int tl3_status_word(void* workspace, void* stream, uint32_t* word);

/* Self-test of the kernels' bounded waits (every wait inside the kernels gives up after 2 s,
 * records a code in the status word and lets the kernel return).  Enqueues a one-CTA kernel that
 * waits on a barrier nothing ever arrives at; about 2 s after it starts, tl3_status() on the
 * same workspace reports DEVICE_TIMEOUT (code 1), the second word of the workspace holds 2
 * ("gave up"; 1 would mean the wait completed), and the device is usable as before.  Clear the
 * workspace with tl3_workspace_init() before using it for a product again. */
int tl3_selftest_bounded_wait(void* workspace, void* stream);

/* (No counterpart in the paper.)  Launch tuning, process-wide, read by every later tl3_spmm* call.
 *   decode_before_x  launches with at most this many tiles per CTA decode a block as soon as it is
 *                    in shared memory instead of waiting for its X tile as well (X may come from the
 *                    kernel before, which the launch overlaps; the weights never do).  Measured on
 *                    B200: 9 % faster at one tile per CTA (1024 x 1024), level or up to 1 % slower
 *                    from seven tiles per CTA on.  0 = never, -1 = always.
 * tl3_set_tuning(NULL) restores the default.  Errors: INVALID_ARG. */
#define TL3_DEFAULT_DECODE_BEFORE_X 4
typedef struct {
  int32_t decode_before_x;
} tl3_tuning;
int tl3_get_tuning(tl3_tuning* out);
int tl3_set_tuning(const tl3_tuning* t);

/* Kernel launch geometry of the last tl3_spmm on this handle (for reporting): CTAs, stages. */
int tl3_last_launch(const tl3_matrix* m, int* ctas, int* stages, int* smem_bytes);

const char* tl3_strerror(int code);
int tl3_last_cuda_error(void);      /* cudaError_t of the last failed runtime call, this thread */

#ifdef __cplusplus
}
#endif
#endif /* TL3_H_ */
