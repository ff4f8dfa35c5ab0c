/*
 * TEST INFRASTRUCTURE ONLY -- the CPU oracle of the three-layer sparse format and its SpMM.
 *
 * Plain, slow, single-purpose C.  Nothing in the product path may call, link or import this
 * file; it shares no code, header, table or helper with the CUDA library.  Only the tests, the
 * smoke check and the CPU-baseline leg of the benchmark use it.
 *
 * What it implements (paper sections in brackets):
 *   oracle_encode      dense masked fp16 W  ->  Sparse-TC / Slot-Filling (PDD) / Residual layers
 *                      [Sec. 3.2 "Multi-layer Storage Format"], one tile at a time [Sec. 4.2:
 *                      the matrix is partitioned into tiles]
 *   oracle_decode      the inverse: Algorithm 1 (PDD decoding) run on the CPU, then the 2:4
 *                      expansion of the Sparse-TC layer and the Residual entries
 *   oracle_spmm        Y = W X walked layer by layer over the container [Sec. 4.1 workflow,
 *                      Sec. 5.1 problem statement: W is M x K, X is K x N, Y is M x N],
 *                      fp32 accumulation, fp16 round-to-nearest-even output
 *
 * Where the paper is silent the container below fixes a reading (listed in the design notes of
 * the repository).  Container, for tile size TM x TK (TK % 8 == 0, TM*TK/2 <= 65535), H = TK/2:
 *   tc_vals  u16[M_pad][K_pad/2]   two value slots per window of four consecutive weights
 *   tc_meta  u8 [M_pad][K_pad/8]   one nibble per window: idx0 | idx1<<2 (2 bits per value,
 *                                  Sec. 3.2 Sparse-TC layer), even window in the low nibble
 *   chain_tau0, chain_rho0 u16[tiles][TM]   16-bit first positions of Algorithm 1 (its initial offsets)
 *   chain_len u8[tiles][TM]        number of delta bytes of the chain (replaces BitLen(code))
 *   pdd_bytes u8[]                 delta bytes, low nibble = offset_t delta, high nibble =
 *                                  offset_r delta (Algorithm 1, the two 4-bit advances); a zero nibble marks a
 *                                  dummy point (Sec. 3.2: spans above the 4-bit range are broken up)
 *   tile_dir u32[tiles][4]         {pdd_off, pdd_len, res_off, res_cnt}
 *   res_rho u16[], res_val u16[]   Residual layer: (position, value) per tile [Sec. 3.2]
 * Coordinates inside a tile (local row r, local window q):
 *   tau = r*H + 2q + s   index of value slot s of window q  (offset_t of Algorithm 1, into W_t)
 *   rho = r*H + 2q + (i-2) for a surplus weight at in-window index i in {2,3}
 *                        (offset_r of Algorithm 1, into W_r); its column is 4q + i.
 *
 * Pins: tests/test_oracle_*.py (worked examples under tests/golden, brute force, closed forms,
 * round trips, dense fp64 products).  The dummy range MAXD and the split of the code into one
 * chain per tile row are readings the paper does not fix: parity unpinned for those two choices.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
  int64_t M, K, M_pad, K_pad;
  int32_t tile_m, tile_k, maxd;
  int64_t n_tiles;
  uint16_t* tc_vals;   int64_t tc_vals_n;
  uint8_t* tc_meta;    int64_t tc_meta_n;
  uint16_t* chain_tau0; uint16_t* chain_rho0; uint8_t* chain_len; int64_t chain_n;
  uint8_t* pdd_bytes;  int64_t pdd_n, pdd_cap;
  uint32_t* tile_dir;
  uint16_t* res_rho; uint16_t* res_val; int64_t res_n, res_cap;
  /* statistics (counts of non-zeros by layer, Sec. 3.2 quotes their shares) */
  int64_t nnz, n_tc, n_sf, n_res, n_dummy, n_slots_unused;
} oracle_container;

static int is_nonzero(uint16_t bits) { return (bits & 0x7FFF) != 0; }

/* ---------------------------------------------------------------- fp16 <-> fp32 --------- */
static float half_to_float(uint16_t h) {
  uint32_t sign = (uint32_t)(h >> 15) << 31;
  uint32_t exp = (h >> 10) & 0x1F;
  uint32_t man = h & 0x3FF;
  uint32_t bits;
  if (exp == 0) {
    if (man == 0) {
      bits = sign;
    } else { /* subnormal: value = man * 2^-24 */
      int e = -1;
      do { man <<= 1; ++e; } while ((man & 0x400) == 0);
      bits = sign | (uint32_t)(127 - 15 - e) << 23 | (man & 0x3FF) << 13;
    }
  } else if (exp == 31) {
    bits = sign | 0x7F800000u | man << 13;
  } else {
    bits = sign | (exp + 112) << 23 | man << 13;
  }
  float f;
  memcpy(&f, &bits, 4);
  return f;
}

static uint16_t float_to_half_rne(float f) {
  uint32_t x;
  memcpy(&x, &f, 4);
  uint16_t sign = (uint16_t)((x >> 16) & 0x8000);
  uint32_t abs = x & 0x7FFFFFFFu;
  if (abs >= 0x7F800000u) { /* Inf or NaN */
    return (uint16_t)(sign | 0x7C00 | (abs > 0x7F800000u ? 0x200 | ((abs >> 13) & 0x3FF) : 0));
  }
  if (abs >= 0x477FF000u) { /* rounds to >= 65520 -> Inf */
    return (uint16_t)(sign | 0x7C00);
  }
  if (abs < 0x33000001u) { /* <= 2^-25: rounds to zero (2^-25 itself ties to even = 0) */
    return sign;
  }
  int32_t e = (int32_t)(abs >> 23) - 127;
  uint32_t man = (abs & 0x7FFFFF) | 0x800000; /* 24-bit significand */
  int shift;                                   /* bits dropped from the 24-bit significand */
  uint32_t half_exp;
  if (e < -14) { shift = 13 + (-14 - e); half_exp = 0; } else { shift = 13; half_exp = (uint32_t)(e + 15); }
  uint32_t kept = man >> shift;
  uint32_t rem = man & ((1u << shift) - 1);
  uint32_t halfway = 1u << (shift - 1);
  if (rem > halfway || (rem == halfway && (kept & 1))) ++kept;
  uint32_t out;
  if (half_exp == 0) out = kept;                      /* subnormal; a carry into bit 10 makes it normal */
  else out = ((half_exp - 1) << 10) + kept;           /* kept carries the implicit bit (0x400) */
  return (uint16_t)(sign | out);
}

/* exported so the tests can pin the conversions against numpy's */
float oracle_half_to_float(uint16_t h) { return half_to_float(h); }
uint16_t oracle_float_to_half(float f) { return float_to_half_rne(f); }

/* ---------------------------------------------------------------- container memory ------ */
void oracle_free(oracle_container* c) {
  if (!c) return;
  free(c->tc_vals); free(c->tc_meta); free(c->chain_tau0); free(c->chain_rho0); free(c->chain_len);
  free(c->pdd_bytes); free(c->tile_dir); free(c->res_rho); free(c->res_val);
  free(c);
}

static void push_pdd(oracle_container* c, uint8_t b) {
  if (c->pdd_n == c->pdd_cap) {
    c->pdd_cap = c->pdd_cap ? c->pdd_cap * 2 : 1024;
    c->pdd_bytes = (uint8_t*)realloc(c->pdd_bytes, (size_t)c->pdd_cap);
  }
  c->pdd_bytes[c->pdd_n++] = b;
}

static void push_res(oracle_container* c, uint16_t rho, uint16_t val) {
  if (c->res_n == c->res_cap) {
    c->res_cap = c->res_cap ? c->res_cap * 2 : 1024;
    c->res_rho = (uint16_t*)realloc(c->res_rho, (size_t)c->res_cap * 2);
    c->res_val = (uint16_t*)realloc(c->res_val, (size_t)c->res_cap * 2);
  }
  c->res_rho[c->res_n] = rho;
  c->res_val[c->res_n] = val;
  ++c->res_n;
}

typedef struct { uint16_t rho; uint16_t val; } surplus_t;

static int cmp_surplus(const void* a, const void* b) {
  return (int)((const surplus_t*)a)->rho - (int)((const surplus_t*)b)->rho;
}

/* ---------------------------------------------------------------- encode ---------------- */
/* W: fp16 bit patterns, row-major M x K, already masked (pruned weights are exact zeros). */
int oracle_encode(const uint16_t* W, int64_t M, int64_t K, int tile_m, int tile_k, int maxd,
                  oracle_container** out) {
  if (!W || !out || M <= 0 || K <= 0 || tile_m <= 0 || tile_k <= 0 || tile_k % 8 != 0) return -1;
  if ((int64_t)tile_m * tile_k / 2 > 65535 || maxd < 1 || maxd > 15) return -1;
  oracle_container* c = (oracle_container*)calloc(1, sizeof(*c));
  const int H = tile_k / 2, QW = tile_k / 4;
  c->M = M; c->K = K; c->tile_m = tile_m; c->tile_k = tile_k; c->maxd = maxd;
  c->M_pad = (M + tile_m - 1) / tile_m * tile_m;
  c->K_pad = (K + tile_k - 1) / tile_k * tile_k;
  const int64_t tiles_m = c->M_pad / tile_m, tiles_k = c->K_pad / tile_k;
  c->n_tiles = tiles_m * tiles_k;
  c->tc_vals_n = c->M_pad * c->K_pad / 2;
  c->tc_meta_n = c->M_pad * c->K_pad / 8;
  c->chain_n = c->n_tiles * tile_m;
  c->tc_vals = (uint16_t*)calloc((size_t)c->tc_vals_n, 2);
  c->tc_meta = (uint8_t*)calloc((size_t)c->tc_meta_n, 1);
  c->chain_tau0 = (uint16_t*)malloc((size_t)c->chain_n * 2);
  c->chain_rho0 = (uint16_t*)malloc((size_t)c->chain_n * 2);
  c->chain_len = (uint8_t*)calloc((size_t)c->chain_n, 1);
  c->tile_dir = (uint32_t*)calloc((size_t)c->n_tiles * 4, 4);

  const int64_t slots = (int64_t)tile_m * H;
  surplus_t* S = (surplus_t*)malloc((size_t)slots * sizeof(surplus_t));   /* surplus, sorted by rho */
  uint16_t* E = (uint16_t*)malloc((size_t)slots * 2);                     /* empty slots, sorted by tau */
  surplus_t* R = (surplus_t*)malloc((size_t)slots * sizeof(surplus_t));   /* residual of this tile */

  for (int64_t tm = 0; tm < tiles_m; ++tm) {
    for (int64_t tk = 0; tk < tiles_k; ++tk) {
      const int64_t tile = tm * tiles_k + tk;
      int64_t nS = 0, nE = 0, nR = 0;

      /* Step 1: Sparse-TC split of every window of four consecutive weights. */
      for (int r = 0; r < tile_m; ++r) {
        const int64_t row = tm * tile_m + r;
        for (int q = 0; q < QW; ++q) {
          uint16_t w[4];
          for (int i = 0; i < 4; ++i) {
            const int64_t col = tk * tile_k + 4 * q + i;
            w[i] = (row < M && col < K) ? W[row * K + col] : 0;
          }
          int nz[4], c_nz = 0;
          for (int i = 0; i < 4; ++i) if (is_nonzero(w[i])) nz[c_nz++] = i;
          c->nnz += c_nz;
          /* the first two non-zeros stay; the 3rd and 4th are surplus */
          int idx[2], is_kept[2];
          if (c_nz >= 2)      { idx[0] = nz[0]; idx[1] = nz[1]; is_kept[0] = 1; is_kept[1] = 1; }
          else if (c_nz == 1) {
            if (nz[0] == 0)   { idx[0] = 0; idx[1] = 1;     is_kept[0] = 1; is_kept[1] = 0; }
            else              { idx[0] = 0; idx[1] = nz[0]; is_kept[0] = 0; is_kept[1] = 1; }
          } else              { idx[0] = 0; idx[1] = 1;     is_kept[0] = 0; is_kept[1] = 0; }
          const int64_t gq = tk * QW + q;                    /* window index in the padded row */
          for (int s = 0; s < 2; ++s) {
            if (is_kept[s]) {
              c->tc_vals[row * (c->K_pad / 2) + 2 * gq + s] = w[idx[s]];
              ++c->n_tc;
            } else {
              E[nE++] = (uint16_t)(r * H + 2 * q + s);
            }
          }
          const uint8_t nib = (uint8_t)(idx[0] | idx[1] << 2);
          c->tc_meta[row * (c->K_pad / 8) + gq / 2] |= (uint8_t)(gq % 2 ? nib << 4 : nib);
          for (int j = 2; j < c_nz; ++j) {
            S[nS].rho = (uint16_t)(r * H + 2 * q + (nz[j] - 2));
            S[nS].val = w[nz[j]];
            ++nS;
          }
        }
      }

      /* Step 3: the i-th surplus weight goes to the i-th empty slot. */
      const int64_t P = nS < nE ? nS : nE;
      for (int64_t i = P; i < nS; ++i) R[nR++] = S[i];
      c->n_slots_unused += nE - P;

      /* Step 4: one PDD chain per tile row (the row of rho). */
      c->tile_dir[tile * 4 + 0] = (uint32_t)c->pdd_n;
      int64_t i = 0;
      for (int r = 0; r < tile_m; ++r) {
        const int64_t ch = tile * tile_m + r;
        c->chain_tau0[ch] = 0xFFFF; c->chain_rho0[ch] = 0xFFFF; c->chain_len[ch] = 0;
        if (i >= P || S[i].rho / H != r) continue;
        /* first pair: absolute 16-bit positions */
        int tau = E[i], rho = S[i].rho;
        c->chain_tau0[ch] = (uint16_t)tau; c->chain_rho0[ch] = (uint16_t)rho;
        c->tc_vals[(tm * tile_m + tau / H) * (c->K_pad / 2) + tk * H + tau % H] = S[i].val;
        ++c->n_sf;
        ++i;
        int len = 0, cut = 0;
        while (i < P && S[i].rho / H == r) {
          if (!cut) {
            int gt = E[i] - tau, gr = S[i].rho - rho;
            int need = 1 + (gt - 1) / maxd + (gr - 1) / maxd;   /* dummies for both spans + the real byte */
            if (len + need > 255) cut = 1;
            else {
              while (gt > maxd) { push_pdd(c, (uint8_t)maxd); gt -= maxd; ++c->n_dummy; }
              while (gr > maxd) { push_pdd(c, (uint8_t)(maxd << 4)); gr -= maxd; ++c->n_dummy; }
              push_pdd(c, (uint8_t)(gt | gr << 4));
              len += need;
              tau = E[i]; rho = S[i].rho;
              c->tc_vals[(tm * tile_m + tau / H) * (c->K_pad / 2) + tk * H + tau % H] = S[i].val;
              ++c->n_sf;
            }
          }
          if (cut) { R[nR++] = S[i]; ++c->n_slots_unused; }   /* chain full: rest of the row -> Residual */
          ++i;
        }
        c->chain_len[ch] = (uint8_t)len;
      }
      c->tile_dir[tile * 4 + 1] = (uint32_t)(c->pdd_n - c->tile_dir[tile * 4 + 0]);

      /* Step 5: Residual layer of the tile, sorted by rho. */
      qsort(R, (size_t)nR, sizeof(surplus_t), cmp_surplus);
      c->tile_dir[tile * 4 + 2] = (uint32_t)c->res_n;
      c->tile_dir[tile * 4 + 3] = (uint32_t)nR;
      for (int64_t j = 0; j < nR; ++j) push_res(c, R[j].rho, R[j].val);
      c->n_res += nR;
    }
  }
  free(S); free(E); free(R);
  *out = c;
  return 0;
}

/* field access for the Python side: which = 0..8 in the order of the header comment */
int oracle_get(const oracle_container* c, int which, const void** ptr, int64_t* bytes) {
  if (!c || !ptr || !bytes) return -1;
  switch (which) {
    case 0: *ptr = c->tc_vals;    *bytes = c->tc_vals_n * 2; break;
    case 1: *ptr = c->tc_meta;    *bytes = c->tc_meta_n; break;
    case 2: *ptr = c->chain_tau0; *bytes = c->chain_n * 2; break;
    case 3: *ptr = c->chain_rho0; *bytes = c->chain_n * 2; break;
    case 4: *ptr = c->chain_len;  *bytes = c->chain_n; break;
    case 5: *ptr = c->pdd_bytes;  *bytes = c->pdd_n; break;
    case 6: *ptr = c->tile_dir;   *bytes = c->n_tiles * 16; break;
    case 7: *ptr = c->res_rho;    *bytes = c->res_n * 2; break;
    case 8: *ptr = c->res_val;    *bytes = c->res_n * 2; break;
    default: return -1;
  }
  return 0;
}

/* stats[0..5] = nnz, n_tc, n_sf, n_res, n_dummy, n_slots_unused */
void oracle_stats(const oracle_container* c, int64_t* stats) {
  stats[0] = c->nnz; stats[1] = c->n_tc; stats[2] = c->n_sf; stats[3] = c->n_res;
  stats[4] = c->n_dummy; stats[5] = c->n_slots_unused;
}

/* ---------------------------------------------------------------- walking a container --- */
/*
 * Both the decoder and the SpMM visit every stored non-zero exactly once, in the order
 *   Slot-Filling (Algorithm 1: chain by chain, moving W_t[offset_t] to position offset_r and
 *   zeroing W_t[offset_t]), Residual, then what remains of the Sparse-TC layer,
 * and hand (row, column, value bits) to a visitor.
 */
typedef void (*visit_fn)(void* ctx, int64_t row, int64_t col, uint16_t val);

static int walk_tile(int64_t M_pad, int64_t K_pad, int tile_m, int tile_k,
                     const uint16_t* tc_vals, const uint8_t* tc_meta,
                     const uint16_t* chain_tau0, const uint16_t* chain_rho0, const uint8_t* chain_len,
                     const uint8_t* pdd_bytes, const uint32_t* tile_dir,
                     const uint16_t* res_rho, const uint16_t* res_val,
                     int64_t tm, int64_t tk, uint16_t* V /* tile_m*H scratch */, visit_fn visit, void* ctx) {
  const int H = tile_k / 2, QW = tile_k / 4;
  const int64_t tiles_k = K_pad / tile_k;
  const int64_t tile = tm * tiles_k + tk;
  const int64_t slots = (int64_t)tile_m * H;
  (void)M_pad;
  /* W_t of this tile */
  for (int r = 0; r < tile_m; ++r)
    memcpy(V + (int64_t)r * H, tc_vals + (tm * tile_m + r) * (K_pad / 2) + tk * H, (size_t)H * 2);
  /* Algorithm 1, one chain per "thread" */
  const uint8_t* code = pdd_bytes + tile_dir[tile * 4 + 0];
  for (int t = 0; t < tile_m; ++t) {
    const int64_t ch = tile * tile_m + t;
    const int len = chain_len[ch];
    if (chain_tau0[ch] == 0xFFFF && chain_rho0[ch] == 0xFFFF && len == 0) continue;   /* empty chain */
    int64_t offset_t = chain_tau0[ch], offset_r = chain_rho0[ch];
    if (offset_t >= slots || offset_r >= slots) return -2;
    visit(ctx, tm * tile_m + offset_r / H, tk * tile_k + 4 * ((offset_r % H) / 2) + 2 + (offset_r & 1), V[offset_t]);
    V[offset_t] = 0;
    for (int i = 0; i < len; ++i) {
      const int dt = code[i] & 0xF, dr = code[i] >> 4;
      offset_t += dt;
      offset_r += dr;
      if (dt == 0 || dr == 0) continue;           /* dummy point: only advances the cursors */
      if (offset_t >= slots || offset_r >= slots) return -2;
      visit(ctx, tm * tile_m + offset_r / H, tk * tile_k + 4 * ((offset_r % H) / 2) + 2 + (offset_r & 1), V[offset_t]);
      V[offset_t] = 0;
    }
    code += len;
  }
  /* Residual layer */
  const int64_t r0 = tile_dir[tile * 4 + 2], rn = tile_dir[tile * 4 + 3];
  for (int64_t j = r0; j < r0 + rn; ++j) {
    const int64_t rho = res_rho[j];
    if (rho >= slots) return -2;
    visit(ctx, tm * tile_m + rho / H, tk * tile_k + 4 * ((rho % H) / 2) + 2 + (rho & 1), res_val[j]);
  }
  /* what is left of the Sparse-TC layer: slot s of window q sits at column 4q + idx_s */
  for (int r = 0; r < tile_m; ++r) {
    const int64_t row = tm * tile_m + r;
    for (int q = 0; q < QW; ++q) {
      const int64_t gq = tk * QW + q;
      const uint8_t byte = tc_meta[row * (K_pad / 8) + gq / 2];
      const int nib = gq % 2 ? byte >> 4 : byte & 0xF;
      const int idx[2] = { nib & 3, nib >> 2 };
      for (int s = 0; s < 2; ++s) {
        const uint16_t v = V[(int64_t)r * H + 2 * q + s];
        if (is_nonzero(v)) visit(ctx, row, tk * tile_k + 4 * q + idx[s], v);
      }
    }
  }
  return 0;
}

/* ---------------------------------------------------------------- decode ---------------- */
typedef struct { uint16_t* W; int64_t M, K; int err; } decode_ctx;

static void decode_visit(void* p, int64_t row, int64_t col, uint16_t val) {
  decode_ctx* d = (decode_ctx*)p;
  if (!is_nonzero(val)) return;
  if (row >= d->M || col >= d->K) { d->err = 1; return; }    /* a non-zero in the padding */
  if (d->W[row * d->K + col] != 0) { d->err = 2; return; }   /* two layers claim one position */
  d->W[row * d->K + col] = val;
}

int oracle_decode(int64_t M, int64_t K, int tile_m, int tile_k,
                  const uint16_t* tc_vals, const uint8_t* tc_meta,
                  const uint16_t* chain_tau0, const uint16_t* chain_rho0, const uint8_t* chain_len,
                  const uint8_t* pdd_bytes, const uint32_t* tile_dir,
                  const uint16_t* res_rho, const uint16_t* res_val, uint16_t* W_out) {
  const int64_t M_pad = (M + tile_m - 1) / tile_m * tile_m, K_pad = (K + tile_k - 1) / tile_k * tile_k;
  memset(W_out, 0, (size_t)(M * K) * 2);
  uint16_t* V = (uint16_t*)malloc((size_t)tile_m * (tile_k / 2) * 2);
  decode_ctx d = { W_out, M, K, 0 };
  int rc = 0;
  for (int64_t tm = 0; tm < M_pad / tile_m && !rc; ++tm)
    for (int64_t tk = 0; tk < K_pad / tile_k && !rc; ++tk)
      rc = walk_tile(M_pad, K_pad, tile_m, tile_k, tc_vals, tc_meta, chain_tau0, chain_rho0, chain_len,
                     pdd_bytes, tile_dir, res_rho, res_val, tm, tk, V, decode_visit, &d);
  free(V);
  if (rc) return rc;
  return d.err ? -3 : 0;
}

/* ---------------------------------------------------------------- SpMM ------------------ */
typedef struct { float* acc; const uint16_t* X; int64_t row0, K; int N; int64_t ldx; } spmm_ctx;

static void spmm_visit(void* p, int64_t row, int64_t col, uint16_t val) {
  spmm_ctx* s = (spmm_ctx*)p;
  if (col >= s->K) return;                     /* padding columns hold no weight */
  const float w = half_to_float(val);
  float* a = s->acc + (row - s->row0) * s->N;
  const uint16_t* x = s->X + col * s->ldx;
  for (int j = 0; j < s->N; ++j) a[j] += w * half_to_float(x[j]);
}

/* Y[M x N] (fp16 bits, ld = ldy) = W * X[K x N] (fp16 bits, ld = ldx); fp32 accumulation. */
int oracle_spmm(int64_t M, int64_t K, int tile_m, int tile_k,
                const uint16_t* tc_vals, const uint8_t* tc_meta,
                const uint16_t* chain_tau0, const uint16_t* chain_rho0, const uint8_t* chain_len,
                const uint8_t* pdd_bytes, const uint32_t* tile_dir,
                const uint16_t* res_rho, const uint16_t* res_val,
                const uint16_t* X, int64_t ldx, uint16_t* Y, int64_t ldy, int N) {
  const int64_t M_pad = (M + tile_m - 1) / tile_m * tile_m, K_pad = (K + tile_k - 1) / tile_k * tile_k;
  const int64_t tiles_m = M_pad / tile_m, tiles_k = K_pad / tile_k;
  int rc_all = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t tm = 0; tm < tiles_m; ++tm) {
    uint16_t* V = (uint16_t*)malloc((size_t)tile_m * (tile_k / 2) * 2);
    float* acc = (float*)calloc((size_t)tile_m * N, sizeof(float));
    spmm_ctx s = { acc, X, tm * tile_m, K, N, ldx };
    int rc = 0;
    for (int64_t tk = 0; tk < tiles_k && !rc; ++tk)
      rc = walk_tile(M_pad, K_pad, tile_m, tile_k, tc_vals, tc_meta, chain_tau0, chain_rho0, chain_len,
                     pdd_bytes, tile_dir, res_rho, res_val, tm, tk, V, spmm_visit, &s);
    for (int r = 0; r < tile_m; ++r) {
      const int64_t row = tm * tile_m + r;
      if (row >= M) break;
      for (int j = 0; j < N; ++j) Y[row * ldy + j] = float_to_half_rne(acc[(int64_t)r * N + j]);
    }
    free(V); free(acc);
    if (rc) {
#pragma omp critical
      rc_all = rc;
    }
  }
  return rc_all;
}

#ifdef _OPENMP
#include <omp.h>
int oracle_threads(void) { return omp_get_max_threads(); }
#else
int oracle_threads(void) { return 1; }
#endif
