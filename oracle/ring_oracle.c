/*
 * CPU oracle for the ring collectives.  TEST INFRASTRUCTURE ONLY: nothing on the product path
 * may include, link or call this file; the CUDA library shares no code with it.
 *
 * What it follows.  The paper (HOCCL) moves collective data with copy engines and treats
 * AllGather and point-to-point send/recv as pure byte moves (Sec. 3.3 "Zero-SM Point-to-Point
 * Executor", Sec. 5 "Communication benchmarks"); it states that reductions are outside its scope
 * (Sec. 4 "Limitations").  The reduction is therefore the textbook ring reduce-scatter in a fixed
 * order: R ranks, R ring chunks, data travels r -> (r+1) mod R, rank r
 * ends the reduce-scatter owning chunk r, the travelling partial is stored in the I/O dtype at every
 * hop, and each hop is ONE IEEE binary32 add followed by round-to-nearest-even to the I/O dtype.
 *
 *   oracle_ring_allreduce / oracle_ring_reduce_scatter : the schedule executed step by step with
 *       R separate arenas (inbox I_r, partial P_r), moves are memcpy, sums are scalar loops.
 *   oracle_allgather   : the definition (concatenation), written as the ring of moves.
 *   oracle_sendrecv    : the definition (identity on bytes).
 *   oracle_alltoall    : the definition (block transpose).
 *   oracle_chain_sum   : closed form of the ring order for one chunk,
 *                        ((x_{c+1} + x_{c+2}) + ... + x_{c+R-1}) + x_c, used to pin the step-by-step code.
 *   oracle_sum_f64     : fp64 sum and fp64 sum of magnitudes (for the error bound).
 *
 * dtype: 0 = fp32, 1 = bf16 (stored as uint16_t, the high half of a binary32).
 * Build with: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp (no FTZ/DAZ, no FMA).
 * `threads` only splits element loops across OpenMP threads; every element is computed by the same
 * scalar code in the same order, so the result does not depend on it.
 *
 * Pins (tests/test_oracle_pins.py): two hand-worked order fingerprints, exact integer sums,
 * R=2 commutativity, the chain closed form, allgather == concatenation, all ranks identical,
 * the fp64 error bound, and an independent exact-rational bf16 rounding.
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { DT_F32 = 0, DT_BF16 = 1 };

static size_t esize(int dtype) { return dtype == DT_F32 ? 4 : 2; }

static float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* round-to-nearest-even binary32 -> bf16; NaN stays NaN */
static uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
  u += 0x7fffu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

/* one hop: out = rn_T( f32(a) + f32(b) ), a = what arrived in the inbox, b = the local contribution */
static void sum_span(int dtype, const void* inbox, const void* local, void* out, size_t n, int threads) {
  (void)threads;
  if (dtype == DT_F32) {
    const float* a = (const float*)inbox;
    const float* b = (const float*)local;
    float* o = (float*)out;
#pragma omp parallel for num_threads(threads) schedule(static) if (threads > 1)
    for (size_t i = 0; i < n; i++) {
      volatile float s = a[i] + b[i];
      o[i] = s;
    }
  } else {
    const uint16_t* a = (const uint16_t*)inbox;
    const uint16_t* b = (const uint16_t*)local;
    uint16_t* o = (uint16_t*)out;
#pragma omp parallel for num_threads(threads) schedule(static) if (threads > 1)
    for (size_t i = 0; i < n; i++) {
      volatile float s = bf16_to_f32(a[i]) + bf16_to_f32(b[i]);
      o[i] = f32_to_bf16_rne(s);
    }
  }
}

static void move_span(void* dst, const void* src, size_t bytes, int threads) {
  if (threads <= 1 || bytes < (1u << 20)) {
    memmove(dst, src, bytes);
    return;
  }
  size_t per = (bytes + (size_t)threads - 1) / (size_t)threads;
#pragma omp parallel for num_threads(threads) schedule(static)
  for (int t = 0; t < threads; t++) {
    size_t lo = (size_t)t * per;
    if (lo < bytes) {
      size_t len = bytes - lo < per ? bytes - lo : per;
      memmove((char*)dst + lo, (const char*)src + lo, len);
    }
  }
}

/* allreduce partition of n elements into R ring chunks: q = ceil(n/R); chunk c = [min(cq,n), min((c+1)q,n)) */
void oracle_chunk_range(size_t n, int R, int c, size_t* lo, size_t* hi) {
  size_t q = (n + (size_t)R - 1) / (size_t)R;
  size_t a = (size_t)c * q, b = ((size_t)c + 1) * q;
  *lo = a < n ? a : n;
  *hi = b < n ? b : n;
}

static int mod(int a, int R) { return ((a % R) + R) % R; }

/*
 * Ring reduce-scatter over explicit chunk ranges.  X[r] is rank r's full send buffer; after the
 * call final_out[r] + final_off[r] holds the reduced chunk r.  lo/hi give chunk boundaries in
 * elements (R entries each).
 */
static int ring_rs(int R, int dtype, const void* const* X, void* const* final_out, const size_t* final_off_el,
                   const size_t* lo, const size_t* hi, int threads) {
  size_t e = esize(dtype);
  size_t maxlen = 0;
  for (int c = 0; c < R; c++)
    if (hi[c] - lo[c] > maxlen) maxlen = hi[c] - lo[c];
  char** I = (char**)calloc((size_t)R, sizeof(char*));
  char** P = (char**)calloc((size_t)R, sizeof(char*));
  if (!I || !P) return -1;
  for (int r = 0; r < R; r++) {
    I[r] = (char*)malloc(maxlen * e + 1);
    P[r] = (char*)malloc(maxlen * e + 1);
    if (!I[r] || !P[r]) return -1;
  }
  for (int s = 0; s <= R - 2; s++) {
    /* MOVE(s, r): chunk c = (r-1-s) mod R leaves rank r for the inbox of rank next(r) */
    for (int r = 0; r < R; r++) {
      int c = mod(r - 1 - s, R);
      size_t len = hi[c] - lo[c];
      const char* src = (s == 0) ? (const char*)X[r] + lo[c] * e : P[r];
      move_span(I[(r + 1) % R], src, len * e, threads);
    }
    /* SUM(s, r): chunk c = (r-2-s) mod R; arrived partial + rank r's own contribution */
    for (int r = 0; r < R; r++) {
      int c = mod(r - 2 - s, R);
      size_t len = hi[c] - lo[c];
      void* out = (s < R - 2) ? (void*)P[r] : (void*)((char*)final_out[r] + final_off_el[r] * e);
      sum_span(dtype, I[r], (const char*)X[r] + lo[c] * e, out, len, threads);
    }
  }
  for (int r = 0; r < R; r++) {
    free(I[r]);
    free(P[r]);
  }
  free(I);
  free(P);
  return 0;
}

/* ring all-gather of chunk ranges already in place: Y[next(r)][chunk] <- Y[r][chunk], chunk = (r-s) mod R */
static void ring_ag(int R, int dtype, void* const* Y, const size_t* lo, const size_t* hi, int threads) {
  size_t e = esize(dtype);
  for (int s = 0; s <= R - 2; s++)
    for (int r = 0; r < R; r++) {
      int c = mod(r - s, R);
      move_span((char*)Y[(r + 1) % R] + lo[c] * e, (const char*)Y[r] + lo[c] * e, (hi[c] - lo[c]) * e, threads);
    }
}

/* allreduce(sum): X[r], Y[r] hold n elements each; X[r] may equal Y[r] (in place). */
int oracle_ring_allreduce(int R, size_t n, int dtype, const void* const* X, void* const* Y, int threads) {
  if (R < 1 || (dtype != DT_F32 && dtype != DT_BF16)) return -2;
  size_t e = esize(dtype);
  if (R == 1) {
    if (X[0] != Y[0]) memmove(Y[0], X[0], n * e);
    return 0;
  }
  size_t* lo = (size_t*)malloc(sizeof(size_t) * (size_t)R * 3);
  if (!lo) return -1;
  size_t *hi = lo + R, *off = hi + R;
  for (int c = 0; c < R; c++) {
    oracle_chunk_range(n, R, c, &lo[c], &hi[c]);
    off[c] = lo[c];
  }
  int rc = ring_rs(R, dtype, X, Y, off, lo, hi, threads);
  if (rc == 0) ring_ag(R, dtype, Y, lo, hi, threads);
  free(lo);
  return rc;
}

/* reduce_scatter(sum): X[r] holds R*count elements, Y[r] receives count elements (chunk r of the sum). */
int oracle_ring_reduce_scatter(int R, size_t count, int dtype, const void* const* X, void* const* Y, int threads) {
  if (R < 1 || (dtype != DT_F32 && dtype != DT_BF16)) return -2;
  size_t e = esize(dtype);
  if (R == 1) {
    if (X[0] != Y[0]) memmove(Y[0], X[0], count * e);
    return 0;
  }
  size_t* lo = (size_t*)malloc(sizeof(size_t) * (size_t)R * 3);
  if (!lo) return -1;
  size_t *hi = lo + R, *off = hi + R;
  for (int c = 0; c < R; c++) {
    lo[c] = (size_t)c * count;
    hi[c] = lo[c] + count;
    off[c] = 0;
  }
  int rc = ring_rs(R, dtype, X, Y, off, lo, hi, threads);
  free(lo);
  return rc;
}

/* allgather: X[r] holds count elements, Y[r] receives R*count = X[0] | X[1] | ... | X[R-1]. */
int oracle_allgather(int R, size_t count, int dtype, const void* const* X, void* const* Y, int threads) {
  if (R < 1 || (dtype != DT_F32 && dtype != DT_BF16)) return -2;
  size_t e = esize(dtype);
  size_t* lo = (size_t*)malloc(sizeof(size_t) * (size_t)R * 2);
  if (!lo) return -1;
  size_t* hi = lo + R;
  for (int c = 0; c < R; c++) {
    lo[c] = (size_t)c * count;
    hi[c] = lo[c] + count;
  }
  for (int r = 0; r < R; r++) {
    char* own = (char*)Y[r] + lo[r] * e;
    if ((const void*)own != X[r]) memmove(own, X[r], count * e);
  }
  ring_ag(R, dtype, Y, lo, hi, threads);
  free(lo);
  return 0;
}

/* all-to-all (the paper's second benchmarked collective, Sec. 5): X[r], Y[r] hold R blocks of count elements;
 * block j of Y[r] is block r of X[j].  Written as the definition, block by block. */
int oracle_alltoall(int R, size_t count, int dtype, const void* const* X, void* const* Y) {
  if (R < 1 || (dtype != DT_F32 && dtype != DT_BF16)) return -2;
  size_t b = count * esize(dtype);
  for (int r = 0; r < R; r++)
    for (int j = 0; j < R; j++) memcpy((char*)Y[r] + (size_t)j * b, (const char*)X[j] + (size_t)r * b, b);
  return 0;
}

/* user-defined pattern (all-to-allv; the paper routes arbitrary patterns through its traffic matrix, Sec. 3.4):
 * rank u sends sendcounts[u*R+v] elements from X[u] + sdispls[u*R+v] to rank v at Y[v] + rdispls[v*R+u].  The definition. */
int oracle_alltoallv(int R, int dtype, const void* const* X, const size_t* sendcounts, const size_t* sdispls, void* const* Y,
                     const size_t* rdispls) {
  if (R < 1 || (dtype != DT_F32 && dtype != DT_BF16)) return -2;
  size_t e = esize(dtype);
  for (int u = 0; u < R; u++)
    for (int v = 0; v < R; v++)
      memcpy((char*)Y[v] + rdispls[(size_t)v * R + u] * e, (const char*)X[u] + sdispls[(size_t)u * R + v] * e,
             sendcounts[(size_t)u * R + v] * e);
  return 0;
}

/* point-to-point: the receiver's buffer becomes a byte copy of the sender's. */
int oracle_sendrecv(const void* src, void* dst, size_t count, int dtype) {
  memmove(dst, src, count * esize(dtype));
  return 0;
}

/*
 * Closed form of the ring order for elements [lo,hi) that all belong to chunk c:
 * acc = x_{c+1}; acc = acc (+) x_{c+2}; ... ; acc = acc (+) x_{c+R-1}; acc = acc (+) x_c  (indices mod R).
 */
int oracle_chain_sum(int R, int c, size_t lo, size_t hi, int dtype, const void* const* X, void* out) {
  if (R < 1) return -2;
  for (size_t i = lo; i < hi; i++) {
    if (dtype == DT_F32) {
      volatile float acc = ((const float*)X[(c + 1) % R])[i];
      for (int k = 2; k <= R; k++) {
        float b = ((const float*)X[(c + k) % R])[i];
        acc = acc + b;
      }
      ((float*)out)[i - lo] = (R == 1) ? ((const float*)X[0])[i] : acc;
    } else {
      uint16_t acc = ((const uint16_t*)X[(c + 1) % R])[i];
      for (int k = 2; k <= R; k++) {
        volatile float s = bf16_to_f32(acc) + bf16_to_f32(((const uint16_t*)X[(c + k) % R])[i]);
        acc = f32_to_bf16_rne(s);
      }
      ((uint16_t*)out)[i - lo] = (R == 1) ? ((const uint16_t*)X[0])[i] : acc;
    }
  }
  return 0;
}

/* fp64 reference: sum_r x_r[i] and sum_r |x_r[i]| accumulated in double in rank order. */
int oracle_sum_f64(int R, size_t n, int dtype, const void* const* X, double* sum, double* sum_abs) {
  for (size_t i = 0; i < n; i++) {
    double s = 0.0, a = 0.0;
    for (int r = 0; r < R; r++) {
      double v = dtype == DT_F32 ? (double)((const float*)X[r])[i] : (double)bf16_to_f32(((const uint16_t*)X[r])[i]);
      s += v;
      a += fabs(v);
    }
    sum[i] = s;
    if (sum_abs) sum_abs[i] = a;
  }
  return 0;
}

int oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
