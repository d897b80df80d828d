// roles_kernel: the stage-decomposed all-reduce / reduce-scatter of the SM path as ONE cooperative launch whose CTAs have roles.
//
// Why.  Under the SM budget for sums the chain sum is the long pole (a 40 MiB bucket over 8 ranks: 292 us on 8 SMs), and the
// moves (the reduce-scatter's copies into the owners' inbox slots, the all-gather's fan-out) can run beside it as long as they
// stay below ~3.5 TB/s (faster copies lengthen the loads of the few summing SMs and slow the sum down).  The graph form gets
// that overlap from kernels of different pieces that run side by side and pays a launch and a pipeline ramp per piece and
// kernel; here the pieces are pipelined inside one kernel through counters instead:
//   * the first `n_sum` CTAs only sum: for piece p they wait until every mover has finished the reduce-scatter moves of piece p,
//     run the chain sum of that piece (the software-pipelined loop of chain_pipe_kernel) and count themselves done;
//   * the other CTAs only move: RS(0), RS(1), AG(0), RS(2), AG(1), ...; before the all-gather moves of piece p they wait until
//     every summing CTA has finished piece p.
// The counters are device words (one pair per piece); a count is a release reduction after a CTA barrier, a wait is an acquire
// poll by one thread followed by a CTA barrier, and everything a CTA reads that another CTA wrote in this launch is loaded
// with ld.global.cg (L2, never a stale L1 line).  The launch is cooperative, so all CTAs are resident together and no wait
// can be for a CTA that has not started; the order above has no cycle (the moves a sum waits for never wait for that sum).
// Every wait is bounded (kRingSpinLimit polls): a CTA that runs out sets a flag, every CTA that sees it skips the rest, the
// kernel ends by itself and the host reads the error word; the last CTA out clears the counters for the next launch.
// Rank locality holds as in the graph form: a mover copies a rank's own data, a summing CTA works in the owner's memory.
// The order of the adds and their rounding are those of chain_kernel: the bits are the oracle's.
//
// Measured (B200, R = 8, bf16, 8 summing + 40 moving CTAs, against the graph form with the same pieces and budgets): 25 MiB per
// rank 0.248 vs 0.245 ms, 40 MiB 0.377 vs 0.380, 64 MiB 0.599 vs 0.613, 128 MiB 1.14 vs 1.22, 256 MiB 2.28 vs 2.32.  So one
// launch instead of 24 to 48 buys a few per cent at best: every piece still drains and refills the register pipelines of both
// roles (4 to 5 us per piece for the sums, measured with the movers switched off), which is what the launches cost the graph
// form too.  Three things mattered more than the form: tables in shared memory (walking them in device memory cost the movers
// 24 us per piece), the three role bodies as functions of their own (inlined into one kernel the chain loop was scheduled
// 8 % slower, and any added variable pushed the kernel over its 128 registers), and scratch regions that start on 128-byte
// lines (plan.cpp).
#include <cuda_bf16.h>

#include "comm.h"
#include "device_common.cuh"

namespace hoccl {

namespace {

constexpr int kRolesThreads = 512;
constexpr int kCopyU = 8;    // vectors in flight per thread of a mover's copy tile (128 KiB per CTA)
constexpr int kFanU = 8;     // vectors per thread of a fan-out tile (64 KiB read once, stored ndst times)
constexpr int kChainP = 3;   // tiles of loads in flight per thread of a summing CTA
constexpr int kCtlWords = 4; // exits, gave-up flag, (unused) in front of the per-piece counters

struct RolesCopySeg {
  const void* src;
  void* dst;
  unsigned long long bytes, nvec, tiles_end, scalars_end;   // tiles_end, scalars_end: running counts over the segments of the group
  unsigned head, pad;
};
struct RolesChainSeg {
  const void* first;
  const void* local;
  void* out;
  unsigned long long n, stride, nvec, tiles_end, scalars_end;
  unsigned head;
  int nsrc;
};
struct RolesFanSeg {
  const void* src;
  unsigned long long bytes, nvec, tiles_end, scalars_end;
  unsigned head;
  int first_dst, ndst, pad;
};
struct RolesPiece {
  int c_first, c_n;   // reduce-scatter moves
  int h_first, h_n;   // chain sums
  int f_first, f_n;   // all-gather fan-out segments
  int x_first, x_n;   // all-gather moves that no fan-out segment carries (plain copies)
};
struct RolesArgs {
  const char* tab;     // the tables in device memory: pieces | copy segments | chain segments | fan segments | fan destinations
  unsigned o_c, o_h, o_f, o_d, total;   // byte offsets of the parts (multiples of 256) and the size of the whole
  unsigned pad0;
  unsigned* ctl;   // kCtlWords control words, then per piece {moved, summed}
  int* host_err;
  int npieces, n_sum, missing, pad;
};

// L2 eviction hints: what a mover puts into an inbox slot is read once, by a summing CTA, a piece later: it should stay in
// L2 until then and go first afterwards; what the all-gather stores is not read again in this launch.  (Measured: 2 % at
// 40 MiB per rank, nothing at 256 MiB; the L2 hit rate of the launch stays near 10 %.)
constexpr bool kL2Hints = true;
__device__ __forceinline__ unsigned long long policy_evict_last() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ unsigned long long policy_evict_first() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void st_hint(uint4* a, uint4 v, unsigned long long pol) {
  asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(pol) : "memory");
}
__device__ __forceinline__ uint4 ldcg_hint(const uint4* a, unsigned long long pol) {
  uint4 v;
  asm volatile("ld.global.cg.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(a), "l"(pol));
  return v;
}

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Everything this CTA wrote so far becomes visible to whoever sees the count.
__device__ __forceinline__ void count_done(unsigned* ctr) {
  __syncthreads();
  if (threadIdx.x == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");
}

// Returns false (for every thread of the CTA) once any CTA has given up.
// `seen`: a value of the counter that thread 0 read (with acquire) earlier; no poll if it already says enough.
__device__ __forceinline__ bool wait_count(const unsigned* ctr, unsigned target, unsigned* ctl, int* host_err, int* s_bail, unsigned seen = 0) {
  if (threadIdx.x == 0 && seen < target) {
    bool ok = true;
    unsigned it = 0;
    while (ld_acquire(ctr) < target) {
      if (++it > kRingSpinLimit || ((it & 63u) == 0 && ld_acquire(&ctl[1]) != 0)) {
        ok = false;
        break;
      }
      if (it > 1024) __nanosleep(64);
    }
    if (!ok) {
      atomicExch(&ctl[1], 1u);
      *reinterpret_cast<volatile int*>(host_err) = 1;
      *s_bail = 1;
    }
  }
  __syncthreads();
  return *reinterpret_cast<volatile int*>(s_bail) == 0;
}

// the last, short tile of a segment, in predicated quarter tiles (its own function: inlined, its registers pushed the kernel into spills)
__device__ __noinline__ void copy_ragged(const uint4* a, uint4* o, unsigned n_here, bool cg) {
  constexpr int UR = 4;
  for (unsigned base = 0; base < n_here; base += UR * kRolesThreads) {
    uint4 v[UR];
#pragma unroll
    for (int u = 0; u < UR; u++) {
      const unsigned i = base + threadIdx.x + u * kRolesThreads;
      if (i < n_here) v[u] = cg ? __ldcg(a + i) : __ldcs(a + i);
    }
#pragma unroll
    for (int u = 0; u < UR; u++) {
      const unsigned i = base + threadIdx.x + u * kRolesThreads;
      if (i < n_here) o[i] = v[u];
    }
  }
}

// ---- a mover's share of one group of plain copies: tiles m, m + M, ... of the group's flattened tile space (a tile = kCopyU
// vectors per thread, all loads of a tile issued before its stores).  Equal contiguous byte ranges per mover instead were tried:
// the extra live 64-bit values pushed the kernel over its 128 registers and every role got slower.
template <bool CG>
__device__ __noinline__ void copy_share(const RolesCopySeg* seg, int nseg, unsigned m, unsigned M) {
  if (nseg <= 0) return;
  constexpr unsigned tile_v = kCopyU * kRolesThreads;
  const unsigned long long keep = policy_evict_last();
  {
    const unsigned long long T_all = seg[nseg - 1].tiles_end;
    int k = 0;
    for (unsigned long long t = m; t < T_all; t += M) {
      while (t >= seg[k].tiles_end) k++;
      const unsigned long long first = (t - (k ? seg[k - 1].tiles_end : 0ull)) * tile_v;
      const unsigned long long left = seg[k].nvec - first;
      const unsigned n_here = left < tile_v ? (unsigned)left : tile_v;
      const uint4* a = reinterpret_cast<const uint4*>(static_cast<const char*>(seg[k].src) + seg[k].head) + first;
      uint4* o = reinterpret_cast<uint4*>(static_cast<char*>(seg[k].dst) + seg[k].head) + first;
      if (n_here == tile_v) {
        uint4 v[kCopyU];
#pragma unroll
        for (int u = 0; u < kCopyU; u++) v[u] = CG ? __ldcg(a + threadIdx.x + u * kRolesThreads) : __ldcs(a + threadIdx.x + u * kRolesThreads);
#pragma unroll
        for (int u = 0; u < kCopyU; u++) {
          if (kL2Hints && !CG) st_hint(o + threadIdx.x + u * kRolesThreads, v[u], keep);
          else o[threadIdx.x + u * kRolesThreads] = v[u];
        }
      } else {
        copy_ragged(a, o, n_here, CG);
      }
    }
  }
  {
    const unsigned long long total = (unsigned long long)M * kRolesThreads;
    const unsigned long long S = seg[nseg - 1].scalars_end;
    int k = 0;
    for (unsigned long long j = (unsigned long long)m * kRolesThreads + threadIdx.x; j < S; j += total) {
      while (j >= seg[k].scalars_end) k++;
      unsigned long long i = j - (k ? seg[k - 1].scalars_end : 0ull);
      if (i >= seg[k].head) i += seg[k].nvec * 16;
      static_cast<unsigned char*>(seg[k].dst)[i] = __ldcg(static_cast<const unsigned char*>(seg[k].src) + i);
    }
  }
}

// ---- a mover's share of the fan-out segments of one piece (a tile is loaded once and stored to every destination)
__device__ __noinline__ void fan_share(const RolesFanSeg* seg, int nseg, void* const* dst_all, unsigned m, unsigned M) {
  if (nseg <= 0) return;
  constexpr unsigned tile_v = kFanU * kRolesThreads;
  {
    const unsigned long long T_all = seg[nseg - 1].tiles_end;
    int k = 0;
    for (unsigned long long t = m; t < T_all; t += M) {
      while (t >= seg[k].tiles_end) k++;
      const unsigned long long first = (t - (k ? seg[k - 1].tiles_end : 0ull)) * tile_v;
      const unsigned long long left = seg[k].nvec - first;
      const unsigned n_here = left < tile_v ? (unsigned)left : tile_v;
      const uint4* a = reinterpret_cast<const uint4*>(static_cast<const char*>(seg[k].src) + seg[k].head) + first;
      void* const* dsts = dst_all + seg[k].first_dst;
      const int nd = seg[k].ndst;
      uint4 v[kFanU];
#pragma unroll
      for (int u = 0; u < kFanU; u++) {
        const unsigned i = threadIdx.x + u * kRolesThreads;
        if (i < n_here) v[u] = __ldcg(a + i);
      }
      for (int d = 0; d < nd; d++) {
        uint4* o = reinterpret_cast<uint4*>(static_cast<char*>(dsts[d]) + seg[k].head) + first;
#pragma unroll
        for (int u = 0; u < kFanU; u++) {
          const unsigned i = threadIdx.x + u * kRolesThreads;
          if (i < n_here) {
            if (kL2Hints) __stcs(o + i, v[u]);
            else o[i] = v[u];
          }
        }
      }
    }
  }
  {
    const unsigned long long total = (unsigned long long)M * kRolesThreads;
    const unsigned long long S = seg[nseg - 1].scalars_end;
    int k = 0;
    for (unsigned long long j = (unsigned long long)m * kRolesThreads + threadIdx.x; j < S; j += total) {
      while (j >= seg[k].scalars_end) k++;
      unsigned long long i = j - (k ? seg[k - 1].scalars_end : 0ull);
      if (i >= seg[k].head) i += seg[k].nvec * 16;
      const unsigned char v = __ldcg(static_cast<const unsigned char*>(seg[k].src) + i);
      void* const* dsts = dst_all + seg[k].first_dst;
      for (int d = 0; d < seg[k].ndst; d++) static_cast<unsigned char*>(dsts[d])[i] = v;
    }
  }
}

// one element of a chain segment, element-wise, operands from L2
template <int DT>
__device__ __forceinline__ void chain_scalar_cg(const RolesChainSeg& sg, unsigned long long i) {
  if (DT == 0) {
    float acc = __ldcg(static_cast<const float*>(sg.first) + i);
    for (int q = 1; q < sg.nsrc; q++) acc = __fadd_rn(acc, __ldcg(reinterpret_cast<const float*>(static_cast<const char*>(sg.first) + (size_t)q * sg.stride) + i));
    static_cast<float*>(sg.out)[i] = __fadd_rn(acc, __ldcg(static_cast<const float*>(sg.local) + i));
  } else {
    unsigned short acc = __ldcg(static_cast<const unsigned short*>(sg.first) + i);
    for (int q = 1; q <= sg.nsrc; q++) {
      const unsigned short b = q < sg.nsrc ? __ldcg(reinterpret_cast<const unsigned short*>(static_cast<const char*>(sg.first) + (size_t)q * sg.stride) + i)
                                           : __ldcg(static_cast<const unsigned short*>(sg.local) + i);
      const float s2 = __fadd_rn(__uint_as_float((uint32_t)acc << 16), __uint_as_float((uint32_t)b << 16));
      acc = __bfloat16_as_ushort(__float2bfloat16_rn(s2));
    }
    static_cast<unsigned short*>(sg.out)[i] = acc;
  }
}

// ---- a summing CTA's share of the chain sums of one piece: a contiguous range of the flattened tile space, the full tiles of a
// segment through a branch-free loop with kChainP tiles of loads in flight per thread (see chain_pipe_kernel)
template <int DT, int NOPS>
__device__ __noinline__ void chain_share(const RolesChainSeg* seg, int nseg, unsigned s, unsigned S) {
  using T = Traits<DT>;
  if (nseg <= 0) return;
  constexpr int P = kChainP, THREADS = kRolesThreads;
  const unsigned long long drop = policy_evict_first();
  {
    const unsigned long long T_all = seg[nseg - 1].tiles_end;
    const unsigned long long A = T_all / S * s + min((unsigned long long)s, T_all % S);
    const unsigned long long B = A + T_all / S + (s < T_all % S ? 1 : 0);
    int k = 0;
    while (k < nseg && seg[k].tiles_end <= A) k++;
    for (; k < nseg && (k ? seg[k - 1].tiles_end : 0ull) < B; k++) {
      const unsigned long long t0 = k ? seg[k - 1].tiles_end : 0ull;
      const unsigned long long a = (A > t0 ? A : t0) - t0;
      const unsigned long long b = (B < seg[k].tiles_end ? B : seg[k].tiles_end) - t0;
      const unsigned long long nvec = seg[k].nvec;
      const unsigned long long bf = b < nvec / THREADS ? b : nvec / THREADS;
      const size_t off0 = (size_t)seg[k].head * T::E + (size_t)threadIdx.x * 16;
      const char* src = static_cast<const char*>(seg[k].first) + off0;
      const char* loc = static_cast<const char*>(seg[k].local) + off0;
      char* out = static_cast<char*>(seg[k].out) + off0;
      const size_t stride = seg[k].stride;
      uint4 buf[P][NOPS];
      auto load = [&](uint4(&bb)[NOPS], unsigned long long t) {
        const size_t o = (size_t)t * THREADS * 16;
#pragma unroll
        for (int q = 0; q < NOPS - 1; q++)
          bb[q] = kL2Hints ? ldcg_hint(reinterpret_cast<const uint4*>(src + (size_t)q * stride + o), drop)
                                 : __ldcg(reinterpret_cast<const uint4*>(src + (size_t)q * stride + o));
        bb[NOPS - 1] = __ldcg(reinterpret_cast<const uint4*>(loc + o));
      };
      auto finish = [&](const uint4(&bb)[NOPS], unsigned long long t) {
        uint4 acc = bb[0];
#pragma unroll
        for (int q = 1; q < NOPS; q++) acc = DT == 1 ? add_vec_bf16_native(acc, bb[q]) : T::add_vec(acc, bb[q]);
        *reinterpret_cast<uint4*>(out + (size_t)t * THREADS * 16) = acc;
      };
      unsigned long long i = a;
      if (bf > a && bf - a >= (unsigned long long)P) {
#pragma unroll
        for (int p = 0; p < P - 1; p++) load(buf[p], i + p);
        for (; i + 2 * P - 1 <= bf; i += P) {
#pragma unroll
          for (int p = 0; p < P; p++) {
            load(buf[(p + P - 1) % P], i + p + P - 1);
            finish(buf[p], i + p);
          }
        }
#pragma unroll
        for (int p = 0; p < P - 1; p++) finish(buf[p], i + p);
        i += P - 1;
      }
      for (; i < bf; i++) {
        load(buf[0], i);
        finish(buf[0], i);
      }
      if (i < b && i * THREADS + threadIdx.x < nvec) {
        load(buf[0], i);
        finish(buf[0], i);
      }
    }
  }
  {
    const unsigned long long total = (unsigned long long)S * THREADS;
    const unsigned long long N = seg[nseg - 1].scalars_end;
    int k = 0;
    for (unsigned long long j = (unsigned long long)s * THREADS + threadIdx.x; j < N; j += total) {
      while (j >= seg[k].scalars_end) k++;
      unsigned long long i = j - (k ? seg[k - 1].scalars_end : 0ull);
      if (i >= seg[k].head) i += seg[k].nvec * T::VE;
      chain_scalar_cg<DT>(seg[k], i);
    }
  }
}

template <int DT, int NOPS>
__global__ void __launch_bounds__(kRolesThreads, 1) roles_kernel(const __grid_constant__ RolesArgs a) {
  // Every CTA first brings the tables of its role into shared memory: walking them in device memory cost a chain of dependent
  // loads per piece and phase (tens of microseconds per piece for the movers).
  extern __shared__ uint4 s_tab4[];
  char* s_tab = reinterpret_cast<char*>(s_tab4);
  __shared__ int s_bail;
  if (threadIdx.x == 0) s_bail = 0;
  const unsigned S = (unsigned)a.n_sum, M = gridDim.x - S;
  {
    const bool sums = blockIdx.x < S;
    const unsigned r0[2] = {0u, sums ? a.o_h : a.o_f}, r1[2] = {sums ? a.o_c : a.o_h, sums ? a.o_f : a.total};
    for (int part = 0; part < 2; part++)
      for (unsigned i = r0[part] / 16 + threadIdx.x; i < r1[part] / 16; i += kRolesThreads)
        s_tab4[i] = __ldg(reinterpret_cast<const uint4*>(a.tab) + i);
  }
  __syncthreads();
  const RolesPiece* piece = reinterpret_cast<const RolesPiece*>(s_tab);
  const RolesCopySeg* cseg = reinterpret_cast<const RolesCopySeg*>(s_tab + a.o_c);
  const RolesChainSeg* hseg = reinterpret_cast<const RolesChainSeg*>(s_tab + a.o_h);
  const RolesFanSeg* fseg = reinterpret_cast<const RolesFanSeg*>(s_tab + a.o_f);
  void* const* fdst = reinterpret_cast<void* const*>(s_tab + a.o_d);
  unsigned* moved = a.ctl + kCtlWords;          // moved[2 p]: movers that finished RS(p);  moved[2 p + 1]: summing CTAs that finished piece p
  const int P = a.npieces;
  if (blockIdx.x < S) {
    const unsigned s = blockIdx.x;
    unsigned seen = 0;
    for (int p = 0; p < P; p++) {
      if (!wait_count(&moved[2 * p], M + (unsigned)a.missing, a.ctl, a.host_err, &s_bail, seen)) break;
      // the next piece's counter is read now and looked at after this piece's sums: mostly it is complete by then, and no poll is needed
      seen = (threadIdx.x == 0 && p + 1 < P) ? ld_acquire(&moved[2 * (p + 1)]) : 0u;
      const RolesPiece pc = piece[p];
      chain_share<DT, NOPS>(hseg + pc.h_first, pc.h_n, s, S);
      count_done(&moved[2 * p + 1]);
    }
  } else {
    const unsigned m = blockIdx.x - S;
    bool ok = true;
    // The movers stay one piece ahead of the sums with the reduce-scatter moves; two to four pieces ahead measured the same or worse.
    constexpr int L = 1;
    for (int step = 0; step < P + L && ok; step++) {
      if (step < P) {   // the reduce-scatter moves of piece `step`: sources are the ranks' send buffers, written before the launch
        const RolesPiece pc = piece[step];
        copy_share<false>(cseg + pc.c_first, pc.c_n, m, M);
        count_done(&moved[2 * step]);
      }
      if (step >= L) {  // the all-gather moves of piece step - L: sources were written by summing CTAs in this launch
        const int p = step - L;
        const RolesPiece pc = piece[p];
        if (pc.f_n > 0 || pc.x_n > 0) {
          ok = wait_count(&moved[2 * p + 1], S, a.ctl, a.host_err, &s_bail);
          if (ok) {
            fan_share(fseg + pc.f_first, pc.f_n, fdst, m, M);
            copy_share<true>(cseg + pc.x_first, pc.x_n, m, M);
          }
        }
      }
    }
  }
  // leave: the last CTA out clears the counters, so that the next launch starts from zero even after a give-up
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned gone = atomicAdd(&a.ctl[0], 1u);
    if (gone == gridDim.x - 1) {
      for (int p = 0; p < 2 * P; p++) moved[p] = 0;
      a.ctl[1] = 0;
      __threadfence();
      a.ctl[0] = 0;
    }
  }
}

template <int DT>
const void* roles_entry_t(int nops) {
  switch (nops) {
    case 2: return reinterpret_cast<const void*>(&roles_kernel<DT, 2>);
    case 3: return reinterpret_cast<const void*>(&roles_kernel<DT, 3>);
    case 4: return reinterpret_cast<const void*>(&roles_kernel<DT, 4>);
    case 5: return reinterpret_cast<const void*>(&roles_kernel<DT, 5>);
    case 6: return reinterpret_cast<const void*>(&roles_kernel<DT, 6>);
    case 7: return reinterpret_cast<const void*>(&roles_kernel<DT, 7>);
    case 8: return reinterpret_cast<const void*>(&roles_kernel<DT, 8>);
    default: return nullptr;
  }
}
const void* roles_entry(int dtype, int nops) { return dtype == 0 ? roles_entry_t<0>(nops) : roles_entry_t<1>(nops); }

void split_bytes(const void* a, const void* b, unsigned long long bytes, unsigned long long* tiles, unsigned long long* scalars, unsigned* head,
                 unsigned long long* nvec) {
  constexpr unsigned long long tile_v = (unsigned long long)kCopyU * kRolesThreads;
  const unsigned ma = (unsigned)((uintptr_t)a & 15), mb = (unsigned)((uintptr_t)b & 15);
  unsigned long long ns;
  split_segment(bytes, ma, ma == mb, 1, 16, head, nvec, &ns);
  *tiles += (*nvec + tile_v - 1) / tile_v;
  *scalars += ns;
}

}  // namespace

constexpr size_t kRolesTabMax = 200 << 10;   // the tables of one launch live in every CTA's shared memory
constexpr size_t kRolesCtlBytes = 1024;
constexpr int kRolesMaxPieces = 64;

// Control words and counters of the roles kernel are the library's own (1 KiB of device memory and 4 bytes of mapped pinned
// host memory per communicator), allocated on first use; every cached call signature keeps its table in device memory of its own.
static hoccl_result_t ensure_roles_ctrl(hoccl_comm* c) {
  if (c->roles_ctl) return HOCCL_OK;
  char* ctl = nullptr;
  CU_TRY(c, cudaMalloc(&ctl, kRolesCtlBytes));
  cudaError_t e = cudaMemset(ctl, 0, kRolesCtlBytes);
  int* err = nullptr;
  int* err_dev = nullptr;
  if (e == cudaSuccess) {
    e = cudaHostAlloc(&err, sizeof(int), cudaHostAllocMapped);
    if (e == cudaSuccess) {
      *err = 0;
      e = cudaHostGetDevicePointer(&err_dev, err, 0);
    }
  }
  for (int dt = 0; dt < 2 && e == cudaSuccess; dt++)
    for (int nops = 2; nops <= 8 && e == cudaSuccess; nops++) {
      // (this also loads the kernel now, not at its first launch)
      e = cudaFuncSetAttribute(roles_entry(dt, nops), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRolesTabMax);
    }
  if (e != cudaSuccess) {
    cudaFree(ctl);
    if (err) cudaFreeHost(err);
    return cuda_fail(c, e, "roles kernel control memory");
  }
  c->roles_err = err;
  c->roles_err_dev = err_dev;
  c->roles_ctl = ctl;
  return HOCCL_OK;
}

// Turns the resolved plan (direct reduce-scatter, optionally with the direct all-gather behind it, SM path) into the table of one
// roles_kernel launch.  UNSUPPORTED if the plan does not have that shape or does not fit: the caller then builds the graph.
hoccl_result_t build_roles(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry) {
  if (!P.rs_direct || P.R < 2 || P.R > 8 || P.pieces > kRolesMaxPieces) return HOCCL_ERR_UNSUPPORTED;
  const int nops = P.R;   // R - 1 inbox operands and the local one
  const long n_sum = std::max<long>(1, std::min<long>(c->sum_ctas, 64));
  const long n_move = std::max<long>(1, c->copy_ctas);
  int per_sm = 0;
  hoccl_result_t rc = ensure_roles_ctrl(c);
  if (rc != HOCCL_OK) return rc;
  std::vector<RolesPiece> pieces((size_t)P.pieces, RolesPiece{0, 0, 0, 0, 0, 0, 0, 0});
  std::vector<RolesCopySeg> cseg;
  std::vector<RolesChainSeg> hseg;
  std::vector<RolesFanSeg> fseg;
  std::vector<void*> fdst;
  const size_t E = P.elem;
  long moves = 0;
  for (int p = 0; p < P.pieces; p++) {
    RolesPiece& pc = pieces[(size_t)p];
    // reduce-scatter moves of the piece
    pc.c_first = (int)cseg.size();
    unsigned long long tiles = 0, scalars = 0;
    for (const RGroup& g : groups) {
      if (g.piece != p || g.kind != OP_MOVE || g.phase != PHASE_RS) continue;
      for (const Seg& s : g.segs) {
        RolesCopySeg r = {s.src, s.dst, (unsigned long long)s.bytes, 0, 0, 0, 0, 0};
        split_bytes(s.src, s.dst, s.bytes, &tiles, &scalars, &r.head, &r.nvec);
        r.tiles_end = tiles;
        r.scalars_end = scalars;
        cseg.push_back(r);
        moves++;
      }
    }
    pc.c_n = (int)cseg.size() - pc.c_first;
    // chain sums
    pc.h_first = (int)hseg.size();
    tiles = scalars = 0;
    for (const RGroup& g : groups) {
      if (g.piece != p || g.kind == OP_MOVE) continue;
      if (g.kind != OP_CHAIN) return HOCCL_ERR_UNSUPPORTED;
      for (const Seg& s : g.segs) {
        if (s.nsrc + 1 != nops) return HOCCL_ERR_UNSUPPORTED;
        RolesChainSeg r = {s.src, s.local, s.dst, (unsigned long long)(s.bytes / E), (unsigned long long)s.src_stride, 0, 0, 0, 0, s.nsrc};
        const unsigned ma = (unsigned)((uintptr_t)s.src & 15), mb = (unsigned)((uintptr_t)s.local & 15), mo = (unsigned)((uintptr_t)s.dst & 15);
        unsigned long long ns;
        split_segment(r.n, ma, ma == mb && mb == mo && (s.src_stride & 15) == 0, (int)E, (int)(16 / E), &r.head, &r.nvec, &ns);
        tiles += (r.nvec + kRolesThreads - 1) / kRolesThreads;
        scalars += ns;
        r.tiles_end = tiles;
        r.scalars_end = scalars;
        hseg.push_back(r);
      }
    }
    pc.h_n = (int)hseg.size() - pc.h_first;
    // all-gather moves: fan-out segments where a source repeats, plain copies otherwise
    pc.f_first = (int)fseg.size();
    pc.x_first = (int)cseg.size();
    unsigned long long ftiles = 0, fscalars = 0;
    tiles = scalars = 0;
    for (const RGroup& g : groups) {
      if (g.piece != p || g.kind != OP_MOVE || g.phase == PHASE_RS) continue;
      std::vector<FanBatch> fans;
      std::vector<double> fb;
      std::vector<long> fm;
      if (build_fan_batches(g, &fans, &fb, &fm)) {
        for (const FanBatch& b : fans)
          for (int k = 0; k < b.nseg; k++) {
            const FanSeg& fs = b.seg[k];
            RolesFanSeg r = {fs.src, fs.bytes, 0, 0, 0, 0, (int)fdst.size(), fs.ndst, 0};
            const unsigned ms = (unsigned)((uintptr_t)fs.src & 15);
            bool same = true;
            for (int d = 0; d < fs.ndst; d++) {
              same = same && ((unsigned)((uintptr_t)b.dst[fs.first_dst + d] & 15) == ms);
              fdst.push_back(b.dst[fs.first_dst + d]);
            }
            unsigned long long ns;
            split_segment(fs.bytes, ms, same, 1, 16, &r.head, &r.nvec, &ns);
            ftiles += (r.nvec + (unsigned long long)kFanU * kRolesThreads - 1) / ((unsigned long long)kFanU * kRolesThreads);
            fscalars += ns;
            r.tiles_end = ftiles;
            r.scalars_end = fscalars;
            fseg.push_back(r);
            moves += fs.ndst;
          }
      } else {
        for (const Seg& s : g.segs) {
          RolesCopySeg r = {s.src, s.dst, (unsigned long long)s.bytes, 0, 0, 0, 0, 0};
          split_bytes(s.src, s.dst, s.bytes, &tiles, &scalars, &r.head, &r.nvec);
          r.tiles_end = tiles;
          r.scalars_end = scalars;
          cseg.push_back(r);
          moves++;
        }
      }
    }
    pc.f_n = (int)fseg.size() - pc.f_first;
    pc.x_n = (int)cseg.size() - pc.x_first;
  }
  // layout of the table: pieces | copy segments | chain segments | fan segments | fan destinations
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  const size_t o_piece = 0, o_c = up(pieces.size() * sizeof(RolesPiece)), o_h = o_c + up(cseg.size() * sizeof(RolesCopySeg)),
               o_f = o_h + up(hseg.size() * sizeof(RolesChainSeg)), o_d = o_f + up(fseg.size() * sizeof(RolesFanSeg)),
               total = o_d + up(fdst.size() * sizeof(void*));
  if (total > kRolesTabMax) return HOCCL_ERR_UNSUPPORTED;
  CU_TRY(c, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, roles_entry(P.dtype, nops), kRolesThreads, total));
  if (n_sum + n_move > (long)per_sm * c->num_sms) return HOCCL_ERR_UNSUPPORTED;   // all CTAs must be resident together
  std::vector<char> host(total, 0);
  std::memcpy(host.data() + o_piece, pieces.data(), pieces.size() * sizeof(RolesPiece));
  if (!cseg.empty()) std::memcpy(host.data() + o_c, cseg.data(), cseg.size() * sizeof(RolesCopySeg));
  if (!hseg.empty()) std::memcpy(host.data() + o_h, hseg.data(), hseg.size() * sizeof(RolesChainSeg));
  if (!fseg.empty()) std::memcpy(host.data() + o_f, fseg.data(), fseg.size() * sizeof(RolesFanSeg));
  if (!fdst.empty()) std::memcpy(host.data() + o_d, fdst.data(), fdst.size() * sizeof(void*));
  char* dev = nullptr;
  CU_TRY(c, cudaMalloc(&dev, total));
  {
    cudaError_t ce = cudaMemcpy(dev, host.data(), total, cudaMemcpyHostToDevice);   // once, when the signature is first seen
    if (ce != cudaSuccess) {
      cudaFree(dev);
      return cuda_fail(c, ce, "roles kernel table");
    }
  }
  entry->roles_tab = dev;
  RolesArgs a = {};
  a.tab = dev;
  a.o_c = (unsigned)o_c;
  a.o_h = (unsigned)o_h;
  a.o_f = (unsigned)o_f;
  a.o_d = (unsigned)o_d;
  a.total = (unsigned)total;
  a.ctl = reinterpret_cast<unsigned*>(c->roles_ctl);
  a.host_err = c->roles_err_dev;
  a.npieces = P.pieces;
  a.n_sum = (int)n_sum;
  a.missing = (int)c->roles_missing;
  entry->roles_args.assign(sizeof(RolesArgs), 0);
  std::memcpy(entry->roles_args.data(), &a, sizeof(RolesArgs));
  entry->roles_grid = (int)(n_sum + n_move);
  entry->roles_sum_ctas = (int)n_sum;
  entry->roles_smem = total;
  entry->roles_fn = roles_entry(P.dtype, nops);
  entry->n_moves = moves;
  entry->n_move_launches = 1;
  entry->n_sum_launches = 0;
  entry->n_pieces = P.pieces;
  return HOCCL_OK;
}

hoccl_result_t launch_roles(hoccl_comm* c, GraphEntry* entry, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)entry->roles_grid);
  cfg.blockDim = dim3((unsigned)kRolesThreads);
  cfg.dynamicSmemBytes = entry->roles_smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  void* args[] = {entry->roles_args.data()};
  CU_TRY(c, cudaLaunchKernelExC(&cfg, entry->roles_fn, args));
  return HOCCL_OK;
}

}  // namespace hoccl
