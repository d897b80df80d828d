// ring_kernel: a whole collective of the SM path in ONE cooperative launch.
//
// The host hands over the plan's groups as a table of phases (a MOVE phase = the copies of one ring step for all ranks,
// a SUM phase = that step's chunk sums).  All CTAs work through the table together; where a phase depends on an earlier
// one they meet at a grid-wide barrier first.  The barrier is the usual arrive-and-poll on one device word; every wait
// is bounded (kRingSpinLimit polls): a CTA that runs out sets a flag, every CTA that sees the flag skips the rest of
// the table, and the kernel ends by itself.  The last CTA to leave clears the barrier words for the next launch.
// The launch is cooperative, so all CTAs are resident together and the barrier cannot wait for a CTA that has not
// started.
//
// Data written by one CTA in a phase is read by another CTA in a later phase: stores are followed by __threadfence()
// before the arrival (a release reduction), the poll is an acquire load (measured faster than relaxed polls plus one fence), and operands are loaded with ld.global.cg (L2, never a stale L1 line).
#include <cuda_bf16.h>

#include "device_common.cuh"

namespace hoccl {

namespace {

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Returns false (for every thread of the CTA) once any CTA has given up.
__device__ __forceinline__ bool grid_barrier(unsigned* bar, unsigned target, int* host_err, int* s_bail) {
  __syncthreads();
  if (threadIdx.x == 0) {
    // release: everything this CTA wrote (ordered before by the bar.sync above) is visible to whoever sees the arrival
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(bar) : "memory");
    bool ok = true;
    unsigned it = 0;
    while (ld_acquire_u32(&bar[0]) < target) {
      if (++it > kRingSpinLimit || ((it & 63u) == 0 && ld_acquire_u32(&bar[2]) != 0)) {
        ok = false;
        break;
      }
      if (it > 2048) __nanosleep(128);
    }
    if (!ok) {
      atomicExch(&bar[2], 1u);
      *reinterpret_cast<volatile int*>(host_err) = 1;
      *s_bail = 1;
    }
  }
  __syncthreads();
  return *reinterpret_cast<volatile int*>(s_bail) == 0;
}

// element-wise add with L2 loads (heads, tails and segments without a common 16-byte phase)
template <int DT>
__device__ __forceinline__ void add_scalar_cg(const void* a, const void* b, void* o, unsigned long long i) {
  if (DT == 0) {
    static_cast<float*>(o)[i] = __fadd_rn(__ldcg(static_cast<const float*>(a) + i), __ldcg(static_cast<const float*>(b) + i));
  } else {
    const unsigned short xa = __ldcg(static_cast<const unsigned short*>(a) + i), xb = __ldcg(static_cast<const unsigned short*>(b) + i);
    const float s = __fadd_rn(__uint_as_float((uint32_t)xa << 16), __uint_as_float((uint32_t)xb << 16));
    static_cast<unsigned short*>(o)[i] = __bfloat16_as_ushort(__float2bfloat16_rn(s));
  }
}

// A phase needs no set-up: the host has split every segment into head / vector body / tail and written the running
// totals of tiles and element-wise items of the phase next to it (RingSeg::tiles_end, ::scalars_end).
template <int DT, int U, int THREADS>
__device__ __forceinline__ void sum_phase(const RingSeg* seg, int nseg) {
  using T = Traits<DT>;
  constexpr unsigned tile_v = U * THREADS;
  {
    const unsigned long long T_all = seg[nseg - 1].tiles_end;
    int k = 0;
    for (unsigned long long t = blockIdx.x; t < T_all; t += gridDim.x) {
      while (t >= seg[k].tiles_end) k++;
      const unsigned long long first = (t - (k ? seg[k - 1].tiles_end : 0ull)) * tile_v;
      const unsigned long long left = seg[k].nvec - first;
      const unsigned n_here = left < tile_v ? (unsigned)left : tile_v;
      const size_t h = (size_t)seg[k].head * T::E;
      const uint4* a = reinterpret_cast<const uint4*>(static_cast<const char*>(seg[k].src) + h) + first;
      const uint4* b = reinterpret_cast<const uint4*>(static_cast<const char*>(seg[k].local) + h) + first;
      uint4* o = reinterpret_cast<uint4*>(static_cast<char*>(seg[k].dst) + h) + first;
      uint4 va[U], vb[U];
      if (n_here == tile_v) {
#pragma unroll
        for (int u = 0; u < U; u++) {
          va[u] = __ldcg(a + threadIdx.x + u * THREADS);
          vb[u] = __ldcg(b + threadIdx.x + u * THREADS);
        }
#pragma unroll
        for (int u = 0; u < U; u++) o[threadIdx.x + u * THREADS] = T::add_vec(va[u], vb[u]);
      } else {
        for (unsigned i = threadIdx.x; i < n_here; i += THREADS) o[i] = T::add_vec(__ldcg(a + i), __ldcg(b + i));
      }
    }
  }
  {
    const unsigned long long total = (unsigned long long)gridDim.x * THREADS;
    const unsigned long long S = seg[nseg - 1].scalars_end;
    int k = 0;
    for (unsigned long long j = (unsigned long long)blockIdx.x * THREADS + threadIdx.x; j < S; j += total) {
      while (j >= seg[k].scalars_end) k++;
      unsigned long long i = j - (k ? seg[k - 1].scalars_end : 0ull);
      if (i >= seg[k].head) i += seg[k].nvec * T::VE;
      add_scalar_cg<DT>(seg[k].src, seg[k].local, seg[k].dst, i);
    }
  }
}

template <int U, int THREADS>
__device__ __forceinline__ void copy_phase(const RingSeg* seg, int nseg) {
  constexpr unsigned tile_v = U * THREADS;
  {
    const unsigned long long T_all = seg[nseg - 1].tiles_end;
    int k = 0;
    for (unsigned long long t = blockIdx.x; t < T_all; t += gridDim.x) {
      while (t >= seg[k].tiles_end) k++;
      const unsigned long long first = (t - (k ? seg[k - 1].tiles_end : 0ull)) * tile_v;
      const unsigned long long left = seg[k].nvec - first;
      const unsigned n_here = left < tile_v ? (unsigned)left : tile_v;
      const uint4* a = reinterpret_cast<const uint4*>(static_cast<const char*>(seg[k].src) + seg[k].head) + first;
      uint4* o = reinterpret_cast<uint4*>(static_cast<char*>(seg[k].dst) + seg[k].head) + first;
      uint4 va[U];
      if (n_here == tile_v) {
#pragma unroll
        for (int u = 0; u < U; u++) va[u] = __ldcg(a + threadIdx.x + u * THREADS);
#pragma unroll
        for (int u = 0; u < U; u++) o[threadIdx.x + u * THREADS] = va[u];
      } else {
        for (unsigned i = threadIdx.x; i < n_here; i += THREADS) o[i] = __ldcg(a + i);
      }
    }
  }
  {
    const unsigned long long total = (unsigned long long)gridDim.x * THREADS;
    const unsigned long long S = seg[nseg - 1].scalars_end;
    int k = 0;
    for (unsigned long long j = (unsigned long long)blockIdx.x * THREADS + threadIdx.x; j < S; j += total) {
      while (j >= seg[k].scalars_end) k++;
      unsigned long long i = j - (k ? seg[k - 1].scalars_end : 0ull);
      if (i >= seg[k].head) i += seg[k].nvec * 16;
      static_cast<unsigned char*>(seg[k].dst)[i] = __ldcg(static_cast<const unsigned char*>(seg[k].src) + i);
    }
  }
}

template <int DT, int THREADS, int NPH, int NSEG>
__global__ void __launch_bounds__(THREADS, 1) ring_kernel(const __grid_constant__ RingArgsT<NPH, NSEG> a) {
  __shared__ int s_bail;
  if (threadIdx.x == 0) s_bail = 0;
  unsigned nbar = 0;
  for (int ph = 0; ph < a.nphase; ph++) {
    const RingPhase P = a.phase[ph];
    if (P.barrier_before) {
      nbar++;
      if (!grid_barrier(a.bar, nbar * (gridDim.x + (unsigned)a.missing_arrivals), a.host_err, &s_bail)) break;
    }
    if (P.kind == 1) sum_phase<DT, 4, THREADS>(a.seg + P.first_seg, P.nseg);
    else copy_phase<(THREADS == 1024 ? 8 : 4), THREADS>(a.seg + P.first_seg, P.nseg);
  }
  // leave: the last CTA out clears the barrier words, so that the next launch starts from zero even after a give-up
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned gone = atomicAdd(&a.bar[1], 1u);
    if (gone == gridDim.x - 1) {
      a.bar[0] = 0;
      a.bar[2] = 0;
      __threadfence();
      a.bar[1] = 0;
    }
  }
}

template <int NPH, int NSEG>
const void* ring_entry(int dtype, int threads) {
  if (threads == 1024)
    return dtype == 0 ? reinterpret_cast<const void*>(&ring_kernel<0, 1024, NPH, NSEG>) : reinterpret_cast<const void*>(&ring_kernel<1, 1024, NPH, NSEG>);
  return dtype == 0 ? reinterpret_cast<const void*>(&ring_kernel<0, 512, NPH, NSEG>) : reinterpret_cast<const void*>(&ring_kernel<1, 512, NPH, NSEG>);
}

template <int NPH, int NSEG>
cudaError_t launch_ring_t(const RingArgsT<NPH, NSEG>& a, int grid, int threads, cudaStream_t stream) {
  if (a.nphase <= 0) return cudaSuccess;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  void* args[] = {const_cast<RingArgsT<NPH, NSEG>*>(&a)};
  return cudaLaunchKernelExC(&cfg, ring_entry<NPH, NSEG>(a.dtype, threads), args);
}

}  // namespace

cudaError_t launch_ring(const RingArgsSmall& a, int grid, int threads, cudaStream_t stream) { return launch_ring_t(a, grid, threads, stream); }
cudaError_t launch_ring(const RingArgsLarge& a, int grid, int threads, cudaStream_t stream) { return launch_ring_t(a, grid, threads, stream); }

void prepare_ring_phase(RingSeg* seg, int nseg, int kind, int dtype, int threads) {
  const int E = kind == 1 ? (dtype == 0 ? 4 : 2) : 1, VE = 16 / E;
  const unsigned long long tile_v = (unsigned long long)threads * (kind == 1 ? 4 : (threads == 1024 ? 8 : 4));
  unsigned long long tiles = 0, scalars = 0;
  for (int k = 0; k < nseg; k++) {
    RingSeg& s = seg[k];
    const unsigned ms = (unsigned)((uintptr_t)s.src & 15), md = (unsigned)((uintptr_t)s.dst & 15);
    const bool congruent = kind == 1 ? (ms == md && ms == (unsigned)((uintptr_t)s.local & 15)) : (ms == md);
    unsigned long long nv, ns;
    unsigned h;
    split_segment(s.bytes / E, ms, congruent, E, VE, &h, &nv, &ns);
    s.head = h;
    s.nvec = nv;
    s.pad = 0;
    tiles += (nv + tile_v - 1) / tile_v;
    scalars += ns;
    s.tiles_end = tiles;
    s.scalars_end = scalars;
  }
}

cudaError_t ring_max_grid(int threads, int dtype, bool large, int num_sms, int* grid) {
  int per_sm = 0;
  const void* fn = large ? ring_entry<kRingLargePhases, kRingLargeSegs>(dtype, threads) : ring_entry<kRingSmallPhases, kRingSmallSegs>(dtype, threads);
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, 0);
  if (e != cudaSuccess) return e;
  *grid = per_sm * num_sms;
  return cudaSuccess;
}

cudaError_t preload_ring_kernels() {
  for (int dtype = 0; dtype < 2; dtype++)
    for (int threads : {512, 1024})
      for (int large = 0; large < 2; large++) {
        cudaFuncAttributes at;
        const void* fn = large ? ring_entry<kRingLargePhases, kRingLargeSegs>(dtype, threads) : ring_entry<kRingSmallPhases, kRingSmallSegs>(dtype, threads);
        cudaError_t e = cudaFuncGetAttributes(&at, fn);
        if (e != cudaSuccess) return e;
      }
  return cudaSuccess;
}

}  // namespace hoccl
