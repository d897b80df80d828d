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

// Prefix sums over the (at most 32) segments of a phase by the first warp: tile counts and element-wise item counts.
// Every thread of the CTA calls it; lanes >= nseg contribute zero.  Ends with the CTA barrier that publishes the view.
__device__ __forceinline__ void flatten_prefix(Flat& f, int nseg, unsigned long long my_tiles, unsigned long long my_scalars) {
  if (threadIdx.x < 32) {
    unsigned long long t = my_tiles, s = my_scalars;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned long long tu = __shfl_up_sync(0xffffffffu, t, d), su = __shfl_up_sync(0xffffffffu, s, d);
      if ((int)threadIdx.x >= d) {
        t += tu;
        s += su;
      }
    }
    if (threadIdx.x == 0) {
      f.tpre[0] = 0;
      f.spre[0] = 0;
    }
    if ((int)threadIdx.x < nseg) {
      f.tpre[threadIdx.x + 1] = t;
      f.spre[threadIdx.x + 1] = s;
    }
  }
  __syncthreads();
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

template <int DT, int U, int THREADS>
__device__ __forceinline__ void sum_phase(Flat& f, const RingSeg* seg, int nseg) {
  using T = Traits<DT>;
  unsigned long long my_tiles = 0, my_scalars = 0;
  if ((int)threadIdx.x < nseg) {
    const RingSeg& s = seg[threadIdx.x];
    unsigned ma = (unsigned)((uintptr_t)s.src & 15), mb = (unsigned)((uintptr_t)s.local & 15), mo = (unsigned)((uintptr_t)s.dst & 15);
    unsigned long long nv, ns;
    unsigned h;
    split_segment(s.bytes / T::E, ma, ma == mb && mb == mo, T::E, T::VE, &h, &nv, &ns);
    f.head[threadIdx.x] = h;
    f.nvec[threadIdx.x] = nv;
    my_tiles = (nv + (unsigned long long)U * THREADS - 1) / ((unsigned long long)U * THREADS);   // a shift
    my_scalars = ns;
  }
  flatten_prefix(f, nseg, my_tiles, my_scalars);
  {
    const unsigned long long T_all = f.tpre[nseg];
    const unsigned tile_v = U * blockDim.x;
    int k = 0;
    for (unsigned long long t = blockIdx.x; t < T_all; t += gridDim.x) {
      while (t >= f.tpre[k + 1]) k++;
      const unsigned long long first = (t - f.tpre[k]) * tile_v;
      const unsigned long long left = f.nvec[k] - first;
      const unsigned n_here = left < tile_v ? (unsigned)left : tile_v;
      const size_t h = (size_t)f.head[k] * T::E;
      const uint4* a = reinterpret_cast<const uint4*>(static_cast<const char*>(seg[k].src) + h) + first;
      const uint4* b = reinterpret_cast<const uint4*>(static_cast<const char*>(seg[k].local) + h) + first;
      uint4* o = reinterpret_cast<uint4*>(static_cast<char*>(seg[k].dst) + h) + first;
      uint4 va[U], vb[U];
      if (n_here == tile_v) {
#pragma unroll
        for (int u = 0; u < U; u++) {
          va[u] = __ldcg(a + threadIdx.x + u * blockDim.x);
          vb[u] = __ldcg(b + threadIdx.x + u * blockDim.x);
        }
#pragma unroll
        for (int u = 0; u < U; u++) o[threadIdx.x + u * blockDim.x] = T::add_vec(va[u], vb[u]);
      } else {
        for (unsigned i = threadIdx.x; i < n_here; i += blockDim.x) o[i] = T::add_vec(__ldcg(a + i), __ldcg(b + i));
      }
    }
  }
  {
    const unsigned long long total = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long S = f.spre[nseg];
    int k = 0;
    for (unsigned long long j = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; j < S; j += total) {
      while (j >= f.spre[k + 1]) k++;
      unsigned long long i = j - f.spre[k];
      if (i >= f.head[k]) i += f.nvec[k] * T::VE;
      add_scalar_cg<DT>(seg[k].src, seg[k].local, seg[k].dst, i);
    }
  }
}

template <int U, int THREADS>
__device__ __forceinline__ void copy_phase(Flat& f, const RingSeg* seg, int nseg) {
  unsigned long long my_tiles = 0, my_scalars = 0;
  if ((int)threadIdx.x < nseg) {
    const RingSeg& s = seg[threadIdx.x];
    unsigned ms = (unsigned)((uintptr_t)s.src & 15), md = (unsigned)((uintptr_t)s.dst & 15);
    unsigned long long nv, ns;
    unsigned h;
    split_segment(s.bytes, ms, ms == md, 1, 16, &h, &nv, &ns);
    f.head[threadIdx.x] = h;
    f.nvec[threadIdx.x] = nv;
    my_tiles = (nv + (unsigned long long)U * THREADS - 1) / ((unsigned long long)U * THREADS);   // a shift
    my_scalars = ns;
  }
  flatten_prefix(f, nseg, my_tiles, my_scalars);
  {
    const unsigned long long T_all = f.tpre[nseg];
    const unsigned tile_v = U * blockDim.x;
    int k = 0;
    for (unsigned long long t = blockIdx.x; t < T_all; t += gridDim.x) {
      while (t >= f.tpre[k + 1]) k++;
      const unsigned long long first = (t - f.tpre[k]) * tile_v;
      const unsigned long long left = f.nvec[k] - first;
      const unsigned n_here = left < tile_v ? (unsigned)left : tile_v;
      const uint4* a = reinterpret_cast<const uint4*>(static_cast<const char*>(seg[k].src) + f.head[k]) + first;
      uint4* o = reinterpret_cast<uint4*>(static_cast<char*>(seg[k].dst) + f.head[k]) + first;
      uint4 va[U];
      if (n_here == tile_v) {
#pragma unroll
        for (int u = 0; u < U; u++) va[u] = __ldcg(a + threadIdx.x + u * blockDim.x);
#pragma unroll
        for (int u = 0; u < U; u++) o[threadIdx.x + u * blockDim.x] = va[u];
      } else {
        for (unsigned i = threadIdx.x; i < n_here; i += blockDim.x) o[i] = __ldcg(a + i);
      }
    }
  }
  {
    const unsigned long long total = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long S = f.spre[nseg];
    int k = 0;
    for (unsigned long long j = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; j < S; j += total) {
      while (j >= f.spre[k + 1]) k++;
      unsigned long long i = j - f.spre[k];
      if (i >= f.head[k]) i += f.nvec[k] * 16;
      static_cast<unsigned char*>(seg[k].dst)[i] = __ldcg(static_cast<const unsigned char*>(seg[k].src) + i);
    }
  }
}

template <int DT, int THREADS, int NPH, int NSEG>
__global__ void __launch_bounds__(THREADS, 1) ring_kernel(const __grid_constant__ RingArgsT<NPH, NSEG> a) {
  __shared__ Flat f;
  __shared__ int s_bail;
  if (threadIdx.x == 0) s_bail = 0;
  unsigned nbar = 0;
  bool ok = true;
  for (int ph = 0; ph < a.nphase && ok; ph++) {
    const RingPhase P = a.phase[ph];
    if (P.barrier_before) {
      nbar++;
      ok = grid_barrier(a.bar, nbar * gridDim.x, a.host_err, &s_bail);
      if (!ok) break;
    } else {
      __syncthreads();   // the flattened view of the previous phase is about to be overwritten
    }
    if (P.kind == 1) sum_phase<DT, 4, THREADS>(f, a.seg + P.first_seg, P.nseg);
    else copy_phase<(THREADS == 1024 ? 8 : 4), THREADS>(f, a.seg + P.first_seg, P.nseg);
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
