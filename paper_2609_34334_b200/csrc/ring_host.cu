// Host side of the whole-collective kernel ("fused" setting of the SM path): control words, the parameter block built
// from a resolved plan, and the self-test of the bounded barrier wait.  The kernel itself is in ring.cu.
#include "comm.h"

namespace hoccl {

// The barrier words and the error word of the "fused" setting are the library's own (16 bytes of device memory and
// 4 bytes of mapped pinned host memory), allocated on first use.
static hoccl_result_t ensure_ring_ctrl(hoccl_comm* c) {
  if (c->ring_bar) return HOCCL_OK;
  unsigned* bar = nullptr;
  int* err = nullptr;
  int* err_dev = nullptr;
  CU_TRY(c, cudaMalloc(&bar, 16));
  cudaError_t e = cudaMemset(bar, 0, 16);
  if (e == cudaSuccess) e = cudaHostAlloc(&err, sizeof(int), cudaHostAllocMapped);
  if (e == cudaSuccess) {
    *err = 0;
    e = cudaHostGetDevicePointer(&err_dev, err, 0);
  }
  if (e == cudaSuccess) e = preload_ring_kernels();
  if (e != cudaSuccess) {
    cudaFree(bar);
    if (err) cudaFreeHost(err);
    return cuda_fail(c, e, "ring kernel control words");
  }
  c->ring_bar = bar;
  c->ring_err = err;
  c->ring_err_dev = err_dev;
  return HOCCL_OK;
}

template <typename Args, int NPH, int NSEG>
static bool fill_ring_args(const std::vector<RGroup>& groups, int dtype, int threads, unsigned* bar, int* err_dev, Args* a,
                           size_t* max_phase_bytes) {
  int nph = 0, nseg = 0;
  *max_phase_bytes = 0;
  a->dtype = dtype;
  a->bar = bar;
  a->host_err = err_dev;
  for (const RGroup& g : groups) {
    bool first_of_group = true;
    for (size_t first = 0; first < g.segs.size(); first += kMaxSegs) {
      const size_t n = std::min<size_t>(kMaxSegs, g.segs.size() - first);
      if (nph >= NPH || nseg + (int)n > NSEG) return false;
      RingPhase& ph = a->phase[nph++];
      ph.first_seg = nseg;
      ph.nseg = (int)n;
      ph.kind = g.kind == OP_SUM ? 1 : 0;
      ph.barrier_before = (first_of_group && !g.deps.empty()) ? 1 : 0;
      first_of_group = false;
      size_t bytes = 0;
      for (size_t i = 0; i < n; i++) {
        const Seg& sg = g.segs[first + i];
        RingSeg rs = {};
        rs.src = sg.src;
        rs.local = g.kind == OP_SUM ? sg.local : nullptr;
        rs.dst = sg.dst;
        rs.bytes = (unsigned long long)sg.bytes;
        a->seg[nseg++] = rs;
        bytes += sg.bytes;
      }
      prepare_ring_phase(a->seg + ph.first_seg, ph.nseg, ph.kind, dtype, threads);
      *max_phase_bytes = std::max(*max_phase_bytes, bytes);
    }
  }
  a->nphase = nph;
  return true;
}

// Turns the resolved plan into the parameter block of one ring_kernel launch.  UNSUPPORTED if the plan does not fit
// into the kernel's parameter space (very many ranks): the caller then falls back to the graph.
hoccl_result_t build_ring(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry) {
  hoccl_result_t rc = ensure_ring_ctrl(c);
  if (rc != HOCCL_OK) return rc;
  size_t max_phase_bytes = 0;
  bool has_sum = false;
  for (const RGroup& g : groups) {
    if (g.kind == OP_CHAIN) return HOCCL_ERR_UNSUPPORTED;   // the ring kernel walks ring steps only
    has_sum = has_sum || g.kind == OP_SUM;
  }
  // CTA budget: never more than either budget of the SM path; never more CTAs than the largest phase has tiles for
  // (a barrier costs more the more CTAs take part); never more than can be resident together.
  long budget = has_sum ? std::min(c->sum_ctas, c->copy_ctas) : c->copy_ctas;
  const int threads = budget >= 128 ? 512 : 1024;
  entry->ring_args.assign(sizeof(RingArgsSmall), 0);
  entry->ring_large = false;
  if (!fill_ring_args<RingArgsSmall, kRingSmallPhases, kRingSmallSegs>(groups, P.dtype, threads, c->ring_bar, c->ring_err_dev,
                                                                     reinterpret_cast<RingArgsSmall*>(entry->ring_args.data()), &max_phase_bytes)) {
    entry->ring_args.assign(sizeof(RingArgsLarge), 0);
    entry->ring_large = true;
    if (!fill_ring_args<RingArgsLarge, kRingLargePhases, kRingLargeSegs>(groups, P.dtype, threads, c->ring_bar, c->ring_err_dev,
                                                                       reinterpret_cast<RingArgsLarge*>(entry->ring_args.data()), &max_phase_bytes)) {
      entry->ring_args.clear();
      return HOCCL_ERR_UNSUPPORTED;
    }
  }
  const size_t tile_bytes = (size_t)threads * 4 * 16;
  const long tiles = (long)((max_phase_bytes + tile_bytes - 1) / tile_bytes);
  int max_grid = 0;
  CU_TRY(c, ring_max_grid(threads, P.dtype, entry->ring_large, c->num_sms, &max_grid));
  long grid = std::max<long>(1, std::min<long>(std::min<long>(budget, tiles), max_grid));
  entry->ring_grid = (int)grid;
  entry->ring_threads = threads;
  entry->ring_has_sum = has_sum;
  entry->n_moves = 0;
  for (const RGroup& g : groups)
    if (g.kind != OP_SUM) entry->n_moves += (long)g.segs.size();
  entry->n_move_launches = 1;   // the one launch of the collective
  entry->n_sum_launches = 0;
  return HOCCL_OK;
}

// Self-test of the bounded barrier wait: two copy phases with a barrier between them that waits for one arrival more
// than the grid can deliver.  The kernel must give up by itself, report it, and leave the barrier words clean.
hoccl_result_t ring_barrier_selftest(hoccl_comm* c, void* dst, const void* src, size_t bytes, cudaStream_t stream) {
  hoccl_result_t rc = ensure_ring_ctrl(c);
  if (rc != HOCCL_OK) return rc;
  std::vector<char> store(sizeof(RingArgsSmall), 0);
  RingArgsSmall* a = reinterpret_cast<RingArgsSmall*>(store.data());
  a->nphase = 2;
  a->dtype = 0;
  a->missing_arrivals = 1;
  a->bar = c->ring_bar;
  a->host_err = c->ring_err_dev;
  const size_t half = bytes / 2;
  for (int ph = 0; ph < 2; ph++) {
    a->phase[ph] = RingPhase{ph, 1, 0, ph};   // phase 1 sits behind the barrier and must never run
    RingSeg rs = {};
    rs.src = (const char*)src + ph * half;
    rs.dst = (char*)dst + ph * half;
    rs.bytes = half;
    a->seg[ph] = rs;
    prepare_ring_phase(a->seg + ph, 1, 0, 0, 1024);
  }
  CU_TRY(c, launch_ring(*a, 4, 1024, stream));
  return HOCCL_OK;
}

}  // namespace hoccl
