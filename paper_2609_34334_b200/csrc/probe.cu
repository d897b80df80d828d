// Diagnostics that answer one question by measurement: does a given way of moving bytes need an SM?
//
// The paper's premise (Sec. 2.3 "DMA Engines") is that copy-engine transfers occupy no SM.  Whether a copy INSIDE one
// device is given to a copy engine is the driver's decision, so the library measures it: a kernel that takes every
// thread slot of every SM sleeps for a fixed time (bounded by the global timer, it waits on nothing) while the move
// is enqueued on another stream.  A move that ends while that kernel is still resident used no SM.
#include <cuda.h>

#include <functional>

#include "comm.h"

namespace hoccl {

namespace {

struct Occupied {
  int needs_sm = 0;
  double end_us = 0;
};

// Runs `enqueue(stream)` while all SMs are taken for spin_us; the enqueued work must complete on `stream`.
hoccl_result_t measure_under_occupancy(hoccl_comm* c, int spin_us, const std::function<cudaError_t(cudaStream_t)>& enqueue, Occupied* out) {
  CU_TRY(c, cudaDeviceSynchronize());
  cudaEvent_t a0, a1, b1;
  CU_TRY(c, cudaEventCreate(&a0));
  CU_TRY(c, cudaEventCreate(&a1));
  CU_TRY(c, cudaEventCreate(&b1));
  hoccl_result_t rc = HOCCL_OK;
  cudaError_t e = cudaEventRecord(a0, c->lane[0]);
  int ctas = 0;
  if (e == cudaSuccess) e = launch_occupy_all_sms((unsigned long long)spin_us * 1000ull, c->num_sms, c->lane[0], &ctas);
  if (e == cudaSuccess) e = cudaEventRecord(a1, c->lane[0]);
  // let the occupying kernel become resident before the move is enqueued
  const double t0 = now_us();
  while (now_us() - t0 < std::min(300.0, spin_us * 0.25)) {
  }
  cudaError_t move_err = cudaSuccess;
  if (e == cudaSuccess) move_err = enqueue(c->lane[1]);
  if (e == cudaSuccess) e = cudaEventRecord(b1, c->lane[1]);
  cudaError_t se = cudaDeviceSynchronize();   // always drain the occupancy kernel, also after a failed enqueue
  if (e == cudaSuccess) e = se;
  if (e == cudaSuccess) e = move_err;
  float spin_ms = 0, end_ms = 0;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&spin_ms, a0, a1);
  if (e == cudaSuccess) e = cudaEventElapsedTime(&end_ms, a0, b1);
  if (e != cudaSuccess) {
    rc = cuda_fail(c, e, "move under full occupancy");
    (void)cudaGetLastError();
  } else {
    out->needs_sm = end_ms >= 0.9f * spin_ms ? 1 : 0;
    out->end_us = end_ms * 1e3;
  }
  cudaEventDestroy(a0);
  cudaEventDestroy(a1);
  cudaEventDestroy(b1);
  return rc;
}

template <typename Fn>
Fn driver_entry(const char* name) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qr;
  if (cudaGetDriverEntryPoint(name, &fn, cudaEnableDefault, &qr) != cudaSuccess || qr != cudaDriverEntryPointSuccess) return nullptr;
  return reinterpret_cast<Fn>(fn);
}

}  // namespace
}  // namespace hoccl

using namespace hoccl;

extern "C" {

hoccl_result_t hoccl_probe_move_needs_sm(hoccl_comm_t c, hoccl_path_t path, void* dst, const void* src, size_t bytes, int spin_us,
                                         int* needs_sm, double* move_end_us) {
  if (!c || !dst || !src || !needs_sm || bytes == 0 || spin_us < 100 || spin_us > 20000) return HOCCL_ERR_INVALID_ARG;
  if (path == HOCCL_PATH_CE_HOST && (!c->host_staging || bytes > c->host_staging_bytes)) return HOCCL_ERR_SCRATCH;
  CU_TRY(c, cudaSetDevice(c->device));
  Occupied r;
  hoccl_result_t rc = measure_under_occupancy(c, spin_us, [&](cudaStream_t s) -> cudaError_t {
    if (path == HOCCL_PATH_CE) return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, s);  // src may be pinned host memory (control)
    if (path == HOCCL_PATH_CE_HOST) {
      cudaError_t e = cudaMemcpyAsync(c->host_staging, src, bytes, cudaMemcpyDeviceToHost, s);
      if (e == cudaSuccess) e = cudaMemcpyAsync(dst, c->host_staging, bytes, cudaMemcpyHostToDevice, s);
      return e;
    }
    CopyBatch b;
    b.nseg = 1;
    b.pad = 0;
    b.seg[0] = CopySeg{src, dst, (unsigned long long)bytes};
    return launch_copy(b, (int)c->copy_ctas, s);
  }, &r);
  if (rc != HOCCL_OK) return rc;
  *needs_sm = r.needs_sm;
  if (move_end_us) *move_end_us = r.end_us;
  return HOCCL_OK;
}

hoccl_result_t hoccl_probe_copy_routes(hoccl_comm_t c, void* dst, const void* src, size_t bytes, int spin_us, hoccl_route_probe_t* out,
                                       int max_out, int* n_out) {
  if (!c || !dst || !src || !out || !n_out || max_out < 1 || bytes < 4 || spin_us < 100 || spin_us > 20000) return HOCCL_ERR_INVALID_ARG;
  CU_TRY(c, cudaSetDevice(c->device));
  const int dev = c->device;
  typedef CUresult (*dtod_fn)(CUdeviceptr, CUdeviceptr, size_t, CUstream);
  typedef CUresult (*write32_fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
  dtod_fn dtod = driver_entry<dtod_fn>("cuMemcpyDtoDAsync");
  write32_fn write32 = driver_entry<write32_fn>("cuStreamWriteValue32");
  // a one-node memcpy graph, instantiated before the measurement
  cudaGraphExec_t gexec = nullptr;
  {
    cudaGraph_t g = nullptr;
    cudaGraphNode_t n;
    if (cudaGraphCreate(&g, 0) == cudaSuccess) {
      if (cudaGraphAddMemcpyNode1D(&n, g, nullptr, 0, dst, src, bytes, cudaMemcpyDeviceToDevice) == cudaSuccess)
        (void)cudaGraphInstantiate(&gexec, g, 0);
      cudaGraphDestroy(g);
    }
    (void)cudaGetLastError();
  }
  // first device access to freshly pinned pages is slow (measured: +2 ms for 16 MiB); touch them once, untimed
  if (c->host_staging && c->host_staging_bytes >= bytes) {
    CU_TRY(c, cudaMemcpyAsync(c->host_staging, src, bytes, cudaMemcpyDeviceToHost, c->lane[1]));
    CU_TRY(c, cudaMemcpyAsync(dst, c->host_staging, bytes, cudaMemcpyHostToDevice, c->lane[1]));
    CU_TRY(c, cudaStreamSynchronize(c->lane[1]));
  }
  const size_t pitch = 4096;
  struct Route {
    const char* name;
    bool available;
    std::function<cudaError_t(cudaStream_t)> fn;
  };
  const Route routes[] = {
      {"cudaMemcpyAsync device->device", true, [&](cudaStream_t s) { return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, s); }},
      {"cudaMemcpyPeerAsync (same device)", true, [&](cudaStream_t s) { return cudaMemcpyPeerAsync(dst, dev, src, dev, bytes, s); }},
      {"cuMemcpyDtoDAsync", dtod != nullptr,
       [&](cudaStream_t s) { return dtod((CUdeviceptr)(uintptr_t)dst, (CUdeviceptr)(uintptr_t)src, bytes, (CUstream)s) == CUDA_SUCCESS ? cudaSuccess : cudaErrorUnknown; }},
      {"memcpy node of a CUDA graph", gexec != nullptr, [&](cudaStream_t s) { return cudaGraphLaunch(gexec, s); }},
      {"cudaMemcpy2DAsync device->device", bytes >= pitch,
       [&](cudaStream_t s) { return cudaMemcpy2DAsync(dst, pitch, src, pitch, pitch, bytes / pitch, cudaMemcpyDeviceToDevice, s); }},
      {"cudaMemsetAsync", true, [&](cudaStream_t s) { return cudaMemsetAsync(dst, 0, bytes, s); }},
      {"copy_kernel (this library, by construction)", true,
       [&](cudaStream_t s) {
         CopyBatch b;
         b.nseg = 1;
         b.pad = 0;
         b.seg[0] = CopySeg{src, dst, (unsigned long long)bytes};
         return launch_copy(b, (int)c->copy_ctas, s);
       }},
      {"control: cuStreamWriteValue32", write32 != nullptr,
       [&](cudaStream_t s) { return write32((CUstream)s, (CUdeviceptr)(uintptr_t)dst, 1u, 0u) == CUDA_SUCCESS ? cudaSuccess : cudaErrorUnknown; }},
      {"control: device->pinned host", c->host_staging && c->host_staging_bytes >= bytes,
       [&](cudaStream_t s) { return cudaMemcpyAsync(c->host_staging, src, bytes, cudaMemcpyDeviceToHost, s); }},
      {"control: pinned host->device", c->host_staging && c->host_staging_bytes >= bytes,
       [&](cudaStream_t s) { return cudaMemcpyAsync(dst, c->host_staging, bytes, cudaMemcpyHostToDevice, s); }},
  };
  int n = 0;
  hoccl_result_t rc = HOCCL_OK;
  for (const Route& r : routes) {
    if (n >= max_out) break;
    if (!r.available) continue;
    Occupied o;
    rc = measure_under_occupancy(c, spin_us, r.fn, &o);
    if (rc != HOCCL_OK) break;
    hoccl_route_probe_t* dstp = &out[n++];
    std::memset(dstp, 0, sizeof(*dstp));
    std::strncpy(dstp->name, r.name, sizeof(dstp->name) - 1);
    dstp->needs_sm = o.needs_sm;
    dstp->end_us = o.end_us;
  }
  if (gexec) cudaGraphExecDestroy(gexec);
  *n_out = n;
  return rc;
}

}  // extern "C"
