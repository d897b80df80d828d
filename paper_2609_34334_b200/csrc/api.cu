// The C ABI declared in include/hoccl.h: communicator life cycle, parameters, collectives, send/recv, the user-defined
// pattern executor, diagnostics, and the host-only planner / scheduler inspection calls.
#include "comm.h"
#include "options.h"
#include "../../include/hoccl_diag.h"

using namespace hoccl;

extern "C" {

hoccl_result_t hoccl_comm_init(hoccl_comm_t* comm, int R, int device) {
  if (!comm || R < 1 || R > kMaxRanks) return HOCCL_ERR_INVALID_ARG;
  *comm = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
    cudaGetLastError();
    return HOCCL_ERR_CUDA;
  }
  hoccl_comm* c = new hoccl_comm();
  c->R = R;
  c->device = device;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, device);
  for (int i = 0; i < kMaxLanes && e == cudaSuccess; i++) e = cudaStreamCreateWithFlags(&c->lane[i], cudaStreamNonBlocking);
  // SUM launches get the highest priority: a SUM CTA needs a whole SM (1024 threads x 64 registers), and when a
  // SUM and the next piece's copies become ready at the same moment the copies' small CTAs would otherwise take
  // every SM first and the SUM would start only after them, which serialises the pipeline.
  int prio_least = 0, prio_greatest = 0;
  if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest);
  c->sum_priority = prio_greatest;
  if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&c->sum_stream, cudaStreamNonBlocking, prio_greatest);
  if (e != cudaSuccess) {
    for (int i = 0; i < kMaxLanes; i++)
      if (c->lane[i]) cudaStreamDestroy(c->lane[i]);
    if (c->sum_stream) cudaStreamDestroy(c->sum_stream);
    delete c;
    return HOCCL_ERR_CUDA;
  }
  *comm = c;
  return HOCCL_OK;
}

hoccl_result_t hoccl_comm_destroy(hoccl_comm_t c) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (c->n_pending > 0) return HOCCL_ERR_PENDING;
  bool forced = false;
  if (c->proxy) {
    const bool drained = c->proxy->drain(c->watchdog_ms);
    if (c->proxy->pending_p2p() > 0) return HOCCL_ERR_PENDING;
    // Hand-overs that are still open (a stream that has not reached its post yet, work that has not finished) are
    // released by the proxy on its way out, so no stream keeps waiting on a communicator that is gone; if a stream could
    // not be seen past its hand-over in time, the flag memory outlives the proxy (see Proxy::shutdown).
    const bool passed = c->proxy->shutdown(2 * c->watchdog_ms + 100);
    forced = !drained || !passed;
    delete c->proxy;
    c->proxy = nullptr;
  }
  cudaSetDevice(c->device);
  for (int i = 0; i < kMaxLanes; i++)
    if (c->lane[i]) {
      cudaStreamSynchronize(c->lane[i]);
      cudaStreamDestroy(c->lane[i]);
    }
  if (c->sum_stream) {
    cudaStreamSynchronize(c->sum_stream);
    cudaStreamDestroy(c->sum_stream);
  }
  for (auto& e : c->cache) destroy_entry(&e);
  if (c->ring_bar) cudaFree(c->ring_bar);
  if (c->ring_err) cudaFreeHost(c->ring_err);
  if (c->roles_ctl) cudaFree(c->roles_ctl);
  if (c->roles_err) cudaFreeHost(c->roles_err);
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : c->post_events) cudaEventDestroy(e);
  for (auto& p : c->prof_pool) {
    cudaEventDestroy(p.first);
    cudaEventDestroy(p.second);
  }
  for (auto& p : c->prof_open) {
    cudaEventDestroy(p.first.first);
    cudaEventDestroy(p.first.second);
  }
  delete c;
  return forced ? HOCCL_ERR_TIMEOUT : HOCCL_OK;
}

size_t hoccl_scratch_bytes(int R, size_t max_count, hoccl_dtype_t dtype) {
  size_t e = dtype_size((int)dtype);
  if (R <= 1 || e == 0 || max_count == 0) return 0;
  return 2 * (size_t)R * slot_bytes_for(R, max_count, e);
}

size_t hoccl_scratch_bytes_direct(int R, size_t max_count, hoccl_dtype_t dtype) {
  size_t e = dtype_size((int)dtype);
  if (R <= 1 || e == 0 || max_count == 0) return 0;
  return (size_t)std::max(2, R - 1) * (size_t)R * slot_bytes_for(R, max_count, e);
}

hoccl_result_t hoccl_comm_set_scratch(hoccl_comm_t c, void* dev_ptr, size_t bytes) {
  if (!c || ((uintptr_t)dev_ptr & 255)) return HOCCL_ERR_INVALID_ARG;
  c->scratch = dev_ptr;
  c->scratch_bytes = dev_ptr ? bytes : 0;
  return HOCCL_OK;
}

hoccl_result_t hoccl_comm_set_staging(hoccl_comm_t c, void* dev_ptr, size_t bytes) {
  if (!c || ((uintptr_t)dev_ptr & 255)) return HOCCL_ERR_INVALID_ARG;
  c->staging = dev_ptr;
  c->staging_bytes = dev_ptr ? bytes : 0;
  return HOCCL_OK;
}

hoccl_result_t hoccl_comm_set_host_staging(hoccl_comm_t c, void* pinned_host_ptr, size_t bytes) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (pinned_host_ptr) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, pinned_host_ptr) != cudaSuccess || attr.type != cudaMemoryTypeHost) {
      cudaGetLastError();
      return HOCCL_ERR_INVALID_ARG;   // pageable memory would turn the copies into staged, synchronous ones
    }
  }
  c->host_staging = static_cast<char*>(pinned_host_ptr);
  c->host_staging_bytes = pinned_host_ptr ? bytes : 0;
  return HOCCL_OK;
}

hoccl_result_t hoccl_comm_set_path(hoccl_comm_t c, hoccl_path_t path) {
  if (!c || (path != HOCCL_PATH_CE && path != HOCCL_PATH_SM && path != HOCCL_PATH_CE_HOST)) return HOCCL_ERR_INVALID_ARG;
  c->path = path;
  return HOCCL_OK;
}

static long* param_slot(hoccl_comm* c, const char* key, long* lo, long* hi) {
  struct Row {
    const char* name;
    long* p;
    long lo, hi;
  } rows[] = {{"sum_ctas", &c->sum_ctas, 1, 1024},      {"copy_ctas", &c->copy_ctas, 1, 1024},
              {"piece_bytes", &c->piece_bytes, 1024, 1L << 40}, {"max_pieces", &c->max_pieces, 1, 4096},
              {"lanes", &c->lanes, 1, kMaxLanes},       {"use_graph", &c->use_graph, 0, 1},
              {"profile", &c->profile, 0, 1},           {"p2p_split", &c->p2p_split, 1, kMaxLanes},
              {"ce_sub_bytes", &c->ce_sub_bytes, 0, 1L << 40}, {"handshake", &c->handshake, 0, 1},
              {"watchdog_ms", &c->watchdog_ms, 10, 600000},    {"onepass", &c->onepass, 0, 1},
              {"forward", &c->forward, 0, 1},           {"fused", &c->fused, 0, 1},
              {"ag_direct", &c->ag_direct, 0, 2},
              {"order_kernels", &c->order_kernels, 0, 1},
              {"rs_direct", &c->rs_direct, 0, 2},
              {"ce_small_bytes", &c->ce_small_bytes, 0, 1L << 40},
              {"ce_small_ctas", &c->ce_small_ctas, 1, 1024},
              {"p2p_strict", &c->p2p_strict, 0, 1},
              {"roles", &c->roles, 0, 1},
              {"piece_grade", &c->piece_grade, -1, 1},
              {"ce_overlap", &c->ce_overlap, -1, 64},
              {"model_gpus_per_node", &c->model_gpus_per_node, 0, kMaxRanks},
              {"model_rdma_sub_bytes", &c->model_rdma_sub_bytes, 0, 1L << 40},
              {"host_pieces", &c->host_pieces, 1, 64}};
  for (auto& r : rows)
    if (std::strcmp(r.name, key) == 0) {
      *lo = r.lo;
      *hi = r.hi;
      return r.p;
    }
  return nullptr;
}

hoccl_result_t hoccl_comm_set_param(hoccl_comm_t c, const char* key, long value) {
  if (!c || !key) return HOCCL_ERR_INVALID_ARG;
  long lo, hi;
  long* p = param_slot(c, key, &lo, &hi);
  if (!p) return HOCCL_ERR_UNSUPPORTED;
  if (value < lo || value > hi) return HOCCL_ERR_INVALID_ARG;
  if (std::strcmp(key, "piece_bytes") == 0) {
    value = (value + 1023) / 1024 * 1024;
    c->piece_bytes_set = true;
  }
  *p = value;
  return HOCCL_OK;
}

hoccl_result_t hoccl_comm_get_param(hoccl_comm_t c, const char* key, long* value) {
  if (!c || !key || !value) return HOCCL_ERR_INVALID_ARG;
  long lo, hi;
  long* p = param_slot(c, key, &lo, &hi);
  if (!p) return HOCCL_ERR_UNSUPPORTED;
  *value = *p;
  return HOCCL_OK;
}

hoccl_result_t hoccl_allreduce(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype, hoccl_op_t op,
                               hoccl_comm_t c, hoccl_stream_t stream) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (op != HOCCL_SUM) return HOCCL_ERR_UNSUPPORTED;
  size_t e = dtype_size((int)dtype);
  Call call{PLAN_ALLREDUCE, count, (int)dtype, false, count * e, count * e, send, recv};
  return run_collective(c, &call, (cudaStream_t)stream);
}

hoccl_result_t hoccl_reduce_scatter(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype, hoccl_op_t op,
                                    hoccl_comm_t c, hoccl_stream_t stream) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (op != HOCCL_SUM) return HOCCL_ERR_UNSUPPORTED;
  size_t e = dtype_size((int)dtype);
  Call call{PLAN_REDUCE_SCATTER, count, (int)dtype, false, (size_t)c->R * count * e, count * e, send, recv};
  return run_collective(c, &call, (cudaStream_t)stream);
}

hoccl_result_t hoccl_allgather(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype, hoccl_comm_t c,
                               hoccl_stream_t stream) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  size_t e = dtype_size((int)dtype);
  Call call{PLAN_ALLGATHER, count, (int)dtype, false, count * e, (size_t)c->R * count * e, send, recv};
  return run_collective(c, &call, (cudaStream_t)stream);
}

hoccl_result_t hoccl_alltoall(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype, hoccl_comm_t c,
                              hoccl_stream_t stream) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  size_t e = dtype_size((int)dtype);
  Call call{PLAN_ALLTOALL, count, (int)dtype, false, (size_t)c->R * count * e, (size_t)c->R * count * e, send, recv};
  return run_collective(c, &call, (cudaStream_t)stream);
}

hoccl_result_t hoccl_send(const void* buf, size_t count, hoccl_dtype_t dtype, int src, int dst, hoccl_comm_t c, hoccl_stream_t stream) {
  return p2p_post(c, true, const_cast<void*>(buf), count, (int)dtype, src, dst, (cudaStream_t)stream);
}

hoccl_result_t hoccl_recv(void* buf, size_t count, hoccl_dtype_t dtype, int src, int dst, hoccl_comm_t c, hoccl_stream_t stream) {
  return p2p_post(c, false, buf, count, (int)dtype, src, dst, (cudaStream_t)stream);
}

int hoccl_comm_pending(hoccl_comm_t c) {
  if (!c) return 0;
  return c->n_pending + (c->proxy ? c->proxy->pending_p2p() : 0);
}

hoccl_result_t hoccl_comm_async_error(hoccl_comm_t c, int clear) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (c->ring_err && *reinterpret_cast<volatile int*>(c->ring_err) != 0) {
    if (clear) *reinterpret_cast<volatile int*>(c->ring_err) = 0;
    return HOCCL_ERR_TIMEOUT;   // a barrier wait of the whole-collective kernel ran out
  }
  if (c->roles_err && *reinterpret_cast<volatile int*>(c->roles_err) != 0) {
    if (clear) *reinterpret_cast<volatile int*>(c->roles_err) = 0;
    return HOCCL_ERR_TIMEOUT;   // a wait of the roles kernel ran out
  }
  if (!c->proxy) return HOCCL_OK;
  int e = c->proxy->async_error();
  if (clear) c->proxy->clear_error();
  switch (e) {
    case PROXY_OK: return HOCCL_OK;
    case PROXY_TIMEOUT: return HOCCL_ERR_TIMEOUT;
    case PROXY_MISMATCH: return HOCCL_ERR_MISMATCH;
    default: return HOCCL_ERR_CUDA;
  }
}

hoccl_result_t hoccl_selftest_barrier_timeout(hoccl_comm_t c, void* dst, const void* src, size_t bytes, hoccl_stream_t stream) {
  if (!c || !dst || !src || bytes < 32 || (bytes & 31)) return HOCCL_ERR_INVALID_ARG;
  CU_TRY(c, cudaSetDevice(c->device));
  return ring_barrier_selftest(c, dst, src, bytes, (cudaStream_t)stream);
}

hoccl_result_t hoccl_selftest_roles_timeout(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype, hoccl_comm_t c,
                                            hoccl_stream_t stream) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (!c->roles) return HOCCL_ERR_UNSUPPORTED;
  c->roles_missing = 1;
  hoccl_result_t rc = hoccl_allreduce(send, recv, count, dtype, HOCCL_SUM, c, stream);
  c->roles_missing = 0;
  return rc;
}

long hoccl_comm_handshakes(hoccl_comm_t c) { return (c && c->proxy) ? c->proxy->handshakes() : 0; }

hoccl_result_t hoccl_comm_proxy_stats(hoccl_comm_t c, double* busy_us, double* span_us, int reset) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (busy_us) *busy_us = 0;
  if (span_us) *span_us = 0;
  if (!c->proxy) return HOCCL_OK;
  c->proxy->work_stats(busy_us, span_us);
  if (reset) c->proxy->reset_work_stats();
  return HOCCL_OK;
}

hoccl_result_t hoccl_host_allreduce(const void* const* h_send, void* const* h_recv, size_t count, hoccl_dtype_t dtype, hoccl_op_t op,
                                    hoccl_comm_t c, hoccl_stream_t stream) {
  if (!c || !h_send || !h_recv) return HOCCL_ERR_INVALID_ARG;
  if (op != HOCCL_SUM) return HOCCL_ERR_UNSUPPORTED;
  size_t e = dtype_size((int)dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  const int R = c->R;
  for (int r = 0; r < R; r++)
    if (!h_send[r] || !h_recv[r]) return HOCCL_ERR_INVALID_ARG;
  if (count == 0) return HOCCL_OK;
  const size_t per = (count * e + 255) / 256 * 256;
  if (!c->staging || c->staging_bytes < 2 * (size_t)R * per) return HOCCL_ERR_SCRATCH;
  CU_TRY(c, cudaSetDevice(c->device));
  cudaStream_t st = (cudaStream_t)stream;
  const void* dsend[kMaxRanks];
  void* drecv[kMaxRanks];
  for (int r = 0; r < R; r++) {
    dsend[r] = (char*)c->staging + (size_t)r * per;
    drecv[r] = (char*)c->staging + (size_t)(R + r) * per;
  }
  // Pipelined form: one graph holds, per piece of every ring chunk, the host-to-device copies, the ring on that piece and
  // the device-to-host copies, so that the three overlap across pieces (PCIe is full duplex and the ring is short).
  const bool pipelined = c->use_graph && c->host_pieces > 1 && !c->handshake && !c->onepass && c->path != HOCCL_PATH_CE_HOST &&
                         !(c->fused && c->path == HOCCL_PATH_SM);
  if (pipelined) {
    // host buffers of different ranks must not overlap each other (a receive buffer is written while others are read)
    for (int a = 0; a < R; a++)
      for (int b = 0; b < R; b++) {
        if (a < b && ranges_overlap((const char*)h_recv[a], count * e, (const char*)h_recv[b], count * e)) return HOCCL_ERR_INVALID_ARG;
        if (h_send[a] != h_recv[b] && ranges_overlap((const char*)h_send[a], count * e, (const char*)h_recv[b], count * e)) return HOCCL_ERR_INVALID_ARG;
      }
    Call call{PLAN_ALLREDUCE, count, (int)dtype, false, count * e, count * e, dsend, drecv};
    call.h_send = h_send;
    call.h_recv = h_recv;
    return run_collective(c, &call, st);
  }
  {   // a combination of settings that the all-reduce will refuse must be refused before the inbound copies are enqueued
    hoccl_result_t orc = check_options(c, PLAN_ALLREDUCE, count, (int)dtype);
    if (orc != HOCCL_OK) return orc;
  }
  for (int r = 0; r < R; r++) CU_TRY(c, cudaMemcpyAsync(const_cast<void*>(dsend[r]), h_send[r], count * e, cudaMemcpyHostToDevice, st));
  hoccl_result_t rc = hoccl_allreduce(dsend, drecv, count, dtype, op, c, stream);
  if (rc != HOCCL_OK) return rc;
  for (int r = 0; r < R; r++) CU_TRY(c, cudaMemcpyAsync(h_recv[r], drecv[r], count * e, cudaMemcpyDeviceToHost, st));
  return HOCCL_OK;
}

hoccl_result_t hoccl_alltoallv(const void* const* send, const size_t* sendcounts, const size_t* sdispls, void* const* recv,
                               const size_t* rdispls, hoccl_dtype_t dtype, hoccl_comm_t c, hoccl_stream_t stream) {
  const double t0 = now_us();
  if (!c || !send || !recv || !sendcounts || !sdispls || !rdispls) return HOCCL_ERR_INVALID_ARG;
  const size_t e = dtype_size((int)dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  if (c->handshake || c->path == HOCCL_PATH_CE_HOST) return HOCCL_ERR_UNSUPPORTED;
  const int R = c->R;
  for (int r = 0; r < R; r++) {
    if (!send[r] || !recv[r]) return HOCCL_ERR_INVALID_ARG;
    if (((uintptr_t)send[r] % e) || ((uintptr_t)recv[r] % e)) return HOCCL_ERR_INVALID_ARG;
  }
  // the flows of the user-defined pattern as the origin traffic matrix C (bytes); one NVLink domain, no RDMA
  Topology topo;
  topo.G = R;
  topo.gpus_per_node = (c->model_gpus_per_node > 0 && c->model_gpus_per_node < R) ? (int)c->model_gpus_per_node : R;
  const bool modelled = topo.gpus_per_node < R;   // more than one modelled node: forwarding copies and "RDMA" legs exist
  if (modelled && !c->use_graph) return HOCCL_ERR_UNSUPPORTED;
  std::vector<uint64_t> C((size_t)R * R);
  uint64_t total = 0;
  for (int u = 0; u < R; u++)
    for (int v = 0; v < R; v++) {
      C[(size_t)u * R + v] = (uint64_t)sendcounts[(size_t)u * R + v] * e;
      total += C[(size_t)u * R + v];
    }
  // A pattern that was issued before with the same buffers (same counts, displacements, pointers and settings) replays
  // its cached graph: validation, Algorithm 1 and the per-operation host cost were paid when it was built.
  std::vector<uint64_t> key;
  if (c->use_graph && total != 0) {
    key.reserve(8 + 2 * (size_t)R + 3 * (size_t)R * R);
    key.push_back(0xA11704117ull);   // tag: not a ring collective
    key.push_back((uint64_t)dtype);
    key.push_back((uint64_t)c->path);
    key.push_back((uint64_t)c->copy_ctas);
    key.push_back((uint64_t)c->piece_bytes);
    key.push_back((uint64_t)c->order_kernels);
    key.push_back((uint64_t)topo.gpus_per_node);
    key.push_back((uint64_t)c->model_rdma_sub_bytes);
    key.push_back((uint64_t)(uintptr_t)c->staging);
    key.push_back((uint64_t)c->staging_bytes);
    for (int r = 0; r < R; r++) {
      key.push_back((uint64_t)(uintptr_t)send[r]);
      key.push_back((uint64_t)(uintptr_t)recv[r]);
    }
    for (size_t i = 0; i < (size_t)R * R; i++) {
      key.push_back((uint64_t)sendcounts[i]);
      key.push_back((uint64_t)sdispls[i]);
      key.push_back((uint64_t)rdispls[i]);
    }
    for (auto& en : c->cache)
      if (en.key == key) {
        c->stats = hoccl_stats_t{};
        c->stats.graph_hit = 1;
        CU_TRY(c, cudaSetDevice(c->device));
        en.last_use = ++c->use_counter;
        CU_TRY(c, cudaGraphLaunch(en.exec, (cudaStream_t)stream));
        c->stats.n_moves = en.n_moves;
        c->stats.n_move_launches = en.n_move_launches;
        c->stats.max_copy_ctas = en.n_move_launches ? c->copy_ctas : 0;
        c->stats.n_pieces = en.n_pieces;
        c->stats.host_launch_us = now_us() - t0;
        return HOCCL_OK;
      }
  }
  // receive regions of one rank must not overlap each other, and no send region may overlap a receive region
  for (int v = 0; v < R; v++)
    for (int a = 0; a < R; a++) {
      const char* ra = (const char*)recv[v] + rdispls[(size_t)v * R + a] * e;
      const size_t la = C[(size_t)a * R + v];
      for (int b = a + 1; b < R; b++)
        if (ranges_overlap(ra, la, (const char*)recv[v] + rdispls[(size_t)v * R + b] * e, C[(size_t)b * R + v])) return HOCCL_ERR_INVALID_ARG;
      for (int u = 0; u < R; u++)
        for (int w = 0; w < R; w++)
          if (ranges_overlap(ra, la, (const char*)send[u] + sdispls[(size_t)u * R + w] * e, C[(size_t)u * R + w])) return HOCCL_ERR_INVALID_ARG;
    }
  c->stats = hoccl_stats_t{};
  if (total == 0) return HOCCL_OK;
  Schedule S;
  const uint64_t chunk_bytes = (uint64_t)std::max<long>(c->piece_bytes, 65536);
  if (!build_schedule(topo, C, chunk_bytes, &S)) return HOCCL_ERR_INTERNAL;
  CU_TRY(c, cudaSetDevice(c->device));
  cudaStream_t user = (cudaStream_t)stream;
  if (c->use_graph) {
    GraphEntry entry;
    entry.key = key;
    hoccl_result_t grc;
    if (modelled) {
      // staging for the flows between modelled nodes: what has left the sender's side and what has arrived at the receiver's
      std::vector<uint64_t> off((size_t)R * R, 0);
      uint64_t need = 0;
      for (int u = 0; u < R; u++)
        for (int v = 0; v < R; v++)
          if (u != v && !topo.same_node(u, v) && C[(size_t)u * R + v]) {
            off[(size_t)u * R + v] = need;
            need += (C[(size_t)u * R + v] + 255) / 256 * 256;
          }
      if (need && (!c->staging || c->staging_bytes < 2 * need)) return HOCCL_ERR_SCRATCH;
      for (int r = 0; r < R && need; r++)
        if (ranges_overlap((const char*)c->staging, 2 * need, (const char*)send[r], 1) || ranges_overlap((const char*)c->staging, 2 * need, (const char*)recv[r], 1))
          return HOCCL_ERR_INVALID_ARG;
      grc = build_pattern_graph_modelled(c, S, send, sdispls, recv, rdispls, e, (char*)c->staging, (char*)c->staging + need, off,
                                         (size_t)chunk_bytes, (size_t)c->model_rdma_sub_bytes, &entry);
    } else {
      grc = build_pattern_graph(c, S, send, sdispls, recv, rdispls, e, &entry);
    }
    if (grc != HOCCL_OK) return grc;
    GraphEntry* en = cache_put(c, std::move(entry));
    en->last_use = ++c->use_counter;
    CU_TRY(c, cudaGraphLaunch(en->exec, user));
    c->stats.n_moves = en->n_moves;
    c->stats.n_move_launches = en->n_move_launches;
    c->stats.max_copy_ctas = en->n_move_launches ? c->copy_ctas : 0;
    c->stats.n_pieces = en->n_pieces;
    c->stats.host_launch_us = now_us() - t0;
    return HOCCL_OK;
  }
  const int lanes = c->path == HOCCL_PATH_SM ? 1 : (int)std::max<long>(1, std::min<long>(c->lanes, kMaxLanes));
  c->ev_next = 0;
  cudaEvent_t fork = next_event(c);
  if (!fork) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
  CU_TRY(c, cudaEventRecord(fork, user));
  for (int l = 0; l < lanes; l++) CU_TRY(c, cudaStreamWaitEvent(c->lane[l], fork, 0));
  long moves = 0, launches = 0;
  for (size_t si = 0; si < S.stages.size(); si++) {
    const Stage& st = S.stages[si];
    auto endpoints = [&](const ChunkItem& it, const char** src, char** dst) {
      const StageFlow& f = st.flows[it.flow];
      const size_t so = sdispls[(size_t)f.origin_src * R + f.origin_dst] * e + f.origin_offset + it.offset;
      const size_t dofs = rdispls[(size_t)f.origin_dst * R + f.origin_src] * e + f.origin_offset + it.offset;
      *src = (const char*)send[f.origin_src] + so;
      *dst = (char*)recv[f.origin_dst] + dofs;
    };
    // Service order is the scheduler's; chunks that follow one another in a queue and continue the same flow are
    // issued as one operation (a queue that serves a single flow, the uniform case, becomes one copy per flow).
    std::vector<std::vector<ChunkItem>> queues(R);
    for (int g = 0; g < R; g++)
      for (const ChunkItem& it : st.queues[g]) {
        if (!queues[g].empty() && queues[g].back().flow == it.flow && queues[g].back().offset + queues[g].back().bytes == it.offset)
          queues[g].back().bytes += it.bytes;
        else
          queues[g].push_back(it);
      }
    if (c->path == HOCCL_PATH_CE) {
      // every DMA queue (one per source rank) is a serial chain on its lane, in the interleaved chunk order
      for (int g = 0; g < R; g++) {
        cudaStream_t lane = c->lane[g % lanes];
        for (const ChunkItem& it : queues[g]) {
          const char* src;
          char* dst;
          endpoints(it, &src, &dst);
          CU_TRY(c, cudaMemcpyAsync(dst, src, it.bytes, cudaMemcpyDeviceToDevice, lane));
          moves++;
        }
      }
    } else {
      // SM path: the k-th chunk of every queue goes into one batched copy launch (the queues advance in lock step,
      // which is what R engines of equal speed would do), so a stage costs as many launches as its longest queue
      size_t depth = 0;
      for (int g = 0; g < R; g++) depth = std::max(depth, queues[g].size());
      for (size_t k = 0; k < depth; k++) {
        CopyBatch b;
        b.nseg = 0;
        b.pad = 0;
        for (int g = 0; g < R; g++) {
          if (k >= queues[g].size()) continue;
          const ChunkItem& it = queues[g][k];
          const char* src;
          char* dst;
          endpoints(it, &src, &dst);
          b.seg[b.nseg++] = CopySeg{src, dst, (unsigned long long)it.bytes};
          moves++;
          if (b.nseg == kMaxSegs) {
            CU_TRY(c, launch_copy(b, (int)c->copy_ctas, c->lane[0]));
            launches++;
            b.nseg = 0;
          }
        }
        if (b.nseg > 0) {
          CU_TRY(c, launch_copy(b, (int)c->copy_ctas, c->lane[0]));
          launches++;
        }
      }
    }
    // stages run one after the other (the paper's serial stages): barrier over the lanes
    if (si + 1 < S.stages.size() && lanes > 1) {
      std::vector<cudaEvent_t> evs(lanes);
      for (int l = 0; l < lanes; l++) {
        evs[l] = next_event(c);
        if (!evs[l]) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
        CU_TRY(c, cudaEventRecord(evs[l], c->lane[l]));
      }
      for (int l = 0; l < lanes; l++)
        for (int m = 0; m < lanes; m++)
          if (m != l) CU_TRY(c, cudaStreamWaitEvent(c->lane[l], evs[m], 0));
    }
  }
  for (int l = 0; l < lanes; l++) {
    cudaEvent_t ev = next_event(c);
    if (!ev) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    CU_TRY(c, cudaEventRecord(ev, c->lane[l]));
    CU_TRY(c, cudaStreamWaitEvent(user, ev, 0));
  }
  c->stats.n_moves = moves;
  c->stats.n_move_launches = launches;
  c->stats.max_copy_ctas = launches ? c->copy_ctas : 0;
  c->stats.n_pieces = (long)S.stages.size();
  c->stats.host_launch_us = now_us() - t0;
  return HOCCL_OK;
}

// ---------------------------------------------------------------- scheduler inspection (host only) ----
struct hoccl_sched {
  Schedule s;
};

hoccl_result_t hoccl_sched_build(hoccl_sched_t* out, int G, int gpus_per_node, double bw_nvlink, double bw_rdma, const uint64_t* C,
                                 uint64_t chunk_bytes) {
  if (!out) return HOCCL_ERR_INVALID_ARG;
  *out = nullptr;
  if (!C || G < 1 || G > 256 || gpus_per_node < 1 || chunk_bytes == 0) return HOCCL_ERR_INVALID_ARG;
  Topology t;
  t.G = G;
  t.gpus_per_node = gpus_per_node;
  if (bw_nvlink > 0) t.bw_nvlink = bw_nvlink;
  if (bw_rdma > 0) t.bw_rdma = bw_rdma;
  hoccl_sched* h = new hoccl_sched();
  std::vector<uint64_t> Cv(C, C + (size_t)G * G);
  if (!build_schedule(t, Cv, chunk_bytes, &h->s)) {
    delete h;
    return HOCCL_ERR_INVALID_ARG;
  }
  *out = h;
  return HOCCL_OK;
}

void hoccl_sched_destroy(hoccl_sched_t s) { delete s; }
int hoccl_sched_num_stages(hoccl_sched_t s) { return s ? (int)s->s.stages.size() : 0; }
double hoccl_sched_stage_tau(hoccl_sched_t s, int stage) {
  return (s && stage >= 0 && stage < (int)s->s.stages.size()) ? s->s.stages[stage].tau : -1.0;
}
double hoccl_sched_total_tau(hoccl_sched_t s) { return s ? s->s.total_tau : -1.0; }
double hoccl_sched_lower_bound(hoccl_sched_t s) { return s ? s->s.lower_bound : -1.0; }

hoccl_result_t hoccl_sched_matrix(hoccl_sched_t s, int which, uint64_t* out) {
  if (!s || !out) return HOCCL_ERR_INVALID_ARG;
  const int G = s->s.topo.G;
  const size_t n = (size_t)G * G;
  if (which == -1) {
    std::copy(s->s.T.begin(), s->s.T.end(), out);
  } else if (which == -2) {
    std::copy(s->s.C.begin(), s->s.C.end(), out);
  } else if (which >= 0 && which < (int)s->s.stages.size()) {
    std::fill(out, out + n, 0);
    for (const StageFlow& f : s->s.stages[which].flows) out[(size_t)f.u * G + f.v] += f.bytes;
  } else {
    return HOCCL_ERR_INVALID_ARG;
  }
  return HOCCL_OK;
}

int hoccl_sched_num_flows(hoccl_sched_t s, int stage) {
  return (s && stage >= 0 && stage < (int)s->s.stages.size()) ? (int)s->s.stages[stage].flows.size() : -1;
}

hoccl_result_t hoccl_sched_get_flow(hoccl_sched_t s, int stage, int index, hoccl_sched_flow_t* out) {
  if (!s || !out || stage < 0 || stage >= (int)s->s.stages.size()) return HOCCL_ERR_INVALID_ARG;
  const Stage& st = s->s.stages[stage];
  if (index < 0 || index >= (int)st.flows.size()) return HOCCL_ERR_INVALID_ARG;
  const StageFlow& f = st.flows[index];
  out->src = f.u;
  out->dst = f.v;
  out->cls = f.cls;
  out->origin_src = f.origin_src;
  out->origin_dst = f.origin_dst;
  out->bytes = f.bytes;
  out->origin_offset = f.origin_offset;
  return HOCCL_OK;
}

int hoccl_sched_queue_len(hoccl_sched_t s, int stage, int gpu) {
  if (!s || stage < 0 || stage >= (int)s->s.stages.size() || gpu < 0 || gpu >= s->s.topo.G) return -1;
  return (int)s->s.stages[stage].queues[gpu].size();
}

hoccl_result_t hoccl_sched_queue_get(hoccl_sched_t s, int stage, int gpu, int index, int* flow, uint64_t* offset, uint64_t* bytes) {
  if (!s || !flow || !offset || !bytes || stage < 0 || stage >= (int)s->s.stages.size() || gpu < 0 || gpu >= s->s.topo.G)
    return HOCCL_ERR_INVALID_ARG;
  const auto& q = s->s.stages[stage].queues[gpu];
  if (index < 0 || index >= (int)q.size()) return HOCCL_ERR_INVALID_ARG;
  *flow = q[index].flow;
  *offset = q[index].offset;
  *bytes = q[index].bytes;
  return HOCCL_OK;
}

const char* hoccl_error_string(hoccl_result_t code) {
  switch (code) {
    case HOCCL_OK: return "ok";
    case HOCCL_ERR_INVALID_ARG: return "invalid argument";
    case HOCCL_ERR_UNSUPPORTED: return "unsupported operation, dtype or parameter";
    case HOCCL_ERR_CUDA: return "CUDA error";
    case HOCCL_ERR_MISMATCH: return "send/recv mismatch";
    case HOCCL_ERR_PENDING: return "unmatched send/recv posts pending";
    case HOCCL_ERR_SCRATCH: return "scratch or staging memory missing or too small";
    case HOCCL_ERR_INTERNAL: return "internal error";
    case HOCCL_ERR_TIMEOUT: return "watchdog timeout in the stream hand-over (the stream was released)";
  }
  return "unknown error code";
}

const char* hoccl_last_cuda_error(hoccl_comm_t c) { return c ? c->cuda_err.c_str() : ""; }

hoccl_result_t hoccl_last_stats(hoccl_comm_t c, hoccl_stats_t* out) {
  if (!c || !out) return HOCCL_ERR_INVALID_ARG;
  // profile numbers: read events of work that has completed (the caller synchronises first)
  harvest_profile(c);
  *out = c->stats;
  out->sum_kernel_ms = c->prof_ms;
  out->sum_kernel_launches_timed = c->prof_n;
  out->sum_kernel_bytes = c->prof_bytes;
  out->copy_kernel_ms = c->prof_copy_ms;
  out->copy_kernel_launches_timed = c->prof_copy_n;
  out->copy_kernel_bytes = c->prof_copy_bytes;
  return HOCCL_OK;
}

hoccl_result_t hoccl_profile_reset(hoccl_comm_t c) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  harvest_profile(c);
  c->prof_ms = 0;
  c->prof_bytes = 0;
  c->prof_n = 0;
  c->prof_copy_ms = 0;
  c->prof_copy_bytes = 0;
  c->prof_copy_n = 0;
  return HOCCL_OK;
}

hoccl_result_t hoccl_sum_launch(const void* inbox, const void* local, void* out, size_t count, hoccl_dtype_t dtype, int ctas,
                                hoccl_stream_t stream) {
  size_t e = dtype_size((int)dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  if (!inbox || !local || !out || ctas < 1 || ctas > 1024) return HOCCL_ERR_INVALID_ARG;
  if (((uintptr_t)inbox % e) || ((uintptr_t)local % e) || ((uintptr_t)out % e)) return HOCCL_ERR_INVALID_ARG;
  if (count == 0) return HOCCL_OK;
  SumBatch b;
  b.nseg = 1;
  b.dtype = (int)dtype;
  b.seg[0] = SumSeg{inbox, local, out, (unsigned long long)count};
  return launch_sum(b, ctas, (cudaStream_t)stream) == cudaSuccess ? HOCCL_OK : HOCCL_ERR_CUDA;
}

hoccl_result_t hoccl_port_probe(int mode, void* buf, size_t bytes, int ctas, unsigned int* sink, hoccl_stream_t stream) {
  if ((mode != 0 && mode != 1) || !buf || !sink || ((uintptr_t)buf & 15) || bytes < (128u << 10) || ctas < 1 || ctas > 1024) return HOCCL_ERR_INVALID_ARG;
  return launch_port_probe(mode, buf, bytes, ctas, sink, (cudaStream_t)stream) == cudaSuccess ? HOCCL_OK : HOCCL_ERR_CUDA;
}

hoccl_result_t hoccl_flatten_inspect(int kind, hoccl_dtype_t dtype, int ctas, int nseg, const uint64_t* a_addr, const uint64_t* b_addr,
                                     const uint64_t* out_addr, const uint64_t* len, uint64_t* tiles_end, uint64_t* scalars_end, uint64_t* nvec,
                                     uint32_t* head, uint64_t* tile_vectors) {
  if ((kind != 0 && kind != 1) || nseg < 1 || nseg > kMaxSegs || !a_addr || !out_addr || (kind == 0 && !b_addr) || !len || !tiles_end ||
      !scalars_end || !nvec || !head || !tile_vectors || ctas < 1)
    return HOCCL_ERR_INVALID_ARG;
  if (kind == 0 && dtype_size((int)dtype) == 0) return HOCCL_ERR_UNSUPPORTED;
  const Flat* f = nullptr;
  SumBatch sb;
  CopyBatch cb;
  if (kind == 0) {
    sb.nseg = nseg;
    sb.dtype = (int)dtype;
    for (int k = 0; k < nseg; k++)
      sb.seg[k] = SumSeg{(const void*)(uintptr_t)a_addr[k], (const void*)(uintptr_t)b_addr[k], (void*)(uintptr_t)out_addr[k], len[k]};
    prepare_sum_batch(&sb, ctas);
    f = &sb.flat;
    int threads = 0;
    (void)sum_kernel_entry((int)dtype, ctas, &threads);
    *tile_vectors = 4ull * (uint64_t)threads;
  } else {
    cb.nseg = nseg;
    cb.pad = 0;
    for (int k = 0; k < nseg; k++) cb.seg[k] = CopySeg{(const void*)(uintptr_t)a_addr[k], (void*)(uintptr_t)out_addr[k], len[k]};
    prepare_copy_batch(&cb, ctas);
    f = &cb.flat;
    int threads = 0;
    (void)copy_kernel_entry(ctas, &threads);
    *tile_vectors = (threads == 1024 ? 8ull : 4ull) * (uint64_t)threads;
  }
  for (int k = 0; k < nseg; k++) {
    tiles_end[k] = f->tpre[k + 1];
    scalars_end[k] = f->spre[k + 1];
    nvec[k] = f->nvec[k];
    head[k] = f->head[k];
  }
  return HOCCL_OK;
}

hoccl_result_t hoccl_chain_launch(const void* first, size_t stride_bytes, int nsrc, const void* local, void* out, size_t count,
                                  hoccl_dtype_t dtype, int ctas, hoccl_stream_t stream) {
  const size_t e = dtype_size((int)dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  if (!first || !local || !out || nsrc < 1 || nsrc > kMaxChainSrcs || (stride_bytes & 15) || ctas < 1 || ctas > 1024 ||
      ((uintptr_t)first % e) || ((uintptr_t)local % e) || ((uintptr_t)out % e))
    return HOCCL_ERR_INVALID_ARG;
  if (count == 0) return HOCCL_OK;
  ChainBatch b;
  b.nseg = 1;
  b.dtype = (int)dtype;
  b.seg[0] = ChainSeg{first, local, out, (unsigned long long)count, (unsigned long long)stride_bytes, nsrc, 0};
  return launch_chain(b, ctas, (cudaStream_t)stream) == cudaSuccess ? HOCCL_OK : HOCCL_ERR_CUDA;
}

hoccl_result_t hoccl_selftest_bf16_add(unsigned long long* counts, hoccl_stream_t stream) {
  if (!counts) return HOCCL_ERR_INVALID_ARG;
  return launch_bf16_add_selftest(counts, (cudaStream_t)stream) == cudaSuccess ? HOCCL_OK : HOCCL_ERR_CUDA;
}

hoccl_result_t hoccl_fanout_inspect(int n, const uint64_t* src, const uint64_t* dst, const uint64_t* len, int ctas, int seg_cap,
                                    int* seg_launch, uint64_t* seg_src, uint64_t* seg_len, int* seg_ndst, uint32_t* seg_head,
                                    uint64_t* seg_nvec, uint64_t* dst_out, int* n_seg, int* n_launch) {
  if (n < 1 || !src || !dst || !len || ctas < 1 || seg_cap < 1 || !seg_launch || !seg_src || !seg_len || !seg_ndst || !seg_head ||
      !seg_nvec || !dst_out || !n_seg || !n_launch)
    return HOCCL_ERR_INVALID_ARG;
  RGroup g;
  g.kind = OP_MOVE;
  g.piece = 0;
  g.chain_dep = -1;
  for (int i = 0; i < n; i++) {
    Seg sg = {};
    sg.src = (const char*)(uintptr_t)src[i];
    sg.dst = (char*)(uintptr_t)dst[i];
    sg.bytes = len[i];
    g.segs.push_back(sg);
  }
  std::vector<FanBatch> fans;
  std::vector<double> hbm;
  std::vector<long> moves;
  *n_seg = 0;
  *n_launch = 0;
  if (!build_fan_batches(g, &fans, &hbm, &moves)) return HOCCL_OK;
  int k = 0;
  size_t nd = 0;
  for (size_t b = 0; b < fans.size(); b++) {
    prepare_fan_batch(&fans[b], ctas);
    for (int j = 0; j < fans[b].nseg; j++) {
      const FanSeg& fs = fans[b].seg[j];
      if (k >= seg_cap || nd + (size_t)fs.ndst > (size_t)n) return HOCCL_ERR_INVALID_ARG;
      seg_launch[k] = (int)b;
      seg_src[k] = (uint64_t)(uintptr_t)fs.src;
      seg_len[k] = fs.bytes;
      seg_ndst[k] = fs.ndst;
      seg_head[k] = fans[b].flat.head[j];
      seg_nvec[k] = fans[b].flat.nvec[j];
      for (int d = 0; d < fs.ndst; d++) dst_out[nd++] = (uint64_t)(uintptr_t)fans[b].dst[fs.first_dst + d];
      k++;
    }
  }
  *n_seg = k;
  *n_launch = (int)fans.size();
  return HOCCL_OK;
}

hoccl_result_t hoccl_kernel_sms(int kind, const void* a, const void* b, void* out, size_t bytes, hoccl_dtype_t dtype, int ctas,
                                unsigned int* smid_out, hoccl_stream_t stream) {
  size_t e = dtype_size((int)dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  if ((kind != 0 && kind != 1) || !a || !out || (kind == 0 && !b) || !smid_out || ctas < 1 || ctas > 1024) return HOCCL_ERR_INVALID_ARG;
  if (((uintptr_t)smid_out & 3) || (kind == 0 && (((uintptr_t)a | (uintptr_t)b | (uintptr_t)out) % e))) return HOCCL_ERR_INVALID_ARG;
  if (bytes == 0) return HOCCL_OK;
  if (kind == 0) {
    SumBatch sb;
    sb.nseg = 1;
    sb.dtype = (int)dtype;
    sb.seg[0] = SumSeg{a, b, out, (unsigned long long)(bytes / e)};
    sb.smid_out = smid_out;
    return launch_sum(sb, ctas, (cudaStream_t)stream) == cudaSuccess ? HOCCL_OK : HOCCL_ERR_CUDA;
  }
  CopyBatch cb;
  cb.nseg = 1;
  cb.pad = 0;
  cb.seg[0] = CopySeg{a, out, (unsigned long long)bytes};
  cb.smid_out = smid_out;
  return launch_copy(cb, ctas, (cudaStream_t)stream) == cudaSuccess ? HOCCL_OK : HOCCL_ERR_CUDA;
}

hoccl_result_t hoccl_copy_launch(const void* src, void* dst, size_t bytes, int ctas, hoccl_stream_t stream) {
  if (!src || !dst || ctas < 1 || ctas > 1024) return HOCCL_ERR_INVALID_ARG;
  if (bytes == 0) return HOCCL_OK;
  CopyBatch b;
  b.nseg = 1;
  b.pad = 0;
  b.seg[0] = CopySeg{src, dst, (unsigned long long)bytes};
  return launch_copy(b, ctas, (cudaStream_t)stream) == cudaSuccess ? HOCCL_OK : HOCCL_ERR_CUDA;
}

hoccl_result_t hoccl_fanout_launch(const void* src, void* const* dsts, int ndst, size_t bytes, int ctas, hoccl_stream_t stream) {
  if (!src || !dsts || ndst < 1 || ndst > kMaxFanDsts || ctas < 1 || ctas > 1024) return HOCCL_ERR_INVALID_ARG;
  for (int d = 0; d < ndst; d++) {
    if (!dsts[d] || ranges_overlap((const char*)src, bytes, (const char*)dsts[d], bytes)) return HOCCL_ERR_INVALID_ARG;
    for (int k = 0; k < d; k++)
      if (ranges_overlap((const char*)dsts[k], bytes, (const char*)dsts[d], bytes)) return HOCCL_ERR_INVALID_ARG;
  }
  if (bytes == 0) return HOCCL_OK;
  // the same grouping as the collectives use: one segment per 16-byte phase of the destinations
  RGroup g;
  g.kind = OP_MOVE;
  g.piece = 0;
  g.chain_dep = -1;
  for (int d = 0; d < ndst; d++) {
    Seg s = {};
    s.src = (const char*)src;
    s.dst = (char*)dsts[d];
    s.bytes = bytes;
    g.segs.push_back(s);
  }
  std::vector<FanBatch> fans;
  std::vector<double> hbm;
  std::vector<long> moves;
  if (!build_fan_batches(g, &fans, &hbm, &moves)) {   // no two destinations share a phase (or there is only one): plain copies
    for (size_t first = 0; first < g.segs.size(); first += kMaxSegs) {
      const size_t n = std::min<size_t>(kMaxSegs, g.segs.size() - first);
      CopyBatch b;
      fill_copy_batch(g, first, n, &b);
      if (launch_copy(b, ctas, (cudaStream_t)stream) != cudaSuccess) return HOCCL_ERR_CUDA;
    }
    return HOCCL_OK;
  }
  for (const FanBatch& f : fans)
    if (launch_fan(f, ctas, (cudaStream_t)stream) != cudaSuccess) return HOCCL_ERR_CUDA;
  return HOCCL_OK;
}

// ---------------------------------------------------------------- plan inspection ----------------
struct hoccl_plan {
  Plan p;
};

hoccl_result_t hoccl_plan_build(hoccl_plan_t* plan, int kind, int R, size_t count, hoccl_dtype_t dtype, int in_place, size_t piece_bytes,
                                int max_pieces, const unsigned char* send_align) {
  if (!plan) return HOCCL_ERR_INVALID_ARG;
  *plan = nullptr;
  if (R < 1 || R > kMaxRanks) return HOCCL_ERR_INVALID_ARG;
  if (dtype_size((int)dtype) == 0) return HOCCL_ERR_UNSUPPORTED;
  hoccl_plan* h = new hoccl_plan();
  if (!build_plan(&h->p, kind, R, count, (int)dtype, in_place != 0, piece_bytes, max_pieces, send_align)) {
    delete h;
    return HOCCL_ERR_INVALID_ARG;
  }
  *plan = h;
  return HOCCL_OK;
}

void hoccl_plan_destroy(hoccl_plan_t plan) { delete plan; }
size_t hoccl_plan_slot_bytes(hoccl_plan_t plan) { return plan ? plan->p.slot_bytes : 0; }
int hoccl_plan_inbox_slots(hoccl_plan_t plan) { return plan ? plan->p.inbox_slots : 0; }
size_t hoccl_plan_scratch_bytes(hoccl_plan_t plan) { return plan ? plan->p.scratch_need() : 0; }
int hoccl_plan_num_ops(hoccl_plan_t plan) { return plan ? (int)plan->p.ops.size() : 0; }
int hoccl_plan_num_groups(hoccl_plan_t plan) { return plan ? (int)plan->p.groups.size() : 0; }

hoccl_result_t hoccl_plan_get_op(hoccl_plan_t plan, int index, hoccl_plan_op_t* out) {
  if (!plan || !out || index < 0 || index >= (int)plan->p.ops.size()) return HOCCL_ERR_INVALID_ARG;
  const PlanOp& o = plan->p.ops[index];
  out->kind = o.kind;
  out->phase = o.phase;
  out->step = o.step;
  out->piece = o.piece;
  out->rank = o.rank;
  out->dst_rank = o.dst_rank;
  out->chunk = o.chunk;
  out->src_buf = o.src_buf;
  out->dst_buf = o.dst_buf;
  out->local_buf = o.local_buf;
  out->src_off = o.src_off;
  out->dst_off = o.dst_off;
  out->local_off = o.local_off;
  out->bytes = o.bytes;
  out->group = o.group;
  out->nsrc = o.nsrc;
  out->src_stride = o.src_stride;
  return HOCCL_OK;
}

int hoccl_plan_group_deps(hoccl_plan_t plan, int group, int* deps, int cap) {
  if (!plan || group < 0 || group >= (int)plan->p.groups.size()) return -1;
  const PlanGroup& g = plan->p.groups[group];
  int n = 0;
  for (int d : g.deps) {
    if (deps && n < cap) deps[n] = d;
    n++;
  }
  if (g.chain_dep >= 0 && std::find(g.deps.begin(), g.deps.end(), g.chain_dep) == g.deps.end()) {
    if (deps && n < cap) deps[n] = g.chain_dep;
    n++;
  }
  return n;
}


}  // extern "C"

extern "C" hoccl_result_t hoccl_options_resolve(const hoccl_options_t* o, hoccl_resolved_t* out) {
  if (!o || !out) return HOCCL_ERR_INVALID_ARG;
  hoccl::OptionsIn in{o->kind, o->R, o->count, o->dtype, o->path, o->onepass, o->forward, o->fused, o->rs_direct, o->ag_direct,
                      o->handshake, o->use_graph, o->ce_small_bytes, o->ce_small_ctas, o->copy_ctas, o->scratch_bytes, o->host_call, o->roles};
  hoccl::OptionsOut r;
  hoccl_result_t rc = hoccl::resolve_options(in, &r);
  if (rc != HOCCL_OK) return rc;
  out->plan_kind = r.plan_kind;
  out->executor = r.executor;
  out->path = r.path;
  out->copy_ctas = r.copy_ctas;
  out->small_switch = r.small_switch;
  return HOCCL_OK;
}
