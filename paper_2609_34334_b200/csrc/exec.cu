// libhoccl: communicator, executors and the C ABI declared in include/hoccl.h.
//
// A collective call = plan (host, plan.cpp) -> resolve the plan's buffer offsets against the caller's
// pointers -> issue.  Two issue engines consume the same plan and give the same bits:
//   * graph executor (default): the plan's group DAG becomes an explicit CUDA graph (memcpy nodes for
//     moves on the copy route, kernel nodes for sums and SM copies), instantiated once per distinct
//     call signature, cached, and replayed with one cudaGraphLaunch into the caller's stream.  A graph
//     launch is stream ordered, which is exactly the operator-level ordering the paper's stream
//     manager provides (Sec. 3.2), and it removes the per-operation host cost that the paper reports
//     as its launch overhead (Sec. 5 "CPU launch overhead").
//   * stream executor: internal move lanes plus one sum stream, ordered with CUDA events
//     (fork from the caller's stream, join back into it).
// SUM launches are chained (one at a time) so that the SM budget for sums is global, not per piece.
#include "comm.h"

namespace hoccl {

hoccl_result_t validate(hoccl_comm* c, Call* call) {
  const int R = c->R;
  const size_t e = dtype_size(call->dtype);
  if (!call->send || !call->recv) return HOCCL_ERR_INVALID_ARG;
  for (int r = 0; r < R; r++) {
    if (!call->send[r] || !call->recv[r]) return HOCCL_ERR_INVALID_ARG;
    if (((uintptr_t)call->send[r] % e) || ((uintptr_t)call->recv[r] % e)) return HOCCL_ERR_INVALID_ARG;
  }
  // in-place forms
  int n_in = 0;
  for (int r = 0; r < R; r++) {
    const char* s = (const char*)call->send[r];
    const char* d = (const char*)call->recv[r];
    bool in;
    if (call->kind == PLAN_ALLREDUCE) in = (s == d);
    else if (call->kind == PLAN_REDUCE_SCATTER) in = (d == s + (size_t)r * call->count * e);
    else if (call->kind == PLAN_ALLTOALL) in = false;   // no in-place form: any overlap of send[r] and recv[r] is an error
    else in = (s == d + (size_t)r * call->count * e);
    if (in) n_in++;
    else if (ranges_overlap(s, call->send_bytes, d, call->recv_bytes)) return HOCCL_ERR_INVALID_ARG;
  }
  if (n_in != 0 && n_in != R) return HOCCL_ERR_INVALID_ARG;
  call->in_place = (n_in == R);
  // buffers of different ranks must be disjoint
  for (int a = 0; a < R; a++)
    for (int b = a + 1; b < R; b++) {
      const char *sa = (const char*)call->send[a], *sb = (const char*)call->send[b];
      const char *da = (const char*)call->recv[a], *db = (const char*)call->recv[b];
      if (ranges_overlap(sa, call->send_bytes, sb, call->send_bytes) || ranges_overlap(da, call->recv_bytes, db, call->recv_bytes) ||
          ranges_overlap(sa, call->send_bytes, db, call->recv_bytes) || ranges_overlap(da, call->recv_bytes, sb, call->send_bytes))
        return HOCCL_ERR_INVALID_ARG;
    }
  return HOCCL_OK;
}

// Turns plan offsets into addresses (the plan already places pieces inside the scratch slots).
void resolve(hoccl_comm* c, const Plan& P, const Call& call, std::vector<RGroup>* out, size_t* host_need) {
  *host_need = 0;
  const int R = P.R;
  char* inbox0 = (char*)c->scratch;
  char* partial0 = inbox0 + (size_t)R * P.slot_bytes;
  auto addr = [&](int buf, int rank, int chunk, uint64_t off) -> char* {
    (void)chunk;
    switch (buf) {
      case BUF_SEND: return (char*)call.send[rank] + off;
      case BUF_RECV: return (char*)call.recv[rank] + off;
      case BUF_INBOX: return inbox0 + (size_t)rank * P.slot_bytes + off;
      default: return partial0 + (size_t)rank * P.slot_bytes + off;
    }
  };
  out->clear();
  out->resize(P.groups.size());
  for (size_t g = 0; g < P.groups.size(); g++) {
    const PlanGroup& pg = P.groups[g];
    RGroup& rg = (*out)[g];
    rg.kind = pg.kind;
    rg.deps = pg.deps;
    rg.chain_dep = pg.chain_dep;
    for (int i = 0; i < pg.num_ops; i++) {
      const PlanOp& op = P.ops[pg.first_op + i];
      Seg s;
      s.bytes = op.bytes;
      if (op.kind == OP_MOVE) {
        s.src = addr(op.src_buf, op.rank, op.chunk, op.src_off);
        s.dst = addr(op.dst_buf, op.dst_rank, op.chunk, op.dst_off);
        s.local = nullptr;
      } else {
        s.src = addr(op.src_buf, op.rank, op.chunk, op.src_off);
        s.local = addr(op.local_buf, op.rank, op.chunk, op.local_off);
        s.dst = addr(op.dst_buf, op.dst_rank, op.chunk, op.dst_off);  // dst_rank == rank except in the forward variant
      }
      if (op.kind == OP_MOVE && c->path == HOCCL_PATH_CE_HOST) {
        s.host_off = *host_need;
        *host_need += (s.bytes + 255) / 256 * 256;
      }
      rg.segs.push_back(s);
    }
  }
  // SM path: the stages of an all-to-all are independent (disjoint blocks, no dependencies), so their moves go into as few
  // batched launches as the segment table allows instead of one launch per stage
  if (c->path == HOCCL_PATH_SM && P.kind == PLAN_ALLTOALL && out->size() > 1) {
    bool independent = true;
    for (const RGroup& g : *out) independent = independent && g.deps.empty() && g.kind == OP_MOVE;
    if (independent) {
      RGroup all = (*out)[0];
      for (size_t g = 1; g < out->size(); g++) all.segs.insert(all.segs.end(), (*out)[g].segs.begin(), (*out)[g].segs.end());
      out->assign(1, all);
    }
  }
}

void fill_sum_batch(const RGroup& g, size_t first, size_t n, int dtype, size_t elem, SumBatch* b) {
  b->nseg = (int)n;
  b->dtype = dtype;
  for (size_t i = 0; i < n; i++) {
    const Seg& s = g.segs[first + i];
    b->seg[i] = SumSeg{s.src, s.local, s.dst, (unsigned long long)(s.bytes / elem)};
  }
}
void fill_copy_batch(const RGroup& g, size_t first, size_t n, CopyBatch* b) {
  b->nseg = (int)n;
  b->pad = 0;
  for (size_t i = 0; i < n; i++) {
    const Seg& s = g.segs[first + i];
    b->seg[i] = CopySeg{s.src, s.dst, (unsigned long long)s.bytes};
  }
}

struct Tally {
  long moves = 0, move_launches = 0, sum_launches = 0;
};

// ------------------------------------------------------------------ stream executor -------------
hoccl_result_t run_streams(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, cudaStream_t user, Tally* tally) {
  const int lanes = (int)std::max<long>(1, std::min<long>(c->lanes, kMaxLanes));
  c->ev_next = 0;
  std::vector<cudaStream_t> where(groups.size(), nullptr);
  std::vector<cudaEvent_t> done(groups.size(), nullptr);
  std::vector<char> lane_used(lanes, 0);
  bool sum_used = false;
  cudaEvent_t fork = next_event(c);
  if (!fork) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
  CU_TRY(c, cudaEventRecord(fork, user));
  auto touch = [&](cudaStream_t s, char* used) -> cudaError_t {
    if (*used) return cudaSuccess;
    *used = 1;
    return cudaStreamWaitEvent(s, fork, 0);
  };
  int move_rr = 0;
  for (size_t g = 0; g < groups.size(); g++) {
    const RGroup& rg = groups[g];
    cudaStream_t s;
    if (rg.kind == OP_SUM) {
      s = c->sum_stream;
      char u = sum_used ? 1 : 0;
      CU_TRY(c, touch(s, &u));
      sum_used = true;
    } else {
      int l = c->path == HOCCL_PATH_SM ? 0 : move_rr++ % lanes;   // SM copies share one lane: global CTA budget
      s = c->lane[l];
      CU_TRY(c, touch(s, &lane_used[l]));
    }
    where[g] = s;
    for (int d : rg.deps)
      if (where[d] != s) CU_TRY(c, cudaStreamWaitEvent(s, done[d], 0));
    // chain_dep needs no event here: every SUM is on the one sum stream
    if (rg.kind == OP_SUM) {
      for (size_t first = 0; first < rg.segs.size(); first += kMaxSegs) {
        size_t n = std::min<size_t>(kMaxSegs, rg.segs.size() - first);
        SumBatch b;
        fill_sum_batch(rg, first, n, P.dtype, P.elem, &b);
        std::pair<cudaEvent_t, cudaEvent_t> pe{nullptr, nullptr};
        if (c->profile) {
          if (c->prof_pool.empty()) {
            cudaEvent_t a, z;
            CU_TRY(c, cudaEventCreate(&a));
            CU_TRY(c, cudaEventCreate(&z));
            pe = {a, z};
          } else {
            pe = c->prof_pool.back();
            c->prof_pool.pop_back();
          }
          CU_TRY(c, cudaEventRecord(pe.first, s));
        }
        CU_TRY(c, launch_sum(b, (int)c->sum_ctas, s));
        if (c->profile) {
          CU_TRY(c, cudaEventRecord(pe.second, s));
          double bytes = 0;
          for (size_t i = 0; i < n; i++) bytes += 3.0 * (double)rg.segs[first + i].bytes;
          c->prof_open.push_back({pe, bytes});
        }
        tally->sum_launches++;
      }
    } else if (c->path == HOCCL_PATH_CE) {
      for (const Seg& sg : rg.segs) {
        CU_TRY(c, cudaMemcpyAsync(sg.dst, sg.src, sg.bytes, cudaMemcpyDeviceToDevice, s));
        tally->moves++;
      }
    } else if (c->path == HOCCL_PATH_CE_HOST) {
      // two copy-engine legs through pinned host memory: no SM takes part in the move
      for (const Seg& sg : rg.segs) {
        CU_TRY(c, cudaMemcpyAsync(c->host_staging + sg.host_off, sg.src, sg.bytes, cudaMemcpyDeviceToHost, s));
        CU_TRY(c, cudaMemcpyAsync(sg.dst, c->host_staging + sg.host_off, sg.bytes, cudaMemcpyHostToDevice, s));
        tally->moves++;
      }
    } else {
      for (size_t first = 0; first < rg.segs.size(); first += kMaxSegs) {
        size_t n = std::min<size_t>(kMaxSegs, rg.segs.size() - first);
        CopyBatch b;
        fill_copy_batch(rg, first, n, &b);
        CU_TRY(c, launch_copy(b, (int)c->copy_ctas, s));
        tally->moves += (long)n;
        tally->move_launches++;
      }
    }
    cudaEvent_t ev = next_event(c);
    if (!ev) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    CU_TRY(c, cudaEventRecord(ev, s));
    done[g] = ev;
  }
  // join: the caller's stream waits for every internal stream that was used
  for (int l = 0; l < lanes; l++)
    if (lane_used[l]) {
      cudaEvent_t ev = next_event(c);
      if (!ev) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
      CU_TRY(c, cudaEventRecord(ev, c->lane[l]));
      CU_TRY(c, cudaStreamWaitEvent(user, ev, 0));
    }
  if (sum_used) {
    cudaEvent_t ev = next_event(c);
    if (!ev) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    CU_TRY(c, cudaEventRecord(ev, c->sum_stream));
    CU_TRY(c, cudaStreamWaitEvent(user, ev, 0));
  }
  return HOCCL_OK;
}

// ------------------------------------------------------------------ graph executor --------------
void destroy_entry(GraphEntry* e) {
  if (e->exec) cudaGraphExecDestroy(e->exec);
  for (cudaGraphExec_t pe : e->piece_exec)
    if (pe) cudaGraphExecDestroy(pe);
  e->piece_exec.clear();
  for (auto& p : e->prof_events) {
    cudaEventDestroy(p.first);
    cudaEventDestroy(p.second);
  }
  e->exec = nullptr;
  e->prof_events.clear();
}

// Host <-> staging copies of one piece of one rank (all-reduce layout): piece p of every ring chunk, i.e. rows of
// `piece` bytes at a pitch of one chunk.  Chunks that hold the full piece go as one 2-D copy; a shorter trailing piece
// as a 1-D copy.
static void add_host_copies(const Plan& P, int p, char* dev, char* host, std::vector<HostCopy>* out) {
  const size_t e = P.elem, q_bytes = P.chunk_elems * e;
  const size_t off = (size_t)p * P.piece_bytes;
  size_t full_rows = 0, full_len = 0;
  for (int cidx = 0; cidx < P.R; cidx++) {
    size_t lo, hi;
    P.chunk_range(cidx, &lo, &hi);
    const size_t len_bytes = (hi - lo) * e;
    const size_t a = std::min(off, len_bytes), b = std::min(off + P.piece_bytes, len_bytes);
    const size_t len = b - a;
    if (len == 0) continue;
    if (cidx == 0) full_len = len;
    if (len == full_len && (size_t)cidx == full_rows) {
      full_rows++;
      continue;
    }
    out->push_back(HostCopy{dev + lo * e + a, host + lo * e + a, len, len, 1});
  }
  if (full_rows > 0) out->push_back(HostCopy{dev + off, host + off, q_bytes, full_len, full_rows});
}

static cudaError_t enqueue_host_copy(const HostCopy& hc, bool to_device, cudaStream_t s) {
  const cudaMemcpyKind kind = to_device ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost;
  void* dst = to_device ? (void*)hc.dev : (void*)hc.host;
  const void* src = to_device ? (const void*)hc.host : (const void*)hc.dev;
  if (hc.rows == 1) return cudaMemcpyAsync(dst, src, hc.width, kind, s);
  return cudaMemcpy2DAsync(dst, hc.pitch, src, hc.pitch, hc.width, hc.rows, kind, s);
}

// only_piece >= 0 builds the graph of that piece alone (dependencies never cross pieces) and stores it in *out_exec.
hoccl_result_t build_graph(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry, int only_piece,
                           cudaGraphExec_t* out_exec) {
  cudaGraph_t g = nullptr;
  CU_TRY(c, cudaGraphCreate(&g, 0));
  std::vector<cudaGraphNode_t> tail(groups.size(), nullptr);
  cudaGraphNode_t last_copy_node = nullptr;
  hoccl_result_t rc = HOCCL_OK;
  auto fail = [&](cudaError_t e, const char* what) {
    rc = cuda_fail(c, e, what);
  };
  for (size_t gi = 0; gi < groups.size() && rc == HOCCL_OK; gi++) {
    if (only_piece >= 0 && P.groups[gi].piece != only_piece) continue;
    const RGroup& rg = groups[gi];
    std::vector<cudaGraphNode_t> deps;
    for (int d : rg.deps)
      if (tail[d]) deps.push_back(tail[d]);
    if (rg.chain_dep >= 0 && tail[rg.chain_dep] && std::find(rg.deps.begin(), rg.deps.end(), rg.chain_dep) == rg.deps.end())
      deps.push_back(tail[rg.chain_dep]);
    std::vector<cudaGraphNode_t> nodes;
    cudaError_t e = cudaSuccess;
    if (rg.kind == OP_SUM) {
      for (size_t first = 0; first < rg.segs.size() && e == cudaSuccess; first += kMaxSegs) {
        size_t n = std::min<size_t>(kMaxSegs, rg.segs.size() - first);
        SumBatch b;
        fill_sum_batch(rg, first, n, P.dtype, P.elem, &b);
        prepare_sum_batch(&b, (int)c->sum_ctas);
        void* args[] = {&b};
        cudaKernelNodeParams kp = {};
        int sum_threads = 0;
        kp.func = const_cast<void*>(sum_kernel_entry(P.dtype, (int)c->sum_ctas, &sum_threads));
        kp.gridDim = dim3((unsigned)c->sum_ctas);
        kp.blockDim = dim3((unsigned)sum_threads);
        kp.kernelParams = args;
        // launches of one group are chained too (they share the SM budget)
        std::vector<cudaGraphNode_t> d2 = nodes.empty() ? deps : std::vector<cudaGraphNode_t>{nodes.back()};
        cudaGraphNode_t start_rec = nullptr;
        std::pair<cudaEvent_t, cudaEvent_t> pe{nullptr, nullptr};
        if (c->profile) {
          if ((e = cudaEventCreate(&pe.first)) != cudaSuccess) break;
          if ((e = cudaEventCreate(&pe.second)) != cudaSuccess) break;
          entry->prof_events.push_back(pe);
          double bytes = 0;
          for (size_t i = 0; i < n; i++) bytes += 3.0 * (double)rg.segs[first + i].bytes;
          entry->prof_bytes.push_back(bytes);
          if ((e = cudaGraphAddEventRecordNode(&start_rec, g, d2.data(), d2.size(), pe.first)) != cudaSuccess) break;
          d2.assign(1, start_rec);
        }
        cudaGraphNode_t kn;
        e = cudaGraphAddKernelNode(&kn, g, d2.data(), d2.size(), &kp);
        if (e != cudaSuccess) break;
        cudaLaunchAttributeValue prio = {};
        prio.priority = c->sum_priority;
        e = cudaGraphKernelNodeSetAttribute(kn, cudaLaunchAttributePriority, &prio);
        if (e != cudaSuccess) break;
        if (c->profile) {
          cudaGraphNode_t end_rec;
          if ((e = cudaGraphAddEventRecordNode(&end_rec, g, &kn, 1, pe.second)) != cudaSuccess) break;
          kn = end_rec;
        }
        nodes.assign(1, kn);
        entry->n_sum_launches++;
      }
    } else if (c->path == HOCCL_PATH_CE) {
      for (const Seg& sg : rg.segs) {
        // optional sub-copies: driver copies of 4-8 MiB pay a ~4 us serialised start-up that smaller ones do not
        size_t sub = sg.bytes;
        if (c->ce_sub_bytes > 0 && sg.bytes > (size_t)c->ce_sub_bytes && sg.bytes < ((size_t)16 << 20))
          sub = ((size_t)c->ce_sub_bytes + 255) / 256 * 256;
        for (size_t off = 0; off < sg.bytes && e == cudaSuccess; off += sub) {
          cudaGraphNode_t n;
          e = cudaGraphAddMemcpyNode1D(&n, g, deps.data(), deps.size(), sg.dst + off, sg.src + off, std::min(sub, sg.bytes - off),
                                       cudaMemcpyDeviceToDevice);
          if (e != cudaSuccess) break;
          nodes.push_back(n);
          entry->n_moves++;
        }
        if (e != cudaSuccess) break;
      }
    } else if (c->path == HOCCL_PATH_CE_HOST) {
      for (const Seg& sg : rg.segs) {
        cudaGraphNode_t d2h, h2d;
        e = cudaGraphAddMemcpyNode1D(&d2h, g, deps.data(), deps.size(), c->host_staging + sg.host_off, sg.src, sg.bytes,
                                     cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) break;
        e = cudaGraphAddMemcpyNode1D(&h2d, g, &d2h, 1, sg.dst, c->host_staging + sg.host_off, sg.bytes, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) break;
        nodes.push_back(h2d);
        entry->n_moves++;
      }
    } else {
      for (size_t first = 0; first < rg.segs.size() && e == cudaSuccess; first += kMaxSegs) {
        size_t n = std::min<size_t>(kMaxSegs, rg.segs.size() - first);
        CopyBatch b;
        fill_copy_batch(rg, first, n, &b);
        prepare_copy_batch(&b, (int)c->copy_ctas);
        void* args[] = {&b};
        cudaKernelNodeParams kp = {};
        int copy_threads = 0;
        kp.func = const_cast<void*>(copy_kernel_entry((int)c->copy_ctas, &copy_threads));
        kp.gridDim = dim3((unsigned)c->copy_ctas);
        kp.blockDim = dim3((unsigned)copy_threads);
        kp.kernelParams = args;
        // copy launches are chained as well: the CTA budget for copies is global, two never run at the same time
        std::vector<cudaGraphNode_t> d2 = deps;
        if (last_copy_node && std::find(d2.begin(), d2.end(), last_copy_node) == d2.end()) d2.push_back(last_copy_node);
        std::pair<cudaEvent_t, cudaEvent_t> pe{nullptr, nullptr};
        if (c->profile) {
          if ((e = cudaEventCreate(&pe.first)) != cudaSuccess) break;
          if ((e = cudaEventCreate(&pe.second)) != cudaSuccess) break;
          entry->prof_events.push_back(pe);
          double bytes = 0;
          for (size_t i = 0; i < n; i++) bytes += 2.0 * (double)rg.segs[first + i].bytes;
          entry->prof_bytes.push_back(-bytes);   // negative: a copy launch (read + write), kept apart from the sums
          cudaGraphNode_t start_rec;
          if ((e = cudaGraphAddEventRecordNode(&start_rec, g, d2.data(), d2.size(), pe.first)) != cudaSuccess) break;
          d2.assign(1, start_rec);
        }
        cudaGraphNode_t kn;
        e = cudaGraphAddKernelNode(&kn, g, d2.data(), d2.size(), &kp);
        if (e != cudaSuccess) break;
        if (c->profile) {
          cudaGraphNode_t end_rec;
          if ((e = cudaGraphAddEventRecordNode(&end_rec, g, &kn, 1, pe.second)) != cudaSuccess) break;
          kn = end_rec;
        }
        last_copy_node = kn;
        nodes.push_back(kn);
        entry->n_moves += (long)n;
        entry->n_move_launches++;
      }
    }
    if (e != cudaSuccess) {
      fail(e, "graph node");
      break;
    }
    if (nodes.size() == 1) {
      tail[gi] = nodes[0];
    } else if (nodes.size() > 1) {
      cudaGraphNode_t join;
      e = cudaGraphAddEmptyNode(&join, g, nodes.data(), nodes.size());
      if (e != cudaSuccess) {
        fail(e, "graph join node");
        break;
      }
      tail[gi] = join;
    }
  }
  if (rc == HOCCL_OK) {
    cudaError_t e = cudaGraphInstantiate(out_exec, g, 0);
    if (e != cudaSuccess) rc = cuda_fail(c, e, "cudaGraphInstantiate");
  }
  cudaGraphDestroy(g);
  if (rc != HOCCL_OK) destroy_entry(entry);
  return rc;
}

// Inserts an entry into the graph cache (evicting the least recently used one when it is full) and returns it.
GraphEntry* cache_put(hoccl_comm* c, GraphEntry&& entry) {
  if (c->cache.size() >= kGraphCacheCap) {
    if (c->proxy) c->proxy->drain(c->watchdog_ms);  // a queued hand-over may still refer to the victim
    size_t victim = 0;
    for (size_t i = 1; i < c->cache.size(); i++)
      if (c->cache[i].last_use < c->cache[victim].last_use) victim = i;
    destroy_entry(&c->cache[victim]);
    c->cache.erase(c->cache.begin() + victim);
  }
  c->cache.push_back(std::move(entry));
  return &c->cache.back();
}

// The schedule of a user-defined pattern (paper Sec. 3.4) as a CUDA graph: stages one after the other (a join node between
// them), inside a stage every source rank's queue is a serial chain in the scheduler's service order (copy route), or the
// k-th operations of all queues share one batched copy launch and the launches form one chain (SM path).
hoccl_result_t build_pattern_graph(hoccl_comm* c, const Schedule& S, const void* const* send, const size_t* sdispls, void* const* recv,
                                   const size_t* rdispls, size_t e, GraphEntry* entry) {
  const int R = c->R;
  cudaGraph_t g = nullptr;
  CU_TRY(c, cudaGraphCreate(&g, 0));
  cudaError_t err = cudaSuccess;
  cudaGraphNode_t stage_dep = nullptr;
  for (size_t si = 0; si < S.stages.size() && err == cudaSuccess; si++) {
    const Stage& st = S.stages[si];
    auto endpoints = [&](const ChunkItem& it, const char** src, char** dst) {
      const StageFlow& f = st.flows[it.flow];
      *src = (const char*)send[f.origin_src] + sdispls[(size_t)f.origin_src * R + f.origin_dst] * e + f.origin_offset + it.offset;
      *dst = (char*)recv[f.origin_dst] + rdispls[(size_t)f.origin_dst * R + f.origin_src] * e + f.origin_offset + it.offset;
    };
    // chunks that follow one another in a queue and continue the same flow are one operation
    std::vector<std::vector<ChunkItem>> queues(R);
    for (int q = 0; q < R; q++)
      for (const ChunkItem& it : st.queues[q]) {
        if (!queues[q].empty() && queues[q].back().flow == it.flow && queues[q].back().offset + queues[q].back().bytes == it.offset)
          queues[q].back().bytes += it.bytes;
        else
          queues[q].push_back(it);
      }
    std::vector<cudaGraphNode_t> tails;
    if (c->path == HOCCL_PATH_CE) {
      for (int q = 0; q < R && err == cudaSuccess; q++) {
        cudaGraphNode_t prev = stage_dep;
        for (const ChunkItem& it : queues[q]) {
          const char* src;
          char* dst;
          endpoints(it, &src, &dst);
          cudaGraphNode_t n;
          err = cudaGraphAddMemcpyNode1D(&n, g, prev ? &prev : nullptr, prev ? 1 : 0, dst, src, it.bytes, cudaMemcpyDeviceToDevice);
          if (err != cudaSuccess) break;
          prev = n;
          entry->n_moves++;
        }
        if (prev && prev != stage_dep) tails.push_back(prev);
      }
    } else {
      size_t depth = 0;
      for (int q = 0; q < R; q++) depth = std::max(depth, queues[q].size());
      cudaGraphNode_t prev = stage_dep;
      auto add_launch = [&](CopyBatch& b) {
        prepare_copy_batch(&b, (int)c->copy_ctas);
        void* args[] = {&b};
        cudaKernelNodeParams kp = {};
        int threads = 0;
        kp.func = const_cast<void*>(copy_kernel_entry((int)c->copy_ctas, &threads));
        kp.gridDim = dim3((unsigned)c->copy_ctas);
        kp.blockDim = dim3((unsigned)threads);
        kp.kernelParams = args;
        cudaGraphNode_t n;
        err = cudaGraphAddKernelNode(&n, g, prev ? &prev : nullptr, prev ? 1 : 0, &kp);
        if (err == cudaSuccess) {
          prev = n;
          entry->n_move_launches++;
        }
        b.nseg = 0;
      };
      for (size_t k = 0; k < depth && err == cudaSuccess; k++) {
        CopyBatch b;
        b.nseg = 0;
        b.pad = 0;
        for (int q = 0; q < R && err == cudaSuccess; q++) {
          if (k >= queues[q].size()) continue;
          const char* src;
          char* dst;
          endpoints(queues[q][k], &src, &dst);
          b.seg[b.nseg++] = CopySeg{src, dst, (unsigned long long)queues[q][k].bytes};
          entry->n_moves++;
          if (b.nseg == kMaxSegs) add_launch(b);
        }
        if (b.nseg > 0 && err == cudaSuccess) add_launch(b);
      }
      if (prev && prev != stage_dep) tails.push_back(prev);
    }
    if (err != cudaSuccess) break;
    if (tails.size() == 1) {
      stage_dep = tails[0];
    } else if (tails.size() > 1) {
      cudaGraphNode_t join;
      err = cudaGraphAddEmptyNode(&join, g, tails.data(), tails.size());
      if (err == cudaSuccess) stage_dep = join;
    }
  }
  hoccl_result_t rc = HOCCL_OK;
  if (err == cudaSuccess) err = cudaGraphInstantiate(&entry->exec, g, 0);
  if (err != cudaSuccess) rc = cuda_fail(c, err, "pattern graph");
  cudaGraphDestroy(g);
  entry->n_pieces = (long)S.stages.size();
  if (rc != HOCCL_OK) destroy_entry(entry);
  return rc;
}

std::vector<uint64_t> make_key(hoccl_comm* c, const Call& call) {
  std::vector<uint64_t> k;
  k.reserve(17 + 2 * c->R);
  k.push_back((uint64_t)call.kind);
  k.push_back((uint64_t)call.count);
  k.push_back((uint64_t)call.dtype);
  k.push_back((uint64_t)c->path);
  k.push_back((uint64_t)c->sum_ctas);
  k.push_back((uint64_t)c->copy_ctas);
  k.push_back((uint64_t)c->piece_bytes);
  k.push_back((uint64_t)c->piece_bytes_set);
  k.push_back((uint64_t)c->max_pieces);
  k.push_back((uint64_t)c->profile);
  k.push_back((uint64_t)c->ce_sub_bytes);
  k.push_back((uint64_t)c->forward);
  k.push_back((uint64_t)(c->fused && c->path == HOCCL_PATH_SM && !c->handshake));
  k.push_back((uint64_t)(uintptr_t)c->scratch);
  k.push_back((uint64_t)c->scratch_bytes);
  k.push_back((uint64_t)(uintptr_t)c->host_staging);
  k.push_back((uint64_t)c->host_staging_bytes);
  for (int r = 0; r < c->R; r++) {
    k.push_back((uint64_t)(uintptr_t)call.send[r]);
    k.push_back((uint64_t)(uintptr_t)call.recv[r]);
  }
  k.push_back(call.h_send ? (uint64_t)c->host_pieces : 0);
  if (call.h_send)
    for (int r = 0; r < c->R; r++) {
      k.push_back((uint64_t)(uintptr_t)call.h_send[r]);
      k.push_back((uint64_t)(uintptr_t)call.h_recv[r]);
    }
  return k;
}

// reads back the profile events of finished work (the caller has synchronised)
void harvest_profile(hoccl_comm* c) {
  for (auto& rec : c->prof_open) {
    float ms = 0;
    if (cudaEventElapsedTime(&ms, rec.first.first, rec.first.second) == cudaSuccess) {
      c->prof_ms += ms;
      c->prof_bytes += rec.second;
      c->prof_n++;
    }
    c->prof_pool.push_back(rec.first);
  }
  c->prof_open.clear();
  // cached graphs keep their own events; a replay overwrites them, so only the latest replay is readable
  for (auto& e : c->cache) {
    if (!e.prof_pending) continue;
    e.prof_pending = false;
    for (size_t i = 0; i < e.prof_events.size(); i++) {
      float ms = 0;
      if (cudaEventElapsedTime(&ms, e.prof_events[i].first, e.prof_events[i].second) == cudaSuccess) {
        if (e.prof_bytes[i] < 0) {
          c->prof_copy_ms += ms;
          c->prof_copy_bytes -= e.prof_bytes[i];
          c->prof_copy_n++;
        } else {
          c->prof_ms += ms;
          c->prof_bytes += e.prof_bytes[i];
          c->prof_n++;
        }
      }
    }
  }
}

// The CPU proxy of the handshake mode is created on first use.
hoccl_result_t ensure_proxy(hoccl_comm* c) {
  if (c->proxy) {
    c->proxy->set_watchdog_ms(c->watchdog_ms);
    return HOCCL_OK;
  }
  Proxy* p = new Proxy(c->device, c->watchdog_ms);
  cudaError_t e = p->init();
  if (e != cudaSuccess) {
    delete p;
    return cuda_fail(c, e, "proxy init (stream memory operations)");
  }
  c->proxy = p;
  return HOCCL_OK;
}

// ------------------------------------------------------------------ whole-collective kernel ------
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
static hoccl_result_t build_ring(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry) {
  hoccl_result_t rc = ensure_ring_ctrl(c);
  if (rc != HOCCL_OK) return rc;
  size_t max_phase_bytes = 0;
  bool has_sum = false;
  for (const RGroup& g : groups) has_sum = has_sum || g.kind == OP_SUM;
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

// Replays a cached graph into the caller's stream (directly, or through the CPU proxy in handshake mode).
static hoccl_result_t launch_entry(hoccl_comm* c, GraphEntry* hit, cudaStream_t user, double t0) {
  hit->last_use = ++c->use_counter;
  if (!hit->ring_args.empty()) {
    if (hit->ring_large)
      CU_TRY(c, launch_ring(*reinterpret_cast<const RingArgsLarge*>(hit->ring_args.data()), hit->ring_grid, hit->ring_threads, user));
    else
      CU_TRY(c, launch_ring(*reinterpret_cast<const RingArgsSmall*>(hit->ring_args.data()), hit->ring_grid, hit->ring_threads, user));
    c->stats.n_pieces = hit->n_pieces;
    c->stats.n_moves = hit->n_moves;
    c->stats.n_move_launches = 1;
    c->stats.n_sum_launches = 0;
    c->stats.max_copy_ctas = hit->ring_grid;
    c->stats.max_sum_ctas = hit->ring_has_sum ? hit->ring_grid : 0;
    c->stats.host_launch_us = now_us() - t0;
    return HOCCL_OK;
  }
  if (!hit->piece_exec.empty()) {
    // Pipelined host all-reduce: the inbound copies run on one internal stream, the outbound copies on another, and the
    // caller's stream runs the ring piece by piece as each piece arrives; PCIe carries both directions at once.
    cudaStream_t in = c->lane[0], out = c->lane[1];
    c->ev_next = 0;
    cudaEvent_t fork = next_event(c);
    if (!fork) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    CU_TRY(c, cudaEventRecord(fork, user));
    CU_TRY(c, cudaStreamWaitEvent(in, fork, 0));
    CU_TRY(c, cudaStreamWaitEvent(out, fork, 0));
    const size_t np = hit->piece_exec.size();
    std::vector<cudaEvent_t> arrived(np, nullptr);
    for (size_t p = 0; p < np; p++) {
      for (const HostCopy& hc : hit->h2d[p]) CU_TRY(c, enqueue_host_copy(hc, true, in));
      arrived[p] = next_event(c);
      if (!arrived[p]) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
      CU_TRY(c, cudaEventRecord(arrived[p], in));
    }
    for (size_t p = 0; p < np; p++) {
      CU_TRY(c, cudaStreamWaitEvent(user, arrived[p], 0));
      if (hit->piece_exec[p]) CU_TRY(c, cudaGraphLaunch(hit->piece_exec[p], user));
      cudaEvent_t reduced = next_event(c);
      if (!reduced) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
      CU_TRY(c, cudaEventRecord(reduced, user));
      CU_TRY(c, cudaStreamWaitEvent(out, reduced, 0));
      for (const HostCopy& hc : hit->d2h[p]) CU_TRY(c, enqueue_host_copy(hc, false, out));
    }
    cudaEvent_t done = next_event(c);
    if (!done) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    CU_TRY(c, cudaEventRecord(done, out));
    CU_TRY(c, cudaStreamWaitEvent(user, done, 0));
  } else if (c->handshake) {
    // paper Sec. 3.2: the stream hands itself to the CPU proxy, which runs the schedule and hands it back
    ProxyTask t;
    t.kind = ProxyTask::GRAPH;
    t.exec = hit->exec;
    CU_TRY(c, c->proxy->submit(user, t));
  } else {
    CU_TRY(c, cudaGraphLaunch(hit->exec, user));
  }
  hit->prof_pending = !hit->prof_events.empty();
  c->stats.n_pieces = hit->n_pieces;
  c->stats.n_moves = hit->n_moves;
  c->stats.n_move_launches = hit->n_move_launches;
  c->stats.n_sum_launches = hit->n_sum_launches;
  c->stats.max_sum_ctas = hit->n_sum_launches ? c->sum_ctas : 0;
  c->stats.max_copy_ctas = hit->n_move_launches ? c->copy_ctas : 0;
  c->stats.host_launch_us = now_us() - t0;
  return HOCCL_OK;
}

hoccl_result_t run_collective(hoccl_comm* c, Call* call, cudaStream_t user) {
  const double t0 = now_us();
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (dtype_size(call->dtype) == 0) return HOCCL_ERR_UNSUPPORTED;
  if (!call->send || !call->recv) return HOCCL_ERR_INVALID_ARG;
  const bool onepass_case = c->onepass && !c->handshake && (call->kind == PLAN_ALLREDUCE || call->kind == PLAN_REDUCE_SCATTER);
  const bool fused = c->fused && c->path == HOCCL_PATH_SM && !c->handshake && !onepass_case && !call->h_send;
  const bool graphs = (c->use_graph || c->handshake || fused) && !onepass_case;
  std::vector<uint64_t> key;
  if (graphs && call->count != 0) {
    // Fast path: a call whose signature (operation, count, dtype, every pointer, every setting that shapes the graph)
    // was seen before was validated and planned then; replaying its graph is all that is left to do.
    if (c->handshake && c->path != HOCCL_PATH_SM) return HOCCL_ERR_UNSUPPORTED;
    key = make_key(c, *call);
    for (auto& e : c->cache)
      if (e.key == key) {
        c->stats = hoccl_stats_t{};
        c->stats.graph_hit = 1;
        CU_TRY(c, cudaSetDevice(c->device));
        if (c->handshake) {
          hoccl_result_t prc = ensure_proxy(c);
          if (prc != HOCCL_OK) return prc;
        }
        return launch_entry(c, &e, user, t0);
      }
  }
  hoccl_result_t rc = validate(c, call);
  if (rc != HOCCL_OK) return rc;
  c->stats = hoccl_stats_t{};
  if (call->count == 0) return HOCCL_OK;
  CU_TRY(c, cudaSetDevice(c->device));

  if (c->onepass && !c->handshake && (call->kind == PLAN_ALLREDUCE || call->kind == PLAN_REDUCE_SCATTER)) {
    // comparison point: the whole reduction in one kernel, same order and rounding as the ring, no moves, no scratch
    OnePassArgs a;
    a.R = c->R;
    a.dtype = call->dtype;
    a.write_all = call->kind == PLAN_ALLREDUCE ? 1 : 0;
    a.pad = 0;
    if (call->kind == PLAN_ALLREDUCE) {
      a.count = call->count;
      a.q = (call->count + (size_t)c->R - 1) / (size_t)c->R;
    } else {
      a.count = (unsigned long long)call->count * c->R;
      a.q = call->count;
    }
    for (int r = 0; r < c->R; r++) {
      a.x[r] = call->send[r];
      a.y[r] = call->recv[r];
    }
    CU_TRY(c, launch_onepass(a, (int)c->sum_ctas, user));
    c->stats.n_sum_launches = 1;
    c->stats.max_sum_ctas = c->sum_ctas;
    c->stats.n_pieces = 1;
    c->stats.host_launch_us = now_us() - t0;
    return HOCCL_OK;
  }
  Plan P;
  unsigned char align[kMaxRanks];
  for (int r = 0; r < c->R; r++) align[r] = (unsigned char)((uintptr_t)call->send[r] & 15);
  int plan_kind = call->kind;
  if (c->forward && call->kind == PLAN_ALLREDUCE) plan_kind = PLAN_ALLREDUCE_FWD;
  if (c->forward && call->kind == PLAN_REDUCE_SCATTER) plan_kind = PLAN_REDUCE_SCATTER_FWD;
  // Piece size: the caller's, else 4 MiB; on the SM path under CTA budgets a reduction is cut into at least two pieces
  // (the copy kernel of one piece then overlaps the sum kernel of the other: measured 1.6x on a 3 MiB chunk with 8 + 8
  // CTAs), which does not pay with driver copies or whole-GPU grids.
  size_t piece_bytes = (size_t)c->piece_bytes;
  int max_pieces = (int)c->max_pieces;
  if (call->h_send) {   // pipelined host all-reduce: host_pieces pieces per chunk, whatever the chunk size
    const size_t q = (call->count + c->R - 1) / c->R;
    const size_t chunk = q * dtype_size(call->dtype);
    max_pieces = (int)c->host_pieces;
    piece_bytes = std::max<size_t>((size_t)64 << 10, ((chunk + max_pieces - 1) / max_pieces + 1023) / 1024 * 1024);
  } else if (fused) {   // one kernel walks the steps in order; whole chunks measured faster than pieces (fewer barriers and tails)
    piece_bytes = (size_t)1 << 60;
    max_pieces = 1;
  } else if (!c->piece_bytes_set && c->path == HOCCL_PATH_SM && std::max(c->sum_ctas, c->copy_ctas) < 64 &&
      (call->kind == PLAN_ALLREDUCE || call->kind == PLAN_REDUCE_SCATTER)) {
    const size_t q = call->kind == PLAN_ALLREDUCE ? (call->count + c->R - 1) / c->R : call->count;
    const size_t chunk = q * dtype_size(call->dtype);
    if (chunk >= ((size_t)1 << 20)) piece_bytes = std::min(piece_bytes, (chunk / 2 + 1023) / 1024 * 1024);
  }
  if (!build_plan(&P, plan_kind, c->R, call->count, call->dtype, call->in_place, piece_bytes, max_pieces, align))
    return HOCCL_ERR_INVALID_ARG;
  if (P.slot_bytes) {
    size_t need = 2 * (size_t)c->R * P.slot_bytes;
    if (!c->scratch || c->scratch_bytes < need) return HOCCL_ERR_SCRATCH;
    // scratch must not overlap any rank buffer
    for (int r = 0; r < c->R; r++)
      if (ranges_overlap((const char*)c->scratch, need, (const char*)call->send[r], call->send_bytes) ||
          ranges_overlap((const char*)c->scratch, need, (const char*)call->recv[r], call->recv_bytes))
        return HOCCL_ERR_INVALID_ARG;
  }
  c->stats.n_pieces = P.pieces;
  c->stats.max_sum_ctas = 0;
  std::vector<RGroup> groups;
  size_t host_need = 0;
  resolve(c, P, *call, &groups, &host_need);
  if (c->path == HOCCL_PATH_CE_HOST && (!c->host_staging || host_need > c->host_staging_bytes)) return HOCCL_ERR_SCRATCH;
  if (graphs) {
    if (c->handshake) {
      // Driver copies share a hardware queue with the copies the parked stream has queued behind its hand-over; a copy
      // issued by the proxy can end up behind them and never start (observed).  Kernels do not have that problem.
      // (Checked before the cache lookup; the proxy is created on first use.)
      rc = ensure_proxy(c);
      if (rc != HOCCL_OK) return rc;
    }
    GraphEntry entry;
    entry.key = key;
    entry.n_pieces = P.pieces;
    if (call->h_send) {
      entry.piece_exec.assign(P.pieces, nullptr);
      entry.h2d.resize(P.pieces);
      entry.d2h.resize(P.pieces);
      for (int p = 0; p < P.pieces; p++) {
        for (int r = 0; r < c->R; r++) {
          add_host_copies(P, p, (char*)call->send[r], (char*)call->h_send[r], &entry.h2d[p]);
          add_host_copies(P, p, (char*)call->recv[r], (char*)call->h_recv[r], &entry.d2h[p]);
        }
        bool any = false;
        for (const PlanGroup& pg : P.groups) any = any || pg.piece == p;
        if (!any) continue;   // e.g. one rank copying in place: nothing to run between the copies
        rc = build_graph(c, P, groups, &entry, p, &entry.piece_exec[p]);
        if (rc != HOCCL_OK) return rc;
      }
    } else {
      rc = fused ? build_ring(c, P, groups, &entry) : HOCCL_ERR_UNSUPPORTED;
      if (rc == HOCCL_ERR_UNSUPPORTED) rc = build_graph(c, P, groups, &entry, -1, &entry.exec);   // not asked for, or too many ranks for one launch
      if (rc != HOCCL_OK) return rc;
    }
    // handshake mode: place the graph on the device now; the proxy must not meet first-launch work later
    if (c->handshake) {
      cudaError_t ue = cudaGraphUpload(entry.exec, c->proxy->work_stream());
      if (ue != cudaSuccess) {
        destroy_entry(&entry);
        return cuda_fail(c, ue, "cudaGraphUpload");
      }
    }
    return launch_entry(c, cache_put(c, std::move(entry)), user, t0);
  }
  Tally tally;
  rc = run_streams(c, P, groups, user, &tally);
  if (rc != HOCCL_OK) return rc;
  c->stats.n_moves = tally.moves;
  c->stats.n_move_launches = tally.move_launches;
  c->stats.n_sum_launches = tally.sum_launches;
  c->stats.max_sum_ctas = tally.sum_launches ? c->sum_ctas : 0;
  c->stats.max_copy_ctas = tally.move_launches ? c->copy_ctas : 0;
  c->stats.host_launch_us = now_us() - t0;
  return HOCCL_OK;
}

}  // namespace hoccl
