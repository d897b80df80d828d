// Graph side of libhoccl: a resolved plan (or the schedule of a user-defined pattern) becomes an explicit CUDA graph:
// memcpy nodes for moves on the copy route, kernel nodes for sums and SM copies, empty nodes as joins.  Also the graph
// cache and the host copies of the pipelined host all-reduce.
#include <tuple>

#include "comm.h"

namespace hoccl {

void destroy_entry(GraphEntry* e) {
  if (e->exec) cudaGraphExecDestroy(e->exec);
  for (cudaGraphExec_t pe : e->piece_exec)
    if (pe) cudaGraphExecDestroy(pe);
  e->piece_exec.clear();
  for (cudaGraphExec_t pe : e->part_exec)
    if (pe) cudaGraphExecDestroy(pe);
  e->part_exec.clear();
  for (auto& p : e->prof_events) {
    cudaEventDestroy(p.first);
    cudaEventDestroy(p.second);
  }
  e->exec = nullptr;
  e->prof_events.clear();
  if (e->roles_tab) {
    cudaFree(e->roles_tab);   // waits for launches still in flight
    e->roles_tab = nullptr;
    e->roles_fn = nullptr;
  }
}

// Host <-> staging copies of one piece of one rank (all-reduce layout): piece p of every ring chunk, i.e. rows of
// `piece` bytes at a pitch of one chunk.  Chunks that hold the full piece go as one 2-D copy; a shorter trailing piece
// as a 1-D copy.
void add_host_copies(const Plan& P, int p, char* dev, char* host, std::vector<HostCopy>* out) {
  const size_t e = P.elem, q_bytes = P.chunk_elems * e;
  const size_t off = (size_t)P.piece_off[(size_t)p], end = (size_t)P.piece_off[(size_t)p + 1];
  size_t full_rows = 0, full_len = 0;
  for (int cidx = 0; cidx < P.R; cidx++) {
    size_t lo, hi;
    P.chunk_range(cidx, &lo, &hi);
    const size_t len_bytes = (hi - lo) * e;
    const size_t a = std::min(off, len_bytes), b = std::min(end, len_bytes);
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

cudaError_t enqueue_host_copy(const HostCopy& hc, bool to_device, cudaStream_t s) {
  const cudaMemcpyKind kind = to_device ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost;
  void* dst = to_device ? (void*)hc.dev : (void*)hc.host;
  const void* src = to_device ? (const void*)hc.host : (const void*)hc.dev;
  if (hc.rows == 1) return cudaMemcpyAsync(dst, src, hc.width, kind, s);
  return cudaMemcpy2DAsync(dst, hc.pitch, src, hc.pitch, hc.width, hc.rows, kind, s);
}

// only_piece >= 0 builds the graph of that piece alone (dependencies never cross pieces) and stores it in *out_exec.
hoccl_result_t build_graph(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry, int only_piece,
                           cudaGraphExec_t* out_exec, int part) {
  // which groups this graph holds
  auto included = [&](size_t gi) {
    const RGroup& rg = groups[gi];
    if (only_piece >= 0 && rg.piece != only_piece) return false;
    if (part < 0) return true;
    const int cls = rg.kind != OP_MOVE ? 1 : (rg.phase == PHASE_RS ? 0 : 2);
    return cls == part;
  };
  {
    bool any = false;
    for (size_t gi = 0; gi < groups.size(); gi++) any = any || (included(gi) && !groups[gi].segs.empty());
    if (!any && part >= 0) {
      *out_exec = nullptr;
      return HOCCL_OK;
    }
  }
  cudaGraph_t g = nullptr;
  CU_TRY(c, cudaGraphCreate(&g, 0));
  std::vector<std::vector<cudaGraphNode_t>> tail(groups.size());   // the node(s) a consumer of the group waits for
  cudaGraphNode_t last_copy_node = nullptr;
  // Copy nodes without a predecessor each wait for the stream's earlier work on their own, which costs ~4 us per node when
  // that work is still running (measured behind a reduce-scatter: 240 instead of 65 us for the 56 root copies of a direct
  // all-gather of the gradient bucket; back-to-back 4 KiB all-to-alls: 65 us per call instead of 24).  One empty kernel as
  // their common predecessor takes that wait once (an empty graph node does not: it changes nothing).
  cudaGraphNode_t root = nullptr;
  bool many_root_copies = false;
  auto inner_deps = [&](size_t gi) {   // dependencies of group gi on groups of this graph
    size_t n = 0;
    for (int d : groups[gi].deps) n += included((size_t)d) ? 1 : 0;
    if (groups[gi].chain_dep >= 0 && included((size_t)groups[gi].chain_dep)) n++;
    return n;
  };
  if (c->order_kernels && (c->path == HOCCL_PATH_CE || c->path == HOCCL_PATH_CE_HOST)) {
    size_t n_root = 0;
    for (size_t gi = 0; gi < groups.size(); gi++)
      if (included(gi) && groups[gi].kind == OP_MOVE && inner_deps(gi) == 0) n_root += groups[gi].segs.size();
    many_root_copies = n_root >= 2;
  }
  // The same holds behind a group of copies: copy nodes (or the end of the graph) that wait for several copy nodes start
  // late; an empty kernel as the join of such a group fixes it (ring all-gather of the gradient bucket, seven stages of eight
  // copies: 88 -> 68 us; the 56 copies of the direct one: 61 -> 51 us).  A SUM kernel that waits for its copies directly does
  // not need it (a kernel in between costs ~1 us per step there), so groups that only feed SUMs keep the empty join.
  std::vector<char> kernel_join(groups.size(), 0), terminal(groups.size(), 0);
  if (c->order_kernels && (c->path == HOCCL_PATH_CE || c->path == HOCCL_PATH_CE_HOST)) {
    std::vector<char> move_user(groups.size(), 0), any_user(groups.size(), 0);
    for (size_t gi = 0; gi < groups.size(); gi++) {
      if (!included(gi)) continue;
      for (int d : groups[gi].deps) {
        any_user[d] = 1;
        if (groups[gi].kind == OP_MOVE) move_user[d] = 1;
      }
    }
    // groups of copies that nothing in this graph waits for share ONE such kernel at the end of the graph (one per group cost
    // 2 us of kernel time each and bought nothing more)
    for (size_t gi = 0; gi < groups.size(); gi++) {
      kernel_join[gi] = groups[gi].kind == OP_MOVE && move_user[gi];
      terminal[gi] = groups[gi].kind == OP_MOVE && !any_user[gi];
    }
  }
  std::vector<cudaGraphNode_t> terminal_nodes;
  hoccl_result_t rc = HOCCL_OK;
  auto fail = [&](cudaError_t e, const char* what) {
    rc = cuda_fail(c, e, what);
  };
  // Issue order.  Copy launches of the SM path form one chain (the CTA budget for copies is global), so the order in which
  // the groups are added is the order in which their copies run.  For the direct schedule cut into pieces the plan lists a
  // piece's reduce-scatter moves, its sum and its all-gather moves together; taken in that order the next piece's moves would
  // wait behind this piece's all-gather, which waits for this piece's sum: nothing would overlap.  So the moves are ordered
  // as a software pipeline: RS(0), RS(1), AG(0), RS(2), AG(1), ...; every dependency still points to an earlier position.
  std::vector<size_t> order(groups.size());
  for (size_t gi = 0; gi < groups.size(); gi++) order[gi] = gi;
  if (c->path == HOCCL_PATH_SM && P.rs_direct && P.pieces > 1 && only_piece < 0 && part < 0) {
    auto key = [&](size_t gi) {
      const RGroup& rg = groups[gi];
      const long p = rg.piece;
      if (rg.kind != OP_MOVE) return 8 * p + 2;
      return rg.phase == PHASE_RS ? 8 * p : 8 * p + 9;
    };
    std::stable_sort(order.begin(), order.end(), [&](size_t a, size_t b) { return key(a) < key(b); });
  }
  for (size_t oi = 0; oi < order.size() && rc == HOCCL_OK; oi++) {
    const size_t gi = order[oi];
    if (!included(gi)) continue;
    const RGroup& rg = groups[gi];
    std::vector<cudaGraphNode_t> deps;   // groups outside this graph have no tail here: their order is the caller's (events)
    for (int d : rg.deps)
      deps.insert(deps.end(), tail[d].begin(), tail[d].end());
    if (rg.chain_dep >= 0 && std::find(rg.deps.begin(), rg.deps.end(), rg.chain_dep) == rg.deps.end())
      deps.insert(deps.end(), tail[rg.chain_dep].begin(), tail[rg.chain_dep].end());
    std::vector<cudaGraphNode_t> nodes;
    cudaError_t e = cudaSuccess;
    if (deps.empty() && many_root_copies && rg.kind == OP_MOVE) {
      if (!root) {
        cudaKernelNodeParams kp = {};
        kp.func = const_cast<void*>(graph_root_kernel_entry());
        kp.gridDim = dim3(1);
        kp.blockDim = dim3(32);
        kp.kernelParams = nullptr;
        e = cudaGraphAddKernelNode(&root, g, nullptr, 0, &kp);
        if (e != cudaSuccess) {
          fail(e, "graph root node");
          break;
        }
        entry->n_order_launches++;
      }
      deps.push_back(root);
    }
    if (rg.kind == OP_SUM || rg.kind == OP_CHAIN) {
      for (size_t first = 0; first < rg.segs.size() && e == cudaSuccess; first += kMaxSegs) {
        size_t n = std::min<size_t>(kMaxSegs, rg.segs.size() - first);
        SumBatch b;
        ChainBatch cb;
        void* args[1];
        cudaKernelNodeParams kp = {};
        int sum_threads = 0;
        double bytes = 0;
        if (rg.kind == OP_SUM) {
          fill_sum_batch(rg, first, n, P.dtype, P.elem, &b);
          prepare_sum_batch(&b, (int)c->sum_ctas);
          args[0] = &b;
          kp.func = const_cast<void*>(sum_kernel_entry(P.dtype, (int)c->sum_ctas, &sum_threads));
          for (size_t i = 0; i < n; i++) bytes += 3.0 * (double)rg.segs[first + i].bytes;
        } else {
          fill_chain_batch(rg, first, n, P.dtype, P.elem, &cb);
          prepare_chain_batch(&cb, (int)c->sum_ctas);
          args[0] = &cb;
          kp.func = const_cast<void*>(chain_kernel_entry(cb, (int)c->sum_ctas, &sum_threads));
          for (size_t i = 0; i < n; i++) bytes += (2.0 + (double)rg.segs[first + i].nsrc) * (double)rg.segs[first + i].bytes;
        }
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
      std::map<uint64_t, cudaGraphNode_t> outbound;   // staging offset -> the outbound copy that fills it
      for (const Seg& sg : rg.segs) {
        cudaGraphNode_t d2h, h2d;
        if (sg.host_first) {
          e = cudaGraphAddMemcpyNode1D(&d2h, g, deps.data(), deps.size(), c->host_staging + sg.host_off, sg.src, sg.bytes,
                                       cudaMemcpyDeviceToHost);
          if (e != cudaSuccess) break;
          outbound[sg.host_off] = d2h;
        } else {
          d2h = outbound[sg.host_off];   // filled by an earlier move of this group (same source, same bytes)
        }
        e = cudaGraphAddMemcpyNode1D(&h2d, g, &d2h, 1, sg.dst, c->host_staging + sg.host_off, sg.bytes, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) break;
        nodes.push_back(h2d);
        entry->n_moves++;
      }
    } else {
      // one kernel node per batch; `batch` is copied into the node when it is added
      auto add_move_node = [&](void* batch, const void* func, int threads, double hbm_bytes, long n_moves) -> cudaError_t {
        void* args[] = {batch};
        cudaKernelNodeParams kp = {};
        kp.func = const_cast<void*>(func);
        kp.gridDim = dim3((unsigned)c->copy_ctas);
        kp.blockDim = dim3((unsigned)threads);
        kp.kernelParams = args;
        // copy launches are chained as well: the CTA budget for copies is global, two never run at the same time
        std::vector<cudaGraphNode_t> d2 = deps;
        if (last_copy_node && std::find(d2.begin(), d2.end(), last_copy_node) == d2.end()) d2.push_back(last_copy_node);
        std::pair<cudaEvent_t, cudaEvent_t> pe{nullptr, nullptr};
        cudaError_t err;
        if (c->profile) {
          if ((err = cudaEventCreate(&pe.first)) != cudaSuccess) return err;
          if ((err = cudaEventCreate(&pe.second)) != cudaSuccess) return err;
          entry->prof_events.push_back(pe);
          entry->prof_bytes.push_back(-hbm_bytes);   // negative: a copy launch (reads + writes), kept apart from the sums
          cudaGraphNode_t start_rec;
          if ((err = cudaGraphAddEventRecordNode(&start_rec, g, d2.data(), d2.size(), pe.first)) != cudaSuccess) return err;
          d2.assign(1, start_rec);
        }
        cudaGraphNode_t kn;
        if ((err = cudaGraphAddKernelNode(&kn, g, d2.data(), d2.size(), &kp)) != cudaSuccess) return err;
        if (c->profile) {
          cudaGraphNode_t end_rec;
          if ((err = cudaGraphAddEventRecordNode(&end_rec, g, &kn, 1, pe.second)) != cudaSuccess) return err;
          kn = end_rec;
        }
        last_copy_node = kn;
        nodes.push_back(kn);
        entry->n_moves += n_moves;
        entry->n_move_launches++;
        return cudaSuccess;
      };
      std::vector<FanBatch> fans;
      std::vector<double> fan_bytes;
      std::vector<long> fan_moves;
      int move_threads = 0;
      if (P.ag_direct && build_fan_batches(rg, &fans, &fan_bytes, &fan_moves)) {
        const void* fn = fan_kernel_entry((int)c->copy_ctas, &move_threads);
        for (size_t i = 0; i < fans.size() && e == cudaSuccess; i++) {
          prepare_fan_batch(&fans[i], (int)c->copy_ctas);
          e = add_move_node(&fans[i], fn, move_threads, fan_bytes[i], fan_moves[i]);
        }
      } else {
        const void* fn = copy_kernel_entry((int)c->copy_ctas, &move_threads);
        for (size_t first = 0; first < rg.segs.size() && e == cudaSuccess; first += kMaxSegs) {
          size_t n = std::min<size_t>(kMaxSegs, rg.segs.size() - first);
          CopyBatch b;
          fill_copy_batch(rg, first, n, &b);
          prepare_copy_batch(&b, (int)c->copy_ctas);
          double bytes = 0;
          for (size_t i = 0; i < n; i++) bytes += 2.0 * (double)rg.segs[first + i].bytes;
          e = add_move_node(&b, fn, move_threads, bytes, (long)n);
        }
      }
    }
    if (e != cudaSuccess) {
      fail(e, "graph node");
      break;
    }
    if (terminal[gi]) {
      terminal_nodes.insert(terminal_nodes.end(), nodes.begin(), nodes.end());
    } else if (nodes.size() == 1) {
      tail[gi].assign(1, nodes[0]);
    } else if (nodes.size() > 1) {
      cudaGraphNode_t join;
      if (kernel_join[gi]) {
        cudaKernelNodeParams kp = {};
        kp.func = const_cast<void*>(graph_root_kernel_entry());
        kp.gridDim = dim3(1);
        kp.blockDim = dim3(32);
        kp.kernelParams = nullptr;
        e = cudaGraphAddKernelNode(&join, g, nodes.data(), nodes.size(), &kp);
        if (e == cudaSuccess) entry->n_order_launches++;
      } else {
        e = cudaGraphAddEmptyNode(&join, g, nodes.data(), nodes.size());
      }
      if (e != cudaSuccess) {
        fail(e, "graph join node");
        break;
      }
      tail[gi].assign(1, join);
    }
  }
  if (rc == HOCCL_OK && terminal_nodes.size() > 1) {
    cudaGraphNode_t join;
    cudaKernelNodeParams kp = {};
    kp.func = const_cast<void*>(graph_root_kernel_entry());
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(32);
    kp.kernelParams = nullptr;
    cudaError_t e = cudaGraphAddKernelNode(&join, g, terminal_nodes.data(), terminal_nodes.size(), &kp);
    if (e == cudaSuccess) entry->n_order_launches++;
    else rc = cuda_fail(c, e, "graph end node");
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
  if (c->path == HOCCL_PATH_CE && c->order_kernels) {   // one empty kernel in front of the first stage's copy chains (see build_graph)
    cudaKernelNodeParams kp = {};
    kp.func = const_cast<void*>(graph_root_kernel_entry());
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(32);
    kp.kernelParams = nullptr;
    err = cudaGraphAddKernelNode(&stage_dep, g, nullptr, 0, &kp);
    if (err == cudaSuccess) entry->n_order_launches++;
  }
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
      if (c->path == HOCCL_PATH_CE && c->order_kernels) {   // copy chains wait for copy chains: an empty kernel as the join (see build_graph)
        cudaKernelNodeParams kp = {};
        kp.func = const_cast<void*>(graph_root_kernel_entry());
        kp.gridDim = dim3(1);
        kp.blockDim = dim3(32);
        kp.kernelParams = nullptr;
        err = cudaGraphAddKernelNode(&join, g, tails.data(), tails.size(), &kp);
        if (err == cudaSuccess) entry->n_order_launches++;
      } else {
        err = cudaGraphAddEmptyNode(&join, g, tails.data(), tails.size());
      }
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

// The same for a MODELLED topology with more than one node (paper Sec. 3.4, Eq. 2-4 and Algorithm 1 run as real copies on one
// device).  A logical flow u -> v between two nodes is carried, portion by portion as Algorithm 1 stages it, by three copies
// per chunk: the sender-side forwarding copy f' from u's send buffer into a staging slot at u's symmetric peer, the "RDMA"
// leg f from that slot into a staging slot at v's symmetric peer (optionally cut into serial sub-copies of `rdma_sub` bytes, a
// crude stand-in for the slower domain), and the receiver-side forwarding copy f'' from there into v's receive buffer.
// Staging: `out_stage` + the flow's offset holds what left u, `in_stage` + the same offset what arrived at v's side.
// Copy route: chunk-level DAG; a source GPU's native and forwarding chunks form one serial queue in the scheduler's
// interleaved order (its DMA engine), the RDMA legs of one source form a second serial queue (its NIC), and chunk k of f
// waits for chunk k of f', chunk k of f'' for chunk k of f.  SM path: per stage three batched phases (all f' and native
// chunks, all f, all f'') in one chain of launches.  Stages run one after the other.
hoccl_result_t build_pattern_graph_modelled(hoccl_comm* c, const Schedule& S, const void* const* send, const size_t* sdispls,
                                            void* const* recv, const size_t* rdispls, size_t e, char* out_stage, char* in_stage,
                                            const std::vector<uint64_t>& flow_stage_off, size_t chunk_bytes, size_t rdma_sub,
                                            GraphEntry* entry) {
  const int R = c->R;
  const Topology& topo = S.topo;
  cudaGraph_t g = nullptr;
  CU_TRY(c, cudaGraphCreate(&g, 0));
  cudaError_t err = cudaSuccess;
  auto order_kernel = [&](cudaGraphNode_t* out, const cudaGraphNode_t* deps, size_t nd) {
    cudaKernelNodeParams kp = {};
    kp.func = const_cast<void*>(graph_root_kernel_entry());
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(32);
    kp.kernelParams = nullptr;
    cudaError_t e2 = cudaGraphAddKernelNode(out, g, deps, nd, &kp);
    if (e2 == cudaSuccess) entry->n_order_launches++;
    return e2;
  };
  cudaGraphNode_t stage_dep = nullptr;
  const bool ce = c->path == HOCCL_PATH_CE;
  if (ce && c->order_kernels) err = order_kernel(&stage_dep, nullptr, 0);
  // where the bytes [off, off + n) of the logical flow (u, v) sit at each of the four places they pass through
  auto place = [&](int cls_src, int u, int v, uint64_t off) -> char* {
    // cls_src: 0 = u's send buffer, 1 = staging at u's peer, 2 = staging at v's peer, 3 = v's receive buffer
    switch (cls_src) {
      case 0: return (char*)send[u] + sdispls[(size_t)u * R + v] * e + off;
      case 1: return out_stage + flow_stage_off[(size_t)u * R + v] + off;
      case 2: return in_stage + flow_stage_off[(size_t)u * R + v] + off;
      default: return (char*)recv[v] + rdispls[(size_t)v * R + u] * e + off;
    }
  };
  struct Op {
    const char* src;
    char* dst;
    uint64_t bytes;
  };
  for (size_t si = 0; si < S.stages.size() && err == cudaSuccess; si++) {
    const Stage& st = S.stages[si];
    auto op_of = [&](const StageFlow& f, uint64_t off, uint64_t n) -> Op {
      const int u = f.origin_src, v = f.origin_dst;
      const uint64_t o = f.origin_offset + off;
      const bool has_pu = topo.peer_of(u) != u, has_pv = topo.peer_of(v) != v;
      switch (f.cls) {
        case FLOW_NATIVE: return Op{place(0, u, v, o), place(3, u, v, o), n};
        case FLOW_FWD_SEND: return Op{place(0, u, v, o), place(1, u, v, o), n};
        case FLOW_FWD_RECV: return Op{place(2, u, v, o), place(3, u, v, o), n};
        default: return Op{place(has_pu ? 1 : 0, u, v, o), place(has_pv ? 2 : 3, u, v, o), n};   // the RDMA leg
      }
    };
    auto key_of = [&](const StageFlow& f, uint64_t off) { return std::make_tuple(f.origin_src, f.origin_dst, f.origin_offset + off); };
    std::vector<cudaGraphNode_t> tails;
    if (ce) {
      std::map<std::tuple<int, int, uint64_t>, cudaGraphNode_t> sent, arrived;   // chunk -> its f' node, its f node
      auto add_copy = [&](const Op& op, std::vector<cudaGraphNode_t> deps, size_t sub, cudaGraphNode_t* last) {
        const size_t step = sub ? sub : op.bytes;
        for (uint64_t o = 0; o < op.bytes && err == cudaSuccess; o += step) {
          const uint64_t n = std::min<uint64_t>(step, op.bytes - o);
          cudaGraphNode_t nd;
          err = cudaGraphAddMemcpyNode1D(&nd, g, deps.data(), deps.size(), op.dst + o, op.src + o, n, cudaMemcpyDeviceToDevice);
          if (err != cudaSuccess) return;
          deps.assign(1, nd);
          *last = nd;
          entry->n_moves++;
        }
      };
      // pass 1: the DMA queues' native and sender-side chunks; pass 2: the NIC queues; pass 3: the receiver-side chunks, in
      // their queues' order behind whatever that queue issued in pass 1
      std::vector<cudaGraphNode_t> qtail(R, nullptr);
      for (int pass = 0; pass < 3 && err == cudaSuccess; pass++) {
        if (pass == 1) {
          for (int u = 0; u < R && err == cudaSuccess; u++) {
            cudaGraphNode_t nic = nullptr;
            for (const StageFlow& f : st.flows) {
              if (f.cls != FLOW_RDMA || f.u != u) continue;
              for (uint64_t off = 0; off < f.bytes && err == cudaSuccess; off += chunk_bytes) {
                const uint64_t n = std::min<uint64_t>(chunk_bytes, f.bytes - off);
                std::vector<cudaGraphNode_t> deps;
                if (nic) deps.push_back(nic);
                auto it = sent.find(key_of(f, off));
                if (it != sent.end()) deps.push_back(it->second);
                if (deps.empty() && stage_dep) deps.push_back(stage_dep);
                cudaGraphNode_t last = nullptr;
                add_copy(op_of(f, off, n), deps, rdma_sub, &last);
                if (err != cudaSuccess) break;
                nic = last;
                arrived[key_of(f, off)] = last;
              }
            }
            if (nic) tails.push_back(nic);
          }
          continue;
        }
        for (int q = 0; q < R && err == cudaSuccess; q++) {
          for (const ChunkItem& it : st.queues[q]) {
            const StageFlow& f = st.flows[it.flow];
            const bool recv_side = f.cls == FLOW_FWD_RECV;
            if ((pass == 0) == recv_side) continue;
            std::vector<cudaGraphNode_t> deps;
            if (qtail[q]) deps.push_back(qtail[q]);
            if (recv_side) {
              auto a = arrived.find(key_of(f, it.offset));
              if (a != arrived.end()) deps.push_back(a->second);
            }
            if (deps.empty() && stage_dep) deps.push_back(stage_dep);
            cudaGraphNode_t last = nullptr;
            add_copy(op_of(f, it.offset, it.bytes), deps, 0, &last);
            if (err != cudaSuccess) break;
            qtail[q] = last;
            if (f.cls == FLOW_FWD_SEND) sent[key_of(f, it.offset)] = last;
          }
        }
      }
      for (int q = 0; q < R; q++)
        if (qtail[q]) tails.push_back(qtail[q]);
    } else {
      cudaGraphNode_t prev = stage_dep;
      auto run_phase = [&](const std::vector<Op>& ops) {
        for (size_t first = 0; first < ops.size() && err == cudaSuccess; first += kMaxSegs) {
          CopyBatch b;
          b.nseg = (int)std::min<size_t>(kMaxSegs, ops.size() - first);
          b.pad = 0;
          for (int i = 0; i < b.nseg; i++) b.seg[i] = CopySeg{ops[first + i].src, ops[first + i].dst, (unsigned long long)ops[first + i].bytes};
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
            entry->n_moves += b.nseg;
          }
        }
      };
      std::vector<Op> a, b, d;
      for (const StageFlow& f : st.flows) {
        if (!f.bytes) continue;
        (f.cls == FLOW_RDMA ? b : f.cls == FLOW_FWD_RECV ? d : a).push_back(op_of(f, 0, f.bytes));
      }
      run_phase(a);
      run_phase(b);
      run_phase(d);
      if (prev && prev != stage_dep) tails.push_back(prev);
    }
    if (err != cudaSuccess) break;
    if (tails.size() == 1) {
      stage_dep = tails[0];
    } else if (tails.size() > 1) {
      cudaGraphNode_t join;
      if (ce && c->order_kernels) err = order_kernel(&join, tails.data(), tails.size());
      else err = cudaGraphAddEmptyNode(&join, g, tails.data(), tails.size());
      if (err == cudaSuccess) stage_dep = join;
    }
  }
  hoccl_result_t rc = HOCCL_OK;
  if (err == cudaSuccess) err = cudaGraphInstantiate(&entry->exec, g, 0);
  if (err != cudaSuccess) rc = cuda_fail(c, err, "modelled pattern graph");
  cudaGraphDestroy(g);
  entry->n_pieces = (long)S.stages.size();
  if (rc != HOCCL_OK) destroy_entry(entry);
  return rc;
}

}  // namespace hoccl
