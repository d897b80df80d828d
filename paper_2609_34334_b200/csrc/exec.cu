// libhoccl: how a collective call is executed (the graphs themselves are built in graph.cu, the one-kernel form in ring_host.cu).
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
#include <tuple>

#include "comm.h"
#include "options.h"

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

// Host-bounce path: moves of one group with the same source and length get the same place in the host staging; the first
// of them (host_first = true) carries the outbound copy, the others only their inbound copy behind it.  Recomputes *host_need.
static void share_host_legs(std::vector<RGroup>* groups, size_t* host_need) {
  *host_need = 0;
  for (RGroup& g : *groups) {
    if (g.kind != OP_MOVE) continue;
    std::map<std::pair<const char*, uint64_t>, size_t> first_of;   // (source, bytes) -> index of the seg that owns the staging
    for (size_t i = 0; i < g.segs.size(); i++) {
      Seg& s = g.segs[i];
      auto it = first_of.find({s.src, s.bytes});
      if (it == first_of.end()) {
        first_of.emplace(std::make_pair(s.src, s.bytes), i);
        s.host_off = *host_need;
        s.host_first = true;
        *host_need += (s.bytes + 255) / 256 * 256;
      } else {
        s.host_off = g.segs[it->second].host_off;
        s.host_first = false;
      }
    }
  }
}

// Turns plan offsets into addresses (the plan already places pieces inside the scratch slots).
void resolve(hoccl_comm* c, const Plan& P, const Call& call, std::vector<RGroup>* out, size_t* host_need) {
  *host_need = 0;
  const int R = P.R;
  char* inbox0 = (char*)c->scratch;
  const size_t inbox_bytes = (size_t)P.inbox_slots * P.slot_bytes;   // one rank's inbox: 1 slot, or R-1 for the direct reduce-scatter
  char* partial0 = inbox0 + (size_t)R * inbox_bytes;
  auto addr = [&](int buf, int rank, int chunk, uint64_t off) -> char* {
    (void)chunk;
    switch (buf) {
      case BUF_SEND: return (char*)call.send[rank] + off;
      case BUF_RECV: return (char*)call.recv[rank] + off;
      case BUF_INBOX: return inbox0 + (size_t)rank * inbox_bytes + off;
      default: return partial0 + (size_t)rank * P.slot_bytes + off;
    }
  };
  out->clear();
  out->resize(P.groups.size());
  for (size_t g = 0; g < P.groups.size(); g++) {
    const PlanGroup& pg = P.groups[g];
    RGroup& rg = (*out)[g];
    rg.kind = pg.kind;
    rg.piece = pg.piece;
    rg.phase = pg.phase;
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
        s.nsrc = op.nsrc;
        s.src_stride = op.src_stride;
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
  // SM path, direct all-gather: its stages (the trailing MOVE groups of a piece, nothing depends on them) wait for the same
  // thing, so consecutive ones with equal dependencies become one group = one batched launch (or one phase of the ring kernel).
  // Host-bounce path: the same merge lets the moves of a group that read the same bytes share ONE outbound copy into the
  // host staging (see share_host_legs): a chunk crosses PCIe once outbound and R-1 times inbound instead of R-1 times each way.
  if ((c->path == HOCCL_PATH_SM || c->path == HOCCL_PATH_CE_HOST) && P.ag_direct && P.kind != PLAN_ALLTOALL) {
    std::vector<char> has_user(out->size(), 0);
    for (const RGroup& g : *out) {
      for (int d : g.deps) has_user[d] = 1;
      if (g.chain_dep >= 0) has_user[g.chain_dep] = 1;
    }
    std::vector<RGroup> merged;
    std::vector<int> remap(out->size(), -1);
    for (size_t g = 0; g < out->size(); g++) {
      RGroup& cur = (*out)[g];
      for (int& d : cur.deps) d = remap[d];
      if (cur.chain_dep >= 0) cur.chain_dep = remap[cur.chain_dep];
      const bool tail_move = cur.kind == OP_MOVE && !has_user[g] && P.groups[g].phase != PHASE_RS;
      if (tail_move && !merged.empty() && g > 0 && remap[g - 1] == (int)merged.size() - 1 && merged.back().kind == OP_MOVE &&
          !has_user[g - 1] && P.groups[g - 1].phase != PHASE_RS && merged.back().piece == cur.piece && merged.back().deps == cur.deps) {
        merged.back().segs.insert(merged.back().segs.end(), cur.segs.begin(), cur.segs.end());
        remap[g] = (int)merged.size() - 1;
      } else {
        merged.push_back(cur);
        remap[g] = (int)merged.size() - 1;
      }
    }
    out->swap(merged);
    if (c->path == HOCCL_PATH_CE_HOST) share_host_legs(out, host_need);
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
void fill_chain_batch(const RGroup& g, size_t first, size_t n, int dtype, size_t elem, ChainBatch* b) {
  b->nseg = (int)n;
  b->dtype = dtype;
  for (size_t i = 0; i < n; i++) {
    const Seg& s = g.segs[first + i];
    b->seg[i] = ChainSeg{s.src, s.local, s.dst, (unsigned long long)(s.bytes / elem), (unsigned long long)s.src_stride, s.nsrc, 0};
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

bool build_fan_batches(const RGroup& g, std::vector<FanBatch>* out, std::vector<double>* bytes_out, std::vector<long>* moves_out) {
  out->clear();
  bytes_out->clear();
  moves_out->clear();
  if (g.kind != OP_MOVE) return false;
  // classes: same source, same length, same 16-byte phase of the destination (so that a class is all-vector or all-element-wise)
  struct Class {
    const char* src;
    size_t bytes;
    unsigned phase;
    std::vector<void*> dsts;
  };
  std::vector<Class> classes;
  std::map<std::tuple<const char*, size_t, unsigned>, size_t> index;
  bool repeats = false;
  for (const Seg& s : g.segs) {
    auto key = std::make_tuple((const char*)s.src, (size_t)s.bytes, (unsigned)((uintptr_t)s.dst & 15));
    auto it = index.find(key);
    if (it == index.end()) {
      index.emplace(key, classes.size());
      classes.push_back(Class{s.src, s.bytes, std::get<2>(key), {s.dst}});
    } else {
      classes[it->second].dsts.push_back(s.dst);
      repeats = true;
    }
  }
  if (!repeats) return false;
  FanBatch cur;
  cur.nseg = 0;
  cur.ndst_total = 0;
  double cur_bytes = 0;
  long cur_moves = 0;
  auto flush = [&]() {
    if (cur.nseg == 0) return;
    out->push_back(cur);
    bytes_out->push_back(cur_bytes);
    moves_out->push_back(cur_moves);
    cur.nseg = 0;
    cur.ndst_total = 0;
    cur_bytes = 0;
    cur_moves = 0;
  };
  for (const Class& cl : classes) {
    size_t done = 0;
    while (done < cl.dsts.size()) {   // a class with more destinations than a batch holds is cut
      if (cur.nseg == kMaxSegs || cur.ndst_total == kMaxFanDsts) flush();
      const size_t n = std::min<size_t>(cl.dsts.size() - done, (size_t)(kMaxFanDsts - cur.ndst_total));
      cur.seg[cur.nseg++] = FanSeg{cl.src, (unsigned long long)cl.bytes, cur.ndst_total, (int)n};
      for (size_t i = 0; i < n; i++) cur.dst[cur.ndst_total++] = cl.dsts[done + i];
      cur_bytes += (double)cl.bytes * (1.0 + (double)n);
      cur_moves += (long)n;
      done += n;
    }
  }
  flush();
  return true;
}

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
    if (rg.kind != OP_MOVE) {
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
    if (rg.kind == OP_CHAIN) {
      for (size_t first = 0; first < rg.segs.size(); first += kMaxSegs) {
        size_t n = std::min<size_t>(kMaxSegs, rg.segs.size() - first);
        ChainBatch b;
        fill_chain_batch(rg, first, n, P.dtype, P.elem, &b);
        CU_TRY(c, launch_chain(b, (int)c->sum_ctas, s));
        tally->sum_launches++;
      }
    } else if (rg.kind == OP_SUM) {
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
        // a seg that shares another seg's outbound copy comes after it in the same group, hence later on this stream
        if (sg.host_first) CU_TRY(c, cudaMemcpyAsync(c->host_staging + sg.host_off, sg.src, sg.bytes, cudaMemcpyDeviceToHost, s));
        CU_TRY(c, cudaMemcpyAsync(sg.dst, c->host_staging + sg.host_off, sg.bytes, cudaMemcpyHostToDevice, s));
        tally->moves++;
      }
    } else {
      std::vector<FanBatch> fans;
      std::vector<double> fan_bytes;
      std::vector<long> fan_moves;
      if (P.ag_direct && build_fan_batches(rg, &fans, &fan_bytes, &fan_moves)) {
        for (size_t i = 0; i < fans.size(); i++) {
          CU_TRY(c, launch_fan(fans[i], (int)c->copy_ctas, s));
          tally->moves += fan_moves[i];
          tally->move_launches++;
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
  k.push_back((uint64_t)c->ag_direct);
  k.push_back((uint64_t)c->order_kernels);
  k.push_back((uint64_t)c->rs_direct);
  k.push_back((uint64_t)c->ce_overlap);
  k.push_back((uint64_t)(c->fused && c->path == HOCCL_PATH_SM && !c->handshake));
  k.push_back((uint64_t)c->roles);
  k.push_back((uint64_t)c->piece_grade);
  k.push_back((uint64_t)c->roles_missing);
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
  if (hit->roles_fn) {
    hoccl_result_t rrc = launch_roles(c, hit, user);
    if (rrc != HOCCL_OK) return rrc;
    c->stats.n_pieces = hit->n_pieces;
    c->stats.n_moves = hit->n_moves;
    c->stats.n_move_launches = 1;
    c->stats.n_sum_launches = 0;
    c->stats.max_copy_ctas = hit->roles_grid - hit->roles_sum_ctas;
    c->stats.max_sum_ctas = hit->roles_sum_ctas;
    c->stats.host_launch_us = now_us() - t0;
    return HOCCL_OK;
  }
  if (!hit->part_exec.empty()) {
    // Copy route with overlap: the reduce-scatter's moves of every piece on one internal stream, the sums on the sum stream
    // (one at a time: the SM budget stays global), the all-gather's moves on a second internal stream; events carry the
    // per-piece dependencies between them.
    cudaStream_t rs = c->lane[0], sm = c->sum_stream, ag = c->lane[1];
    c->ev_next = 0;
    cudaEvent_t fork = next_event(c);
    if (!fork) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    CU_TRY(c, cudaEventRecord(fork, user));
    CU_TRY(c, cudaStreamWaitEvent(rs, fork, 0));
    CU_TRY(c, cudaStreamWaitEvent(sm, fork, 0));
    CU_TRY(c, cudaStreamWaitEvent(ag, fork, 0));
    const size_t np = hit->part_exec.size() / 3;
    for (size_t p = 0; p < np; p++) {
      cudaGraphExec_t g_rs = hit->part_exec[3 * p], g_sum = hit->part_exec[3 * p + 1], g_ag = hit->part_exec[3 * p + 2];
      if (g_rs) {
        CU_TRY(c, cudaGraphLaunch(g_rs, rs));
        cudaEvent_t moved = next_event(c);
        if (!moved) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
        CU_TRY(c, cudaEventRecord(moved, rs));
        CU_TRY(c, cudaStreamWaitEvent(sm, moved, 0));
      }
      if (g_sum) CU_TRY(c, cudaGraphLaunch(g_sum, sm));
      if (g_ag) {
        cudaEvent_t summed = next_event(c);
        if (!summed) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
        CU_TRY(c, cudaEventRecord(summed, sm));
        CU_TRY(c, cudaStreamWaitEvent(ag, summed, 0));
        CU_TRY(c, cudaGraphLaunch(g_ag, ag));
      }
    }
    for (cudaStream_t s : {rs, sm, ag}) {
      cudaEvent_t done = next_event(c);
      if (!done) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
      CU_TRY(c, cudaEventRecord(done, s));
      CU_TRY(c, cudaStreamWaitEvent(user, done, 0));
    }
  } else if (!hit->piece_exec.empty()) {
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
  c->stats.n_order_launches = hit->n_order_launches;
  c->stats.max_sum_ctas = hit->n_sum_launches ? c->sum_ctas : 0;
  c->stats.max_copy_ctas = hit->n_move_launches ? c->copy_ctas : 0;
  c->stats.host_launch_us = now_us() - t0;
  return HOCCL_OK;
}

static OptionsIn options_of(hoccl_comm* c, int kind, size_t count, int dtype, bool host_call) {
  return OptionsIn{kind, c->R, count, dtype, (int)c->path, c->onepass, c->forward, c->fused, c->rs_direct, c->ag_direct,
                   c->handshake, c->use_graph, c->ce_small_bytes, c->ce_small_ctas, c->copy_ctas, c->scratch ? c->scratch_bytes : 0,
                   host_call ? 1 : 0, c->roles};
}

hoccl_result_t check_options(hoccl_comm* c, int kind, size_t count, int dtype) {
  OptionsOut o;
  return resolve_options(options_of(c, kind, count, dtype, false), &o);
}

hoccl_result_t run_collective(hoccl_comm* c, Call* call, cudaStream_t user) {
  const double t0 = now_us();
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (dtype_size(call->dtype) == 0) return HOCCL_ERR_UNSUPPORTED;
  if (!call->send || !call->recv) return HOCCL_ERR_INVALID_ARG;
  // One place decides how the settings combine for this call (options.h); a contradictory combination is refused here.
  const OptionsIn oin = options_of(c, call->kind, call->count, call->dtype, call->h_send != nullptr);
  OptionsOut opt;
  {
    hoccl_result_t orc = resolve_options(oin, &opt);
    if (orc != HOCCL_OK) return orc;
  }
  // a small message on the copy route runs on the copy kernel's route: the communicator shows that route for this call only
  struct RouteGuard {
    hoccl_comm* c;
    hoccl_path_t path;
    long ctas;
    ~RouteGuard() {
      c->path = path;
      c->copy_ctas = ctas;
    }
  } guard{c, c->path, c->copy_ctas};
  c->path = (hoccl_path_t)opt.path;
  c->copy_ctas = opt.copy_ctas;
  const bool onepass_case = opt.executor == EXEC_ONEPASS;
  const bool fused = opt.executor == EXEC_ONE_KERNEL;
  const bool roles = opt.executor == EXEC_ROLES;
  const bool graphs = opt.executor != EXEC_STREAMS && !onepass_case;
  std::vector<uint64_t> key;
  if (graphs && call->count != 0) {
    // Fast path: a call whose signature (operation, count, dtype, every pointer, every setting that shapes the graph)
    // was seen before was validated and planned then; replaying its graph is all that is left to do.
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

  if (onepass_case) {
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
  const int plan_kind = opt.plan_kind;
  // Piece size: the caller's if set.  Otherwise: on the SM path under CTA budgets a reduction is cut into at least two
  // pieces (the copy kernel of one piece then overlaps the sum kernel of the other: measured 1.6x on a 3 MiB chunk with
  // 8 + 8 CTAs) of at most 4 MiB.  That does not pay with driver copies (they take the whole GPU and never overlap a sum:
  // every extra copy only adds its start-up) nor with whole-GPU grids (two kernels then share the same SMs), so the
  // copy route and the SM path with 128 CTAs or more for both kernels keep whole chunks up to 256 MiB (measured, R = 8,
  // bf16, 64 MiB to 1 GiB per rank: 7-15 % faster than 4 MiB pieces on the copy route with 8-CTA sums, 19-33 % with
  // 148-CTA sums, 3-14 % on the whole-GPU SM path).
  size_t piece_bytes = (size_t)c->piece_bytes;
  int max_pieces = (int)c->max_pieces;
  const bool reduction = call->kind == PLAN_ALLREDUCE || call->kind == PLAN_REDUCE_SCATTER;
  const size_t ring_chunk = (call->kind == PLAN_ALLREDUCE ? (call->count + c->R - 1) / c->R : call->count) * dtype_size(call->dtype);
  // Copy route with overlap ("ce_overlap"): the direct schedule cut into pieces whose three parts run on three internal
  // streams (see launch_entry).  Automatic (-1): 2 pieces from 2 MiB per ring chunk, from 4 MiB on pieces of about 4 MiB, at
  // least 4 and at most 32 of them; below that the ~30 us of host time per call and the extra copies cost more than the overlap
  // gives (measured on B200, R = 8, bf16, 8-CTA sums: 25 MiB per rank 0.290 -> 0.280 ms with 2 pieces; 40 MiB 0.468 -> 0.421 with
  // 4; 256 MiB 2.97 -> 2.44 with 8; 1 GiB 11.8 -> 9.72 with 8, 9.52 with 32).
  long overlap_pieces = c->ce_overlap;
  if (overlap_pieces < 0) {
    // (whole-GPU sums are short: beside them more than 8 pieces only add copies; 1 GiB per rank 6.34 ms with 8, 6.80 with 32)
    const size_t most = c->sum_ctas >= 64 ? 8 : 32;
    overlap_pieces = ring_chunk >= ((size_t)4 << 20) ? (long)std::min<size_t>(most, std::max<size_t>(4, ring_chunk >> 22))
                                                     : ring_chunk >= ((size_t)2 << 20) ? 2 : 0;
  }
  const bool overlap = overlap_pieces > 1 && c->path == HOCCL_PATH_CE && opt.executor == EXEC_GRAPH && !call->h_send &&
                       (plan_kind & PLAN_FLAG_RS_DIRECT) && c->R > 1 && !c->piece_bytes_set;
  if (overlap) {
    max_pieces = (int)overlap_pieces;
    piece_bytes = std::max<size_t>((size_t)64 << 10, ((ring_chunk + max_pieces - 1) / max_pieces + 1023) / 1024 * 1024);
  } else if (!c->piece_bytes_set && c->path == HOCCL_PATH_SM && opt.executor == EXEC_GRAPH && !call->h_send && reduction &&
             (plan_kind & PLAN_FLAG_RS_DIRECT) && c->sum_ctas < 64 && c->copy_ctas < 128 && ring_chunk >= ((size_t)1 << 20)) {
    // SM path, direct schedule under CTA budgets: pieces of an eighth of a ring chunk, between 640 KiB and 2 MiB, issued as a
    // software pipeline (see build_graph): a piece's copies run beside another piece's chain sum (measured, 8-CTA sums and
    // 40 copy CTAs: 40 MiB per rank 0.46 ms with 2 pieces, 0.41 with 4, 0.38 with 8, 0.45 with 10; 25 MiB 0.30 / 0.26 / 0.245 /
    // 0.29 ms with 2 / 4 / 5 / 7 pieces; 256 MiB 2.92 / 2.57 / 2.40 / 2.32 ms with 2 / 4 / 8 / 16 pieces)
    piece_bytes = std::min<size_t>((size_t)2 << 20, std::max<size_t>((size_t)640 << 10, (ring_chunk / 8 + 1023) / 1024 * 1024));
    max_pieces = 64;
  } else if (call->h_send) {   // pipelined host all-reduce: host_pieces pieces per chunk, whatever the chunk size
    const size_t q = (call->count + c->R - 1) / c->R;
    const size_t chunk = q * dtype_size(call->dtype);
    max_pieces = (int)c->host_pieces;
    piece_bytes = std::max<size_t>((size_t)64 << 10, ((chunk + max_pieces - 1) / max_pieces + 1023) / 1024 * 1024);
  } else if (roles) {
    // the piece rule of the graph form of the same schedule (above): both forms measured best with the same pieces
    if (!c->piece_bytes_set)
      piece_bytes = std::min<size_t>((size_t)2 << 20, std::max<size_t>((size_t)640 << 10, (ring_chunk / 8 + 1023) / 1024 * 1024));
    max_pieces = 64;   // (when the tables of that many pieces do not fit into shared memory the graph form runs the plan)
  } else if (fused) {   // one kernel walks the steps in order; whole chunks measured faster than pieces (fewer barriers and tails)
    piece_bytes = (size_t)1 << 60;
    max_pieces = 1;
  } else if (!c->piece_bytes_set && reduction &&
             (c->path == HOCCL_PATH_CE || (c->path == HOCCL_PATH_SM && std::min(c->sum_ctas, c->copy_ctas) >= 128))) {
    // "whole" stops at 256 MiB: several concurrent driver copies of 512 MiB each ran at half speed (R = 2, 1 GiB per rank)
    piece_bytes = (size_t)256 << 20;
  } else if (!c->piece_bytes_set && c->path == HOCCL_PATH_SM && std::max(c->sum_ctas, c->copy_ctas) < 64 &&
      (call->kind == PLAN_ALLREDUCE || call->kind == PLAN_REDUCE_SCATTER)) {
    const size_t q = call->kind == PLAN_ALLREDUCE ? (call->count + c->R - 1) / c->R : call->count;
    const size_t chunk = q * dtype_size(call->dtype);
    if (chunk >= ((size_t)1 << 20)) piece_bytes = std::min(piece_bytes, (chunk / 2 + 1023) / 1024 * 1024);
  }
  // graded pieces ("piece_grade"; -1 = automatic): measured on B200 (R = 8, bf16, 8-CTA sums) they gain 1-5 % from 64 MiB per rank
  // on (256 MiB: copy route 2.46 -> 2.44 ms, SM path 8 + 40 CTAs 2.32 -> 2.27, roles kernel 2.32 -> 2.25) and lose below (40 MiB
  // buckets: copy route 0.423 -> 0.444 ms, SM path 0.380 -> 0.431: the small outer pieces cost more in fixed time per piece than
  // their shorter fill saves), so automatic means: from 8 MiB per ring chunk, under a SUM budget (with whole-GPU sums the outer
  // pieces' moves are no longer what is exposed: 256 MiB per rank, copy route, 148-CTA sums 1.51 -> 1.53 ms)
  const bool graded = reduction && !call->h_send && !fused && (plan_kind & PLAN_FLAG_RS_DIRECT) &&
                      (c->piece_grade == 1 || (c->piece_grade < 0 && ring_chunk >= ((size_t)8 << 20) && c->sum_ctas < 64));
  if (!build_plan(&P, plan_kind | (graded ? PLAN_FLAG_GRADED : 0), c->R, call->count, call->dtype, call->in_place, piece_bytes, max_pieces, align))
    return HOCCL_ERR_INVALID_ARG;
  if (P.slot_bytes) {
    size_t need = P.scratch_need();
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
        if (rc != HOCCL_OK) {
          destroy_entry(&entry);   // the pieces built so far, and any profile events
          return rc;
        }
      }
    } else if (overlap && P.pieces > 1) {   // with one piece there is nothing to overlap: one graph
      entry.part_exec.assign((size_t)P.pieces * 3, nullptr);
      for (int p = 0; p < P.pieces && rc == HOCCL_OK; p++)
        for (int part = 0; part < 3 && rc == HOCCL_OK; part++) rc = build_graph(c, P, groups, &entry, p, &entry.part_exec[(size_t)p * 3 + part], part);
      if (rc != HOCCL_OK) {
        destroy_entry(&entry);
        return rc;
      }
    } else {
      rc = fused ? build_ring(c, P, groups, &entry) : roles ? build_roles(c, P, groups, &entry) : HOCCL_ERR_UNSUPPORTED;
      // not asked for, too many ranks for one launch (fused), or more CTAs than can be resident together (roles)
      if (rc == HOCCL_ERR_UNSUPPORTED) rc = build_graph(c, P, groups, &entry, -1, &entry.exec);
      if (rc != HOCCL_OK) {
        destroy_entry(&entry);
        return rc;
      }
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
