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
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cstdio>
#include <cstring>
#include <deque>
#include <map>
#include <string>
#include <utility>
#include <vector>

#include "../../include/hoccl.h"
#include "kernels.cuh"
#include "plan.h"
#include "proxy.h"
#include "sched.h"

using namespace hoccl;

namespace {

constexpr int kMaxRanks = 64;
constexpr int kMaxLanes = 8;
constexpr size_t kGraphCacheCap = 48;

double now_us() {
  return std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

struct Seg {
  const char* src;    // MOVE: source; SUM: inbox
  const char* local;  // SUM only
  char* dst;
  uint64_t bytes;
};

struct RGroup {
  int kind;
  std::vector<Seg> segs;
  std::vector<int> deps;
  int chain_dep;
};

struct Post {
  bool is_send;
  void* buf;
  size_t count;
  int dtype;
  cudaStream_t stream;
};

struct GraphEntry {
  std::vector<uint64_t> key;
  cudaGraphExec_t exec = nullptr;
  uint64_t last_use = 0;
  long n_moves = 0, n_move_launches = 0, n_sum_launches = 0, n_pieces = 0;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof_events;  // owned; only with profile = 1
  std::vector<double> prof_bytes;
  bool prof_pending = false;  // replayed since the profile events were last read
};

}  // namespace

struct hoccl_comm {
  int R = 0, device = 0, num_sms = 0;
  hoccl_path_t path = HOCCL_PATH_CE;
  long sum_ctas = 8, copy_ctas = 8, piece_bytes = 4 << 20, max_pieces = 8, lanes = 4, use_graph = 1, profile = 0, p2p_split = 1, ce_sub_bytes = 0,
       handshake = 0, watchdog_ms = 10000, onepass = 0;
  Proxy* proxy = nullptr;
  cudaStream_t lane[kMaxLanes] = {};
  cudaStream_t sum_stream = nullptr;
  int sum_priority = 0;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_next = 0;
  void* scratch = nullptr;
  size_t scratch_bytes = 0;
  void* staging = nullptr;
  size_t staging_bytes = 0;
  std::map<std::pair<int, int>, std::deque<Post>> pending;
  int n_pending = 0;
  unsigned p2p_rr = 0;
  std::vector<GraphEntry> cache;
  uint64_t use_counter = 0;
  hoccl_stats_t stats = {};
  std::string cuda_err;
  // profile accumulation
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof_pool;   // timing events of the stream executor
  std::vector<std::pair<std::pair<cudaEvent_t, cudaEvent_t>, double>> prof_open;  // recorded, not yet read
  double prof_ms = 0, prof_bytes = 0;
  long prof_n = 0;
};

namespace {

hoccl_result_t cuda_fail(hoccl_comm* c, cudaError_t e, const char* what) {
  if (c) {
    c->cuda_err = std::string(what) + ": " + cudaGetErrorString(e);
  }
  return HOCCL_ERR_CUDA;
}

#define CU_TRY(c, call)                                   \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return cuda_fail(c, e__, #call); \
  } while (0)

cudaEvent_t next_event(hoccl_comm* c) {
  if (c->ev_next == c->ev_pool.size()) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    c->ev_pool.push_back(e);
  }
  return c->ev_pool[c->ev_next++];
}

bool ranges_overlap(const char* a, size_t an, const char* b, size_t bn) {
  if (an == 0 || bn == 0) return false;
  return a < b + bn && b < a + an;
}

struct Call {
  int kind;  // PlanKind
  size_t count;
  int dtype;
  bool in_place;
  size_t send_bytes, recv_bytes;
  const void* const* send;
  void* const* recv;
};

// Argument checks shared by the three collectives.  Sets call->in_place.
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
void resolve(hoccl_comm* c, const Plan& P, const Call& call, std::vector<RGroup>* out) {
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
        s.dst = addr(op.dst_buf, op.rank, op.chunk, op.dst_off);
      }
      rg.segs.push_back(s);
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
  for (auto& p : e->prof_events) {
    cudaEventDestroy(p.first);
    cudaEventDestroy(p.second);
  }
  e->exec = nullptr;
  e->prof_events.clear();
}

hoccl_result_t build_graph(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry) {
  cudaGraph_t g = nullptr;
  CU_TRY(c, cudaGraphCreate(&g, 0));
  std::vector<cudaGraphNode_t> tail(groups.size(), nullptr);
  cudaGraphNode_t last_copy_node = nullptr;
  hoccl_result_t rc = HOCCL_OK;
  auto fail = [&](cudaError_t e, const char* what) {
    rc = cuda_fail(c, e, what);
  };
  for (size_t gi = 0; gi < groups.size() && rc == HOCCL_OK; gi++) {
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
    } else {
      for (size_t first = 0; first < rg.segs.size() && e == cudaSuccess; first += kMaxSegs) {
        size_t n = std::min<size_t>(kMaxSegs, rg.segs.size() - first);
        CopyBatch b;
        fill_copy_batch(rg, first, n, &b);
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
        cudaGraphNode_t kn;
        e = cudaGraphAddKernelNode(&kn, g, d2.data(), d2.size(), &kp);
        if (e != cudaSuccess) break;
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
    cudaError_t e = cudaGraphInstantiate(&entry->exec, g, 0);
    if (e != cudaSuccess) rc = cuda_fail(c, e, "cudaGraphInstantiate");
  }
  cudaGraphDestroy(g);
  if (rc != HOCCL_OK) destroy_entry(entry);
  return rc;
}

std::vector<uint64_t> make_key(hoccl_comm* c, const Call& call) {
  std::vector<uint64_t> k;
  k.reserve(12 + 2 * c->R);
  k.push_back((uint64_t)call.kind);
  k.push_back((uint64_t)call.count);
  k.push_back((uint64_t)call.dtype);
  k.push_back((uint64_t)c->path);
  k.push_back((uint64_t)c->sum_ctas);
  k.push_back((uint64_t)c->copy_ctas);
  k.push_back((uint64_t)c->piece_bytes);
  k.push_back((uint64_t)c->max_pieces);
  k.push_back((uint64_t)c->profile);
  k.push_back((uint64_t)c->ce_sub_bytes);
  k.push_back((uint64_t)(uintptr_t)c->scratch);
  for (int r = 0; r < c->R; r++) {
    k.push_back((uint64_t)(uintptr_t)call.send[r]);
    k.push_back((uint64_t)(uintptr_t)call.recv[r]);
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
        c->prof_ms += ms;
        c->prof_bytes += e.prof_bytes[i];
        c->prof_n++;
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

hoccl_result_t run_collective(hoccl_comm* c, Call* call, cudaStream_t user) {
  const double t0 = now_us();
  if (!c) return HOCCL_ERR_INVALID_ARG;
  if (dtype_size(call->dtype) == 0) return HOCCL_ERR_UNSUPPORTED;
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
  if (!build_plan(&P, call->kind, c->R, call->count, call->dtype, call->in_place, (size_t)c->piece_bytes, (int)c->max_pieces, align))
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
  Tally tally;
  if (c->handshake) {
    // Driver copies share a hardware queue with the copies the parked stream has queued behind its hand-over; a copy
    // issued by the proxy can end up behind them and never start (observed).  Kernels do not have that problem.
    if (c->path == HOCCL_PATH_CE) return HOCCL_ERR_UNSUPPORTED;
    rc = ensure_proxy(c);
    if (rc != HOCCL_OK) return rc;
  }
  if (c->use_graph || c->handshake) {
    std::vector<uint64_t> key = make_key(c, *call);
    GraphEntry* hit = nullptr;
    for (auto& e : c->cache)
      if (e.key == key) {
        hit = &e;
        break;
      }
    c->stats.graph_hit = hit ? 1 : 0;
    if (!hit) {
      std::vector<RGroup> groups;
      resolve(c, P, *call, &groups);
      GraphEntry entry;
      entry.key = key;
      entry.n_pieces = P.pieces;
      rc = build_graph(c, P, groups, &entry);
      if (rc != HOCCL_OK) return rc;
      // handshake mode: place the graph on the device now; the proxy must not meet first-launch work later
      if (c->handshake) CU_TRY(c, cudaGraphUpload(entry.exec, c->proxy->work_stream()));
      if (c->cache.size() >= kGraphCacheCap) {
        if (c->proxy) c->proxy->drain(c->watchdog_ms);  // a queued hand-over may still refer to the victim
        size_t victim = 0;
        for (size_t i = 1; i < c->cache.size(); i++)
          if (c->cache[i].last_use < c->cache[victim].last_use) victim = i;
        destroy_entry(&c->cache[victim]);
        c->cache.erase(c->cache.begin() + victim);
      }
      c->cache.push_back(std::move(entry));
      hit = &c->cache.back();
    }
    hit->last_use = ++c->use_counter;
    if (c->handshake) {
      // paper Sec. 3.2: the stream hands itself to the CPU proxy, which runs the schedule and hands it back
      ProxyTask t;
      t.kind = ProxyTask::GRAPH;
      t.exec = hit->exec;
      CU_TRY(c, c->proxy->submit(user, t));
    } else {
      CU_TRY(c, cudaGraphLaunch(hit->exec, user));
    }
    hit->prof_pending = !hit->prof_events.empty();
    tally.moves = hit->n_moves;
    tally.move_launches = hit->n_move_launches;
    tally.sum_launches = hit->n_sum_launches;
  } else {
    std::vector<RGroup> groups;
    resolve(c, P, *call, &groups);
    rc = run_streams(c, P, groups, user, &tally);
    if (rc != HOCCL_OK) return rc;
  }
  c->stats.n_moves = tally.moves;
  c->stats.n_move_launches = tally.move_launches;
  c->stats.n_sum_launches = tally.sum_launches;
  c->stats.max_sum_ctas = tally.sum_launches ? c->sum_ctas : 0;
  c->stats.max_copy_ctas = tally.move_launches ? c->copy_ctas : 0;
  c->stats.host_launch_us = now_us() - t0;
  return HOCCL_OK;
}

hoccl_result_t p2p_post(hoccl_comm* c, bool is_send, void* buf, size_t count, int dtype, int src, int dst, cudaStream_t stream) {
  const double t0 = now_us();
  if (!c || !buf) return HOCCL_ERR_INVALID_ARG;
  const size_t e = dtype_size(dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  if (src < 0 || src >= c->R || dst < 0 || dst >= c->R || src == dst) return HOCCL_ERR_INVALID_ARG;
  if ((uintptr_t)buf % e) return HOCCL_ERR_INVALID_ARG;
  if (c->handshake) {
    // the post is handed to the proxy at once; matching happens there, after the stream has reached the post
    if (c->path == HOCCL_PATH_CE) return HOCCL_ERR_UNSUPPORTED;   // see run_collective
    hoccl_result_t rc = ensure_proxy(c);
    if (rc != HOCCL_OK) return rc;
    ProxyTask t;
    t.kind = ProxyTask::P2P;
    t.is_send = is_send;
    t.src = src;
    t.dst = dst;
    t.buf = buf;
    t.count = count;
    t.elem = e;
    t.dtype = dtype;
    t.path = (int)c->path;
    t.copy_ctas = (int)c->copy_ctas;
    CU_TRY(c, cudaSetDevice(c->device));
    CU_TRY(c, c->proxy->submit(stream, t));
    c->stats = hoccl_stats_t{};
    c->stats.n_moves = 1;
    c->stats.host_launch_us = now_us() - t0;
    return HOCCL_OK;
  }
  auto key = std::make_pair(src, dst);
  std::deque<Post>& q = c->pending[key];
  if (q.empty() || q.front().is_send == is_send) {
    q.push_back(Post{is_send, buf, count, dtype, stream});
    c->n_pending++;
    return HOCCL_OK;
  }
  Post peer = q.front();
  q.pop_front();
  c->n_pending--;
  if (peer.count != count || peer.dtype != dtype) return HOCCL_ERR_MISMATCH;
  c->stats = hoccl_stats_t{};
  if (count == 0) return HOCCL_OK;
  const void* sbuf = is_send ? buf : peer.buf;
  void* dbuf = is_send ? peer.buf : buf;
  const size_t bytes = count * e;
  if (ranges_overlap((const char*)sbuf, bytes, (const char*)dbuf, bytes)) return HOCCL_ERR_INVALID_ARG;
  CU_TRY(c, cudaSetDevice(c->device));
  const bool two_streams = (peer.stream != stream);
  // Large messages on the copy route are cut into up to 4 slices that run on different lanes: one driver copy of
  // 64 MiB reaches ~5.4 TB/s of HBM traffic, two to four concurrent ones ~6.5 TB/s (the same idea as keeping several
  // chunks in flight per connection, paper Sec. 3.3.1 "Multi-QP parallelism").
  int nsplit = 1;
  if (c->path == HOCCL_PATH_CE && bytes >= ((size_t)32 << 20)) {
    nsplit = (int)std::min<size_t>((size_t)c->p2p_split, bytes / ((size_t)16 << 20));
    nsplit = std::max(1, std::min<int>(nsplit, kMaxLanes));
  }
  long n_moves = 0;
  if (!two_streams && nsplit == 1) {
    // both posts came from the same stream: its own order is the whole dependency
    if (c->path == HOCCL_PATH_CE) {
      CU_TRY(c, cudaMemcpyAsync(dbuf, sbuf, bytes, cudaMemcpyDeviceToDevice, stream));
    } else {
      CopyBatch b;
      b.nseg = 1;
      b.pad = 0;
      b.seg[0] = CopySeg{sbuf, dbuf, (unsigned long long)bytes};
      CU_TRY(c, launch_copy(b, (int)c->copy_ctas, stream));
      c->stats.n_move_launches = 1;
      c->stats.max_copy_ctas = c->copy_ctas;
    }
    n_moves = 1;
  } else {
    // the move runs on internal lanes after both posting streams, and both wait for it
    c->ev_next = 0;
    cudaEvent_t ea = next_event(c), eb = two_streams ? next_event(c) : nullptr;
    if (!ea || (two_streams && !eb)) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    CU_TRY(c, cudaEventRecord(ea, peer.stream));
    if (two_streams) CU_TRY(c, cudaEventRecord(eb, stream));
    const size_t slice = ((bytes + nsplit - 1) / nsplit + 255) / 256 * 256;
    for (int i = 0; i < nsplit; i++) {
      const size_t off = (size_t)i * slice;
      if (off >= bytes) break;
      const size_t len = std::min(slice, bytes - off);
      // copy route: rotate lanes so that independent messages overlap; SM copies share one lane so that the CTA
      // budget stays global (two copy kernels never run at the same time)
      cudaStream_t run = c->path == HOCCL_PATH_CE ? c->lane[(c->p2p_rr++) % kMaxLanes] : c->lane[0];
      CU_TRY(c, cudaStreamWaitEvent(run, ea, 0));
      if (two_streams) CU_TRY(c, cudaStreamWaitEvent(run, eb, 0));
      if (c->path == HOCCL_PATH_CE) {
        CU_TRY(c, cudaMemcpyAsync((char*)dbuf + off, (const char*)sbuf + off, len, cudaMemcpyDeviceToDevice, run));
      } else {
        CopyBatch b;
        b.nseg = 1;
        b.pad = 0;
        b.seg[0] = CopySeg{(const char*)sbuf + off, (char*)dbuf + off, (unsigned long long)len};
        CU_TRY(c, launch_copy(b, (int)c->copy_ctas, run));
        c->stats.n_move_launches++;
        c->stats.max_copy_ctas = c->copy_ctas;
      }
      n_moves++;
      cudaEvent_t ed = next_event(c);
      if (!ed) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
      CU_TRY(c, cudaEventRecord(ed, run));
      CU_TRY(c, cudaStreamWaitEvent(peer.stream, ed, 0));
      if (two_streams) CU_TRY(c, cudaStreamWaitEvent(stream, ed, 0));
    }
  }
  c->stats.n_moves = n_moves;
  c->stats.host_launch_us = now_us() - t0;
  return HOCCL_OK;
}

}  // namespace

// ====================================================================== C ABI ====================
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
  if (c->proxy) {
    c->proxy->drain(c->watchdog_ms);
    if (c->proxy->pending_p2p() > 0) return HOCCL_ERR_PENDING;
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
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  for (auto& p : c->prof_pool) {
    cudaEventDestroy(p.first);
    cudaEventDestroy(p.second);
  }
  for (auto& p : c->prof_open) {
    cudaEventDestroy(p.first.first);
    cudaEventDestroy(p.first.second);
  }
  delete c;
  return HOCCL_OK;
}

size_t hoccl_scratch_bytes(int R, size_t max_count, hoccl_dtype_t dtype) {
  size_t e = dtype_size((int)dtype);
  if (R <= 1 || e == 0 || max_count == 0) return 0;
  return 2 * (size_t)R * slot_bytes_for(R, max_count, e);
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

hoccl_result_t hoccl_comm_set_path(hoccl_comm_t c, hoccl_path_t path) {
  if (!c || (path != HOCCL_PATH_CE && path != HOCCL_PATH_SM)) return HOCCL_ERR_INVALID_ARG;
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
              {"watchdog_ms", &c->watchdog_ms, 10, 600000},    {"onepass", &c->onepass, 0, 1}};
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
  if (std::strcmp(key, "piece_bytes") == 0) value = (value + 1023) / 1024 * 1024;
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

long hoccl_comm_handshakes(hoccl_comm_t c) { return (c && c->proxy) ? c->proxy->handshakes() : 0; }

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
    CU_TRY(c, cudaMemcpyAsync(const_cast<void*>(dsend[r]), h_send[r], count * e, cudaMemcpyHostToDevice, st));
  }
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
  if (c->handshake) return HOCCL_ERR_UNSUPPORTED;
  const int R = c->R;
  for (int r = 0; r < R; r++) {
    if (!send[r] || !recv[r]) return HOCCL_ERR_INVALID_ARG;
    if (((uintptr_t)send[r] % e) || ((uintptr_t)recv[r] % e)) return HOCCL_ERR_INVALID_ARG;
  }
  // the flows of the user-defined pattern as the origin traffic matrix C (bytes); one NVLink domain, no RDMA
  Topology topo;
  topo.G = R;
  topo.gpus_per_node = R;
  std::vector<uint64_t> C((size_t)R * R);
  uint64_t total = 0;
  for (int u = 0; u < R; u++)
    for (int v = 0; v < R; v++) {
      C[(size_t)u * R + v] = (uint64_t)sendcounts[(size_t)u * R + v] * e;
      total += C[(size_t)u * R + v];
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
  if (!build_schedule(topo, C, (uint64_t)std::max<long>(c->piece_bytes, 65536), &S)) return HOCCL_ERR_INTERNAL;
  CU_TRY(c, cudaSetDevice(c->device));
  cudaStream_t user = (cudaStream_t)stream;
  const int lanes = c->path == HOCCL_PATH_SM ? 1 : (int)std::max<long>(1, std::min<long>(c->lanes, kMaxLanes));
  c->ev_next = 0;
  cudaEvent_t fork = next_event(c);
  if (!fork) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
  CU_TRY(c, cudaEventRecord(fork, user));
  for (int l = 0; l < lanes; l++) CU_TRY(c, cudaStreamWaitEvent(c->lane[l], fork, 0));
  long moves = 0, launches = 0;
  for (size_t si = 0; si < S.stages.size(); si++) {
    const Stage& st = S.stages[si];
    // every DMA queue (one per source rank) is a serial chain on its lane, in the interleaved chunk order
    for (int g = 0; g < R; g++) {
      cudaStream_t lane = c->lane[g % lanes];
      for (const ChunkItem& it : st.queues[g]) {
        const StageFlow& f = st.flows[it.flow];
        const size_t so = sdispls[(size_t)f.origin_src * R + f.origin_dst] * e + f.origin_offset + it.offset;
        const size_t dofs = rdispls[(size_t)f.origin_dst * R + f.origin_src] * e + f.origin_offset + it.offset;
        const char* src = (const char*)send[f.origin_src] + so;
        char* dst = (char*)recv[f.origin_dst] + dofs;
        if (c->path == HOCCL_PATH_CE) {
          CU_TRY(c, cudaMemcpyAsync(dst, src, it.bytes, cudaMemcpyDeviceToDevice, lane));
        } else {
          CopyBatch b;
          b.nseg = 1;
          b.pad = 0;
          b.seg[0] = CopySeg{src, dst, (unsigned long long)it.bytes};
          CU_TRY(c, launch_copy(b, (int)c->copy_ctas, lane));
          launches++;
        }
        moves++;
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
  return HOCCL_OK;
}

hoccl_result_t hoccl_profile_reset(hoccl_comm_t c) {
  if (!c) return HOCCL_ERR_INVALID_ARG;
  harvest_profile(c);
  c->prof_ms = 0;
  c->prof_bytes = 0;
  c->prof_n = 0;
  return HOCCL_OK;
}

hoccl_result_t hoccl_probe_move_needs_sm(hoccl_comm_t c, hoccl_path_t path, void* dst, const void* src, size_t bytes, int spin_us,
                                         int* needs_sm, double* move_end_us) {
  if (!c || !dst || !src || !needs_sm || bytes == 0 || spin_us < 100 || spin_us > 20000) return HOCCL_ERR_INVALID_ARG;
  CU_TRY(c, cudaSetDevice(c->device));
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
  if (e == cudaSuccess) {
    if (path == HOCCL_PATH_CE) {
      e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, c->lane[1]);  // src may be pinned host memory (control)
    } else {
      CopyBatch b;
      b.nseg = 1;
      b.pad = 0;
      b.seg[0] = CopySeg{src, dst, (unsigned long long)bytes};
      e = launch_copy(b, (int)c->copy_ctas, c->lane[1]);
    }
  }
  if (e == cudaSuccess) e = cudaEventRecord(b1, c->lane[1]);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  float spin_ms = 0, end_ms = 0;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&spin_ms, a0, a1);
  if (e == cudaSuccess) e = cudaEventElapsedTime(&end_ms, a0, b1);
  if (e != cudaSuccess) rc = cuda_fail(c, e, "probe_move_needs_sm");
  else {
    *needs_sm = end_ms >= 0.9f * spin_ms ? 1 : 0;
    if (move_end_us) *move_end_us = end_ms * 1e3;
  }
  cudaEventDestroy(a0);
  cudaEventDestroy(a1);
  cudaEventDestroy(b1);
  return rc;
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

hoccl_result_t hoccl_copy_launch(const void* src, void* dst, size_t bytes, int ctas, hoccl_stream_t stream) {
  if (!src || !dst || ctas < 1 || ctas > 1024) return HOCCL_ERR_INVALID_ARG;
  if (bytes == 0) return HOCCL_OK;
  CopyBatch b;
  b.nseg = 1;
  b.pad = 0;
  b.seg[0] = CopySeg{src, dst, (unsigned long long)bytes};
  return launch_copy(b, ctas, (cudaStream_t)stream) == cudaSuccess ? HOCCL_OK : HOCCL_ERR_CUDA;
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
