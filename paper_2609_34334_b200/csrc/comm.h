// Shared internals of libhoccl: the communicator object and small helpers used by the executors, the point-to-point
// path, the pattern executor and the C ABI.
#pragma once
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
#include "../../include/hoccl_diag.h"
#include "kernels.cuh"
#include "plan.h"
#include "proxy.h"
#include "sched.h"

namespace hoccl {

constexpr int kMaxRanks = 64;
constexpr int kMaxLanes = 8;
constexpr size_t kGraphCacheCap = 48;

inline double now_us() {
  return std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

struct Seg {
  const char* src;    // MOVE: source; SUM: inbox
  const char* local;  // SUM only
  char* dst;
  uint64_t bytes;
  uint64_t host_off = 0;  // HOCCL_PATH_CE_HOST: where this move bounces in the pinned host staging
  int nsrc = 1;           // OP_CHAIN: inbox operands at src + j * src_stride
  uint64_t src_stride = 0;
  bool host_first = true; // HOCCL_PATH_CE_HOST: this move issues the outbound copy into host_off (false: another move of the group did)
};

struct RGroup {
  int kind;
  int piece;
  int phase = 0;   // plan phase of the group (reduce-scatter, all-gather, own chunk, all-to-all stage)
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
  cudaEvent_t at_post;   // recorded on `stream` when the post was made: the move waits for this point, not for later work
};

// One host <-> staging copy of the pipelined host all-reduce: `rows` rows of `width` bytes at `pitch` (rows == 1: plain).
struct HostCopy {
  char* dev;
  char* host;
  size_t pitch, width, rows;
};

struct GraphEntry {
  std::vector<uint64_t> key;
  cudaGraphExec_t exec = nullptr;
  uint64_t last_use = 0;
  long n_moves = 0, n_move_launches = 0, n_sum_launches = 0, n_pieces = 0, n_order_launches = 0;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof_events;  // owned; only with profile = 1
  std::vector<double> prof_bytes;
  bool prof_pending = false;  // replayed since the profile events were last read
  // pipelined host all-reduce: one graph per piece, and the host copies in front of and behind each of them
  std::vector<cudaGraphExec_t> piece_exec;
  std::vector<std::vector<HostCopy>> h2d, d2h;   // [piece]
  // "ce_overlap" setting: per piece three graphs (the reduce-scatter's moves, the sum, the all-gather's moves) that run on three
  // internal streams, so that one piece's driver copies overlap another piece's sum (inside ONE graph they never did)
  std::vector<cudaGraphExec_t> part_exec;   // [piece * 3 + part], null where a part is empty
  // "fused" setting: the whole plan as one cooperative kernel instead of a graph (exec stays null)
  std::vector<char> ring_args;  // a RingArgsSmall or RingArgsLarge, by value
  bool ring_large = false;
  int ring_grid = 0, ring_threads = 0;
  bool ring_has_sum = false;
  // "roles" setting: the direct schedule as one cooperative kernel with summing and moving CTAs (exec stays null)
  char* roles_tab = nullptr;    // owned device memory: the segment tables of this call signature
  std::vector<char> roles_args; // a RolesArgs, by value
  const void* roles_fn = nullptr;
  int roles_grid = 0, roles_sum_ctas = 0;
  size_t roles_smem = 0;        // dynamic shared memory of the launch = size of the tables
};

}  // namespace hoccl

struct hoccl_comm {
  int R = 0, device = 0, num_sms = 0;
  hoccl_path_t path = HOCCL_PATH_CE;
  long sum_ctas = 8, copy_ctas = 8, piece_bytes = 4 << 20, max_pieces = 8, lanes = 4, use_graph = 1, profile = 0, p2p_split = 1, ce_sub_bytes = 0,
       handshake = 0, watchdog_ms = 10000, onepass = 0, forward = 0, fused = 0, host_pieces = 8, ag_direct = 2, order_kernels = 1, rs_direct = 2,
       ce_small_bytes = 8 << 20, ce_small_ctas = 148, p2p_strict = 0, ce_overlap = -1, model_gpus_per_node = 0, model_rdma_sub_bytes = 0, roles = 0, piece_grade = -1,
       roles_missing = 0 /* self-test only: summing CTAs wait for this many movers that do not exist */;
  bool piece_bytes_set = false;  // the caller chose a piece size: no automatic choice
  hoccl::Proxy* proxy = nullptr;
  cudaStream_t lane[hoccl::kMaxLanes] = {};
  cudaStream_t sum_stream = nullptr;
  int sum_priority = 0;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_next = 0;
  void* scratch = nullptr;
  size_t scratch_bytes = 0;
  void* staging = nullptr;
  size_t staging_bytes = 0;
  unsigned* ring_bar = nullptr;  // "fused" setting: three device words of the grid barrier (library owned, 16 bytes)
  int* ring_err = nullptr;       // mapped pinned host word the ring kernel sets when a barrier wait ran out
  int* ring_err_dev = nullptr;   // the same word as the device sees it
  char* roles_ctl = nullptr;     // "roles" setting: control words and per-piece counters of the roles kernel (library owned, 1 KiB)
  int* roles_err = nullptr;      // mapped pinned host word the roles kernel sets when a wait ran out
  int* roles_err_dev = nullptr;
  char* host_staging = nullptr;  // pinned host memory of the CE_HOST path
  size_t host_staging_bytes = 0;
  std::map<std::pair<int, int>, std::deque<hoccl::Post>> pending;
  std::vector<cudaEvent_t> post_events;   // free list of the events that mark parked posts
  int n_pending = 0;
  unsigned p2p_rr = 0;
  std::vector<hoccl::GraphEntry> cache;
  uint64_t use_counter = 0;
  hoccl_stats_t stats = {};
  std::string cuda_err;
  // profile accumulation
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof_pool;   // timing events of the stream executor
  std::vector<std::pair<std::pair<cudaEvent_t, cudaEvent_t>, double>> prof_open;  // recorded, not yet read
  double prof_ms = 0, prof_bytes = 0;
  long prof_n = 0;
  double prof_copy_ms = 0, prof_copy_bytes = 0;   // copy_kernel launches (graph executor)
  long prof_copy_n = 0;
};

namespace hoccl {

inline hoccl_result_t cuda_fail(hoccl_comm* c, cudaError_t e, const char* what) {
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

inline cudaEvent_t next_event(hoccl_comm* c) {
  if (c->ev_next == c->ev_pool.size()) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    c->ev_pool.push_back(e);
  }
  return c->ev_pool[c->ev_next++];
}

inline bool ranges_overlap(const char* a, size_t an, const char* b, size_t bn) {
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
  // hoccl_host_allreduce, pipelined form: the caller's HOST buffers; send/recv then point into the device staging and
  // the graph carries, per piece, the host-to-device copies in front of the ring and the device-to-host copies behind it
  const void* const* h_send = nullptr;
  void* const* h_recv = nullptr;
};


struct Tally {
  long moves = 0, move_launches = 0, sum_launches = 0;
};

// exec.cu
void fill_sum_batch(const RGroup& g, size_t first, size_t n, int dtype, size_t elem, SumBatch* b);
void fill_copy_batch(const RGroup& g, size_t first, size_t n, CopyBatch* b);
void fill_chain_batch(const RGroup& g, size_t first, size_t n, int dtype, size_t elem, ChainBatch* b);
// Moves of a group that read the same bytes (same source and length; the direct all-gather on the SM path) become fan-out
// segments: one read, one store per destination.  Returns false (and leaves *out empty) if no source repeats: the plain
// copy batches are used then.  bytes_out[i] = HBM bytes of batch i (reads + writes), moves_out[i] = moves it carries.
bool build_fan_batches(const RGroup& g, std::vector<FanBatch>* out, std::vector<double>* bytes_out, std::vector<long>* moves_out);
// graph.cu
// part < 0: every group (of `only_piece`, if that is >= 0); part 0 / 1 / 2: only the reduce-scatter's MOVE groups / the SUM and
// CHAIN groups / the remaining MOVE groups; dependencies on groups outside the part are left to the caller (events).
// *out_exec stays null when nothing falls into the selection.
hoccl_result_t build_graph(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry, int only_piece,
                           cudaGraphExec_t* out_exec, int part = -1);
void add_host_copies(const Plan& P, int p, char* dev, char* host, std::vector<HostCopy>* out);
cudaError_t enqueue_host_copy(const HostCopy& hc, bool to_device, cudaStream_t s);
// ring_host.cu
hoccl_result_t build_ring(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry);
// roles.cu
hoccl_result_t build_roles(hoccl_comm* c, const Plan& P, const std::vector<RGroup>& groups, GraphEntry* entry);
hoccl_result_t launch_roles(hoccl_comm* c, GraphEntry* entry, cudaStream_t stream);
// exec.cu
hoccl_result_t run_collective(hoccl_comm* c, Call* call, cudaStream_t user);
// HOCCL_OK if the communicator's settings fit together for such a call (see options.h); nothing is enqueued
hoccl_result_t check_options(hoccl_comm* c, int kind, size_t count, int dtype);
hoccl_result_t ensure_proxy(hoccl_comm* c);
void harvest_profile(hoccl_comm* c);
void destroy_entry(GraphEntry* e);
GraphEntry* cache_put(hoccl_comm* c, GraphEntry&& entry);
hoccl_result_t build_pattern_graph(hoccl_comm* c, const Schedule& S, const void* const* send, const size_t* sdispls, void* const* recv,
                                   const size_t* rdispls, size_t e, GraphEntry* entry);
hoccl_result_t build_pattern_graph_modelled(hoccl_comm* c, const Schedule& S, const void* const* send, const size_t* sdispls,
                                            void* const* recv, const size_t* rdispls, size_t e, char* out_stage, char* in_stage,
                                            const std::vector<uint64_t>& flow_stage_off, size_t chunk_bytes, size_t rdma_sub,
                                            GraphEntry* entry);
hoccl_result_t ring_barrier_selftest(hoccl_comm* c, void* dst, const void* src, size_t bytes, cudaStream_t stream);
// p2p.cu
hoccl_result_t p2p_post(hoccl_comm* c, bool is_send, void* buf, size_t count, int dtype, int src, int dst, cudaStream_t stream);

}  // namespace hoccl
