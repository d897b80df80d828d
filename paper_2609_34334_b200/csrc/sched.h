// Collective scheduler of the paper (Sec. 3.4), host only:
//   origin traffic matrix C  ->  HOCCL traffic matrix T (Eq. 2-4: forwarding copies on the (u, u-bar) edges)
//   ->  stages T^1..T^n by the Birkhoff-like decomposition (Algorithm 1; completeness Eq. 5-6, per-stage RDMA
//   degree bound Eq. 7, stage time Eq. 8-9, objective Eq. 10)  ->  per stage and per DMA engine a weighted
//   interleaving of fixed-size chunks ("Flow-size-aware chunk scheduling").
//
// Topology model: G GPUs in nodes of `gpus_per_node`; GPUs of one node form an NVLink domain, entries between nodes
// form the RDMA domain; the symmetric peer of GPU u is u ^ 1 inside its node (the GPU under the same PCIe switch).
// With one node (the single-device build: G = R logical ranks) the RDMA domain is empty, T = C, and the stages are
// the matching components of the native traffic.
//
// Readings where the paper is informal: the "largest removable portion" of a matching is the smallest entry on
// it; NVLink slack of a stage = tau * B_nvlink - the largest forwarding load on an edge of that domain; a DMA
// engine is the one of the SOURCE GPU of a copy (it serves that GPU's native sends and both kinds of forwarding
// copies that start there).
#pragma once
#include <cstdint>
#include <vector>

namespace hoccl {

struct Topology {
  int G = 1;
  int gpus_per_node = 1;
  double bw_nvlink = 400e9;  // bytes per second per NVLink edge
  double bw_rdma = 50e9;     // bytes per second per NIC
  int node_of(int g) const { return g / gpus_per_node; }
  int peer_of(int g) const {
    int p = g ^ 1;
    return (p < G && node_of(p) == node_of(g)) ? p : g;
  }
  bool same_node(int a, int b) const { return node_of(a) == node_of(b); }
  int num_nodes() const { return (G + gpus_per_node - 1) / gpus_per_node; }
};

enum FlowClass { FLOW_NATIVE = 0, FLOW_RDMA = 1, FLOW_FWD_SEND = 2, FLOW_FWD_RECV = 3 };

// One entry of a stage: `bytes` of traffic from u to v of a given class.  For forwarding copies `origin_src` /
// `origin_dst` name the logical (inter-node) flow they belong to.
struct StageFlow {
  int u, v;
  int cls;
  int origin_src, origin_dst;
  uint64_t bytes;
  uint64_t origin_offset;  // position of these bytes inside the logical flow C[origin_src][origin_dst]
};

struct ChunkItem {
  int flow;  // index into Stage::flows
  uint64_t offset, bytes;  // inside that stage flow
};

struct Stage {
  std::vector<StageFlow> flows;
  double tau = 0;                               // Eq. 9
  std::vector<std::vector<ChunkItem>> queues;   // per GPU (DMA engine of the source), service order
};

struct Schedule {
  Topology topo;
  std::vector<uint64_t> C, T;  // G x G, row = source
  std::vector<Stage> stages;
  double total_tau = 0;        // Eq. 10
  double lower_bound = 0;      // max over endpoints and domains of load / bandwidth (no schedule can beat it)
};

// Eq. 2-4.  C and T are G x G row-major byte counts; diagonal entries (local copies) are passed through.
void expand_traffic(const Topology& topo, const std::vector<uint64_t>& C, std::vector<uint64_t>* T);

// Algorithm 1 + chunk scheduling.  chunk_bytes > 0.  Returns false on bad arguments.
bool build_schedule(const Topology& topo, const std::vector<uint64_t>& C, uint64_t chunk_bytes, Schedule* out);

// Weighted interleaving of the chunks of several flows on one serial queue: flow i has bytes[i] bytes, cut into
// chunks of chunk_bytes (the last one shorter).  Service is proportional to flow size (smooth weighted round-robin on
// the chunk counts), so all flows finish near the end and no flow waits long.  Output: (flow index, chunk index).
void interleave_chunks(const std::vector<uint64_t>& bytes, uint64_t chunk_bytes, std::vector<std::pair<int, uint64_t>>* order);

}  // namespace hoccl
