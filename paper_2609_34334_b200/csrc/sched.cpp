// Collective scheduler (see sched.h): traffic-matrix expansion, Birkhoff-like stage decomposition, chunk interleaving.
#include "sched.h"

#include <algorithm>
#include <functional>
#include <map>
#include <numeric>

namespace hoccl {

void expand_traffic(const Topology& topo, const std::vector<uint64_t>& C, std::vector<uint64_t>* T) {
  const int G = topo.G;
  *T = C;
  for (int u = 0; u < G; u++)
    for (int v = 0; v < G; v++) {
      const uint64_t f = C[(size_t)u * G + v];
      if (!f || u == v || topo.same_node(u, v)) continue;
      // f => f' + f + f'': sender-side copy on (u, u-bar), the RDMA transfer, receiver-side copy on (v-bar, v)
      const int pu = topo.peer_of(u), pv = topo.peer_of(v);
      if (pu != u) (*T)[(size_t)u * G + pu] += f;  // A_u
      if (pv != v) (*T)[(size_t)pv * G + v] += f;  // B_v
    }
}

void interleave_chunks(const std::vector<uint64_t>& bytes, uint64_t chunk_bytes, std::vector<std::pair<int, uint64_t>>* order) {
  order->clear();
  const int n = (int)bytes.size();
  std::vector<long long> w(n), cur(n, 0);
  std::vector<uint64_t> next(n, 0);
  long long total = 0;
  for (int i = 0; i < n; i++) {
    w[i] = (long long)((bytes[i] + chunk_bytes - 1) / chunk_bytes);
    total += w[i];
  }
  order->reserve((size_t)total);
  // smooth weighted round-robin: every slot each flow earns its weight, the richest flow is served and pays `total`
  for (long long slot = 0; slot < total; slot++) {
    int best = -1;
    for (int i = 0; i < n; i++) {
      if (next[i] >= (uint64_t)w[i]) continue;
      cur[i] += w[i];
      if (best < 0 || cur[i] > cur[best]) best = i;
    }
    cur[best] -= total;
    order->push_back({best, next[best]++});
  }
}

namespace {

typedef std::vector<std::pair<int, int>> Matching;

// Maximum-cardinality matching on the positive entries of M restricted by `allowed`; heavy rows and heavy entries
// are tried first so that large flows are peeled early.
Matching max_matching(int G, const std::vector<uint64_t>& M, const std::function<bool(int, int)>& allowed) {
  std::vector<std::vector<int>> adj(G);
  std::vector<uint64_t> rowsum(G, 0);
  for (int u = 0; u < G; u++) {
    for (int v = 0; v < G; v++)
      if (M[(size_t)u * G + v] && allowed(u, v)) {
        adj[u].push_back(v);
        rowsum[u] += M[(size_t)u * G + v];
      }
    std::sort(adj[u].begin(), adj[u].end(), [&](int a, int b) { return M[(size_t)u * G + a] > M[(size_t)u * G + b]; });
  }
  std::vector<int> rows(G);
  std::iota(rows.begin(), rows.end(), 0);
  std::stable_sort(rows.begin(), rows.end(), [&](int a, int b) { return rowsum[a] > rowsum[b]; });
  std::vector<int> match_col(G, -1);
  std::function<bool(int, std::vector<char>&)> augment = [&](int u, std::vector<char>& seen) -> bool {
    for (int v : adj[u]) {
      if (seen[v]) continue;
      seen[v] = 1;
      if (match_col[v] < 0 || augment(match_col[v], seen)) {
        match_col[v] = u;
        return true;
      }
    }
    return false;
  };
  for (int u : rows) {
    if (adj[u].empty()) continue;
    std::vector<char> seen(G, 0);
    augment(u, seen);
  }
  Matching m;
  for (int v = 0; v < G; v++)
    if (match_col[v] >= 0) m.push_back({match_col[v], v});
  std::sort(m.begin(), m.end());
  return m;
}

struct Component {
  Matching m;
  uint64_t amount;
};

}  // namespace

bool build_schedule(const Topology& topo, const std::vector<uint64_t>& C, uint64_t chunk_bytes, Schedule* out) {
  const int G = topo.G;
  if (G < 1 || topo.gpus_per_node < 1 || chunk_bytes == 0 || C.size() != (size_t)G * G || topo.bw_nvlink <= 0 || topo.bw_rdma <= 0)
    return false;
  Schedule& S = *out;
  S = Schedule();
  S.topo = topo;
  S.C = C;
  expand_traffic(topo, C, &S.T);
  auto at = [&](std::vector<uint64_t>& M, int u, int v) -> uint64_t& { return M[(size_t)u * G + v]; };

  // residuals: inter-node logical flows, native intra-node flows, local copies
  std::vector<uint64_t> Rr((size_t)G * G, 0), Rn((size_t)G * G, 0), off((size_t)G * G, 0);
  std::vector<std::pair<int, uint64_t>> local;
  for (int u = 0; u < G; u++)
    for (int v = 0; v < G; v++) {
      uint64_t f = C[(size_t)u * G + v];
      if (!f) continue;
      if (u == v) local.push_back({u, f});
      else if (topo.same_node(u, v)) at(Rn, u, v) = f;
      else at(Rr, u, v) = f;
    }

  // Algorithm 1, line 2: native NVLink traffic of every domain as matching components
  const int nodes = topo.num_nodes();
  std::vector<std::vector<Component>> comps(nodes);
  for (int d = 0; d < nodes; d++) {
    for (;;) {
      Matching m = max_matching(G, Rn, [&](int u, int v) { return topo.node_of(u) == d && topo.node_of(v) == d; });
      if (m.empty()) break;
      uint64_t amt = UINT64_MAX;
      for (auto& e : m) amt = std::min(amt, at(Rn, e.first, e.second));
      for (auto& e : m) at(Rn, e.first, e.second) -= amt;
      comps[d].push_back(Component{m, amt});
    }
  }
  std::vector<size_t> comp_next(nodes, 0);
  auto add_native = [&](Stage& st, int d, uint64_t budget) -> uint64_t {
    // moves up to `budget` bytes per entry of domain d's next matching component(s) into the stage
    uint64_t used_max = 0;
    while (budget > 0 && comp_next[d] < comps[d].size()) {
      Component& c = comps[d][comp_next[d]];
      uint64_t p = std::min(c.amount, budget);
      for (auto& e : c.m) {
        st.flows.push_back(StageFlow{e.first, e.second, FLOW_NATIVE, e.first, e.second, p, at(off, e.first, e.second)});
        at(off, e.first, e.second) += p;
      }
      c.amount -= p;
      budget -= p;
      used_max += p;
      if (c.amount == 0) comp_next[d]++;
      // one component per stage and domain keeps every GPU at one native send and one native receive
      break;
    }
    return used_max;
  };

  bool locals_placed = false;
  auto place_locals = [&](Stage& st) {
    if (locals_placed) return;
    locals_placed = true;
    for (auto& l : local) st.flows.push_back(StageFlow{l.first, l.first, FLOW_NATIVE, l.first, l.first, l.second, 0});
  };

  // Algorithm 1, lines 3-10
  for (;;) {
    Matching m = max_matching(G, Rr, [&](int, int) { return true; });
    if (m.empty()) break;
    Stage st;
    uint64_t amt = UINT64_MAX;
    for (auto& e : m) amt = std::min(amt, at(Rr, e.first, e.second));  // largest portion removable from every entry
    std::map<std::pair<int, int>, uint64_t> edge_load;                   // forwarding bytes per NVLink edge
    for (auto& e : m) {
      const int u = e.first, v = e.second;
      const uint64_t o = at(off, u, v);
      st.flows.push_back(StageFlow{u, v, FLOW_RDMA, u, v, amt, o});
      const int pu = topo.peer_of(u), pv = topo.peer_of(v);
      if (pu != u) {
        st.flows.push_back(StageFlow{u, pu, FLOW_FWD_SEND, u, v, amt, o});
        edge_load[{u, pu}] += amt;
      }
      if (pv != v) {
        st.flows.push_back(StageFlow{pv, v, FLOW_FWD_RECV, u, v, amt, o});
        edge_load[{pv, v}] += amt;
      }
      at(off, u, v) += amt;
      at(Rr, u, v) -= amt;
    }
    std::vector<uint64_t> fwd_max(nodes, 0);
    uint64_t fwd_all = 0;
    for (auto& kv : edge_load) {
      fwd_max[topo.node_of(kv.first.first)] = std::max(fwd_max[topo.node_of(kv.first.first)], kv.second);
      fwd_all = std::max(fwd_all, kv.second);
    }
    double tau = std::max((double)amt / topo.bw_rdma, (double)fwd_all / topo.bw_nvlink);
    // line 8: fill the NVLink slack of every domain with a native matching component
    for (int d = 0; d < nodes; d++) {
      double slack = tau * topo.bw_nvlink - (double)fwd_max[d];
      if (slack >= 1.0) add_native(st, d, (uint64_t)slack);
    }
    place_locals(st);
    st.tau = tau;
    S.stages.push_back(std::move(st));
  }
  // what is left is native NVLink traffic only: one matching component per domain and stage
  for (;;) {
    bool any = false;
    for (int d = 0; d < nodes; d++) any = any || comp_next[d] < comps[d].size();
    if (!any) break;
    Stage st;
    uint64_t biggest = 0;
    for (int d = 0; d < nodes; d++) biggest = std::max(biggest, add_native(st, d, UINT64_MAX));
    place_locals(st);
    st.tau = (double)biggest / topo.bw_nvlink;
    S.stages.push_back(std::move(st));
  }
  if (!locals_placed && !local.empty()) {
    Stage st;
    place_locals(st);
    S.stages.push_back(std::move(st));
  }

  // flow-size-aware chunk scheduling: one serial queue per DMA engine (source GPU) and stage
  for (Stage& st : S.stages) {
    st.queues.assign(G, {});
    for (int g = 0; g < G; g++) {
      std::vector<int> mine;
      std::vector<uint64_t> bytes;
      for (size_t i = 0; i < st.flows.size(); i++)
        if (st.flows[i].u == g && st.flows[i].cls != FLOW_RDMA) {  // the NIC, not the DMA engine, carries the RDMA leg
          mine.push_back((int)i);
          bytes.push_back(st.flows[i].bytes);
        }
      std::vector<std::pair<int, uint64_t>> order;
      interleave_chunks(bytes, chunk_bytes, &order);
      for (auto& o : order) {
        const uint64_t b = bytes[o.first];
        const uint64_t lo = o.second * chunk_bytes;
        st.queues[g].push_back(ChunkItem{mine[o.first], lo, std::min(chunk_bytes, b - lo)});
      }
    }
    S.total_tau += st.tau;
  }

  // a bound no schedule can beat: the busiest RDMA endpoint and the busiest NVLink edge
  double lb = 0;
  for (int u = 0; u < G; u++) {
    uint64_t out_r = 0, in_r = 0;
    for (int v = 0; v < G; v++) {
      if (u != v && !topo.same_node(u, v)) {
        out_r += C[(size_t)u * G + v];
        in_r += C[(size_t)v * G + u];
      }
      if (u != v && topo.same_node(u, v)) lb = std::max(lb, (double)S.T[(size_t)u * G + v] / topo.bw_nvlink);
    }
    lb = std::max(lb, std::max((double)out_r, (double)in_r) / topo.bw_rdma);
  }
  S.lower_bound = lb;
  return true;
}

}  // namespace hoccl
