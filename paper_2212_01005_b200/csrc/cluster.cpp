// Acyclic graph partitioning of the frontend (Section IV, Algorithm 1 "Cluster"), host only:
// operator weights (Eq. 1), topological stages (Definition 2), affix sets (Definition 3) and the
// greedy clustering loop. Where the paper leaves a choice open, this file fixes it:
//   * "nodes v can connect to" (Definition 3) are the nodes adjacent to v in the quotient graph;
//   * ties: the heaviest candidate with the smallest member id; the lightest affix node with
//     the smallest member id;
//   * c and b of Eq. 1 are the caller's (the paper fits them to tuning budgets and prints no values).
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <set>
#include <vector>

#include "../../include/ago.h"

namespace ago {
ago_status_t report_failure(ago_status_t s, const char* msg);   // records the thread's last error (api.cu)
}

namespace {

struct Hyper {
  std::vector<int> members;   // original node ids, ascending
  double weight = 0.0;
  bool alive = true, cand = true;
  int first() const { return members.front(); }
};

// Longest-path stage of every live hyper node (roots = 1); false if the quotient graph has a cycle.
bool topological_stages(const std::vector<Hyper>& h, const std::vector<std::set<int>>& succ,
                        const std::vector<std::set<int>>& pred, std::vector<int>* ts) {
  const int n = (int)h.size();
  std::vector<int> indeg(n, 0), order;
  ts->assign(n, 0);
  int live = 0;
  for (int v = 0; v < n; ++v)
    if (h[v].alive) { ++live; indeg[v] = (int)pred[v].size(); if (!indeg[v]) { order.push_back(v); (*ts)[v] = 1; } }
  for (size_t i = 0; i < order.size(); ++i) {
    const int v = order[i];
    for (int w : succ[v]) {
      (*ts)[w] = std::max((*ts)[w], (*ts)[v] + 1);
      if (--indeg[w] == 0) order.push_back(w);
    }
  }
  return (int)order.size() == live;
}

}  // namespace

extern "C" double ago_op_weight(const int64_t* loop_extents, int32_t num_loops, double c, double b) {
  if (!loop_extents || num_loops <= 0) return b;
  double prod = 1.0;
  for (int i = 0; i < num_loops; ++i) prod *= std::log((double)loop_extents[i]);
  return c * prod + b;
}

extern "C" ago_status_t ago_graph_cluster(const ago_graph_desc_t* g, int32_t* subgraph_of_node, int32_t* num_subgraphs) {
  auto fail = [](ago_status_t st, const char* msg) { return ago::report_failure(st, msg); };
  if (!g || !subgraph_of_node || !num_subgraphs) return fail(AGO_ERR_INVALID_ARG, "ago_graph_cluster: NULL argument");
  if (g->struct_size != sizeof(ago_graph_desc_t)) return fail(AGO_ERR_INVALID_ARG, "ago_graph_cluster: struct_size mismatch");
  const int n = g->num_nodes;
  if (n <= 0 || !g->weights || g->num_edges < 0 || (g->num_edges > 0 && !g->edges))
    return fail(AGO_ERR_INVALID_ARG, "ago_graph_cluster: empty graph or missing arrays");
  std::vector<Hyper> h(n);
  std::vector<std::set<int>> succ(n), pred(n);
  for (int v = 0; v < n; ++v) { h[v].members = {v}; h[v].weight = g->weights[v]; }
  for (int e = 0; e < g->num_edges; ++e) {
    const int u = g->edges[2 * e], v = g->edges[2 * e + 1];
    if (u < 0 || u >= n || v < 0 || v >= n || u == v) return fail(AGO_ERR_INVALID_ARG, "ago_graph_cluster: bad edge");
    succ[u].insert(v); pred[v].insert(u);
  }
  std::vector<int> ts;
  if (!topological_stages(h, succ, pred, &ts)) return fail(AGO_ERR_INVALID_ARG, "ago_graph_cluster: the graph has a cycle");

  while (true) {
    // the heaviest candidate
    int v = -1;
    for (int i = 0; i < n; ++i)
      if (h[i].alive && h[i].cand && (v < 0 || h[i].weight > h[v].weight || (h[i].weight == h[v].weight && h[i].first() < h[v].first()))) v = i;
    if (v < 0) break;
    // the lightest node of its affix set: adjacent, one stage above or below
    int u = -1;
    auto consider = [&](int w) {
      if (std::abs(ts[w] - ts[v]) != 1) return;
      if (u < 0 || h[w].weight < h[u].weight || (h[w].weight == h[u].weight && h[w].first() < h[u].first())) u = w;
    };
    for (int w : succ[v]) consider(w);
    for (int w : pred[v]) consider(w);
    if (u >= 0 && h[v].weight + h[u].weight < g->threshold) {
      // u joins v; the hyper node stays a candidate
      h[v].members.insert(h[v].members.end(), h[u].members.begin(), h[u].members.end());
      std::sort(h[v].members.begin(), h[v].members.end());
      h[v].weight += h[u].weight;
      h[u].alive = false;
      for (int w : succ[u]) { pred[w].erase(u); if (w != v) { succ[v].insert(w); pred[w].insert(v); } }
      for (int w : pred[u]) { succ[w].erase(u); if (w != v) { pred[v].insert(w); succ[w].insert(v); } }
      succ[u].clear(); pred[u].clear();
      succ[v].erase(v); pred[v].erase(v);
      if (!topological_stages(h, succ, pred, &ts)) return fail(AGO_ERR_INVALID_ARG, "ago_graph_cluster: internal: partition became cyclic");
    } else {
      h[v].cand = false;
    }
  }
  // number the subgraphs by their smallest member
  std::vector<int> live;
  for (int i = 0; i < n; ++i) if (h[i].alive) live.push_back(i);
  std::sort(live.begin(), live.end(), [&](int a, int b) { return h[a].first() < h[b].first(); });
  for (size_t s = 0; s < live.size(); ++s)
    for (int m : h[live[s]].members) subgraph_of_node[m] = (int32_t)s;
  *num_subgraphs = (int32_t)live.size();
  return AGO_OK;
}
