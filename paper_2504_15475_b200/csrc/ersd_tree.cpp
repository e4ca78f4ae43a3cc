// Host-side construction of the draft tree with the largest expected number of accepted tokens
// (Algorithm 3 of the paper): vertices are added greedily in order of acceptance probability,
// candidates kept in a priority queue; a popped vertex offers its first child and its next
// sibling.  Acceptance probabilities follow the 0-th order model of the paper's experiments:
// R(j_1..j_m) = a[j_1] * ... * a[j_m], a[r] = acceptance probability of a node's child of rank r.
#include <stdint.h>

#include <algorithm>
#include <queue>
#include <vector>

#include "ersd.h"

namespace {

struct Vertex {
  double r;                  // acceptance probability of the vertex
  std::vector<uint8_t> path;  // child ranks from the root
};

struct Worse {  // priority queue order: highest r first; ties: shallower, then lexicographic
  bool operator()(const Vertex& a, const Vertex& b) const {
    if (a.r != b.r) return a.r < b.r;
    if (a.path.size() != b.path.size()) return a.path.size() > b.path.size();
    return a.path > b.path;
  }
};

}  // namespace

extern "C" int ersd_optimal_tree(const double* accept, int max_children, int k, int32_t* parent_out,
                                 double* expected_tokens) {
  if (!accept || !parent_out || max_children < 1 || k < 0) return ERSD_EINVAL;
  if (k + 1 > ERSD_MAX_ROWS) return ERSD_EUNSUPPORTED;
  const int C = std::min(max_children, (int)ERSD_MAX_TOP_C);
  for (int r = 0; r < C; ++r) {
    if (!(accept[r] >= 0.0 && accept[r] <= 1.0)) return ERSD_EINVAL;
    if (r > 0 && accept[r] > accept[r - 1]) return ERSD_EINVAL;  // ranks are ordered by acceptance
  }
  std::priority_queue<Vertex, std::vector<Vertex>, Worse> queue;
  queue.push(Vertex{accept[0], {0}});
  std::vector<Vertex> tree;
  double total = 0.0;
  for (int i = 0; i < k && !queue.empty(); ++i) {
    Vertex v = queue.top();
    queue.pop();
    total += v.r;
    Vertex child = v;
    child.path.push_back(0);
    child.r = v.r * accept[0];
    queue.push(child);
    const int rank = v.path.back();
    if (rank + 1 < C) {
      Vertex sib = v;
      sib.path.back() = (uint8_t)(rank + 1);
      sib.r = accept[rank] > 0.0 ? v.r / accept[rank] * accept[rank + 1] : 0.0;
      queue.push(sib);
    }
    tree.push_back(v);
  }
  // parent array in lexicographic vertex order: parents precede children, siblings ascend by rank
  std::sort(tree.begin(), tree.end(), [](const Vertex& a, const Vertex& b) { return a.path < b.path; });
  parent_out[0] = -1;
  for (size_t n = 0; n < tree.size(); ++n) {
    const std::vector<uint8_t>& p = tree[n].path;
    int parent = 0;
    if (p.size() > 1) {
      const std::vector<uint8_t> up(p.begin(), p.end() - 1);
      const auto it = std::lower_bound(tree.begin(), tree.end(), up,
                                       [](const Vertex& v, const std::vector<uint8_t>& q) { return v.path < q; });
      parent = (int)(it - tree.begin()) + 1;
    }
    parent_out[n + 1] = parent;
  }
  if (expected_tokens) *expected_tokens = total;
  return ERSD_OK;
}
