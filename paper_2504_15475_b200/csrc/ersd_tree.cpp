// Host-side helpers around draft trees (no GPU work).
//
// ersd_optimal_tree: the draft tree with the largest expected number of accepted tokens
// (Section 4 of the paper, "Optimal tree construction").  Because a vertex can only be accepted
// when its ancestors are, the optimum is the set of the k vertices of highest acceptance
// probability, and those can be collected best-first: the frontier holds every vertex that is not
// in the tree yet but whose parent and previous sibling are; taking the best frontier vertex makes
// exactly two more vertices eligible, its first child and its next sibling.  Acceptance
// probabilities follow the 0-th order model of the paper's experiments: a vertex reached through
// child ranks (j_1, .., j_m) has R = a[j_1] * ... * a[j_m].  R is formed from the COUNT of each
// rank on the path, multiplied out in ascending rank order, so two vertices that use the same
// ranks in another order get bit-identical R and the stated tie order (shallower first, then
// lexicographic) really decides between them.
//
// ersd_acceptance_profile: the empirical a[r] of Section 5 from verified paths.
#include <stdint.h>

#include <algorithm>
#include <queue>
#include <vector>

#include "ersd.h"

namespace {

struct Node {
  int parent;   // arena index of the parent vertex, -1 for children of the root
  int rank;     // child rank under its parent
  int depth;    // 1 for children of the root
  double r;     // acceptance probability
};

class Arena {
 public:
  Arena(const double* accept, int C) : accept_(accept), C_(C) {}

  int add(int parent, int rank) {
    Node n;
    n.parent = parent;
    n.rank = rank;
    n.depth = parent < 0 ? 1 : nodes_[parent].depth + 1;
    nodes_.push_back(n);
    const int id = (int)nodes_.size() - 1;
    nodes_[id].r = probability(id);
    return id;
  }
  const Node& operator[](int id) const { return nodes_[id]; }

  // child ranks from the root, for the lexicographic tie order
  std::vector<int> path(int id) const {
    std::vector<int> p;
    for (int v = id; v >= 0; v = nodes_[v].parent) p.push_back(nodes_[v].rank);
    std::reverse(p.begin(), p.end());
    return p;
  }

 private:
  // product of accept[rank] over the path, taken rank by rank in ascending order
  double probability(int id) const {
    std::vector<int> count(C_, 0);
    for (int v = id; v >= 0; v = nodes_[v].parent) ++count[nodes_[v].rank];
    double r = 1.0;
    for (int q = 0; q < C_; ++q)
      for (int n = 0; n < count[q]; ++n) r *= accept_[q];
    return r;
  }
  const double* accept_;
  int C_;
  std::vector<Node> nodes_;
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
  Arena arena(accept, C);
  // frontier order: highest R first; ties: shallower, then lexicographically smaller path
  auto worse = [&arena](int a, int b) {
    if (arena[a].r != arena[b].r) return arena[a].r < arena[b].r;
    if (arena[a].depth != arena[b].depth) return arena[a].depth > arena[b].depth;
    return arena.path(a) > arena.path(b);
  };
  std::priority_queue<int, std::vector<int>, decltype(worse)> frontier(worse);
  frontier.push(arena.add(-1, 0));
  std::vector<int> chosen;
  double total = 0.0;
  while ((int)chosen.size() < k && !frontier.empty()) {
    const int v = frontier.top();
    frontier.pop();
    chosen.push_back(v);
    total += arena[v].r;
    frontier.push(arena.add(v, 0));                                           // its first child
    if (arena[v].rank + 1 < C) frontier.push(arena.add(arena[v].parent, arena[v].rank + 1));  // its next sibling
  }
  // Node ids in lexicographic vertex order (parents before children, siblings by rank): a
  // depth-first walk over the chosen vertices' child lists.
  std::vector<int> slot_of_arena;  // arena id -> index in `chosen`
  {
    int max_id = 0;
    for (int v : chosen) max_id = std::max(max_id, v);
    slot_of_arena.assign((size_t)max_id + 1, -1);
    for (size_t s = 0; s < chosen.size(); ++s) slot_of_arena[chosen[s]] = (int)s;
  }
  // children lists: a vertex of rank r hangs behind its sibling of rank r - 1 (which was chosen before it)
  std::vector<std::vector<int>> kids(chosen.size() + 1);  // index 0: the root, 1 + slot: a chosen vertex
  for (size_t s = 0; s < chosen.size(); ++s) {
    const Node& n = arena[chosen[s]];
    const int holder = n.parent < 0 ? 0 : 1 + slot_of_arena[n.parent];
    if ((int)kids[holder].size() <= n.rank) kids[holder].resize((size_t)n.rank + 1, -1);
    kids[holder][n.rank] = (int)s;
  }
  parent_out[0] = -1;
  int next_id = 1;
  // (to number in lexicographic order the walk finishes a child's subtree before its next sibling)
  struct Frame {
    int holder, holder_id, next_rank;
  };
  std::vector<Frame> frames;
  frames.push_back(Frame{0, 0, 0});
  while (!frames.empty()) {
    Frame& f = frames.back();
    if (f.next_rank >= (int)kids[f.holder].size()) {
      frames.pop_back();
      continue;
    }
    const int s = kids[f.holder][f.next_rank++];
    if (s < 0) continue;
    const int id = next_id++;
    parent_out[id] = f.holder_id;
    frames.push_back(Frame{1 + s, id, 0});
  }
  if (expected_tokens) *expected_tokens = total;
  return ERSD_OK;
}

// Empirical acceptance profile (Section 5 of the paper: the acceptance probability function R is
// estimated from observed acceptances and treated as a 0-th order Markov source).  From the
// accepted paths of B verified sequences over one draft tree: every node on a path was verified,
// which put each of its children to the test -- a trial for that child's rank -- and the path's
// next node, if any, is the child that was accepted.  accept[r] = acceptances / trials of rank r.
extern "C" int ersd_acceptance_profile(const int32_t* paths, const int32_t* parent, int B, int N,
                                       int max_children, double* accept, int64_t* trials) {
  if (!paths || !parent || !accept || B < 0 || N < 0 || max_children < 1) return ERSD_EINVAL;
  if (N + 1 > ERSD_MAX_ROWS) return ERSD_EUNSUPPORTED;
  const int nodes = N + 1;
  if (parent[0] != -1) return ERSD_EINVAL;
  std::vector<int> nchild(nodes, 0), rank(nodes, 0), depth(nodes, 0);
  int D = 0;
  for (int n = 1; n < nodes; ++n) {
    if (parent[n] < 0 || parent[n] >= n) return ERSD_EINVAL;
    rank[n] = nchild[parent[n]]++;
    depth[n] = depth[parent[n]] + 1;
    D = std::max(D, depth[n]);
  }
  std::vector<int64_t> hit(max_children, 0), tried(max_children, 0);
  for (int b = 0; b < B; ++b) {
    const int32_t* path = paths + (int64_t)b * (D + 1);
    for (int d = 0; d <= D; ++d) {
      const int n = path[d];
      if (n < 0) break;
      if (n >= nodes || (d == 0 && n != 0) || (d > 0 && parent[n] != path[d - 1])) return ERSD_EINVAL;
      for (int r = 0; r < nchild[n] && r < max_children; ++r) ++tried[r];
      if (d < D && path[d + 1] >= 0 && path[d + 1] < nodes && rank[path[d + 1]] < max_children)
        ++hit[rank[path[d + 1]]];
    }
  }
  for (int r = 0; r < max_children; ++r) {
    accept[r] = tried[r] > 0 ? (double)hit[r] / (double)tried[r] : 0.0;
    // ersd_optimal_tree wants ranks ordered by acceptance: an estimate that rises with the rank
    // (sampling noise; an untried rank after a tried one) is capped at its predecessor
    if (r > 0 && accept[r] > accept[r - 1]) accept[r] = accept[r - 1];
    if (trials) trials[r] = tried[r];
  }
  return ERSD_OK;
}
