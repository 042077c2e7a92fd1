// CPU oracle for per-step draft construction (arXiv 2503.05330, Method section
// and Algorithm 1).  TEST INFRASTRUCTURE ONLY: a plain, slow, brute-force
// restatement of the method, used to check the CUDA library and timed as the
// CPU baseline.  It shares no code with the CUDA path and is never called by it.
//
// What each step follows:
//   state      - paths y_1..y_N that grow token by token ("Dynamic Draft Pool
//                Construction"), with the model probability of every generated
//                token (the p_theta of Eq. 5).
//   match      - Eq. 3: every position of every OTHER path of the same prompt
//                whose prefix ends with the query path's k-token suffix; with a
//                tolerance eps (Eq. 4, "Fuzzy Suffix Matching") every position
//                where some window s' ends with edit distance delta(q, s') <= eps.
//   candidates - the tokens following each match (at most D of them).
//   DAG        - "Consensus-Driven Draft Extraction": layer d holds the distinct
//                d-th follower tokens; edge (u,v) between layers d-1 and d
//                carries Eq. 5: alpha * sum_i p_i + (1-alpha) * Freq(u->v).
//   search     - greedy walk: at each layer take the token whose summed
//                in-edge weight is highest; stop at length D or at a leaf.
//   accept     - "Draft acceptance": longest prefix of the draft equal to the
//                sampled tokens.
//   trim       - a sliding window for runs longer than the capacity: a path forgets
//                its oldest tokens (the paper's runs are short; not part of its method).
//   tree, list - the two weaker draft pools of the "Ablation Study": a tree merges
//                candidates only along identical prefixes, a list does not merge.
//
// Readings where the paper is silent (all restated in the design notes):
//   * followers start one position after the matched suffix;
//   * a match needs at least one follower; a path never searches itself;
//   * probabilities are held as integers pq = round_half_even(exp(logprob)*2^30),
//     sums S are exact 64-bit integers, so results do not depend on the order
//     of accumulation;  Freq(u->v) is the raw instance count;
//   * weight = alpha*(S/2^30) + (1-alpha)*cnt evaluated in double, each
//     operation rounded separately (build with -ffp-contract=off);
//   * the walk only moves to successors of the node it stands on (mode 0);
//     mode 1 takes the best node of each layer regardless of the previous one;
//     mode 2 replaces the greedy walk by the path of the DAG with the largest sum of
//     node weights (not in the paper's method; its introduction motivates it);
//   * ties go to the smallest token id;
//   * optionally (max_matches = R > 0) a query keeps, of its matches in one source path, only
//     the R with the largest end positions; the default keeps all, as Eq. 3 does.
//
// Pins (tests/, CPU only): hand-worked example from Eq. 3 / Eq. 5 with dyadic
// probabilities; match set against regex/numpy searches and closed-form counts;
// alpha = 0 against collections.Counter; conservation invariants; enumeration
// of every root-to-node DAG path; fuzzy matches against exact search for every
// string within one edit of the query; pq against 50-digit decimal arithmetic;
// acceptance against os.path.commonprefix; the match cap against slices of the
// uncapped match set and a hand-worked case.  Behaviour on real model traces
// (the paper's Table 1) is "parity unpinned": it needs the models and datasets.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <thread>
#include <utility>
#include <vector>
#include <algorithm>

namespace {

constexpr int64_t ONE_Q30 = int64_t(1) << 30;

enum : uint32_t {
  ST_BAD_COUNT = 1u, ST_CAPACITY = 2u, ST_BAD_TOKEN = 4u, ST_BAD_LOGPROB = 8u,
};

struct Acc { int64_t S = 0; int64_t cnt = 0; };

struct PathResult {
  bool valid = false;                       // query existed (len >= k, path not full)
  int root = -1;
  std::vector<std::pair<int, int>> matches; // (path j, index e of last matched token)
  // layers[d-1] for d = 1..D
  std::vector<std::map<int, Acc>> nodes;
  std::vector<std::map<std::pair<int, int>, Acc>> edges;  // key (u, v)
  std::vector<int> draft;
  std::vector<double> score, edge_w;
  // several drafts (beams) of the best-path search, best first
  std::vector<std::vector<int>> beam_tok;
  std::vector<double> beam_value;
};

struct Ctx {
  int G, N, L, V, D, mode;
  int eps = 0;                                  // edit-distance tolerance of the suffix match (Eq. 4)
  int pool = 0;                                 // draft pool of the ablation: 0 DAG, 1 tree, 2 list
  int max_matches = 0;                          // R: per (query path, source path) only the R most recent matches count; 0 = all
  double alpha;
  std::vector<std::vector<int32_t>> tok, pq;
  std::vector<PathResult> res;
};

// Eq. 5 with S in units of 2^-30 (probability sum) and cnt = Freq.
double weight(double alpha, int64_t S, int64_t cnt) {
  double t1 = alpha * (double)S;
  t1 = t1 * (1.0 / (double)ONE_Q30);
  double t2 = (1.0 - alpha) * (double)cnt;
  return t1 + t2;
}

// pq = round_half_even(exp(logprob) * 2^30), clamped to [0, 2^30]; NaN -> 0.
int32_t prob_to_fixed(float lp, uint32_t* status) {
  if (std::isnan(lp)) { if (status) *status |= ST_BAD_LOGPROB; return 0; }
  if (lp >= 0.0f) return (int32_t)ONE_Q30;
  long double y = expl((long double)lp) * (long double)ONE_Q30;
  long double r = rintl(y);   // default rounding mode: to nearest, ties to even
  if (r < 0) r = 0;
  if (r > (long double)ONE_Q30) r = (long double)ONE_Q30;
  return (int32_t)r;
}

uint32_t append_impl(Ctx* c, const int32_t* tokens, const float* logprobs, const int32_t* pqs,
                     const int32_t* counts, int a_max) {
  uint32_t st = 0;
  int P = c->G * c->N;
  for (int p = 0; p < P; ++p) {
    int n = counts[p];
    if (n < 0) { st |= ST_BAD_COUNT; n = 0; }
    if (n > a_max) { st |= ST_BAD_COUNT; n = a_max; }
    int room = c->L - (int)c->tok[p].size();
    if (n > room) { st |= ST_CAPACITY; n = room; }
    for (int a = 0; a < n; ++a) {
      int32_t t = tokens[(size_t)p * a_max + a];
      if (t < 0 || t >= c->V) { st |= ST_BAD_TOKEN; break; }   // path keeps what came before
      int32_t q = pqs ? pqs[(size_t)p * a_max + a]
                      : prob_to_fixed(logprobs[(size_t)p * a_max + a], &st);
      c->tok[p].push_back(t);
      c->pq[p].push_back(q);
    }
  }
  return st;
}

// Textbook Levenshtein distance (unit costs) between a[0..na) and b[0..nb).
int edit_distance(const int32_t* a, int na, const int32_t* b, int nb) {
  std::vector<std::vector<int>> dp(na + 1, std::vector<int>(nb + 1, 0));
  for (int x = 0; x <= na; ++x) dp[x][0] = x;
  for (int y = 0; y <= nb; ++y) dp[0][y] = y;
  for (int x = 1; x <= na; ++x)
    for (int y = 1; y <= nb; ++y)
      dp[x][y] = std::min({dp[x - 1][y] + 1, dp[x][y - 1] + 1, dp[x - 1][y - 1] + (a[x - 1] != b[y - 1] ? 1 : 0)});
  return dp[na][nb];
}

// Eq. 4: does some window s' of path y that ends at e satisfy delta(q, s') <= eps?  Windows within eps of
// the query's length are the only ones that can; the empty window is not a match.
bool fuzzy_end(const std::vector<int32_t>& y, int e, const int32_t* q, int k, int eps) {
  for (int n = std::max(1, k - eps); n <= k + eps; ++n) {
    if (e - n + 1 < 0) continue;
    if (edit_distance(q, k, y.data() + (e - n + 1), n) <= eps) return true;
  }
  return false;
}

void build_path(Ctx* c, int k, int i) {
  PathResult& r = c->res[i];
  r = PathResult();
  r.nodes.resize(c->D);
  r.edges.resize(c->D);
  const std::vector<int32_t>& yi = c->tok[i];
  int len_i = (int)yi.size();
  if (k < 1 || len_i < k || len_i >= c->L) return;    // no query: too short, or path is full
  r.valid = true;
  r.root = yi[len_i - 1];
  int g = i / c->N;
  // Eq. 3: every other path j of the prompt, every end position e with a follower.
  for (int j = g * c->N; j < (g + 1) * c->N; ++j) {
    if (j == i) continue;
    const std::vector<int32_t>& yj = c->tok[j];
    int len_j = (int)yj.size();
    const size_t first_of_j = r.matches.size();
    if (c->eps > 0) {                              // "Fuzzy Suffix Matching": each end position counts once
      for (int e = 0; e <= len_j - 2; ++e)
        if (fuzzy_end(yj, e, yi.data() + (len_i - k), k, c->eps)) r.matches.push_back({j, e});
    } else {
      for (int e = k - 1; e <= len_j - 2; ++e) {
        bool same = true;
        for (int t = 0; t < k; ++t)
          if (yj[e - k + 1 + t] != yi[len_i - k + t]) { same = false; break; }
        if (same) r.matches.push_back({j, e});
      }
    }
    // Optional cap (Eq. 3 itself has none; the paper's experiments stress that its candidate set is small and
    // its limitations name the cost of aggregating over many paths): of the matches of query path i in source
    // path j only the R with the largest end position e, i.e. the most recent ones, stay in the pool.
    if (c->max_matches > 0 && r.matches.size() - first_of_j > (size_t)c->max_matches)
      r.matches.erase(r.matches.begin() + first_of_j, r.matches.end() - c->max_matches);   // found in ascending e
  }
  // Layered DAG: one instance per (candidate, layer).
  for (const auto& m : r.matches) {
    int j = m.first, e = m.second;
    int len_j = (int)c->tok[j].size();
    int n_m = std::min(c->D, len_j - 1 - e);
    for (int d = 1; d <= n_m; ++d) {
      int u = c->tok[j][e + d - 1];
      int v = c->tok[j][e + d];
      int64_t p = c->pq[j][e + d];
      Acc& ed = r.edges[d - 1][{u, v}];
      ed.S += p; ed.cnt += 1;
      Acc& nd = r.nodes[d - 1][v];
      nd.S += p; nd.cnt += 1;
    }
  }
  if (c->pool == 1) {
    // Tree pool (ablation study): candidates merge only while their whole prefix is the same, so a
    // node is a prefix.  Walk: among the candidates that spell the draft so far, group by next token,
    // weigh each child by Eq. 5 over its own instances, take the heaviest (ties: smaller token).
    std::vector<std::pair<int, int>> live(r.matches);
    for (int d = 1; d <= c->D; ++d) {
      std::map<int, Acc> child;
      for (const auto& m : live) {
        int j = m.first, e = m.second;
        if (e + d > (int)c->tok[j].size() - 1) continue;
        Acc& a = child[c->tok[j][e + d]];
        a.S += c->pq[j][e + d]; a.cnt += 1;
      }
      bool found = false; int best_v = -1; double best_w = 0.0;
      for (const auto& kv : child) {
        double w = weight(c->alpha, kv.second.S, kv.second.cnt);
        if (!found || w > best_w) { found = true; best_v = kv.first; best_w = w; }
      }
      if (!found) break;
      r.draft.push_back(best_v); r.score.push_back(best_w); r.edge_w.push_back(best_w);
      std::vector<std::pair<int, int>> next;
      for (const auto& m : live)
        if (m.second + d <= (int)c->tok[m.first].size() - 1 && c->tok[m.first][m.second + d] == best_v) next.push_back(m);
      live.swap(next);
    }
    return;
  }
  if (c->pool == 2) {
    // List pool (ablation study): no merging at all.  The draft is the candidate whose own tokens
    // weigh most by Eq. 5 (S = sum of its probabilities, Freq = its length); ties go to the
    // candidate that comes first in (path, position) order.
    bool found = false; double best_w = 0.0; std::pair<int, int> best;
    for (const auto& m : r.matches) {
      int j = m.first, e = m.second;
      int n_m = std::min(c->D, (int)c->tok[j].size() - 1 - e);
      int64_t S = 0;
      for (int d = 1; d <= n_m; ++d) S += c->pq[j][e + d];
      double w = weight(c->alpha, S, n_m);
      if (!found || w > best_w) { found = true; best_w = w; best = m; }
    }
    if (!found) return;
    int j = best.first, e = best.second;
    int n_m = std::min(c->D, (int)c->tok[j].size() - 1 - e);
    for (int d = 1; d <= n_m; ++d) {
      double w = weight(c->alpha, c->pq[j][e + d], 1);
      r.draft.push_back(c->tok[j][e + d]); r.score.push_back(w); r.edge_w.push_back(w);
    }
    return;
  }
  if (c->mode == 2) {
    // Best path instead of the greedy walk (the introduction asks for the highest-likelihood
    // sequence of the pool; the greedy rule of "Consensus-Driven Draft Extraction" only looks one
    // layer ahead).  Value of a path = sum of its nodes' in-weights (the greedy rule's own score),
    // added from the path's end towards its start:  best(d, v) = w(d, v) + max over successors v'
    // of best(d+1, v'), and 0 for the max of nothing.  Weights are >= 0, so a path is never cut
    // short of a leaf.  The walk takes, among the successors of the node it stands on, the one with
    // the highest best(); ties go to the smaller token.
    const bool virtual_root = c->eps > 0;
    std::vector<std::map<int, double>> best(c->D);
    for (int d = c->D; d >= 1; --d) {
      for (const auto& kv : r.nodes[d - 1]) {
        double succ = 0.0;
        if (d < c->D)
          for (const auto& e : r.edges[d])          // edges between layer d and layer d + 1
            if (e.first.first == kv.first) succ = std::max(succ, best[d].at(e.first.second));
        best[d - 1][kv.first] = weight(c->alpha, kv.second.S, kv.second.cnt) + succ;
      }
    }
    int cur = r.root;
    for (int d = 1; d <= c->D; ++d) {
      bool found = false; int best_v = -1; double best_b = 0.0;
      for (const auto& kv : r.nodes[d - 1]) {       // ascending token id
        const bool succ = (d == 1 && virtual_root) || r.edges[d - 1].count({cur, kv.first});
        if (!succ) continue;
        const double b = best[d - 1].at(kv.first);
        if (!found || b > best_b) { found = true; best_v = kv.first; best_b = b; }
      }
      if (!found) break;
      const Acc& nd = r.nodes[d - 1].at(best_v);
      r.draft.push_back(best_v);
      r.score.push_back(weight(c->alpha, nd.S, nd.cnt));
      if (d == 1 && virtual_root) r.edge_w.push_back(r.score.back());
      else { const Acc& ed = r.edges[d - 1].at({cur, best_v}); r.edge_w.push_back(weight(c->alpha, ed.S, ed.cnt)); }
      cur = best_v;
    }
    return;
  }
  // Greedy extraction.
  int cur = r.root;
  for (int d = 1; d <= c->D; ++d) {
    bool found = false; int best_v = -1; double best_w = 0.0; double best_e = 0.0;
    for (const auto& kv : r.nodes[d - 1]) {       // ascending token id
      int v = kv.first;
      auto it = r.edges[d - 1].find({cur, v});
      bool succ = it != r.edges[d - 1].end();
      // fuzzy matches may end in different tokens: the walk then starts from a virtual root that
      // precedes all of them, so every first-layer node is a successor and the edge taken carries
      // everything that enters the node
      const bool from_virtual_root = d == 1 && c->eps > 0;
      if (c->mode == 0 && !succ && !from_virtual_root) continue;
      double w = weight(c->alpha, kv.second.S, kv.second.cnt);
      if (!found || w > best_w) {                 // strict: ties keep the smaller token
        found = true; best_v = v; best_w = w;
        best_e = from_virtual_root ? w : (succ ? weight(c->alpha, it->second.S, it->second.cnt) : 0.0);
      }
    }
    if (!found) break;
    r.draft.push_back(best_v);
    r.score.push_back(best_w);
    r.edge_w.push_back(best_e);
    cur = best_v;
  }
}

struct NodeRow { int tok; int64_t S, cnt; double w; };

// The B best paths of the pool instead of the single best one (several drafts per query path, e.g. for
// tree verification; the paper's method extracts one sequence, its introduction asks for the
// highest-likelihood one).  Same value as search mode 2: a path is worth the sum of its nodes'
// Eq. 5 in-weights, added from its end towards its start, and only paths that run on to a leaf (or to
// layer D) count.  Every node keeps its B best continuations:
//   leaf (d, v):      [ w(d, v) ]
//   otherwise:        the B best of { w(d, v) + x : x a kept continuation of a successor v' },
// ordered by value (larger first), then by v' (smaller first), then by the rank of x in the list of
// v'.  As long as no two different sums round to the same double (never with alpha = 1: all sums
// are exact) this is the order "value, then token sequence read as a word", and the result is the B
// best root-to-leaf paths of the DAG.
struct Cont { double value; int next; int rank; };
void build_beams(Ctx* c, int i, int B) {
  PathResult& r = c->res[i];
  r.beam_tok.clear(); r.beam_value.clear();
  if (!r.valid || r.matches.empty() || B < 1) return;
  auto better = [](const Cont& a, const Cont& b) {
    if (a.value != b.value) return a.value > b.value;
    if (a.next != b.next) return a.next < b.next;
    return a.rank < b.rank;
  };
  std::vector<std::map<int, std::vector<Cont>>> keep(c->D);
  for (int d = c->D; d >= 1; --d) {
    for (const auto& kv : r.nodes[d - 1]) {
      const double w = weight(c->alpha, kv.second.S, kv.second.cnt);
      std::vector<Cont> cand;
      if (d < c->D)
        for (const auto& e : r.edges[d])            // edges between layer d and layer d + 1
          if (e.first.first == kv.first) {
            const std::vector<Cont>& of = keep[d].at(e.first.second);
            for (size_t x = 0; x < of.size(); ++x) cand.push_back({w + of[x].value, e.first.second, (int)x});
          }
      if (cand.empty()) cand.push_back({w, -1, 0});
      std::sort(cand.begin(), cand.end(), better);
      if ((int)cand.size() > B) cand.resize(B);
      keep[d - 1][kv.first] = cand;
    }
  }
  std::vector<Cont> top;
  for (const auto& kv : r.nodes[0]) {
    if (!(c->eps > 0) && !r.edges[0].count({r.root, kv.first})) continue;   // always true with exact matching
    const std::vector<Cont>& of = keep[0].at(kv.first);
    for (size_t x = 0; x < of.size(); ++x) top.push_back({of[x].value, kv.first, (int)x});
  }
  std::sort(top.begin(), top.end(), better);
  if ((int)top.size() > B) top.resize(B);
  for (const Cont& t : top) {
    std::vector<int> seq;
    int v = t.next, rank = t.rank;
    for (int d = 1; d <= c->D && v >= 0; ++d) {
      seq.push_back(v);
      const Cont& e = keep[d - 1].at(v)[rank];
      v = e.next; rank = e.rank;
    }
    r.beam_tok.push_back(seq);
    r.beam_value.push_back(t.value);
  }
}

}  // namespace

extern "C" {

void* orc_create(int G, int N, int L, int V, int D, float alpha, int mode) {
  Ctx* c = new Ctx();
  c->G = G; c->N = N; c->L = L; c->V = V; c->D = D; c->mode = mode;
  c->alpha = (double)alpha;
  c->tok.resize((size_t)G * N); c->pq.resize((size_t)G * N); c->res.resize((size_t)G * N);
  return c;
}

void orc_destroy(void* h) { delete (Ctx*)h; }

// Edit-distance tolerance of the suffix match (Eq. 4); 0 = exact matching.
void orc_set_epsilon(void* h, int eps) { ((Ctx*)h)->eps = eps; }

// Cap R on the matches kept per (query path, source path): the R most recent ones; 0 = no cap (Eq. 3 as printed).
void orc_set_max_matches(void* h, int R) { ((Ctx*)h)->max_matches = R; }

// Draft pool structure of the paper's ablation: 0 = DAG (the method), 1 = tree, 2 = list.
void orc_set_pool(void* h, int pool) { ((Ctx*)h)->pool = pool; }

int orc_edit_distance(const int32_t* a, int na, const int32_t* b, int nb) { return edit_distance(a, na, b, nb); }

int32_t orc_prob_to_fixed(float lp) { return prob_to_fixed(lp, nullptr); }

double orc_weight(float alpha, int64_t S, int64_t cnt) { return weight((double)alpha, S, cnt); }

uint32_t orc_append(void* h, const int32_t* tokens, const float* logprobs, const int32_t* counts, int a_max) {
  return append_impl((Ctx*)h, tokens, logprobs, nullptr, counts, a_max);
}

// Same as orc_append but with the fixed-point probabilities given directly
// (used by the hand-worked examples, whose probabilities are dyadic).
uint32_t orc_append_fixed(void* h, const int32_t* tokens, const int32_t* pq, const int32_t* counts, int a_max) {
  return append_impl((Ctx*)h, tokens, nullptr, pq, counts, a_max);
}

// Sliding window over the histories (not in the paper, whose runs end before any limit): path p
// forgets all but its newest keep[p] tokens; keep[p] >= its length changes nothing, keep[p] < 0 is
// reported as a bad count and changes nothing.  What a later build sees is exactly the shorter
// history, as if only those tokens had ever been appended.
uint32_t orc_trim(void* h, const int32_t* keep) {
  Ctx* c = (Ctx*)h;
  uint32_t st = 0;
  for (size_t p = 0; p < c->tok.size(); ++p) {
    if (keep[p] < 0) { st |= ST_BAD_COUNT; continue; }
    const size_t len = c->tok[p].size();
    if ((size_t)keep[p] >= len) continue;
    c->tok[p].erase(c->tok[p].begin(), c->tok[p].begin() + (len - keep[p]));
    c->pq[p].erase(c->pq[p].begin(), c->pq[p].begin() + (len - keep[p]));
  }
  return st;
}

void orc_get_lengths(void* h, int32_t* out) {
  Ctx* c = (Ctx*)h;
  for (size_t p = 0; p < c->tok.size(); ++p) out[p] = (int32_t)c->tok[p].size();
}

void orc_get_history(void* h, int p, int32_t* tok, int32_t* pq) {
  Ctx* c = (Ctx*)h;
  std::memcpy(tok, c->tok[p].data(), c->tok[p].size() * 4);
  std::memcpy(pq, c->pq[p].data(), c->pq[p].size() * 4);
}

void orc_build_path(void* h, int k, int i) { build_path((Ctx*)h, k, i); }

// All paths; nthreads > 1 fans the (independent) query paths out over threads.
void orc_build_all(void* h, int k, int nthreads) {
  Ctx* c = (Ctx*)h;
  int P = c->G * c->N;
  if (nthreads <= 1) { for (int i = 0; i < P; ++i) build_path(c, k, i); return; }
  std::vector<std::thread> th;
  for (int t = 0; t < nthreads; ++t)
    th.emplace_back([=]() { for (int i = t; i < P; i += nthreads) build_path(c, k, i); });
  for (auto& x : th) x.join();
}

// Beams of query path i from the pool of its last build (DAG pool): at most B drafts, best first.
// tok is [B][D] (unused -1), len [B], value [B]; returns the number of beams found.
int orc_build_beams(void* h, int i, int B, int32_t* tok, int32_t* len, double* value) {
  Ctx* c = (Ctx*)h;
  build_beams(c, i, B);
  const PathResult& r = c->res[i];
  for (int b = 0; b < B; ++b) {
    len[b] = 0; value[b] = 0.0;
    for (int d = 0; d < c->D; ++d) tok[(size_t)b * c->D + d] = -1;
  }
  for (size_t b = 0; b < r.beam_tok.size(); ++b) {
    len[b] = (int32_t)r.beam_tok[b].size(); value[b] = r.beam_value[b];
    for (size_t d = 0; d < r.beam_tok[b].size(); ++d) tok[b * c->D + d] = r.beam_tok[b][d];
  }
  return (int)r.beam_tok.size();
}

int orc_num_matches(void* h, int i) { return (int)((Ctx*)h)->res[i].matches.size(); }

// Global positions j*L + e, ascending.
void orc_get_matches(void* h, int i, int32_t* gpos) {
  Ctx* c = (Ctx*)h;
  size_t n = 0;
  for (const auto& m : c->res[i].matches) gpos[n++] = m.first * c->L + m.second;
}

void orc_layer_counts(void* h, int i, int d, int32_t* n_nodes, int32_t* n_edges) {
  const PathResult& r = ((Ctx*)h)->res[i];
  *n_nodes = (int32_t)r.nodes[d - 1].size();
  *n_edges = (int32_t)r.edges[d - 1].size();
}

void orc_get_nodes(void* h, int i, int d, int32_t* tok, int64_t* S, int64_t* cnt) {
  size_t n = 0;
  for (const auto& kv : ((Ctx*)h)->res[i].nodes[d - 1]) { tok[n] = kv.first; S[n] = kv.second.S; cnt[n] = kv.second.cnt; ++n; }
}

void orc_get_edges(void* h, int i, int d, int32_t* u, int32_t* v, int64_t* S, int64_t* cnt) {
  size_t n = 0;
  for (const auto& kv : ((Ctx*)h)->res[i].edges[d - 1]) {
    u[n] = kv.first.first; v[n] = kv.first.second; S[n] = kv.second.S; cnt[n] = kv.second.cnt; ++n;
  }
}

int orc_get_draft(void* h, int i, int32_t* tok, double* score, double* edge_w) {
  const PathResult& r = ((Ctx*)h)->res[i];
  for (size_t d = 0; d < r.draft.size(); ++d) { tok[d] = r.draft[d]; score[d] = r.score[d]; edge_w[d] = r.edge_w[d]; }
  return (int)r.draft.size();
}

// Drafts of all paths in the library's output layout: tok [P][D] (unused = -1),
// len [P], score / edge_w [P][D] as float (unused = 0).
void orc_get_drafts(void* h, int32_t* tok, int32_t* len, float* score, float* edge_w) {
  Ctx* c = (Ctx*)h;
  int P = c->G * c->N;
  for (int i = 0; i < P; ++i) {
    const PathResult& r = c->res[i];
    len[i] = (int32_t)r.draft.size();
    for (int d = 0; d < c->D; ++d) {
      bool on = d < (int)r.draft.size();
      tok[(size_t)i * c->D + d] = on ? r.draft[d] : -1;
      score[(size_t)i * c->D + d] = on ? (float)r.score[d] : 0.0f;
      edge_w[(size_t)i * c->D + d] = on ? (float)r.edge_w[d] : 0.0f;
    }
  }
}

// Truncated view of the DAG of path i: per layer the B best nodes by
// (weight desc, token asc); per kept node of layer d its Ke best out-edges to
// layer d+1 by (weight desc, destination token asc).  Unused slots: token -1.
// node_* are [D][B], node_count [D], edge_* are [D][B][Ke], out_degree [D][B].
void orc_get_export(void* h, int i, int B, int Ke,
                    int32_t* node_tok, int64_t* node_S, int32_t* node_cnt, int32_t* node_count,
                    int32_t* edge_dst, int64_t* edge_S, int32_t* edge_cnt, int32_t* out_degree) {
  Ctx* c = (Ctx*)h;
  const PathResult& r = c->res[i];
  int D = c->D;
  for (int x = 0; x < D * B; ++x) { node_tok[x] = -1; node_S[x] = 0; node_cnt[x] = 0; out_degree[x] = 0; }
  for (int x = 0; x < D * B * Ke; ++x) { edge_dst[x] = -1; edge_S[x] = 0; edge_cnt[x] = 0; }
  for (int d = 1; d <= D; ++d) {
    node_count[d - 1] = (int32_t)r.nodes[d - 1].size();
    std::vector<NodeRow> rows;
    for (const auto& kv : r.nodes[d - 1])
      rows.push_back({kv.first, kv.second.S, kv.second.cnt, weight(c->alpha, kv.second.S, kv.second.cnt)});
    std::stable_sort(rows.begin(), rows.end(), [](const NodeRow& a, const NodeRow& b) {
      return a.w > b.w || (a.w == b.w && a.tok < b.tok); });
    for (int b = 0; b < B && b < (int)rows.size(); ++b) {
      size_t nx = (size_t)(d - 1) * B + b;
      node_tok[nx] = rows[b].tok; node_S[nx] = rows[b].S; node_cnt[nx] = (int32_t)rows[b].cnt;
      if (d == D) continue;
      std::vector<NodeRow> out;
      for (const auto& kv : r.edges[d])              // edges between layers d and d+1
        if (kv.first.first == rows[b].tok)
          out.push_back({kv.first.second, kv.second.S, kv.second.cnt, weight(c->alpha, kv.second.S, kv.second.cnt)});
      out_degree[nx] = (int32_t)out.size();
      std::stable_sort(out.begin(), out.end(), [](const NodeRow& a, const NodeRow& b) {
        return a.w > b.w || (a.w == b.w && a.tok < b.tok); });
      for (int e = 0; e < Ke && e < (int)out.size(); ++e) {
        size_t ex = nx * Ke + e;
        edge_dst[ex] = out[e].tok; edge_S[ex] = out[e].S; edge_cnt[ex] = (int32_t)out[e].cnt;
      }
    }
  }
}

// "Draft acceptance": tau_p = longest t <= draft_len[p] with draft[0..t) == sampled[0..t).
void orc_accept(void* h, const int32_t* draft_tok, const int32_t* draft_len, const int32_t* sampled,
                int32_t* accept_len) {
  Ctx* c = (Ctx*)h;
  int P = c->G * c->N, D = c->D;
  for (int p = 0; p < P; ++p) {
    int t = 0;
    while (t < draft_len[p] && t < D && draft_tok[(size_t)p * D + t] == sampled[(size_t)p * (D + 1) + t]) ++t;
    accept_len[p] = t;
  }
}

// Acceptance followed by the state update: path p appends sampled[p][0 .. tau_p]
// (the accepted tokens plus the model's own next token), at most max_append
// tokens, cut at capacity (no status for that cut) and before a token outside [0, V).
uint32_t orc_accept_commit(void* h, const int32_t* draft_tok, const int32_t* draft_len, const int32_t* sampled,
                           const float* sampled_logprobs, int max_append, int32_t* accept_len) {
  Ctx* c = (Ctx*)h;
  int P = c->G * c->N, D = c->D;
  orc_accept(h, draft_tok, draft_len, sampled, accept_len);
  std::vector<int32_t> counts(P);
  for (int p = 0; p < P; ++p) {
    int n = std::min(accept_len[p] + 1, max_append);
    n = std::min(n, c->L - (int)c->tok[p].size());
    counts[p] = n;
  }
  return append_impl(c, sampled, sampled_logprobs, nullptr, counts.data(), D + 1);
}

}  // extern "C"
