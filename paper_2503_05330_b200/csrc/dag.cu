// Follower gather, layered DAG aggregation (Eq. 5) and greedy extraction, plus
// the single-launch build for small prompts.
//
// Every match m of query path i contributes, at layer d = 1..D, its d-th
// follower v = tok[e+d] with the fixed-point probability pq[e+d].  A node is a
// distinct token of a layer, an edge a distinct (previous token, token) pair; S
// and cnt of nodes and edges are integer sums, so the order of accumulation
// (atomics, warp shuffles) cannot change a result.
//
// Two ways through, both per query path in one CTA:
//   dag_small (M <= 32 matches, the common case): lane m owns candidate m and
//     each WARP owns a layer, so all layers aggregate at the same time.  Lanes
//     with the same follower token (__match_any_sync) form a node, lanes that
//     also share the previous token form an edge; sums run over the lanes of a
//     group, ranks over the group leaders, and each layer also decides the best
//     way out of every source node.  One barrier, then one warp walks the layers
//     by looking those decisions up.
//   dag_block (any M): layers in sequence.  Followers are staged in shared memory
//     when they fit; every candidate adds into a shared-memory hash table keyed
//     by token (32-bit atomics with explicit carry).  Unstaged fan-out past the
//     first layer runs in two phases - claim a slot for every successor of the
//     current node, then add only the candidates that land on a claimed slot -
//     so the table holds the successors of one node instead of a whole layer.
//     One warp then picks the best successor.  A layer with more distinct tokens
//     than the table holds is processed in several passes, each over the tokens
//     of one residue class, so any fan-out fits the same tables.
//   The EXPORT instantiation (sdms_get_dag) also keeps an edge table and lets
//   other warps rank the B best nodes of the layer and the Ke best out-edges of
//   the nodes kept one layer up.  tree / list pools reuse the same passes with a
//   prefix filter / a single arg-max over candidates.
#include "sdms_internal.h"
#include "append_dev.cuh"
#include "wide_dev.cuh"

namespace sdms {

namespace {

typedef unsigned long long u64;
constexpr unsigned FULL = 0xffffffffu;
constexpr int CAP = kDagCap;
constexpr int MAXB = SDMS_MAX_DAG_NODES;
constexpr int MAXKE = SDMS_MAX_DAG_EDGES;
constexpr int kRollMax = 2 * 8192 / 3;   // candidates whose followers are staged layer by layer (three arrays in the staging area)
constexpr int kStageWords = 8192;      // followers (token, pq) of all matches staged in shared memory when M*D fits
constexpr int kLoadBatch = 4;          // candidates a thread loads before it touches the tables
constexpr int kListCap = 2048;         // matches a fused CTA keeps in shared memory besides its global slice
static_assert(kStageWords >= 4 * 32 * SDMS_MAX_DRAFT, "dag_small keeps its per-layer lanes in the staging area");

// Loads of path state (tokens, probabilities, lengths, records, index buckets).  In the one-launch
// step other CTAs write this state earlier in the same launch, so it is read with ordinary loads,
// which a cluster-scope acquire keeps coherent, never through the read-only (non-coherent) path.
template <class T>
__device__ __forceinline__ T ldm(const T* p) { return *p; }

struct Cand {            // a node or an edge competing in a selection
  double w; u64 S; unsigned cnt; int tok; int valid;
};

// Lane holding the first candidate in rank order (largest weight, then smallest
// token) among the lanes with valid set, or -1.  Weights are non-negative, so
// their bit patterns order like the values: three full-warp reductions settle it.
__device__ __forceinline__ int warp_arg_first(bool valid, double w, int tok) {
  const u64 bits = (u64)__double_as_longlong(w);
  const unsigned hi = (unsigned)(bits >> 32), lo = (unsigned)bits;
  if (__ballot_sync(FULL, valid) == 0) return -1;
  const unsigned mh = __reduce_max_sync(FULL, valid ? hi : 0u);
  const bool c1 = valid && hi == mh;
  const unsigned ml = __reduce_max_sync(FULL, c1 ? lo : 0u);
  const bool c2 = c1 && lo == ml;
  const unsigned mt = __reduce_min_sync(FULL, c2 ? (unsigned)tok : 0xffffffffu);
  return __ffs(__ballot_sync(FULL, c2 && (unsigned)tok == mt)) - 1;
}

__device__ __forceinline__ Cand warp_best(Cand c) {
  const int src = warp_arg_first(c.valid != 0, c.w, c.tok);
  const int from = src < 0 ? 0 : src;
  Cand r;
  r.valid = src >= 0;
  r.w = __shfl_sync(FULL, c.w, from);
  r.S = __shfl_sync(FULL, c.S, from);
  r.cnt = __shfl_sync(FULL, c.cnt, from);
  r.tok = __shfl_sync(FULL, c.tok, from);
  return r;
}

// The K first candidates in rank order among get(0..ncand-1); lane 0 stores them.
// Tokens are distinct among valid candidates, so "strictly after the previous
// pick" enumerates them one by one.  Returns how many were found.
template <class Get>
__device__ int warp_topk(int ncand, Get get, int K, int* out_tok, u64* out_S, unsigned* out_cnt) {
  const int lane = threadIdx.x & 31;
  double prev_w = 0.0; int prev_tok = 0;
  int r = 0;
  for (; r < K; ++r) {
    Cand best; best.valid = 0; best.w = 0.0; best.S = 0; best.cnt = 0; best.tok = 0;
    for (int x = lane; x < ncand; x += 32) {
      const Cand c = get(x);
      if (!c.valid) continue;
      if (r > 0 && !ranks_before(prev_w, prev_tok, c.w, c.tok)) continue;
      if (!best.valid || ranks_before(c.w, c.tok, best.w, best.tok)) best = c;
    }
    best = warp_best(best);
    if (!best.valid) break;
    if (lane == 0) { out_tok[r] = best.tok; out_S[r] = best.S; out_cnt[r] = best.cnt; }
    prev_w = best.w; prev_tok = best.tok;
  }
  __syncwarp();
  return r;
}

// Sums of val over the lanes of group a and of group b; `live` (warp-uniform)
// lists the lanes worth visiting.
__device__ __forceinline__ void group_sums(unsigned live, unsigned a, unsigned b, unsigned val, u64* sa, u64* sb) {
  u64 x = 0, y = 0;
  for (unsigned rem = live; rem; rem &= rem - 1) {
    const int src = __ffs(rem) - 1;
    const unsigned t = __shfl_sync(FULL, val, src);
    if (a >> src & 1) x += t;
    if (b >> src & 1) y += t;
  }
  *sa = x; *sb = y;
}

// 64-bit add on a (lo, hi) pair of shared words with 32-bit atomics: whoever
// makes the low word wrap carries into the high word.
__device__ __forceinline__ void add64(unsigned* lo, unsigned* hi, u64 v) {
  const unsigned l = (unsigned)v;
  unsigned h = (unsigned)(v >> 32);
  const unsigned old = atomicAdd(lo, l);
  if (old + l < old) ++h;
  if (h) atomicAdd(hi, h);
}
__device__ __forceinline__ u64 get64(const unsigned* lo, const unsigned* hi, int x) {
  return ((u64)hi[x] << 32) | lo[x];
}

struct Smem {
  // node table: key = token; sums over all candidates and over those coming from the current node
  int* n_key; unsigned* n_Slo; unsigned* n_Shi; unsigned* n_Clo; unsigned* n_Chi; unsigned* n_call; unsigned* n_ccur;
  int* n_touch;
  // edge table (export): key = token * MAXB + slot of the kept source node
  int* e_key; unsigned* e_Slo; unsigned* e_Shi; unsigned* e_c; int* e_touch;
  // export lists
  u64* r_node_S; int* r_node_tok; unsigned* r_node_cnt;
  u64* r_edge_S; int* r_edge_dst; unsigned* r_edge_cnt;
  u64* t_S; int* t_tok; unsigned* t_cnt;        // per-warp scratch for merging
  int* kept; int* r_nedge; int* r_outdeg;
  int* st_tok; int* st_pq;                      // staged followers [m*D + d-1], token -1 = past the path's end
  int* list;                                    // fused kernel: first kListCap matches
};

constexpr int kMaxWarps = 32;

template <bool EXPORT>
__host__ __device__ constexpr size_t dag_smem_bytes() {
  size_t b = (size_t)CAP * 8 * 4 + (size_t)kStageWords * 8 + (size_t)kListCap * 4;
  if (EXPORT) {
    b += (size_t)CAP * 5 * 4;
    b += (size_t)MAXB * 16 + (size_t)MAXB * MAXKE * 16 + (size_t)kMaxWarps * 32 * 16 + (size_t)MAXB * 12;
  }
  return b;
}

template <bool EXPORT>
__device__ Smem carve(unsigned char* base) {
  Smem m;
  u64* p8 = reinterpret_cast<u64*>(base);
  if (EXPORT) {
    m.r_node_S = p8; p8 += MAXB;
    m.r_edge_S = p8; p8 += MAXB * MAXKE;
    m.t_S = p8; p8 += kMaxWarps * 32;
  }
  int* p4 = reinterpret_cast<int*>(p8);
  m.st_tok = p4; p4 += kStageWords;
  m.st_pq = p4; p4 += kStageWords;
  m.n_key = p4; p4 += CAP;
  m.n_Slo = reinterpret_cast<unsigned*>(p4); p4 += CAP;
  m.n_Shi = reinterpret_cast<unsigned*>(p4); p4 += CAP;
  m.n_Clo = reinterpret_cast<unsigned*>(p4); p4 += CAP;
  m.n_Chi = reinterpret_cast<unsigned*>(p4); p4 += CAP;
  m.n_call = reinterpret_cast<unsigned*>(p4); p4 += CAP;
  m.n_ccur = reinterpret_cast<unsigned*>(p4); p4 += CAP;
  m.n_touch = p4; p4 += CAP;
  m.list = p4; p4 += kListCap;
  if (EXPORT) {
    m.e_key = p4; p4 += CAP;
    m.e_Slo = reinterpret_cast<unsigned*>(p4); p4 += CAP;
    m.e_Shi = reinterpret_cast<unsigned*>(p4); p4 += CAP;
    m.e_c = reinterpret_cast<unsigned*>(p4); p4 += CAP;
    m.e_touch = p4; p4 += CAP;
    m.r_node_tok = p4; p4 += MAXB;
    m.r_node_cnt = reinterpret_cast<unsigned*>(p4); p4 += MAXB;
    m.r_edge_dst = p4; p4 += MAXB * MAXKE;
    m.r_edge_cnt = reinterpret_cast<unsigned*>(p4); p4 += MAXB * MAXKE;
    m.t_tok = p4; p4 += kMaxWarps * 32;
    m.t_cnt = reinterpret_cast<unsigned*>(p4); p4 += kMaxWarps * 32;
    m.kept = p4; p4 += MAXB;
    m.r_nedge = p4; p4 += MAXB;
    m.r_outdeg = p4; p4 += MAXB;
  }
  return m;
}

// 16-bit tag of a token, never 0 (0 marks "no token")
__device__ __forceinline__ unsigned short tag_of(int tok) { return (unsigned short)(0x8000u | (((unsigned)tok * 2654435761u) >> 17)); }
__device__ __forceinline__ unsigned slot_hash(unsigned x) { return (x * 2654435761u) >> 22; }   // 10 bits = CAP
static_assert(CAP == 1024, "slot_hash yields 10 bits");

// Defaults of one query path: no draft, empty export.
template <bool EXPORT>
__device__ void write_defaults(const Dev& s, int i, int32_t* draft_tok, float* draft_score, float* draft_edge_w) {
  const int tid = threadIdx.x, D = s.D, B = s.B, Ke = s.Ke;
  for (int d = tid; d < D; d += blockDim.x) {
    draft_tok[(size_t)i * D + d] = -1;
    if (draft_score) draft_score[(size_t)i * D + d] = 0.0f;
    if (draft_edge_w) draft_edge_w[(size_t)i * D + d] = 0.0f;
  }
  if (EXPORT) {
    for (int x = tid; x < D * B; x += blockDim.x) {
      const size_t nx = (size_t)i * D * B + x;
      s.x_node_tok[nx] = -1; s.x_node_S[nx] = 0; s.x_node_cnt[nx] = 0; s.x_out_degree[nx] = 0;
    }
    for (int x = tid; x < D * B * Ke; x += blockDim.x) {
      const size_t ex = (size_t)i * D * B * Ke + x;
      s.x_edge_dst[ex] = -1; s.x_edge_S[ex] = 0; s.x_edge_cnt[ex] = 0;
    }
    for (int d = tid; d < D; d += blockDim.x) s.x_node_count[(size_t)i * D + d] = 0;
  }
}

// ---------------------------------------------------------------------------
// M <= 32: one warp per layer, then one warp walks.  The export rows must hold
// their defaults already (write_defaults followed by a barrier).
// ---------------------------------------------------------------------------
template <bool EXPORT>
__device__ void dag_small(const Dev& s, const Smem& sm, int i, int M, const int32_t* mlist,
                          const int32_t* plen, int poff, int root, int32_t* __restrict__ draft_tok, int32_t* __restrict__ draft_len,
                          float* __restrict__ draft_score, float* __restrict__ draft_edge_w) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int D = s.D, B = s.B, Ke = s.Ke;
  // per layer and lane: follower token, previous token, node score, edge weight; per layer: leader masks
  int* L_v = sm.st_tok;
  int* L_u = sm.st_tok + 32 * SDMS_MAX_DRAFT;
  unsigned* L_lead = reinterpret_cast<unsigned*>(sm.st_tok + 2 * 32 * SDMS_MAX_DRAFT);
  unsigned* L_elead = L_lead + SDMS_MAX_DRAFT;
  unsigned* L_best = L_elead + SDMS_MAX_DRAFT;      // per layer: the best edge out of each source / the best node
  int* L_p = sm.st_tok + 3 * 32 * SDMS_MAX_DRAFT;   // fixed-point probability of the follower (tree pool)
  double* L_W = reinterpret_cast<double*>(sm.st_pq);
  double* L_we = L_W + 32 * SDMS_MAX_DRAFT;

  int gpos = 0, n_m = 0;
  if (lane < M) {
    gpos = mlist[lane];
    const int j = path_of(s, gpos);
    n_m = min(D, plen[j - poff] - 1 - (gpos - j * s.L));
  }
  for (int d = warp + 1; d <= D; d += nwarps) {
    const bool alive = d <= n_m;                        // candidate reaches layer d
    const bool alive_prev = lane < M && d - 1 <= n_m;   // ... reached layer d-1 (layer 0 is the root)
    const int v = alive ? ldm(s.tok + gpos + d) : -1;
    const unsigned p = alive ? (unsigned)ldm(s.pq + gpos + d) : 0u;
    const int u = !alive_prev ? -1 : (d == 1 ? root : ldm(s.tok + gpos + d - 1));
    const unsigned live = __ballot_sync(FULL, alive);
    const unsigned gv = __match_any_sync(FULL, v);                     // lanes on the same node
    const unsigned gu = __match_any_sync(FULL, u);                     // lanes with the same previous node
    const unsigned ge = gv & gu;                                       // lanes on the same edge
    u64 S_all, S_uv;
    group_sums(live, gv, ge, p, &S_all, &S_uv);
    const unsigned c_all = __popc(gv), c_uv = __popc(ge);
    const bool leader = alive && lane == __ffs(gv) - 1;
    const bool eleader = alive && lane == __ffs(ge) - 1;
    const double W = eq5_weight(s.alpha, S_all, c_all);
    const double w_uv = eq5_weight(s.alpha, S_uv, c_uv);
    const unsigned leaders = __ballot_sync(FULL, leader), eleaders = __ballot_sync(FULL, eleader);
    // is this edge the best way out of its source, judged by the score of its destination?
    bool beaten = false;
    for (unsigned rem = eleaders; rem; rem &= rem - 1) {
      const int src = __ffs(rem) - 1;
      const int ou = __shfl_sync(FULL, u, src);
      const int ot = __shfl_sync(FULL, v, src);
      const double oW = __shfl_sync(FULL, W, src);
      if (ou == u && ranks_before(oW, ot, W, v)) beaten = true;
    }
    const unsigned best_out = __ballot_sync(FULL, eleader && !beaten);
    const int top = s.mode == 1 ? warp_arg_first(leader, W, v) : -1;   // best node of the layer
    L_v[(d - 1) * 32 + lane] = v; L_u[(d - 1) * 32 + lane] = u; L_p[(d - 1) * 32 + lane] = (int)p;
    L_W[(d - 1) * 32 + lane] = W; L_we[(d - 1) * 32 + lane] = w_uv;
    if (lane == 0) {
      L_lead[d - 1] = leaders; L_elead[d - 1] = eleaders;
      L_best[d - 1] = s.mode == 1 ? (top >= 0 ? 1u << top : 0u) : best_out;
    }
    if (EXPORT && live) {
      int rank = 0;
      for (unsigned rem = leaders; rem; rem &= rem - 1) {
        const int src = __ffs(rem) - 1;
        const double ow = __shfl_sync(FULL, W, src);
        const int ot = __shfl_sync(FULL, v, src);
        if (ranks_before(ow, ot, W, v)) ++rank;
      }
      if (leader && rank < B) {
        const size_t nx = ((size_t)i * D + (d - 1)) * B + rank;
        s.x_node_tok[nx] = v; s.x_node_S[nx] = (int64_t)S_all; s.x_node_cnt[nx] = (int32_t)c_all;
      }
      if (lane == 0) s.x_node_count[(size_t)i * D + (d - 1)] = __popc(leaders);
      if (d > 1) {
        // rank of each previous-layer node, recomputed here so that layers stay independent
        const unsigned pu = alive_prev ? (unsigned)ldm(s.pq + gpos + d - 1) : 0u;
        const unsigned live_prev = __ballot_sync(FULL, alive_prev);
        u64 S_u, unused;
        group_sums(live_prev, gu, 0u, pu, &S_u, &unused);
        const double W_u = eq5_weight(s.alpha, S_u, __popc(gu));
        const bool uleader = alive_prev && lane == __ffs(gu) - 1;
        const unsigned uleaders = __ballot_sync(FULL, uleader);
        int urank = 0;
        for (unsigned rem = uleaders; rem; rem &= rem - 1) {
          const int src = __ffs(rem) - 1;
          const double ow = __shfl_sync(FULL, W_u, src);
          const int ot = __shfl_sync(FULL, u, src);
          if (ranks_before(ow, ot, W_u, u)) ++urank;
        }
        const int slot_u = __shfl_sync(FULL, urank, __ffs(gu) - 1);     // export slot of this lane's source node
        int erank = 0, deg = 0;
        for (unsigned rem = eleaders; rem; rem &= rem - 1) {
          const int src = __ffs(rem) - 1;
          const double ow = __shfl_sync(FULL, w_uv, src);
          const int ot = __shfl_sync(FULL, v, src);
          const int ou = __shfl_sync(FULL, u, src);
          if (ou == u) { ++deg; if (ranks_before(ow, ot, w_uv, v)) ++erank; }
        }
        if (eleader && slot_u < B) {
          const size_t nb = ((size_t)i * D + (d - 2)) * B + slot_u;
          if (erank < Ke) {
            s.x_edge_dst[nb * Ke + erank] = v; s.x_edge_S[nb * Ke + erank] = (int64_t)S_uv;
            s.x_edge_cnt[nb * Ke + erank] = (int32_t)c_uv;
          }
          if (erank == 0) s.x_out_degree[nb] = deg;
        }
      }
    }
  }
  __syncthreads();
  if (warp != 0) return;
  if (!EXPORT && s.pool == 1) {
    // tree pool: only the candidates that spell the draft so far stay in play
    bool in_play = lane < M;
    int emitted = 0;
    for (int d = 1; d <= D; ++d) {
      const int v = L_v[(d - 1) * 32 + lane];
      const bool on = in_play && v >= 0;
      const unsigned live = __ballot_sync(FULL, on);
      if (live == 0) break;
      const unsigned gv = __match_any_sync(FULL, on ? v : -1);
      u64 S, unused;
      group_sums(live, gv, 0u, (unsigned)L_p[(d - 1) * 32 + lane], &S, &unused);
      const double W = eq5_weight(s.alpha, S, __popc(gv));
      const int src = warp_arg_first(on && lane == __ffs(gv) - 1, W, v);
      const int tok = __shfl_sync(FULL, v, src);
      const double Wb = __shfl_sync(FULL, W, src);
      if (lane == 0) {
        draft_tok[(size_t)i * D + (d - 1)] = tok;
        if (draft_score) draft_score[(size_t)i * D + (d - 1)] = (float)Wb;
        if (draft_edge_w) draft_edge_w[(size_t)i * D + (d - 1)] = (float)Wb;
      }
      in_play = on && v == tok;
      ++emitted;
    }
    if (lane == 0) draft_len[i] = emitted;
    return;
  }
  int cur = root, emitted = 0;
  for (int d = 1; d <= D; ++d) {
    const int v = L_v[(d - 1) * 32 + lane], u = L_u[(d - 1) * 32 + lane];
    const unsigned from_cur = __ballot_sync(FULL, u == cur);
    const unsigned pick = s.mode == 1 ? L_best[d - 1] : (L_best[d - 1] & from_cur);
    if (pick == 0) break;
    const int src = __ffs(pick) - 1;
    const int tok = __shfl_sync(FULL, v, src);
    const double W = __shfl_sync(FULL, L_W[(d - 1) * 32 + lane], src);
    // the edge taken: in mode 0 the picked lane leads it; in mode 1 it may not exist
    const unsigned emask = L_elead[d - 1] & from_cur & __ballot_sync(FULL, v == tok);
    const double we = __shfl_sync(FULL, L_we[(d - 1) * 32 + lane], emask ? __ffs(emask) - 1 : 0);
    if (lane == 0) {
      draft_tok[(size_t)i * D + (d - 1)] = tok;
      if (draft_score) draft_score[(size_t)i * D + (d - 1)] = (float)W;
      if (draft_edge_w) draft_edge_w[(size_t)i * D + (d - 1)] = emask ? (float)we : 0.0f;
    }
    cur = tok;
    ++emitted;
  }
  if (lane == 0) draft_len[i] = emitted;
}

// ---------------------------------------------------------------------------
// any M: layers in sequence, shared-memory hash tables
// ---------------------------------------------------------------------------
template <bool EXPORT>
__device__ void dag_block(const Dev& s, const Smem& sm, int i, int M, const int32_t* mlist,
                          const int32_t* plen, int poff, int root, int32_t* __restrict__ draft_tok, int32_t* __restrict__ draft_len,
                          float* __restrict__ draft_score, float* __restrict__ draft_edge_w) {
  __shared__ int sh_nn, sh_ne, sh_overflow, sh_found, sh_cur, sh_nkept, sh_nnode_run, sh_node_total;
  __shared__ int sh_draft[SDMS_MAX_DRAFT];
  __shared__ double sh_best_w, sh_best_ew;
  __shared__ int sh_best_tok, sh_best_valid;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int D = s.D, B = s.B, Ke = s.Ke;

  // stage every follower once: one round trip to memory instead of one per layer
  const bool staged = M * D <= kStageWords;
  if (staged) {
    for (int x = tid; x < M * D; x += blockDim.x) {
      const int m = x / D, dd = x - m * D + 1;
      const int gpos = mlist[m];
      const int j = path_of(s, gpos);
      const int e = gpos - j * s.L;
      const bool on = e + dd <= plen[j - poff] - 1;
      sm.st_tok[x] = on ? ldm(s.tok + gpos + dd) : -1;
      sm.st_pq[x] = on ? ldm(s.pq + gpos + dd) : 0;
    }
  }
  // too many followers to stage them all: stage one layer at a time (token and probability of every
  // candidate; the layer before stays, it holds the edges' sources), so that the passes and phases of
  // a layer read shared memory and only one sweep per layer goes to L2
  const bool rolling = !staged && M <= kRollMax && !(!EXPORT && s.pool == 1);
  // more candidates than that: the staging area is free and keeps a 16-bit tag of every candidate's token
  // of the layer before (written by the last sweep of that layer), so that the sweep that claims the
  // successors of the current node (phase 0 below) reads shared memory and goes to the histories only
  // for the candidates whose tag is the current node's
  const bool tagged = !EXPORT && !staged && !rolling && s.pool == 0 && M <= 4 * kStageWords;
  unsigned short* const tag = reinterpret_cast<unsigned short*>(sm.st_tok);
  int* const roll_odd = sm.st_tok;
  int* const roll_even = sm.st_tok + kRollMax;
  int* const roll_p = sm.st_tok + 2 * kRollMax;
  for (int x = tid; x < CAP; x += blockDim.x) {
    sm.n_key[x] = -1; sm.n_Slo[x] = 0; sm.n_Shi[x] = 0; sm.n_Clo[x] = 0; sm.n_Chi[x] = 0;
    sm.n_call[x] = 0; sm.n_ccur[x] = 0;
    if (EXPORT) { sm.e_key[x] = -1; sm.e_Slo[x] = 0; sm.e_Shi[x] = 0; sm.e_c[x] = 0; }
  }
  if (tid == 0) { sh_nn = 0; sh_ne = 0; sh_overflow = 0; sh_cur = root; sh_nkept = 0; }
  __syncthreads();

  const int npart_max = (int)(((long long)s.V * (EXPORT ? max(1, B) : 1) + CAP / 2 - 1) / (CAP / 2));
  int npart = 1;
  int emitted = 0;
  bool walking = true;

  for (int d = 1; d <= D; ++d) {
    if (!walking && !EXPORT) break;
    const int cur = sh_cur;
    const int nkept = EXPORT ? sh_nkept : 0;
    const bool tree = !EXPORT && s.pool == 1;       // only candidates that spell the draft so far take part
    const bool restricted = !EXPORT && !staged && !tree && s.mode != 1 && d > 1;   // staged candidates are cheap to revisit
    if (!EXPORT) {
      // first layer (or every layer in mode 1): every distinct follower is a node.  The guess is
      // optimistic, one node per 32 candidates (popular n-grams have far fewer distinct followers than
      // occurrences): a sweep that finds the table three quarters full stops at once and the layer is
      // redone with twice the residue classes, so a wrong guess costs a fraction of a sweep, while a
      // cautious one costs a full sweep for every class too many.  Restricted layers only hold the
      // successors of one node.
      npart = 1;
      if (!restricted) while (npart * (CAP / 2) * 32 < M && npart < npart_max) npart *= 2;
    }
    const unsigned short cur_tag = tag_of(cur);
    int* const cur_v = (d & 1) ? roll_odd : roll_even;
    const int* const prev_v = (d & 1) ? roll_even : roll_odd;
    if (rolling) {
      constexpr int kRollBatch = 8;
      for (int m0 = tid; m0 < M; m0 += kRollBatch * blockDim.x) {
        int tv[kRollBatch], tp[kRollBatch];
#pragma unroll
        for (int r = 0; r < kRollBatch; ++r) {
          const int m = m0 + r * blockDim.x;
          tv[r] = -1; tp[r] = 0;
          if (m >= M) continue;
          const int gpos = mlist[m];
          const int j = path_of(s, gpos);
          if (gpos - j * s.L + d <= plen[j - poff] - 1) { tv[r] = ldm(s.tok + gpos + d); tp[r] = ldm(s.pq + gpos + d); }
        }
#pragma unroll
        for (int r = 0; r < kRollBatch; ++r) {
          const int m = m0 + r * blockDim.x;
          if (m < M) { cur_v[m] = tv[r]; roll_p[m] = tp[r]; }
        }
      }
    }
    bool layer_done = false;
    // the tags describe the layer before only until the last residue class of a pass has overwritten them with
    // this layer's: a pass that is given up after that point and done again must not filter by them
    bool tags_fresh = true;
    while (!layer_done) {
      if (tid == 0) { sh_best_valid = 0; sh_nnode_run = 0; sh_node_total = 0; }
      if (EXPORT && tid < MAXB) { sm.r_nedge[tid] = 0; sm.r_outdeg[tid] = 0; }
      __syncthreads();
      bool overflowed = false;
      // while the layer can still be split further, a claim that does not find its slot within 64 probes gives the
      // pass up (it is redone): a first batch of 2048 claims can fill the table before any thread looks at the count
      const int probe_max = npart < npart_max ? 64 : CAP;
      const bool part_pow2 = (npart & (npart - 1)) == 0;        // nearly always: residue and quotient without a division
      const int part_shift = __ffs(npart) - 1;
      for (int part = 0; part < npart && !overflowed; ++part) {
        // ---- accumulate this residue class of follower tokens ----
        // Walking in mode 0 past the first layer, only successors of the current node can be chosen:
        // phase 0 claims a slot for each of them, phase 1 adds every candidate that lands on a claimed
        // slot.  Otherwise one phase claims and adds.
        for (int phase = restricted ? 0 : 1; phase < 2; ++phase) {
          for (int m0 = tid; m0 < M; m0 += kLoadBatch * blockDim.x) {
            if (npart < npart_max && *(volatile int*)&sh_nn > CAP * 3 / 4) break;   // too many nodes for this pass: it is redone
            int v[kLoadBatch], u[kLoadBatch];
            unsigned p[kLoadBatch];
#pragma unroll
            for (int r = 0; r < kLoadBatch; ++r) {                    // loads of the whole batch go out together
              const int m = m0 + r * blockDim.x;
              v[r] = -1; u[r] = -1; p[r] = 0;
              if (m >= M) continue;
              if (staged) {
                v[r] = sm.st_tok[m * D + d - 1];
                if (v[r] >= 0) { u[r] = d == 1 ? root : sm.st_tok[m * D + d - 2]; p[r] = (unsigned)sm.st_pq[m * D + d - 1]; }
                if (tree) for (int x = 1; x < d && v[r] >= 0; ++x) if (sm.st_tok[m * D + x - 1] != sh_draft[x - 1]) v[r] = -1;
              } else if (rolling) {
                v[r] = cur_v[m];
                if (v[r] >= 0) { u[r] = d == 1 ? root : prev_v[m]; p[r] = (unsigned)roll_p[m]; }
              } else {
                if (tagged && phase == 0 && tags_fresh && tag[m] != cur_tag) continue;   // its token of the layer before is not the current node
                const int gpos = mlist[m];
                const int j = path_of(s, gpos);
                if (gpos - j * s.L + d <= plen[j - poff] - 1) {
                  v[r] = ldm(s.tok + gpos + d);
                  u[r] = d == 1 ? root : ldm(s.tok + gpos + d - 1);
                  p[r] = (unsigned)ldm(s.pq + gpos + d);
                  if (tree) for (int x = 1; x < d && v[r] >= 0; ++x) if (ldm(s.tok + gpos + x) != sh_draft[x - 1]) v[r] = -1;
                }
                if (tagged && phase == 1 && part == npart - 1) tag[m] = v[r] >= 0 ? tag_of(v[r]) : (unsigned short)0;
              }
            }
#pragma unroll
            for (int r = 0; r < kLoadBatch; ++r) {
              const int vv = v[r], uu = u[r];
              const unsigned pp = p[r];
              if (vv < 0 || (npart > 1 && (part_pow2 ? (vv & (npart - 1)) : vv % npart) != part)) continue;
              if (phase == 0 && uu != cur) continue;
              const unsigned vq = part_pow2 ? (unsigned)vv >> part_shift : (unsigned)(vv / npart);
              unsigned h = slot_hash(vq);
              int slot = -1;
              if (phase == 1 && restricted) {                          // read-only: is vv a claimed successor?
                for (int probe = 0; probe < CAP; ++probe) {
                  const int key = sm.n_key[h];
                  if (key == vv) { slot = (int)h; break; }
                  if (key == -1) break;
                  h = (h + 1) & (CAP - 1);
                }
                if (slot < 0) continue;
              } else {
                for (int probe = 0; probe < probe_max; ++probe) {
                  const int old = atomicCAS(&sm.n_key[h], -1, vv);
                  if (old == -1) sm.n_touch[atomicAdd(&sh_nn, 1)] = (int)h;
                  if (old == -1 || old == vv) { slot = (int)h; break; }
                  h = (h + 1) & (CAP - 1);
                }
                if (slot < 0) { sh_overflow = 1; continue; }
                if (phase == 0) continue;
              }
              add64(&sm.n_Slo[slot], &sm.n_Shi[slot], pp);
              atomicAdd(&sm.n_call[slot], 1u);
              if (uu == cur) { add64(&sm.n_Clo[slot], &sm.n_Chi[slot], pp); atomicAdd(&sm.n_ccur[slot], 1u); }
              if (EXPORT && d > 1) {
                int b = -1;
                for (int x = 0; x < nkept; ++x) if (sm.kept[x] == uu) { b = x; break; }
                if (b >= 0) {
                  const int ekey = vv * MAXB + b;               // (destination, kept source) in one word
                  unsigned he = slot_hash(vq * 37u + (unsigned)b);
                  int es = -1;
                  for (int probe = 0; probe < CAP; ++probe) {
                    const int old = atomicCAS(&sm.e_key[he], -1, ekey);
                    if (old == -1) sm.e_touch[atomicAdd(&sh_ne, 1)] = (int)he;
                    if (old == -1 || old == ekey) { es = (int)he; break; }
                    he = (he + 1) & (CAP - 1);
                  }
                  if (es < 0) { sh_overflow = 1; continue; }
                  add64(&sm.e_Slo[es], &sm.e_Shi[es], pp);
                  atomicAdd(&sm.e_c[es], 1u);
                }
              }
            }
          }
          if (phase == 0) __syncthreads();
        }
        __syncthreads();
        const int nn = sh_nn, ne = EXPORT ? sh_ne : 0;
        overflowed = sh_overflow || (npart < npart_max && (nn > CAP * 3 / 4 || ne > CAP * 3 / 4));
        if (!overflowed) {
          // ---- selections, one warp each ----
          if (warp == 0 && walking) {
            Cand best; best.valid = 0; best.w = 0; best.tok = 0; best.S = 0; best.cnt = 0;
            for (int x = lane; x < nn; x += 32) {
              const int sl = sm.n_touch[x];
              Cand c;
              c.tok = sm.n_key[sl]; c.S = 0;
              c.valid = s.mode == 1 || tree || sm.n_ccur[sl] > 0;
              c.w = eq5_weight(s.alpha, get64(sm.n_Slo, sm.n_Shi, sl), sm.n_call[sl]);
              c.cnt = (unsigned)sl;                  // carry the slot: the edge weight is read from it below
              if (c.valid && (!best.valid || ranks_before(c.w, c.tok, best.w, best.tok))) best = c;
            }
            best = warp_best(best);
            if (lane == 0 && best.valid &&
                (!sh_best_valid || ranks_before(best.w, best.tok, sh_best_w, sh_best_tok))) {
              const int sl = (int)best.cnt;
              sh_best_valid = 1; sh_best_w = best.w; sh_best_tok = best.tok;
              sh_best_ew = tree ? best.w
                         : sm.n_ccur[sl] ? eq5_weight(s.alpha, get64(sm.n_Clo, sm.n_Chi, sl), sm.n_ccur[sl]) : 0.0;
            }
          }
          if (EXPORT && warp == 1) {
            const int nrun = sh_nnode_run;
            auto get = [&](int x) {
              Cand c; c.valid = 1;
              if (x < nn) { const int sl = sm.n_touch[x]; c.tok = sm.n_key[sl]; c.S = get64(sm.n_Slo, sm.n_Shi, sl); c.cnt = sm.n_call[sl]; }
              else { c.tok = sm.r_node_tok[x - nn]; c.S = sm.r_node_S[x - nn]; c.cnt = sm.r_node_cnt[x - nn]; }
              c.w = eq5_weight(s.alpha, c.S, c.cnt);
              return c;
            };
            int* tt = sm.t_tok + warp * 32; u64* tS = sm.t_S + warp * 32; unsigned* tc = sm.t_cnt + warp * 32;
            const int got = warp_topk(nn + nrun, get, B, tt, tS, tc);
            for (int x = lane; x < got; x += 32) { sm.r_node_tok[x] = tt[x]; sm.r_node_S[x] = tS[x]; sm.r_node_cnt[x] = tc[x]; }
            if (lane == 0) { sh_nnode_run = got; sh_node_total += nn; }
          }
          if (EXPORT && warp >= 2 && d > 1) {
            for (int b = warp - 2; b < nkept; b += nwarps - 2) {
              const int nrun = sm.r_nedge[b];
              int deg = 0;
              for (int x = lane; x < ne; x += 32) deg += sm.e_key[sm.e_touch[x]] % MAXB == b;
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) deg += __shfl_xor_sync(FULL, deg, o);
              auto get = [&](int x) {
                Cand c;
                if (x < ne) {
                  const int sl = sm.e_touch[x];
                  c.valid = sm.e_key[sl] % MAXB == b; c.tok = sm.e_key[sl] / MAXB;
                  c.S = get64(sm.e_Slo, sm.e_Shi, sl); c.cnt = sm.e_c[sl];
                } else {
                  const int y = b * MAXKE + (x - ne);
                  c.valid = 1; c.tok = sm.r_edge_dst[y]; c.S = sm.r_edge_S[y]; c.cnt = sm.r_edge_cnt[y];
                }
                c.w = eq5_weight(s.alpha, c.S, c.cnt);
                return c;
              };
              int* tt = sm.t_tok + warp * 32; u64* tS = sm.t_S + warp * 32; unsigned* tc = sm.t_cnt + warp * 32;
              const int got = warp_topk(ne + nrun, get, Ke, tt, tS, tc);
              for (int x = lane; x < got; x += 32) {
                const int y = b * MAXKE + x;
                sm.r_edge_dst[y] = tt[x]; sm.r_edge_S[y] = tS[x]; sm.r_edge_cnt[y] = tc[x];
              }
              if (lane == 0) { sm.r_nedge[b] = got; sm.r_outdeg[b] += deg; }
              __syncwarp();
            }
          }
        }
        __syncthreads();
        // ---- wipe the touched slots for the next pass ----
        for (int x = tid; x < nn; x += blockDim.x) {
          const int sl = sm.n_touch[x];
          sm.n_key[sl] = -1; sm.n_Slo[sl] = 0; sm.n_Shi[sl] = 0; sm.n_Clo[sl] = 0; sm.n_Chi[sl] = 0;
          sm.n_call[sl] = 0; sm.n_ccur[sl] = 0;
        }
        if (EXPORT)
          for (int x = tid; x < ne; x += blockDim.x) {
            const int sl = sm.e_touch[x];
            sm.e_key[sl] = -1; sm.e_Slo[sl] = 0; sm.e_Shi[sl] = 0; sm.e_c[sl] = 0;
          }
        __syncthreads();
        if (tid == 0) { sh_nn = 0; sh_ne = 0; sh_overflow = 0; }
        __syncthreads();
      }
      if (overflowed && npart < npart_max) {
        npart = min(npart * 2, npart_max);          // redo the layer with smaller residue classes
        tags_fresh = false;
      } else {
        layer_done = true;
      }
    }
    // ---- close the layer ----
    if (tid == 0) {
      sh_found = 0;
      if (walking && sh_best_valid) {
        sh_found = 1;
        draft_tok[(size_t)i * D + (d - 1)] = sh_best_tok;
        sh_draft[d - 1] = sh_best_tok;
        if (draft_score) draft_score[(size_t)i * D + (d - 1)] = (float)sh_best_w;
        if (draft_edge_w) draft_edge_w[(size_t)i * D + (d - 1)] = (float)sh_best_ew;
        sh_cur = sh_best_tok;
      }
    }
    if (EXPORT) {
      const int nrun = sh_nnode_run;
      if (d > 1)
        for (int x = tid; x < nkept * Ke; x += blockDim.x) {
          const int b = x / Ke, r = x % Ke;
          if (r < sm.r_nedge[b]) {
            const size_t ex = (((size_t)i * D + (d - 2)) * B + b) * Ke + r;
            const int y = b * MAXKE + r;
            s.x_edge_dst[ex] = sm.r_edge_dst[y]; s.x_edge_S[ex] = (int64_t)sm.r_edge_S[y];
            s.x_edge_cnt[ex] = (int32_t)sm.r_edge_cnt[y];
          }
          if (r == 0) s.x_out_degree[((size_t)i * D + (d - 2)) * B + b] = sm.r_outdeg[b];
        }
      __syncthreads();
      for (int x = tid; x < nrun; x += blockDim.x) {
        const size_t nx = ((size_t)i * D + (d - 1)) * B + x;
        s.x_node_tok[nx] = sm.r_node_tok[x]; s.x_node_S[nx] = (int64_t)sm.r_node_S[x];
        s.x_node_cnt[nx] = (int32_t)sm.r_node_cnt[x];
        sm.kept[x] = sm.r_node_tok[x];
      }
      if (tid == 0) { s.x_node_count[(size_t)i * D + (d - 1)] = sh_node_total; sh_nkept = nrun; }
    }
    __syncthreads();
    if (walking) {
      if (sh_found) ++emitted; else walking = false;
    }
    // expected growth of the next layer decides where its pass count starts
    if (EXPORT) {
      const int tot = sh_node_total;
      int next = 1;
      while (next * (CAP / 2) < 2 * tot && next < npart_max) next *= 2;
      npart = min(next, npart_max);
      if (tot == 0) { break; }                      // no candidate reaches this depth: nor any deeper one
    }
    __syncthreads();
  }
  if (tid == 0) draft_len[i] = emitted;
}

// List pool (ablation): no merging; the draft is the single candidate that weighs most by Eq. 5 on
// its own tokens (S = sum of its probabilities, Freq = its length), ties to the smaller position.
__device__ void list_pool(const Dev& s, int i, int M, const int32_t* mlist, const int32_t* plen, int poff,
                          int32_t* __restrict__ draft_tok, int32_t* __restrict__ draft_len,
                          float* __restrict__ draft_score, float* __restrict__ draft_edge_w) {
  __shared__ double sh_w[kMaxWarps];
  __shared__ int sh_g[kMaxWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int D = s.D;
  double best_w = 0.0;
  int best_g = -1;
  for (int m = tid; m < M; m += blockDim.x) {
    const int gpos = mlist[m];
    const int j = path_of(s, gpos);
    const int n_m = min(D, plen[j - poff] - 1 - (gpos - j * s.L));
    u64 S = 0;
    for (int d = 1; d <= n_m; ++d) S += (unsigned)ldm(s.pq + gpos + d);
    const double w = eq5_weight(s.alpha, S, (unsigned)n_m);
    if (best_g < 0 || ranks_before(w, gpos, best_w, best_g)) { best_w = w; best_g = gpos; }
  }
  int src = warp_arg_first(best_g >= 0, best_w, best_g);
  if (src < 0) src = 0;
  best_w = __shfl_sync(FULL, best_w, src); best_g = __shfl_sync(FULL, best_g, src);
  if (lane == 0) { sh_w[warp] = best_w; sh_g[warp] = best_g; }
  __syncthreads();
  if (warp != 0) return;
  best_w = lane < nwarps ? sh_w[lane] : 0.0; best_g = lane < nwarps ? sh_g[lane] : -1;
  src = warp_arg_first(best_g >= 0, best_w, best_g);
  best_g = __shfl_sync(FULL, best_g, src < 0 ? 0 : src);
  const int j = best_g / s.L;
  const int n_m = min(D, plen[j - poff] - 1 - (best_g - j * s.L));
  if (lane < n_m) {
    const float w = (float)eq5_weight(s.alpha, (unsigned)ldm(s.pq + best_g + 1 + lane), 1u);
    draft_tok[(size_t)i * D + lane] = ldm(s.tok + best_g + 1 + lane);
    if (draft_score) draft_score[(size_t)i * D + lane] = w;
    if (draft_edge_w) draft_edge_w[(size_t)i * D + lane] = w;
  }
  if (lane == 0) draft_len[i] = n_m;
}

// ---- all layers at once (DAG pool, no export, a few hundred matches) ------------------------------
// dag_block takes the layers one after the other because the walk decides which node's successors
// count; each layer then costs a few barriers and a chain of shared-memory atomics whatever M is.
// Here every layer is aggregated at the same time into tables of its own:
//   node table of layer d : follower token v -> sum of probabilities, count          (Eq. 5 inputs)
//   pred table of layer d : token u of layer d - 1 -> its best successor v at layer d
// and the walk is D table look-ups.  The pool of shared words (staging area and dag_block's tables,
// kPoolWords in a row) holds the staged followers and as many layers' tables as fit; more layers
// take more rounds.
constexpr int kPoolWords = 2 * kStageWords + 8 * CAP;
constexpr int kLayerWords = 8;                    // per table slot: pred weight (2), node key/Slo/Shi/cnt, pred key/token

struct LayerTables {
  unsigned* p_whi; unsigned* p_wlo; int* n_key; unsigned* n_Slo; unsigned* n_Shi; unsigned* n_cnt; int* p_key; int* p_tok;
};
__device__ __forceinline__ LayerTables layer_tables(int* pool, int cap, int l) {
  int* b = pool + (size_t)l * kLayerWords * cap;
  LayerTables t;
  t.p_whi = reinterpret_cast<unsigned*>(b); t.p_wlo = reinterpret_cast<unsigned*>(b + cap);
  t.n_key = b + 2 * cap; t.n_Slo = reinterpret_cast<unsigned*>(b + 3 * cap); t.n_Shi = reinterpret_cast<unsigned*>(b + 4 * cap);
  t.n_cnt = reinterpret_cast<unsigned*>(b + 5 * cap); t.p_key = b + 6 * cap; t.p_tok = b + 7 * cap;
  return t;
}
// slot of `key` in an open-addressing table of `cap` (power of two) slots; claims one if INSERT
template <bool INSERT>
__device__ __forceinline__ int table_slot(int* keys, int cap, int shift, int key) {
  unsigned h = ((unsigned)key * 2654435761u) >> shift;
#pragma unroll 1
  for (int probe = 0; probe < cap; ++probe) {
    const int old = INSERT ? atomicCAS(&keys[h], -1, key) : keys[h];
    if (old == key || (INSERT && old == -1)) return (int)h;
    if (!INSERT && old == -1) return -1;
    h = (h + 1) & (cap - 1);
  }
  return -1;
}
// Sums of 30-bit probabilities are kept as two 32-bit sums, of the low 16 bits and of the rest: each
// stays below 2^32 for any number of candidates a CTA handles, and an add needs no result back (no
// carry to pass on), so the adds do not stall their thread.
__device__ __forceinline__ void add_split(unsigned* lo16, unsigned* hi, unsigned* cnt, unsigned pq) {
  atomicAdd(lo16, pq & 0xffffu);
  atomicAdd(hi, pq >> 16);
  atomicAdd(cnt, 1u);
}
__device__ __forceinline__ u64 weight_bits(double alpha, const unsigned* lo16, const unsigned* hi, const unsigned* cnt, int x) {
  return (u64)__double_as_longlong(eq5_weight(alpha, ((u64)hi[x] << 16) + lo16[x], cnt[x]));
}

// How many layers' tables fit beside the staged followers (0: use dag_block).  Three words are staged
// per follower: token, probability, and the table slots found for it (so that no pass probes twice).
__device__ __forceinline__ int layers_per_round(int M, int D, int* cap_out) {
  const int staged = (3 * M * D + 1) & ~1;
  int cap = 64;                                    // more slots than keys: a probe always ends at a free slot
  while (cap <= M) cap *= 2;
  // twice the slots shorten the probe sequences (a warp waits for its longest); taken when all
  // layers still fit in one round
  if ((kPoolWords - staged) / (kLayerWords * 2 * cap) >= D) cap *= 2;
  *cap_out = cap;
  return (kPoolWords - staged) / (kLayerWords * cap);
}

__device__ __forceinline__ bool layers_in_round_ok(int M, int D) {
  int cap;
  return layers_per_round(M, D, &cap) >= min(D, 2);
}

__device__ void dag_layers(const Dev& s, const Smem& sm, int i, int M, const int32_t* mlist, const int32_t* plen,
                           int poff, int root, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                           float* draft_edge_w) {
  __shared__ int sh_draft[SDMS_MAX_DRAFT];
  __shared__ unsigned sh_lwhi[SDMS_MAX_DRAFT], sh_lwlo[SDMS_MAX_DRAFT];   // mode 1: heaviest node of the layer
  __shared__ int sh_lt[SDMS_MAX_DRAFT];
  __shared__ unsigned sh_eSlo[SDMS_MAX_DRAFT], sh_eShi[SDMS_MAX_DRAFT], sh_ec[SDMS_MAX_DRAFT];
  __shared__ int sh_cur, sh_emitted, sh_walking;
  const int tid = threadIdx.x, D = s.D;
  int cap;
  const int per_round = min(D, layers_per_round(M, D, &cap));
  const int lcap = 31 - __clz(cap), shift = 32 - lcap;
  int* st_tok = sm.st_tok;                         // [m * D + d - 1], -1 past the end of the path
  int* st_pq = sm.st_tok + M * D;
  int* st_slot = sm.st_tok + 2 * M * D;            // node slot | pred slot << 16 of each staged follower
  int* pool = sm.st_tok + ((3 * M * D + 1) & ~1);
  const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int nchunk = (M + 31) >> 5;                // a warp takes 32 matches of one layer at a time

  if (tid < D) { sh_lwhi[tid] = 0; sh_lwlo[tid] = 0; sh_lt[tid] = INT_MAX; sh_eSlo[tid] = 0; sh_eShi[tid] = 0; sh_ec[tid] = 0; }
  if (tid == 0) { sh_cur = root; sh_emitted = 0; sh_walking = 1; }
  // stage the followers: a thread asks for four entries before it stores the first
  {
    int lD = 0;
    while ((1 << lD) < D) ++lD;                    // entries are numbered m << lD | d - 1: no division
    constexpr int kBatch = 4;
#pragma unroll 1
    for (int x0 = tid; x0 < (M << lD); x0 += kBatch * blockDim.x) {
      int tk[kBatch], pr[kBatch];
#pragma unroll
      for (int r = 0; r < kBatch; ++r) {
        const int x = x0 + r * blockDim.x;
        const int m = x >> lD, dd = (x & ((1 << lD) - 1)) + 1;
        tk[r] = -1; pr[r] = 0;
        if (m >= M || dd > D) continue;
        const int gpos = mlist[m];
        const int j = path_of(s, gpos);
        if (gpos - j * s.L + dd <= plen[j - poff] - 1) { tk[r] = ldm(s.tok + gpos + dd); pr[r] = ldm(s.pq + gpos + dd); }
      }
#pragma unroll
      for (int r = 0; r < kBatch; ++r) {
        const int x = x0 + r * blockDim.x;
        const int m = x >> lD, dd = (x & ((1 << lD) - 1)) + 1;
        if (m < M && dd <= D) { st_tok[m * D + dd - 1] = tk[r]; st_pq[m * D + dd - 1] = pr[r]; }
      }
    }
  }

#pragma unroll 1
  for (int d0 = 1; d0 <= D; d0 += per_round) {
    const int nl = min(per_round, D - d0 + 1);
    // empty tables: keys -1, sums 0, best weight 0, best token "none"
#pragma unroll 1
    for (int x = tid; x < ((nl * kLayerWords) << lcap); x += blockDim.x) {
      const int w = (x >> lcap) & (kLayerWords - 1);
      pool[x] = (w == 2 || w == 6) ? -1 : (w == 7 ? INT_MAX : 0);
    }
    __syncthreads();
    if (!sh_walking) break;
    // pass 0: node sums; passes 1, 2: heaviest successor weight of every predecessor, the upper half of
    // the weight's bit pattern first, then the lower half among those (weights are >= 0, so the
    // patterns order like the values); pass 3: the smallest token that has this weight
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
#pragma unroll 1
      for (int task = warp; task < nl * nchunk; task += nwarps) {
        const int l = task / nchunk, m = ((task - l * nchunk) << 5) + lane;
        const int d = d0 + l, at = m * D + d - 1;
        const int v = m < M ? st_tok[at] : -1;
        if (v < 0) continue;
        const LayerTables t = layer_tables(pool, cap, l);
        if (pass == 0) {
          const int sl = table_slot<true>(t.n_key, cap, shift, v);
          st_slot[at] = sl;
          add_split(&t.n_Slo[sl], &t.n_Shi[sl], &t.n_cnt[sl], (unsigned)st_pq[at]);
          continue;
        }
        const u64 w = weight_bits(s.alpha, t.n_Slo, t.n_Shi, t.n_cnt, st_slot[at] & 0xffff);
        const unsigned whi = (unsigned)(w >> 32), wlo = (unsigned)w;
        if (pass == 1) {
          const int claimed = table_slot<true>(t.p_key, cap, shift, d == 1 ? root : st_tok[at - 1]);
          st_slot[at] |= claimed << 16;
          atomicMax(&t.p_whi[claimed], whi);
          if (s.mode == 1) atomicMax(&sh_lwhi[d - 1], whi);
          continue;
        }
        const int ps = (unsigned)st_slot[at] >> 16;
        if (pass == 2) {
          if (t.p_whi[ps] == whi) atomicMax(&t.p_wlo[ps], wlo);
          if (s.mode == 1 && sh_lwhi[d - 1] == whi) atomicMax(&sh_lwlo[d - 1], wlo);
        } else {
          if (t.p_whi[ps] == whi && t.p_wlo[ps] == wlo) atomicMin(&t.p_tok[ps], v);
          if (s.mode == 1 && sh_lwhi[d - 1] == whi && sh_lwlo[d - 1] == wlo) atomicMin(&sh_lt[d - 1], v);
        }
      }
      __syncthreads();
    }
    // the walk through this round's layers
    if (tid == 0) {
      int cur = sh_cur, emitted = sh_emitted;
#pragma unroll 1
      for (int l = 0; l < nl; ++l) {
        const int d = d0 + l;
        const LayerTables t = layer_tables(pool, cap, l);
        int next;
        u64 w;
        if (s.mode == 1) {
          next = sh_lt[d - 1]; w = ((u64)sh_lwhi[d - 1] << 32) | sh_lwlo[d - 1];
          if (next == INT_MAX) { sh_walking = 0; break; }
        } else {
          const int ps = table_slot<false>(t.p_key, cap, shift, cur);
          if (ps < 0) { sh_walking = 0; break; }
          next = t.p_tok[ps]; w = ((u64)t.p_whi[ps] << 32) | t.p_wlo[ps];
        }
        draft_tok[(size_t)i * D + d - 1] = next;
        if (draft_score) draft_score[(size_t)i * D + d - 1] = (float)__longlong_as_double((long long)w);
        sh_draft[d - 1] = next;
        cur = next; ++emitted;
      }
      sh_cur = cur; sh_emitted = emitted;
    }
    __syncthreads();
  }
  // weight of the edges the draft took (Eq. 5 over the candidates that contain the edge)
  const int emitted = sh_emitted;
#pragma unroll 1
  for (int task = warp; task < emitted * nchunk; task += nwarps) {
    const int l = task / nchunk, m = ((task - l * nchunk) << 5) + lane;
    const int d = l + 1, at = m * D + d - 1;
    if (m < M && st_tok[at] == sh_draft[d - 1] && (d == 1 || st_tok[at - 1] == sh_draft[d - 2]))
      add_split(&sh_eSlo[d - 1], &sh_eShi[d - 1], &sh_ec[d - 1], (unsigned)st_pq[at]);
  }
  __syncthreads();
  if (tid < emitted && draft_edge_w)
    draft_edge_w[(size_t)i * D + tid] =
        sh_ec[tid] ? (float)__longlong_as_double((long long)weight_bits(s.alpha, sh_eSlo, sh_eShi, sh_ec, tid)) : 0.0f;
  if (tid == 0) draft_len[i] = emitted;
}

// ---- best path instead of the greedy walk (search mode 2) ------------------------------------------
// best(d, v) = w(d, v) + max over the successors v' of v of best(d + 1, v')  (0 for no successor), w the
// node's Eq. 5 in-weight; the draft follows, from the root, the successor with the largest best(), ties
// to the smaller token.  All D layers' node tables stay in shared memory at once; the layers are
// taken from the last to the first for best(), then every node's choice of successor is made for
// all layers together, and the walk is D look-ups.
constexpr int kPathWords = 9;     // per slot: best (2), largest successor best (2), key, sum lo16 / hi, count, chosen successor

struct PathTables {
  u64* best; u64* succ; int* key; unsigned* Slo; unsigned* Shi; unsigned* cnt; int* next;
};
__device__ __forceinline__ PathTables path_tables(int* pool, int cap, int l) {
  int* b = pool + (size_t)l * kPathWords * cap;
  PathTables t;
  t.best = reinterpret_cast<u64*>(b); t.succ = reinterpret_cast<u64*>(b + 2 * cap);
  t.key = b + 4 * cap; t.Slo = reinterpret_cast<unsigned*>(b + 5 * cap); t.Shi = reinterpret_cast<unsigned*>(b + 6 * cap);
  t.cnt = reinterpret_cast<unsigned*>(b + 7 * cap); t.next = b + 8 * cap;
  return t;
}
// Do the tables of all D layers fit beside the staged followers?
__device__ __forceinline__ bool best_path_fits(int M, int D, int* cap_out) {
  int cap = 64;
  while (cap <= M) cap *= 2;
  *cap_out = cap;
  return (long long)((2 * M * D + 1) & ~1) + (long long)D * kPathWords * cap <= kPoolWords;
}

__device__ void dag_best_path(const Dev& s, const Smem& sm, int i, int M, int cap, const int32_t* mlist,
                              const int32_t* plen, int poff, int32_t* draft_tok, int32_t* draft_len,
                              float* draft_score, float* draft_edge_w) {
  __shared__ int sh_draft[SDMS_MAX_DRAFT];
  __shared__ unsigned sh_eSlo[SDMS_MAX_DRAFT], sh_eShi[SDMS_MAX_DRAFT], sh_ec[SDMS_MAX_DRAFT];
  __shared__ u64 sh_root_succ;
  __shared__ int sh_root_next, sh_emitted;
  const int tid = threadIdx.x, D = s.D;
  const int lcap = 31 - __clz(cap), shift = 32 - lcap;
  int* st_tok = sm.st_tok;                         // [m * D + d - 1], -1 past the end of the path
  int* st_pq = sm.st_tok + M * D;
  int* pool = sm.st_tok + ((2 * M * D + 1) & ~1);
  int lD = 0;
  while ((1 << lD) < D) ++lD;                      // items are numbered m << lD | d - 1

  for (int x = tid; x < (M << lD); x += blockDim.x) {
    const int m = x >> lD, dd = (x & ((1 << lD) - 1)) + 1;
    if (dd > D) continue;
    const int gpos = mlist[m];
    const int j = path_of(s, gpos);
    const bool on = gpos - j * s.L + dd <= plen[j - poff] - 1;
    st_tok[m * D + dd - 1] = on ? ldm(s.tok + gpos + dd) : -1;
    st_pq[m * D + dd - 1] = on ? ldm(s.pq + gpos + dd) : 0;
  }
  for (int x = tid; x < D * kPathWords * cap; x += blockDim.x) {
    const int w = (x >> lcap) % kPathWords;
    pool[x] = w == 4 ? -1 : (w == 8 ? INT_MAX : 0);
  }
  if (tid < D) { sh_eSlo[tid] = 0; sh_eShi[tid] = 0; sh_ec[tid] = 0; }
  if (tid == 0) { sh_root_succ = 0; sh_root_next = INT_MAX; sh_emitted = 0; }
  __syncthreads();
  // node sums of every layer
  for (int x = tid; x < (M << lD); x += blockDim.x) {
    const int m = x >> lD, l = x & ((1 << lD) - 1);
    if (l >= D) continue;
    const int v = st_tok[m * D + l];
    if (v < 0) continue;
    const PathTables t = path_tables(pool, cap, l);
    const int sl = table_slot<true>(t.key, cap, shift, v);
    add_split(&t.Slo[sl], &t.Shi[sl], &t.cnt[sl], (unsigned)st_pq[m * D + l]);
  }
  __syncthreads();
  // best(), last layer first: a candidate hands the best() of its next node to its node of this layer
  for (int d = D; d >= 1; --d) {
    const PathTables t = path_tables(pool, cap, d - 1);
    if (d < D) {
      const PathTables tn = path_tables(pool, cap, d);
      for (int m = tid; m < M; m += blockDim.x) {
        const int v = st_tok[m * D + d - 1], vn = st_tok[m * D + d];
        if (v < 0 || vn < 0) continue;
        atomicMax(&t.succ[table_slot<false>(t.key, cap, shift, v)], tn.best[table_slot<false>(tn.key, cap, shift, vn)]);
      }
      __syncthreads();
    }
    for (int x = tid; x < cap; x += blockDim.x)     // sums are only added to once per key: every slot on its own
      if (t.key[x] >= 0) {
        const double w = eq5_weight(s.alpha, ((u64)t.Shi[x] << 16) + t.Slo[x], t.cnt[x]);
        t.best[x] = (u64)__double_as_longlong(__dadd_rn(w, __longlong_as_double((long long)t.succ[x])));
      }
    __syncthreads();
  }
  // the root's best successor value (every first-layer node follows the root), then every node's
  // choice: the smallest successor token whose best() is the largest
  {
    const PathTables t = path_tables(pool, cap, 0);
    for (int x = tid; x < cap; x += blockDim.x)
      if (t.key[x] >= 0) atomicMax(&sh_root_succ, t.best[x]);
  }
  __syncthreads();
  for (int x = tid; x < (M << lD); x += blockDim.x) {
    const int m = x >> lD, l = x & ((1 << lD) - 1);
    if (l >= D) continue;
    const int v = st_tok[m * D + l];
    if (v < 0) continue;
    const PathTables t = path_tables(pool, cap, l);
    const u64 b = t.best[table_slot<false>(t.key, cap, shift, v)];
    if (l == 0) {
      if (b == sh_root_succ) atomicMin(&sh_root_next, v);
    } else {
      const PathTables tp = path_tables(pool, cap, l - 1);
      const int ps = table_slot<false>(tp.key, cap, shift, st_tok[m * D + l - 1]);
      if (b == tp.succ[ps]) atomicMin(&tp.next[ps], v);
    }
  }
  __syncthreads();
  if (tid == 0) {
    int next = sh_root_next, emitted = 0;
    for (int d = 1; d <= D && next != INT_MAX; ++d) {
      const PathTables t = path_tables(pool, cap, d - 1);
      const int sl = table_slot<false>(t.key, cap, shift, next);
      draft_tok[(size_t)i * D + d - 1] = next;
      if (draft_score)
        draft_score[(size_t)i * D + d - 1] = (float)eq5_weight(s.alpha, ((u64)t.Shi[sl] << 16) + t.Slo[sl], t.cnt[sl]);
      sh_draft[d - 1] = next;
      ++emitted;
      next = t.next[sl];
    }
    sh_emitted = emitted;
  }
  __syncthreads();
  // weight of the edges the draft took (Eq. 5 over the candidates that contain the edge)
  const int emitted = sh_emitted;
  for (int x = tid; x < (M << lD); x += blockDim.x) {
    const int m = x >> lD, d = (x & ((1 << lD) - 1)) + 1, at = m * D + d - 1;
    if (d > emitted || st_tok[at] != sh_draft[d - 1] || (d > 1 && st_tok[at - 1] != sh_draft[d - 2])) continue;
    add_split(&sh_eSlo[d - 1], &sh_eShi[d - 1], &sh_ec[d - 1], (unsigned)st_pq[at]);
  }
  __syncthreads();
  if (tid < emitted && draft_edge_w)
    draft_edge_w[(size_t)i * D + tid] =
        (float)eq5_weight(s.alpha, ((u64)sh_eShi[tid] << 16) + sh_eSlo[tid], sh_ec[tid]);
  if (tid == 0) draft_len[i] = emitted;
}

// Optional cap on the pool: of the matches of the query in one source path only the R with the largest end
// positions stay.  `list` holds the query's M matches (global memory, any order) and is compacted in
// place; the new count is returned (the same in every thread).  scratch: kStageWords * 2 shared words.
// Paths with at most R matches keep them all; for each of the others the R-th largest end position is
// found digit by digit, most significant first: one counting sweep over the list per digit fills a
// histogram of the digit for every such path (over the matches that agree with the digits found so
// far), and the path reads off which digit value its R-th largest position has.  No order among the
// matches is needed.
__device__ int cap_matches(const Dev& s, int g, int M, int32_t* list, int* scratch) {
  __shared__ int sh_warp_tot[kMaxWarps];
  __shared__ int sh_out;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int N = s.N, R = s.R, poff = g * N;
  // digits of `bits` bits: as wide as the histograms of N paths fit beside three words per path
  int bits = 5;
  while (bits > 1 && 3 * N + (N << bits) > 2 * kStageWords) --bits;
  int* cnt = scratch; int* lo = scratch + N; int* need = scratch + 2 * N; int* hist = scratch + 3 * N;   // hist[n << bits | digit]
  for (int n = tid; n < N; n += blockDim.x) { cnt[n] = 0; lo[n] = 0; need[n] = R; }
  __syncthreads();
  for (int m = tid; m < M; m += blockDim.x) atomicAdd(&cnt[path_of(s, list[m]) - poff], 1);
  __syncthreads();
  int over = 0;
  for (int n = tid; n < N; n += blockDim.x) over |= cnt[n] > R;
  if (!__syncthreads_or(over)) return M;
  int top = 0;
  while ((1 << top) < s.L) ++top;                     // positions have `top` bits
  // per path: the R-th largest position lies in [lo, lo + 2^shift) and is the need-th largest in there
  for (int shift = top; shift > 0;) {
    const int width = min(bits, shift);
    shift -= width;
    for (int x = tid; x < (N << bits); x += blockDim.x) hist[x] = 0;
    __syncthreads();
    for (int m = tid; m < M; m += blockDim.x) {
      const int gpos = list[m];
      const int j = path_of(s, gpos), n = j - poff;
      if (cnt[n] <= R) continue;
      const int rel = gpos - j * s.L - lo[n];
      if (rel >= 0 && (rel >> (shift + width)) == 0) atomicAdd(&hist[(n << bits) | (rel >> shift)], 1);
    }
    __syncthreads();
    for (int n = tid; n < N; n += blockDim.x)
      if (cnt[n] > R) {
        int left = need[n], digit = (1 << width) - 1;
        while (digit > 0 && hist[(n << bits) | digit] < left) { left -= hist[(n << bits) | digit]; --digit; }
        lo[n] += digit << shift; need[n] = left;
      }
    __syncthreads();
  }
  // keep what ends at or after the path's threshold; a chunk is read whole before any of it is written,
  // and what is written lands at or before the places already read
  if (tid == 0) sh_out = 0;
  __syncthreads();
  for (int base = 0; base < M; base += blockDim.x) {
    const int m = base + tid;
    int gpos = 0;
    bool keep = false;
    if (m < M) {
      gpos = list[m];
      const int j = path_of(s, gpos), n = j - poff;
      keep = cnt[n] <= R || gpos - j * s.L >= lo[n];
    }
    const unsigned b = __ballot_sync(FULL, keep);
    if (lane == 0) sh_warp_tot[warp] = __popc(b);
    __syncthreads();
    int before = sh_out;
    for (int w = 0; w < warp; ++w) before += sh_warp_tot[w];
    if (keep) list[before + __popc(b & ((1u << lane) - 1u))] = gpos;
    __syncthreads();
    if (tid == 0) { int t = sh_out; for (int w = 0; w < nwarps; ++w) t += sh_warp_tot[w]; sh_out = t; }
    __syncthreads();
  }
  return sh_out;
}

// Gather + DAG + search for query path i over its M (> 0) matches in mlist
// (shared or global memory).  Called by all threads of the CTA, after a barrier
// that follows write_defaults.
template <bool EXPORT>
__device__ __forceinline__ void dag_phase(const Dev& s, const Smem& sm, int i, int M, const int32_t* mlist,
                                          const int32_t* plen, int poff, int root, int32_t* draft_tok,
                                          int32_t* draft_len, float* draft_score, float* draft_edge_w) {
  // plen[j - poff] = length of path j (the prompt's lengths in shared memory, or the global array)
  if (!EXPORT && s.mode == 2) {
    int cap;
    if (best_path_fits(M, s.D, &cap)) {
      dag_best_path(s, sm, i, M, cap, mlist, plen, poff, draft_tok, draft_len, draft_score, draft_edge_w);
      return;
    }
    // too many matches for tables in shared memory: the path gets the greedy draft for now and is marked; the
    // launch that follows a best-path build (beams.cu) searches the marked paths over node tables in the
    // workspace's table area and replaces their drafts.  Without a table area the greedy draft stays, and says so.
    if (s.beam_stride > 0) {
      if (threadIdx.x == 0) s.bp_todo[i] = 1;
    } else if (threadIdx.x == 0) {
      atomicOr(s.status, SDMS_STATUS_SEARCH_FALLBACK);
    }
  }
  if (!EXPORT && s.pool == 2) list_pool(s, i, M, mlist, plen, poff, draft_tok, draft_len, draft_score, draft_edge_w);
  else if (M <= 32) dag_small<EXPORT>(s, sm, i, M, mlist, plen, poff, root, draft_tok, draft_len, draft_score, draft_edge_w);
  else if (!EXPORT && s.pool == 0 && M * s.D <= kStageWords && layers_in_round_ok(M, s.D))
    dag_layers(s, sm, i, M, mlist, plen, poff, root, draft_tok, draft_len, draft_score, draft_edge_w);
  else dag_block<EXPORT>(s, sm, i, M, mlist, plen, poff, root, draft_tok, draft_len, draft_score, draft_edge_w);
}

template <bool EXPORT>
__global__ void __launch_bounds__(kDagThreads, EXPORT ? 1 : 2) dag_kernel(Dev s, int32_t* __restrict__ draft_tok,
                                                          int32_t* __restrict__ draft_len,
                                                          float* __restrict__ draft_score,
                                                          float* __restrict__ draft_edge_w, int round, int k,
                                                          int32_t* __restrict__ used_k) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const Smem sm = carve<EXPORT>(smem_raw);
  __shared__ int32_t sh_len[SDMS_MAX_PATHS_PER_GROUP];
  const int i = blockIdx.x;
  // the path lengths are older than the kernels this one follows (probe, scan: their CTAs let it start only after
  // their own wait): fetched while those drain
  for (int n = threadIdx.x; n < s.N; n += blockDim.x) sh_len[n] = ldm(s.len + (i / s.N) * s.N + n);
  const int32_t root = ldm(s.rec + (size_t)i * kRecWords + 1);
  grid_wait();
  grid_release();
  // what probe and scan left for this path, in one round trip
  const int32_t q_mode = s.q_mode[i];
  const int q_found = min(s.q_cursor[i], s.q_reserved[i]), q_off = s.q_off[i];
  if (i == 0) {                                       // probe and scan are done with these: the next build finds them at zero
    for (int x = threadIdx.x; x < s.G; x += blockDim.x) s.g_nscan[x] = 0;
    // (the slices of a back-off build's earlier rounds stay where they are until its last round)
    if (threadIdx.x == 0 && (!(round & kRoundBackoff) || (round & kRoundLast))) *s.match_cursor = 0ull;
  }
  if ((round & kRoundNotFirst) && q_mode == Q_DONE) return;     // drafted in an earlier round, from a longer suffix
  write_defaults<EXPORT>(s, i, draft_tok, draft_score, draft_edge_w);
  const int M = q_mode == Q_NONE ? 0 : q_found;
  if (M == 0) {
    if (threadIdx.x == 0) { draft_len[i] = 0; if (used_k) used_k[i] = 0; }
    return;
  }
  if ((round & kRoundBackoff) && threadIdx.x == 0) { s.q_mode[i] = Q_DONE; if (used_k) used_k[i] = k; }
  const int g = i / s.N;
  __syncthreads();
  int32_t* const mlist = s.matches + q_off;
  int Mk = M;
  if (s.R > 0) {                                    // (a second pass over the same build finds nothing left to cut)
    Mk = cap_matches(s, g, M, mlist, sm.st_tok);
    if (threadIdx.x == 0) s.q_cursor[i] = Mk;
    __syncthreads();
  }
  // more matches than a warp holds: all SMs share the work (the pass that follows this kernel)
  if (!EXPORT && s.pool == 0 && s.mode != 2 && Mk > 32 && wide_register(s, i, Mk)) return;
  dag_phase<EXPORT>(s, sm, i, Mk, mlist, sh_len, g * s.N, root, draft_tok, draft_len, draft_score, draft_edge_w);
}

// Whole draft construction of one query path in one CTA, for prompts whose
// histories are small enough that every CTA can afford to read them itself:
// probe the index; a k-gram with at most kInlineSlots occurrences is answered
// from its bucket, any other by streaming the other paths of the prompt with
// 128-bit loads (last token first, the rest of the window on a hit); then the
// gather / DAG / search phase runs on the matches just found.  The matches also
// go to the path's private slice of the match list for inspection.
// Do the first k - 2 tokens of the window that ends at `at` equal the query's?  (The last two have been
// compared by the caller.)
__device__ __forceinline__ bool window_head_equal(const int32_t* at, int k, const int32_t* q) {
  for (int t = 0; t < k - 2; ++t)
    if (ldm(at - (k - 1) + t) != q[t]) return false;
  return true;
}

// ---- a thread-block cluster shares the scan of its prompt ------------------------------------------
// In the single-launch build every query that its index bucket cannot answer streams the other paths
// of the prompt; with many such queries the same histories cross the chip once per query.  When the
// CTAs of a launch form clusters (paths [c * csize, (c + 1) * csize) of a prompt), each CTA instead
// scans 1 / csize of the prompt's tokens for ALL scan queries of its cluster and appends what it finds
// to the owning path's match slice (a cursor in global memory).  Queries are exchanged through
// distributed shared memory; two cluster barriers frame the scan.
constexpr int kShareMinTokens = 32768;   // below this a CTA reads its prompt faster than it talks to its cluster
constexpr int kPubWords = SDMS_MAX_K + 2;

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned cluster_rank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// word `w` of the array `local` (shared memory) as CTA `rank` of the cluster holds it
__device__ __forceinline__ int32_t ld_cluster(const int32_t* local, unsigned rank) {
  const uint32_t mine = (uint32_t)__cvta_generic_to_shared(local);
  uint32_t theirs;
  int32_t v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(theirs) : "r"(mine), "r"(rank));
  asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(theirs) : "memory");
  return v;
}

// This CTA's share of the prompt's tokens against the nq scan queries of the cluster.  cq[q] holds
// {path index of the query, unused, k tokens}.  16-byte chunks as in the single-CTA scan: a position
// passes on to the full comparison only if its own token and the one before it fit.
__device__ void shared_scan(const Dev& s, int g, int k, int nq, const int32_t (*cq)[kPubWords], const int32_t* sh_len,
                            unsigned crank, int csize) {
  const int tid = threadIdx.x;
  const int32_t* gtok = s.tok + (size_t)g * s.N * s.L;
  const int pos0 = g * s.N * s.L, slice = s.N * s.L;
  const int per = s.L >> 2, total = s.N * per;
  const int4* g4 = reinterpret_cast<const int4*>(gtok);
  const int lo = (int)((long long)total * crank / csize), hi = (int)((long long)total * (crank + 1) / csize);
  constexpr int kBatch = 8;
  for (int base = lo; base < hi; base += kBatch * blockDim.x) {           // same trip count for every thread
    int4 w[kBatch];
    int e0[kBatch], e_hi[kBatch], jn[kBatch];
#pragma unroll
    for (int r = 0; r < kBatch; ++r) {
      const int x = base + r * blockDim.x + tid;
      jn[r] = x < hi ? x / per : -1;
      e0[r] = jn[r] >= 0 ? 4 * x - jn[r] * s.L : 0;
      e_hi[r] = jn[r] >= 0 ? sh_len[jn[r]] - 2 : -1;
      w[r] = make_int4(-1, -1, -1, -1);
      if (e0[r] <= e_hi[r]) w[r] = ldm(g4 + x);
    }
    int left[kBatch];
#pragma unroll
    for (int r = 0; r < kBatch; ++r) left[r] = __shfl_up_sync(FULL, w[r].w, 1);   // last token of the chunk before this one
#pragma unroll 1
    for (int q = 0; q < nq; ++q) {
      const int i = cq[q][0], own = i - g * s.N;
      const int last = cq[q][2 + k - 1], before_last = k >= 2 ? cq[q][2 + k - 2] : -1;
      unsigned cand = 0;                                              // bit 4 r + u: position u of chunk r is a candidate
#pragma unroll
      for (int r = 0; r < kBatch; ++r) {
        const int v[5] = {left[r], w[r].x, w[r].y, w[r].z, w[r].w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const bool ok = v[u + 1] == last && jn[r] != own && e0[r] + u >= k - 1 && e0[r] + u <= e_hi[r] &&
                          (k < 2 || v[u] == before_last || (u == 0 && (tid & 31) == 0));
          cand |= (unsigned)ok << (4 * r + u);
        }
      }
      while (cand) {
        const int bit = __ffs(cand) - 1;
        cand &= cand - 1;
        const int at = 4 * (base + (bit >> 2) * (int)blockDim.x + tid) + (bit & 3);   // position within the prompt
        if (k >= 2 && (bit & 3) == 0 && (tid & 31) == 0 && ldm(gtok + at - 1) != before_last) continue;
        if (k >= 3 && !window_head_equal(gtok + at, k, &cq[q][2])) continue;
        const int n = atomicAdd(&s.q_cursor[i], 1);
        s.matches[(size_t)i * slice + n] = pos0 + at;
      }
    }
  }
}

// SHARE: the code of the cluster-shared scan is compiled in (kernels for prompts below kShareMinTokens leave it
// out: after a cold start the step fetches every instruction it may run past)
template <bool EXPORT, bool SHARE>
__device__ void build_phase(const Dev& s, const Smem& sm, int k_hi, int k_lo, int32_t* draft_tok, int32_t* draft_len,
                            float* draft_score, float* draft_edge_w, int32_t* used_k,
                            const int32_t* own_rec = nullptr, int csize = 0) {
  __shared__ int sh_mode, sh_M;
  __shared__ int32_t sh_pub[kPubWords];                     // this CTA's query as its cluster sees it: path, mode, tokens
  __shared__ int32_t sh_cq[kMaxClusterPaths][kPubWords];    // the scan queries of the cluster
  __shared__ int sh_nq;
  __shared__ uint32_t sh_count, sh_pos[kInlineSlots];
  __shared__ int32_t sh_q[SDMS_MAX_K];
  __shared__ int32_t sh_len[SDMS_MAX_PATHS_PER_GROUP];
  const int i = blockIdx.x, tid = threadIdx.x;
  const int g = i / s.N;
  for (int n = tid; n < s.N; n += blockDim.x) sh_len[n] = ldm(s.len + g * s.N + n);
  const int slice = s.N * s.L;
  int32_t* my_matches = s.matches + (size_t)i * slice;

  write_defaults<EXPORT>(s, i, draft_tok, draft_score, draft_edge_w);
  // the cluster shares its scans (same decision in every CTA of the launch)
  const bool share = SHARE && csize > 1 && k_lo == k_hi && s.eps == 0 && (s.L & 3) == 0 && slice >= kShareMinTokens;
  // With k_lo < k_hi the suffix length backs off: the longest k in [k_lo, k_hi] that has a match wins.
  int k = k_hi;
  for (;; --k) {
  if (tid == 0) {
    // the path's record: length and last tokens (newest first) in one 128-byte line (or the copy
    // the caller already holds in shared memory)
    const int32_t* rec = own_rec ? own_rec : s.rec + (size_t)i * kRecWords;
    const int len_i = ldm(rec);
    int mode = Q_NONE;
    uint32_t fp = 0, count = 0;
    if (len_i >= k && len_i < s.L && s.eps > 0) {      // fuzzy matches are found by scanning only
      for (int t = 0; t < k; ++t) sh_q[t] = ldm(rec + k - t);
      mode = Q_SCAN;
    } else if (len_i >= k && len_i < s.L) {
      // the index is asked for the query's last nx tokens: all k of them unless the context keeps fewer tables
      const int nx = min(k, s.idx_n);
      uint64_t h = gram_init(nx);
      for (int t = 0; t < k; ++t) { const int32_t x = ldm(rec + k - t); sh_q[t] = x; if (t >= k - nx) h = gram_step(h, x); }
      h = gram_final(h);
      fp = gram_fp(h);
      const uint32_t* table = index_table(s, g, nx);
      uint32_t b = gram_bucket(h, s.table_cap);
      for (uint32_t probe = 0; probe < s.table_cap; ++probe) {
        const uint4* cand = reinterpret_cast<const uint4*>(table + (size_t)b * kBucketWords);
        const uint4 lo = ldm(cand), hi = ldm(cand + 1);      // both halves in flight together
        if (lo.x == fp) {
          count = lo.y;
          sh_pos[0] = lo.z; sh_pos[1] = lo.w; sh_pos[2] = hi.x; sh_pos[3] = hi.y; sh_pos[4] = hi.z; sh_pos[5] = hi.w;
          mode = count <= (uint32_t)kInlineSlots ? Q_INLINE : Q_SCAN;
          break;
        }
        if (lo.x == 0u) break;
        b = (b + 1) & (s.table_cap - 1);
      }
    }
    sh_mode = mode; sh_count = count; sh_M = 0;
    s.q_fp[i] = fp; s.q_mode[i] = mode; s.q_reserved[i] = mode == Q_NONE ? 0 : slice; s.q_off[i] = i * slice;
    if (share) {
      sh_pub[0] = i; sh_pub[1] = mode;
      for (int t = 0; t < k; ++t) sh_pub[2 + t] = sh_q[t];
      if (mode == Q_SCAN) s.q_cursor[i] = 0;              // the cluster's scanners count this query's matches here
    }
  }
  __syncthreads();
  const int mode = sh_mode;
  if (mode == Q_INLINE) {
    if (tid < (int)sh_count) {
      const uint32_t lpos = sh_pos[tid];
      const int jn = (int)(lpos / (uint32_t)s.L);
      const int j = g * s.N + jn;
      const int e = (int)(lpos % (uint32_t)s.L);
      if (j != i && e >= k - 1 && e <= sh_len[jn] - 2) {
        const int32_t* c = s.tok + (size_t)j * s.L + (e - k + 1);
        bool same = true;
        for (int t = 0; t < k; ++t) same = same && (ldm(c + t) == sh_q[t]);
        if (same) {
          const int at = atomicAdd(&sh_M, 1);
          sm.list[at] = j * s.L + e;
          my_matches[at] = j * s.L + e;
        }
      }
    }
  }
  if (share) {
    cluster_sync_all();                                     // every query of the cluster is published
    const unsigned crank = cluster_rank();
    for (int x = tid; x < csize * (k + 2); x += blockDim.x) {
      const int r = x / (k + 2), w = x - r * (k + 2);
      sh_cq[r][w] = ld_cluster(&sh_pub[w], (unsigned)r);
    }
    __syncthreads();
    if (tid == 0) {                                         // keep the scan queries, in rank order
      int nq = 0;
      for (int r = 0; r < csize; ++r)
        if (sh_cq[r][1] == Q_SCAN) {
          if (nq != r) for (int w = 0; w < k + 2; ++w) sh_cq[nq][w] = sh_cq[r][w];
          ++nq;
        }
      sh_nq = nq;
    }
    __syncthreads();
    if (sh_nq > 0) shared_scan(s, g, k, sh_nq, sh_cq, sh_len, crank, csize);
    cluster_sync_all();                                     // all shares scanned; nobody reads a neighbour's memory any more
    if (mode == Q_SCAN) {
      const int M = __ldcg(s.q_cursor + i);
      for (int x = tid; x < min(M, kListCap); x += blockDim.x) sm.list[x] = __ldcg(my_matches + x);
      if (tid == 0) sh_M = M;
    }
  } else if (mode == Q_SCAN && s.eps > 0) {
    // Eq. 4 with tolerance 1.  A window s' is within one edit of the query q iff, with a = their common
    // prefix and b = their common suffix (each at most the shorter length), a + b >= max(|q|, |s'|) - 1.
    // For the windows that end at e, b is shared; a is looked at only as far as it can still decide.
    const int32_t* gtok = s.tok + (size_t)g * s.N * s.L;
    for (int jn = 0; jn < s.N; ++jn) {
      if (g * s.N + jn == i) continue;
      const int32_t* row = gtok + (size_t)jn * s.L;
      const int e_hi = sh_len[jn] - 2;
      for (int e = tid; e <= e_hi; e += blockDim.x) {
        int b = 0;
        while (b < k && b <= e && ldm(row + e - b) == sh_q[k - 1 - b]) ++b;
        bool found = false;
        for (int n = max(1, k - 1); n <= k + 1 && !found; ++n) {
          if (e - n + 1 < 0) break;
          const int shorter = min(k, n), need = max(k, n) - 1 - min(b, shorter);
          if (need <= 0) { found = true; break; }
          if (need > shorter) continue;
          int a = 0;
          while (a < need && ldm(row + e - n + 1 + a) == sh_q[a]) ++a;
          found = a >= need;
        }
        if (found) {
          const int at = atomicAdd(&sh_M, 1);
          const int pos = (g * s.N + jn) * s.L + e;
          if (at < kListCap) sm.list[at] = pos;
          my_matches[at] = pos;
        }
      }
    }
  } else if (mode == Q_SCAN) {
    // every other path of the prompt, all loads independent of each other:
    // compare the last token of the query first, the rest of the window on a hit
    const int last = sh_q[k - 1];
    const int32_t* gtok = s.tok + (size_t)g * s.N * s.L;
    const int own = i - g * s.N;
    const int pos0 = g * s.N * s.L;
    if ((s.L & 3) == 0) {
      // 16-byte chunks, chunk x = path x / per, tokens 4 * (x % per) ..; a thread keeps eight loads in flight.
      // A position passes on to the full comparison only if the token before it fits as well: that token
      // sits in the same chunk or in the neighbouring lane's, so the filter costs no dependent load.
      const int per = s.L >> 2, total = s.N * per;
      const int4* g4 = reinterpret_cast<const int4*>(gtok);
      const int before_last = k >= 2 ? sh_q[k - 2] : -1;
      constexpr int kBatch = 8;
      for (int base = 0; base < total; base += kBatch * blockDim.x) {       // same trip count for every thread
        int4 w[kBatch];
        int e0[kBatch], e_hi[kBatch];
#pragma unroll
        for (int r = 0; r < kBatch; ++r) {
          const int x = base + r * blockDim.x + tid;
          const int jn = x < total ? x / per : own;
          e0[r] = 4 * x - jn * s.L;                                   // 4 * (x % per)
          e_hi[r] = jn != own ? sh_len[jn] - 2 : -1;                  // last position with a follower
          w[r] = make_int4(-1, -1, -1, -1);
          if (e0[r] <= e_hi[r]) w[r] = ldm(g4 + x);
        }
        unsigned cand = 0;                                            // bit 4 r + u: position u of chunk r is a candidate
#pragma unroll
        for (int r = 0; r < kBatch; ++r) {
          const int left = __shfl_up_sync(FULL, w[r].w, 1);           // last token of the chunk before this one
          const int v[5] = {left, w[r].x, w[r].y, w[r].z, w[r].w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const bool ok = v[u + 1] == last && e0[r] + u >= k - 1 && e0[r] + u <= e_hi[r] &&
                            (k < 2 || v[u] == before_last || (u == 0 && (tid & 31) == 0));
            cand |= (unsigned)ok << (4 * r + u);
          }
        }
        // one copy of the code that looks closer, run once per candidate
        while (cand) {
          const int bit = __ffs(cand) - 1;
          cand &= cand - 1;
          const int at = 4 * (base + (bit >> 2) * (int)blockDim.x + tid) + (bit & 3);   // position within the prompt
          if (k >= 2 && (bit & 3) == 0 && (tid & 31) == 0 && ldm(gtok + at - 1) != before_last) continue;
          if (k >= 3 && !window_head_equal(gtok + at, k, sh_q)) continue;
          const int n = atomicAdd(&sh_M, 1);
          if (n < kListCap) sm.list[n] = pos0 + at;
          my_matches[n] = pos0 + at;
        }
      }
    } else {
      const int total = s.N * s.L;
      for (int x = tid; x < total; x += blockDim.x) {
        const int jn = x / s.L, e = x - jn * s.L;
        if (jn == own || e < k - 1 || e > sh_len[jn] - 2) continue;
        if (ldm(gtok + x) != last) continue;
        if (k >= 2 && (ldm(gtok + x - 1) != sh_q[k - 2] || !window_head_equal(gtok + x, k, sh_q))) continue;
        const int n = atomicAdd(&sh_M, 1);
        if (n < kListCap) sm.list[n] = pos0 + x;
        my_matches[n] = pos0 + x;
      }
    }
  }
  __syncthreads();
  if (sh_M > 0 || k <= k_lo) break;
  __syncthreads();                                   // everybody has read sh_M before the next probe resets it
  }
  int M = sh_M;
  if (s.R > 0 && M > s.R) {                          // (uniform) the cap can only bite with more than R matches
    const int M0 = M;
    M = cap_matches(s, g, M0, my_matches, sm.st_tok);
    if (M < M0 && M <= kListCap)
      for (int x = tid; x < M; x += blockDim.x) sm.list[x] = my_matches[x];
    __syncthreads();
  }
  if (tid == 0) { s.q_cursor[i] = M; if (used_k) used_k[i] = M > 0 ? k : 0; }
  if (M == 0) {
    if (tid == 0) draft_len[i] = 0;
    return;
  }
  dag_phase<EXPORT>(s, sm, i, M, M <= kListCap ? sm.list : my_matches, sh_len, g * s.N, sh_q[k - 1], draft_tok,
                    draft_len, draft_score, draft_edge_w);
}

template <bool EXPORT, bool SHARE>
__global__ void __launch_bounds__(kFusedThreads, 1) build_fused_kernel(Dev s, int k_hi, int k_lo, int32_t* draft_tok,
                                                                  int32_t* draft_len, float* draft_score,
                                                                  float* draft_edge_w, int32_t* used_k, int csize) {
  grid_wait();
  grid_release();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const Smem sm = carve<EXPORT>(smem_raw);
  build_phase<EXPORT, SHARE>(s, sm, k_hi, k_lo, draft_tok, draft_len, draft_score, draft_edge_w, used_k, nullptr, csize);
}

// One launch per decode step.  The CTAs of a prompt form a thread-block cluster.  Each CTA first
// checks its path's previous draft against the sampled tokens and appends what was accepted (tokens,
// probabilities, index entries); after a cluster-wide barrier with release/acquire semantics every
// path of the prompt is up to date and each CTA builds its path's next draft.  draft_tok / draft_len
// hold the previous drafts on entry and the new ones on exit.
// k_lo < k: the suffix length backs off from k to k_lo (used_k, if given, receives each path's choice).
template <bool SHARE>
__global__ void __launch_bounds__(kFusedThreads, 1) step_kernel(Dev s, int k, int k_lo, const int32_t* sampled,
                                                           const float* sampled_lp, int32_t* accept_len,
                                                           int32_t* draft_tok, int32_t* draft_len,
                                                           float* draft_score, float* draft_edge_w,
                                                           int32_t* used_k) {
  grid_wait();
  grid_release();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const Smem sm = carve<false>(smem_raw);
  __shared__ int32_t sh_own_rec[kRecWords];
  accept_commit_phase(s, blockIdx.x, draft_tok, draft_len, sampled, sampled_lp, accept_len, sh_own_rec, k);
  // every thread of every CTA of the cluster gets here exactly once (no early exit above)
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  build_phase<false, SHARE>(s, sm, k, k_lo, draft_tok, draft_len, draft_score, draft_edge_w, used_k, sh_own_rec, s.N);
}

}  // namespace

cudaError_t dag_kernel_setup() {
  cudaError_t e = cudaFuncSetAttribute(dag_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)dag_smem_bytes<false>());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(dag_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)dag_smem_bytes<true>());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(build_fused_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)dag_smem_bytes<false>());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(build_fused_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)dag_smem_bytes<false>());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(step_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dag_smem_bytes<false>());
  if (e == cudaSuccess) e = cudaFuncSetAttribute(step_kernel<false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(step_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dag_smem_bytes<false>());
  if (e == cudaSuccess) e = cudaFuncSetAttribute(step_kernel<true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  return e;
}

namespace {
void step_launch_config(const Dev& s, cudaStream_t stream, cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr) {
  *cfg = cudaLaunchConfig_t{};
  cfg->gridDim = dim3(s.P); cfg->blockDim = dim3(kFusedThreads);
  cfg->dynamicSmemBytes = dag_smem_bytes<false>(); cfg->stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = s.N; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg->attrs = attr; cfg->numAttrs = 2;
}
}  // namespace

// Can the prompts of this context run as clusters (one CTA per path) on this device?
bool step_kernel_fits(const Dev& s) {
  if (!s.fused || s.N > kMaxClusterPaths) return false;
  cudaLaunchConfig_t cfg; cudaLaunchAttribute attr[2];
  step_launch_config(s, 0, &cfg, attr);
  cfg.numAttrs = 1;                                   // occupancy only looks at the cluster shape
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, step_kernel<true>, &cfg) != cudaSuccess) { cudaGetLastError(); return false; }
  // every prompt's cluster resident at once: large clusters leave SMs of a GPC idle, and a launch whose
  // clusters queue up for the device is slower than the separate accept and build launches
  return (long long)clusters * s.N >= s.P;
}

cudaError_t launch_step(const Dev& s, int k, int k_lo, const int32_t* sampled, const float* sampled_lp,
                        int32_t* accept_len, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                        float* draft_edge_w, int32_t* used_k, cudaStream_t stream) {
  cudaLaunchConfig_t cfg; cudaLaunchAttribute attr[2];
  step_launch_config(s, stream, &cfg, attr);
  const bool share = (s.L & 3) == 0 && (long long)s.N * s.L >= kShareMinTokens;       // the prompt is worth sharing its scan
  return cudaLaunchKernelEx(&cfg, share ? step_kernel<true> : step_kernel<false>, s, k, k_lo, sampled, sampled_lp, accept_len,
                            draft_tok, draft_len, draft_score, draft_edge_w, used_k);
}

cudaError_t launch_dag(const Dev& s, bool with_export, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                       float* draft_edge_w, cudaStream_t stream, int round, int k, int32_t* used_k) {
  if (with_export)
    return launch_overlapped(dag_kernel<true>, dim3(s.P), dim3(kDagThreads), dag_smem_bytes<true>(), stream, s,
                             draft_tok, draft_len, draft_score, draft_edge_w, 0, 0, (int32_t*)nullptr);
  return launch_overlapped(dag_kernel<false>, dim3(s.P), dim3(kDagThreads), dag_smem_bytes<false>(), stream, s,
                           draft_tok, draft_len, draft_score, draft_edge_w, round, k, used_k);
}

// Cluster size (CTAs = consecutive paths of one prompt) of the single-launch build, 1 for none.  A cluster
// shares the scan of its prompt (shared_scan), which shortens the longest CTA of a launch but adds two
// barriers to every CTA: it pays when the whole launch is resident at once, i.e. when the launch's
// time is its slowest CTA's, and loses when CTAs queue for SMs anyway.  Sizes above 8 leave too many
// SMs of a GPC idle.
int build_cluster_size(const Dev& s) {
  if (!s.fused || (s.L & 3) != 0 || (long long)s.N * s.L < kShareMinTokens) return 1;
  for (int c = 8; c >= 2; --c) {
    if (s.N % c) continue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(s.P); cfg.blockDim = dim3(kFusedThreads); cfg.dynamicSmemBytes = dag_smem_bytes<false>();
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, build_fused_kernel<false, true>, &cfg) != cudaSuccess) { cudaGetLastError(); continue; }
    if ((long long)clusters * c >= s.P) return c;
  }
  return 1;
}

cudaError_t launch_build_fused(const Dev& s, int k_hi, int k_lo, int32_t* draft_tok, int32_t* draft_len,
                               float* draft_score, float* draft_edge_w, int32_t* used_k, cudaStream_t stream) {
  if (s.build_cluster <= 1 || k_lo != k_hi)
    return launch_overlapped(build_fused_kernel<false, false>, dim3(s.P), dim3(kFusedThreads), dag_smem_bytes<false>(), stream,
                             s, k_hi, k_lo, draft_tok, draft_len, draft_score, draft_edge_w, used_k, 0);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(s.P); cfg.blockDim = dim3(kFusedThreads);
  cfg.dynamicSmemBytes = dag_smem_bytes<false>(); cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = s.build_cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, build_fused_kernel<false, true>, s, k_hi, k_lo, draft_tok, draft_len, draft_score, draft_edge_w,
                            used_k, (int)s.build_cluster);
}

}  // namespace sdms
