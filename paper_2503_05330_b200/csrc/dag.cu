// Follower gather, layered DAG aggregation (Eq. 5) and greedy extraction.
//
// dag_kernel : one CTA per query path.  Layer by layer (d = 1..D) every match m
//              contributes its d-th follower v = tok[e+d] with the fixed-point
//              probability pq[e+d]; contributions to the same token merge in a
//              shared-memory hash table (node = distinct token of the layer):
//                S_all / c_all : sum over every candidate      -> node score
//                S_cur / c_cur : candidates coming from the node the walk stands
//                                on                             -> successor test
//                                                                  and edge weight
//              All sums are integers, so the order of the atomics cannot change
//              a result.  After the pass one warp picks the best successor; with
//              the export enabled other warps select the B best nodes of the
//              layer and the Ke best out-edges of the nodes kept one layer up.
//              A layer with more distinct tokens than the table holds is
//              processed in several passes, each over the tokens of one residue
//              class, so that any fan-out fits a fixed amount of shared memory.
#include "sdms_internal.h"

namespace sdms {

namespace {

typedef unsigned long long u64;
constexpr int CAP = kDagCap;
constexpr int kWarps = kDagThreads / 32;
constexpr int MAXB = SDMS_MAX_DAG_NODES;
constexpr int MAXKE = SDMS_MAX_DAG_EDGES;

struct Cand {            // a node or an edge competing in a selection
  double w; u64 S; unsigned cnt; int tok; int valid;
};

__device__ __forceinline__ Cand warp_best(Cand c) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Cand x;
    x.w = __shfl_xor_sync(0xffffffffu, c.w, o);
    x.S = __shfl_xor_sync(0xffffffffu, c.S, o);
    x.cnt = __shfl_xor_sync(0xffffffffu, c.cnt, o);
    x.tok = __shfl_xor_sync(0xffffffffu, c.tok, o);
    x.valid = __shfl_xor_sync(0xffffffffu, c.valid, o);
    if (x.valid && (!c.valid || ranks_before(x.w, x.tok, c.w, c.tok))) c = x;
  }
  return c;
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

struct Smem {
  u64* n_Sall; u64* n_Scur; u64* e_S;
  int* n_key; unsigned* n_call; unsigned* n_ccur; int* n_touch;
  int* e_key; unsigned* e_c; int* e_touch;
  // export lists
  u64* r_node_S; int* r_node_tok; unsigned* r_node_cnt;
  u64* r_edge_S; int* r_edge_dst; unsigned* r_edge_cnt;
  u64* t_S; int* t_tok; unsigned* t_cnt;        // per-warp scratch for merging
  int* kept; int* r_nedge; int* r_outdeg;
};

template <bool EXPORT>
__host__ __device__ constexpr size_t dag_smem_bytes() {
  size_t b = (size_t)CAP * (8 + 8 + 4 + 4 + 4 + 4);
  if (EXPORT) {
    b += (size_t)CAP * (8 + 4 + 4 + 4);
    b += (size_t)MAXB * 16 + (size_t)MAXB * MAXKE * 16 + (size_t)kWarps * 32 * 16 + (size_t)MAXB * 12;
  }
  return b;
}

template <bool EXPORT>
__device__ Smem carve(unsigned char* base) {
  Smem m;
  u64* p8 = reinterpret_cast<u64*>(base);
  m.n_Sall = p8; p8 += CAP;
  m.n_Scur = p8; p8 += CAP;
  if (EXPORT) {
    m.e_S = p8; p8 += CAP;
    m.r_node_S = p8; p8 += MAXB;
    m.r_edge_S = p8; p8 += MAXB * MAXKE;
    m.t_S = p8; p8 += kWarps * 32;
  }
  int* p4 = reinterpret_cast<int*>(p8);
  m.n_key = p4; p4 += CAP;
  m.n_call = reinterpret_cast<unsigned*>(p4); p4 += CAP;
  m.n_ccur = reinterpret_cast<unsigned*>(p4); p4 += CAP;
  m.n_touch = p4; p4 += CAP;
  if (EXPORT) {
    m.e_key = p4; p4 += CAP;
    m.e_c = reinterpret_cast<unsigned*>(p4); p4 += CAP;
    m.e_touch = p4; p4 += CAP;
    m.r_node_tok = p4; p4 += MAXB;
    m.r_node_cnt = reinterpret_cast<unsigned*>(p4); p4 += MAXB;
    m.r_edge_dst = p4; p4 += MAXB * MAXKE;
    m.r_edge_cnt = reinterpret_cast<unsigned*>(p4); p4 += MAXB * MAXKE;
    m.t_tok = p4; p4 += kWarps * 32;
    m.t_cnt = reinterpret_cast<unsigned*>(p4); p4 += kWarps * 32;
    m.kept = p4; p4 += MAXB;
    m.r_nedge = p4; p4 += MAXB;
    m.r_outdeg = p4; p4 += MAXB;
  }
  return m;
}

__device__ __forceinline__ unsigned slot_hash(unsigned x) { return (x * 2654435761u) >> 22; }   // 10 bits = CAP
static_assert(CAP == 1024, "slot_hash yields 10 bits");

template <bool EXPORT>
__global__ void __launch_bounds__(kDagThreads) dag_kernel(Dev s, int32_t* __restrict__ draft_tok,
                                                          int32_t* __restrict__ draft_len,
                                                          float* __restrict__ draft_score,
                                                          float* __restrict__ draft_edge_w) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem sm = carve<EXPORT>(smem_raw);
  __shared__ int sh_nn, sh_ne, sh_overflow, sh_found, sh_cur, sh_nkept, sh_nnode_run, sh_node_total;
  __shared__ double sh_best_w, sh_best_ew;
  __shared__ int sh_best_tok, sh_best_valid;

  const int i = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = s.D, B = s.B, Ke = s.Ke;

  // defaults: no draft, empty export
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
  const int M = s.q_mode[i] == Q_NONE ? 0 : min(s.q_cursor[i], s.q_reserved[i]);
  if (M == 0) {
    if (tid == 0) draft_len[i] = 0;
    return;
  }
  const int32_t* mlist = s.matches + s.q_off[i];
  const int root = s.tok[(size_t)i * s.L + s.len[i] - 1];

  for (int x = tid; x < CAP; x += blockDim.x) {
    sm.n_key[x] = -1; sm.n_Sall[x] = 0; sm.n_Scur[x] = 0; sm.n_call[x] = 0; sm.n_ccur[x] = 0;
    if (EXPORT) { sm.e_key[x] = -1; sm.e_S[x] = 0; sm.e_c[x] = 0; }
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
    bool layer_done = false;
    while (!layer_done) {
      if (tid == 0) { sh_best_valid = 0; sh_nnode_run = 0; sh_node_total = 0; }
      if (EXPORT && tid < MAXB) { sm.r_nedge[tid] = 0; sm.r_outdeg[tid] = 0; }
      __syncthreads();
      bool overflowed = false;
      for (int part = 0; part < npart && !overflowed; ++part) {
        // ---- accumulate this residue class of follower tokens ----
        for (int m = tid; m < M; m += blockDim.x) {
          const int gpos = mlist[m];
          const int j = gpos / s.L;
          const int e = gpos - j * s.L;
          if (e + d > s.len[j] - 1) continue;
          const int v = __ldg(s.tok + gpos + d);
          if (npart > 1 && v % npart != part) continue;
          const int u = d == 1 ? root : __ldg(s.tok + gpos + d - 1);
          const u64 p = (u64)(unsigned)__ldg(s.pq + gpos + d);
          unsigned h = slot_hash((unsigned)(v / npart));
          int slot = -1;
          for (int probe = 0; probe < CAP; ++probe) {
            const int old = atomicCAS(&sm.n_key[h], -1, v);
            if (old == -1) sm.n_touch[atomicAdd(&sh_nn, 1)] = (int)h;
            if (old == -1 || old == v) { slot = (int)h; break; }
            h = (h + 1) & (CAP - 1);
          }
          if (slot < 0) { sh_overflow = 1; continue; }
          atomicAdd(&sm.n_Sall[slot], p);
          atomicAdd(&sm.n_call[slot], 1u);
          if (u == cur) { atomicAdd(&sm.n_Scur[slot], p); atomicAdd(&sm.n_ccur[slot], 1u); }
          if (EXPORT && d > 1) {
            int b = -1;
            for (int x = 0; x < nkept; ++x) if (sm.kept[x] == u) { b = x; break; }
            if (b >= 0) {
              const int ekey = v * MAXB + b;                 // (destination, kept source) in one word
              unsigned he = slot_hash((unsigned)(v / npart) * 37u + (unsigned)b);
              int es = -1;
              for (int probe = 0; probe < CAP; ++probe) {
                const int old = atomicCAS(&sm.e_key[he], -1, ekey);
                if (old == -1) sm.e_touch[atomicAdd(&sh_ne, 1)] = (int)he;
                if (old == -1 || old == ekey) { es = (int)he; break; }
                he = (he + 1) & (CAP - 1);
              }
              if (es < 0) { sh_overflow = 1; continue; }
              atomicAdd(&sm.e_S[es], p);
              atomicAdd(&sm.e_c[es], 1u);
            }
          }
        }
        __syncthreads();
        const int nn = sh_nn, ne = EXPORT ? sh_ne : 0;
        overflowed = sh_overflow || (npart < npart_max && (nn > CAP * 3 / 4 || ne > CAP * 3 / 4));
        if (!overflowed) {
          // ---- selections, one warp each ----
          if (warp == 0 && walking) {
            auto get = [&](int x) {
              const int sl = sm.n_touch[x];
              Cand c;
              c.tok = sm.n_key[sl]; c.S = sm.n_Sall[sl]; c.cnt = sm.n_call[sl];
              c.valid = s.mode == 1 || sm.n_ccur[sl] > 0;
              c.w = eq5_weight(s.alpha, c.S, c.cnt);
              // carry the slot in place of the count: the edge weight is read from it below
              c.cnt = (unsigned)sl;
              return c;
            };
            Cand best; best.valid = 0; best.w = 0; best.tok = 0; best.S = 0; best.cnt = 0;
            for (int x = lane; x < nn; x += 32) {
              const Cand c = get(x);
              if (c.valid && (!best.valid || ranks_before(c.w, c.tok, best.w, best.tok))) best = c;
            }
            best = warp_best(best);
            if (lane == 0 && best.valid &&
                (!sh_best_valid || ranks_before(best.w, best.tok, sh_best_w, sh_best_tok))) {
              const int sl = (int)best.cnt;
              sh_best_valid = 1; sh_best_w = best.w; sh_best_tok = best.tok;
              sh_best_ew = sm.n_ccur[sl] ? eq5_weight(s.alpha, sm.n_Scur[sl], sm.n_ccur[sl]) : 0.0;
            }
          }
          if (EXPORT && warp == 1) {
            const int nrun = sh_nnode_run;
            auto get = [&](int x) {
              Cand c; c.valid = 1;
              if (x < nn) { const int sl = sm.n_touch[x]; c.tok = sm.n_key[sl]; c.S = sm.n_Sall[sl]; c.cnt = sm.n_call[sl]; }
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
            for (int b = warp - 2; b < nkept; b += kWarps - 2) {
              const int nrun = sm.r_nedge[b];
              int deg = 0;
              for (int x = lane; x < ne; x += 32) deg += sm.e_key[sm.e_touch[x]] % MAXB == b;
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) deg += __shfl_xor_sync(0xffffffffu, deg, o);
              auto get = [&](int x) {
                Cand c;
                if (x < ne) {
                  const int sl = sm.e_touch[x];
                  c.valid = sm.e_key[sl] % MAXB == b; c.tok = sm.e_key[sl] / MAXB; c.S = sm.e_S[sl]; c.cnt = sm.e_c[sl];
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
          sm.n_key[sl] = -1; sm.n_Sall[sl] = 0; sm.n_Scur[sl] = 0; sm.n_call[sl] = 0; sm.n_ccur[sl] = 0;
        }
        if (EXPORT)
          for (int x = tid; x < ne; x += blockDim.x) {
            const int sl = sm.e_touch[x];
            sm.e_key[sl] = -1; sm.e_S[sl] = 0; sm.e_c[sl] = 0;
          }
        __syncthreads();
        if (tid == 0) { sh_nn = 0; sh_ne = 0; sh_overflow = 0; }
        __syncthreads();
      }
      if (overflowed && npart < npart_max) {
        npart = min(npart * 2, npart_max);          // redo the layer with smaller residue classes
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

}  // namespace

cudaError_t dag_kernel_setup() {
  cudaError_t e = cudaFuncSetAttribute(dag_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)dag_smem_bytes<false>());
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(dag_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)dag_smem_bytes<true>());
}

cudaError_t launch_dag(const Dev& s, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                       float* draft_edge_w, cudaStream_t stream) {
  if (s.B > 0)
    dag_kernel<true><<<s.P, kDagThreads, dag_smem_bytes<true>(), stream>>>(s, draft_tok, draft_len, draft_score,
                                                                          draft_edge_w);
  else
    dag_kernel<false><<<s.P, kDagThreads, dag_smem_bytes<false>(), stream>>>(s, draft_tok, draft_len, draft_score,
                                                                            draft_edge_w);
  return cudaGetLastError();
}

}  // namespace sdms
