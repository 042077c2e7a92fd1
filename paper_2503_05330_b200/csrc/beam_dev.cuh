// The B best paths of a query's pool (several drafts per path), by one CTA over node tables in global
// memory.  Value of a path: the sum of its nodes' Eq. 5 in-weights, added from its end towards its
// start (the search-mode-2 value); only paths that run on to a leaf or to layer D count.
//
// Every node keeps its B best continuations, best first:
//   leaf (d, v):  [ w(d, v) ]
//   otherwise:    the B best of { w(d, v) + x : x a kept continuation of a successor v' },
// ordered by value (larger first), then v' (smaller first), then the rank of x in the list of v'.
// The layers are taken from the last to the first.  Rank r of a layer is found by two sweeps over the
// layer's (candidate, successor) items: every item offers the best of its successor's continuations
// that still comes strictly after the node's rank r - 1 entry (64-bit max on the value's bit pattern),
// then the items that hold exactly that value compete with (~v', rank) packed in 64 bits.  Equal
// offers from different items are the same entry, so duplicates do no harm.
#pragma once
#include "wide_dev.cuh"

namespace sdms {

constexpr u64 kBeamLeaf = 1ull;          // `next` of a continuation that ends at its node
struct BeamEnt { u64 value; u64 next; };  // value: bit pattern of the double; next: ~token << 32 | (7 - rank) << 24 | slot; 0 = no entry

__device__ __forceinline__ u64 beam_next(uint32_t tok, int rank, int slot) {
  return ((u64)(~tok) << 32) | ((u64)(7 - rank) << 24) | (u64)(unsigned)slot;
}
__device__ __forceinline__ bool beam_after(u64 v, u64 nx, const BeamEnt& prev) {   // (v, nx) comes strictly after prev
  return v < prev.value || (v == prev.value && nx < prev.next);
}

// One CTA (kWideThreads threads), query path i with M matches in `list`.  Needs D << lcap table slots
// starting at `base`, all zero (they are left zero).  Writes beam_tok [B][D], beam_len [B], beam_value [B]
// of the path.  `ent` = s.b_ent + base * stride.  With score0 / edge0 (each [D], either may be NULL; the
// caller asks with want0) the first beam also gets what a draft carries: the Eq. 5 in-weight of each of
// its nodes and the weight of each edge it takes.
__device__ __forceinline__ void beams_of_query(const Dev& s, int i, int M, const int32_t* list, unsigned base, int lcap, int B,
                               int32_t* beam_tok, int32_t* beam_len, float* beam_value, bool want0 = false,
                               float* score0 = nullptr, float* edge0 = nullptr) {
  __shared__ BeamEnt sh_root[SDMS_MAX_BEAMS];
  __shared__ int sh_bslot[SDMS_MAX_DRAFT];
  __shared__ u64 sh_bedge[SDMS_MAX_DRAFT];
  __shared__ int sh_blen;
  const int tid = threadIdx.x, D = s.D, stride = s.beam_stride;
  const unsigned cap = 1u << lcap;
  WideSlot* const tab = s.w_tab + base;
  BeamEnt* const ent = s.b_ent + (size_t)base * stride;
  const int* const item = s.w_item + base;           // [(d - 1) * M + m]
  for (int m0 = 0; m0 < M; m0 += kWideChunk) wide_insert_unit(s, list, base, lcap, M, m0);
  if (tid < SDMS_MAX_BEAMS) sh_root[tid] = BeamEnt{0ull, 0ull};
  __threadfence();
  __syncthreads();

  for (int d = D; d >= 0; --d) {
    // d >= 1: the lists of the nodes of layer d from those of layer d + 1; d = 0: the root's from layer 1
    if (d < D) {
      for (int r = 0; r < B; ++r) {
        for (int stage = 0; stage < 2; ++stage) {
          for (int m = tid; m < M; m += blockDim.x) {
            const int sv = __ldcg(item + (size_t)d * M + m);                 // the candidate's node at layer d + 1
            if (sv < 0) continue;
            BeamEnt* mine;                                                 // the list this item feeds
            double w_u = 0.0;
            if (d == 0) {
              mine = sh_root;
            } else {
              const int su = __ldcg(item + (size_t)(d - 1) * M + m);
              mine = ent + ((size_t)((d - 1) << lcap) + su) * stride;
              const u64 sum = __ldcg(&tab[((size_t)(d - 1) << lcap) + su].sum);
              w_u = eq5_weight(s.alpha, sum & ((1ull << kWideSumShift) - 1), (unsigned)(sum >> kWideSumShift));
            }
            BeamEnt prev{0ull, 0ull};
            if (r > 0) {
              prev = d == 0 ? sh_root[r - 1] : BeamEnt{__ldcg(&mine[r - 1].value), __ldcg(&mine[r - 1].next)};
              if (prev.next == 0ull) continue;                             // the node ran out of continuations before
            }
            const BeamEnt* theirs = ent + ((size_t)(d << lcap) + sv) * stride;
            const uint32_t tok = __ldcg(&tab[((size_t)d << lcap) + sv].tok1) - 1u;
            for (int j = 0; j < B; ++j) {                                  // best first: the first that qualifies is the offer
              const u64 nx = __ldcg(&theirs[j].next);
              if (nx == 0ull) break;
              const double x = __longlong_as_double((long long)__ldcg(&theirs[j].value));
              const u64 val = (u64)__double_as_longlong(d == 0 ? x : __dadd_rn(w_u, x));
              const u64 key = beam_next(tok, j, sv);
              if (r > 0 && !beam_after(val, key, prev)) continue;
              if (stage == 0) atomicMax(&mine[r].value, val);
              else if ((d == 0 ? mine[r].value : __ldcg(&mine[r].value)) == val) atomicMax(&mine[r].next, key);
              break;
            }
          }
          __threadfence();
          __syncthreads();
        }
      }
    }
    if (d >= 1) {
      // a node that nothing was offered to is a leaf: its only continuation is to stop
      for (unsigned x = tid; x < cap; x += blockDim.x) {
        const size_t sl = ((size_t)(d - 1) << lcap) + x;
        if (__ldcg(&s.w_key[base + sl]) == 0u) continue;
        BeamEnt* mine = ent + sl * stride;
        if (__ldcg(&mine[0].next) != 0ull) continue;
        const u64 sum = __ldcg(&tab[sl].sum);
        mine[0].value = (u64)__double_as_longlong(eq5_weight(s.alpha, sum & ((1ull << kWideSumShift) - 1), (unsigned)(sum >> kWideSumShift)));
        mine[0].next = kBeamLeaf;
      }
      __threadfence();
      __syncthreads();
    }
  }

  // the beams: follow the entries from the root
  if (tid < B) {
    BeamEnt e = sh_root[tid];
    int len = 0;
    if (e.next != 0ull) beam_value[tid] = (float)__longlong_as_double((long long)e.value);
    else beam_value[tid] = 0.0f;
    for (int d = 1; d <= D && e.next != 0ull && e.next != kBeamLeaf; ++d) {
      const uint32_t tok = ~(uint32_t)(e.next >> 32);
      const int rank = 7 - (int)((e.next >> 24) & 7u), slot = (int)(e.next & 0xffffffu);
      beam_tok[tid * D + len++] = (int32_t)tok;
      const BeamEnt* at = ent + ((size_t)((d - 1) << lcap) + slot) * stride + rank;
      e = BeamEnt{__ldcg(&at->value), __ldcg(&at->next)};
    }
    for (int d = len; d < D; ++d) beam_tok[tid * D + d] = -1;
    beam_len[tid] = len;
  }
  if (want0) {
    // the first beam once more, slot by slot; then the probabilities of the items on its edges
    if (tid < SDMS_MAX_DRAFT) sh_bedge[tid] = 0ull;
    if (tid == 0) {
      BeamEnt e = sh_root[0];
      int len = 0;
      for (int d = 1; d <= D && e.next != 0ull && e.next != kBeamLeaf; ++d) {
        const int rank = 7 - (int)((e.next >> 24) & 7u), slot = (int)(e.next & 0xffffffu);
        sh_bslot[len++] = slot;
        if (score0) {
          const u64 sum = __ldcg(&tab[((size_t)(d - 1) << lcap) + slot].sum);
          score0[d - 1] = (float)eq5_weight(s.alpha, sum & ((1ull << kWideSumShift) - 1), (unsigned)(sum >> kWideSumShift));
        }
        const BeamEnt* at = ent + ((size_t)((d - 1) << lcap) + slot) * stride + rank;
        e = BeamEnt{__ldcg(&at->value), __ldcg(&at->next)};
      }
      sh_blen = len;
    }
    __syncthreads();
    const int len = sh_blen;
    if (edge0) {
      for (int d = 1; d <= len; ++d) {
        for (int m0 = 0; m0 < M; m0 += blockDim.x) {             // whole warps: the lanes add up together
          const int m = m0 + tid;
          bool on = false;
          if (m < M) on = __ldcg(item + (size_t)(d - 1) * M + m) == sh_bslot[d - 1] &&
                          (d == 1 || __ldcg(item + (size_t)(d - 2) * M + m) == sh_bslot[d - 2]);
          const unsigned group = __ballot_sync(FULL, on);
          if (group == 0u) continue;
          const u64 sum = group_sum(group, group, on ? (unsigned)__ldg(s.pq + list[m] + d) : 0u);
          if ((tid & 31) == __ffs(group) - 1) atomicAdd(&sh_bedge[d - 1], ((u64)__popc(group) << kWideSumShift) | sum);
        }
      }
      __syncthreads();
      if (tid < len) {
        const u64 sum = sh_bedge[tid];
        edge0[tid] = (float)eq5_weight(s.alpha, sum & ((1ull << kWideSumShift) - 1), (unsigned)(sum >> kWideSumShift));
      }
    }
  }
  __syncthreads();
  // leave the tables as they were found
  uint4* z = reinterpret_cast<uint4*>(tab);
  for (size_t x = tid; x < ((size_t)D << lcap) * 2; x += blockDim.x) z[x] = make_uint4(0u, 0u, 0u, 0u);
  uint4* zk = reinterpret_cast<uint4*>(s.w_key + base);
  for (size_t x = tid; x < ((size_t)D << lcap) / 4; x += blockDim.x) zk[x] = make_uint4(0u, 0u, 0u, 0u);
  uint4* ze = reinterpret_cast<uint4*>(ent);
  for (size_t x = tid; x < ((size_t)D << lcap) * stride; x += blockDim.x) ze[x] = make_uint4(0u, 0u, 0u, 0u);
}

}  // namespace sdms
