// Hand-over of a query with many matches to the device-wide aggregation pass (dag_wide.cu).
#pragma once
#include "sdms_dev.cuh"

namespace sdms {

// log2 of the slots of one layer's node table: a power of two above 5/2 of the matches.  A layer in which
// every candidate is a node of its own fills at most 40 % of it: the whole grid waits for the unluckiest
// lane of a pass, that is for the fullest eight-key sector of all tables (every claimer that meets
// somebody else's token there pays another round trip), and how full that sector is grows quickly with the fill.
__device__ __forceinline__ int wide_lcap(int M) {
  int l = 6;
  while ((1ll << l) < (5ll * M) / 2 + 1) ++l;
  return l;
}

// The same for the one-CTA-per-path beam kernel, which nobody waits for: above 5/4 of the matches.
__device__ __forceinline__ int beam_lcap(int M) {
  int l = 6;
  while ((1ll << l) < (long long)M + (M >> 2) + 1) ++l;
  return l;
}

// Called by every thread of the query's CTA.  Reserves table slots for all D layers and enters the
// query in the list the wide pass works through; false (for all threads) if the pass is not in use,
// the list is full or the slots have run out - the caller then aggregates the query itself.
__device__ __forceinline__ bool wide_register(const Dev& s, int i, int M) {
  __shared__ int sh_wide_q;
  if (s.w_grid == 0 || M > kWideMaxMatches) return false;
  if (threadIdx.x == 0) {
    int q = -1;
    const int lcap = wide_lcap(M);
    const unsigned long long need = (unsigned long long)s.D << lcap;
    const unsigned long long first = atomicAdd(&s.w_ctl[1], need);
    if (first + need <= s.w_slots) {
      const unsigned long long n = atomicAdd(&s.w_ctl[0], 1ull);
      if (n < (unsigned long long)kMaxWide) {
        q = (int)n;
        s.w_desc[q] = make_int4(i, M, lcap, (int)(unsigned)first);
        atomicMax(&s.w_ctl[3], first + need);
      }
    }
    sh_wide_q = q;
  }
  __syncthreads();
  const int q = sh_wide_q;
  if (q >= 0 && threadIdx.x < SDMS_MAX_DRAFT) {
    s.w_pred[(size_t)q * SDMS_MAX_DRAFT + threadIdx.x] = WidePred{0ull, 0ull};
    s.w_edge[(size_t)q * SDMS_MAX_DRAFT + threadIdx.x] = 0ull;
  }
  return q >= 0;
}


typedef unsigned long long u64;
constexpr unsigned FULL = 0xffffffffu;
constexpr int kWideThreads = 512;
constexpr int kWideChunk = 128;                      // matches per unit of work: thread t owns match t % 128 ...
constexpr int kLayerWays = kWideThreads / kWideChunk;  // ... and the layers d = t / 128 + 1, + 5, + 9, ...
constexpr int kMaxRounds = 4;                          // layers of a thread that are in flight together (16 layers of the query)
static_assert(kMaxRounds * 8 <= 32, "eight slot bits per layer in flight fit one word");

// Sum of p over the lanes of this lane's group (`group` from __match_any_sync).  The same loop in every
// lane, over the lanes that share their group with somebody (`shared`: whole groups only); a lane that is
// not among them keeps its own p.  One shuffle per visited lane: the shuffle pipe is what this costs.
__device__ __forceinline__ u64 group_sum(unsigned group, unsigned shared, unsigned p) {
  u64 sum = (shared >> (threadIdx.x & 31) & 1u) ? 0ull : (u64)p;
  for (unsigned rem = shared; rem; rem &= rem - 1) {
    const int src = __ffs(rem) - 1;
    const unsigned q = __shfl_sync(FULL, p, src);
    if (group >> src & 1u) sum += q;
  }
  return sum;
}

// Node sums of one unit: the matches list[m0 .. m0 + 128) of a query with M matches, all layers, into the
// query's tables (first slot `base`, 2^lcap slots per layer).  Called by all kWideThreads threads of a
// CTA.  The lanes of a warp hold 32 matches at the same layer; lanes whose followers are the same token
// form a group and the group's leader claims the node's slot and sends one add for all of them.
// Every item's slot (-1: the candidate has ended) is noted in w_item[base + (d - 1) * M + m].
// A thread's layers are d_first + 4 r; with r_lo / r_hi the call takes only the rounds r_lo <= r < r_hi of them (a unit
// split by layers: more, shorter units when there are fewer units than CTAs).
__device__ __forceinline__ void wide_insert_unit(const Dev& s, const int32_t* list, unsigned base, int lcap, int M, int m0,
                                                 int r_lo = 0, int r_hi = SDMS_MAX_DRAFT) {
  const int tid = threadIdx.x, lane = tid & 31;
  const int D = s.D;
  const int ml = tid & (kWideChunk - 1), d_first = tid / kWideChunk + 1;   // d_first is the same in all lanes of a warp
  const int nm = min(kWideChunk, M - m0);
    const unsigned mask = (1u << lcap) - 1u;
    int* const item = s.w_item + base + m0 + ml;      // + (d - 1) * M: the item's slot, layer by layer
    int gpos = 0, n_m = 0;
    if (ml < nm) {
      gpos = list[m0 + ml];
      const int j = path_of(s, gpos);
      n_m = min(D, __ldg(s.len + j) - 1 - (gpos - j * s.L));
    }
  for (int r0 = r_lo; r0 < r_hi && d_first + r0 * kLayerWays <= D; r0 += kMaxRounds) {     // the same trip count for the whole warp
    const int d_base = d_first + r0 * kLayerWays;
    const int d_end = min(D, d_first + (r_hi - 1) * kLayerWays);    // the last layer of this thread that belongs to the unit
    int v[kMaxRounds];
    unsigned p[kMaxRounds];
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {            // every follower this thread needs is asked for before the first is used
      const int d = d_base + r * kLayerWays;
      v[r] = -1; p[r] = 0u;
      if (d <= n_m && d <= d_end) { v[r] = __ldg(s.tok + gpos + d); p[r] = (unsigned)__ldg(s.pq + gpos + d); }
    }
    // the key sector and the slot every follower hashes to are asked for now: when the rounds below get to
    // them (one after the other, the lanes of a warp in step) they are on their way from memory
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
      const int d = d_base + r * kLayerWays;
      if (v[r] >= 0) {
        const size_t at = base + ((size_t)(d - 1) << lcap) + (((unsigned)v[r] * 2654435761u) >> (32 - lcap));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(s.w_key + at));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(s.w_tab + at));
      }
    }
    // Who speaks for which node, for all of the thread's layers at once; then the leaders' probe
    // sequences of those layers run side by side (a round trip to L2 costs the same for one request
    // as for four), and last the slots go back to the groups.
    int leader[kMaxRounds], sv[kMaxRounds];
    u64 add[kMaxRounds];
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
      const int d = d_base + r * kLayerWays;
      leader[r] = 0; sv[r] = -1; add[r] = 0ull;
      if (d > d_end) continue;                          // the same for the whole warp
      const unsigned group = __match_any_sync(FULL, v[r]);          // lanes whose items are the same node
      leader[r] = __ffs(group) - 1;
      const unsigned shared = __ballot_sync(FULL, v[r] >= 0 && (group & (group - 1)) != 0u);
      add[r] = ((u64)__popc(group) << kWideSumShift) | group_sum(group, shared, p[r]);
    }
    // Open addressing by sectors of eight keys (one round trip each).  A token's home sector is given by its hash; it
    // may sit in any of the sector's eight slots, and only a sector without a free slot sends it on to the next one.
    // Within a sector every claimer of a token tries the free slots in the same order (from the hash's low bits on,
    // wrapping), so two claimers of one token end up at one slot: the slots before it in that order were taken by
    // other tokens when the first of them passed, and slots are never given back during a pass.
    unsigned h[kMaxRounds];
    unsigned todo = 0;                                  // layers whose slot this thread still has to find
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
      const int d = d_base + r * kLayerWays;
      h[r] = ((unsigned)v[r] * 2654435761u) >> (32 - lcap);
      if (d <= d_end && v[r] >= 0 && lane == leader[r]) todo |= 1u << r;
    }
    uint4 ka[kMaxRounds], kb[kMaxRounds];                // the sector of keys each sequence is looking at
    unsigned fresh = 0;                                 // layers whose sector is in ka / kb
    unsigned taken = 0;                                 // eight bits per layer: slots of that sector a failed claim has shown to be somebody else's
    for (unsigned step = 0; step <= 2u * mask + 16u && todo; ++step) {   // every step finds the slot, rules one out or leaves a full sector
#pragma unroll
      for (int r = 0; r < kMaxRounds; ++r) {
        if (!(todo >> r & 1u) || (fresh >> r & 1u)) continue;
        const uint32_t* keys = s.w_key + base + ((size_t)(d_base + r * kLayerWays - 1) << lcap) + (h[r] & ~7u);
        ka[r] = __ldcg(reinterpret_cast<const uint4*>(keys));
        kb[r] = __ldcg(reinterpret_cast<const uint4*>(keys + 4));
      }
      fresh |= todo;
      int at[kMaxRounds];                               // the slot that holds the token, else the first free one in the token's order
      uint32_t seen[kMaxRounds];
#pragma unroll
      for (int r = 0; r < kMaxRounds; ++r) {
        at[r] = -1; seen[r] = 0u;
        if (!(todo >> r & 1u)) continue;
        const uint32_t want = (uint32_t)v[r] + 1u;
        const uint32_t kk[8] = {ka[r].x, ka[r].y, ka[r].z, ka[r].w, kb[r].x, kb[r].y, kb[r].z, kb[r].w};
        unsigned hit = 0u, vacant = 0u;
#pragma unroll
        for (int x = 0; x < 8; ++x) { hit |= (unsigned)(kk[x] == want) << x; vacant |= (unsigned)(kk[x] == 0u) << x; }
        vacant &= ~(taken >> (8 * r));
        const unsigned start = h[r] & 7u;
        if (hit) { at[r] = __ffs(hit) - 1; seen[r] = want; }
        else if (vacant) { at[r] = (int)((start + __ffs(((vacant | (vacant << 8)) >> start) & 0xffu) - 1) & 7u); }
      }
      unsigned claims = 0;
#pragma unroll
      for (int r = 0; r < kMaxRounds; ++r) {             // the claims of all layers go out together ...
        if (!(todo >> r & 1u) || at[r] < 0 || seen[r] != 0u) continue;
        uint32_t* keys = s.w_key + base + ((size_t)(d_base + r * kLayerWays - 1) << lcap) + (h[r] & ~7u);
        seen[r] = atomicCAS(&keys[at[r]], 0u, (uint32_t)v[r] + 1u);
        claims |= 1u << r;
      }
#pragma unroll
      for (int r = 0; r < kMaxRounds; ++r) {             // ... and with them a new look at their sectors: should a claim fail (the
        if (!(claims >> r & 1u)) continue;               // sector was read before its other claimers arrived), the next one knows better
        const uint32_t* keys = s.w_key + base + ((size_t)(d_base + r * kLayerWays - 1) << lcap) + (h[r] & ~7u);
        ka[r] = __ldcg(reinterpret_cast<const uint4*>(keys));
        kb[r] = __ldcg(reinterpret_cast<const uint4*>(keys + 4));
      }
#pragma unroll
      for (int r = 0; r < kMaxRounds; ++r) {
        if (!(claims >> r & 1u) || seen[r] != 0u) continue;
        seen[r] = (uint32_t)v[r] + 1u;
        s.w_tab[base + ((size_t)(d_base + r * kLayerWays - 1) << lcap) + (h[r] & ~7u) + at[r]].tok1 = seen[r];
      }
#pragma unroll
      for (int r = 0; r < kMaxRounds; ++r) {
        if (!(todo >> r & 1u)) continue;
        if (at[r] < 0) {                                  // no room in this sector: on to the next, same order within it
          h[r] = (((h[r] & ~7u) + 8u) & mask) | (h[r] & 7u);
          fresh &= ~(1u << r); taken &= ~(0xffu << (8 * r));
          continue;
        }
        if (seen[r] == (uint32_t)v[r] + 1u) { sv[r] = (int)((h[r] & ~7u) + at[r]); todo &= ~(1u << r); continue; }
        taken |= 1u << (8 * r + at[r]);                   // somebody else's token got there first: the next free slot of the (stale) sector
      }
    }
    if (todo) atomicOr(s.status, SDMS_STATUS_INDEX_FULL);             // more nodes than slots: cannot happen
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
      const int d = d_base + r * kLayerWays;
      if (d > d_end) continue;
      if (sv[r] >= 0) atomicAdd(&s.w_tab[base + ((size_t)(d - 1) << lcap) + sv[r]].sum, add[r]);
      const int mine = __shfl_sync(FULL, sv[r], leader[r]);
      if (ml < nm) item[(size_t)(d - 1) * M] = v[r] >= 0 ? mine : -1;
    }
  }
}

}  // namespace sdms
