// Follower gather, DAG aggregation (Eq. 5) and the greedy walk for queries with many matches, spread
// over the whole device.
//
// One CTA aggregates a query of a few dozen matches in its own shared memory (dag.cu).  A query with
// hundreds or tens of thousands of matches keeps one SM busy for as long while the others idle, so
// dag_kernel hands such queries over (wide_register) and this pass works through all of them at
// once: every (match, layer) pair is one item, 128 matches are one unit of work (split by layers into
// two or four units when that still leaves CTAs without one), and the units of all queries are dealt
// out to a grid that covers the device.  Each query owns, for every layer, a node
// table in global memory (open addressing, one 32-byte slot per node and the keys apart, eight to a
// sector; all of it zero when the pass begins and again when it ends).  Sums are integers and every choice has a tie rule, so the atomics'
// order cannot show in a result.
//
// Within a unit a thread owns one match and every fourth layer, so the lanes of a warp hold 32
// matches at the SAME layer: lanes whose items fall on the same node (or the same edge) are found
// with __match_any_sync and send ONE atomic for the group.  Popular n-grams are followed by the same
// tokens over and over; without this thousands of adds queue up on one address in L2.
//
//   pass A  item (m, d): the group's leader claims the slot of the follower token v in the table of
//           layer d and adds the group's probabilities and count (one 64-bit add).  Every item notes
//           its slot.
//   pass B  every node's Eq. 5 weight is final: an item offers it to the node of the token before it
//           (64-bit max on the weight's bit pattern; layer 1 offers to the root, and under the
//           layer-wise rule every layer to a record of its own).
//   pass C  items whose node carries exactly that largest weight compete with their token: the
//           smallest wins (64-bit max of ~token), and its slot travels with it.
//   pass D  the walk is one dependent load per layer; each unit walks its own query (no barrier
//           between walk and use) and then adds the probabilities of the items on the edges the draft
//           takes.
//   pass E  edge weights out; the slots that were used are zeroed again.
// Between the passes all CTAs meet at a grid barrier (bounded wait; the launch is cooperative, so all
// CTAs are resident).
#include <cstddef>
#include "sdms_internal.h"
#include "wide_dev.cuh"

namespace sdms {

namespace {

constexpr long long kBarrierCycles = 200000000LL;    // about a tenth of a second (the pass takes 0.1-0.3 ms): a barrier that takes that long has failed
constexpr u64 kSumMask = (1ull << kWideSumShift) - 1;
constexpr int kRivalsFrom = 4096;                    // matches of a query from which offers to one node are reduced in the warp first
static_assert(offsetof(WideSlot, succ) == offsetof(WideSlot, succ_w) + 8 && offsetof(WidePred, succ) == offsetof(WidePred, succ_w) + 8,
              "the best successor sits right behind its weight");

__device__ __forceinline__ u64 ld_u64(const u64* p) { return __ldcg(p); }
__device__ __forceinline__ uint32_t ld_u32(const uint32_t* p) { return __ldcg(p); }

// All CTAs of the grid arrive; returns false (in every thread of the CTA) if the others did not show
// up in time.  Arrivals are spread over kWideBarrierWays counters in lines of their own (hundreds of
// atomics on one address take microseconds); one thread per counter waits for it.
__device__ __forceinline__ bool wait_for_count(const u64* ctr, u64 target, long long cycles) {
  const long long t0 = clock64();
  while (ld_u64(ctr) < target) {
    if (clock64() - t0 > cycles) return false;
    __nanosleep(32);
  }
  return true;
}

__device__ bool grid_barrier(const Dev& s, unsigned phase) {
  __syncthreads();
  int ok = 1;
  const int t = threadIdx.x;
  if (t < kWideBarrierWays) {
    u64* ctr = s.w_ctl + kWideBarrierAt + t * kWideBarrierStride;
    if (t == (int)(blockIdx.x & (kWideBarrierWays - 1))) { __threadfence(); atomicAdd(ctr, 1ull); }
    const u64 target = (u64)((gridDim.x + kWideBarrierWays - 1 - t) / kWideBarrierWays) * phase;
    ok = wait_for_count(ctr, target, kBarrierCycles);
    __threadfence();
  }
  return __syncthreads_and(ok) != 0;
}

// sdms_debug_wait_timeout: the bounded wait of the grid barrier on a count that nobody raises.
__global__ void wait_timeout_kernel(Dev s, long long cycles) {
  if (threadIdx.x == 0 && !wait_for_count(s.b_ctl + 1, ~0ull, cycles)) atomicOr(s.status, SDMS_STATUS_TIMEOUT);
}

__device__ __forceinline__ double weight_of(const Dev& s, u64 sum) {
  return eq5_weight(s.alpha, sum & kSumMask, (unsigned)(sum >> kWideSumShift));
}

__global__ void __launch_bounds__(kWideThreads, 1)
dag_wide_kernel(Dev s, int32_t* __restrict__ draft_tok, int32_t* __restrict__ draft_len,
                float* __restrict__ draft_score, float* __restrict__ draft_edge_w) {
  grid_wait();                                       // scheduled while dag_kernel drains; its list is complete from here on
  const u64 registered = ld_u64(&s.w_ctl[0]);
  if (registered == 0) return;                       // the same for every CTA: nobody waits for anybody
  const int nq = (int)(registered < (u64)kMaxWide ? registered : (u64)kMaxWide);
  __shared__ int4 sh_desc[kMaxWide];
  __shared__ int sh_cbase[kMaxWide + 1];
  __shared__ int sh_warp[kWideThreads / 32];
  __shared__ int sh_dslot[SDMS_MAX_DRAFT];
  __shared__ int sh_emitted;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = s.D;
  const int ml = tid & (kWideChunk - 1), d_first = tid / kWideChunk + 1;   // d_first is the same in all lanes of a warp

  // the list of queries and, by a prefix sum, the first unit of each
  {
    static_assert(kMaxWide == 2 * kWideThreads, "two list entries per thread");
    int c[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int q = 2 * tid + r;
      c[r] = 0;
      if (q < nq) { const int4 de = __ldcg(&s.w_desc[q]); sh_desc[q] = de; c[r] = (de.y + kWideChunk - 1) / kWideChunk; }
    }
    int x = c[0] + c[1];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(FULL, x, o); if (lane >= o) x += y; }
    if (lane == 31) sh_warp[warp] = x;
    __syncthreads();
    if (warp == 0) {
      int w = lane < kWideThreads / 32 ? sh_warp[lane] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(FULL, w, o); if (lane >= o) w += y; }
      if (lane < kWideThreads / 32) sh_warp[lane] = w;
    }
    __syncthreads();
    const int before = (warp ? sh_warp[warp - 1] : 0) + x - c[0] - c[1];
    if (2 * tid < nq) sh_cbase[2 * tid] = before;
    if (2 * tid + 1 < nq) sh_cbase[2 * tid + 1] = before + c[0];
    if (tid == kWideThreads - 1) sh_cbase[nq] = before + c[0] + c[1];
    __syncthreads();
  }
  const int chunks = sh_cbase[nq];
  // With fewer chunks than CTAs a chunk is split by layers as well: a thread's rounds (its layers d_first + 4 r) go to
  // `split` units that run on different SMs.
  const int rounds_all = (D + kLayerWays - 1) / kLayerWays;
  int split = 1;
  while (split * 2 <= rounds_all && chunks * split * 2 <= (int)gridDim.x) split *= 2;   // never two units for a CTA because of it: each unit walks the draft again
  const int rounds_per = (rounds_all + split - 1) / split;
  const int units = chunks * split;

  // unit c belongs to the last query whose first unit is not after c
  auto query_of = [&](int c) {
    int lo = 0, hi = nq;                              // sh_cbase[lo] <= c < sh_cbase[hi]
    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (sh_cbase[mid] <= c) lo = mid; else hi = mid; }
    return lo;
  };

  // ---- pass A: node sums -------------------------------------------------------------------------
  for (int u = blockIdx.x; u < units; u += gridDim.x) {
    const int c = u / split, r_lo = (u - c * split) * rounds_per;
    const int q = query_of(c);
    const int4 de = sh_desc[q];
    const int i = de.x, M = de.y, lcap = de.z;
    const unsigned base = (unsigned)de.w;
    const int m0 = (c - sh_cbase[q]) * kWideChunk;
    wide_insert_unit(s, s.matches + s.q_off[i], base, lcap, M, m0, r_lo, r_lo + rounds_per);
  }
  if (!grid_barrier(s, 1)) { if (tid == 0) atomicOr(s.status, SDMS_STATUS_TIMEOUT); return; }

  // ---- passes B and C: the best successor of every node ------------------------------------------
  for (int pass = 0; pass < 2; ++pass) {
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
      const int c = u / split, r_lo = (u - c * split) * rounds_per;
      const int q = query_of(c);
      const int4 de = sh_desc[q];
      const int M = de.y, lcap = de.z;
      const unsigned base = (unsigned)de.w;
      const int m0 = (c - sh_cbase[q]) * kWideChunk, nm = min(kWideChunk, M - m0);
      const int* const item = s.w_item + base + m0 + ml;
      const int d_end = min(D, d_first + (r_lo + rounds_per - 1) * kLayerWays);
      // a thread's layers four at a time: the loads of all four are on their way before the first is used
#pragma unroll 1
      for (int d0 = d_first + r_lo * kLayerWays; d0 <= d_end; d0 += kMaxRounds * kLayerWays) {
        int sv[kMaxRounds], su[kMaxRounds];
#pragma unroll
        for (int r = 0; r < kMaxRounds; ++r) {
          const int d = d0 + r * kLayerWays;
          sv[r] = -1; su[r] = -1;
          if (d <= d_end && ml < nm) {
            sv[r] = item[(size_t)(d - 1) * M];
            if (d > 1 && s.mode != 1) su[r] = item[(size_t)(d - 2) * M];
          }
        }
        unsigned lead = 0;                             // layers in which this lane speaks for its edge
        u64 sum[kMaxRounds];
        u64* best_w[kMaxRounds];
#pragma unroll
        for (int r = 0; r < kMaxRounds; ++r) {
          const int d = d0 + r * kLayerWays;
          sum[r] = 0ull; best_w[r] = nullptr;
          if (d > d_end) continue;                     // the same for the whole warp
          const bool on = sv[r] >= 0 && (d == 1 || s.mode == 1 || su[r] >= 0);
          // items on the same edge (same node, under the layer-wise rule) bring the same offer: one lane speaks for them
          const u64 edge = on ? ((u64)(unsigned)su[r] << 32) | (u64)(unsigned)sv[r] : ~(u64)lane;
          const unsigned group = __match_any_sync(FULL, edge);
          if (!on || lane != __ffs(group) - 1) continue;
          lead |= 1u << r;
          sum[r] = ld_u64(&s.w_tab[base + ((size_t)(d - 1) << lcap) + sv[r]].sum);
          best_w[r] = d == 1 || s.mode == 1 ? &s.w_pred[(size_t)q * SDMS_MAX_DRAFT + (d - 1)].succ_w
                                            : &s.w_tab[base + ((size_t)(d - 2) << lcap) + su[r]].succ_w;
        }
        if (pass == 0) {
#pragma unroll
          for (int r = 0; r < kMaxRounds; ++r) {
            if (d0 + r * kLayerWays > d_end) continue;   // the same for the whole warp
            // Of the lanes that offer to the same node only the one with the largest weight needs to: a popular
            // n-gram's root or first nodes would otherwise take thousands of atomics on one address.
            const bool on = lead >> r & 1u;
            const u64 w = on ? (u64)__double_as_longlong(weight_of(s, sum[r])) : 0ull;
            if (M < kRivalsFrom) { if (on) atomicMax(best_w[r], w); continue; }   // few offers per node: not worth the shuffles
            const unsigned rivals = __match_any_sync(FULL, on ? (u64)(uintptr_t)best_w[r] : (u64)lane);
            u64 top = w;
            for (unsigned rem = __ballot_sync(FULL, on && (rivals & (rivals - 1)) != 0u); rem; rem &= rem - 1) {
              const int src = __ffs(rem) - 1;
              const u64 other = __shfl_sync(FULL, w, src);
              if ((rivals >> src & 1u) && other > top) top = other;
            }
            if (on && w == top) atomicMax(best_w[r], w);
          }
        } else {
          u64 cur[kMaxRounds];
          uint32_t tok1[kMaxRounds];
#pragma unroll
          for (int r = 0; r < kMaxRounds; ++r) {
            cur[r] = 0ull; tok1[r] = 0u;
            if (!(lead >> r & 1u)) continue;
            cur[r] = ld_u64(best_w[r]);
            tok1[r] = ld_u32(&s.w_tab[base + ((size_t)(d0 + r * kLayerWays - 1) << lcap) + sv[r]].tok1);
          }
#pragma unroll
          for (int r = 0; r < kMaxRounds; ++r) {
            if (!(lead >> r & 1u) || cur[r] != (u64)__double_as_longlong(weight_of(s, sum[r]))) continue;
            atomicMax(best_w[r] + 1, ((u64)(~(tok1[r] - 1u)) << 32) | (u64)(unsigned)sv[r]);   // succ sits behind succ_w
          }
        }
      }
    }
    if (!grid_barrier(s, 2 + pass)) { if (tid == 0) atomicOr(s.status, SDMS_STATUS_TIMEOUT); return; }
  }

  // ---- pass D: walk, then the sums of the edges taken ---------------------------------------------
  for (int u = blockIdx.x; u < units; u += gridDim.x) {
    const int c = u / split, r_lo = (u - c * split) * rounds_per;
    const int q = query_of(c);
    const int4 de = sh_desc[q];
    const int i = de.x, M = de.y, lcap = de.z;
    const unsigned base = (unsigned)de.w;
    const int m0 = (c - sh_cbase[q]) * kWideChunk, nm = min(kWideChunk, M - m0);
    // what the edge sums below need of this thread's first four layers is asked for now: it arrives while
    // thread 0 walks (a dependent load per layer)
    const int* const item = s.w_item + base + m0 + ml;
    const int gpos = ml < nm ? s.matches[(size_t)s.q_off[i] + m0 + ml] : 0;
    const int d_lo = d_first + r_lo * kLayerWays, d_hi = min(D, d_first + (r_lo + rounds_per - 1) * kLayerWays);
    int it1[kMaxRounds], it0[kMaxRounds];
    unsigned pv[kMaxRounds];
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
      const int d = d_lo + r * kLayerWays;
      it1[r] = -1; it0[r] = -1; pv[r] = 0u;
      if (ml < nm && d <= d_hi) {
        it1[r] = item[(size_t)(d - 1) * M];
        if (d > 1) it0[r] = item[(size_t)(d - 2) * M];
      }
    }
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r)
      if (it1[r] >= 0) pv[r] = (unsigned)__ldg(s.pq + gpos + d_lo + r * kLayerWays);    // the item exists, so its follower does
    if (tid == 0) {
      const bool writer = m0 == 0 && r_lo == 0;       // the query's first unit writes the draft out
      const WidePred* pr = s.w_pred + (size_t)q * SDMS_MAX_DRAFT;
      u64 next = ld_u64(&pr[0].succ);
      int emitted = 0;
      for (int d = 1; d <= D; ++d) {
        if (s.mode == 1) next = ld_u64(&pr[d - 1].succ);
        if (next == 0ull) break;
        const int slot = (int)(unsigned)next;
        const WideSlot* node = s.w_tab + base + ((size_t)(d - 1) << lcap) + slot;
        sh_dslot[d - 1] = slot;
        if (writer) {
          draft_tok[(size_t)i * D + d - 1] = (int32_t)~(uint32_t)(next >> 32);
          if (draft_score) draft_score[(size_t)i * D + d - 1] = (float)weight_of(s, ld_u64(&node->sum));
        }
        ++emitted;
        if (s.mode != 1) next = ld_u64(&node->succ);
      }
      if (writer) draft_len[i] = emitted;
      sh_emitted = emitted;
    }
    __syncthreads();
    const int emitted = sh_emitted;
    const int d_end = min(emitted, d_hi);
#pragma unroll 1
    for (int d0 = d_lo; d0 <= d_end; d0 += kMaxRounds * kLayerWays) {
      if (d0 != d_lo) {                                 // more than four layers per thread (D > 16, unit not split): the next four
#pragma unroll
        for (int r = 0; r < kMaxRounds; ++r) {
          const int d = d0 + r * kLayerWays;
          it1[r] = -1; it0[r] = -1; pv[r] = 0u;
          if (ml < nm && d <= d_end) {
            it1[r] = item[(size_t)(d - 1) * M];
            it0[r] = item[(size_t)(d - 2) * M];
            if (it1[r] >= 0) pv[r] = (unsigned)__ldg(s.pq + gpos + d);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kMaxRounds; ++r) {
        const int d = d0 + r * kLayerWays;
        if (d > d_end) continue;                        // the same for the whole warp
        const bool on = it1[r] >= 0 && it1[r] == sh_dslot[d - 1] && (d == 1 || it0[r] == sh_dslot[d - 2]);
        const unsigned group = __ballot_sync(FULL, on);
        if (group == 0u) continue;
        const u64 sum = group_sum(group, group, on ? pv[r] : 0u);
        if (lane == __ffs(group) - 1)
          atomicAdd(&s.w_edge[(size_t)q * SDMS_MAX_DRAFT + d - 1], ((u64)__popc(group) << kWideSumShift) | sum);
      }
    }
    __syncthreads();
  }
  if (!grid_barrier(s, 4)) { if (tid == 0) atomicOr(s.status, SDMS_STATUS_TIMEOUT); return; }

  // ---- pass E: edge weights; leave the tables empty ------------------------------------------------
  if (draft_edge_w)
    for (int q = blockIdx.x; q < nq; q += gridDim.x) {
      const int i = sh_desc[q].x;
      if (tid < __ldcg(draft_len + i)) {
        const u64 sum = ld_u64(&s.w_edge[(size_t)q * SDMS_MAX_DRAFT + tid]);
        draft_edge_w[(size_t)i * D + tid] = (sum >> kWideSumShift) ? (float)weight_of(s, sum) : 0.0f;
      }
    }
  const u64 used = ld_u64(&s.w_ctl[3]);
  uint4* const z = reinterpret_cast<uint4*>(s.w_tab);
  for (u64 x = (u64)blockIdx.x * blockDim.x + tid; x < 2 * used; x += (u64)gridDim.x * blockDim.x)
    z[x] = make_uint4(0u, 0u, 0u, 0u);
  uint4* const zk = reinterpret_cast<uint4*>(s.w_key);              // slots are handed out in multiples of 64
  for (u64 x = (u64)blockIdx.x * blockDim.x + tid; x < used / 4; x += (u64)gridDim.x * blockDim.x)
    zk[x] = make_uint4(0u, 0u, 0u, 0u);
}

}  // namespace

// Largest grid whose CTAs are all resident at once on the current device (0: no cooperative launch here).
int wide_kernel_grid() {
  int dev = 0, coop = 0, sms = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) { cudaGetLastError(); return 0; }
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dag_wide_kernel, kWideThreads, 0) != cudaSuccess) { cudaGetLastError(); return 0; }
  return sms * (per_sm < 1 ? per_sm : 1);
}

cudaError_t launch_wait_timeout(const Dev& s, long long cycles, cudaStream_t stream) {
  wait_timeout_kernel<<<1, 32, 0, stream>>>(s, cycles);
  return cudaGetLastError();
}

cudaError_t launch_dag_wide(const Dev& s, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                            float* draft_edge_w, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(s.w_grid); cfg.blockDim = dim3(kWideThreads); cfg.dynamicSmemBytes = 0; cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  // Scheduled early as well (its CTAs take their SMs while the kernel before drains: that kernel's CTAs have all
  // started by then and wait for nobody) where the runtime takes both attributes together, else cooperative only.
  static bool early = true;
  if (early) {
    cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, dag_wide_kernel, s, draft_tok, draft_len, draft_score, draft_edge_w);
    if (e == cudaSuccess) return e;
    cudaGetLastError();                               // whatever the reason: once more without the second attribute
    early = false;
  }
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, dag_wide_kernel, s, draft_tok, draft_len, draft_score, draft_edge_w);
}

}  // namespace sdms
