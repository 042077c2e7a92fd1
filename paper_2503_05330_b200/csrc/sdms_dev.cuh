// Device-side view of a context and helpers shared by the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "sdms.h"

namespace sdms {

constexpr int kBucketWords = 8;        // one 32-byte sector: fingerprint, count, 6 positions
constexpr int kInlineSlots = kBucketWords - 2;
constexpr int kRecWords = 32;          // one 128-byte line per path: what a step needs first, in one load
constexpr int kHalo = SDMS_MAX_K;      // tokens staged in front of a scan tile
constexpr int kScanTile = 1024;        // history tokens per scan CTA
constexpr int kScanThreads = 256;
constexpr int kDagThreads = 512;
constexpr int kMaxClusterPaths = 16;    // largest thread-block cluster (one CTA per path of a prompt)
constexpr int kFusedThreads = 512;     // the single-launch build: more loads in flight while it scans
constexpr int kDagCap = 1024;          // entries of the shared-memory node / edge tables
constexpr int kFusedMaxTokens = 131072; // largest N*L a CTA scans on its own
constexpr int kMaxWide = 1024;          // queries one build can hand to the device-wide aggregation pass
constexpr int kWideSumShift = 47;       // packed node sums: count in the upper 17 bits, sum of probabilities below
constexpr int kWideMaxMatches = (1 << 17) - 1;   // so that both parts of a packed sum fit
constexpr int kWideBarrierWays = 8;     // grid-barrier arrivals are spread over this many counters ...
constexpr int kWideBarrierAt = 16, kWideBarrierStride = 16;   // ... at w_ctl[16], [32], ...: a 128-byte line each
constexpr int kWideCtlWords = kWideBarrierAt + kWideBarrierWays * kWideBarrierStride;

// Q_DONE: a back-off build on a large prompt has found this path's matches at a longer suffix length
enum QueryMode : int32_t { Q_NONE = 0, Q_INLINE = 1, Q_SCAN = 2, Q_DONE = 3 };
constexpr int kRoundBackoff = 1, kRoundNotFirst = 2, kRoundLast = 4;   // flags of one round of such a build

// One slot of a wide query's node table of one layer (32 bytes, one sector).  All-zero = empty.  The keys
// (token + 1) that the probing looks at lie in an array of their own, eight to a sector.
struct WideSlot {
  uint32_t tok1;                 // token + 1, written by whoever claimed the slot
  uint32_t unused;
  unsigned long long sum;        // count << kWideSumShift | sum of fixed-point probabilities of the node
  unsigned long long succ_w;     // bit pattern of the largest Eq. 5 weight among the node's successors
  unsigned long long succ;       // ~token << 32 | slot of the successor with that weight and the smallest token; 0 = none
};
struct BeamEnt;
struct WidePred { unsigned long long succ_w, succ; };   // the same two words for the root (and, in mode 1, for each layer)

// Everything a kernel needs, passed by value.
struct Dev {
  int32_t G, N, L, V, k_max, D, max_append, B, Ke, mode, P;
  int32_t idx_n;                       // n-gram lengths 1..idx_n have index tables (<= k_max)
  int32_t pool;                        // 0 DAG, 1 tree, 2 list
  int32_t eps;                         // edit-distance tolerance of the suffix match (0 or 1)
  int32_t fused;                       // one kernel per build (small prompts) instead of probe + scan + dag
  int32_t build_cluster;               // CTAs per cluster of the single-launch build (they share their prompt's scan); 1 = none
  int32_t R;                           // matches kept per (query path, source path): the R most recent; 0 = all
  double alpha;
  uint32_t table_cap;                  // buckets per (prompt, n) table, power of two
  uint32_t L_magic; int32_t L_shift;   // x / L for 0 <= x < 2^31 as (x * L_magic) >> L_shift (path_of)
  int64_t match_cap;
  // path store
  int32_t* tok;                        // [P][L]
  int32_t* pq;                         // [P][L] fixed-point probabilities
  int32_t* len;                        // [P]
  int32_t* rec;                        // [P][kRecWords] per path: length, then its last k_max tokens, newest first
  uint32_t* status;
  uint32_t* index;                     // [G][k_max][table_cap][kBucketWords]
  // per-query scratch of the last build
  uint32_t* q_fp;                      // [P]
  int32_t* q_mode;                     // [P]
  int32_t* q_reserved;                 // [P] match slots reserved (index count)
  int32_t* q_off;                      // [P] start in `matches`
  int32_t* q_cursor;                   // [P] matches written
  unsigned long long* match_cursor;    // match slots handed to scan queries by the probe; zero between builds
  int32_t* g_nscan;                    // [G] queries of the prompt that need the scan; zero between builds
  int32_t* g_trim;                     // [G] a path of the prompt was trimmed: its index is rebuilt
  int32_t* matches;                    // [match_cap] global positions j*L+e
  // device-wide aggregation of queries with many matches (dag_wide.cu); w_slots = 0: not in use
  unsigned long long* w_ctl;           // [kWideCtlWords] queries registered, slots handed out, -, end of the slots in use; barrier counters
  int4* w_desc;                        // [kMaxWide] query path, matches, log2 of the slots per layer, first slot
  WidePred* w_pred;                    // [kMaxWide][SDMS_MAX_DRAFT]
  unsigned long long* w_edge;          // [kMaxWide][SDMS_MAX_DRAFT] packed sums of the edges the draft takes
  WideSlot* w_tab;                     // [w_slots]
  uint32_t* w_key;                     // [w_slots] token + 1 of the node in the slot, 0 = free
  int32_t* w_item;                     // [w_slots] per (layer, match): slot of the item's token in the layer's table
  unsigned long long w_slots;
  BeamEnt* b_ent;                      // [w_slots][beam_stride] continuations kept per node (sdms_get_beams)
  unsigned long long* b_ctl;           // [2] slots handed out by the beam kernel / by the best-path launch after a build
  int32_t beam_stride;                 // continuations kept per node: the context's max_beams, 1 for search mode 2 alone
  int32_t* bp_todo;                    // [P] search mode 2: the path's best path is still to be searched over global tables
  int32_t w_grid;                      // CTAs of the wide pass (all resident at once)
  // DAG export of the last build
  int32_t* x_node_tok; int64_t* x_node_S; int32_t* x_node_cnt; int32_t* x_node_count;
  int32_t* x_edge_dst; int64_t* x_edge_S; int32_t* x_edge_cnt; int32_t* x_out_degree;
};

// 64-bit hash of an n-gram, fed token by token (oldest first).
__device__ __forceinline__ uint64_t gram_init(int n) {
  return 0x9E3779B97F4A7C15ull * (uint64_t)(n + 1);
}
__device__ __forceinline__ uint64_t gram_step(uint64_t h, int32_t tok) {
  h = (h ^ (uint64_t)(uint32_t)tok) * 0xFF51AFD7ED558CCDull;
  return h ^ (h >> 29);
}
__device__ __forceinline__ uint64_t gram_final(uint64_t h) {
  h *= 0xC4CEB9FE1A85EC53ull;
  return h ^ (h >> 32);
}
// Non-zero 32-bit fingerprint (0 marks an empty bucket) and bucket number.
__device__ __forceinline__ uint32_t gram_fp(uint64_t h) { return (uint32_t)(h >> 32) | 1u; }
__device__ __forceinline__ uint32_t gram_bucket(uint64_t h, uint32_t cap) { return (uint32_t)h & (cap - 1); }

__device__ __forceinline__ uint32_t* index_table(const Dev& s, int g, int n) {
  return s.index + ((size_t)(g * s.idx_n + (n - 1)) * s.table_cap) * kBucketWords;
}

// Path (row of the store) a global position x = j * L + e lies in, without a division: L_magic =
// ceil(2^(31 + l) / L) with l = ceil(log2 L) fits 32 bits and gives the exact quotient for every
// 0 <= x < 2^31 (round-up method of division by an invariant integer).
__device__ __forceinline__ int path_of(const Dev& s, int x) {
  return (int)(((uint64_t)(uint32_t)x * s.L_magic) >> s.L_shift);
}

// Eq. 5 on integer sums: alpha * S / 2^30 + (1 - alpha) * cnt, every operation
// rounded on its own (no fused multiply-add), so that any two evaluations of
// the same (S, cnt) agree bit for bit.
__device__ __forceinline__ double eq5_weight(double alpha, unsigned long long S, unsigned int cnt) {
  double t1 = __dmul_rn(alpha, (double)S);
  t1 = __dmul_rn(t1, 1.0 / 1073741824.0);
  double t2 = __dmul_rn(__dsub_rn(1.0, alpha), (double)cnt);
  return __dadd_rn(t1, t2);
}

// Programmatic dependent launch: a kernel launched with launch_overlapped() may be scheduled while
// the kernel before it on the stream is still draining.  grid_wait() returns once that kernel has
// completed and its writes are visible; everything that touches memory comes after it.
// grid_release() lets the next kernel on the stream start being scheduled.
__device__ __forceinline__ void grid_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Total order of the export and of the search: larger weight first, then smaller token.
__device__ __forceinline__ bool ranks_before(double wa, int ta, double wb, int tb) {
  return wa > wb || (wa == wb && ta < tb);
}

}  // namespace sdms
