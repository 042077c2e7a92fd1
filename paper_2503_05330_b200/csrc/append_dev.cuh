// Device code of the state update and of the acceptance check, shared by the kernels that run it
// (append_kernel, accept_kernel, and the one-launch step).
#pragma once
#include "sdms_dev.cuh"

namespace sdms {
namespace {

struct dd { double hi, lo; };

__device__ __forceinline__ dd two_sum(double a, double b) {
  double s = __dadd_rn(a, b);
  double bb = __dsub_rn(s, a);
  double e = __dadd_rn(__dsub_rn(a, __dsub_rn(s, bb)), __dsub_rn(b, bb));
  return {s, e};
}
__device__ __forceinline__ dd quick_two_sum(double a, double b) {   // |a| >= |b|
  double s = __dadd_rn(a, b);
  return {s, __dsub_rn(b, __dsub_rn(s, a))};
}
__device__ __forceinline__ dd two_prod(double a, double b) {
  double p = __dmul_rn(a, b);
  return {p, __fma_rn(a, b, -p)};
}
__device__ __forceinline__ dd dd_add(dd a, dd b) {
  dd s = two_sum(a.hi, b.hi);
  dd t = two_sum(a.lo, b.lo);
  s.lo = __dadd_rn(s.lo, t.hi);
  s = quick_two_sum(s.hi, s.lo);
  s.lo = __dadd_rn(s.lo, t.lo);
  return quick_two_sum(s.hi, s.lo);
}
__device__ __forceinline__ dd dd_mul(dd a, dd b) {
  dd p = two_prod(a.hi, b.hi);
  p.lo = __dadd_rn(p.lo, __dadd_rn(__dmul_rn(a.hi, b.lo), __dmul_rn(a.lo, b.hi)));
  return quick_two_sum(p.hi, p.lo);
}
__device__ __forceinline__ dd dd_div_small(dd a, double n) {        // n a small positive integer
  double q = __ddiv_rn(a.hi, n);
  double rem = __fma_rn(-q, n, a.hi);                                // exact remainder
  double ql = __ddiv_rn(__dadd_rn(rem, a.lo), n);
  return quick_two_sum(q, ql);
}

// round_half_even(exp(lp) * 2^30) clamped to [0, 2^30].  exp is evaluated in
// double-double arithmetic (about 100 bits) so that the rounding decision is
// that of the exact real number: argument reduction by a split ln 2, Taylor
// series of exp on |r| <= ln2/2, scaling by a power of two.
__device__ int32_t prob_to_fixed(float lp, uint32_t* st) {
  const int32_t one = 1 << 30;
  if (lp != lp) { *st |= SDMS_STATUS_BAD_LOGPROB; return 0; }
  if (lp >= 0.0f) return one;
  if (lp < -40.0f) return 0;                       // exp(-40) * 2^30 < 1e-8
  const double x = (double)lp;
  {
    // plain double first: exp() is within 1 ulp, so y is within 2e-7 of the true value;
    // only a fraction that close to one half needs the exact evaluation below
    const double y = __dmul_rn(exp(x), 1073741824.0);
    const double fl = floor(y);
    const double frac = __dsub_rn(y, fl);
    if (fabs(__dsub_rn(frac, 0.5)) > 1e-5) return (int32_t)fl + (frac > 0.5 ? 1 : 0);
  }
  const double ln2_hi = 6.93147180369123816490e-01;  // 32 significant bits: m * ln2_hi is exact
  const double ln2_lo = 1.90821492927058770002e-10;  // ln 2 - ln2_hi
  const double m = rint(__dmul_rn(x, 1.44269504088896338700e+00));
  dd r = {__fma_rn(-m, ln2_hi, x), 0.0};             // exact: the difference fits in 53 bits
  dd ml = two_prod(m, ln2_lo);
  r = dd_add(r, dd{-ml.hi, -ml.lo});
  dd sum = {1.0, 0.0};
  dd term = {1.0, 0.0};
  for (int n = 1; n <= 24; ++n) {
    term = dd_div_small(dd_mul(term, r), (double)n);
    sum = dd_add(sum, term);
  }
  const int sh = (int)m + 30;
  const double yh = ldexp(sum.hi, sh), yl = ldexp(sum.lo, sh);
  long long n = __double2ll_rn(yh);
  const double d = __dadd_rn(__dsub_rn(yh, (double)n), yl);
  if (d > 0.5 || (d == 0.5 && (n & 1))) ++n;
  else if (d < -0.5 || (d == -0.5 && (n & 1))) --n;
  if (n < 0) n = 0;
  if (n > one) n = one;
  return (int32_t)n;
}

// Adds one occurrence of an n-gram (hash h) ending at prompt-local position lpos.
__device__ void index_insert(const Dev& s, int g, int n, uint64_t h, uint32_t lpos, uint32_t* st) {
  uint32_t* table = index_table(s, g, n);
  const uint32_t fp = gram_fp(h);
  uint32_t b = gram_bucket(h, s.table_cap);
  for (uint32_t probe = 0; probe < s.table_cap; ++probe) {
    uint32_t* bucket = table + (size_t)b * kBucketWords;
    // {fingerprint, count} is one 64-bit word: an empty bucket is claimed and counted in one atomic
    unsigned long long* head = reinterpret_cast<unsigned long long*>(bucket);
    const unsigned long long old = atomicCAS(head, 0ull, (1ull << 32) | fp);
    if (old == 0ull) { bucket[2] = lpos; return; }
    if ((uint32_t)old == fp) {
      const uint32_t slot = (uint32_t)(atomicAdd(head, 1ull << 32) >> 32);
      if (slot < (uint32_t)kInlineSlots) bucket[2 + slot] = lpos;
      return;
    }
    b = (b + 1) & (s.table_cap - 1);
  }
  *st |= SDMS_STATUS_INDEX_FULL;
}

// Block-cooperative append of n validated tokens to path p whose length is len0.  rec is the
// path's record as it was before the call (shared memory): rec[1 + t] = token at len0 - 1 - t.
// Also writes the path's new record and length (and a copy of the record to rec_out, shared
// memory, if given); no barrier inside.
__device__ void append_tokens(const Dev& s, int p, int len0, int n, const int32_t* in_tok,
                              const float* in_lp, const int32_t* rec, uint32_t* st, int32_t* rec_out = nullptr) {
  int32_t* tok = s.tok + (size_t)p * s.L;
  int32_t* pq = s.pq + (size_t)p * s.L;
  // the stores start from the last thread, the index inserts (below) from the first: with few new
  // tokens different warps do the two and the atomics are in flight during the exponentials
  const int r = (int)blockDim.x - 1 - (int)threadIdx.x;
  for (int a = r; a < n; a += blockDim.x) {
    tok[len0 + a] = in_tok[a];
    pq[len0 + a] = prob_to_fixed(in_lp[a], st);
  }
  const int g = p / s.N;
  const uint32_t lbase = (uint32_t)(p - g * s.N) * (uint32_t)s.L;
  for (int w = threadIdx.x; w < n * s.idx_n; w += blockDim.x) {
    const int a = w / s.idx_n, nn = w % s.idx_n + 1;
    const int pos = len0 + a;
    if (pos + 1 < nn) continue;
    uint64_t h = gram_init(nn);
    for (int t = pos - nn + 1; t <= pos; ++t)
      h = gram_step(h, t < len0 ? rec[len0 - t] : in_tok[t - len0]);   // old tokens from the record, new from the input
    index_insert(s, g, nn, gram_final(h), lbase + (uint32_t)pos, st);
  }
  // the record after the append: new length, then the newest k_max tokens
  int32_t* out = s.rec + (size_t)p * kRecWords;
  // (the last threads write it, so that the warps with inserts to do are not held up)
  if (r < s.k_max) {
    const int x = len0 + n - 1 - r;                                      // position of the token this word holds
    const int32_t v = x >= len0 ? in_tok[x - len0] : (x >= 0 ? rec[len0 - x] : 0);
    out[1 + r] = v;
    if (rec_out) rec_out[1 + r] = v;
  }
  if (r == s.k_max) {
    out[0] = len0 + n; s.len[p] = len0 + n;
    if (rec_out) rec_out[0] = len0 + n;
  }
}

// "Draft acceptance" for path p, then (if sampled_lp is given) the commit: the path appends
// sampled[0 .. min(tau + 1, max_append)).  Block-cooperative, any block size >= 64; every thread of
// the CTA must call it.  draft_tok / draft_len are only read.  If rec_out is given (shared memory,
// kRecWords words) it receives the path's record as it is after the call.  next_k > 0 announces
// the suffix length of the query the path makes next: its index bucket is prefetched into L2.
__device__ void accept_commit_phase(const Dev& s, int p, const int32_t* draft_tok, const int32_t* draft_len,
                                    const int32_t* sampled, const float* sampled_lp, int32_t* accept_len,
                                    int32_t* rec_out = nullptr, int next_k = 0) {
  __shared__ int sh_len0, sh_n;
  __shared__ uint32_t sh_st;
  __shared__ int32_t sh_rec[kRecWords];
  __shared__ int32_t sh_smp[SDMS_MAX_DRAFT + 1];
  __shared__ float sh_lp[SDMS_MAX_DRAFT + 1];
  const int32_t* smp = sampled + (size_t)p * (s.D + 1);
  const int lane = threadIdx.x;
  if (lane < 32) {
    static_assert(kRecWords == 32 && SDMS_MAX_DRAFT <= 32, "one record word, one draft position per lane");
    // every load of this phase is issued before the first use: one round trip to memory
    const int32_t mine = sampled_lp ? s.rec[(size_t)p * kRecWords + lane] : 0;
    int dl = draft_len[p];
    const int32_t drafted = lane < s.D ? draft_tok[(size_t)p * s.D + lane] : -1;
    const int32_t got = lane <= s.D ? smp[lane] : -1;
    const int32_t got_last = lane == 0 && s.D == 32 ? smp[32] : -1;       // position D when D fills the warp
    float lp = 0.0f, lp_last = 0.0f;
    if (sampled_lp) {
      const float* slp = sampled_lp + (size_t)p * (s.D + 1);
      if (lane <= s.D) lp = slp[lane];
      if (lane == 0 && s.D == 32) lp_last = slp[32];
    }
    sh_rec[lane] = mine;
    sh_smp[lane] = got; sh_lp[lane] = lp;
    if (lane == 0) { sh_smp[32] = got_last; sh_lp[32] = lp_last; }
    dl = dl < 0 ? 0 : (dl > s.D ? s.D : dl);
    const bool differs = lane >= dl || drafted != got;
    const unsigned first = __ffs(__ballot_sync(0xffffffffu, differs));   // 0 only if all 32 lanes agree
    const int tau = first ? (int)first - 1 : 32;
    int n = 0, len0 = 0;
    if (sampled_lp) {
      len0 = __shfl_sync(0xffffffffu, mine, 0);         // lane 0 holds the length
      n = min(min(tau + 1, s.max_append), s.L - len0);
      // the commit stops before the first token outside the vocabulary
      const bool bad = lane < n && (got < 0 || got >= s.V);
      const bool bad_last = lane == 0 && n == 33 && (got_last < 0 || got_last >= s.V);      // only lane 0 can see it
      const unsigned bad_mask = __ballot_sync(0xffffffffu, bad);
      const unsigned bad_last_any = __ballot_sync(0xffffffffu, bad_last);
      int ok = bad_mask ? __ffs(bad_mask) - 1 : (bad_last_any ? 32 : n);
      if (lane == 0) { sh_st = ok < n ? SDMS_STATUS_BAD_TOKEN : 0u; sh_len0 = len0; sh_n = ok; }
    }
    if (lane == 0) accept_len[p] = tau;
  }
  if (!sampled_lp) return;                            // uniform: check only
  __syncthreads();
  uint32_t st = 0;
  if (next_k > 0 && s.eps == 0 && threadIdx.x == blockDim.x - 64) {
    const int len0 = sh_len0, len1 = len0 + sh_n;
    if (len1 >= next_k && len1 < s.L) {
      const int nx = min(next_k, s.idx_n);               // the query's last nx tokens are what the index is asked for
      uint64_t h = gram_init(nx);
      for (int x = len1 - nx; x < len1; ++x) h = gram_step(h, x >= len0 ? sh_smp[x - len0] : sh_rec[len0 - x]);
      const uint32_t* bucket =
          index_table(s, p / s.N, nx) + (size_t)gram_bucket(gram_final(h), s.table_cap) * kBucketWords;
      asm volatile("prefetch.global.L2 [%0];" ::"l"(bucket));
    }
  }
  append_tokens(s, p, sh_len0, sh_n, sh_smp, sh_lp, sh_rec, &st, rec_out);
  if (st) atomicOr(&sh_st, st);
  __syncthreads();
  if (threadIdx.x == 0 && sh_st) atomicOr(s.status, sh_st);
}

}  // namespace
}  // namespace sdms
