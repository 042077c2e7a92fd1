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
    const uint32_t old = atomicCAS(&bucket[0], 0u, fp);
    if (old == 0u || old == fp) {
      const uint32_t slot = atomicAdd(&bucket[1], 1u);
      if (slot < (uint32_t)kInlineSlots) bucket[2 + slot] = lpos;
      return;
    }
    b = (b + 1) & (s.table_cap - 1);
  }
  *st |= SDMS_STATUS_INDEX_FULL;
}

// Block-cooperative append of n validated tokens to path p whose length is len0.  rec is the
// path's record as it was before the call (shared memory): rec[1 + t] = token at len0 - 1 - t.
// Ends with a barrier-free write of the new record by the first k_max threads; the caller
// updates nothing else.
__device__ void append_tokens(const Dev& s, int p, int len0, int n, const int32_t* in_tok,
                              const float* in_lp, const int32_t* rec, uint32_t* st) {
  int32_t* tok = s.tok + (size_t)p * s.L;
  int32_t* pq = s.pq + (size_t)p * s.L;
  for (int a = threadIdx.x; a < n; a += blockDim.x) {
    tok[len0 + a] = in_tok[a];
    pq[len0 + a] = prob_to_fixed(in_lp[a], st);
  }
  const int g = p / s.N;
  const uint32_t lbase = (uint32_t)(p - g * s.N) * (uint32_t)s.L;
  for (int w = threadIdx.x; w < n * s.k_max; w += blockDim.x) {
    const int a = w / s.k_max, nn = w % s.k_max + 1;
    const int pos = len0 + a;
    if (pos + 1 < nn) continue;
    uint64_t h = gram_init(nn);
    for (int t = pos - nn + 1; t <= pos; ++t)
      h = gram_step(h, t < len0 ? rec[len0 - t] : in_tok[t - len0]);   // old tokens from the record, new from the input
    index_insert(s, g, nn, gram_final(h), lbase + (uint32_t)pos, st);
  }
  // the record after the append: new length, then the newest k_max tokens
  int32_t* out = s.rec + (size_t)p * kRecWords;
  if (threadIdx.x < s.k_max) {
    const int x = len0 + n - 1 - (int)threadIdx.x;                       // position of the token this word holds
    out[1 + threadIdx.x] = x >= len0 ? in_tok[x - len0] : (x >= 0 ? rec[len0 - x] : 0);
  }
  if (threadIdx.x == 0) { out[0] = len0 + n; s.len[p] = len0 + n; }
}

// "Draft acceptance" for path p, then (if sampled_lp is given) the commit: the path appends
// sampled[0 .. min(tau + 1, max_append)).  Block-cooperative, any block size >= 32; every thread of
// the CTA must call it.  draft_tok / draft_len are only read.
__device__ void accept_commit_phase(const Dev& s, int p, const int32_t* draft_tok, const int32_t* draft_len,
                                    const int32_t* sampled, const float* sampled_lp, int32_t* accept_len) {
  __shared__ int sh_len0, sh_n, sh_bad;
  __shared__ uint32_t sh_st;
  __shared__ int32_t sh_rec[kRecWords];
  const int32_t* smp = sampled + (size_t)p * (s.D + 1);
  if (threadIdx.x < 32) {
    static_assert(kRecWords == 32, "one record word per lane");
    const int32_t mine = sampled_lp ? s.rec[(size_t)p * kRecWords + threadIdx.x] : 0;   // in flight with the draft
    sh_rec[threadIdx.x] = mine;
    int dl = draft_len[p];
    dl = dl < 0 ? 0 : (dl > s.D ? s.D : dl);
    const int d = threadIdx.x;
    const bool differs = d >= dl || draft_tok[(size_t)p * s.D + d] != smp[d];
    const unsigned first = __ffs(__ballot_sync(0xffffffffu, differs));   // 0 only if all 32 lanes agree
    const int tau = first ? (int)first - 1 : 32;
    if (d == 0) {
      accept_len[p] = tau;
      int n = 0, len0 = 0;
      if (sampled_lp) {
        len0 = mine;                                  // lane 0 holds the length
        n = min(min(tau + 1, s.max_append), s.L - len0);
      }
      sh_len0 = len0; sh_n = n; sh_bad = n; sh_st = 0;
    }
  }
  if (!sampled_lp) return;                            // uniform: check only
  __syncthreads();
  for (int a = threadIdx.x; a < sh_n; a += blockDim.x) {
    const int32_t t = smp[a];
    if (t < 0 || t >= s.V) atomicMin(&sh_bad, a);
  }
  __syncthreads();
  uint32_t st = 0;
  const int n = sh_bad;
  if (threadIdx.x == 0 && n < sh_n) st |= SDMS_STATUS_BAD_TOKEN;
  append_tokens(s, p, sh_len0, n, smp, sampled_lp + (size_t)p * (s.D + 1), sh_rec, &st);
  if (st) atomicOr(&sh_st, st);
  __syncthreads();
  if (threadIdx.x == 0 && sh_st) atomicOr(s.status, sh_st);
}

}  // namespace
}  // namespace sdms
