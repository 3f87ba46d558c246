// Top-k sparsification of the workers' parameter deltas (Section 2, "Compressed Communication";
// Algorithm 2 with top-k as the compressor C; Appendix, "Assumptions around the collective used":
// each worker's delta is sparsified once, the sparse deltas are averaged, nothing is compressed
// after the mean).
//
// Per (tensor, worker) the kk-th largest magnitude is found by a radix select on the bit pattern
// of |x| (31 bits: 11 + 10 + 10), one histogram pass over the data per digit; the entries with
// |x| >= that threshold are kept (ties all kept), so the kept set is unique and the same on every
// implementation that forms x with the same float32 operations.  The fused pass then forms the
// mean of the kept entries, takes the outer Nesterov step and writes the K replicas, like the
// other outer-sync kernels.
//
// x = theta - theta_k, or with error feedback x = fl(fl(beta E_k) + (theta - theta_k)); every
// pass recomputes it with the same single float32 operations.
#include <float.h>

#include "internal.h"

namespace muloco {

namespace {

constexpr int TK_THREADS = 256;
constexpr int TK_WARPS = TK_THREADS / 32;
constexpr int TK_UNIT = 128;                // elements per warp step (4 per lane)
constexpr int TK_UNITS_PER_CTA = 256;       // histogram passes: 32768 elements per CTA and worker (measured: 26.4 ms
                                            // per sync of 400M parameters x 16 workers, against 28.8 with 64 and 32.2 with 32)
constexpr int TK_APPLY_UNITS_PER_CTA = 32;  // fused pass: small CTAs in address order
constexpr int TK_BINS = 2048;               // widest digit (11 bits)

__host__ __device__ constexpr int digit_bits(int pass) { return pass == 0 ? 11 : 10; }
__host__ __device__ constexpr int digit_shift(int pass) { return pass == 0 ? 20 : (pass == 1 ? 10 : 0); }

__device__ __forceinline__ int tk_find_seg(const SyncSeg* __restrict__ segs, int n, int64_t unit) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (segs[mid].unit_begin <= unit) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ void tk_load4(const float* __restrict__ p, bool vec, int nvalid, float (&v)[4]) {
  if (vec) {
    float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = (e < nvalid) ? p[e] : 0.0f;
  }
}

__device__ __forceinline__ void tk_store4(float* __restrict__ p, bool vec, int nvalid, const float (&v)[4]) {
  if (vec) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(v[0], v[1], v[2], v[3]));
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (e < nvalid) __stcs(p + e, v[e]);
  }
}

__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(fabsf(x)); }

// MODE 0: x = theta - theta_k; MODE 1: x = beta E_k + (theta - theta_k); MODE 2: x = theta (a raw array).
template <int MODE>
__device__ __forceinline__ void form_x(const float (&tg)[4], const float (&r)[4], const float (&e)[4], float beta,
                                       float (&x)[4]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (MODE == 2) {
      x[q] = tg[q];
    } else {
      const float d = __fsub_rn(tg[q], r[q]);
      x[q] = (MODE == 1) ? __fadd_rn(__fmul_rn(beta, e[q]), d) : d;
    }
  }
}

// One digit of the radix select: histogram of digit `PASS` over the elements whose higher digits
// equal the prefix found so far.  CTA b handles worker b % K and span b / K of the fragment's
// units (the K CTAs of a span run close together and share theta through L2).  A span that
// crosses a tensor boundary is histogrammed piece by piece.
template <int MODE, int PASS>
__global__ void __launch_bounds__(TK_THREADS)
topk_hist_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps,
                 float* const* __restrict__ efs, int K, int64_t n_units, float ef_beta,
                 const uint32_t* __restrict__ prefix, uint32_t* __restrict__ ghist) {
  __shared__ uint32_t hist[TK_BINS];
  constexpr int NB = 1 << digit_bits(PASS);
  constexpr int SH = digit_shift(PASS);
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int k = (int)(blockIdx.x % (unsigned)K);
  const int64_t span = blockIdx.x / (unsigned)K;
  int64_t u = span * TK_UNITS_PER_CTA;
  int64_t cta_end = u + TK_UNITS_PER_CTA;
  if (cta_end > n_units) cta_end = n_units;
  while (u < cta_end) {
    const int seg = tk_find_seg(segs, n_segs, u);
    const SyncSeg s = segs[seg];
    const int64_t seg_end = (seg + 1 < n_segs) ? segs[seg + 1].unit_begin : n_units;
    const int64_t piece_end = seg_end < cta_end ? seg_end : cta_end;
    const int64_t problem = s.rep_index + k;
    const uint32_t pre = (PASS == 0) ? 0u : prefix[problem];
    for (int b = threadIdx.x; b < NB; b += TK_THREADS) hist[b] = 0u;
    __syncthreads();
    const float* rp = (MODE == 2) ? nullptr : reps[problem];
    const float* ep = (MODE == 1) ? efs[problem] : nullptr;
    const int64_t numel = s.rows * s.cols;
    bool aligned = ((((uintptr_t)s.theta_g) & 15) == 0);
    if (MODE != 2) aligned = aligned && ((((uintptr_t)rp) & 15) == 0);
    if (MODE == 1) aligned = aligned && ((((uintptr_t)ep) & 15) == 0);
    for (int64_t unit = u + warp; unit < piece_end; unit += TK_WARPS) {
      const int64_t off = (unit - s.unit_begin) * TK_UNIT + lane * 4;
      int64_t left = numel - off;
      const int nvalid = left < 0 ? 0 : (left > 4 ? 4 : (int)left);
      const bool vec = aligned && nvalid == 4;
      float tg[4] = {0.f, 0.f, 0.f, 0.f}, r[4] = {0.f, 0.f, 0.f, 0.f}, e[4] = {0.f, 0.f, 0.f, 0.f}, x[4];
      if (nvalid > 0) {
        tk_load4(s.theta_g + off, vec, nvalid, tg);
        if (MODE != 2) tk_load4(rp + off, vec, nvalid, r);
        if (MODE == 1) tk_load4(ep + off, vec, nvalid, e);
      }
      form_x<MODE>(tg, r, e, ef_beta, x);
      uint32_t dg[4];
      bool in[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t key = mag_key(x[q]);
        in[q] = (q < nvalid) && (PASS == 0 || (key >> (SH + digit_bits(PASS))) == pre);
        dg[q] = (key >> SH) & (uint32_t)(NB - 1);
      }
      if (PASS == 0) {
        // The leading digit is the exponent.  A full unit whose 128 keys share it (zero deltas, a
        // constant tensor) adds once; otherwise plain shared-memory atomics: a warp's keys fall
        // into a few dozen bins, a few lanes per bin.
        const uint32_t d0 = __shfl_sync(0xffffffffu, dg[0], 0);
        const bool same = nvalid == 4 && dg[0] == d0 && dg[1] == d0 && dg[2] == d0 && dg[3] == d0;
        if (__all_sync(0xffffffffu, same)) {
          if (lane == 0) atomicAdd(&hist[d0], (uint32_t)TK_UNIT);
          continue;
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (in[q]) atomicAdd(&hist[dg[q]], 1u);
    }
    __syncthreads();
    uint32_t* gh = ghist + problem * TK_BINS;
    for (int b = threadIdx.x; b < NB; b += TK_THREADS) {
      const uint32_t v = hist[b];
      if (v) atomicAdd(gh + b, v);
    }
    __syncthreads();
    u = piece_end;
  }
}

// After a histogram pass: the digit of the kk-th largest key.  One CTA per (tensor of the
// fragment, worker).  Walks the bins from the top; `remaining` is how many of the kk are still
// to be found at or below the chosen bin.  Clears the histogram for the next pass.  After the
// last pass `prefix` is the full 31-bit key of the kk-th largest magnitude.
template <int PASS>
__global__ void __launch_bounds__(TK_THREADS)
topk_scan_kernel(const SyncSeg* __restrict__ segs, const uint32_t* __restrict__ kk_seg,
                 uint32_t* __restrict__ prefix, uint32_t* __restrict__ remaining, uint32_t* __restrict__ ghist) {
  constexpr int NB = 1 << digit_bits(PASS);
  constexpr int PER = NB / TK_THREADS;            // consecutive bins per thread
  __shared__ uint32_t part[TK_THREADS];
  const int64_t problem = segs[blockIdx.x].rep_index + (int64_t)blockIdx.y;
  uint32_t* gh = ghist + problem * TK_BINS;
  const uint32_t need = (PASS == 0) ? kk_seg[blockIdx.x] : remaining[problem];
  // thread t owns bins [NB - (t+1)*PER, NB - t*PER): thread 0 the top ones
  const int hi = NB - (int)threadIdx.x * PER;
  uint32_t c[PER];
  uint32_t mine = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) { c[j] = gh[hi - 1 - j]; mine += c[j]; }
  part[threadIdx.x] = mine;
  __syncthreads();
  // exclusive prefix over threads (counts in bins above this thread's): 256 values, one warp pass each
  uint32_t above = 0;
  for (int t = 0; t < (int)threadIdx.x; ++t) above += part[t];
  __syncthreads();
#pragma unroll
  for (int j = 0; j < PER; ++j) gh[hi - 1 - j] = 0u;
  if (above < need && above + mine >= need) {
    uint32_t acc = above;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (acc < need && acc + c[j] >= need) {
        const uint32_t dg = (uint32_t)(hi - 1 - j);
        const uint32_t pre = (PASS == 0) ? 0u : prefix[problem];
        prefix[problem] = (pre << digit_bits(PASS)) | dg;
        remaining[problem] = need - acc;
      }
      acc += c[j];
    }
  }
}

// The fused pass: mean of the kept entries, outer Nesterov step (Eq. 3), broadcast; with error
// feedback E_k <- x - kept(x).  Same unit/CTA mapping and arithmetic order as the two-stage
// quantised kernel: workers ascending, one float32 operation at a time, then * fl(1/K).
template <bool EF>
__global__ void __launch_bounds__(TK_THREADS)
outer_sync_topk_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps,
                       float* const* __restrict__ efs, int K, int64_t n_units, float eta, float mu,
                       float inv_k, float ef_beta, const uint32_t* __restrict__ thr, int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t cta_begin = (int64_t)blockIdx.x * TK_APPLY_UNITS_PER_CTA;
  int64_t cta_end = cta_begin + TK_APPLY_UNITS_PER_CTA;
  if (cta_end > n_units) cta_end = n_units;
  bool bad = false;
  int64_t unit = cta_begin + warp;
  if (unit < cta_end) {
    int seg = tk_find_seg(segs, n_segs, unit);
    SyncSeg s = segs[seg];
    int64_t seg_end = (seg + 1 < n_segs) ? segs[seg + 1].unit_begin : n_units;
    for (; unit < cta_end; unit += TK_WARPS) {
      while (unit >= seg_end) {
        ++seg;
        s = segs[seg];
        seg_end = (seg + 1 < n_segs) ? segs[seg + 1].unit_begin : n_units;
      }
      const int64_t off = (unit - s.unit_begin) * TK_UNIT + lane * 4;
      const int64_t left = s.rows * s.cols - off;
      const int nvalid = left < 0 ? 0 : (left > 4 ? 4 : (int)left);
      float* const* rp = reps + s.rep_index;
      float* const* ep = EF ? efs + s.rep_index : nullptr;
      const uint32_t* tp = thr + s.rep_index;
      bool vec = ((((uintptr_t)s.theta_g | (uintptr_t)s.u) & 15) == 0) && nvalid == 4;
      for (int k = 0; k < K; ++k) {
        vec = vec && ((((uintptr_t)rp[k]) & 15) == 0);
        if (EF) vec = vec && ((((uintptr_t)ep[k]) & 15) == 0);
      }
      if (nvalid <= 0) continue;
      float tg[4], uu[4], acc[4] = {0.f, 0.f, 0.f, 0.f};
      tk_load4(s.theta_g + off, vec, nvalid, tg);
      tk_load4(s.u + off, vec, nvalid, uu);
      for (int k0 = 0; k0 < K; k0 += 4) {
        float r[4][4], e[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
          for (int q = 0; q < 4; ++q) { r[j][q] = 0.f; e[j][q] = 0.f; }
          if (k0 + j < K) {
            tk_load4(rp[k0 + j] + off, vec, nvalid, r[j]);
            if (EF) tk_load4(ep[k0 + j] + off, vec, nvalid, e[j]);
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (k0 + j < K) {
            const uint32_t t = tp[k0 + j];
            float x[4], sent[4];
            if (EF) form_x<1>(tg, r[j], e[j], ef_beta, x); else form_x<0>(tg, r[j], e[j], ef_beta, x);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              if (q < nvalid && !(fabsf(x[q]) <= FLT_MAX)) bad = true;
              sent[q] = (mag_key(x[q]) >= t) ? x[q] : 0.0f;
              acc[q] = __fadd_rn(acc[q], sent[q]);
            }
            if (EF) {
              float en[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) en[q] = __fsub_rn(x[q], sent[q]);
              tk_store4(ep[k0 + j] + off, vec, nvalid, en);
            }
          }
        }
      }
      float un[4], tn[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float psi = __fmul_rn(acc[q], inv_k);
        const float epq = eta * psi;
        un[q] = fmaf(mu, uu[q], epq);
        tn[q] = tg[q] - fmaf(mu, un[q], epq);
      }
      tk_store4(s.u + off, vec, nvalid, un);
      tk_store4(s.theta_g + off, vec, nvalid, tn);
      for (int k = 0; k < K; ++k) tk_store4(rp[k] + off, vec, nvalid, tn);
    }
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, ST_NONFINITE);
}

// Standalone form: out = x where |x| >= threshold, else 0.
__global__ void topk_apply_raw_kernel(const float* __restrict__ x, int64_t n, const uint32_t* __restrict__ thr,
                                      float* __restrict__ out, int* __restrict__ status) {
  const uint32_t t = thr[0];
  bool bad = false;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const float v = x[i];
    if (!(fabsf(v) <= FLT_MAX)) bad = true;
    out[i] = (mag_key(v) >= t) ? v : 0.0f;
  }
  if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicOr(status, ST_NONFINITE);
}

template <int MODE>
void select_thresholds(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* reps, float* const* efs,
                       int K, int64_t n_units, float ef_beta, const uint32_t* kk_seg, TopkScratch& sc) {
  const int64_t spans = (n_units + TK_UNITS_PER_CTA - 1) / TK_UNITS_PER_CTA;
  const dim3 hgrid((unsigned)(spans * K));
  const dim3 sgrid((unsigned)n_segs, (unsigned)K);
  topk_hist_kernel<MODE, 0><<<hgrid, TK_THREADS, 0, st>>>(segs, n_segs, reps, efs, K, n_units, ef_beta, sc.prefix, sc.hist);
  topk_scan_kernel<0><<<sgrid, TK_THREADS, 0, st>>>(segs, kk_seg, sc.prefix, sc.remaining, sc.hist);
  topk_hist_kernel<MODE, 1><<<hgrid, TK_THREADS, 0, st>>>(segs, n_segs, reps, efs, K, n_units, ef_beta, sc.prefix, sc.hist);
  topk_scan_kernel<1><<<sgrid, TK_THREADS, 0, st>>>(segs, kk_seg, sc.prefix, sc.remaining, sc.hist);
  topk_hist_kernel<MODE, 2><<<hgrid, TK_THREADS, 0, st>>>(segs, n_segs, reps, efs, K, n_units, ef_beta, sc.prefix, sc.hist);
  topk_scan_kernel<2><<<sgrid, TK_THREADS, 0, st>>>(segs, kk_seg, sc.prefix, sc.remaining, sc.hist);
}

}  // namespace

size_t topk_hist_words_per_problem() { return TK_BINS; }

int launch_outer_sync_topk(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas, int K,
                           int64_t n_units, float outer_lr, float mu, int* status, float* const* ef,
                           float ef_beta, const uint32_t* kk_seg, TopkScratch sc) {
  if (n_units <= 0 || n_segs <= 0) return 0;
  if (ef) select_thresholds<1>(st, segs, n_segs, replicas, ef, K, n_units, ef_beta, kk_seg, sc);
  else select_thresholds<0>(st, segs, n_segs, replicas, ef, K, n_units, ef_beta, kk_seg, sc);
  const int64_t ctas = (n_units + TK_APPLY_UNITS_PER_CTA - 1) / TK_APPLY_UNITS_PER_CTA;
  const float inv_k = 1.0f / (float)K;
  if (ef)
    outer_sync_topk_kernel<true><<<(unsigned)ctas, TK_THREADS, 0, st>>>(segs, n_segs, replicas, ef, K, n_units, outer_lr,
                                                                        mu, inv_k, ef_beta, sc.prefix, status);
  else
    outer_sync_topk_kernel<false><<<(unsigned)ctas, TK_THREADS, 0, st>>>(segs, n_segs, replicas, ef, K, n_units,
                                                                         outer_lr, mu, inv_k, ef_beta, sc.prefix, status);
  return 7;
}

int launch_topk_raw(cudaStream_t st, const SyncSeg* seg_dev, int64_t n, const float* x, float* out,
                    const uint32_t* kk_dev, TopkScratch sc, int* status) {
  if (n <= 0) return 0;
  const int64_t n_units = (n + TK_UNIT - 1) / TK_UNIT;
  select_thresholds<2>(st, seg_dev, 1, nullptr, nullptr, 1, n_units, 0.0f, kk_dev, sc);
  const int blocks = (int)((n + 255) / 256 < 4096 ? (n + 255) / 256 : 4096);
  topk_apply_raw_kernel<<<blocks, 256, 0, st>>>(x, n, sc.prefix, out, status);
  return 7;
}

}  // namespace muloco
