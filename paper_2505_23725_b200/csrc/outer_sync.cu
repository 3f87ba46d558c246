// Outer synchronisation (outer step of Algorithm 1, Eqs. 2-3) as ONE pass over memory:
// pseudogradient over the K replicas, optional per-block quantise->dequantise,
// Nesterov outer step, broadcast into the K replicas.  Pure HBM streaming:
// (K+2) fp32 reads and (K+2) fp32 writes per parameter.
//
// Work unit = one block of `block` (<= 128) consecutive elements of one row,
// handled by one warp, four elements per lane (128-bit accesses when the row
// pitch allows).  A CTA owns a short contiguous span of units; CTAs are launched
// in address order.
#include <float.h>

#include "internal.h"

namespace muloco {

namespace {

constexpr int SYNC_THREADS = 256;
constexpr int SYNC_WARPS = SYNC_THREADS / 32;
// Units per warp.  Small CTAs in launch order: the CTAs resident at any moment then work on
// one narrow window of each of the K+2 streams, which keeps DRAM pages open (measured: 6.56 TB/s
// with 4 units per warp against 5.8 TB/s with a few long spans per SM).
constexpr int SYNC_UNITS_PER_WARP = 4;

__device__ __forceinline__ int find_seg(const SyncSeg* __restrict__ segs, int n, int64_t unit) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (segs[mid].unit_begin <= unit) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Quantise -> dequantise the (up to) four values of this lane; the block is the
// whole warp.  Exact fp32 operations, no contraction: amax, inv = qmax / amax,
// q = rint(x * inv) clamped, scale = amax / qmax, x^ = q * scale.
template <int QB>
__device__ __forceinline__ void quant_dequant4(float (&x)[4], int nvalid, int (&q)[4], float& scale,
                                               bool& bad) {
  constexpr float qmax = (QB == 8) ? 127.0f : (QB == 4 ? 7.0f : 1.0f);
  float lmax = 0.0f;
#pragma unroll
  for (int e = 0; e < 4; ++e)
    if (e < nvalid) {
      float a = fabsf(x[e]);
      if (!(a <= FLT_MAX)) bad = true;
      lmax = fmaxf(lmax, a);
    }
  const float amax = warp_max(lmax);
  if (amax > 0.0f && amax <= FLT_MAX) {
    const float inv = __fdiv_rn(qmax, amax);
    scale = __fdiv_rn(amax, qmax);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float r = rintf(__fmul_rn(x[e], inv));
      r = fminf(fmaxf(r, -qmax), qmax);
      q[e] = (int)r;
      x[e] = __fmul_rn(r, scale);
    }
  } else {
    scale = 0.0f;
#pragma unroll
    for (int e = 0; e < 4; ++e) { q[e] = 0; x[e] = 0.0f; }
  }
}

__device__ __forceinline__ void load4(const float* __restrict__ p, bool vec, int nvalid, float (&v)[4]) {
  if (vec) {
    float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = (e < nvalid) ? __ldcs(p + e) : 0.0f;
  }
}

__device__ __forceinline__ void store4(float* __restrict__ p, bool vec, int nvalid, const float (&v)[4]) {
  if (vec) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(v[0], v[1], v[2], v[3]));
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (e < nvalid) __stcs(p + e, v[e]);
  }
}

// KT > 0: K known at compile time (all replica loads in flight at once).
template <int KT, int QB>
__global__ void __launch_bounds__(SYNC_THREADS)
outer_sync_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps,
                  int Krt, int64_t n_units, int64_t units_per_cta, int block, float eta, float mu,
                  float inv_k, int* __restrict__ status) {
  const int K = (KT > 0) ? KT : Krt;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t cta_begin = (int64_t)blockIdx.x * units_per_cta;
  int64_t cta_end = cta_begin + units_per_cta;
  if (cta_end > n_units) cta_end = n_units;
  bool bad = false;

  int64_t unit = cta_begin + warp;
  if (unit < cta_end) {
    int seg = find_seg(segs, n_segs, unit);
    SyncSeg s = segs[seg];
    int64_t seg_end = (seg + 1 < n_segs) ? segs[seg + 1].unit_begin : n_units;
    bool aligned = ((s.cols & 3) == 0) && ((((uintptr_t)s.theta_g | (uintptr_t)s.u) & 15) == 0);
    for (; unit < cta_end; unit += SYNC_WARPS) {
      while (unit >= seg_end) {
        ++seg;
        if (!MULOCO_IN_BOUNDS(seg < n_segs, status)) return;
        s = segs[seg];
        seg_end = (seg + 1 < n_segs) ? segs[seg + 1].unit_begin : n_units;
        aligned = ((s.cols & 3) == 0) && ((((uintptr_t)s.theta_g | (uintptr_t)s.u) & 15) == 0);
      }
      const int64_t ul = unit - s.unit_begin;
      if (!MULOCO_IN_BOUNDS(ul >= 0 && ul < s.rows * s.nblk, status)) return;
      const int64_t row = ul / s.nblk;
      const int64_t blk = ul - row * s.nblk;
      const int64_t col0 = blk * block + lane * 4;
      int64_t blk_end = (blk + 1) * block;
      if (blk_end > s.cols) blk_end = s.cols;
      int nvalid = (int)(blk_end - col0);
      nvalid = nvalid < 0 ? 0 : (nvalid > 4 ? 4 : nvalid);
      const int64_t off = row * s.cols + col0;
      float* const* rp = reps + s.rep_index;

      float tg[4], uu[4], acc[4] = {0.f, 0.f, 0.f, 0.f};
      bool vec = aligned && nvalid == 4;
      if (nvalid > 0) {
        if (KT > 0) {
          float r[KT > 0 ? KT : 1][4];
          bool v2 = vec;
#pragma unroll
          for (int k = 0; k < KT; ++k) v2 = v2 && ((((uintptr_t)rp[k]) & 15) == 0);
          vec = v2;
          load4(s.theta_g + off, vec, nvalid, tg);
          load4(s.u + off, vec, nvalid, uu);
#pragma unroll
          for (int k = 0; k < KT; ++k) load4(rp[k] + off, vec, nvalid, r[k]);
#pragma unroll
          for (int k = 0; k < KT; ++k)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[e] = __fadd_rn(acc[e], __fsub_rn(tg[e], r[k][e]));
        } else {
          for (int k = 0; k < K; ++k) vec = vec && ((((uintptr_t)rp[k]) & 15) == 0);
          load4(s.theta_g + off, vec, nvalid, tg);
          load4(s.u + off, vec, nvalid, uu);
          for (int k0 = 0; k0 < K; k0 += 4) {
            float r[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (k0 + j < K) load4(rp[k0 + j] + off, vec, nvalid, r[j]);
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (k0 + j < K)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[e] = __fadd_rn(acc[e], __fsub_rn(tg[e], r[j][e]));
          }
        }
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) { tg[e] = 0.f; uu[e] = 0.f; }
      }
      float psi[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) psi[e] = __fmul_rn(acc[e], inv_k);
      if (QB != 0) {
        int q[4]; float sc;
        quant_dequant4<(QB == 0 ? 8 : QB)>(psi, nvalid, q, sc, bad);
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (e < nvalid && !(fabsf(psi[e]) <= FLT_MAX)) bad = true;
      }
      if (nvalid > 0) {
        float un[4], tn[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float ep = eta * psi[e];
          un[e] = fmaf(mu, uu[e], ep);
          tn[e] = tg[e] - fmaf(mu, un[e], ep);
        }
        store4(s.u + off, vec, nvalid, un);
        store4(s.theta_g + off, vec, nvalid, tn);
        for (int k = 0; k < K; ++k) store4(rp[k] + off, vec, nvalid, tn);
      }
    }
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, ST_NONFINITE);
}

// Algorithm 2 with two quantisations (Section 2, "Collectives for compressed communication"):
// every worker's delta (or error-feedback accumulator) is quantised -> dequantised per block,
// the mean of those is taken in fp32 (k ascending, then * 1/K) and quantised again.  Workers are
// read four at a time.  Same unit/CTA mapping as outer_sync_kernel; with error feedback the
// accumulators add one fp32 read and one write per worker and parameter.
template <int QB, bool EF>
__global__ void __launch_bounds__(SYNC_THREADS)
outer_sync2_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps,
                   float* const* __restrict__ efs, int K, int64_t n_units, int64_t units_per_cta, int block,
                   float eta, float mu, float inv_k, float ef_beta, int* __restrict__ status) {
  // workers per batch (their loads are in flight together).  Measured at 400M parameters, int4:
  // without error feedback 2 beats 4, 8, 16 (K=16: 5.64 / 5.56 / 4.91 / 5.42 TB/s; K=5: 5.27 / 4.81 / 4.11 /
  // 3.88), with error feedback 4 beats 2, 8, 16 (6.42 / 5.84 / 6.08 / 4.15 TB/s).  Fetching the next batch
  // before the current one is reduced (double-buffered registers) was slower in both (4.94 and 5.60 TB/s).
  constexpr int WB = EF ? 4 : 2;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t cta_begin = (int64_t)blockIdx.x * units_per_cta;
  int64_t cta_end = cta_begin + units_per_cta;
  if (cta_end > n_units) cta_end = n_units;
  bool bad = false;
  int64_t unit = cta_begin + warp;
  if (unit < cta_end) {
    int seg = find_seg(segs, n_segs, unit);
    SyncSeg s = segs[seg];
    int64_t seg_end = (seg + 1 < n_segs) ? segs[seg + 1].unit_begin : n_units;
    for (; unit < cta_end; unit += SYNC_WARPS) {
      while (unit >= seg_end) {
        ++seg;
        if (!MULOCO_IN_BOUNDS(seg < n_segs, status)) return;
        s = segs[seg];
        seg_end = (seg + 1 < n_segs) ? segs[seg + 1].unit_begin : n_units;
      }
      const int64_t ul = unit - s.unit_begin;
      if (!MULOCO_IN_BOUNDS(ul >= 0 && ul < s.rows * s.nblk, status)) return;
      const int64_t row = ul / s.nblk;
      const int64_t blk = ul - row * s.nblk;
      const int64_t col0 = blk * block + lane * 4;
      int64_t blk_end = (blk + 1) * block;
      if (blk_end > s.cols) blk_end = s.cols;
      int nvalid = (int)(blk_end - col0);
      nvalid = nvalid < 0 ? 0 : (nvalid > 4 ? 4 : nvalid);
      const int64_t off = row * s.cols + col0;
      float* const* rp = reps + s.rep_index;
      float* const* ep = EF ? efs + s.rep_index : nullptr;
      bool vec = ((s.cols & 3) == 0) && ((((uintptr_t)s.theta_g | (uintptr_t)s.u) & 15) == 0) && nvalid == 4;
      for (int k = 0; k < K; ++k) {
        vec = vec && ((((uintptr_t)rp[k]) & 15) == 0);
        if (EF) vec = vec && ((((uintptr_t)ep[k]) & 15) == 0);
      }
      float tg[4] = {0.f, 0.f, 0.f, 0.f}, uu[4] = {0.f, 0.f, 0.f, 0.f}, acc[4] = {0.f, 0.f, 0.f, 0.f};
      if (nvalid > 0) {
        load4(s.theta_g + off, vec, nvalid, tg);
        load4(s.u + off, vec, nvalid, uu);
      }
      for (int k0 = 0; k0 < K; k0 += WB) {
        float r[WB][4], e[EF ? WB : 1][4];
#pragma unroll
        for (int j = 0; j < WB; ++j) {
#pragma unroll
          for (int q = 0; q < 4; ++q) { r[j][q] = 0.f; e[EF ? j : 0][q] = 0.f; }
          if (k0 + j < K && nvalid > 0) {
            load4(rp[k0 + j] + off, vec, nvalid, r[j]);
            if (EF) load4(ep[k0 + j] + off, vec, nvalid, e[EF ? j : 0]);
          }
        }
#pragma unroll
        for (int j = 0; j < WB; ++j) {
          if (k0 + j < K) {            // uniform over the warp: the block reduction below needs every lane
            float x[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float d = __fsub_rn(tg[q], r[j][q]);
              x[q] = EF ? __fadd_rn(__fmul_rn(ef_beta, e[EF ? j : 0][q]), d) : d;
            }
            float sent[4] = {x[0], x[1], x[2], x[3]};
            int qq[4]; float sc;
            quant_dequant4<QB>(sent, nvalid, qq, sc, bad);
            if (EF && nvalid > 0) {
              float en[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) en[q] = __fsub_rn(x[q], sent[q]);
              store4(ep[k0 + j] + off, vec, nvalid, en);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[q] = __fadd_rn(acc[q], sent[q]);
          }
        }
      }
      float psi[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) psi[q] = __fmul_rn(acc[q], inv_k);
      {
        int qq[4]; float sc;
        quant_dequant4<QB>(psi, nvalid, qq, sc, bad);
      }
      if (nvalid > 0) {
        float un[4], tn[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float epq = eta * psi[q];
          un[q] = fmaf(mu, uu[q], epq);
          tn[q] = tg[q] - fmaf(mu, un[q], epq);
        }
        store4(s.u + off, vec, nvalid, un);
        store4(s.theta_g + off, vec, nvalid, tn);
        for (int k = 0; k < K; ++k) store4(rp[k] + off, vec, nvalid, tn);
      }
    }
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, ST_NONFINITE);
}

// Row-wise quantisation (one absmax block per row; Section 6.3 and the row-wise panels of the
// quantisation ablation): one CTA per row.  The row's pseudogradient (or, with two stages, the mean
// of the workers' dequantised deltas) is staged in shared memory between the pass that finds the
// row's absmax and the pass that quantises it.  With two stages a worker's row is needed twice (for
// its absmax, then to be quantised with it): outer_sync_row1_kernel stages it in shared memory
// beside the running sum, so every replica (and error-feedback accumulator) is read from memory
// once; rows too long for two staged copies take outer_sync_row_kernel, which reads them twice.
// Arithmetic and order are those of the block kernels, so codes are bit-exact against the same reference.
constexpr int ROW_THREADS = 256;
constexpr int ROW_PIECES = 4;            // pieces of four columns a thread can hold in registers

__device__ __forceinline__ float block_max(float v, float* red) {
  v = warp_max(v);
  __syncthreads();                       // red may still be read from the previous reduction
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float m = red[0];
#pragma unroll
  for (int w = 1; w < ROW_THREADS / 32; ++w) m = fmaxf(m, red[w]);
  return m;
}

template <int QB>
__device__ __forceinline__ float quant_dequant1(float x, float amax, bool& bad) {
  constexpr float qmax = (QB == 8) ? 127.0f : (QB == 4 ? 7.0f : 1.0f);
  if (!(fabsf(x) <= FLT_MAX)) bad = true;
  if (!(amax > 0.0f && amax <= FLT_MAX)) return 0.0f;
  const float inv = __fdiv_rn(qmax, amax);
  const float scale = __fdiv_rn(amax, qmax);
  float r = rintf(__fmul_rn(x, inv));
  r = fminf(fmaxf(r, -qmax), qmax);
  return __fmul_rn(r, scale);
}

// Two quantisations per sync, every array read once.  Shared memory: xbuf[cols4] (the current
// worker's delta, or its error-feedback sum) and acc[cols4] (running sum of what the workers sent);
// every thread only ever touches the entries of its own columns, so the two arrays need no barrier
// of their own.  Pieces of four columns per thread (16-byte accesses when the row allows it).
// Without error feedback, rows of up to ROW_PIECES * ROW_THREADS pieces (4096 columns) run software-pipelined: theta stays
// in registers for the whole row, and the next worker's replica (and accumulator) is already on
// its way while the current worker's absmax is reduced over the CTA.
template <int QB, bool EF>
__global__ void __launch_bounds__(ROW_THREADS)
outer_sync_row1_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps,
                       float* const* __restrict__ efs, int K, int64_t n_rows, int64_t cols_pad, float eta,
                       float mu, float inv_k, float ef_beta, int* __restrict__ status) {
  extern __shared__ float rowbuf[];      // [cols_pad] xbuf, [cols_pad] acc
  __shared__ float red[ROW_THREADS / 32];
  __shared__ int vec_ok;
  const int64_t unit = blockIdx.x;
  if (unit >= n_rows) return;
  const int seg = find_seg(segs, n_segs, unit);
  const SyncSeg s = segs[seg];
  const int64_t row = unit - s.unit_begin;
  if (!MULOCO_IN_BOUNDS(seg >= 0 && seg < n_segs && row >= 0 && row < s.rows, status)) return;
  const int64_t cols = s.cols;
  const int64_t off0 = row * cols;
  float* const* rp = reps + s.rep_index;
  float* const* ep = EF ? efs + s.rep_index : nullptr;
  float* xbuf = rowbuf;
  float* accb = rowbuf + cols_pad;
  bool bad = false;
  float* tgp = s.theta_g + off0;
  float* up = s.u + off0;
  if (threadIdx.x == 0) {
    uintptr_t bits = (uintptr_t)tgp | (uintptr_t)up;
    for (int k = 0; k < K; ++k) {
      bits |= (uintptr_t)(rp[k] + off0);
      if (EF) bits |= (uintptr_t)(ep[k] + off0);
    }
    vec_ok = ((bits & 15) == 0) ? 1 : 0;
  }
  __syncthreads();
  const bool vec = vec_ok != 0;
  const int64_t n4 = (cols + 3) >> 2;    // pieces of four columns; the last one may be short
  auto nvalid_of = [&](int64_t c) { return (cols - c >= 4) ? 4 : (int)(cols - c); };
  auto load_theta = [&](int64_t c, bool v4, int nvalid, float (&t)[4]) {
    if (v4) {
      const float4 tt = *reinterpret_cast<const float4*>(tgp + c);
      t[0] = tt.x; t[1] = tt.y; t[2] = tt.z; t[3] = tt.w;
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q) t[q] = (q < nvalid) ? tgp[c + q] : 0.f;
    }
  };

  for (int64_t i = threadIdx.x; i < n4; i += ROW_THREADS)
    *reinterpret_cast<float4*>(accb + 4 * i) = make_float4(0.f, 0.f, 0.f, 0.f);

  if (!EF && n4 <= (int64_t)ROW_PIECES * ROW_THREADS) {
    // ---- pipelined (without error feedback: with it the accumulators double the registers in
    // flight and the occupancy lost costs more than the overlap gains: 0.75 against 0.83 of the copy
    // bandwidth at 4096 columns, K = 16): this thread's pieces are i = threadIdx.x + j * ROW_THREADS, j < ROW_PIECES ----
    float t[ROW_PIECES][4], rv[ROW_PIECES][4], ev[ROW_PIECES][4];
    auto fetch = [&](int k) {
#pragma unroll
      for (int j = 0; j < ROW_PIECES; ++j) {
        const int64_t i = threadIdx.x + (int64_t)j * ROW_THREADS;
#pragma unroll
        for (int q = 0; q < 4; ++q) { rv[j][q] = 0.f; ev[j][q] = 0.f; }
        if (i < n4) {
          const int64_t c = 4 * i;
          const int nvalid = nvalid_of(c);
          const bool v4 = vec && nvalid == 4;
          load4(rp[k] + off0 + c, v4, nvalid, rv[j]);
          if (EF) load4(ep[k] + off0 + c, v4, nvalid, ev[j]);
        }
      }
    };
#pragma unroll
    for (int j = 0; j < ROW_PIECES; ++j) {
      const int64_t i = threadIdx.x + (int64_t)j * ROW_THREADS;
#pragma unroll
      for (int q = 0; q < 4; ++q) t[j][q] = 0.f;
      if (i < n4) load_theta(4 * i, vec && nvalid_of(4 * i) == 4, nvalid_of(4 * i), t[j]);
    }
    fetch(0);
    for (int k = 0; k < K; ++k) {
      float lm = 0.f;
#pragma unroll
      for (int j = 0; j < ROW_PIECES; ++j) {
        const int64_t i = threadIdx.x + (int64_t)j * ROW_THREADS;
        if (i < n4) {
          const int64_t c = 4 * i;
          const int nvalid = nvalid_of(c);
          float x[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float d = __fsub_rn(t[j][q], rv[j][q]);
            x[q] = EF ? __fadd_rn(__fmul_rn(ef_beta, ev[j][q]), d) : d;
            if (q >= nvalid) x[q] = 0.f;
            const float a = fabsf(x[q]);
            if (!(a <= FLT_MAX)) bad = true;
            lm = fmaxf(lm, a);
          }
          *reinterpret_cast<float4*>(xbuf + c) = make_float4(x[0], x[1], x[2], x[3]);
        }
      }
      if (k + 1 < K) fetch(k + 1);       // in flight during the reduction and the quantising pass
      const float amax = block_max(lm, red);
#pragma unroll
      for (int j = 0; j < ROW_PIECES; ++j) {
        const int64_t i = threadIdx.x + (int64_t)j * ROW_THREADS;
        if (i < n4) {
          const int64_t c = 4 * i;
          const int nvalid = nvalid_of(c);
          const bool v4 = vec && nvalid == 4;
          const float4 xv = *reinterpret_cast<const float4*>(xbuf + c);
          float4 av = *reinterpret_cast<const float4*>(accb + c);
          const float x[4] = {xv.x, xv.y, xv.z, xv.w};
          float sent[4], en[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            sent[q] = quant_dequant1<QB>(x[q], amax, bad);
            en[q] = __fsub_rn(x[q], sent[q]);
          }
          if (EF) store4(ep[k] + off0 + c, v4, nvalid, en);
          av.x = __fadd_rn(av.x, sent[0]); av.y = __fadd_rn(av.y, sent[1]);
          av.z = __fadd_rn(av.z, sent[2]); av.w = __fadd_rn(av.w, sent[3]);
          *reinterpret_cast<float4*>(accb + c) = av;
        }
      }
    }
  } else {
    for (int k = 0; k < K; ++k) {
      float* r = rp[k] + off0;
      float* e = EF ? ep[k] + off0 : nullptr;
      float lm = 0.f;
      for (int64_t i = threadIdx.x; i < n4; i += ROW_THREADS) {
        const int64_t c = 4 * i;
        const int nvalid = nvalid_of(c);
        const bool v4 = vec && nvalid == 4;
        float t[4], rv[4], ev[4] = {0.f, 0.f, 0.f, 0.f}, x[4];
        load_theta(c, v4, nvalid, t);                     // read K times: a cache hit after the first
        load4(r + c, v4, nvalid, rv);
        if (EF) load4(e + c, v4, nvalid, ev);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float d = __fsub_rn(t[q], rv[q]);
          x[q] = EF ? __fadd_rn(__fmul_rn(ef_beta, ev[q]), d) : d;
          if (q >= nvalid) x[q] = 0.f;
          const float a = fabsf(x[q]);
          if (!(a <= FLT_MAX)) bad = true;
          lm = fmaxf(lm, a);
        }
        *reinterpret_cast<float4*>(xbuf + c) = make_float4(x[0], x[1], x[2], x[3]);
      }
      const float amax = block_max(lm, red);
      for (int64_t i = threadIdx.x; i < n4; i += ROW_THREADS) {
        const int64_t c = 4 * i;
        const int nvalid = nvalid_of(c);
        const bool v4 = vec && nvalid == 4;
        const float4 xv = *reinterpret_cast<const float4*>(xbuf + c);
        float4 av = *reinterpret_cast<const float4*>(accb + c);
        const float x[4] = {xv.x, xv.y, xv.z, xv.w};
        float sent[4], en[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          sent[q] = quant_dequant1<QB>(x[q], amax, bad);
          en[q] = __fsub_rn(x[q], sent[q]);
        }
        if (EF) store4(e + c, v4, nvalid, en);
        av.x = __fadd_rn(av.x, sent[0]); av.y = __fadd_rn(av.y, sent[1]);
        av.z = __fadd_rn(av.z, sent[2]); av.w = __fadd_rn(av.w, sent[3]);
        *reinterpret_cast<float4*>(accb + c) = av;
      }
    }
  }
  // the mean, its absmax, the second quantisation, the outer step, the broadcast
  float lm = 0.f;
  for (int64_t i = threadIdx.x; i < n4; i += ROW_THREADS) {
    float4 av = *reinterpret_cast<const float4*>(accb + 4 * i);
    av.x = __fmul_rn(av.x, inv_k); av.y = __fmul_rn(av.y, inv_k);
    av.z = __fmul_rn(av.z, inv_k); av.w = __fmul_rn(av.w, inv_k);
    *reinterpret_cast<float4*>(accb + 4 * i) = av;
    lm = fmaxf(fmaxf(lm, fabsf(av.x)), fmaxf(fabsf(av.y), fmaxf(fabsf(av.z), fabsf(av.w))));
  }
  const float amax = block_max(lm, red);
  for (int64_t i = threadIdx.x; i < n4; i += ROW_THREADS) {
    const int64_t c = 4 * i;
    const int nvalid = nvalid_of(c);
    const bool v4 = vec && nvalid == 4;
    const float4 av = *reinterpret_cast<const float4*>(accb + c);
    const float m4[4] = {av.x, av.y, av.z, av.w};
    float t[4], uu[4], un[4], tn[4];
    load_theta(c, v4, nvalid, t);
    load4(up + c, v4, nvalid, uu);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float psi = quant_dequant1<QB>(m4[q], amax, bad);
      const float epq = eta * psi;
      un[q] = fmaf(mu, uu[q], epq);
      tn[q] = t[q] - fmaf(mu, un[q], epq);
    }
    store4(up + c, v4, nvalid, un);
    store4(tgp + c, v4, nvalid, tn);
    for (int k = 0; k < K; ++k) store4(rp[k] + off0 + c, v4, nvalid, tn);
  }
  if (__syncthreads_or(bad) && threadIdx.x == 0) atomicOr(status, ST_NONFINITE);
}

template <int QB, bool TWO, bool EF>
__global__ void __launch_bounds__(ROW_THREADS)
outer_sync_row_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps,
                      float* const* __restrict__ efs, int K, int64_t n_rows, float eta, float mu, float inv_k,
                      float ef_beta, int* __restrict__ status) {
  extern __shared__ float rowbuf[];      // [cols] staged values, then [K] per-worker absmax
  __shared__ float red[ROW_THREADS / 32];
  const int64_t unit = blockIdx.x;
  if (unit >= n_rows) return;
  const int seg = find_seg(segs, n_segs, unit);
  const SyncSeg s = segs[seg];
  const int64_t row = unit - s.unit_begin;
  if (!MULOCO_IN_BOUNDS(seg >= 0 && seg < n_segs && row >= 0 && row < s.rows, status)) return;
  const int64_t cols = s.cols;
  const int64_t off0 = row * cols;
  float* const* rp = reps + s.rep_index;
  float* const* ep = EF ? efs + s.rep_index : nullptr;
  float* amax_k = rowbuf + cols;
  bool bad = false;
  const float* tgp = s.theta_g + off0;

  if (TWO) {
    // pass A: every worker's absmax over the row
    for (int k = 0; k < K; ++k) {
      const float* r = rp[k] + off0;
      const float* e = EF ? ep[k] + off0 : nullptr;
      float lm = 0.f;
      for (int64_t c = threadIdx.x; c < cols; c += ROW_THREADS) {
        const float d = __fsub_rn(tgp[c], r[c]);
        const float x = EF ? __fadd_rn(__fmul_rn(ef_beta, e[c]), d) : d;
        const float a = fabsf(x);
        if (!(a <= FLT_MAX)) bad = true;
        lm = fmaxf(lm, a);
      }
      const float m = block_max(lm, red);
      if (threadIdx.x == 0) amax_k[k] = m;
    }
    __syncthreads();
    // pass B: quantise every worker's value with its own scale, mean in fp32, stage the mean
    float lm = 0.f;
    for (int64_t c = threadIdx.x; c < cols; c += ROW_THREADS) {
      const float t = tgp[c];
      float acc = 0.f;
      for (int k = 0; k < K; ++k) {
        const float d = __fsub_rn(t, rp[k][off0 + c]);
        float x = d;
        if (EF) x = __fadd_rn(__fmul_rn(ef_beta, ep[k][off0 + c]), d);
        const float sent = quant_dequant1<QB>(x, amax_k[k], bad);
        if (EF) ep[k][off0 + c] = __fsub_rn(x, sent);
        acc = __fadd_rn(acc, sent);
      }
      const float mean = __fmul_rn(acc, inv_k);
      rowbuf[c] = mean;
      lm = fmaxf(lm, fabsf(mean));
    }
    const float amax = block_max(lm, red);
    for (int64_t c = threadIdx.x; c < cols; c += ROW_THREADS) rowbuf[c] = quant_dequant1<QB>(rowbuf[c], amax, bad);
  } else {
    float lm = 0.f;
    for (int64_t c = threadIdx.x; c < cols; c += ROW_THREADS) {
      const float t = tgp[c];
      float acc = 0.f;
      for (int k = 0; k < K; ++k) acc = __fadd_rn(acc, __fsub_rn(t, rp[k][off0 + c]));
      const float psi = __fmul_rn(acc, inv_k);
      rowbuf[c] = psi;
      const float a = fabsf(psi);
      if (!(a <= FLT_MAX)) bad = true;
      lm = fmaxf(lm, a);
    }
    const float amax = block_max(lm, red);
    for (int64_t c = threadIdx.x; c < cols; c += ROW_THREADS) rowbuf[c] = quant_dequant1<QB>(rowbuf[c], amax, bad);
  }
  // each thread re-reads only the entries it wrote: no barrier needed before the update pass
  for (int64_t c = threadIdx.x; c < cols; c += ROW_THREADS) {
    const float psi = rowbuf[c];
    const float t = tgp[c];
    const float ep_ = eta * psi;
    const float un = fmaf(mu, s.u[off0 + c], ep_);
    const float tn = t - fmaf(mu, un, ep_);
    s.u[off0 + c] = un;
    s.theta_g[off0 + c] = tn;
    for (int k = 0; k < K; ++k) rp[k][off0 + c] = tn;
  }
  if (__syncthreads_or(bad) && threadIdx.x == 0) atomicOr(status, ST_NONFINITE);
}

__global__ void pseudograd_kernel(const float* __restrict__ tg, float* const* __restrict__ reps, int K,
                                  int64_t n, float inv_k, float* __restrict__ out) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) {
    const float t = tg[i];
    float acc = 0.f;
    for (int k = 0; k < K; ++k) acc = __fadd_rn(acc, __fsub_rn(t, reps[k][i]));
    out[i] = __fmul_rn(acc, inv_k);
  }
}

template <int QB>
__global__ void quantize_kernel(const float* __restrict__ psi, int64_t rows, int64_t cols, int block,
                                int64_t nblk, int8_t* __restrict__ codes, float* __restrict__ scales,
                                float* __restrict__ deq, int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int64_t n_units = rows * nblk;
  bool bad = false;
  for (int64_t unit = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); unit < n_units;
       unit += (int64_t)gridDim.x * (blockDim.x >> 5)) {
    const int64_t row = unit / nblk, blk = unit - row * nblk;
    const int64_t col0 = blk * block + lane * 4;
    int64_t blk_end = (blk + 1) * block;
    if (blk_end > cols) blk_end = cols;
    int nvalid = (int)(blk_end - col0);
    nvalid = nvalid < 0 ? 0 : (nvalid > 4 ? 4 : nvalid);
    const int64_t off = row * cols + col0;
    float x[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) x[e] = (e < nvalid) ? psi[off + e] : 0.f;
    int q[4]; float sc;
    quant_dequant4<QB>(x, nvalid, q, sc, bad);
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (e < nvalid) {
        if (codes) codes[off + e] = (int8_t)q[e];
        if (deq) deq[off + e] = x[e];
      }
    if (scales && lane == 0) scales[row * nblk + blk] = sc;
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, ST_NONFINITE);
}

__global__ void broadcast_kernel(const float* __restrict__ src, float* const* __restrict__ dst, int K,
                                 int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) {
    const float v = src[i];
    for (int k = 0; k < K; ++k) dst[k][i] = v;
  }
}

template <int QB>
void launch_sync_q(cudaStream_t st, dim3 grid, const SyncSeg* segs, int n_segs, float* const* reps,
                   int K, int64_t n_units, int64_t upc, int block, float eta, float mu, float inv_k,
                   int* status) {
#define MULOCO_SYNC_CASE(KT)                                                                      \
  outer_sync_kernel<KT, QB><<<grid, SYNC_THREADS, 0, st>>>(segs, n_segs, reps, K, n_units, upc,   \
                                                           block, eta, mu, inv_k, status)
  switch (K) {
    case 1: MULOCO_SYNC_CASE(1); break;
    case 2: MULOCO_SYNC_CASE(2); break;
    case 4: MULOCO_SYNC_CASE(4); break;
    case 8: MULOCO_SYNC_CASE(8); break;
    case 16: MULOCO_SYNC_CASE(16); break;
    default: MULOCO_SYNC_CASE(0); break;
  }
#undef MULOCO_SYNC_CASE
}

// ---------------------------------------------------------------------------
// Worker-sharded outer synchronisation: the workers are partitioned over G GPUs and the all-reduce
// of the outer delta (Algorithm 1) is taken apart into a reduce-scatter and an all-gather (Section 2,
// "Collectives for compressed communication"; Appendix, "Assumptions around the collective used").
// Three passes on each GPU, the two collectives between them are the caller's:
//   delta     : S = sum over this GPU's workers of (theta - theta_k) (fp32, k ascending; with two
//               quantisation stages every worker's delta, or error-feedback sum, is quantised ->
//               dequantised first)                                 -> staging buffer, then reduce-scatter
//   step      : on this GPU's shard: Psi = (sum over all GPUs) * 1/K_total, the (second)
//               quantisation, u and theta updated in place      -> new theta of the shard, then all-gather
//   broadcast : theta and every local replica <- gathered theta.
// The staging buffers are unit-major with a fixed stride of 128 floats per unit (a unit is a
// block of the quantiser, at most 128 elements of one row; lanes beyond a short block hold zeros), so
// a shard is a range of whole units and every GPU gets the same count.
// ---------------------------------------------------------------------------
struct UnitPos {
  int64_t off;      // element offset of this lane's four values inside the tensor
  int nvalid;
  bool vec;
};

__device__ __forceinline__ UnitPos unit_pos(const SyncSeg& s, int64_t unit, int block, int lane) {
  const int64_t ul = unit - s.unit_begin;
  const int64_t row = ul / s.nblk;
  const int64_t blk = ul - row * s.nblk;
  const int64_t col0 = blk * block + lane * 4;
  int64_t blk_end = (blk + 1) * block;
  if (blk_end > s.cols) blk_end = s.cols;
  int nvalid = (int)(blk_end - col0);
  nvalid = nvalid < 0 ? 0 : (nvalid > 4 ? 4 : nvalid);
  UnitPos p;
  p.off = row * s.cols + col0;
  p.nvalid = nvalid;
  p.vec = (nvalid == 4) && ((s.cols & 3) == 0) && ((((uintptr_t)s.theta_g | (uintptr_t)s.u) & 15) == 0);
  return p;
}

template <int QB, bool TWO, bool EF>
__global__ void __launch_bounds__(SYNC_THREADS)
shard_delta_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps,
                   float* const* __restrict__ efs, int K, int64_t n_units, int64_t units_per_cta, int block,
                   float ef_beta, float* __restrict__ stage, int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t cta_begin = (int64_t)blockIdx.x * units_per_cta;
  int64_t cta_end = cta_begin + units_per_cta;
  if (cta_end > n_units) cta_end = n_units;
  bool bad = false;
  for (int64_t unit = cta_begin + warp; unit < cta_end; unit += SYNC_WARPS) {
    const int seg = find_seg(segs, n_segs, unit);
    if (!MULOCO_IN_BOUNDS(seg >= 0 && seg < n_segs, status)) return;
    const SyncSeg s = segs[seg];
    if (!MULOCO_IN_BOUNDS(unit - s.unit_begin < s.rows * s.nblk, status)) return;
    UnitPos u = unit_pos(s, unit, block, lane);
    float* const* rp = reps + s.rep_index;
    float* const* ep = EF ? efs + s.rep_index : nullptr;
    for (int k = 0; k < K; ++k) {
      u.vec = u.vec && ((((uintptr_t)rp[k]) & 15) == 0);
      if (EF) u.vec = u.vec && ((((uintptr_t)ep[k]) & 15) == 0);
    }
    float tg[4] = {0.f, 0.f, 0.f, 0.f}, acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (u.nvalid > 0) load4(s.theta_g + u.off, u.vec, u.nvalid, tg);
    for (int k0 = 0; k0 < K; k0 += 4) {
      float r[4][4], e[EF ? 4 : 1][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int q = 0; q < 4; ++q) { r[j][q] = 0.f; e[EF ? j : 0][q] = 0.f; }
        if (k0 + j < K && u.nvalid > 0) {
          load4(rp[k0 + j] + u.off, u.vec, u.nvalid, r[j]);
          if (EF) load4(ep[k0 + j] + u.off, u.vec, u.nvalid, e[EF ? j : 0]);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (k0 + j < K) {              // uniform over the warp: the block reduction needs every lane
          float x[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float d = __fsub_rn(tg[q], r[j][q]);
            x[q] = EF ? __fadd_rn(__fmul_rn(ef_beta, e[EF ? j : 0][q]), d) : d;
          }
          float sent[4] = {x[0], x[1], x[2], x[3]};
          if (TWO) {
            int qq[4]; float sc;
            quant_dequant4<(QB == 0 ? 8 : QB)>(sent, u.nvalid, qq, sc, bad);
            if (EF && u.nvalid > 0) {
              float en[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) en[q] = __fsub_rn(x[q], sent[q]);
              store4(ep[k0 + j] + u.off, u.vec, u.nvalid, en);
            }
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) acc[q] = __fadd_rn(acc[q], sent[q]);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (q >= u.nvalid) acc[q] = 0.f;
    __stcs(reinterpret_cast<float4*>(stage + unit * 128 + lane * 4), make_float4(acc[0], acc[1], acc[2], acc[3]));
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, ST_NONFINITE);
}

template <int QB>
__global__ void __launch_bounds__(SYNC_THREADS)
shard_step_kernel(const SyncSeg* __restrict__ segs, int n_segs, int64_t n_units, int64_t unit_begin,
                  int64_t unit_count, int block, float eta, float mu, float inv_k_total,
                  const float* __restrict__ reduced, float* __restrict__ theta_out, int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int64_t j = (int64_t)blockIdx.x * SYNC_WARPS + (threadIdx.x >> 5);
  if (j >= unit_count) return;
  const int64_t unit = unit_begin + j;
  bool bad = false;
  float tn[4] = {0.f, 0.f, 0.f, 0.f};
  if (unit < n_units) {                   // beyond: padding units that make the shards equal
    const int seg = find_seg(segs, n_segs, unit);
    if (!MULOCO_IN_BOUNDS(seg >= 0 && seg < n_segs, status)) return;
    const SyncSeg s = segs[seg];
    if (!MULOCO_IN_BOUNDS(unit - s.unit_begin < s.rows * s.nblk, status)) return;
    const UnitPos u = unit_pos(s, unit, block, lane);
    const float4 rv = __ldcs(reinterpret_cast<const float4*>(reduced + j * 128 + lane * 4));
    float psi[4] = {__fmul_rn(rv.x, inv_k_total), __fmul_rn(rv.y, inv_k_total), __fmul_rn(rv.z, inv_k_total),
                    __fmul_rn(rv.w, inv_k_total)};
    if (QB != 0) {
      int q[4]; float sc;
      quant_dequant4<(QB == 0 ? 8 : QB)>(psi, u.nvalid, q, sc, bad);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (e < u.nvalid && !(fabsf(psi[e]) <= FLT_MAX)) bad = true;
    }
    if (u.nvalid > 0) {
      float tg[4], uu[4], un[4];
      load4(s.theta_g + u.off, u.vec, u.nvalid, tg);
      load4(s.u + u.off, u.vec, u.nvalid, uu);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float ep = eta * psi[e];
        un[e] = fmaf(mu, uu[e], ep);
        tn[e] = tg[e] - fmaf(mu, un[e], ep);
      }
      store4(s.u + u.off, u.vec, u.nvalid, un);
      store4(s.theta_g + u.off, u.vec, u.nvalid, tn);
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (e >= u.nvalid) tn[e] = 0.f;
    }
  }
  __stcs(reinterpret_cast<float4*>(theta_out + j * 128 + lane * 4), make_float4(tn[0], tn[1], tn[2], tn[3]));
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, ST_NONFINITE);
}

__global__ void __launch_bounds__(SYNC_THREADS)
shard_broadcast_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps, int K,
                       int64_t n_units, int64_t units_per_cta, int block, const float* __restrict__ theta_all,
                       int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t cta_begin = (int64_t)blockIdx.x * units_per_cta;
  int64_t cta_end = cta_begin + units_per_cta;
  if (cta_end > n_units) cta_end = n_units;
  for (int64_t unit = cta_begin + warp; unit < cta_end; unit += SYNC_WARPS) {
    const int seg = find_seg(segs, n_segs, unit);
    if (!MULOCO_IN_BOUNDS(seg >= 0 && seg < n_segs, status)) return;
    const SyncSeg s = segs[seg];
    if (!MULOCO_IN_BOUNDS(unit - s.unit_begin < s.rows * s.nblk, status)) return;
    UnitPos u = unit_pos(s, unit, block, lane);
    if (u.nvalid == 0) continue;
    float* const* rp = reps + s.rep_index;
    for (int k = 0; k < K; ++k) u.vec = u.vec && ((((uintptr_t)rp[k]) & 15) == 0);
    const float4 v = __ldcs(reinterpret_cast<const float4*>(theta_all + unit * 128 + lane * 4));
    const float tn[4] = {v.x, v.y, v.z, v.w};
    store4(s.theta_g + u.off, u.vec, u.nvalid, tn);
    for (int k = 0; k < K; ++k) store4(rp[k] + u.off, u.vec, u.nvalid, tn);
  }
}

// Plain data parallelism as a special case (Section 5, the DP baselines): one worker, eta_out = 1,
// mu = 0, no compression.  Eq. 3 then gives theta <- theta - (theta - theta_1) = theta_1 in exact
// arithmetic, so the worker's parameters are copied (exactly: H plain inner steps), u <- theta - theta_1,
// and the replica is left as it is: 16 instead of 24 bytes per parameter.
__global__ void __launch_bounds__(SYNC_THREADS)
dp_sync_kernel(const SyncSeg* __restrict__ segs, int n_segs, float* const* __restrict__ reps, int64_t n_units,
               int64_t units_per_cta, int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int64_t cta_begin = (int64_t)blockIdx.x * units_per_cta;
  int64_t cta_end = cta_begin + units_per_cta;
  if (cta_end > n_units) cta_end = n_units;
  bool bad = false;
  for (int64_t unit = cta_begin + warp; unit < cta_end; unit += SYNC_WARPS) {
    const int seg = find_seg(segs, n_segs, unit);
    if (!MULOCO_IN_BOUNDS(seg >= 0 && seg < n_segs, status)) return;
    const SyncSeg s = segs[seg];
    if (!MULOCO_IN_BOUNDS(unit - s.unit_begin < s.rows * s.nblk, status)) return;
    UnitPos u = unit_pos(s, unit, 128, lane);
    if (u.nvalid == 0) continue;
    float* r1 = reps[s.rep_index];
    u.vec = u.vec && ((((uintptr_t)r1) & 15) == 0);
    float tg[4], r[4], psi[4];
    load4(s.theta_g + u.off, u.vec, u.nvalid, tg);
    load4(r1 + u.off, u.vec, u.nvalid, r);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      psi[e] = __fsub_rn(tg[e], r[e]);
      if (e < u.nvalid && !(fabsf(psi[e]) <= FLT_MAX)) bad = true;
    }
    store4(s.u + u.off, u.vec, u.nvalid, psi);
    store4(s.theta_g + u.off, u.vec, u.nvalid, r);
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, ST_NONFINITE);
}

}  // namespace

void launch_outer_sync(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas,
                       int K, int64_t n_units, int block, int quant_bits, float outer_lr, float mu,
                       int* status, int n_sms, int stages, float* const* ef, float ef_beta) {
  (void)n_sms;
  if (n_units <= 0) return;
  const int64_t upc = (int64_t)SYNC_WARPS * SYNC_UNITS_PER_WARP;
  const int64_t ctas = (n_units + upc - 1) / upc;
  const float inv_k = 1.0f / (float)K;
  dim3 grid((unsigned)ctas);
  if (stages == 2 && quant_bits != 0) {
#define MULOCO_SYNC2_CASE(QB)                                                                        \
  do {                                                                                             \
    if (ef)                                                                                        \
      outer_sync2_kernel<QB, true><<<grid, SYNC_THREADS, 0, st>>>(segs, n_segs, replicas, ef, K, n_units, upc, \
                                                                  block, outer_lr, mu, inv_k, ef_beta, status); \
    else                                                                                           \
      outer_sync2_kernel<QB, false><<<grid, SYNC_THREADS, 0, st>>>(segs, n_segs, replicas, ef, K, n_units, upc, \
                                                                   block, outer_lr, mu, inv_k, ef_beta, status); \
  } while (0)
    if (quant_bits == 8) MULOCO_SYNC2_CASE(8);
    else if (quant_bits == 4) MULOCO_SYNC2_CASE(4);
    else MULOCO_SYNC2_CASE(2);
#undef MULOCO_SYNC2_CASE
    return;
  }
  if (quant_bits == 8)
    launch_sync_q<8>(st, grid, segs, n_segs, replicas, K, n_units, upc, block, outer_lr, mu, inv_k, status);
  else if (quant_bits == 4)
    launch_sync_q<4>(st, grid, segs, n_segs, replicas, K, n_units, upc, block, outer_lr, mu, inv_k, status);
  else if (quant_bits == 2)
    launch_sync_q<2>(st, grid, segs, n_segs, replicas, K, n_units, upc, block, outer_lr, mu, inv_k, status);
  else
    launch_sync_q<0>(st, grid, segs, n_segs, replicas, K, n_units, upc, block, outer_lr, mu, inv_k, status);
}

void launch_dp_sync(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas, int64_t n_units,
                    int* status) {
  if (n_units <= 0) return;
  const int64_t upc = (int64_t)SYNC_WARPS * SYNC_UNITS_PER_WARP;
  dim3 grid((unsigned)((n_units + upc - 1) / upc));
  dp_sync_kernel<<<grid, SYNC_THREADS, 0, st>>>(segs, n_segs, replicas, n_units, upc, status);
}

void launch_shard_delta(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas, int K,
                        int64_t n_units, int block, int quant_bits, int stages, float* const* ef, float ef_beta,
                        float* stage, int* status) {
  if (n_units <= 0) return;
  const int64_t upc = (int64_t)SYNC_WARPS * SYNC_UNITS_PER_WARP;
  dim3 grid((unsigned)((n_units + upc - 1) / upc));
  const bool two = (stages == 2 && quant_bits != 0);
#define MULOCO_SD(QB, TWO, EF)                                                                             \
  shard_delta_kernel<QB, TWO, EF><<<grid, SYNC_THREADS, 0, st>>>(segs, n_segs, replicas, ef, K, n_units, upc, \
                                                                block, ef_beta, stage, status)
  if (!two) MULOCO_SD(0, false, false);
  else if (quant_bits == 8) { if (ef) MULOCO_SD(8, true, true); else MULOCO_SD(8, true, false); }
  else if (quant_bits == 4) { if (ef) MULOCO_SD(4, true, true); else MULOCO_SD(4, true, false); }
  else { if (ef) MULOCO_SD(2, true, true); else MULOCO_SD(2, true, false); }
#undef MULOCO_SD
}

void launch_shard_step(cudaStream_t st, const SyncSeg* segs, int n_segs, int64_t n_units, int64_t unit_begin,
                       int64_t unit_count, int block, int quant_bits, float outer_lr, float mu, float inv_k_total,
                       const float* reduced, float* theta_out, int* status) {
  if (unit_count <= 0) return;
  dim3 grid((unsigned)((unit_count + SYNC_WARPS - 1) / SYNC_WARPS));
#define MULOCO_SS(QB)                                                                                       \
  shard_step_kernel<QB><<<grid, SYNC_THREADS, 0, st>>>(segs, n_segs, n_units, unit_begin, unit_count, block, \
                                                        outer_lr, mu, inv_k_total, reduced, theta_out, status)
  if (quant_bits == 8) MULOCO_SS(8);
  else if (quant_bits == 4) MULOCO_SS(4);
  else if (quant_bits == 2) MULOCO_SS(2);
  else MULOCO_SS(0);
#undef MULOCO_SS
}

void launch_shard_broadcast(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas, int K,
                            int64_t n_units, int block, const float* theta_all, int* status) {
  if (n_units <= 0) return;
  const int64_t upc = (int64_t)SYNC_WARPS * SYNC_UNITS_PER_WARP;
  dim3 grid((unsigned)((n_units + upc - 1) / upc));
  shard_broadcast_kernel<<<grid, SYNC_THREADS, 0, st>>>(segs, n_segs, replicas, K, n_units, upc, block, theta_all,
                                                        status);
}

cudaError_t launch_outer_sync_rows(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas,
                                   int K, int64_t n_rows, int64_t max_cols, int quant_bits, float outer_lr,
                                   float mu, int* status, int stages, float* const* ef, float ef_beta) {
  if (n_rows <= 0) return cudaSuccess;
  const size_t smem = ((size_t)max_cols + (size_t)K) * sizeof(float);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  const float inv_k = 1.0f / (float)K;
  const bool two = (stages == 2);
  // two stages: two staged copies of the row (the worker's values and the running sum) when they fit
  const int64_t cols_pad = (max_cols + 3) / 4 * 4;
  const size_t smem1 = 2 * (size_t)cols_pad * sizeof(float);
  const bool single_read = two && smem1 <= 200 * 1024;
#define MULOCO_ROW_LAUNCH(QB, TWO, EF)                                                                   \
  do {                                                                                                   \
    cudaError_t e_ = cudaFuncSetAttribute(outer_sync_row_kernel<QB, TWO, EF>,                            \
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(200 * 1024)); \
    if (e_ != cudaSuccess) return e_;                                                                    \
    outer_sync_row_kernel<QB, TWO, EF><<<(unsigned)n_rows, ROW_THREADS, smem, st>>>(                     \
        segs, n_segs, replicas, ef, K, n_rows, outer_lr, mu, inv_k, ef_beta, status);                    \
  } while (0)
#define MULOCO_ROW1_LAUNCH(QB, EF)                                                                       \
  do {                                                                                                   \
    cudaError_t e_ = cudaFuncSetAttribute(outer_sync_row1_kernel<QB, EF>,                                \
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(200 * 1024)); \
    if (e_ != cudaSuccess) return e_;                                                                    \
    outer_sync_row1_kernel<QB, EF><<<(unsigned)n_rows, ROW_THREADS, smem1, st>>>(                        \
        segs, n_segs, replicas, ef, K, n_rows, cols_pad, outer_lr, mu, inv_k, ef_beta, status);          \
  } while (0)
#define MULOCO_ROW_BITS(QB)                                   \
  do {                                                        \
    if (single_read && ef) MULOCO_ROW1_LAUNCH(QB, true);      \
    else if (single_read) MULOCO_ROW1_LAUNCH(QB, false);      \
    else if (two && ef) MULOCO_ROW_LAUNCH(QB, true, true);    \
    else if (two) MULOCO_ROW_LAUNCH(QB, true, false);         \
    else MULOCO_ROW_LAUNCH(QB, false, false);                 \
  } while (0)
  if (quant_bits == 8) MULOCO_ROW_BITS(8);
  else if (quant_bits == 4) MULOCO_ROW_BITS(4);
  else MULOCO_ROW_BITS(2);
#undef MULOCO_ROW_BITS
#undef MULOCO_ROW1_LAUNCH
#undef MULOCO_ROW_LAUNCH
  return cudaGetLastError();
}

void launch_pseudogradient(cudaStream_t st, const float* theta_g, float* const* replicas, int K,
                           int64_t n, float* psi_out) {
  if (n <= 0) return;
  int blocks = (int)((n + 255) / 256 < 2048 ? (n + 255) / 256 : 2048);
  pseudograd_kernel<<<blocks, 256, 0, st>>>(theta_g, replicas, K, n, 1.0f / (float)K, psi_out);
}

void launch_quantize(cudaStream_t st, const float* psi, int64_t rows, int64_t cols, int block,
                     int bits, int8_t* codes, float* scales, float* dequant, int* status) {
  const int64_t nblk = (cols + block - 1) / block;
  const int64_t n_units = rows * nblk;
  if (n_units <= 0) return;
  int blocks = (int)((n_units + 7) / 8 < 4096 ? (n_units + 7) / 8 : 4096);
  if (bits == 8)
    quantize_kernel<8><<<blocks, 256, 0, st>>>(psi, rows, cols, block, nblk, codes, scales, dequant, status);
  else if (bits == 2)
    quantize_kernel<2><<<blocks, 256, 0, st>>>(psi, rows, cols, block, nblk, codes, scales, dequant, status);
  else
    quantize_kernel<4><<<blocks, 256, 0, st>>>(psi, rows, cols, block, nblk, codes, scales, dequant, status);
}

void launch_broadcast_init(cudaStream_t st, const float* src, float* const* dst_table, int K, int64_t n) {
  if (n <= 0) return;
  int blocks = (int)((n + 255) / 256 < 4096 ? (n + 255) / 256 : 4096);
  broadcast_kernel<<<blocks, 256, 0, st>>>(src, dst_table, K, n);
}

}  // namespace muloco
