// HBM-bound elementwise kernels of the inner step:
//   - Muon prologue: m <- beta m + g, NS input U staged as bf16/fp32 (transposed
//     when the tensor has more rows than columns), partial sums of U^2 for the
//     Frobenius norm (Section 2, "Muon").
//   - scale finalisation: r = 1 / (||U||_F + eps) per matrix, deterministic order.
//   - fused AdamW (Section 4.3) over a flat list of (worker, tensor) segments.
#include "internal.h"

namespace muloco {

namespace {

constexpr int PRO_TI = 32;    // tile rows of X (the s dimension)
constexpr int PRO_TJ = 128;   // tile cols of X (the l dimension)
constexpr int PRO_THREADS = 256;

__device__ __forceinline__ float load_g(const void* g, int64_t idx, int is_bf16) {
  return is_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(g)[idx])
                 : reinterpret_cast<const float*>(g)[idx];
}

template <typename XT>
__device__ __forceinline__ XT to_x(float v);
template <>
__device__ __forceinline__ float to_x<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 to_x<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ void store_x2(float* p, float a, float b) { *reinterpret_cast<float2*>(p) = make_float2(a, b); }
__device__ __forceinline__ void store_x2(__nv_bfloat16* p, float a, float b) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b);
}
__device__ __forceinline__ void store_x4(float* p, float4 u) { *reinterpret_cast<float4*>(p) = u; }
__device__ __forceinline__ void store_x4(__nv_bfloat16* p, float4 u) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(u.x, u.y), hi = __floats2bfloat162_rn(u.z, u.w);
  uint2 v;
  v.x = *reinterpret_cast<uint32_t*>(&lo);
  v.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = v;
}

// One CTA = one 32 x 128 tile of X (s x l view) of one matrix.
// The value that enters the sum of squares is the fp32 U (before bf16 rounding).
// BF16SRC: the source (gradient, or the standalone call's input) is bf16; only that instantiation
// carries the bf16 access shapes, so the fp32-source kernel keeps its register count.
template <typename XT, bool BF16SRC>
__global__ void __launch_bounds__(PRO_THREADS)
prologue_kernel(const MatDesc* __restrict__ mats, int64_t s, int64_t l, int src_mode, int g_is_bf16,
                float beta, int nesterov, XT* __restrict__ X, int64_t ldx, float* __restrict__ partials,
                int tiles_j, int n_part) {
  __shared__ float tile_raw[PRO_TJ * (PRO_TI + 1)];   // viewed as 128 x 33 or 64 x 65 floats, or 64 x 130 bf16
  float (*tile)[PRO_TI + 1] = reinterpret_cast<float (*)[PRO_TI + 1]>(tile_raw);
  __shared__ float red[PRO_THREADS / 32];
  const int mat = blockIdx.y;
  const MatDesc d = mats[mat];
  // Tile order follows the tensor's own memory order, so that the CTAs resident at one
  // time read neighbouring addresses: tj fastest for a tensor stored s x l, ti fastest for
  // one stored l x s (its rows are the j axis).  Tall tensors with an even s use 64 x 64 tiles
  // (two consecutive i per lane); the grid has max(#32x128 tiles, #64x64 tiles) CTAs per matrix
  // and the CTAs a tensor does not need write a zero partial sum.
  const bool pair_ok = ((((uintptr_t)d.m) & 7) == 0) &&
                       ((((uintptr_t)d.g) & ((src_mode == SRC_RAW_BF16 || (src_mode == SRC_MUON && g_is_bf16)) ? 3 : 7)) == 0);
  const bool src_is_bf16 = BF16SRC && ((src_mode == SRC_RAW_BF16) || (src_mode == SRC_MUON && g_is_bf16));
  // tall tensors with a bf16 source: 128 x 64 tiles, four consecutive i per lane (8-byte pieces of the
  // 2-byte stream, 256 bytes per warp and tensor row; the 64 x 64 path would read it in 128-byte pieces)
  const bool t128 = BF16SRC && d.transposed && src_is_bf16 && sizeof(XT) == 2 && ((s & 3) == 0) &&
                    ((((uintptr_t)d.g) & 7) == 0) && ((((uintptr_t)d.m) & 15) == 0);
  const bool t64 = !t128 && d.transposed && ((s & 1) == 0) && pair_ok;
  XT* Xm = X + (int64_t)mat * s * ldx;
  // bf16 sources of tensors stored s x l: 32 x 256 tiles, eight consecutive j per thread, so that the
  // 2-byte stream is read in 512-byte pieces per tile row like the 4-byte streams of the other paths
  const bool vec8 = BF16SRC && !d.transposed && src_is_bf16 && sizeof(XT) == 2 && ((l & 7) == 0) && ((ldx & 7) == 0) &&
                    ((((uintptr_t)d.g | (uintptr_t)d.m | (uintptr_t)Xm) & 15) == 0);
  const int tiles_i = t128 ? (int)((s + 127) / 128) : (t64 ? (int)((s + 63) / 64) : (int)((s + PRO_TI - 1) / PRO_TI));
  const int tiles_jj = (t64 || t128) ? (int)((l + 63) / 64) : (vec8 ? (int)((l + 255) / 256) : tiles_j);
  if ((int)blockIdx.x >= tiles_i * tiles_jj) {
    if (threadIdx.x == 0) partials[(int64_t)mat * n_part + blockIdx.x] = 0.f;
    return;
  }
  const int ti = d.transposed ? (int)(blockIdx.x % tiles_i) : (int)(blockIdx.x / tiles_jj);
  const int tj = d.transposed ? (int)(blockIdx.x / tiles_i) : (int)(blockIdx.x % tiles_jj);
  const int64_t i0 = (int64_t)ti * (t128 ? 128 : (t64 ? 64 : PRO_TI));
  const int64_t j0 = (int64_t)tj * ((t64 || t128) ? 64 : (vec8 ? 256 : PRO_TJ));
  float ss = 0.f;
  const int tid = threadIdx.x;

  auto produce = [&](int64_t idx) -> float {   // idx: element index in the tensor's own layout
    float u;
    if (src_mode == SRC_MUON) {
      const float g = load_g(d.g, idx, g_is_bf16);
      const float mn = fmaf(beta, d.m[idx], g);
      d.m[idx] = mn;
      u = nesterov ? fmaf(beta, mn, g) : mn;
    } else if (src_mode == SRC_RAW_F32) {
      u = reinterpret_cast<const float*>(d.g)[idx];
    } else {
      u = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(d.g)[idx]);
    }
    return u;
  };

  if (t128) {
    // tensor is l x s with a bf16 source: read rows j (128 consecutive i, four per lane), turn the tile
    // through shared memory (already rounded to bf16, which is what X holds), write rows i of X
    // (64 consecutive j per warp)
    __nv_bfloat16 (*t12)[130] = reinterpret_cast<__nv_bfloat16 (*)[130]>(tile_raw);
    static_assert(64 * 130 * 2 <= PRO_TJ * (PRO_TI + 1) * 4, "staging tile");
    const int lane = tid & 31, w = tid >> 5;
    const int64_t i = i0 + 4 * lane;
#pragma unroll
    for (int half = 0; half < 2; ++half) {          // four rows at a time: their loads before their stores
      uint2 graw[4];
      float4 mv[4];
      bool ok[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int64_t j = j0 + w + 8 * (half * 4 + r);
        ok[r] = (j < l) && (i < s);
        graw[r] = make_uint2(0u, 0u);
        mv[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (!ok[r]) continue;
        const int64_t idx = j * s + i;
        graw[r] = __ldcs(reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(d.g) + idx));
        if (src_mode == SRC_MUON) mv[r] = *reinterpret_cast<const float4*>(d.m + idx);
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int jj = w + 8 * (half * 4 + r);
        float u[4] = {0.f, 0.f, 0.f, 0.f};
        if (ok[r]) {
          const float g[4] = {__uint_as_float(graw[r].x << 16), __uint_as_float(graw[r].x & 0xFFFF0000u),
                              __uint_as_float(graw[r].y << 16), __uint_as_float(graw[r].y & 0xFFFF0000u)};
          if (src_mode == SRC_MUON) {
            const float mold[4] = {mv[r].x, mv[r].y, mv[r].z, mv[r].w};
            float mn[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              mn[e] = fmaf(beta, mold[e], g[e]);
              u[e] = nesterov ? fmaf(beta, mn[e], g[e]) : mn[e];
            }
            *reinterpret_cast<float4*>(d.m + (j0 + jj) * s + i) = make_float4(mn[0], mn[1], mn[2], mn[3]);
          } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) u[e] = g[e];
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) ss = fmaf(u[e], u[e], ss);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) t12[jj][4 * lane + e] = __float2bfloat16_rn(u[e]);
      }
    }
    __syncthreads();
    const int64_t j = j0 + 2 * lane;
#pragma unroll
    for (int r = 0; r < 16; ++r) {
      const int ii = w + 8 * r;
      const int64_t ix = i0 + ii;
      if (ix >= s || j >= l) continue;
      if constexpr (sizeof(XT) == 2) {
        const __nv_bfloat16 a0 = t12[2 * lane][ii], a1 = t12[2 * lane + 1][ii];
        if (j + 1 < l) {
          *reinterpret_cast<__nv_bfloat162*>(Xm + ix * ldx + j) = __halves2bfloat162(a0, a1);
        } else {
          Xm[ix * ldx + j] = a0;
        }
      }
    }
  } else if (t64) {
    // tensor is l x s: read rows j (64 consecutive i = 256 bytes per warp, two per lane), turn the
    // tile through shared memory, write rows i of X (64 consecutive j per warp)
    float (*t6)[65] = reinterpret_cast<float (*)[65]>(&tile[0][0]);
    const int lane = tid & 31, w = tid >> 5;
    const int64_t i = i0 + 2 * lane;
    const bool src_bf16 = (src_mode == SRC_RAW_BF16) || (src_mode == SRC_MUON && g_is_bf16);
    float2 gv[8], mv[8];
    bool ok[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const int64_t j = j0 + w + 8 * r;
      ok[r] = (j < l) && (i < s);
      gv[r] = make_float2(0.f, 0.f);
      mv[r] = gv[r];
      if (!ok[r]) continue;
      const int64_t idx = j * s + i;
      if (src_bf16) {
        const uint32_t raw = __ldcs(reinterpret_cast<const uint32_t*>(reinterpret_cast<const __nv_bfloat16*>(d.g) + idx));
        gv[r] = make_float2(__uint_as_float(raw << 16), __uint_as_float(raw & 0xFFFF0000u));
      } else {
        gv[r] = __ldcs(reinterpret_cast<const float2*>(reinterpret_cast<const float*>(d.g) + idx));
      }
      if (src_mode == SRC_MUON) mv[r] = *reinterpret_cast<const float2*>(d.m + idx);
    }
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const int jj = w + 8 * r;
      float2 u = make_float2(0.f, 0.f);
      if (ok[r]) {
        u = gv[r];
        if (src_mode == SRC_MUON) {
          float2 mn;
          mn.x = fmaf(beta, mv[r].x, gv[r].x);
          mn.y = fmaf(beta, mv[r].y, gv[r].y);
          *reinterpret_cast<float2*>(d.m + (j0 + jj) * s + i) = mn;
          if (nesterov) {
            u.x = fmaf(beta, mn.x, gv[r].x);
            u.y = fmaf(beta, mn.y, gv[r].y);
          } else {
            u = mn;
          }
        }
        ss = fmaf(u.x, u.x, ss);
        ss = fmaf(u.y, u.y, ss);
      }
      t6[jj][2 * lane] = u.x;
      t6[jj][2 * lane + 1] = u.y;
    }
    __syncthreads();
    const int64_t j = j0 + 2 * lane;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const int ii = w + 8 * r;
      const int64_t ix = i0 + ii;
      if (ix >= s || j >= l) continue;
      const float a0 = t6[2 * lane][ii], a1 = t6[2 * lane + 1][ii];
      if (j + 1 < l) {
        store_x2(Xm + ix * ldx + j, a0, a1);
      } else {
        Xm[ix * ldx + j] = to_x<XT>(a0);
      }
    }
  }
  const bool vec4 = !d.transposed && ((l & 3) == 0) && ((ldx & 3) == 0) &&
                    ((((uintptr_t)d.g | (uintptr_t)d.m) & 15) == 0) && ((((uintptr_t)Xm) & 15) == 0);
  if (t64 || t128) {
    // handled above
  } else if (vec8) {
    const int tx = tid & 31, ty = tid >> 5;   // 32 lanes x 8 columns, 8 warps x 4 rows
    const int64_t j = j0 + tx * 8;
#pragma unroll
    for (int half = 0; half < 2; ++half) {    // two rows at a time: all loads of both rows before their stores
      uint4 graw[2];
      float4 mo[2][2];
      bool ok[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int64_t i = i0 + ty + (half * 2 + r) * 8;
        ok[r] = (i < s) && (j < l);
        graw[r] = make_uint4(0u, 0u, 0u, 0u);
        mo[r][0] = make_float4(0.f, 0.f, 0.f, 0.f);
        mo[r][1] = mo[r][0];
        if (!ok[r]) continue;
        const int64_t idx = i * l + j;
        graw[r] = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(d.g) + idx));
        if (src_mode == SRC_MUON) {
          mo[r][0] = *reinterpret_cast<const float4*>(d.m + idx);
          mo[r][1] = *reinterpret_cast<const float4*>(d.m + idx + 4);
        }
      }
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        if (!ok[r]) continue;
        const int64_t i = i0 + ty + (half * 2 + r) * 8;
        const int64_t idx = i * l + j;
        const uint32_t w[4] = {graw[r].x, graw[r].y, graw[r].z, graw[r].w};
        float g[8], u[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          g[2 * q] = __uint_as_float(w[q] << 16);
          g[2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
        }
        if (src_mode == SRC_MUON) {
          const float mold[8] = {mo[r][0].x, mo[r][0].y, mo[r][0].z, mo[r][0].w,
                                 mo[r][1].x, mo[r][1].y, mo[r][1].z, mo[r][1].w};
          float mn[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            mn[e] = fmaf(beta, mold[e], g[e]);
            u[e] = nesterov ? fmaf(beta, mn[e], g[e]) : mn[e];
          }
          *reinterpret_cast<float4*>(d.m + idx) = make_float4(mn[0], mn[1], mn[2], mn[3]);
          *reinterpret_cast<float4*>(d.m + idx + 4) = make_float4(mn[4], mn[5], mn[6], mn[7]);
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) u[e] = g[e];
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) ss = fmaf(u[e], u[e], ss);
        store_x4(Xm + i * ldx + j, make_float4(u[0], u[1], u[2], u[3]));
        store_x4(Xm + i * ldx + j + 4, make_float4(u[4], u[5], u[6], u[7]));
      }
    }
  } else if (vec4) {
    // tensor is s x l with 16-byte aligned rows: four consecutive j per thread.  All loads of
    // the thread's four rows are issued before the first store (the stores to m would
    // otherwise order the later loads behind them).
    const int tx = tid & 31, ty = tid >> 5;   // 32 x 8
    constexpr int R = PRO_TI / 8;
    const int64_t j = j0 + tx * 4;
    const bool src_bf16 = (src_mode == SRC_RAW_BF16) || (src_mode == SRC_MUON && g_is_bf16);
    float4 g[R], mo[R];
    bool ok[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int64_t i = i0 + ty + r * 8;
      ok[r] = (i < s) && (j < l);
      g[r] = make_float4(0.f, 0.f, 0.f, 0.f);
      mo[r] = g[r];
      if (!ok[r]) continue;
      const int64_t idx = i * l + j;
      if (src_bf16) {
        const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(d.g) + idx));
        g[r] = make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u),
                           __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
      } else {
        g[r] = __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(d.g) + idx));
      }
      if (src_mode == SRC_MUON) mo[r] = *reinterpret_cast<const float4*>(d.m + idx);
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (!ok[r]) continue;
      const int64_t i = i0 + ty + r * 8;
      const int64_t idx = i * l + j;
      float4 u = g[r];
      if (src_mode == SRC_MUON) {
        float4 mn;
        mn.x = fmaf(beta, mo[r].x, g[r].x); mn.y = fmaf(beta, mo[r].y, g[r].y);
        mn.z = fmaf(beta, mo[r].z, g[r].z); mn.w = fmaf(beta, mo[r].w, g[r].w);
        *reinterpret_cast<float4*>(d.m + idx) = mn;
        if (nesterov) {
          u.x = fmaf(beta, mn.x, g[r].x); u.y = fmaf(beta, mn.y, g[r].y);
          u.z = fmaf(beta, mn.z, g[r].z); u.w = fmaf(beta, mn.w, g[r].w);
        } else {
          u = mn;
        }
      }
      ss = fmaf(u.x, u.x, ss); ss = fmaf(u.y, u.y, ss); ss = fmaf(u.z, u.z, ss); ss = fmaf(u.w, u.w, ss);
      store_x4(Xm + i * ldx + j, u);
    }
  } else if (!d.transposed) {
    // tensor is s x l: X[i][j] = T[i][j]; lanes run along j
    const int tx = tid & 31, ty = tid >> 5;   // 32 x 8
#pragma unroll
    for (int r = 0; r < PRO_TI / 8; ++r) {
      const int64_t i = i0 + ty + r * 8;
      if (i >= s) continue;
#pragma unroll
      for (int q = 0; q < PRO_TJ / 32; ++q) {
        const int64_t j = j0 + tx + q * 32;
        if (j < l) {
          const float u = produce(i * l + j);
          ss = fmaf(u, u, ss);
          Xm[i * ldx + j] = to_x<XT>(u);
        }
      }
    }
  } else {
    // tensor is l x s: X[i][j] = T[j][i]; read with lanes along i, write with lanes along j
    const int tx = tid & 31, ty = tid >> 5;
    const int64_t i = i0 + tx;
    constexpr int RB = 8;   // rows per batch: their loads are all issued before the first store
#pragma unroll 1
    for (int rb = 0; rb < PRO_TJ / 8; rb += RB) {
      float gv[RB], mv[RB];
      bool ok[RB];
#pragma unroll
      for (int q = 0; q < RB; ++q) {
        const int64_t j = j0 + ty + (rb + q) * 8;
        ok[q] = (j < l) && (i < s);
        gv[q] = 0.f; mv[q] = 0.f;
        if (!ok[q]) continue;
        const int64_t idx = j * s + i;
        if (src_mode == SRC_MUON) {
          gv[q] = load_g(d.g, idx, g_is_bf16);
          mv[q] = d.m[idx];
        } else if (src_mode == SRC_RAW_F32) {
          gv[q] = reinterpret_cast<const float*>(d.g)[idx];
        } else {
          gv[q] = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(d.g)[idx]);
        }
      }
#pragma unroll
      for (int q = 0; q < RB; ++q) {
        const int jj = ty + (rb + q) * 8;
        float u = 0.f;
        if (ok[q]) {
          u = gv[q];
          if (src_mode == SRC_MUON) {
            const float mn = fmaf(beta, mv[q], gv[q]);
            d.m[(j0 + jj) * s + i] = mn;
            u = nesterov ? fmaf(beta, mn, gv[q]) : mn;
          }
          ss = fmaf(u, u, ss);
        }
        tile[jj][tx] = u;
      }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < PRO_TI / 8; ++r) {
      const int ii = ty + r * 8;
      const int64_t i = i0 + ii;
      if (i >= s) continue;
#pragma unroll
      for (int q = 0; q < PRO_TJ / 32; ++q) {
        const int jj = tx + q * 32;
        const int64_t j = j0 + jj;
        if (j < l) Xm[i * ldx + j] = to_x<XT>(tile[jj][ii]);
      }
    }
  }
  // deterministic block reduction
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((tid & 31) == 0) red[tid >> 5] = ss;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < PRO_THREADS / 32; ++w) t += red[w];
    partials[(int64_t)mat * n_part + blockIdx.x] = t;
  }
}

__global__ void finalize_scales_kernel(const float* __restrict__ partials, int n_part, int n_mats,
                                       float eps, float2* __restrict__ scales, int* __restrict__ status) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= n_mats) return;
  const float* p = partials + (int64_t)warp * n_part;
  double acc = 0.0;
  for (int i = lane; i < n_part; i += 32) acc += (double)p[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) {
    const double r = 1.0 / (sqrt(acc) + (double)eps);
    scales[warp] = make_float2((float)(r * r), (float)r);
    // a NaN or infinity anywhere in the input (gradient or momentum) shows up here
    if (status && !(acc <= 1.0e300)) atomicOr(status, ST_NONFINITE);
  }
}

// ---------------------------------------------------------------------------
// AdamW
// ---------------------------------------------------------------------------
constexpr int ADAM_THREADS = 256;

__device__ __forceinline__ int find_adam_seg(const AdamSeg* __restrict__ segs, int n, int64_t unit) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (segs[mid].unit_begin <= unit) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ void adam_elem(float g, float& m, float& v, float& th, float beta1,
                                          float beta2, float eps, const AdamSeg& s) {
  m = fmaf(beta1, m, (1.0f - beta1) * g);
  v = fmaf(beta2, v, (1.0f - beta2) * g * g);
  const float mh = m * s.inv_bc1;
  const float denom = fmaf(sqrtf(v), s.inv_sqrt_bc2, eps);
  th = th - fmaf(s.lr, __fdiv_rn(mh, denom), s.lr_wd * th);
}

__global__ void __launch_bounds__(ADAM_THREADS)
adamw_kernel(const AdamSeg* __restrict__ segs, int n_segs, int64_t n_units, int g_is_bf16, float beta1,
             float beta2, float eps, int* __restrict__ status) {
  // a gradient that is not finite would poison m, v and theta for good: it is flagged (the step is
  // still applied, like every other kernel here: nothing aborts)
  bool bad = false;
  auto check = [&](float g) { bad |= !(fabsf(g) <= 3.402823466e38f); };
  for (int64_t unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
    const int si = find_adam_seg(segs, n_segs, unit);
    const AdamSeg s = segs[si];
    const int64_t base = (unit - s.unit_begin) * ADAM_UNIT;
    if (!MULOCO_IN_BOUNDS(si >= 0 && si < n_segs && base >= 0 && base < s.n, status)) continue;
    int64_t cnt = s.n - base;
    if (cnt > ADAM_UNIT) cnt = ADAM_UNIT;
    // 16-byte accesses when every stream allows it (bf16 gradients: 8 bytes for the same 4 elements)
    const bool vec = ((((uintptr_t)s.m | (uintptr_t)s.v | (uintptr_t)s.theta) & 15) == 0) &&
                     ((((uintptr_t)s.g) & (g_is_bf16 ? 7 : 15)) == 0);
    if (vec) {
      const float4* g4 = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(s.g) + base);
      const uint2* gb = reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(s.g) + base);
      float4* m4 = reinterpret_cast<float4*>(s.m + base);
      float4* v4 = reinterpret_cast<float4*>(s.v + base);
      float4* t4 = reinterpret_cast<float4*>(s.theta + base);
      const int n4 = (int)(cnt >> 2);
#pragma unroll
      for (int r = 0; r < ADAM_UNIT / 4 / ADAM_THREADS; ++r) {
        const int i = threadIdx.x + r * ADAM_THREADS;
        if (i < n4) {
          float4 g;
          if (g_is_bf16) {
            const uint2 raw = __ldcs(gb + i);
            g = make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u),
                            __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
          } else {
            g = __ldcs(g4 + i);
          }
          float4 m = m4[i], v = v4[i], t = t4[i];
          check(g.x); check(g.y); check(g.z); check(g.w);
          adam_elem(g.x, m.x, v.x, t.x, beta1, beta2, eps, s);
          adam_elem(g.y, m.y, v.y, t.y, beta1, beta2, eps, s);
          adam_elem(g.z, m.z, v.z, t.z, beta1, beta2, eps, s);
          adam_elem(g.w, m.w, v.w, t.w, beta1, beta2, eps, s);
          m4[i] = m; v4[i] = v; t4[i] = t;
        }
      }
      for (int64_t i = (int64_t)n4 * 4 + threadIdx.x; i < cnt; i += ADAM_THREADS) {
        float g = load_g(s.g, base + i, g_is_bf16);
        float m = s.m[base + i], v = s.v[base + i], t = s.theta[base + i];
        check(g);
        adam_elem(g, m, v, t, beta1, beta2, eps, s);
        s.m[base + i] = m; s.v[base + i] = v; s.theta[base + i] = t;
      }
    } else {
      for (int64_t i = threadIdx.x; i < cnt; i += ADAM_THREADS) {
        float g = load_g(s.g, base + i, g_is_bf16);
        float m = s.m[base + i], v = s.v[base + i], t = s.theta[base + i];
        check(g);
        adam_elem(g, m, v, t, beta1, beta2, eps, s);
        s.m[base + i] = m; s.v[base + i] = v; s.theta[base + i] = t;
      }
    }
  }
  if (status && __syncthreads_or(bad ? 1 : 0) && threadIdx.x == 0) atomicOr(status, ST_NONFINITE);
}

}  // namespace

int prologue_partials_per_matrix(int64_t s, int64_t l) {
  const int64_t a = ((s + PRO_TI - 1) / PRO_TI) * ((l + PRO_TJ - 1) / PRO_TJ);   // 32 x 128 tiles
  const int64_t b = ((s + 63) / 64) * ((l + 63) / 64);                          // 64 x 64 tiles (tall tensors)
  return (int)(a > b ? a : b);
}

void launch_prologue(cudaStream_t st, const MatDesc* mats, int n_mats, int64_t s, int64_t l,
                     int src_mode, int g_is_bf16, float beta, int nesterov, void* X, int x_is_f32,
                     int64_t ldx, float* partials) {
  if (n_mats <= 0) return;
  const int tiles_j = (int)((l + PRO_TJ - 1) / PRO_TJ);
  const int n_part = prologue_partials_per_matrix(s, l);
  for (int m0 = 0; m0 < n_mats; m0 += 65535) {
    const int nm = (n_mats - m0 < 65535) ? (n_mats - m0) : 65535;
    dim3 grid((unsigned)n_part, (unsigned)nm);
    const bool bf16_src = (src_mode == SRC_RAW_BF16) || (src_mode == SRC_MUON && g_is_bf16);
    if (x_is_f32)
      prologue_kernel<float, false><<<grid, PRO_THREADS, 0, st>>>(
          mats + m0, s, l, src_mode, g_is_bf16, beta, nesterov,
          reinterpret_cast<float*>(X) + (int64_t)m0 * s * ldx, ldx, partials + (int64_t)m0 * n_part,
          tiles_j, n_part);
    else if (bf16_src)
      prologue_kernel<__nv_bfloat16, true><<<grid, PRO_THREADS, 0, st>>>(
          mats + m0, s, l, src_mode, g_is_bf16, beta, nesterov,
          reinterpret_cast<__nv_bfloat16*>(X) + (int64_t)m0 * s * ldx, ldx,
          partials + (int64_t)m0 * n_part, tiles_j, n_part);
    else
      prologue_kernel<__nv_bfloat16, false><<<grid, PRO_THREADS, 0, st>>>(
          mats + m0, s, l, src_mode, g_is_bf16, beta, nesterov,
          reinterpret_cast<__nv_bfloat16*>(X) + (int64_t)m0 * s * ldx, ldx,
          partials + (int64_t)m0 * n_part, tiles_j, n_part);
  }
}

void launch_finalize_scales(cudaStream_t st, const float* partials, int n_part, int n_mats, float eps,
                            float2* scales, int* status) {
  if (n_mats <= 0) return;
  const int threads = 128;
  const int blocks = (n_mats * 32 + threads - 1) / threads;
  finalize_scales_kernel<<<blocks, threads, 0, st>>>(partials, n_part, n_mats, eps, scales, status);
}

void launch_adamw(cudaStream_t st, const AdamSeg* segs, int n_segs, int64_t n_units, int g_is_bf16,
                  float beta1, float beta2, float eps, int* status) {
  if (n_units <= 0 || n_segs <= 0) return;
  // one unit per CTA, launched in address order (the resident CTAs then share DRAM pages)
  int64_t blocks = n_units < 0x7fffffffLL ? n_units : 0x7fffffffLL;
  adamw_kernel<<<(unsigned)blocks, ADAM_THREADS, 0, st>>>(segs, n_segs, n_units, g_is_bf16, beta1,
                                                          beta2, eps, status);
}

}  // namespace muloco
