// Batched bf16 Newton-Schulz engine for sm_100a: tcgen05.mma with fp32
// accumulators in tensor memory, operands staged in shared memory by TMA
// (128-byte swizzle), mbarrier pipeline, warp-specialised persistent CTAs.
//
// One launch computes one of the three products of a Newton-Schulz iteration
// (Section 2, "Muon": X_j = p(X X^T) X, p(x) = a x + b x^3 + c x^5) for every
// matrix of a chunk; tiles of all matrices form one linear work list:
//   GRAM  : A  = r^2 X X^T      symmetric: only tiles touching the upper triangle,
//   POLY  : B  = b A + c A A    each stored directly and mirrored
//   APPLY : X' = r (a X + B X)
//   FINAL : as APPLY, result goes to the parameter update / output sink
// Operand forms: GRAM/POLY multiply a row-major matrix by its own transpose
// (both operands K-major); APPLY needs X with the contraction index as the slow
// axis, i.e. an MN-major B operand, so no transposed copy of X is ever made.
//
// CTA = 6 warps: warp 0 issues TMA loads, warp 1 allocates tensor memory and
// issues the MMAs, warps 2-5 run the epilogue (one 32-lane quarter of the
// accumulator each).  Two accumulators alternate so the epilogue of one tile
// overlaps the main loop of the next.  Every wait is bounded: when one runs out
// the kernel raises ST_TIMEOUT, all roles leave their loops, and the CTA frees
// its tensor memory and returns.
#include <cuda.h>
#include <stdio.h>
#include <string.h>

#include <vector>

#include "internal.h"
#include "sink.cuh"

namespace muloco {

namespace {

constexpr int BM = 128;          // tile rows (UMMA M)
constexpr int BK = 64;           // k slab per stage (64 bf16 = one 128-byte swizzle row)
constexpr int UMMA_K = 16;
constexpr int TC_THREADS = 192;
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;

template <int BN> struct TcCfg {
  static constexpr int STAGES = (BN == 256) ? 4 : 6;
  static constexpr uint32_t B_STAGE_BYTES = BN * BK * 2;
  static constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
  static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + 1024;   // + alignment slack
  static constexpr uint32_t TMEM_COLS = 2 * BN;                          // two accumulators
};

struct TcParams {
  int kind;
  int n_mats;
  int M, N, Kd;
  int n_tiles_per_mat;
  const int2* tiles;
  const __nv_bfloat16* Cin;
  int64_t ldc, strideC;
  __nv_bfloat16* D;
  int64_t ldd, strideD;
  float a, b, c;
  const float2* scales;
  const MatDesc* mats;
  int sink_mode;
  int64_t s, l;
  int* status;
};

// ----------------------------- PTX wrappers --------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait ran out, or another did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_timer_ns() - t0 > WAIT_LIMIT_NS) {
      *abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),
        "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),
        "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),
        "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), version 1.
// K-major operand  : rows of 64 bf16 (128 B) at 128 B pitch, 8-row groups 1024 B apart (SBO).
// MN-major operand : 64-element (128 B) runs along MN, 8 k-rows per 1024 B group (SBO),
//                    next 64-element MN atom `lbo` bytes further.
__device__ __forceinline__ uint64_t make_sdesc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// ------------------------------- the kernel --------------------------------
template <int BN, bool B_MN>
__global__ void __launch_bounds__(TC_THREADS, 1)
ns_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const TcParams p) {
  using Cfg = TcCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[STAGES];
  __shared__ __align__(8) uint64_t bar_empty[STAGES];
  __shared__ __align__(8) uint64_t bar_tfull[2];
  __shared__ __align__(8) uint64_t bar_tempty[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile int abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int total_tiles = p.n_mats * p.n_tiles_per_mat;
  const int num_kb = (p.Kd + BK - 1) / BK;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&bar_tfull[a]), 1);
      mbar_init(smem_u32(&bar_tempty[a]), 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&tmem_base_slot)),
                 "r"(Cfg::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    uint32_t stage = 0, phase = 0;
    bool alive = true;
    for (int tile = blockIdx.x; tile < total_tiles && alive; tile += gridDim.x) {
      const int mat = tile / p.n_tiles_per_mat;
      const int2 tt = p.tiles[tile - mat * p.n_tiles_per_mat];
      for (int kb = 0; kb < num_kb && alive; ++kb) {
        if (lane == 0) {
          if (mbar_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, &abort_flag)) {
            const uint32_t full = smem_u32(&bar_full[stage]);
            const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
            const uint32_t sb = sa + A_STAGE_BYTES;
            mbar_expect_tx(full, Cfg::STAGE_BYTES);
            tma_load_3d(sa, &tmA, full, kb * BK, tt.x * BM, mat);
            if (!B_MN) {
#pragma unroll
              for (int h = 0; h < BN / 128; ++h)
                tma_load_3d(sb + h * (128 * BK * 2), &tmB, full, kb * BK, tt.y * BN + h * 128, mat);
            } else {
#pragma unroll
              for (int q = 0; q < BN / 64; ++q)
                tma_load_3d(sb + q * (BK * 128), &tmB, full, tt.y * BN + q * 64, kb * BK, mat);
            }
          }
        }
        __syncwarp();
        alive = (abort_flag == 0);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((B_MN ? 1u : 0u) << 16) |
                               ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    uint32_t stage = 0, phase = 0;
    int local_tile = 0;
    bool alive = true;
    for (int tile = blockIdx.x; tile < total_tiles && alive; tile += gridDim.x, ++local_tile) {
      const int acc = local_tile & 1;
      const uint32_t acc_phase = (uint32_t)(local_tile >> 1) & 1u;
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
      if (lane == 0) {
        if (mbar_wait(smem_u32(&bar_tempty[acc]), acc_phase ^ 1u, &abort_flag)) tc_fence_after();
      }
      __syncwarp();
      alive = (abort_flag == 0);
      for (int kb = 0; kb < num_kb && alive; ++kb) {
        if (lane == 0) {
          if (mbar_wait(smem_u32(&bar_full[stage]), phase, &abort_flag)) {
            tc_fence_after();
            const uint32_t sa = smem_base + stage * Cfg::STAGE_BYTES;
            const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              const uint64_t adesc = make_sdesc(sa + k * (UMMA_K * 2), 16, 1024);
              const uint64_t bdesc = B_MN ? make_sdesc(sb + k * (UMMA_K * 128), BK * 128, 1024)
                                          : make_sdesc(sb + k * (UMMA_K * 2), 16, 1024);
              tc_mma_bf16(d_tmem, adesc, bdesc, idesc, (kb > 0 || k > 0) ? 1u : 0u);
            }
            tc_commit(smem_u32(&bar_empty[stage]));
          }
        }
        __syncwarp();
        alive = (abort_flag == 0);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (alive && lane == 0) tc_commit(smem_u32(&bar_tfull[acc]));
      __syncwarp();
    }
  } else {
    // -------------------------------- epilogue --------------------------------
    const int quarter = warp & 3;          // TMEM lanes [32*quarter, 32*quarter+32)
    const int row = quarter * 32 + lane;
    int local_tile = 0;
    bool alive = true;
    const bool sym = (p.kind == GEMM_GRAM || p.kind == GEMM_POLY);
    for (int tile = blockIdx.x; tile < total_tiles && alive; tile += gridDim.x, ++local_tile) {
      const int acc = local_tile & 1;
      const uint32_t acc_phase = (uint32_t)(local_tile >> 1) & 1u;
      const int mat = tile / p.n_tiles_per_mat;
      const int2 tt = p.tiles[tile - mat * p.n_tiles_per_mat];
      if (!mbar_wait(smem_u32(&bar_tfull[acc]), acc_phase, &abort_flag)) { alive = false; }
      alive = __all_sync(0xffffffffu, alive);
      if (!alive) break;
      tc_fence_after();
      const int64_t gi = (int64_t)tt.x * BM + row;
      const bool row_ok = gi < p.M;
      float sc = 1.f;
      if (p.scales) sc = (p.kind == GEMM_GRAM) ? p.scales[mat].x : p.scales[mat].y;
      const __nv_bfloat16* Cm = p.Cin ? p.Cin + (int64_t)mat * p.strideC : nullptr;
      __nv_bfloat16* Dm = p.D ? p.D + (int64_t)mat * p.strideD : nullptr;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        const int64_t gj0 = (int64_t)tt.y * BN + c * 32;
        if (gj0 >= p.N) break;                       // warp-uniform
        const int cb = (int)(gj0 / BM);              // 128-column block of this chunk
        if (sym && cb < tt.x) continue;              // lower-triangle block: its mirror image writes it
        uint32_t v[32];
        tc_ld32(t_row + (uint32_t)(c * 32), v);
        float f[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
        const bool full_chunk = (gj0 + 32 <= p.N);
        // ---- addend -----------------------------------------------------------
        if (p.kind != GEMM_GRAM) {
          float add[32];
          const bool vec_in = full_chunk && ((p.ldc & 7) == 0) && ((((uintptr_t)Cm) & 15) == 0);
          if (row_ok) {
            const __nv_bfloat16* src = Cm + gi * p.ldc + gj0;
            if (vec_in) {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const uint4 u = *reinterpret_cast<const uint4*>(src + q * 8);
                add[q * 8 + 0] = bf16_lo(u.x); add[q * 8 + 1] = bf16_hi(u.x);
                add[q * 8 + 2] = bf16_lo(u.y); add[q * 8 + 3] = bf16_hi(u.y);
                add[q * 8 + 4] = bf16_lo(u.z); add[q * 8 + 5] = bf16_hi(u.z);
                add[q * 8 + 6] = bf16_lo(u.w); add[q * 8 + 7] = bf16_hi(u.w);
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e) add[e] = (gj0 + e < p.N) ? __bfloat162float(src[e]) : 0.f;
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) add[e] = 0.f;
          }
          if (p.kind == GEMM_POLY) {
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] = fmaf(p.c, f[e], p.b * add[e]);
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] = sc * fmaf(p.a, add[e], f[e]);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) f[e] *= sc;
        }
        // ---- store --------------------------------------------------------------
        if (p.kind == GEMM_FINAL) {
          if (row_ok) {
            const MatDesc d = p.mats[mat];
            const bool fast = !d.transposed && p.sink_mode != SINK_STORE_BF16 && full_chunk &&
                              ((p.l & 3) == 0) && ((((uintptr_t)d.w) & 15) == 0);
            if (fast) {
              float4* w4 = reinterpret_cast<float4*>(reinterpret_cast<float*>(d.w) + gi * p.l + gj0);
              if (p.sink_mode == SINK_UPDATE_W) {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                  float4 w = w4[q];
                  w.x = fmaf(-d.lr_eff, f[q * 4 + 0], fmaf(-d.wd_term, w.x, w.x));
                  w.y = fmaf(-d.lr_eff, f[q * 4 + 1], fmaf(-d.wd_term, w.y, w.y));
                  w.z = fmaf(-d.lr_eff, f[q * 4 + 2], fmaf(-d.wd_term, w.z, w.z));
                  w.w = fmaf(-d.lr_eff, f[q * 4 + 3], fmaf(-d.wd_term, w.w, w.w));
                  w4[q] = w;
                }
              } else {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                  w4[q] = make_float4(f[q * 4 + 0], f[q * 4 + 1], f[q * 4 + 2], f[q * 4 + 3]);
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (gj0 + e < p.N) sink_element(d, p.sink_mode, p.s, p.l, gi, gj0 + e, f[e]);
            }
          }
        } else {
          if (row_ok) {
            __nv_bfloat16* dst = Dm + gi * p.ldd + gj0;
            const bool vec_out = full_chunk && ((p.ldd & 7) == 0) && ((((uintptr_t)Dm) & 15) == 0);
            if (vec_out) {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                uint4 u;
                u.x = pack_bf16x2(f[q * 8 + 0], f[q * 8 + 1]);
                u.y = pack_bf16x2(f[q * 8 + 2], f[q * 8 + 3]);
                u.z = pack_bf16x2(f[q * 8 + 4], f[q * 8 + 5]);
                u.w = pack_bf16x2(f[q * 8 + 6], f[q * 8 + 7]);
                *reinterpret_cast<uint4*>(dst + q * 8) = u;
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (gj0 + e < p.N) dst[e] = __float2bfloat16_rn(f[e]);
            }
            if (sym && cb > tt.x) {
              // mirror image: D[j][i] = D[i][j]; lanes hold consecutive i
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (gj0 + e < p.N) Dm[(gj0 + e) * p.ldd + gi] = __float2bfloat16_rn(f[e]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bar_tempty[acc]));
    }
  }

  // ------------------------------- teardown ----------------------------------
  if (abort_flag) {
    // give copies and MMAs still in flight time to land before memory is released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    if (threadIdx.x == 0) atomicOr(p.status, ST_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg::TMEM_COLS)
                 : "memory");
  }
}

// ------------------------------ host side ----------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(ptr);
  return fn;
}

// 3-D map over [n_slots][rows][cols] bf16 with row pitch ld; box = box_cols x box_rows x 1.
bool encode_map(CUtensorMap* out, void* base, int64_t cols, int64_t rows, int64_t n_slots, int64_t ld,
                int box_cols, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)n_slots};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)rows * (cuuint64_t)ld * 2};
  cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int BN, bool B_MN>
cudaError_t launch_one(cudaStream_t st, const CUtensorMap& a, const CUtensorMap& b, const TcParams& p,
                       int n_sms) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(ns_tc_kernel<BN, B_MN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)TcCfg<BN>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int total = p.n_mats * p.n_tiles_per_mat;
  const int grid = total < n_sms ? total : n_sms;
  ns_tc_kernel<BN, B_MN><<<grid, TC_THREADS, TcCfg<BN>::SMEM_BYTES, st>>>(a, b, p);
  return cudaGetLastError();
}

}  // namespace

struct TcGroupPlan {
  int64_t s, l, ldx, lds;
  int chunk;
  void* X[2];
  void* A;
  void* B;
  CUtensorMap x_k[2], x_mn[2], a_k, b_k;
  int bn_sym, bn_apply;
  int2* tiles_sym = nullptr;
  int n_tiles_sym = 0;
  int2* tiles_full = nullptr;
  int n_tiles_full = 0;
  int n_sms = 148;
};

int tc_num_sms() {
  static int n = 0;
  if (n) return n;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  return n;
}

TcGroupPlan* tc_plan_create(int64_t s, int64_t l, int chunk, void* X0, void* X1, int64_t ldx, void* A,
                            void* B, int64_t lds, char* err, size_t errlen) {
  TcGroupPlan* pl = new TcGroupPlan();
  pl->s = s; pl->l = l; pl->ldx = ldx; pl->lds = lds; pl->chunk = chunk;
  pl->X[0] = X0; pl->X[1] = X1; pl->A = A; pl->B = B;
  pl->n_sms = tc_num_sms();
  pl->bn_sym = (s > 128) ? 256 : 128;
  pl->bn_apply = (l > 128) ? 256 : 128;
  bool ok = true;
  for (int i = 0; i < 2; ++i) {
    ok = ok && encode_map(&pl->x_k[i], pl->X[i], l, s, chunk, ldx, BK, 128);
    ok = ok && encode_map(&pl->x_mn[i], pl->X[i], l, s, chunk, ldx, 64, BK);
  }
  ok = ok && encode_map(&pl->a_k, A, s, s, chunk, lds, BK, 128);
  ok = ok && encode_map(&pl->b_k, B, s, s, chunk, lds, BK, 128);
  if (!ok) {
    snprintf(err, errlen, "cuTensorMapEncodeTiled failed for shape %lld x %lld", (long long)s, (long long)l);
    delete pl;
    return nullptr;
  }
  std::vector<int2> sym, full;
  const int tm_n = (int)((s + BM - 1) / BM);
  const int tn_sym = (int)((s + pl->bn_sym - 1) / pl->bn_sym);
  for (int tm = 0; tm < tm_n; ++tm)
    for (int tn = 0; tn < tn_sym; ++tn)
      if ((int64_t)(tn + 1) * pl->bn_sym > (int64_t)tm * BM) sym.push_back(make_int2(tm, tn));
  const int tn_full = (int)((l + pl->bn_apply - 1) / pl->bn_apply);
  for (int tm = 0; tm < tm_n; ++tm)
    for (int tn = 0; tn < tn_full; ++tn) full.push_back(make_int2(tm, tn));
  pl->n_tiles_sym = (int)sym.size();
  pl->n_tiles_full = (int)full.size();
  if (cudaMalloc(&pl->tiles_sym, sym.size() * sizeof(int2)) != cudaSuccess ||
      cudaMalloc(&pl->tiles_full, full.size() * sizeof(int2)) != cudaSuccess ||
      cudaMemcpy(pl->tiles_sym, sym.data(), sym.size() * sizeof(int2), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(pl->tiles_full, full.data(), full.size() * sizeof(int2), cudaMemcpyHostToDevice) != cudaSuccess) {
    snprintf(err, errlen, "tile list allocation failed");
    tc_plan_destroy(pl);
    return nullptr;
  }
  return pl;
}

void tc_plan_destroy(TcGroupPlan* pl) {
  if (!pl) return;
  if (pl->tiles_sym) cudaFree(pl->tiles_sym);
  if (pl->tiles_full) cudaFree(pl->tiles_full);
  delete pl;
}

cudaError_t tc_launch(cudaStream_t st, TcGroupPlan* pl, int kind, int n_mats, int xin,
                      const NsIterArgs& args) {
  if (n_mats <= 0) return cudaSuccess;
  TcParams p;
  memset(&p, 0, sizeof(p));
  p.kind = kind; p.n_mats = n_mats;
  p.a = args.a; p.b = args.b; p.c = args.c;
  p.scales = args.scales; p.mats = args.mats; p.sink_mode = args.sink_mode;
  p.s = pl->s; p.l = pl->l; p.status = args.status;
  p.M = (int)pl->s;
  const int64_t sX = pl->s * pl->ldx, sS = pl->s * pl->lds;
  __nv_bfloat16* Xin = reinterpret_cast<__nv_bfloat16*>(pl->X[xin]);
  __nv_bfloat16* Xout = reinterpret_cast<__nv_bfloat16*>(pl->X[1 - xin]);
  __nv_bfloat16* A = reinterpret_cast<__nv_bfloat16*>(pl->A);
  __nv_bfloat16* B = reinterpret_cast<__nv_bfloat16*>(pl->B);
  if (kind == GEMM_GRAM) {
    p.N = (int)pl->s; p.Kd = (int)pl->l; p.tiles = pl->tiles_sym; p.n_tiles_per_mat = pl->n_tiles_sym;
    p.D = A; p.ldd = pl->lds; p.strideD = sS;
    return pl->bn_sym == 256 ? launch_one<256, false>(st, pl->x_k[xin], pl->x_k[xin], p, pl->n_sms)
                             : launch_one<128, false>(st, pl->x_k[xin], pl->x_k[xin], p, pl->n_sms);
  }
  if (kind == GEMM_POLY) {
    p.N = (int)pl->s; p.Kd = (int)pl->s; p.tiles = pl->tiles_sym; p.n_tiles_per_mat = pl->n_tiles_sym;
    p.Cin = A; p.ldc = pl->lds; p.strideC = sS;
    p.D = B; p.ldd = pl->lds; p.strideD = sS;
    return pl->bn_sym == 256 ? launch_one<256, false>(st, pl->a_k, pl->a_k, p, pl->n_sms)
                             : launch_one<128, false>(st, pl->a_k, pl->a_k, p, pl->n_sms);
  }
  p.N = (int)pl->l; p.Kd = (int)pl->s; p.tiles = pl->tiles_full; p.n_tiles_per_mat = pl->n_tiles_full;
  p.Cin = Xin; p.ldc = pl->ldx; p.strideC = sX;
  p.D = (kind == GEMM_APPLY) ? Xout : nullptr; p.ldd = pl->ldx; p.strideD = sX;
  return pl->bn_apply == 256 ? launch_one<256, true>(st, pl->b_k, pl->x_mn[xin], p, pl->n_sms)
                             : launch_one<128, true>(st, pl->b_k, pl->x_mn[xin], p, pl->n_sms);
}

}  // namespace muloco
