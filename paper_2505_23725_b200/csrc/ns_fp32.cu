// fp32 Newton-Schulz engine on CUDA cores (FFMA), used where the result must be
// within 1e-4 of a float64 evaluation (TF32/bf16 inputs are too coarse for that:
// the iteration amplifies input rounding by up to a^5 ~ 485).  One launch = one
// of the three products of an iteration, for every matrix of a chunk:
//   GRAM  : A  = r^2 * X X^T            (r^2 only in the first iteration)
//   POLY  : B  = b A + c A A
//   APPLY : X' = r * (a X + B X)        (r only in the first iteration)
//   FINAL : as APPLY, but the result goes to the sink (parameter update / output)
// (Section 2, "Muon": X_j = p(X X^T) X with p(x) = a x + b x^3 + c x^5.)
#include "internal.h"
#include "sink.cuh"

namespace muloco {

namespace {

constexpr int FT = 64;    // tile edge
constexpr int FK = 16;    // k slab
constexpr int FTHREADS = 256;

// P(i,k) = Pm[i*ldp + k].  Q(k,j) = NT ? Qm[j*ldq + k] : Qm[k*ldq + j].
template <bool NT>
__global__ void __launch_bounds__(FTHREADS)
ns_fp32_kernel(int kind, int64_t M, int64_t N, int64_t Kd, const float* __restrict__ P, int64_t ldp,
               int64_t strideP, const float* __restrict__ Q, int64_t ldq, int64_t strideQ,
               const float* __restrict__ Cin, int64_t ldc, int64_t strideC, float* __restrict__ D,
               int64_t ldd, int64_t strideD, float a, float b, float c, const float2* __restrict__ scales,
               const MatDesc* __restrict__ mats, int sink_mode, int64_t s, int64_t l) {
  __shared__ float Ps[FK][FT + 4];
  __shared__ float Qs[FK][FT + 4];
  const int mat = blockIdx.z;
  const int64_t i0 = (int64_t)blockIdx.y * FT, j0 = (int64_t)blockIdx.x * FT;
  const float* Pm = P + (int64_t)mat * strideP;
  const float* Qm = Q + (int64_t)mat * strideQ;
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  float acc[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[r][q] = 0.f;

  for (int64_t k0 = 0; k0 < Kd; k0 += FK) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int e = tid + r * FTHREADS;
      {
        const int ii = e / FK, kk = e % FK;
        const int64_t i = i0 + ii, k = k0 + kk;
        Ps[kk][ii] = (i < M && k < Kd) ? Pm[i * ldp + k] : 0.f;
      }
      if (NT) {
        const int jj = e / FK, kk = e % FK;
        const int64_t j = j0 + jj, k = k0 + kk;
        Qs[kk][jj] = (j < N && k < Kd) ? Qm[j * ldq + k] : 0.f;
      } else {
        const int kk = e / FT, jj = e % FT;
        const int64_t j = j0 + jj, k = k0 + kk;
        Qs[kk][jj] = (j < N && k < Kd) ? Qm[k * ldq + j] : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < FK; ++kk) {
      float pv[4], qv[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) pv[r] = Ps[kk][ty * 4 + r];
#pragma unroll
      for (int q = 0; q < 4; ++q) qv[q] = Qs[kk][tx * 4 + q];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[r][q] = fmaf(pv[r], qv[q], acc[r][q]);
    }
    __syncthreads();
  }

  float sc = 1.f;
  if (scales) sc = (kind == GEMM_GRAM) ? scales[mat].x : scales[mat].y;
  const float* Cm = Cin ? Cin + (int64_t)mat * strideC : nullptr;
  float* Dm = D ? D + (int64_t)mat * strideD : nullptr;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int64_t i = i0 + ty * 4 + r;
    if (i >= M) continue;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int64_t j = j0 + tx * 4 + q;
      if (j >= N) continue;
      float v = acc[r][q];
      if (kind == GEMM_GRAM) {
        Dm[i * ldd + j] = v * sc;
      } else if (kind == GEMM_POLY) {
        Dm[i * ldd + j] = fmaf(c, v, b * Cm[i * ldc + j]);
      } else {
        v = sc * fmaf(a, Cm[i * ldc + j], v);
        if (kind == GEMM_APPLY) Dm[i * ldd + j] = v;
        else sink_element(mats[mat], sink_mode, s, l, i, j, v);
      }
    }
  }
}

}  // namespace

void launch_ns_fp32(cudaStream_t st, int kind, int n_mats, int64_t s, int64_t l, const float* X,
                    int64_t ldx, const float* A, const float* B, int64_t lds, float* Aout, float* Bout,
                    float* Xout, const NsIterArgs& args) {
  if (n_mats <= 0) return;
  const int64_t sX = s * ldx, sS = s * lds;
  for (int m0 = 0; m0 < n_mats; m0 += 65535) {
    const int nm = (n_mats - m0 < 65535) ? (n_mats - m0) : 65535;
    const float2* sc = args.scales ? args.scales + m0 : nullptr;
    const MatDesc* md = args.mats ? args.mats + m0 : nullptr;
    if (kind == GEMM_GRAM) {
      dim3 grid((unsigned)((s + FT - 1) / FT), (unsigned)((s + FT - 1) / FT), (unsigned)nm);
      ns_fp32_kernel<true><<<grid, FTHREADS, 0, st>>>(kind, s, s, l, X + m0 * sX, ldx, sX, X + m0 * sX, ldx,
                                                      sX, nullptr, 0, 0, Aout + m0 * sS, lds, sS, args.a,
                                                      args.b, args.c, sc, md, args.sink_mode, s, l);
    } else if (kind == GEMM_POLY) {
      dim3 grid((unsigned)((s + FT - 1) / FT), (unsigned)((s + FT - 1) / FT), (unsigned)nm);
      ns_fp32_kernel<true><<<grid, FTHREADS, 0, st>>>(kind, s, s, s, A + m0 * sS, lds, sS, A + m0 * sS, lds,
                                                      sS, A + m0 * sS, lds, sS, Bout + m0 * sS, lds, sS,
                                                      args.a, args.b, args.c, nullptr, md, args.sink_mode,
                                                      s, l);
    } else {
      dim3 grid((unsigned)((l + FT - 1) / FT), (unsigned)((s + FT - 1) / FT), (unsigned)nm);
      ns_fp32_kernel<false><<<grid, FTHREADS, 0, st>>>(
          kind, s, l, s, B + m0 * sS, lds, sS, X + m0 * sX, ldx, sX, X + m0 * sX, ldx, sX,
          Xout ? Xout + m0 * sX : nullptr, ldx, sX, args.a, args.b, args.c, sc, md, args.sink_mode, s, l);
    }
  }
}

}  // namespace muloco
