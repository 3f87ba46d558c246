// muloco_newton_schulz_static: Newton-Schulz on a small batch with NO device
// allocation.  Its scratch (staged X, Gram and polynomial matrices, norm partials,
// descriptor table) lives in one file-scope __device__ array of fixed size, so the
// call never reaches cudaMalloc/cudaFree.  The descriptor table is written by a
// small kernel from by-value arguments, so the call reads no host memory after it
// returns.  It is meant for callers that
// must not allocate: code that runs after a framework's caching allocator has
// reserved the whole device (a raw cudaMalloc there can fail or fragment the pool),
// and latency-sensitive loops that cannot afford the device-wide synchronisation an
// allocation or a free implies.
//
// The array belongs to the library image: every GPU that loads libmuloco keeps
// MULOCO_STATIC_SCRATCH_BYTES of it until the process exits.  All calls on a device
// share it and it keeps the previous call's contents, so two calls whose GPU work
// overlaps (different streams, or threads) race; serialise them.
#include <stdio.h>

#include <mutex>

#include "internal.h"

using namespace muloco;

namespace {

constexpr size_t kScratchBytes = MULOCO_STATIC_SCRATCH_BYTES;
constexpr int kMaxBatch = 64;
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for the runtime (cudaGetSymbolAddress);
// it is NOT a device address and must never be handed to a kernel as one.
static __device__ __align__(256) unsigned char g_ns_scratch[kScratchBytes];

struct DeviceSetup {
  bool ready = false;
  unsigned char* base = nullptr;   // device address of g_ns_scratch on this device
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

size_t up256(size_t v) { return (v + 255) / 256 * 256; }

// One descriptor per matrix of the batch, written on the device: X and O are
// [batch][rows][cols]; the standalone sink stores O and uses no optimizer fields.
__global__ void static_descs_kernel(MatDesc* __restrict__ mats, const float* X, float* O, int batch,
                                    int64_t numel, int transposed) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= batch) return;
  MatDesc d;
  d.g = X + (size_t)j * numel;
  d.m = nullptr;
  d.w = O + (size_t)j * numel;
  d.lr_eff = 0.f;
  d.wd_term = 0.f;
  d.transposed = transposed;
  d.pad = 0;
  d.wmap = nullptr;
  mats[j] = d;
}

muloco_status fail(char* errbuf, size_t errlen, muloco_status s, const char* fmt, long long a = 0,
                   long long b = 0, long long c = 0) {
  if (errbuf && errlen) snprintf(errbuf, errlen, fmt, a, b, c);
  return s;
}

}  // namespace

extern "C" MULOCO_API muloco_status muloco_newton_schulz_static(const float* X, float* O, int32_t batch,
                                                                int64_t rows, int64_t cols,
                                                                void* cuda_stream, char* errbuf,
                                                                size_t errbuf_len) {
  if (errbuf && errbuf_len) errbuf[0] = 0;
  if (!X || !O) return fail(errbuf, errbuf_len, MULOCO_EINVAL, "X or O is NULL");
  if (batch < 0 || rows < 1 || cols < 1) return fail(errbuf, errbuf_len, MULOCO_ESHAPE, "bad batch or shape");
  if (batch == 0) return MULOCO_OK;
  if (batch > kMaxBatch)
    return fail(errbuf, errbuf_len, MULOCO_ESHAPE, "batch %lld exceeds the static limit of %lld matrices",
                (long long)batch, (long long)kMaxBatch);
  const int64_t s = rows < cols ? rows : cols, l = rows < cols ? cols : rows;
  if (l > (1 << 20)) return fail(errbuf, errbuf_len, MULOCO_ESHAPE, "matrix too large");
  const int64_t ldx = (l + 7) / 8 * 8, lds = (s + 7) / 8 * 8;
  const int n_part = prologue_partials_per_matrix(s, l);

  // carve the scratch: descriptors | X0 | X1 | A | B | partials | scales
  size_t off = 0;
  const size_t o_mats = off;   off += up256((size_t)batch * sizeof(MatDesc));
  const size_t xb = up256((size_t)batch * s * ldx * sizeof(float));
  const size_t sb = up256((size_t)batch * s * lds * sizeof(float));
  const size_t o_x0 = off; off += xb;
  const size_t o_x1 = off; off += xb;
  const size_t o_a = off;  off += sb;
  const size_t o_b = off;  off += sb;
  const size_t o_part = off; off += up256((size_t)batch * n_part * sizeof(float));
  const size_t o_scales = off; off += up256((size_t)batch * sizeof(float2));
  if (off > kScratchBytes)
    return fail(errbuf, errbuf_len, MULOCO_ESHAPE,
                "needs %lld bytes of scratch but the static scratch holds %lld: use muloco_newton_schulz",
                (long long)off, (long long)kScratchBytes);

  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(errbuf, errbuf_len, MULOCO_ECUDA, "no current CUDA device (error %lld)", (long long)e);
  if (dev < 0 || dev >= kMaxDevices) return fail(errbuf, errbuf_len, MULOCO_ECUDA, "device index %lld not supported", dev);
  unsigned char* base = nullptr;
  {
    // once per device, with that device current: resolve the symbol to its device address
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_setup[dev].ready) {
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_ns_scratch);
      if (e != cudaSuccess || !p)
        return fail(errbuf, errbuf_len, MULOCO_ECUDA, "cudaGetSymbolAddress failed (error %lld)", (long long)e);
      g_setup[dev].base = static_cast<unsigned char*>(p);
      g_setup[dev].ready = true;
    }
    base = g_setup[dev].base;
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);

  // Every region of the scratch is fully written by this call before it is read (descriptors
  // here, X0 and the partial sums by the prologue, the scales, A, B and X1 by the kernels that
  // follow on the same stream), so nothing has to be cleared and nothing of an earlier call leaks in.
  MatDesc* d_mats = reinterpret_cast<MatDesc*>(base + o_mats);
  static_descs_kernel<<<1, kMaxBatch, 0, st>>>(d_mats, X, O, batch, rows * cols, rows > cols ? 1 : 0);

  float* X0 = reinterpret_cast<float*>(base + o_x0);
  float* X1 = reinterpret_cast<float*>(base + o_x1);
  float* A = reinterpret_cast<float*>(base + o_a);
  float* B = reinterpret_cast<float*>(base + o_b);
  float* partials = reinterpret_cast<float*>(base + o_part);
  float2* scales = reinterpret_cast<float2*>(base + o_scales);
  launch_prologue(st, d_mats, batch, s, l, SRC_RAW_F32, 0, 0.f, 0, X0, 1, ldx, partials);
  launch_finalize_scales(st, partials, n_part, batch, 1e-7f, scales);   // no status word: see the header
  NsIterArgs a;
  a.a = 3.4445f; a.b = -4.7750f; a.c = 2.0315f;   // Section 2, "Muon"
  a.mats = d_mats; a.sink_mode = SINK_STORE_F32; a.status = nullptr;
  float* Xb[2] = {X0, X1};
  for (int it = 0; it < 5; ++it) {
    float* Xin = Xb[it & 1];
    float* Xout = Xb[1 - (it & 1)];
    a.scales = (it == 0) ? scales : nullptr;
    launch_ns_fp32(st, GEMM_GRAM, batch, s, l, Xin, ldx, A, B, lds, A, B, Xout, a);
    a.scales = nullptr;
    launch_ns_fp32(st, GEMM_POLY, batch, s, l, Xin, ldx, A, B, lds, A, B, Xout, a);
    a.scales = (it == 0) ? scales : nullptr;
    launch_ns_fp32(st, it == 4 ? GEMM_FINAL : GEMM_APPLY, batch, s, l, Xin, ldx, A, B, lds, A, B, Xout, a);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(errbuf, errbuf_len, MULOCO_ECUDA, "kernel launch failed (error %lld)", (long long)e);
  return MULOCO_OK;
}
