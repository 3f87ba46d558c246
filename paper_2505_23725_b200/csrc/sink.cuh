// Final stage of the Muon step, shared by the fp32 and the tensor-core engines:
// what happens to one element O[i][j] of the orthogonalised update (s x l view).
#pragma once
#include "internal.h"

namespace muloco {

// SINK_UPDATE_W : W <- W - eta' O - (eta_wd lambda) W   (Section 2 "Muon"; eta' carries sqrt(n/m))
// SINK_STORE_*  : O itself is written (standalone Newton-Schulz call)
__device__ __forceinline__ void sink_element(const MatDesc& d, int sink_mode, int64_t s, int64_t l,
                                             int64_t i, int64_t j, float o) {
  const int64_t idx = d.transposed ? (j * s + i) : (i * l + j);
  if (sink_mode == SINK_UPDATE_W) {
    float* w = reinterpret_cast<float*>(d.w);
    const float wv = w[idx];
    w[idx] = fmaf(-d.lr_eff, o, fmaf(-d.wd_term, wv, wv));
  } else if (sink_mode == SINK_STORE_F32) {
    reinterpret_cast<float*>(d.w)[idx] = o;
  } else {
    reinterpret_cast<__nv_bfloat16*>(d.w)[idx] = __float2bfloat16_rn(o);
  }
}

}  // namespace muloco
