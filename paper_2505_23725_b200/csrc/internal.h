// Internal declarations shared by the CUDA translation units of libmuloco.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/muloco.h"

namespace muloco {

// Device status word bits (OR-ed by kernels, read by muloco_sync_status).
enum : int { ST_NONFINITE = 1, ST_TIMEOUT = 2, ST_BOUNDS = 4 };

// Debug build (-DMULOCO_DEBUG): kernels check the indices they derive (work-list cursors, matrix
// slots, tile coordinates, segment and unit indices) before using them; a failed check raises
// ST_BOUNDS in the status word and the thread skips the access (nothing traps).  In the regular
// build the checks compile to nothing.
#ifdef MULOCO_DEBUG
#define MULOCO_IN_BOUNDS(cond, status) ((cond) ? true : (atomicOr((status), ::muloco::ST_BOUNDS), false))
#else
#define MULOCO_IN_BOUNDS(cond, status) (true)
#endif

// ---------------------------------------------------------------------------
// Muon path: one entry per (worker, hidden matrix) of a chunk.
// The Newton-Schulz workspace always holds X as s x l with s <= l; a matrix
// stored with rows > cols enters and leaves through its transpose.
// ---------------------------------------------------------------------------
struct MatDesc {
  const void* g;   // gradient (fp32 or bf16), tensor layout rows x cols; or raw X for the standalone call
  float* m;        // Muon momentum (fp32), tensor layout; NULL for the standalone call
  void* w;         // parameters W (fp32, updated in place) or output O of the standalone call
  float lr_eff;    // eta' = lr * lr_scale * lr_mult
  float wd_term;   // eta_wd * lambda * wd_mult (multiplies W)
  int32_t transposed;  // 1: tensor is l x s (rows > cols)
  int32_t pad;
  const void* wmap;    // device address of a 128-byte TMA descriptor over W (32 x 32 fp32 boxes) for the
                       // fused parameter update of the tensor-core engine, or NULL (plain accesses)
};

enum SrcMode : int { SRC_MUON = 0, SRC_RAW_F32 = 1, SRC_RAW_BF16 = 2 };
enum SinkMode : int { SINK_UPDATE_W = 0, SINK_STORE_F32 = 1, SINK_STORE_BF16 = 2 };

// prologue: m <- beta m + g; U -> workspace X (bf16 or fp32, s x ldx per slot); partial sums of U^2.
// partial layout: partials[slot * n_part + tile], n_part = ceil(s/32) * ceil(l/128).
void launch_prologue(cudaStream_t st, const MatDesc* mats, int n_mats, int64_t s, int64_t l,
                     int src_mode, int g_is_bf16, float beta, int nesterov, void* X, int x_is_f32,
                     int64_t ldx, float* partials);
int prologue_partials_per_matrix(int64_t s, int64_t l);
// scales[slot] = { r*r, r } with r = 1 / (sqrt(sum partials) + eps)
void launch_finalize_scales(cudaStream_t st, const float* partials, int n_part, int n_mats,
                            float eps, float2* scales, int* status = nullptr);

// fp32 Newton-Schulz engine (CUDA cores).  One call = one of the three products
// of an iteration for all matrices of a chunk.
enum GemmKind : int { GEMM_GRAM = 0, GEMM_POLY = 1, GEMM_APPLY = 2, GEMM_FINAL = 3 };
struct NsIterArgs {
  float a, b, c;            // quintic coefficients
  const float2* scales;     // per-slot {r^2, r}; NULL: no scaling in this call
  const MatDesc* mats;      // for GEMM_FINAL (sink)
  int sink_mode;
  int* status;
  unsigned long long wait_limit_ns = 0;   // tensor-core engine: limit of every device-side wait (0: 2 s)
  int debug_withhold = 0;                 // tensor-core engine, test hook: one operand copy is never issued
};
void launch_ns_fp32(cudaStream_t st, int kind, int n_mats, int64_t s, int64_t l, const float* X,
                    int64_t ldx, const float* A, const float* B, int64_t lds, float* Aout,
                    float* Bout, float* Xout, const NsIterArgs& args);

// bf16 tensor-core engine (tcgen05 / TMEM / TMA); see ns_tc.cu.  One launch runs all products of
// all iterations for the matrices of a chunk; the staged input X0 is chunk-sized, the
// intermediates live in a ring of tc_ring_slots(group) slots.
struct TcGroupPlan;   // opaque per-shape-group plan (tensor maps, tile lists, work lists)
// matrices per group of the work list for min-dimension s (never more than `chunk`)
int tc_group_size(int64_t s, int chunk);
// ring slots for groups of `group` matrices; bytes of the ring (X', X'', A, B for n_slots matrices, bf16)
int tc_ring_slots(int group);
size_t tc_ring_bytes(int64_t s, int64_t ldx, int64_t lds, int n_slots);
// counters: chunk * 3 * ns_steps + 1 ints (tile counters and the ticket counter; zeroed by every launch)
TcGroupPlan* tc_plan_create(int64_t s, int64_t l, int chunk, void* X0, int64_t ldx, void* ring, int64_t lds,
                            int group, int* counters, int ns_steps, char* err, size_t errlen);
void tc_plan_destroy(TcGroupPlan*);
// the whole iteration for the first n_mats matrices of the chunk (args.scales: per-matrix {r^2, r})
cudaError_t tc_launch(cudaStream_t st, TcGroupPlan* plan, int n_mats, const NsIterArgs& args);
int tc_num_sms();
// Encodes (into 128 bytes at `out_host`) the TMA descriptor of a rows x cols fp32 tensor for 32 x 32
// boxes; swizzled for tensors stored s x l, plain for tensors stored l x s.  False when the tensor
// cannot be addressed by TMA (base not 16-byte aligned or cols not a multiple of 4).
bool tc_encode_w_map(void* out_host, void* base, int64_t rows, int64_t cols, int transposed);
constexpr size_t TC_MAP_BYTES = 128;

// AdamW: one entry per (worker, tensor).
struct AdamSeg {
  const void* g;
  float* m;
  float* v;
  float* theta;
  int64_t n;
  int64_t unit_begin;   // first work unit (of ADAM_UNIT elements) of this segment
  float lr;             // alpha
  float lr_wd;          // alpha * lambda * wd_mult
  float inv_bc1;        // 1 / (1 - beta1^t) (1 if no bias correction)
  float inv_sqrt_bc2;   // 1 / sqrt(1 - beta2^t)
};
constexpr int ADAM_UNIT = 2048;
// status: device status word; a non-finite gradient raises ST_NONFINITE (NULL: not checked)
void launch_adamw(cudaStream_t st, const AdamSeg* segs, int n_segs, int64_t n_units, int g_is_bf16,
                  float beta1, float beta2, float eps, int* status);

// Outer sync: one entry per tensor of the fragment.
struct SyncSeg {
  float* theta_g;
  float* u;
  int64_t rows, cols;
  int64_t nblk;         // blocks per row
  int64_t unit_begin;   // first block-unit of this segment
  int64_t rep_index;    // index of this tensor's first replica pointer in the replica table
};
// ef: table of error-feedback accumulators laid out like `replicas` (NULL: no error feedback);
// stages 2 selects the per-worker quantisation of Algorithm 2.
void launch_outer_sync(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas,
                       int K, int64_t n_units, int block, int quant_bits, float outer_lr,
                       float mu, int* status, int n_sms, int stages = 1, float* const* ef = nullptr,
                       float ef_beta = 1.0f);
// Row-wise quantisation (quant_block == 0): units are rows (SyncSeg.nblk == 1); max_cols is the
// longest row of the fragment.  cudaErrorInvalidValue when a row does not fit shared memory.
cudaError_t launch_outer_sync_rows(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas,
                                   int K, int64_t n_rows, int64_t max_cols, int quant_bits, float outer_lr,
                                   float mu, int* status, int stages, float* const* ef, float ef_beta);
// K = 1, eta_out = 1, mu = 0, no compression: theta <- theta_1 (exactly), u <- theta - theta_1.
void launch_dp_sync(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas, int64_t n_units,
                    int* status);
// Worker-sharded outer synchronisation (outer_sync.cu): the three passes around the caller's
// reduce-scatter and all-gather.  Staging buffers are unit-major, 128 floats per unit.
void launch_shard_delta(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas, int K,
                        int64_t n_units, int block, int quant_bits, int stages, float* const* ef, float ef_beta,
                        float* stage, int* status);
void launch_shard_step(cudaStream_t st, const SyncSeg* segs, int n_segs, int64_t n_units, int64_t unit_begin,
                       int64_t unit_count, int block, int quant_bits, float outer_lr, float mu, float inv_k_total,
                       const float* reduced, float* theta_out, int* status);
void launch_shard_broadcast(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas, int K,
                            int64_t n_units, int block, const float* theta_all, int* status);
// Top-k sparsification of the workers' deltas (topk.cu).  Scratch: one histogram of
// topk_hist_words_per_problem() words (zero between calls), one prefix word (the threshold key
// after a call) and one counter per (tensor, worker), indexed like the replica table.
// kk_seg[i] = how many entries segment i keeps.  Segments are flat (rows == 1, 128-element units).
// Returns the number of kernels launched.
struct TopkScratch {
  uint32_t* hist = nullptr;
  uint32_t* prefix = nullptr;
  uint32_t* remaining = nullptr;
};
size_t topk_hist_words_per_problem();
int launch_outer_sync_topk(cudaStream_t st, const SyncSeg* segs, int n_segs, float* const* replicas, int K,
                           int64_t n_units, float outer_lr, float mu, int* status, float* const* ef,
                           float ef_beta, const uint32_t* kk_seg, TopkScratch sc);
// Standalone: out = top-k(x) for one device array of n elements; seg_dev describes x as one flat
// segment (theta_g = x, rep_index = 0), kk_dev holds the count to keep.
int launch_topk_raw(cudaStream_t st, const SyncSeg* seg_dev, int64_t n, const float* x, float* out,
                    const uint32_t* kk_dev, TopkScratch sc, int* status);
void launch_pseudogradient(cudaStream_t st, const float* theta_g, float* const* replicas, int K,
                           int64_t n, float* psi_out);
void launch_quantize(cudaStream_t st, const float* psi, int64_t rows, int64_t cols, int block,
                     int bits, int8_t* codes, float* scales, float* dequant, int* status);
void launch_broadcast_init(cudaStream_t st, const float* src, float* const* dst_table, int K,
                           int64_t n);

}  // namespace muloco
