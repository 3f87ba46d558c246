// C ABI of libmuloco and the host runtime behind it: tensor table, shape
// groups, chunked Newton-Schulz workspace, per-call descriptor tables, phase
// timers.  Every step of the optimizer runs in the kernels of this library; the
// host code only validates, builds tables and launches.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <string>
#include <vector>

#include "internal.h"

using namespace muloco;

namespace {

thread_local std::string g_create_error;

struct TensorInfo {
  int64_t rows, cols;
  int kind, fragment;
  float wd_mult, lr_mult;
  float* theta_g;
  float* u;
  std::vector<float*> theta_k, s1, s2, ef;
  int64_t numel() const { return rows * cols; }
};

struct WsRegion { const char* name; size_t off, bytes; };

struct WsLayout {   // byte offsets inside the workspace for one shape group
  // fp32 engine: x0, x1, a, b are chunk-sized.  bf16 engine: x0 is the chunk-sized staged input and
  // `ring` holds the intermediates of tc_ring_slots(group) matrices; `counters` counts finished tiles.
  // Every region lies between guard zones of at least 1 KB; the 64 bytes right before and right
  // after a region are its canaries (see muloco_check_workspace).
  size_t x0 = 0, x1 = 0, a = 0, b = 0, ring = 0, partials = 0, scales = 0, counters = 0, total = 0;
  std::vector<WsRegion> regions;
};

struct Group {
  int64_t s = 0, l = 0, ldx = 0, lds = 0;
  std::vector<int> tensors;
  int chunk = 0;
  int n_part = 0;
  int elt = 2;
  int mode = MULOCO_NS_BF16;   // engine that serves this group (see engine_for)
  int ring_group = 1;          // bf16 engine: matrices per group of the work list (the ring has tc_ring_slots(ring_group) slots)
  WsLayout ws;
  TcGroupPlan* plan = nullptr;
};

// How many entries top-k keeps of n: floor(fraction * n) in double, at least 1, at most n.
uint32_t topk_keep(int64_t n, float fraction) {
  int64_t kk = (int64_t)floor((double)fraction * (double)n);
  kk = std::max<int64_t>(1, std::min<int64_t>(kk, n));
  return (uint32_t)kk;
}

struct FragTable {
  uint32_t* d_kk = nullptr;     // top-k: entries kept per segment
  SyncSeg* d_segs = nullptr;
  int n_segs = 0;
  int64_t n_units = 0;
  int64_t max_cols = 0;
  std::vector<int> tensors;
};

struct TimedSpan { int phase; cudaEvent_t a, b; };

constexpr int RING = 3;
constexpr uint32_t STATE_MAGIC = 0x4d4c4331u;   // "MLC1"

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// The bf16 engine holds its 2e-2 tolerance from a min-dimension of 64 on (measured against the fp64
// iteration: 1.0-1.5e-2 there, 1.9-3.8e-2 for 8..48 rows, where too few roundings average out), so
// smaller matrices always take the fp32 engine; their cost is negligible.
constexpr int64_t BF16_MIN_S = 64;
int engine_for(int requested_mode, int64_t s) {
  return (requested_mode == MULOCO_NS_BF16 && s >= BF16_MIN_S) ? MULOCO_NS_BF16 : MULOCO_NS_FP32;
}

constexpr size_t WS_GUARD = 1024, WS_CANARY = 64;
constexpr int WS_CANARY_BYTE = 0xC5;

WsLayout make_layout(int64_t s, int64_t ldx, int64_t lds, int chunk, int n_part, int elt, int ring_group,
                     int ns_steps) {
  WsLayout w;
  size_t off = 0;
  auto place = [&](const char* name, size_t bytes) {
    off = align_up(off + WS_GUARD, 1024);
    w.regions.push_back(WsRegion{name, off, bytes});
    const size_t at = off;
    off += bytes;
    return at;
  };
  const size_t xb = (size_t)chunk * s * ldx * elt;
  w.x0 = place("X0", xb);
  if (elt == 2) {
    w.ring = place("ring", tc_ring_bytes(s, ldx, lds, tc_ring_slots(ring_group)));
  } else {
    const size_t sb = (size_t)chunk * s * lds * elt;
    w.x1 = place("X1", xb);
    w.a = place("A", sb);
    w.b = place("B", sb);
  }
  w.partials = place("partials", (size_t)chunk * n_part * sizeof(float));
  w.scales = place("scales", (size_t)chunk * sizeof(float2));
  w.counters = place("counters", ((size_t)chunk * 3 * ns_steps + 16) * sizeof(int));   // tile counters + ticket
  w.total = align_up(off + WS_GUARD, 1024);
  return w;
}

// Matrices per workspace chunk: as many as the budget holds, then evened out so that
// all chunks of a group have (nearly) the same size.
int pick_chunk(int64_t count, size_t per_slot, size_t budget) {
  int64_t ch = (int64_t)(budget / (per_slot ? per_slot : 1));
  if (ch < 1) ch = 1;
  if (ch >= count) return (int)std::max<int64_t>(count, 1);
  const int64_t n_chunks = (count + ch - 1) / ch;
  return (int)((count + n_chunks - 1) / n_chunks);
}

// Chunk size and ring size of a group of `count` same-shape matrices within `budget` bytes.
void size_group(int64_t s, int64_t l, int64_t ldx, int64_t lds, int64_t count, size_t budget, int mode,
                int ns_steps, int* chunk, int* ring_group) {
  const int np = prologue_partials_per_matrix(s, l);
  const int elt = (mode == MULOCO_NS_BF16) ? 2 : 4;
  int rg = 1;
  size_t fixed = 0;
  if (elt == 2) {
    rg = tc_group_size(s, (int)std::min<int64_t>(count, 1 << 30));
    fixed = tc_ring_bytes(s, ldx, lds, tc_ring_slots(rg));
  }
  const size_t per_slot = make_layout(s, ldx, lds, 1, np, elt, 0, ns_steps).total;
  const size_t avail = budget > fixed + per_slot ? budget - fixed : per_slot;
  *chunk = pick_chunk(count, per_slot, avail);
  *ring_group = std::min(rg, *chunk);
}

}  // namespace

struct muloco_ctx {
  muloco_config cfg;
  int n = 0;
  std::vector<TensorInfo> T;
  cudaStream_t st = nullptr;
  int n_sms = 148;
  std::string err;
  int* d_status = nullptr;
  unsigned long long wait_limit_ns = 0;   // limit of the device-side waits of the bf16 engine (0: its default)
  int debug_withhold = 0;                 // test hook, see muloco_debug_set
  bool canaries = false;                  // write and verify the workspace canaries around every chunk
  int corrupt_region = -1;                // test hook: one canary byte of this region is overwritten (one-shot)
  std::string canary_report;              // first violation since the last muloco_check_workspace

  std::vector<int> muon_ids, adam_ids;
  std::vector<Group> groups;
  char* ws = nullptr;
  size_t ws_bytes = 0;

  // standalone Newton-Schulz call: its own cached group + workspace
  Group sa_group;
  char* sa_ws = nullptr;
  size_t sa_ws_bytes = 0;
  int sa_mode = -1;
  MatDesc* sa_d_mats = nullptr;
  int sa_mats_cap = 0;

  std::vector<FragTable> frags;   // J entries + one for "all"
  float** d_replicas = nullptr;   // [n][K]
  float** d_ef = nullptr;         // [n][K] error-feedback accumulators (Algorithm 2), or NULL
  TopkScratch topk;               // radix-select scratch, [n][K] problems (top-k only)

  // per-call tables
  MatDesc* d_mats = nullptr;
  AdamSeg* d_adam = nullptr;
  char* d_wmaps = nullptr;                 // [K][n] TMA descriptors over theta_k (bf16 engine only)
  std::vector<char> wmap_ok;               // [K][n]
  char* h_ring[RING] = {nullptr, nullptr, nullptr};
  cudaEvent_t ring_ev[RING];
  bool ring_used[RING] = {false, false, false};
  int ring_next = 0;
  size_t ring_bytes = 0;

  std::vector<int64_t> worker_step, frag_syncs;

  // host-gradient staging: copies run on their own stream, one section (shape group, or the
  // AdamW tensors) at a time, so that the copy of a section overlaps the compute of the others
  cudaStream_t copy_st = nullptr, copy_st2 = nullptr;   // two streams: per-copy overheads of one hide under the other
  std::vector<cudaEvent_t> ev_copied, ev_copied2, ev_consumed;   // per section
  std::vector<char> consumed_valid;
  bool host_mode = false;                            // set while muloco_inner_step_host runs the step
  char* stage = nullptr;
  size_t stage_bytes = 0;
  std::vector<size_t> stage_off;   // [K][n]

  // timing
  bool timing = false;
  std::vector<TimedSpan> spans;
  std::vector<cudaEvent_t> ev_pool;
  int64_t launches = 0;
};

namespace {

muloco_status fail(muloco_ctx* c, muloco_status s, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c) c->err = buf; else g_create_error = buf;
  return s;
}

#define CK(call)                                                                              \
  do {                                                                                        \
    cudaError_t e_ = (call);                                                                  \
    if (e_ != cudaSuccess)                                                                    \
      return fail(c, MULOCO_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_));           \
  } while (0)

cudaEvent_t get_event(muloco_ctx* c) {
  if (!c->ev_pool.empty()) {
    cudaEvent_t e = c->ev_pool.back();
    c->ev_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

struct PhaseTimer {
  muloco_ctx* c;
  TimedSpan sp;
  bool on;
  cudaStream_t stream;
  PhaseTimer(muloco_ctx* ctx, int phase, cudaStream_t s = nullptr)
      : c(ctx), on(ctx->timing), stream(s ? s : ctx->st) {
    if (on) {
      sp.phase = phase;
      sp.a = get_event(c);
      sp.b = get_event(c);
      cudaEventRecord(sp.a, stream);
    }
  }
  ~PhaseTimer() {
    if (on) {
      cudaEventRecord(sp.b, stream);
      c->spans.push_back(sp);
    }
  }
};

bool valid_block(int b) { return b == 0 || b == 32 || b == 64 || b == 128; }   // 0: one block per row

muloco_status validate_config(const muloco_config* cfg) {
  muloco_ctx* c = nullptr;
  if (!cfg) return fail(c, MULOCO_EINVAL, "config is NULL");
  if (cfg->K < 1 || cfg->K > 64) return fail(c, MULOCO_EINVAL, "K must be in 1..64 (got %d)", cfg->K);
  if (cfg->H < 1) return fail(c, MULOCO_EINVAL, "H must be >= 1");
  if (cfg->J < 1 || cfg->H % cfg->J != 0)
    return fail(c, MULOCO_EINVAL, "J must be >= 1 and divide H (H=%d, J=%d)", cfg->H, cfg->J);
  if (cfg->ns_steps < 1 || cfg->ns_steps > 64) return fail(c, MULOCO_EINVAL, "ns_steps must be in 1..64");
  if (cfg->ns_mode != MULOCO_NS_BF16 && cfg->ns_mode != MULOCO_NS_FP32)
    return fail(c, MULOCO_EINVAL, "unknown ns_mode %d", cfg->ns_mode);
  if (cfg->quant != MULOCO_Q_NONE && cfg->quant != MULOCO_Q_INT2 && cfg->quant != MULOCO_Q_INT4 &&
      cfg->quant != MULOCO_Q_INT8)
    return fail(c, MULOCO_EINVAL, "quant must be 0, 2, 4 or 8");
  if (cfg->quant_stages < 0 || cfg->quant_stages > 2)
    return fail(c, MULOCO_EINVAL, "quant_stages must be 0, 1 or 2");
  if (!(cfg->topk_fraction >= 0.f && cfg->topk_fraction <= 1.f))
    return fail(c, MULOCO_EINVAL, "topk_fraction must be in [0, 1]");
  if (cfg->topk_fraction > 0.f && cfg->quant != MULOCO_Q_NONE)
    return fail(c, MULOCO_EINVAL, "top-k sparsification and quantisation are not combined");
  if (cfg->error_feedback != 0 && !(cfg->topk_fraction > 0.f) &&
      (cfg->quant_stages != 2 || cfg->quant == MULOCO_Q_NONE))
    return fail(c, MULOCO_EINVAL, "error_feedback needs quant_stages == 2 and a quantiser, or topk_fraction > 0");
  if (cfg->error_feedback != 0 && !(cfg->ef_beta >= 0.f && cfg->ef_beta <= 1.f))
    return fail(c, MULOCO_EINVAL, "ef_beta must be in [0, 1]");
  if (!valid_block(cfg->quant_block)) return fail(c, MULOCO_EINVAL, "quant_block must be 0 (row-wise), 32, 64 or 128");
  if (cfg->grad_dtype != MULOCO_F32 && cfg->grad_dtype != MULOCO_BF16)
    return fail(c, MULOCO_EINVAL, "unknown grad_dtype %d", cfg->grad_dtype);
  if (!(cfg->ns_eps >= 0.f)) return fail(c, MULOCO_EINVAL, "ns_eps must be >= 0");
  return MULOCO_OK;
}

void destroy_group(Group& g) {
  if (g.plan) tc_plan_destroy(g.plan);
  g.plan = nullptr;
}

// Sets up a group's layout (and tensor-core plan in bf16 mode) inside workspace `ws`.
muloco_status setup_group(muloco_ctx* c, Group& g, char* ws, int mode) {
  g.mode = mode;
  g.elt = (mode == MULOCO_NS_BF16) ? 2 : 4;
  g.n_part = prologue_partials_per_matrix(g.s, g.l);
  g.ws = make_layout(g.s, g.ldx, g.lds, g.chunk, g.n_part, g.elt, g.ring_group, c->cfg.ns_steps);
  if (mode == MULOCO_NS_BF16) {
    char err[256] = {0};
    g.plan = tc_plan_create(g.s, g.l, g.chunk, ws + g.ws.x0, g.ldx, ws + g.ws.ring, g.lds, g.ring_group,
                            reinterpret_cast<int*>(ws + g.ws.counters), c->cfg.ns_steps, err, sizeof err);
    if (!g.plan) return fail(c, MULOCO_ECUDA, "%s", err);
  }
  return MULOCO_OK;
}

// Canaries of a group's layout inside workspace `ws`: written before a chunk runs ...
muloco_status write_canaries(muloco_ctx* c, const Group& g, char* ws) {
  for (const WsRegion& r : g.ws.regions) {
    CK(cudaMemsetAsync(ws + r.off - WS_CANARY, WS_CANARY_BYTE, WS_CANARY, c->st));
    CK(cudaMemsetAsync(ws + r.off + r.bytes, WS_CANARY_BYTE, WS_CANARY, c->st));
  }
  if (c->corrupt_region >= 0 && c->corrupt_region < (int)g.ws.regions.size()) {
    // test hook: a host-initiated memset stands in for a kernel that wrote past a region's end
    const WsRegion& r = g.ws.regions[c->corrupt_region];
    CK(cudaMemsetAsync(ws + r.off + r.bytes + 3, 0, 1, c->st));
  }
  c->corrupt_region = -1;
  return MULOCO_OK;
}

// ... and verified after it has run (waits for the stream).
muloco_status verify_canaries(muloco_ctx* c, const Group& g, char* ws) {
  const size_t n = g.ws.regions.size();
  std::vector<unsigned char> h(2 * n * WS_CANARY);
  for (size_t i = 0; i < n; ++i) {
    const WsRegion& r = g.ws.regions[i];
    CK(cudaMemcpyAsync(h.data() + (2 * i) * WS_CANARY, ws + r.off - WS_CANARY, WS_CANARY, cudaMemcpyDeviceToHost, c->st));
    CK(cudaMemcpyAsync(h.data() + (2 * i + 1) * WS_CANARY, ws + r.off + r.bytes, WS_CANARY, cudaMemcpyDeviceToHost, c->st));
  }
  CK(cudaStreamSynchronize(c->st));
  for (size_t i = 0; i < n && c->canary_report.empty(); ++i)
    for (int side = 0; side < 2 && c->canary_report.empty(); ++side)
      for (size_t b = 0; b < WS_CANARY; ++b)
        if (h[(2 * i + side) * WS_CANARY + b] != WS_CANARY_BYTE) {
          char buf[256];
          snprintf(buf, sizeof buf, "workspace canary %s region '%s' (shape group %lld x %lld) was overwritten at byte %zu",
                   side ? "after" : "before", g.ws.regions[i].name, (long long)g.s, (long long)g.l, b);
          c->canary_report = buf;
          break;
        }
  return MULOCO_OK;
}

// One chunk of matrices through prologue + Newton-Schulz + sink.
muloco_status run_ns_chunk(muloco_ctx* c, Group& g, char* ws, const MatDesc* d_mats, int n_mats,
                           int mode, int src_mode, int sink_mode, int g_is_bf16) {
  const muloco_config& f = c->cfg;
  float* partials = reinterpret_cast<float*>(ws + g.ws.partials);
  float2* scales = reinterpret_cast<float2*>(ws + g.ws.scales);
  void* X[2] = {ws + g.ws.x0, ws + g.ws.x1};
  if (c->canaries) {
    const muloco_status cs = write_canaries(c, g, ws);
    if (cs != MULOCO_OK) return cs;
  }
  {
    PhaseTimer t(c, MULOCO_PH_PROLOGUE);
    launch_prologue(c->st, d_mats, n_mats, g.s, g.l, src_mode, g_is_bf16, f.muon_beta, f.muon_nesterov,
                    X[0], mode == MULOCO_NS_FP32, g.ldx, partials);
    launch_finalize_scales(c->st, partials, g.n_part, n_mats, f.ns_eps, scales, c->d_status);
    c->launches += 2;
  }
  PhaseTimer t(c, MULOCO_PH_NS);
  NsIterArgs a;
  a.a = f.ns_a; a.b = f.ns_b; a.c = f.ns_c;
  a.mats = d_mats; a.sink_mode = sink_mode; a.status = c->d_status;
  if (mode == MULOCO_NS_BF16) {
    // one launch: every product of every iteration, the parameter update fused into the last one
    a.scales = scales;
    a.wait_limit_ns = c->wait_limit_ns;
    a.debug_withhold = c->debug_withhold;
    c->debug_withhold = 0;                       // one-shot
    CK(tc_launch(c->st, g.plan, n_mats, a));
    c->launches += 1;
    CK(cudaGetLastError());
    return c->canaries ? verify_canaries(c, g, ws) : MULOCO_OK;
  }
  for (int it = 0; it < f.ns_steps; ++it) {
    const int xin = it & 1;
    const bool last = (it == f.ns_steps - 1);
    float* Xin = reinterpret_cast<float*>(X[xin]);
    float* Xout = reinterpret_cast<float*>(X[1 - xin]);
    float* A = reinterpret_cast<float*>(ws + g.ws.a);
    float* B = reinterpret_cast<float*>(ws + g.ws.b);
    a.scales = (it == 0) ? scales : nullptr;
    launch_ns_fp32(c->st, GEMM_GRAM, n_mats, g.s, g.l, Xin, g.ldx, A, B, g.lds, A, B, Xout, a);
    a.scales = nullptr;
    launch_ns_fp32(c->st, GEMM_POLY, n_mats, g.s, g.l, Xin, g.ldx, A, B, g.lds, A, B, Xout, a);
    a.scales = (it == 0) ? scales : nullptr;
    launch_ns_fp32(c->st, last ? GEMM_FINAL : GEMM_APPLY, n_mats, g.s, g.l, Xin, g.ldx, A, B, g.lds,
                   A, B, Xout, a);
    c->launches += 3;
  }
  CK(cudaGetLastError());
  return c->canaries ? verify_canaries(c, g, ws) : MULOCO_OK;
}

muloco_status build_sync_tables(muloco_ctx* c) {
  const int K = c->cfg.K, n = c->n;
  std::vector<float*> reps((size_t)n * K);
  for (int i = 0; i < n; ++i)
    for (int k = 0; k < K; ++k) reps[(size_t)i * K + k] = c->T[i].theta_k[k];
  if (n > 0) {
    CK(cudaMalloc(&c->d_replicas, reps.size() * sizeof(float*)));
    CK(cudaMemcpy(c->d_replicas, reps.data(), reps.size() * sizeof(float*), cudaMemcpyHostToDevice));
    if (c->cfg.error_feedback != 0) {
      for (int i = 0; i < n; ++i)
        for (int k = 0; k < K; ++k) reps[(size_t)i * K + k] = c->T[i].ef[k];
      CK(cudaMalloc(&c->d_ef, reps.size() * sizeof(float*)));
      CK(cudaMemcpy(c->d_ef, reps.data(), reps.size() * sizeof(float*), cudaMemcpyHostToDevice));
    }
  }
  const bool topk = c->cfg.topk_fraction > 0.f;
  if (topk && n > 0) {
    for (int i = 0; i < n; ++i)
      if (c->T[i].numel() >= ((int64_t)1 << 31))
        return fail(c, MULOCO_ESHAPE, "top-k: tensor %d has 2^31 elements or more", i);
    const size_t problems = (size_t)n * K;
    const size_t hist_bytes = problems * topk_hist_words_per_problem() * sizeof(uint32_t);
    CK(cudaMalloc(&c->topk.hist, hist_bytes));
    CK(cudaMalloc(&c->topk.prefix, problems * sizeof(uint32_t)));
    CK(cudaMalloc(&c->topk.remaining, problems * sizeof(uint32_t)));
    CK(cudaMemsetAsync(c->topk.hist, 0, hist_bytes, c->st));
    CK(cudaMemsetAsync(c->topk.prefix, 0, problems * sizeof(uint32_t), c->st));
    CK(cudaMemsetAsync(c->topk.remaining, 0, problems * sizeof(uint32_t), c->st));
  }
  c->frags.resize(c->cfg.J + 1);
  for (int f = 0; f <= c->cfg.J; ++f) {
    FragTable& ft = c->frags[f];
    std::vector<SyncSeg> segs;
    std::vector<uint32_t> kks;
    int64_t units = 0;
    for (int i = 0; i < n; ++i) {
      const TensorInfo& t = c->T[i];
      if (f < c->cfg.J && t.fragment != f) continue;
      ft.tensors.push_back(i);
      SyncSeg s;
      s.theta_g = t.theta_g; s.u = t.u;
      if (c->cfg.quant == MULOCO_Q_NONE) { s.rows = 1; s.cols = t.numel(); }
      else { s.rows = t.rows; s.cols = t.cols; }
      int64_t blk = (c->cfg.quant == MULOCO_Q_NONE) ? 128 : c->cfg.quant_block;
      if (blk == 0) blk = s.cols;                      // row-wise: one unit per row
      s.nblk = (s.cols + blk - 1) / blk;
      ft.max_cols = std::max<int64_t>(ft.max_cols, s.cols);
      s.unit_begin = units;
      s.rep_index = (int64_t)i * K;
      units += s.rows * s.nblk;
      segs.push_back(s);
      if (topk) kks.push_back(topk_keep(t.numel(), c->cfg.topk_fraction));
    }
    ft.n_segs = (int)segs.size();
    ft.n_units = units;
    if (!segs.empty()) {
      CK(cudaMalloc(&ft.d_segs, segs.size() * sizeof(SyncSeg)));
      CK(cudaMemcpy(ft.d_segs, segs.data(), segs.size() * sizeof(SyncSeg), cudaMemcpyHostToDevice));
      if (topk) {
        CK(cudaMalloc(&ft.d_kk, kks.size() * sizeof(uint32_t)));
        CK(cudaMemcpy(ft.d_kk, kks.data(), kks.size() * sizeof(uint32_t), cudaMemcpyHostToDevice));
      }
    }
  }
  return MULOCO_OK;
}

muloco_status acquire_ring(muloco_ctx* c, char** host) {
  const int r = c->ring_next;
  c->ring_next = (r + 1) % RING;
  if (c->ring_used[r]) CK(cudaEventSynchronize(c->ring_ev[r]));
  *host = c->h_ring[r];
  return MULOCO_OK;
}

muloco_status release_ring(muloco_ctx* c, char* host) {
  for (int r = 0; r < RING; ++r)
    if (c->h_ring[r] == host) {
      CK(cudaEventRecord(c->ring_ev[r], c->st));
      c->ring_used[r] = true;
    }
  return MULOCO_OK;
}

}  // namespace

// ===========================================================================
extern "C" {

MULOCO_API muloco_status muloco_create(const muloco_config* cfg, const muloco_tensor_desc* tensors, int32_t n_tensors,
                            const muloco_buffers* bufs, void* cuda_stream, muloco_ctx** out) {
  muloco_ctx* c = nullptr;
  if (!out) return fail(c, MULOCO_EINVAL, "out is NULL");
  *out = nullptr;
  muloco_status vs = validate_config(cfg);
  if (vs != MULOCO_OK) return vs;
  if (n_tensors < 0) return fail(c, MULOCO_EINVAL, "n_tensors < 0");
  if (n_tensors > 0 && (!tensors || !bufs || !bufs->theta_k || !bufs->theta_g || !bufs->outer_u ||
                        !bufs->state1_k || !bufs->state2_k))
    return fail(c, MULOCO_EINVAL, "tensor table or buffer table is NULL");
  const int K = cfg->K;
  if (n_tensors > 0 && cfg->error_feedback != 0 && !bufs->ef_k)
    return fail(c, MULOCO_EINVAL, "error_feedback is set but the ef_k table is NULL");
  for (int i = 0; i < n_tensors; ++i) {
    const muloco_tensor_desc& d = tensors[i];
    if (d.rows < 1 || d.cols < 1) return fail(c, MULOCO_ESHAPE, "tensor %d has an empty shape", i);
    if (d.rows * d.cols > ((int64_t)1 << 40)) return fail(c, MULOCO_ESHAPE, "tensor %d is too large", i);
    if (d.kind != MULOCO_MUON && d.kind != MULOCO_ADAMW) return fail(c, MULOCO_EINVAL, "tensor %d: bad kind", i);
    if (d.fragment < 0 || d.fragment >= cfg->J)
      return fail(c, MULOCO_EINVAL, "tensor %d: fragment %d outside 0..%d", i, d.fragment, cfg->J - 1);
    if (d.kind == MULOCO_MUON && (std::min(d.rows, d.cols) > 32768 || std::max(d.rows, d.cols) > (1 << 20)))
      return fail(c, MULOCO_ESHAPE, "tensor %d: Muon matrix too large", i);
    if (!bufs->theta_g[i] || !bufs->outer_u[i]) return fail(c, MULOCO_EINVAL, "tensor %d: NULL global buffer", i);
    for (int k = 0; k < K; ++k) {
      const size_t e = (size_t)k * n_tensors + i;
      if (!bufs->theta_k[e] || !bufs->state1_k[e]) return fail(c, MULOCO_EINVAL, "tensor %d worker %d: NULL buffer", i, k);
      if (d.kind == MULOCO_ADAMW && !bufs->state2_k[e])
        return fail(c, MULOCO_EINVAL, "tensor %d worker %d: NULL second-moment buffer", i, k);
      if (cfg->error_feedback != 0 && !bufs->ef_k[e])
        return fail(c, MULOCO_EINVAL, "tensor %d worker %d: NULL error-feedback buffer", i, k);
    }
  }
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1)
    return fail(c, MULOCO_ECUDA, "no CUDA device: this library has no CPU path");

  c = new muloco_ctx();
  c->cfg = *cfg;
  c->n = n_tensors;
  c->st = reinterpret_cast<cudaStream_t>(cuda_stream);
  c->n_sms = tc_num_sms();
  c->worker_step.assign(K, 0);
  c->frag_syncs.assign(cfg->J, 0);
  for (int r = 0; r < RING; ++r) c->ring_ev[r] = nullptr;

  auto bail = [&](muloco_status s) {
    g_create_error = c->err;
    muloco_destroy(c);
    return s;
  };
#define CKC(call)                                                                              \
  do {                                                                                         \
    cudaError_t e_ = (call);                                                                   \
    if (e_ != cudaSuccess) {                                                                   \
      fail(c, MULOCO_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_));                   \
      return bail(MULOCO_ECUDA);                                                               \
    }                                                                                          \
  } while (0)

  c->T.resize(n_tensors);
  for (int i = 0; i < n_tensors; ++i) {
    TensorInfo& t = c->T[i];
    const muloco_tensor_desc& d = tensors[i];
    t.rows = d.rows; t.cols = d.cols; t.kind = d.kind; t.fragment = d.fragment;
    t.wd_mult = d.wd_mult;
    t.lr_mult = isnan(d.lr_mult) ? (d.kind == MULOCO_MUON ? (float)sqrt((double)d.cols / (double)d.rows) : 1.0f)
                                 : d.lr_mult;
    t.theta_g = bufs->theta_g[i];
    t.u = bufs->outer_u[i];
    for (int k = 0; k < K; ++k) {
      const size_t e = (size_t)k * n_tensors + i;
      t.theta_k.push_back(bufs->theta_k[e]);
      t.s1.push_back(bufs->state1_k[e]);
      t.s2.push_back(d.kind == MULOCO_ADAMW ? bufs->state2_k[e] : nullptr);
      t.ef.push_back(cfg->error_feedback != 0 ? bufs->ef_k[e] : nullptr);
    }
    (d.kind == MULOCO_MUON ? c->muon_ids : c->adam_ids).push_back(i);
  }

  CKC(cudaMalloc(&c->d_status, sizeof(int)));
  CKC(cudaMemsetAsync(c->d_status, 0, sizeof(int), c->st));

  // shape groups of the hidden matrices (same s x l after orienting to s <= l)
  std::map<std::pair<int64_t, int64_t>, int> gidx;
  for (int i : c->muon_ids) {
    const TensorInfo& t = c->T[i];
    const int64_t s = std::min(t.rows, t.cols), l = std::max(t.rows, t.cols);
    auto key = std::make_pair(s, l);
    if (!gidx.count(key)) {
      gidx[key] = (int)c->groups.size();
      Group g;
      g.s = s; g.l = l; g.ldx = (l + 7) / 8 * 8; g.lds = (s + 7) / 8 * 8;
      c->groups.push_back(g);
    }
    c->groups[gidx[key]].tensors.push_back(i);
  }
  // default budget: 6 GiB, less when the device is nearly full (the state of the largest
  // configurations leaves only a few GiB)
  size_t budget = cfg->workspace_bytes ? (size_t)cfg->workspace_bytes : ((size_t)6 << 30);
  if (!cfg->workspace_bytes) {
    size_t free_b = 0, total_b = 0;
    if (cudaMemGetInfo(&free_b, &total_b) == cudaSuccess && free_b / 2 < budget)
      budget = std::max<size_t>(free_b / 2, (size_t)256 << 20);
  }
  size_t need = 0;
  for (Group& g : c->groups) {
    const int np = prologue_partials_per_matrix(g.s, g.l);
    const int gmode = engine_for(cfg->ns_mode, g.s);
    size_group(g.s, g.l, g.ldx, g.lds, (int64_t)g.tensors.size() * K, budget, gmode, cfg->ns_steps, &g.chunk,
               &g.ring_group);
    need = std::max(need, make_layout(g.s, g.ldx, g.lds, g.chunk, np, gmode == MULOCO_NS_BF16 ? 2 : 4,
                                      g.ring_group, cfg->ns_steps).total);
  }
  if (need) {
    cudaError_t e = cudaMalloc(&c->ws, need);
    if (e != cudaSuccess) {
      fail(c, MULOCO_ENOMEM, "workspace of %zu bytes: %s", need, cudaGetErrorString(e));
      return bail(MULOCO_ENOMEM);
    }
    c->ws_bytes = need;
  }
  for (Group& g : c->groups) {
    muloco_status s = setup_group(c, g, c->ws, engine_for(cfg->ns_mode, g.s));
    if (s != MULOCO_OK) return bail(s);
  }

  // per-call descriptor tables
  const size_t n_mats_max = c->muon_ids.size() * (size_t)K;
  const size_t n_adam_max = c->adam_ids.size() * (size_t)K;
  if (n_mats_max) CKC(cudaMalloc(&c->d_mats, n_mats_max * sizeof(MatDesc)));
  if (n_adam_max) CKC(cudaMalloc(&c->d_adam, n_adam_max * sizeof(AdamSeg)));
  c->ring_bytes = std::max<size_t>(64, n_mats_max * sizeof(MatDesc) + n_adam_max * sizeof(AdamSeg));
  for (int r = 0; r < RING; ++r) {
    CKC(cudaMallocHost(&c->h_ring[r], c->ring_bytes));
    CKC(cudaEventCreateWithFlags(&c->ring_ev[r], cudaEventDisableTiming));
  }

  if (cfg->ns_mode == MULOCO_NS_BF16 && !c->muon_ids.empty()) {
    // one TMA descriptor per (worker, hidden matrix) for the fused parameter update
    std::vector<char> hmaps((size_t)K * n_tensors * TC_MAP_BYTES, 0);
    c->wmap_ok.assign((size_t)K * n_tensors, 0);
    for (int k = 0; k < K; ++k)
      for (int i : c->muon_ids) {
        const TensorInfo& t = c->T[i];
        const size_t e = (size_t)k * n_tensors + i;
        c->wmap_ok[e] = tc_encode_w_map(hmaps.data() + e * TC_MAP_BYTES, t.theta_k[k], t.rows, t.cols,
                                        t.rows > t.cols) ? 1 : 0;
      }
    CKC(cudaMalloc(&c->d_wmaps, hmaps.size()));
    CKC(cudaMemcpy(c->d_wmaps, hmaps.data(), hmaps.size(), cudaMemcpyHostToDevice));
  }

  { const muloco_status bs = build_sync_tables(c); if (bs != MULOCO_OK) return bail(bs); }

  // Algorithm 1, initialisation: u <- 0, inner state <- 0, theta_k <- theta_g
  for (int i = 0; i < n_tensors; ++i) {
    TensorInfo& t = c->T[i];
    const size_t bytes = (size_t)t.numel() * sizeof(float);
    CKC(cudaMemsetAsync(t.u, 0, bytes, c->st));
    for (int k = 0; k < K; ++k) {
      CKC(cudaMemsetAsync(t.s1[k], 0, bytes, c->st));
      if (t.s2[k]) CKC(cudaMemsetAsync(t.s2[k], 0, bytes, c->st));
      if (t.ef[k]) CKC(cudaMemsetAsync(t.ef[k], 0, bytes, c->st));     // Algorithm 2: E_i <- 0
      CKC(cudaMemcpyAsync(t.theta_k[k], t.theta_g, bytes, cudaMemcpyDeviceToDevice, c->st));
    }
  }
#undef CKC
  *out = c;
  return MULOCO_OK;
}

MULOCO_API void muloco_destroy(muloco_ctx* c) {
  if (!c) return;
  cudaStreamSynchronize(c->st);
  for (Group& g : c->groups) destroy_group(g);
  destroy_group(c->sa_group);
  if (c->ws) cudaFree(c->ws);
  if (c->sa_ws) cudaFree(c->sa_ws);
  if (c->sa_d_mats) cudaFree(c->sa_d_mats);
  if (c->d_status) cudaFree(c->d_status);
  if (c->d_replicas) cudaFree(c->d_replicas);
  if (c->d_ef) cudaFree(c->d_ef);
  if (c->topk.hist) cudaFree(c->topk.hist);
  if (c->topk.prefix) cudaFree(c->topk.prefix);
  if (c->topk.remaining) cudaFree(c->topk.remaining);
  if (c->d_mats) cudaFree(c->d_mats);
  if (c->d_adam) cudaFree(c->d_adam);
  if (c->d_wmaps) cudaFree(c->d_wmaps);
  if (c->copy_st) cudaStreamSynchronize(c->copy_st);
  if (c->copy_st2) cudaStreamSynchronize(c->copy_st2);
  for (cudaEvent_t e : c->ev_copied) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_copied2) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_consumed) if (e) cudaEventDestroy(e);
  if (c->copy_st) cudaStreamDestroy(c->copy_st);
  if (c->copy_st2) cudaStreamDestroy(c->copy_st2);
  if (c->stage) cudaFree(c->stage);
  for (FragTable& f : c->frags) {
    if (f.d_segs) cudaFree(f.d_segs);
    if (f.d_kk) cudaFree(f.d_kk);
  }
  for (int r = 0; r < RING; ++r) {
    if (c->h_ring[r]) cudaFreeHost(c->h_ring[r]);
    if (c->ring_ev[r]) cudaEventDestroy(c->ring_ev[r]);
  }
  for (TimedSpan& s : c->spans) { cudaEventDestroy(s.a); cudaEventDestroy(s.b); }
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  delete c;
}

MULOCO_API muloco_status muloco_inner_step(muloco_ctx* c, int32_t worker, const void* const* grads, float lr_scale) {
  if (!c) return MULOCO_EINVAL;
  const muloco_config& f = c->cfg;
  const int K = f.K, n = c->n;
  if (worker < -1 || worker >= K) return fail(c, MULOCO_EINVAL, "worker %d outside -1..%d", worker, K - 1);
  if (!grads && n > 0) return fail(c, MULOCO_EINVAL, "grads is NULL");
  const int k0 = worker < 0 ? 0 : worker, k1 = worker < 0 ? K : worker + 1;
  const int nw = k1 - k0;
  for (int k = k0; k < k1; ++k)
    for (int i = 0; i < n; ++i)
      if (!grads[(size_t)(k - k0) * n + i]) return fail(c, MULOCO_EINVAL, "gradient of tensor %d (worker %d) is NULL", i, k);
  if (n == 0) return MULOCO_OK;
  // the step counters advance only once the whole step has been enqueued (a call that fails on the
  // way leaves them, and with them AdamW's bias correction and the state blob, where they were)
  const int g_is_bf16 = (f.grad_dtype == MULOCO_BF16);

  char* host = nullptr;
  muloco_status rs = acquire_ring(c, &host);
  if (rs != MULOCO_OK) return rs;
  MatDesc* hm = reinterpret_cast<MatDesc*>(host);
  // group-major, worker-major inside a group
  std::vector<size_t> group_begin;
  size_t nm = 0;
  const double lr = (double)f.muon_lr * (double)lr_scale;
  for (const Group& g : c->groups) {
    group_begin.push_back(nm);
    for (int k = k0; k < k1; ++k)
      for (int i : g.tensors) {
        const TensorInfo& t = c->T[i];
        MatDesc d;
        d.g = grads[(size_t)(k - k0) * n + i];
        d.m = t.s1[k];
        d.w = t.theta_k[k];
        const double eta = lr * (double)t.lr_mult;
        d.lr_eff = (float)eta;
        d.wd_term = (float)((f.wd_uses_scaled_lr ? eta : lr) * (double)f.muon_wd * (double)t.wd_mult);
        d.transposed = t.rows > t.cols;
        d.pad = 0;
        const size_t e = (size_t)k * n + i;
        d.wmap = (c->d_wmaps && c->wmap_ok[e]) ? c->d_wmaps + e * TC_MAP_BYTES : nullptr;
        hm[nm++] = d;
      }
  }
  AdamSeg* ha = reinterpret_cast<AdamSeg*>(host + nm * sizeof(MatDesc));
  size_t na = 0;
  int64_t units = 0;
  for (int k = k0; k < k1; ++k) {
    const double t_step = (double)(c->worker_step[k] + 1);
    const double bc1 = f.adam_bias_correction ? 1.0 - pow((double)f.adam_beta1, t_step) : 1.0;
    const double bc2 = f.adam_bias_correction ? 1.0 - pow((double)f.adam_beta2, t_step) : 1.0;
    for (int i : c->adam_ids) {
      const TensorInfo& t = c->T[i];
      AdamSeg s;
      s.g = grads[(size_t)(k - k0) * n + i];
      s.m = t.s1[k]; s.v = t.s2[k]; s.theta = t.theta_k[k];
      s.n = t.numel();
      s.unit_begin = units;
      const double alpha = (double)f.adam_lr * (double)lr_scale * (double)t.lr_mult;
      s.lr = (float)alpha;
      s.lr_wd = (float)(alpha * (double)f.adam_wd * (double)t.wd_mult);
      s.inv_bc1 = (float)(1.0 / bc1);
      s.inv_sqrt_bc2 = (float)(1.0 / sqrt(bc2));
      units += (s.n + ADAM_UNIT - 1) / ADAM_UNIT;
      ha[na++] = s;
    }
  }
  if (nm) CK(cudaMemcpyAsync(c->d_mats, hm, nm * sizeof(MatDesc), cudaMemcpyHostToDevice, c->st));
  if (na) CK(cudaMemcpyAsync(c->d_adam, ha, na * sizeof(AdamSeg), cudaMemcpyHostToDevice, c->st));
  rs = release_ring(c, host);
  if (rs != MULOCO_OK) return rs;

  for (size_t gi = 0; gi < c->groups.size(); ++gi) {
    Group& g = c->groups[gi];
    const int count = (int)g.tensors.size() * nw;
    if (c->host_mode) {
      CK(cudaStreamWaitEvent(c->st, c->ev_copied[gi], 0));
      CK(cudaStreamWaitEvent(c->st, c->ev_copied2[gi], 0));
    }
    for (int m0 = 0; m0 < count; m0 += g.chunk) {
      const int cnt = std::min(g.chunk, count - m0);
      rs = run_ns_chunk(c, g, c->ws, c->d_mats + group_begin[gi] + m0, cnt, g.mode, SRC_MUON,
                        SINK_UPDATE_W, g_is_bf16);
      if (rs != MULOCO_OK) return rs;
    }
    if (c->host_mode) {
      CK(cudaEventRecord(c->ev_consumed[gi], c->st));
      c->consumed_valid[gi] = 1;
    }
  }
  if (na) {
    const size_t sec = c->groups.size();
    if (c->host_mode) {
      CK(cudaStreamWaitEvent(c->st, c->ev_copied[sec], 0));
      CK(cudaStreamWaitEvent(c->st, c->ev_copied2[sec], 0));
    }
    {
      PhaseTimer t(c, MULOCO_PH_ADAMW);
      launch_adamw(c->st, c->d_adam, (int)na, units, g_is_bf16, f.adam_beta1, f.adam_beta2, f.adam_eps, c->d_status);
      c->launches += 1;
    }
    if (c->host_mode) {
      CK(cudaEventRecord(c->ev_consumed[sec], c->st));
      c->consumed_valid[sec] = 1;
    }
  }
  CK(cudaGetLastError());
  for (int k = k0; k < k1; ++k) c->worker_step[k] += 1;
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_inner_step_host(muloco_ctx* c, int32_t worker, const void* const* host_grads,
                                     float lr_scale) {
  if (!c) return MULOCO_EINVAL;
  const int K = c->cfg.K, n = c->n;
  if (worker < -1 || worker >= K) return fail(c, MULOCO_EINVAL, "worker %d outside -1..%d", worker, K - 1);
  if (!host_grads && n > 0) return fail(c, MULOCO_EINVAL, "host_grads is NULL");
  if (n == 0) return MULOCO_OK;
  const size_t elt = (c->cfg.grad_dtype == MULOCO_BF16) ? 2 : 4;
  if (!c->stage) {
    c->stage_off.resize((size_t)K * n);
    size_t off = 0;
    for (int k = 0; k < K; ++k)
      for (int i = 0; i < n; ++i) {
        c->stage_off[(size_t)k * n + i] = off;
        off += align_up((size_t)c->T[i].numel() * elt, 16);
      }
    cudaError_t e = cudaMalloc(&c->stage, off);
    if (e != cudaSuccess) return fail(c, MULOCO_ENOMEM, "gradient staging of %zu bytes: %s", off, cudaGetErrorString(e));
    c->stage_bytes = off;
  }
  const int k0 = worker < 0 ? 0 : worker, k1 = worker < 0 ? K : worker + 1;
  std::vector<const void*> dev((size_t)(k1 - k0) * n);
  for (int k = k0; k < k1; ++k)
    for (int i = 0; i < n; ++i)
      if (!host_grads[(size_t)(k - k0) * n + i])
        return fail(c, MULOCO_EINVAL, "host gradient of tensor %d (worker %d) is NULL", i, k);
  const size_t n_sec = c->groups.size() + 1;           // shape groups, then the AdamW tensors
  if (!c->copy_st) {
    CK(cudaStreamCreateWithFlags(&c->copy_st, cudaStreamNonBlocking));
    CK(cudaStreamCreateWithFlags(&c->copy_st2, cudaStreamNonBlocking));
    c->ev_copied.assign(n_sec, nullptr);
    c->ev_copied2.assign(n_sec, nullptr);
    c->ev_consumed.assign(n_sec, nullptr);
    c->consumed_valid.assign(n_sec, 0);
    for (size_t s2 = 0; s2 < n_sec; ++s2) {
      CK(cudaEventCreateWithFlags(&c->ev_copied[s2], cudaEventDisableTiming));
      CK(cudaEventCreateWithFlags(&c->ev_copied2[s2], cudaEventDisableTiming));
      CK(cudaEventCreateWithFlags(&c->ev_consumed[s2], cudaEventDisableTiming));
    }
  }
  // Section by section, in the order the step consumes them: wait until the previous step has
  // consumed the section's staging area, copy (one copy per tensor: adjacent host pointers may
  // belong to different pinned allocations, which a single copy must not span), signal.
  for (size_t sec = 0; sec < n_sec; ++sec) {
    const std::vector<int>& ids = sec < c->groups.size() ? c->groups[sec].tensors : c->adam_ids;
    if (c->consumed_valid[sec]) {
      CK(cudaStreamWaitEvent(c->copy_st, c->ev_consumed[sec], 0));
      CK(cudaStreamWaitEvent(c->copy_st2, c->ev_consumed[sec], 0));
    }
    {
      // both copy streams are timed; the reported copy phase is the sum of their busy spans
      PhaseTimer t(c, MULOCO_PH_COPY, c->copy_st);
      PhaseTimer t2(c, MULOCO_PH_COPY, c->copy_st2);
      int which = 0;
      for (int k = k0; k < k1; ++k)
        for (int i : ids) {
          const void* src = host_grads[(size_t)(k - k0) * n + i];
          char* dst = c->stage + c->stage_off[(size_t)k * n + i];
          dev[(size_t)(k - k0) * n + i] = dst;
          CK(cudaMemcpyAsync(dst, src, (size_t)c->T[i].numel() * elt, cudaMemcpyHostToDevice,
                             (which++ & 1) ? c->copy_st2 : c->copy_st));
        }
    }
    CK(cudaEventRecord(c->ev_copied[sec], c->copy_st));
    CK(cudaEventRecord(c->ev_copied2[sec], c->copy_st2));
  }
  c->host_mode = true;
  const muloco_status rs = muloco_inner_step(c, worker, dev.data(), lr_scale);
  c->host_mode = false;
  return rs;
}

MULOCO_API muloco_status muloco_outer_sync(muloco_ctx* c, int32_t fragment) {
  if (!c) return MULOCO_EINVAL;
  const muloco_config& f = c->cfg;
  if (fragment < -1 || fragment >= f.J) return fail(c, MULOCO_EINVAL, "fragment %d outside -1..%d", fragment, f.J - 1);
  FragTable& ft = c->frags[fragment < 0 ? f.J : fragment];
  if (fragment < 0) for (auto& s : c->frag_syncs) s += 1; else c->frag_syncs[fragment] += 1;
  if (ft.n_segs == 0) return MULOCO_OK;
  PhaseTimer t(c, MULOCO_PH_SYNC);
  if (f.topk_fraction > 0.f) {
    c->launches += launch_outer_sync_topk(c->st, ft.d_segs, ft.n_segs, c->d_replicas, f.K, ft.n_units, f.outer_lr,
                                          f.outer_momentum, c->d_status, c->d_ef, f.ef_beta, ft.d_kk, c->topk);
    CK(cudaGetLastError());
    return MULOCO_OK;
  }
  if (f.K == 1 && f.quant == MULOCO_Q_NONE && f.outer_lr == 1.0f && f.outer_momentum == 0.0f) {
    // plain data parallelism (Section 5's DP baselines): the outer step is the identity on theta_1
    launch_dp_sync(c->st, ft.d_segs, ft.n_segs, c->d_replicas, ft.n_units, c->d_status);
    c->launches += 1;
    CK(cudaGetLastError());
    return MULOCO_OK;
  }
  const int blk = (f.quant == MULOCO_Q_NONE) ? 128 : f.quant_block;
  if (f.quant != MULOCO_Q_NONE && blk == 0) {
    cudaError_t e = launch_outer_sync_rows(c->st, ft.d_segs, ft.n_segs, c->d_replicas, f.K, ft.n_units, ft.max_cols,
                                           f.quant, f.outer_lr, f.outer_momentum, c->d_status,
                                           f.quant_stages == 2 ? 2 : 1, c->d_ef, f.ef_beta);
    if (e == cudaErrorInvalidValue)
      return fail(c, MULOCO_ESHAPE, "row-wise quantisation: a row of %lld elements does not fit shared memory",
                  (long long)ft.max_cols);
    CK(e);
    c->launches += 1;
    return MULOCO_OK;
  }
  launch_outer_sync(c->st, ft.d_segs, ft.n_segs, c->d_replicas, f.K, ft.n_units, blk, f.quant, f.outer_lr,
                    f.outer_momentum, c->d_status, c->n_sms, f.quant_stages == 2 ? 2 : 1, c->d_ef, f.ef_beta);
  c->launches += 1;
  CK(cudaGetLastError());
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_outer_sync_host(muloco_ctx* c, int32_t fragment, void* const* host_theta_g) {
  if (!c) return MULOCO_EINVAL;
  if (!host_theta_g && c->n > 0) return fail(c, MULOCO_EINVAL, "host_theta_g is NULL");
  muloco_status s = muloco_outer_sync(c, fragment);
  if (s != MULOCO_OK) return s;
  FragTable& ft = c->frags[fragment < 0 ? c->cfg.J : fragment];
  PhaseTimer t(c, MULOCO_PH_COPY);
  for (int i : ft.tensors) {
    if (!host_theta_g[i]) return fail(c, MULOCO_EINVAL, "host buffer of tensor %d is NULL", i);
    CK(cudaMemcpyAsync(host_theta_g[i], c->T[i].theta_g, (size_t)c->T[i].numel() * sizeof(float),
                       cudaMemcpyDeviceToHost, c->st));
  }
  return MULOCO_OK;
}

// ---- worker-sharded outer synchronisation ------------------------------------------------
namespace {
muloco_status shard_check(muloco_ctx* c, int32_t fragment, int32_t world, int32_t rank, FragTable** ft) {
  if (!c) return MULOCO_EINVAL;
  const muloco_config& f = c->cfg;
  if (fragment < -1 || fragment >= f.J) return fail(c, MULOCO_EINVAL, "fragment %d outside -1..%d", fragment, f.J - 1);
  if (world < 1 || rank < 0 || rank >= world) return fail(c, MULOCO_EINVAL, "bad world/rank (%d, %d)", world, rank);
  if (f.topk_fraction > 0.f) return fail(c, MULOCO_EINVAL, "the sharded sync does not do top-k sparsification");
  if (f.quant != MULOCO_Q_NONE && f.quant_block == 0)
    return fail(c, MULOCO_EINVAL, "the sharded sync does not do row-wise quantisation");
  *ft = &c->frags[fragment < 0 ? f.J : fragment];
  return MULOCO_OK;
}
int64_t shard_units(int64_t n_units, int32_t world) { return (n_units + world - 1) / world; }
}  // namespace

MULOCO_API muloco_status muloco_shard_layout(muloco_ctx* c, int32_t fragment, int32_t world, int32_t rank,
                                             int64_t* stage_floats, int64_t* shard_floats) {
  FragTable* ft = nullptr;
  const muloco_status s = shard_check(c, fragment, world, rank, &ft);
  if (s != MULOCO_OK) return s;
  const int64_t us = shard_units(ft->n_units, world);
  if (stage_floats) *stage_floats = us * world * 128;
  if (shard_floats) *shard_floats = us * 128;
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_shard_delta(muloco_ctx* c, int32_t fragment, int32_t world, float* stage) {
  FragTable* ft = nullptr;
  const muloco_status s = shard_check(c, fragment, world, 0, &ft);
  if (s != MULOCO_OK) return s;
  if (ft->n_segs == 0) return MULOCO_OK;
  if (!stage) return fail(c, MULOCO_EINVAL, "stage is NULL");
  const muloco_config& f = c->cfg;
  PhaseTimer t(c, MULOCO_PH_SYNC);
  const int64_t us = shard_units(ft->n_units, world);
  const int64_t pad = us * world - ft->n_units;      // units that only make the shards equal: zeros
  if (pad > 0) CK(cudaMemsetAsync(stage + ft->n_units * 128, 0, (size_t)pad * 128 * sizeof(float), c->st));
  const int blk = (f.quant == MULOCO_Q_NONE) ? 128 : f.quant_block;
  launch_shard_delta(c->st, ft->d_segs, ft->n_segs, c->d_replicas, f.K, ft->n_units, blk, f.quant,
                     f.quant_stages == 2 ? 2 : 1, c->d_ef, f.ef_beta, stage, c->d_status);
  c->launches += 1;
  CK(cudaGetLastError());
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_shard_step(muloco_ctx* c, int32_t fragment, int32_t world, int32_t rank,
                                           const float* reduced, float* theta_shard) {
  FragTable* ft = nullptr;
  const muloco_status s = shard_check(c, fragment, world, rank, &ft);
  if (s != MULOCO_OK) return s;
  if (ft->n_segs == 0) return MULOCO_OK;
  if (!reduced || !theta_shard) return fail(c, MULOCO_EINVAL, "reduced or theta_shard is NULL");
  const muloco_config& f = c->cfg;
  PhaseTimer t(c, MULOCO_PH_SYNC);
  const int64_t us = shard_units(ft->n_units, world);
  const int blk = (f.quant == MULOCO_Q_NONE) ? 128 : f.quant_block;
  const float inv_k_total = 1.0f / (float)((int64_t)f.K * world);
  launch_shard_step(c->st, ft->d_segs, ft->n_segs, ft->n_units, us * rank, us, blk, f.quant, f.outer_lr,
                    f.outer_momentum, inv_k_total, reduced, theta_shard, c->d_status);
  c->launches += 1;
  CK(cudaGetLastError());
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_shard_broadcast(muloco_ctx* c, int32_t fragment, int32_t world, const float* theta_all) {
  FragTable* ft = nullptr;
  const muloco_status s = shard_check(c, fragment, world, 0, &ft);
  if (s != MULOCO_OK) return s;
  const muloco_config& f = c->cfg;
  if (fragment < 0) for (auto& n : c->frag_syncs) n += 1; else c->frag_syncs[fragment] += 1;
  if (ft->n_segs == 0) return MULOCO_OK;
  if (!theta_all) return fail(c, MULOCO_EINVAL, "theta_all is NULL");
  PhaseTimer t(c, MULOCO_PH_SYNC);
  const int blk = (f.quant == MULOCO_Q_NONE) ? 128 : f.quant_block;
  launch_shard_broadcast(c->st, ft->d_segs, ft->n_segs, c->d_replicas, f.K, ft->n_units, blk, theta_all, c->d_status);
  c->launches += 1;
  CK(cudaGetLastError());
  return MULOCO_OK;
}

MULOCO_API int32_t muloco_fragments_due(const muloco_ctx* c, int64_t step, int32_t* out_frags) {
  if (!c || !out_frags) return -1;
  if (step <= 0) return 0;
  const int64_t H = c->cfg.H, J = c->cfg.J;
  int32_t cnt = 0;
  for (int64_t j = 1; j <= J; ++j)
    if (step % H == (j * H / J) % H) out_frags[cnt++] = (int32_t)(j - 1);
  return cnt;
}

MULOCO_API muloco_status muloco_newton_schulz(muloco_ctx* c, const void* X, int32_t x_dtype, void* O, int32_t o_dtype,
                                   int32_t batch, int64_t rows, int64_t cols, int32_t ns_mode) {
  if (!c) return MULOCO_EINVAL;
  if (batch < 0 || rows < 1 || cols < 1) return fail(c, MULOCO_ESHAPE, "bad batch/shape");
  if (batch == 0) return MULOCO_OK;                  // an empty batch: nothing to read or write
  if (!X || !O) return fail(c, MULOCO_EINVAL, "X or O is NULL");
  if ((x_dtype != MULOCO_F32 && x_dtype != MULOCO_BF16) || (o_dtype != MULOCO_F32 && o_dtype != MULOCO_BF16))
    return fail(c, MULOCO_EINVAL, "bad dtype");
  if (ns_mode != MULOCO_NS_BF16 && ns_mode != MULOCO_NS_FP32) return fail(c, MULOCO_EINVAL, "bad ns_mode");
  if (std::min(rows, cols) > 32768 || std::max(rows, cols) > (1 << 20)) return fail(c, MULOCO_ESHAPE, "matrix too large");
  if (batch == 0) return MULOCO_OK;
  const int64_t s = std::min(rows, cols), l = std::max(rows, cols);
  Group& g = c->sa_group;
  ns_mode = engine_for(ns_mode, s);
  const int elt = (ns_mode == MULOCO_NS_BF16) ? 2 : 4;
  const int64_t ldx = (l + 7) / 8 * 8, lds = (s + 7) / 8 * 8;
  const int np = prologue_partials_per_matrix(s, l);
  const size_t budget = c->cfg.workspace_bytes ? (size_t)c->cfg.workspace_bytes : ((size_t)6 << 30);
  int chunk = 1, ring_group = 1;
  size_group(s, l, ldx, lds, batch, budget, ns_mode, c->cfg.ns_steps, &chunk, &ring_group);
  if (g.s != s || g.l != l || c->sa_mode != ns_mode || g.chunk != chunk || !c->sa_ws) {
    CK(cudaStreamSynchronize(c->st));
    destroy_group(g);
    g = Group();
    g.s = s; g.l = l; g.ldx = ldx; g.lds = lds; g.chunk = chunk; g.ring_group = ring_group;
    const size_t need = make_layout(s, ldx, lds, chunk, np, elt, ring_group, c->cfg.ns_steps).total;
    if (need > c->sa_ws_bytes) {
      if (c->sa_ws) cudaFree(c->sa_ws);
      c->sa_ws = nullptr; c->sa_ws_bytes = 0;
      cudaError_t e = cudaMalloc(&c->sa_ws, need);
      if (e != cudaSuccess) return fail(c, MULOCO_ENOMEM, "workspace of %zu bytes: %s", need, cudaGetErrorString(e));
      c->sa_ws_bytes = need;
    }
    c->sa_mode = ns_mode;
    muloco_status st = setup_group(c, g, c->sa_ws, ns_mode);
    if (st != MULOCO_OK) { c->sa_mode = -1; g.s = 0; return st; }
  }
  if (c->sa_mats_cap < chunk) {
    if (c->sa_d_mats) cudaFree(c->sa_d_mats);
    c->sa_d_mats = nullptr; c->sa_mats_cap = 0;
    CK(cudaMalloc(&c->sa_d_mats, (size_t)chunk * sizeof(MatDesc)));
    c->sa_mats_cap = chunk;
  }
  const size_t xe = (x_dtype == MULOCO_BF16) ? 2 : 4, oe = (o_dtype == MULOCO_BF16) ? 2 : 4;
  std::vector<MatDesc> hm(chunk);
  for (int m0 = 0; m0 < batch; m0 += chunk) {
    const int cnt = std::min(chunk, batch - m0);
    for (int j = 0; j < cnt; ++j) {
      MatDesc d;
      d.g = reinterpret_cast<const char*>(X) + (size_t)(m0 + j) * rows * cols * xe;
      d.m = nullptr;
      d.w = reinterpret_cast<char*>(O) + (size_t)(m0 + j) * rows * cols * oe;
      d.lr_eff = 0.f; d.wd_term = 0.f;
      d.transposed = rows > cols;
      d.pad = 0;
      d.wmap = nullptr;
      hm[j] = d;
    }
    // pageable source: the copy is staged before the call returns, so hm may be reused
    CK(cudaMemcpyAsync(c->sa_d_mats, hm.data(), (size_t)cnt * sizeof(MatDesc), cudaMemcpyHostToDevice, c->st));
    CK(cudaStreamSynchronize(c->st));
    muloco_status st = run_ns_chunk(c, g, c->sa_ws, c->sa_d_mats, cnt, ns_mode,
                                    x_dtype == MULOCO_BF16 ? SRC_RAW_BF16 : SRC_RAW_F32,
                                    o_dtype == MULOCO_BF16 ? SINK_STORE_BF16 : SINK_STORE_F32, 0);
    if (st != MULOCO_OK) return st;
    if (m0 + chunk < batch) CK(cudaStreamSynchronize(c->st));
  }
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_quantize(muloco_ctx* c, const float* psi, int64_t rows, int64_t cols, int32_t bits,
                              int8_t* codes, float* scales, float* dequant) {
  if (!c) return MULOCO_EINVAL;
  if (bits != 8 && bits != 4 && bits != 2) return fail(c, MULOCO_EINVAL, "bits must be 8, 4 or 2");
  if (rows < 0 || cols < 0) return fail(c, MULOCO_ESHAPE, "negative shape");
  if (rows == 0 || cols == 0) return MULOCO_OK;      // empty input: nothing to read or write
  if (c->cfg.quant_block == 0)
    return fail(c, MULOCO_ESHAPE, "muloco_quantize works on blocks of 32, 64 or 128; this context is row-wise");
  if (!psi) return fail(c, MULOCO_EINVAL, "psi is NULL");
  launch_quantize(c->st, psi, rows, cols, c->cfg.quant_block, bits, codes, scales, dequant, c->d_status);
  c->launches += 1;
  CK(cudaGetLastError());
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_topk_sparsify(muloco_ctx* c, const float* x, int64_t n, float fraction, float* out) {
  if (!c) return MULOCO_EINVAL;
  if (!(fraction > 0.f && fraction <= 1.f)) return fail(c, MULOCO_EINVAL, "fraction must be in (0, 1]");
  if (n < 0 || n >= ((int64_t)1 << 31)) return fail(c, MULOCO_ESHAPE, "n must be in 0..2^31-1");
  if (n == 0) return MULOCO_OK;                      // empty input: nothing to read or write
  if (!x || !out) return fail(c, MULOCO_EINVAL, "x or out is NULL");
  const size_t words = topk_hist_words_per_problem() + 4;
  char* scratch = nullptr;
  CK(cudaMalloc(&scratch, words * sizeof(uint32_t) + sizeof(SyncSeg)));
  uint32_t* w = reinterpret_cast<uint32_t*>(scratch);
  TopkScratch sc;
  sc.hist = w;
  sc.prefix = w + topk_hist_words_per_problem();
  sc.remaining = sc.prefix + 1;
  uint32_t* d_kk = sc.prefix + 2;
  SyncSeg* d_seg = reinterpret_cast<SyncSeg*>(scratch + words * sizeof(uint32_t));
  SyncSeg seg;
  seg.theta_g = const_cast<float*>(x); seg.u = nullptr;
  seg.rows = 1; seg.cols = n; seg.nblk = (n + 127) / 128; seg.unit_begin = 0; seg.rep_index = 0;
  const uint32_t kk = topk_keep(n, fraction);
  cudaError_t e = cudaMemsetAsync(scratch, 0, words * sizeof(uint32_t), c->st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(d_kk, &kk, sizeof kk, cudaMemcpyHostToDevice, c->st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(d_seg, &seg, sizeof seg, cudaMemcpyHostToDevice, c->st);
  if (e == cudaSuccess) {
    c->launches += launch_topk_raw(c->st, d_seg, n, x, out, d_kk, sc, c->d_status);
    e = cudaGetLastError();
  }
  const cudaError_t e2 = cudaStreamSynchronize(c->st);   // kk and seg are stack variables; scratch is freed below
  cudaFree(scratch);
  CK(e);
  CK(e2);
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_pseudogradient(muloco_ctx* c, int32_t tensor, float* psi_out) {
  if (!c) return MULOCO_EINVAL;
  if (tensor < 0 || tensor >= c->n) return fail(c, MULOCO_EINVAL, "tensor %d outside 0..%d", tensor, c->n - 1);
  if (!psi_out) return fail(c, MULOCO_EINVAL, "psi_out is NULL");
  const TensorInfo& t = c->T[tensor];
  launch_pseudogradient(c->st, t.theta_g, c->d_replicas + (size_t)tensor * c->cfg.K, c->cfg.K, t.numel(), psi_out);
  c->launches += 1;
  CK(cudaGetLastError());
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_get_state(const muloco_ctx* c, void* host_blob, size_t* nbytes) {
  if (!c || !nbytes) return MULOCO_EINVAL;
  const size_t need = 16 + sizeof(int64_t) * (c->worker_step.size() + c->frag_syncs.size());
  if (!host_blob) { *nbytes = need; return MULOCO_OK; }
  if (*nbytes < need) { *nbytes = need; return MULOCO_EINVAL; }
  char* p = reinterpret_cast<char*>(host_blob);
  uint32_t hdr[4] = {STATE_MAGIC, (uint32_t)c->cfg.K, (uint32_t)c->cfg.J, 0};
  memcpy(p, hdr, 16);
  memcpy(p + 16, c->worker_step.data(), sizeof(int64_t) * c->worker_step.size());
  memcpy(p + 16 + sizeof(int64_t) * c->worker_step.size(), c->frag_syncs.data(),
         sizeof(int64_t) * c->frag_syncs.size());
  *nbytes = need;
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_set_state(muloco_ctx* c, const void* host_blob, size_t nbytes) {
  if (!c || !host_blob) return MULOCO_EINVAL;
  const size_t need = 16 + sizeof(int64_t) * (c->worker_step.size() + c->frag_syncs.size());
  if (nbytes != need) return fail(c, MULOCO_ESTATE, "state blob has %zu bytes, expected %zu", nbytes, need);
  const char* p = reinterpret_cast<const char*>(host_blob);
  uint32_t hdr[4];
  memcpy(hdr, p, 16);
  if (hdr[0] != STATE_MAGIC || hdr[1] != (uint32_t)c->cfg.K || hdr[2] != (uint32_t)c->cfg.J)
    return fail(c, MULOCO_ESTATE, "state blob does not match this context (K or J differ)");
  memcpy(c->worker_step.data(), p + 16, sizeof(int64_t) * c->worker_step.size());
  memcpy(c->frag_syncs.data(), p + 16 + sizeof(int64_t) * c->worker_step.size(),
         sizeof(int64_t) * c->frag_syncs.size());
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_set_timing(muloco_ctx* c, int32_t enabled) {
  if (!c) return MULOCO_EINVAL;
  c->timing = enabled != 0;
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_get_timings(muloco_ctx* c, float* ms, int64_t* launches) {
  if (!c) return MULOCO_EINVAL;
  CK(cudaStreamSynchronize(c->st));
  float acc[MULOCO_N_PHASES] = {0, 0, 0, 0, 0};
  for (TimedSpan& s : c->spans) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, s.a, s.b) == cudaSuccess) acc[s.phase] += t;
    c->ev_pool.push_back(s.a);
    c->ev_pool.push_back(s.b);
  }
  c->spans.clear();
  if (ms) memcpy(ms, acc, sizeof acc);
  if (launches) *launches = c->launches;
  c->launches = 0;
  return MULOCO_OK;
}

MULOCO_API muloco_status muloco_debug_set(muloco_ctx* c, int32_t what, int64_t value) {
  if (!c) return MULOCO_EINVAL;
  if (what == MULOCO_DEBUG_WAIT_LIMIT_NS) {
    if (value < 0) return fail(c, MULOCO_EINVAL, "wait limit must be >= 0");
    c->wait_limit_ns = (unsigned long long)value;
    return MULOCO_OK;
  }
  if (what == MULOCO_DEBUG_WITHHOLD_COPY) {
    c->debug_withhold = value != 0;
    return MULOCO_OK;
  }
  if (what == MULOCO_DEBUG_CANARIES) {
    c->canaries = value != 0;
    return MULOCO_OK;
  }
  if (what == MULOCO_DEBUG_CORRUPT_CANARY) {
    c->corrupt_region = (int)value;
    return MULOCO_OK;
  }
  return fail(c, MULOCO_EINVAL, "unknown debug switch %d", what);
}

MULOCO_API muloco_status muloco_check_workspace(muloco_ctx* c) {
  if (!c) return MULOCO_EINVAL;
  if (c->canary_report.empty()) return MULOCO_OK;
  const std::string msg = c->canary_report;
  c->canary_report.clear();
  return fail(c, MULOCO_ESTATE, "%s", msg.c_str());
}

MULOCO_API muloco_status muloco_sync_status(muloco_ctx* c) {
  if (!c) return MULOCO_EINVAL;
  cudaError_t e = cudaStreamSynchronize(c->st);
  if (e != cudaSuccess) return fail(c, MULOCO_ECUDA, "stream synchronize: %s", cudaGetErrorString(e));
  int h = 0;
  CK(cudaMemcpy(&h, c->d_status, sizeof(int), cudaMemcpyDeviceToHost));
  if (h) CK(cudaMemset(c->d_status, 0, sizeof(int)));
  if (h & ST_TIMEOUT) return fail(c, MULOCO_ETIMEOUT, "a bounded wait inside a kernel ran out");
  if (h & ST_BOUNDS) return fail(c, MULOCO_ECUDA, "a kernel rejected an out-of-range index");
  if (h & ST_NONFINITE)
    return fail(c, MULOCO_ENONFINITE, "non-finite value: a pseudogradient, the Newton-Schulz input of a hidden matrix, or a gradient given to AdamW");
  return MULOCO_OK;
}

MULOCO_API const char* muloco_last_error(const muloco_ctx* c) {
  return c ? c->err.c_str() : g_create_error.c_str();
}

}  // extern "C"
