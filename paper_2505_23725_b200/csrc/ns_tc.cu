// Batched bf16 Newton-Schulz engine for sm_100a: tcgen05.mma with fp32
// accumulators in tensor memory, operands staged in shared memory by TMA
// (128-byte swizzle), mbarrier pipeline, warp-specialised persistent CTAs.
//
// ONE launch runs the whole iteration (Section 2, "Muon": X_j = p(X X^T) X,
// p(x) = a x + b x^3 + c x^5, five times) for every matrix of a chunk.  Each
// iteration is three products,
//   GRAM  : A  = r^2 X X^T      symmetric: only the tiles on or above the diagonal are computed
//   POLY  : B' = a I + b A + c A A   AND stored; a consumer fetches a block below the diagonal as
//                               the transpose of its mirror image (an MN-major operand)
//   APPLY : X' = r B' X  (= r (a X + b A X + c A A X); with a on B's diagonal the product needs no addend)
//   FINAL : as APPLY in the last iteration, the result goes to the parameter update / output sink
// and the tiles of all products of all matrices form one linear list of work items that the host
// lays out (a table of blocks, one block = one product of a few matrices).  The list is ordered so
// that a matrix's intermediates are consumed while they are still in L2: the matrices are taken
// in groups of D, a group runs its 15 products one after the other over all its matrices, and the
// intermediates (X', A, B') live in a small ring of 2 D slots that the next group but one reuses;
// only the first Gram and the first apply read the staged input from its chunk-sized buffer.
//
// The tile workers (CTA pairs) take the items in list order from a ticket counter in global memory, and
// all workers are resident at once.  An item only depends on items before it in the list: a product of
// matrix m needs all tiles of m's previous product (and the first product of m needs the ring slot's
// previous user to be finished).  Finished tiles are counted per (matrix, product) in global memory:
// every epilogue warp adds one (release) once its part of the tile is in memory; a worker's
// dispatcher thread claims the next item, waits (acquire) until the count of the product it reads is
// complete and only then hands the item to the worker's other roles.  The unfinished item with the
// smallest index always has its inputs ready, so the list drains; a worker that has to wait for an
// input delays only itself, the others go on claiming items.
// Operand forms: GRAM/POLY multiply a row-major matrix by its own transpose
// (both operands K-major); APPLY needs X with the contraction index as the slow
// axis, i.e. an MN-major B operand, so no transposed copy of X is ever made.
//
// Two tile shapes share one kernel body (template parameter CG):
//   CG = 2 : a pair of CTAs on neighbouring SMs (a cluster of two) computes a
//            256 x 256 tile with tcgen05.mma.cta_group::2.  Each CTA stages its
//            own 128 rows of the left operand and HALF of the right operand, so
//            a stage is 32 KB per SM for 256 x 256 x 64 of work.  The CTA of
//            rank 0 issues the MMAs; every CTA drains its own 128 accumulator
//            rows.  No load is multicast: each CTA fetches its own slabs.
//   CG = 1 : one CTA, 128 x 128 tiles (matrices with at most 128 rows).
//
// CTA = 7 warps: warp 0 issues TMA loads, warp 1 allocates tensor memory and
// (rank 0) issues the MMAs, warps 2-5 run the epilogue (one 32-lane quarter of
// the accumulator each), warp 6 is the dispatcher: one thread (of the rank-0 CTA) that claims and
// decodes the worker's items, waits for their inputs and publishes them in a shared-memory ring of
// both CTAs, one item ahead of the producer, so that no other role ever waits on global memory
// between two tiles.  Two accumulators alternate so the epilogue of one
// tile overlaps the main loop of the next.  The epilogue goes through shared
// memory: the addend (A for POLY) arrives by TMA, results leave as
// bulk tensor stores of whole 32 x 64 blocks, so global memory only sees full lines.
// Every wait is bounded (on a barrier or on a counter): when one runs out the kernel raises
// ST_TIMEOUT (a failed index check of the debug build: ST_BOUNDS), all roles leave their loops, the CTA frees its tensor memory and returns; the other
// CTAs see the flag in the status word at their next counter wait and leave as well.
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <vector>

#include "internal.h"
#include "sink.cuh"

namespace muloco {

namespace {

constexpr int BM = 128;          // rows per CTA (one CTA's share of UMMA M)
constexpr int BK = 64;           // k slab per stage (64 bf16 = one 128-byte swizzle row)
constexpr int UMMA_K = 16;
constexpr int TC_THREADS = 224;      // 7 warps: producer, MMA issuer, 4 epilogue warps, scout
constexpr int TC_STAGES = 5;
// Five pipeline stages beside four staging blocks per epilogue warp (GRAM, APPLY: results; POLY:
// addend + results; FINAL: the parameter ring).
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;        // 16 KB: 128 rows x 64 k
constexpr uint32_t B_STAGE_BYTES = 128 * BK * 2;       // 16 KB: this CTA's 128 columns of the right operand
constexpr uint32_t STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr uint32_t EPI_BLOCK_BYTES = 32 * 64 * 2;      // one 32 x 64 bf16 block
constexpr uint32_t EPI_WARP_BYTES = 4u * EPI_BLOCK_BYTES;
constexpr uint32_t TC_SMEM_BYTES = (uint32_t)TC_STAGES * STAGE_BYTES + 4u * EPI_WARP_BYTES + 1024u;   // + alignment slack

// One block of the work list: the tiles of one product (`ph` = 3 * iteration + {0 Gram, 1 polynomial,
// 2 apply}) of the matrices [mat0, mat0 + n_mats) of the chunk, matrix-major.
struct TcBlock {
  int first_item, n_items;
  int kind, ph;
  int mat0, n_mats;
  int pad0, pad1;
};

// Tensor maps of one shape group.  X0 is the chunk-sized staged input (third coordinate: matrix of
// the chunk); XA, XB, A, B are the ring (third coordinate: slot).  _K: K-major operand boxes
// (64 x 128); _MN: MN-major operand boxes (one 4-D copy per slab when the column count allows it,
// else 64 x 64 boxes); _IO: 64 x 32 boxes for addend loads and result stores.
enum MapId : int {
  MAP_X0_K = 0, MAP_XA_K, MAP_XB_K,
  MAP_X0_MN, MAP_XA_MN, MAP_XB_MN,
  MAP_XA_IO, MAP_XB_IO,
  MAP_A_K, MAP_A_MN, MAP_A_IO,
  MAP_B_K, MAP_B_MN, MAP_B_IO,
  N_MAPS
};
struct TcMaps {
  CUtensorMap m[N_MAPS];
};

struct TcParams {
  const TcBlock* blocks;
  int n_blocks, total_items;
  int n_mats;                 // matrices of the chunk in this launch
  const int2* tiles_sym;      // (tile row, tile col) in units of 128*CG, tiles on or above the diagonal
  const int2* tiles_full;     // all tiles of the s x l result
  int n_sym, n_full;
  int s, l;
  int last_ph;                // 3 * ns_steps - 1: the product whose result goes to the sink
  float a, b, c;
  const float2* scales;       // per matrix of the chunk {r^2, r}; applied in the first iteration
  const MatDesc* mats;        // per matrix of the chunk (sink)
  int sink_mode;
  int x_wide, s_wide;         // the _MN maps of X / of A and B are the 4-D form (both 64-column atoms of a slab in one copy)
  int n_slots;
  int* ticket;                // next unclaimed item (zeroed by every launch)
  int* counters;              // [chunk][cw]: epilogue warps that have finished product ph of matrix m
  int cw;
  int* status;
  unsigned long long wait_limit_ns;
  int debug_withhold;         // test hook: the first operand copy of the list's first item is never issued
};

// One work item, as every role decodes it.
struct Item {
  int kind, ph, it;           // product, its index 3 * it + {0, 1, 2}, iteration
  int m, slot;                // matrix of the chunk, ring slot
  int2 tt;                    // tile
  int N, Kd;                  // result columns, contraction length
};

// ----------------------------- PTX wrappers --------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory offset in the CTA of rank `rank`
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n"
               "barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// arrive on a barrier given by its shared::cluster address (own CTA or the peer)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint64_t limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_timer_ns() - t0 > limit_ns) {
      *abort_flag = 1;
      return false;
    }
  }
}
// TMA load whose completion is counted on a barrier of this CTA.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// TMA load into this CTA's shared memory whose completion is counted on a barrier that may
// live in the peer CTA of the pair (shared::cluster address).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// 4-D forms for the maps that deliver two 64-column atoms of an MN-major operand in one copy
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
// 2-D forms, descriptor in global memory (the per-matrix maps of the parameter tensors)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const void* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void bulk_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_2() { asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory"); }
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

template <int CG>
__device__ __forceinline__ void tc_commit(uint32_t bar_cluster_addr) {
  if (CG == 1)
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster_addr) : "memory");
  else
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster_addr) : "memory");
}
template <int CG>
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  if (CG == 1)
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  else
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
template <int CG>
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem_addr, uint32_t cols) {
  if (CG == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem_addr), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  } else {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem_addr), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
}
template <int CG>
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols) {
  if (CG == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
  else
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
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
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// ----------------------------- work-list helpers ----------------------------
__device__ __forceinline__ Item decode_item(const TcParams& p, int item, int& cur) {
  // items of one worker increase, so the block cursor only moves forward
  const int4* bt = reinterpret_cast<const int4*>(p.blocks);
  Item q;
  q.kind = -1;                                  // stays -1 when a debug-build check fails
  q.ph = q.it = q.m = q.slot = q.N = q.Kd = 0;
  q.tt = make_int2(0, 0);
  if (!MULOCO_IN_BOUNDS(cur >= 0 && cur < p.n_blocks, p.status)) return q;
  int4 b0 = __ldg(bt + 2 * cur);
  while (item >= b0.x + b0.y) {
    ++cur;
    if (!MULOCO_IN_BOUNDS(cur < p.n_blocks, p.status)) return q;
    b0 = __ldg(bt + 2 * cur);
  }
  const int mat0 = __ldg(reinterpret_cast<const int*>(p.blocks) + 8 * cur + 4);
  const bool sym = b0.z <= GEMM_POLY;
  const int tpm = sym ? p.n_sym : p.n_full;
  const int r = item - b0.x;
  const int ml = r / tpm;
  q.ph = b0.w;
  q.it = q.ph / 3;
  q.m = mat0 + ml;
  q.slot = q.m % p.n_slots;
  if (!MULOCO_IN_BOUNDS(r >= 0 && q.m >= 0 && q.m < p.n_mats && b0.z >= GEMM_GRAM && b0.z <= GEMM_FINAL &&
                        q.ph >= 0 && q.ph <= p.last_ph, p.status))
    return q;
  q.tt = (sym ? p.tiles_sym : p.tiles_full)[r - ml * tpm];
  q.N = sym ? p.s : p.l;
  q.Kd = (b0.z == GEMM_GRAM) ? p.l : p.s;
#ifdef MULOCO_DEBUG
  {
    const int T = (p.s > 128) ? 256 : 128;      // tile edge
    if (!MULOCO_IN_BOUNDS(q.tt.x >= 0 && q.tt.y >= 0 && q.tt.x * T < p.s && q.tt.y * T < q.N, p.status)) return q;
  }
#endif
  q.kind = b0.z;
  return q;
}

__device__ __forceinline__ int ld_acquire(const int* ptr) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}

// Waits until the product this item reads is complete (all tiles of the matrix's previous product;
// for a matrix's first product: the last product of the ring slot's previous user).  Called by one
// thread.  Returns false when the CTA is aborting or another CTA has raised ST_TIMEOUT.
template <int CG>
__device__ __forceinline__ bool dep_wait(const TcParams& p, const Item& q, volatile int* abort_flag) {
  const int* cnt;
  int need;
  if (q.ph > 0) {
    cnt = p.counters + (int64_t)q.m * p.cw + (q.ph - 1);
    need = (((q.ph - 1) % 3 == 2) ? p.n_full : p.n_sym) * 4 * CG;
  } else if (q.m >= p.n_slots) {
    cnt = p.counters + (int64_t)(q.m - p.n_slots) * p.cw + p.last_ph;
    need = p.n_full * 4 * CG;
  } else {
    return true;
  }
  if (ld_acquire(cnt) < need) {
    const uint64_t t0 = global_timer_ns();
    for (;;) {
      if (ld_acquire(cnt) >= need) break;
      if (*abort_flag) return false;
      if (ld_acquire(p.status) & (ST_TIMEOUT | ST_BOUNDS)) { *abort_flag = 1; return false; }
      if (global_timer_ns() - t0 > p.wait_limit_ns) { *abort_flag = 1; return false; }
      __nanosleep(64);
    }
  }
  // what the other CTAs wrote through the async proxy is read through the async proxy next
  asm volatile("fence.proxy.async;" ::: "memory");
  return true;
}

// One epilogue warp has finished its part of a tile (its stores are complete): count it.
__device__ __forceinline__ void signal_done(const TcParams& p, const Item& q) {
  int* cnt = p.counters + (int64_t)q.m * p.cw + q.ph;
  asm volatile("fence.proxy.async;" ::: "memory");
  asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(cnt) : "memory");
}

// ---- the item ring --------------------------------------------------------------------------
// The dispatcher (one thread of the worker: warp 6, lane 0 of the rank-0 CTA) claims the worker's next
// item from a ticket counter in global memory, decodes it, waits for its inputs and then publishes
// it, packed into 64 bits, in a ring in shared memory of every CTA of the worker (for the peer CTA
// through distributed shared memory).  The other roles read their n-th item from slot n % RING.
//   bits 63..52 tag = (n + 1) mod 4096 | 51..44 ph | 43..22 m | 21..14 tile row | 13..0 tile column
// ph = RING_STOP marks the end of the work.  A slot is rewritten RING items later; the dispatcher stays
// at most one item ahead of the producer, the producer at most TC_STAGES tiles ahead of the MMA
// issuer (a tile is at least one k slab) and the MMA issuer at most two tiles ahead of the epilogue
// (two accumulators), so no reader is ever RING items behind.
constexpr int RING = 16;
constexpr int RING_STOP = 255;

__device__ __forceinline__ uint64_t ring_pack(int n, int ph, int m, int tx, int ty) {
  return ((uint64_t)((n + 1) & 0xFFF) << 52) | ((uint64_t)(ph & 0xFF) << 44) | ((uint64_t)(m & 0x3FFFFF) << 22) |
         ((uint64_t)(tx & 0xFF) << 14) | (uint64_t)(ty & 0x3FFF);
}
__device__ __forceinline__ void ring_store(uint32_t cluster_addr, uint64_t v) {
  asm volatile("st.release.cluster.shared::cluster.b64 [%0], %1;" ::"r"(cluster_addr), "l"(v) : "memory");
}
__device__ __forceinline__ uint64_t ring_load(uint32_t addr) {
  uint64_t v;
  asm volatile("ld.acquire.cluster.shared::cta.b64 %0, [%1];" : "=l"(v) : "r"(addr) : "memory");
  return v;
}
// The worker's n-th item, once the dispatcher has published it.  Called by one thread; kind = -1 when
// the CTA is aborting, kind = -2 at the end of the work.
__device__ __forceinline__ Item ring_read(const TcParams& p, uint32_t ring0, int n, volatile int* abort_flag,
                                          uint64_t limit_ns) {
  const uint32_t addr = ring0 + (uint32_t)(n % RING) * 8u;
  const uint64_t tag = (uint64_t)((n + 1) & 0xFFF);
  uint64_t v = ring_load(addr);
  Item q;
  q.kind = -1; q.ph = q.it = q.m = q.slot = q.N = q.Kd = 0; q.tt = make_int2(0, 0);
  if ((v >> 52) != tag) {
    const uint64_t t0 = global_timer_ns();
    for (;;) {
      v = ring_load(addr);
      if ((v >> 52) == tag) break;
      if (*abort_flag) return q;
      if (global_timer_ns() - t0 > limit_ns) { *abort_flag = 1; return q; }
    }
  }
  q.ph = (int)((v >> 44) & 0xFF);
  if (q.ph == RING_STOP) { q.kind = -2; return q; }
  q.it = q.ph / 3;
  q.m = (int)((v >> 22) & 0x3FFFFF);
  q.slot = q.m % p.n_slots;
  q.tt = make_int2((int)((v >> 14) & 0xFF), (int)(v & 0x3FFF));
  const int r3 = q.ph - 3 * q.it;
  q.kind = (r3 == 0) ? GEMM_GRAM : (r3 == 1) ? GEMM_POLY : (q.ph == p.last_ph ? GEMM_FINAL : GEMM_APPLY);
  const bool sym = r3 < 2;
  q.N = sym ? p.s : p.l;
  q.Kd = (r3 == 0) ? p.l : p.s;
  return q;
}

// ------------------------------- the kernel --------------------------------
template <int CG>
__global__ void __launch_bounds__(TC_THREADS, 1)
ns_tc_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
  constexpr int STAGES = TC_STAGES;
  constexpr int BN = 128 * CG;                 // accumulator columns = tile columns
  constexpr int TM = 128 * CG;                 // tile rows (over the CTA pair)
  constexpr uint32_t TMEM_COLS = 2 * BN;
  constexpr int NCH = BN / 64;                 // 64-column epilogue blocks per tile
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[STAGES];    // used in the CTA of rank 0
  __shared__ __align__(8) uint64_t bar_empty[STAGES];
  __shared__ __align__(8) uint64_t bar_tfull[2];
  __shared__ __align__(8) uint64_t bar_tempty[2];       // used in the CTA of rank 0
  __shared__ __align__(8) uint64_t bar_cin[4][2];
  __shared__ __align__(8) uint64_t bar_w[4][4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile int abort_flag;
  __shared__ __align__(8) uint64_t item_ring[RING];      // written by the dispatcher (of rank 0)
  __shared__ int prod_started;                           // rank 0: tiles the producer has begun

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = (CG == 2) ? cluster_ctarank() : 0u;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint64_t limit = p.wait_limit_ns;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    prod_started = 0;
    for (int i = 0; i < RING; ++i) item_ring[i] = 0;
#pragma unroll 1
    for (int i = 0; i < N_MAPS; ++i) asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.m[i]) : "memory");
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&bar_tfull[a]), 1);
      mbar_init(smem_u32(&bar_tempty[a]), 4 * CG);
    }
    for (int w = 0; w < 4; ++w) {
      for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&bar_cin[w][b]), 1);
      for (int b = 0; b < 4; ++b) mbar_init(smem_u32(&bar_w[w][b]), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc<CG>(smem_u32(&tmem_base_slot), TMEM_COLS);
  tc_fence_before();
  if (CG == 2) cluster_sync_all(); else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    // One thread runs the whole loop; the other lanes wait at the end.
    if (lane == 0) {
      const uint32_t empty0 = smem_u32(&bar_empty[0]);
      const uint32_t full0 = smem_u32(&bar_full[0]);
      // both CTAs' copies are counted on the barrier of rank 0, which expects the sum
      const uint32_t full0_bar = (CG == 2) ? map_to_rank(full0, 0) : full0;
      uint32_t stage = 0, phase = 0;
      bool alive = true;
      const uint32_t ring0 = smem_u32(&item_ring[0]);
      const uint32_t started_addr = smem_u32(&prod_started);
      for (int n_local = 0; alive; ++n_local) {
        const Item q = ring_read(p, ring0, n_local, &abort_flag, limit);
        if (q.kind < 0) break;                               // end of the work, or aborting
        // the dispatcher may now claim the item after this one
        if (rank == 0) asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(started_addr), "r"(n_local + 1) : "memory");
        // what the other CTAs wrote through the async proxy is read through the async proxy next
        asm volatile("fence.proxy.async;" ::: "memory");
        const bool sym = q.kind <= GEMM_POLY;
        const bool b_is_x = q.kind >= GEMM_APPLY;             // right operand: X, MN-major
        const bool same = sym && (q.tt.x == q.tt.y);          // diagonal tile: right slab == left slab
        const int xsel = (q.it == 0) ? 0 : ((q.it & 1) ? 1 : 2);
        const CUtensorMap* mA;
        const CUtensorMap* mB;
        const CUtensorMap* mS;
        int zA, zB;
        if (q.kind == GEMM_GRAM) {
          mA = mB = &maps.m[MAP_X0_K + xsel];
          zA = zB = (q.it == 0) ? q.m : q.slot;
          mS = mA;
        } else if (q.kind == GEMM_POLY) {
          mA = mB = &maps.m[MAP_A_K];
          zA = zB = q.slot;
          mS = &maps.m[MAP_A_MN];
        } else {
          mA = &maps.m[MAP_B_K];
          zA = q.slot;
          mB = &maps.m[MAP_X0_MN + xsel];
          zB = (q.it == 0) ? q.m : q.slot;
          mS = &maps.m[MAP_B_MN];
        }
        const int a_row = BM * (CG * q.tt.x + (int)rank);
        const int b_off = TM * q.tt.y + 128 * (int)rank;
        const uint32_t cta_bytes = A_STAGE_BYTES + (same ? 0u : B_STAGE_BYTES);
        // blocks of a symmetric operand below the diagonal are not stored: their k slab is fetched
        // from the mirror image as two 64-column atoms (k rows, 64 operand rows each)
        const int ka_mn = (q.kind != GEMM_GRAM) ? (TM / BK) * q.tt.x : 0;
        const int kb_mn = (q.kind == GEMM_POLY) ? (TM / BK) * q.tt.y : 0;
        const int num_kb = (q.Kd + BK - 1) / BK;
        // test hook: the first k slab of the very first item of the list
        bool withhold = (p.debug_withhold != 0) && q.ph == 0 && q.m == 0 && q.tt.x == 0 && q.tt.y == 0;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty0 + stage * 8u, phase ^ 1u, &abort_flag, limit)) { alive = false; break; }
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + A_STAGE_BYTES;
          const uint32_t bar = full0_bar + stage * 8u;
          if (withhold) {
            // test hook: nothing is expected and nothing is copied for this stage, so the MMA
            // issuer's wait for it runs out
            withhold = false;
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            continue;
          }
          if (CG == 1) mbar_expect_tx(bar, cta_bytes);
          else if (rank == 0) mbar_expect_tx(full0 + stage * 8u, 2u * cta_bytes);
          auto load = [&](uint32_t dst, const CUtensorMap* map, int c0, int c1, int z) {
            if (CG == 1) tma_load_3d(dst, map, bar, c0, c1, z);
            else tma_load_3d_pair(dst, map, bar, c0, c1, z);
          };
          // an MN-major slab = two 64-column atoms of 64 k rows: one 4-D copy, or two 64 x 64 boxes
          auto load_mn = [&](uint32_t dst, const CUtensorMap* map, bool wide, int col0, int k, int z) {
            if (wide) {
              if (CG == 1) tma_load_4d(dst, map, bar, 0, k, col0 >> 6, z);
              else tma_load_4d_pair(dst, map, bar, 0, k, col0 >> 6, z);
            } else {
              load(dst, map, col0, k, z);
              load(dst + BK * 128, map, col0 + 64, k, z);
            }
          };
          const int k0 = kb * BK;
          if (kb >= ka_mn) load(sa, mA, k0, a_row, zA);
          else load_mn(sa, mS, p.s_wide != 0, a_row, k0, q.slot);
          if (!same) {
            if (b_is_x) load_mn(sb, mB, p.x_wide != 0, b_off, k0, zB);
            else if (kb >= kb_mn) load(sb, mB, k0, b_off, zB);
            else load_mn(sb, mS, p.s_wide != 0, b_off, k0, q.slot);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    // One thread runs the whole loop (the other lanes wait at the end): per k slab it waits for the
    // stage, issues four MMAs whose descriptors differ from the stage's base by a constant step,
    // and commits the stage to both CTAs' empty barriers.
    if (rank == 0 && lane == 0) {
      // fp32 accumulate, bf16 x bf16; bit 15 / bit 16: left / right operand is MN-major
      constexpr uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) |
                                  ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
      // descriptor halves: high = SBO 1024 B | version 1 | 128-byte swizzle; low = address/16 | LBO/16 << 16
      constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
      constexpr uint32_t LBO_K = (16u >> 4) << 16, LBO_MN = ((uint32_t)(BK * 128) >> 4) << 16;
      constexpr uint32_t STEP_K = (UMMA_K * 2) >> 4, STEP_MN = (UMMA_K * 128) >> 4;
      const uint32_t full0 = smem_u32(&bar_full[0]);
      const uint32_t empty0 = smem_u32(&bar_empty[0]);
      const uint32_t empty0_peer = (CG == 2) ? map_to_rank(empty0, 1) : 0u;
      const uint32_t tfull0 = smem_u32(&bar_tfull[0]);
      const uint32_t tfull0_peer = (CG == 2) ? map_to_rank(tfull0, 1) : 0u;
      uint32_t stage = 0, phase = 0;
      int local_tile = 0;
      bool alive = true;
      const uint32_t ring0 = smem_u32(&item_ring[0]);
      for (; alive; ++local_tile) {
        const Item q = ring_read(p, ring0, local_tile, &abort_flag, limit);
        if (q.kind < 0) break;
        const bool sym = q.kind <= GEMM_POLY;
        const bool same = sym && (q.tt.x == q.tt.y);
        const int num_kb = (q.Kd + BK - 1) / BK;
        // k slabs below these indices come from the mirror image (MN-major), as staged by the producer
        const int ka_mn = (q.kind != GEMM_GRAM) ? (TM / BK) * q.tt.x : 0;
        const int kb_mn = (q.kind >= GEMM_APPLY) ? num_kb : ((q.kind == GEMM_POLY) ? (TM / BK) * q.tt.y : 0);
        const uint32_t acc = (uint32_t)local_tile & 1u;
        const uint32_t acc_phase = (uint32_t)(local_tile >> 1) & 1u;
        const uint32_t d_tmem = tmem_base + acc * (uint32_t)BN;
        if (!mbar_wait(smem_u32(&bar_tempty[acc]), acc_phase ^ 1u, &abort_flag, limit)) break;
        tc_fence_after();
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full0 + stage * 8u, phase, &abort_flag, limit)) { alive = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * STAGE_BYTES;
          const uint32_t sb = same ? sa : sa + A_STAGE_BYTES;
          const bool a_mn = kb < ka_mn, b_mn = kb < kb_mn;
          const uint32_t idesc = idesc0 | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16);
          const uint32_t alo = (sa >> 4) | (a_mn ? LBO_MN : LBO_K), astep = a_mn ? STEP_MN : STEP_K;
          const uint32_t blo = (sb >> 4) | (b_mn ? LBO_MN : LBO_K), bstep = b_mn ? STEP_MN : STEP_K;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adesc = ((uint64_t)DESC_HI << 32) | (uint64_t)(alo + (uint32_t)k * astep);
            const uint64_t bdesc = ((uint64_t)DESC_HI << 32) | (uint64_t)(blo + (uint32_t)k * bstep);
            tc_mma_bf16<CG>(d_tmem, adesc, bdesc, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit<CG>(empty0 + stage * 8u);
          if (CG == 2) tc_commit<CG>(empty0_peer + stage * 8u);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (alive) {
          tc_commit<CG>(tfull0 + acc * 8u);
          if (CG == 2) tc_commit<CG>(tfull0_peer + acc * 8u);
        }
      }
    }
    __syncwarp();
  } else if (warp == 6) {
    // ------------------------------- dispatcher -------------------------------
    if (rank == 0 && lane == 0) {
      const uint32_t ring0 = smem_u32(&item_ring[0]);
      const uint32_t ring0_peer = (CG == 2) ? map_to_rank(ring0, 1) : 0u;
      const uint32_t started_addr = smem_u32(&prod_started);
      auto publish = [&](int n, uint64_t v) {
        ring_store(ring0 + (uint32_t)(n % RING) * 8u, v);
        if (CG == 2) ring_store(ring0_peer + (uint32_t)(n % RING) * 8u, v);
      };
      int cur = 0;
      for (int n = 0;; ++n) {
        // stay one item ahead of the producer: item n is claimed once the producer has begun item n - 1
        // (claiming further ahead was measured slower: a claimed item that waits behind its worker's
        // current tile holds up the items that depend on it)
        if (n >= 1) {
          int st;
          asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(st) : "r"(started_addr) : "memory");
          if (st < n) {
            const uint64_t t0 = global_timer_ns();
            bool ok = true;
            for (;;) {
              asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(st) : "r"(started_addr) : "memory");
              if (st >= n) break;
              if (abort_flag) { ok = false; break; }
              if (global_timer_ns() - t0 > limit) { abort_flag = 1; ok = false; break; }
              __nanosleep(32);
            }
            if (!ok) break;
          }
        }
        const int item = atomicAdd(p.ticket, 1);
        if (item >= p.total_items) { publish(n, ring_pack(n, RING_STOP, 0, 0, 0)); break; }
        const Item q = decode_item(p, item, cur);
        if (q.kind < 0) { abort_flag = 2; break; }
        if (!dep_wait<CG>(p, q, &abort_flag)) break;
        publish(n, ring_pack(n, q.ph, q.m, q.tt.x, q.tt.y));
      }
    }
    __syncwarp();
  } else {
    // -------------------------------- epilogue --------------------------------
    const int quarter = warp & 3;          // TMEM lanes [32*quarter, 32*quarter+32)
    const int ew = warp - 2;               // staging slot of this warp
    const uint32_t epi = smem_base + STAGES * STAGE_BYTES + (uint32_t)ew * EPI_WARP_BYTES;
    // staging blocks of this warp: addend 0/1 (when there is one), then results 0/1
    auto cin_buf = [&](uint32_t b) { return epi + b * EPI_BLOCK_BYTES; };
    const uint32_t cin_bar0 = smem_u32(&bar_cin[ew][0]);
    auto cin_bar = [&](uint32_t b) { return cin_bar0 + b * 8u; };
    // parameter update through TMA: a ring of four 32 x 32 fp32 blocks, the whole staging space of
    // the warp (the final product has no addend and stages no results)
    auto w_buf = [&](uint32_t b) { return epi + b * EPI_BLOCK_BYTES; };
    const uint32_t w_bar0 = smem_u32(&bar_w[ew][0]);
    auto w_bar = [&](uint32_t b) { return w_bar0 + b * 8u; };
    uint32_t w_issued = 0, w_used = 0;
    uint32_t cin_issued = 0, cin_used = 0, st_count = 0, t_count = 0;
    int local_tile = 0;
    bool alive = true;
    int prev_kind = -1;
    const uint32_t ring0 = smem_u32(&item_ring[0]);
    for (; alive; ++local_tile) {
      // lane 0 reads the ring, the packed item goes to the other lanes by shuffle
      Item q;
      {
        Item q0;
        q0.kind = 0; q0.ph = q0.it = q0.m = q0.slot = q0.N = q0.Kd = 0; q0.tt = make_int2(0, 0);
        if (lane == 0) q0 = ring_read(p, ring0, local_tile, &abort_flag, limit);
        q.kind = __shfl_sync(0xffffffffu, q0.kind, 0); q.ph = __shfl_sync(0xffffffffu, q0.ph, 0);
        q.it = __shfl_sync(0xffffffffu, q0.it, 0);     q.m = __shfl_sync(0xffffffffu, q0.m, 0);
        q.slot = __shfl_sync(0xffffffffu, q0.slot, 0); q.N = __shfl_sync(0xffffffffu, q0.N, 0);
        q.Kd = __shfl_sync(0xffffffffu, q0.Kd, 0);
        q.tt.x = __shfl_sync(0xffffffffu, q0.tt.x, 0); q.tt.y = __shfl_sync(0xffffffffu, q0.tt.y, 0);
      }
      if (q.kind < 0) { alive = false; break; }
      const int acc = local_tile & 1;
      const uint32_t acc_phase = (uint32_t)(local_tile >> 1) & 1u;
      const int2 tt = q.tt;
      const int mat = q.m;
      // Only the polynomial has an addend (b A).  Its epilogue also adds a to the diagonal, B' = B + a I,
      // so that the third product of the iteration, a X + B X = B' X, needs none.
      const bool has_cin = (q.kind == GEMM_POLY);
      const bool stores = (q.kind != GEMM_FINAL);
      const bool upd = (q.kind == GEMM_FINAL && p.sink_mode == SINK_UPDATE_W);
      const uint32_t o_first = (q.kind == GEMM_GRAM || q.kind == GEMM_APPLY) ? 0u : 2u;   // addend blocks come first
      auto out_buf = [&](uint32_t b) { return epi + (o_first + b) * EPI_BLOCK_BYTES; };
      const CUtensorMap* mC = &maps.m[MAP_A_IO];
      const CUtensorMap* mD = (q.kind == GEMM_GRAM) ? &maps.m[MAP_A_IO]
                              : (q.kind == GEMM_POLY) ? &maps.m[MAP_B_IO]
                              : &maps.m[(q.it & 1) ? MAP_XB_IO : MAP_XA_IO];
      if (q.kind != prev_kind) {
        // the staging space is laid out per product: everything the previous product handed to the
        // bulk stores has been read before it is reused under another layout
        if (lane == 0) bulk_wait_read_0();
        __syncwarp();
        prev_kind = q.kind;
      }
      const int rb = CG * tt.x + (int)rank;                 // 128-row block of this CTA
      const int gi0 = rb * BM + quarter * 32;               // first row of this warp
      const int gi = gi0 + lane;
      const bool row_ok = gi < p.s;
      // 64-column blocks of this tile that this warp has to produce
      uint32_t todo = 0;
      if (gi0 < p.s) {
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const int gj0 = TM * tt.y + c * 64;
          if (gj0 < q.N) todo |= 1u << c;
        }
      }
      auto issue_cin = [&](int c) {
        if (lane == 0) {
          const uint32_t b = cin_issued & 1u;
          mbar_expect_tx(cin_bar(b), EPI_BLOCK_BYTES);
          tma_load_3d(cin_buf(b), mC, cin_bar(b), TM * tt.y + c * 64, gi0, q.slot);
        }
        ++cin_issued;
      };
      if (has_cin && todo) {
        // the addend is the Gram matrix of this iteration: the item was only published once all of its
        // tiles were in memory
        if (lane == 0) asm volatile("fence.proxy.async;" ::: "memory");
        issue_cin(__ffs(todo) - 1);
      }
      // fused parameter update: the old parameters come in as 32 x 32 blocks, two steps ahead
      MatDesc dsc;
      dsc.wmap = nullptr; dsc.transposed = 0; dsc.lr_eff = 0.f; dsc.wd_term = 0.f;
      if (upd) dsc = p.mats[mat];
      const bool use_tma = upd && dsc.wmap != nullptr && todo != 0;
      int n_hb = 0;                                      // 32-column blocks of this warp in this tile
      if (use_tma) n_hb = min(2 * NCH, (q.N - TM * tt.y + 31) >> 5);
      auto issue_w = [&](int hb) {
        if (lane == 0) {
          const uint32_t b = w_issued & 3u;
          const int gjh = TM * tt.y + hb * 32;
          mbar_expect_tx(w_bar(b), EPI_BLOCK_BYTES);
          if (!dsc.transposed) tma_load_2d(w_buf(b), dsc.wmap, w_bar(b), gjh, gi0);
          else tma_load_2d(w_buf(b), dsc.wmap, w_bar(b), gi0, gjh);
        }
        ++w_issued;
      };
      if (use_tma) {
        if (lane == 0) bulk_wait_read_2();               // blocks stored three and more steps ago have left the ring
        __syncwarp();
        issue_w(0);
        if (n_hb > 1) issue_w(1);
      } else if (upd) {
        if (lane == 0) bulk_wait_read_0();               // plain path reuses the staging space
        __syncwarp();
      }
      if (!mbar_wait(smem_u32(&bar_tfull[acc]), acc_phase, &abort_flag, limit)) alive = false;
      alive = __all_sync(0xffffffffu, alive);
      if (!alive) break;
      tc_fence_after();
      float sc = 1.f;
      if (p.scales && q.it == 0 && q.kind != GEMM_POLY) sc = (q.kind == GEMM_GRAM) ? p.scales[mat].x : p.scales[mat].y;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
      while (todo) {
        const int c = __ffs(todo) - 1;
        todo &= todo - 1;
        const int gj0 = TM * tt.y + c * 64;
        if (has_cin) {
          if (todo) issue_cin(__ffs(todo) - 1);
          bool ok = mbar_wait(cin_bar(cin_used & 1u), (cin_used >> 1) & 1u, &abort_flag, limit);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { alive = false; break; }
        }
        const uint32_t cbuf = cin_buf(cin_used & 1u);
        const uint32_t obuf = out_buf(st_count & 1u);
        if (stores) {
          if (lane == 0) bulk_wait_read_1();     // the block stored two steps ago has left this buffer
          __syncwarp();
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t v[32];
          tc_ld32(t_row + (uint32_t)(c * 64 + h * 32), v);
          float f[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
          if (has_cin) {
            float add[32];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              const uint4 u = lds128(cbuf + (uint32_t)lane * 128u + ((uint32_t)((h * 4 + q4) ^ (lane & 7)) << 4));
              add[q4 * 8 + 0] = bf16_lo(u.x); add[q4 * 8 + 1] = bf16_hi(u.x);
              add[q4 * 8 + 2] = bf16_lo(u.y); add[q4 * 8 + 3] = bf16_hi(u.y);
              add[q4 * 8 + 4] = bf16_lo(u.z); add[q4 * 8 + 5] = bf16_hi(u.z);
              add[q4 * 8 + 6] = bf16_lo(u.w); add[q4 * 8 + 7] = bf16_hi(u.w);
            }
            const int dcol = gi - (gj0 + h * 32);        // this lane's diagonal element, if it is in the block
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] = fmaf(p.c, f[e], p.b * add[e]) + ((e == dcol) ? p.a : 0.0f);
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] *= sc;
          }
          if (!stores) {
            // ---- parameter update / output sink (tensor in its own layout and type) ----
            // Lanes run along the tensor's contiguous axis, so every access of the warp is one
            // full line: for a tensor stored rows x cols as s x l that axis is the tile's column
            // axis and the block is first turned through shared memory; for a tensor stored
            // l x s it is the tile's row axis, which the lanes already hold.
            const int gjh = gj0 + h * 32;
            if (use_tma) {
              if (gjh < q.N) {
                const int hb = 2 * c + h;
                if (lane == 0) bulk_wait_read_1();       // the block stored two steps ago has left the ring
                __syncwarp();
                if (hb + 2 < n_hb) issue_w(hb + 2);
                bool ok = mbar_wait(w_bar(w_used & 3u), (w_used >> 2) & 1u, &abort_flag, limit);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { alive = false; break; }
                const uint32_t wb = w_buf(w_used & 3u);
                if (!dsc.transposed) {
                  // block rows are tile rows: each lane owns one 128-byte row (swizzled)
#pragma unroll
                  for (int q4 = 0; q4 < 8; ++q4) {
                    const uint32_t ad = wb + (uint32_t)lane * 128u + ((uint32_t)(q4 ^ (lane & 7)) << 4);
                    uint4 u = lds128(ad);
                    float w0 = __uint_as_float(u.x), w1 = __uint_as_float(u.y), w2 = __uint_as_float(u.z),
                          w3 = __uint_as_float(u.w);
                    w0 = fmaf(-dsc.lr_eff, f[q4 * 4 + 0], fmaf(-dsc.wd_term, w0, w0));
                    w1 = fmaf(-dsc.lr_eff, f[q4 * 4 + 1], fmaf(-dsc.wd_term, w1, w1));
                    w2 = fmaf(-dsc.lr_eff, f[q4 * 4 + 2], fmaf(-dsc.wd_term, w2, w2));
                    w3 = fmaf(-dsc.lr_eff, f[q4 * 4 + 3], fmaf(-dsc.wd_term, w3, w3));
                    sts128(ad, make_uint4(__float_as_uint(w0), __float_as_uint(w1), __float_as_uint(w2),
                                          __float_as_uint(w3)));
                  }
                } else {
                  // block rows are tile columns: lane i reads element i of every row
#pragma unroll
                  for (int e = 0; e < 32; ++e) {
                    const uint32_t ad = wb + (uint32_t)e * 128u + (uint32_t)lane * 4u;
                    const float wv = __uint_as_float(lds32(ad));
                    sts32(ad, __float_as_uint(fmaf(-dsc.lr_eff, f[e], fmaf(-dsc.wd_term, wv, wv))));
                  }
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                  if (!dsc.transposed) tma_store_2d(dsc.wmap, wb, gjh, gi0);
                  else tma_store_2d(dsc.wmap, wb, gi0, gjh);
                  bulk_commit();
                }
                ++w_used;
              }
            } else if (gjh < q.N) {
              const MatDesc d = p.mats[mat];
              const bool full = (gi0 + 32 <= p.s) && (gjh + 32 <= q.N);
              if (full) {
                float o[32];
                int64_t base, stride;
                if (!d.transposed) {
                  const uint32_t tb = epi + (2u + (t_count & 1u)) * EPI_BLOCK_BYTES;
                  ++t_count;
#pragma unroll
                  for (int q4 = 0; q4 < 8; ++q4)
                    sts128(tb + (uint32_t)lane * 128u + ((uint32_t)(q4 ^ (lane & 7)) << 4),
                           make_uint4(__float_as_uint(f[q4 * 4 + 0]), __float_as_uint(f[q4 * 4 + 1]),
                                      __float_as_uint(f[q4 * 4 + 2]), __float_as_uint(f[q4 * 4 + 3])));
                  __syncwarp();
#pragma unroll
                  for (int r = 0; r < 32; ++r)
                    o[r] = __uint_as_float(lds32(tb + (uint32_t)r * 128u + ((uint32_t)((lane >> 2) ^ (r & 7)) << 4) +
                                                 (uint32_t)(lane & 3) * 4u));
                  base = (int64_t)gi0 * p.l + gjh + lane;
                  stride = p.l;
                } else {
#pragma unroll
                  for (int e = 0; e < 32; ++e) o[e] = f[e];
                  base = (int64_t)gjh * p.s + gi0 + lane;
                  stride = p.s;
                }
                if (p.sink_mode == SINK_UPDATE_W) {
                  float* W = reinterpret_cast<float*>(d.w) + base;
                  float wv[32];
#pragma unroll
                  for (int r = 0; r < 32; ++r) wv[r] = W[(int64_t)r * stride];
#pragma unroll
                  for (int r = 0; r < 32; ++r)
                    W[(int64_t)r * stride] = fmaf(-d.lr_eff, o[r], fmaf(-d.wd_term, wv[r], wv[r]));
                } else if (p.sink_mode == SINK_STORE_F32) {
                  float* O = reinterpret_cast<float*>(d.w) + base;
#pragma unroll
                  for (int r = 0; r < 32; ++r) O[(int64_t)r * stride] = o[r];
                } else {
                  __nv_bfloat16* O = reinterpret_cast<__nv_bfloat16*>(d.w) + base;
#pragma unroll
                  for (int r = 0; r < 32; ++r) O[(int64_t)r * stride] = __float2bfloat16_rn(o[r]);
                }
              } else if (row_ok) {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                  if (gjh + e < q.N) sink_element(d, p.sink_mode, p.s, p.l, gi, gjh + e, f[e]);
              }
            }
          } else {
            // ---- stage the bf16 block for the bulk store ----
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              uint4 u;
              u.x = pack_bf16x2(f[q4 * 8 + 0], f[q4 * 8 + 1]);
              u.y = pack_bf16x2(f[q4 * 8 + 2], f[q4 * 8 + 3]);
              u.z = pack_bf16x2(f[q4 * 8 + 4], f[q4 * 8 + 5]);
              u.w = pack_bf16x2(f[q4 * 8 + 6], f[q4 * 8 + 7]);
              sts128(obuf + (uint32_t)lane * 128u + ((uint32_t)((h * 4 + q4) ^ (lane & 7)) << 4), u);
            }
          }
        }
        if (!alive) break;
        if (has_cin) ++cin_used;
        if (stores) {
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_3d(mD, obuf, gj0, gi0, q.slot);
            bulk_commit();
          }
          ++st_count;
        } else {
          __syncwarp();
        }
      }
      if (!alive) break;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        const uint32_t te = smem_u32(&bar_tempty[acc]);
        mbar_arrive_cluster(CG == 2 ? map_to_rank(te, 0) : te);
        // This warp's part of the tile: for a stored product its results are in memory once the
        // bulk stores have completed; the final product only has to have read its operands, which
        // it has (its accumulator was complete), so the ring slot may be reused.
        if (stores) bulk_wait_all();
        signal_done(p, q);
      }
    }
    bulk_wait_all();
  }

  // ------------------------------- teardown ----------------------------------
  if (abort_flag) {
    // give copies and MMAs still in flight time to land before memory is released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    if (threadIdx.x == 0) atomicOr(p.status, abort_flag == 2 ? ST_BOUNDS : ST_TIMEOUT);
  }
  tc_fence_before();
  if (CG == 2) cluster_sync_all(); else __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<CG>(tmem_base, TMEM_COLS);
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
                int box_cols, int box_rows, bool swizzle128) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)n_slots};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)rows * (cuuint64_t)ld * 2};
  cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// 4-D map over the same array for MN-major operands: [n_slots][cols/64][rows][64], box 64 x 64 x 2 x 1,
// i.e. two consecutive 64-column atoms (64 rows of 128 bytes each, 8 KB apart in shared memory) per copy.
// Needs cols % 64 == 0.
bool encode_map_mn2(CUtensorMap* out, void* base, int64_t cols, int64_t rows, int64_t n_slots, int64_t ld) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn || (cols & 63) != 0) return false;
  cuuint64_t dims[4] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64), (cuuint64_t)n_slots};
  cuuint64_t strides[3] = {(cuuint64_t)ld * 2, 128, (cuuint64_t)rows * (cuuint64_t)ld * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)BK, 2, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

bool tc_encode_w_map(void* out_host, void* base, int64_t rows, int64_t cols, int transposed) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn || (((uintptr_t)base) & 15) != 0 || (cols & 3) != 0) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
  cuuint32_t box[2] = {32, 32};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap m;
  CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, transposed ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  static_assert(sizeof(CUtensorMap) == TC_MAP_BYTES, "TMA descriptor size");
  memcpy(out_host, &m, sizeof m);
  return true;
}

namespace {

// Number of tile workers (CTAs for CG = 1, CTA pairs for CG = 2) that can be resident at once.
template <int CG>
int resident_units(int n_sms, cudaError_t* err) {
  static int cached = 0;
  *err = cudaSuccess;
  if (cached) return cached;
  cudaError_t e = cudaFuncSetAttribute(ns_tc_kernel<CG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)TC_SMEM_BYTES);
  if (e != cudaSuccess) { *err = e; return 0; }
  if (CG == 1) {
    cached = n_sms;
    return cached;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((unsigned)(n_sms / 2 * 2));
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = TC_SMEM_BYTES;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, ns_tc_kernel<CG>, &cfg);
  if (e != cudaSuccess) { *err = e; return 0; }
  if (n < 1) { *err = cudaErrorLaunchOutOfResources; return 0; }
  cached = n;
  return cached;
}

template <int CG>
cudaError_t launch_one(cudaStream_t st, const TcMaps& m, const TcParams& p, int n_sms) {
  cudaError_t e;
  const int units = resident_units<CG>(n_sms, &e);
  if (e != cudaSuccess) return e;
  // every worker must be resident for the whole launch (items wait for items of other workers)
  const int workers = p.total_items < units ? p.total_items : units;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((unsigned)(workers * CG));
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = TC_SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = CG; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, ns_tc_kernel<CG>, m, p);
}

struct BlockTable {
  TcBlock* dev = nullptr;
  int n_blocks = 0, total_items = 0;
};

}  // namespace

struct TcGroupPlan {
  int64_t s, l, ldx, lds;
  int chunk;
  int cg;                       // CTAs per tile worker (1 or 2)
  int group, n_slots;           // matrices per group of the work list, ring slots (tc_ring_slots(group))
  int ns_steps, cw;
  TcMaps maps;
  bool wide_x = false, wide_s = false;
  int2* tiles_sym = nullptr;
  int n_sym = 0;
  int2* tiles_full = nullptr;
  int n_full = 0;
  int* counters = nullptr;
  std::map<int, BlockTable> tables;   // work list per matrix count
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

// Matrices per group of the work list: about one round of the tile workers per block of a symmetric
// product (at least two matrices).  Measured on the four benchmark shape mixes (Newton-Schulz ms per
// inner step against the group size): smaller groups leave a product's tiles still running when the
// matrix's next product comes up, larger ones push the intermediates out of L2.
int tc_group_size(int64_t s, int chunk) {
  const int cg = (s > 128) ? 2 : 1;
  const int64_t T = 128 * cg;
  const int64_t tm = (s + T - 1) / T;
  const int64_t n_sym = tm * (tm + 1) / 2;
  const int units = tc_num_sms() / cg;
  int64_t g = (units + n_sym - 1) / n_sym;
  if (g < 2) g = 2;
  if (const char* e = getenv("MULOCO_NS_GROUP")) {     // tuning studies
    const int v = atoi(e);
    if (v > 0) g = v;
  }
  if (g < 1) g = 1;
  if (g > chunk) g = chunk;
  return (int)g;
}

// Three groups are in flight at a time (see get_table) and a fourth set of slots belongs to the group
// that finished last, so that a new group never waits for its slots.
int tc_ring_slots(int group) { return 4 * group; }

size_t tc_ring_bytes(int64_t s, int64_t ldx, int64_t lds, int n_slots) {
  const size_t xb = ((size_t)n_slots * s * ldx * 2 + 1023) / 1024 * 1024;
  const size_t sb = ((size_t)n_slots * s * lds * 2 + 1023) / 1024 * 1024;
  return 2 * xb + 2 * sb;
}

TcGroupPlan* tc_plan_create(int64_t s, int64_t l, int chunk, void* X0, int64_t ldx, void* ring, int64_t lds,
                            int group, int* counters, int ns_steps, char* err, size_t errlen) {
  TcGroupPlan* pl = new TcGroupPlan();
  pl->s = s; pl->l = l; pl->ldx = ldx; pl->lds = lds; pl->chunk = chunk;
  pl->group = group; pl->n_slots = tc_ring_slots(group);
  pl->ns_steps = ns_steps; pl->cw = 3 * ns_steps;
  pl->counters = counters;
  pl->n_sms = tc_num_sms();
  pl->cg = (s > 128) ? 2 : 1;
  const int ns = pl->n_slots;
  const size_t xb = ((size_t)ns * s * ldx * 2 + 1023) / 1024 * 1024;
  const size_t sb = ((size_t)ns * s * lds * 2 + 1023) / 1024 * 1024;
  char* r = reinterpret_cast<char*>(ring);
  void* XA = r;
  void* XB = r + xb;
  void* A = r + 2 * xb;
  void* B = r + 2 * xb + sb;
  CUtensorMap* m = pl->maps.m;
  bool ok = true;
  ok = ok && encode_map(&m[MAP_X0_K], X0, l, s, chunk, ldx, BK, 128, true);
  ok = ok && encode_map(&m[MAP_XA_K], XA, l, s, ns, ldx, BK, 128, true);
  ok = ok && encode_map(&m[MAP_XB_K], XB, l, s, ns, ldx, BK, 128, true);
  ok = ok && encode_map(&m[MAP_XA_IO], XA, l, s, ns, ldx, 64, 32, true);
  ok = ok && encode_map(&m[MAP_XB_IO], XB, l, s, ns, ldx, 64, 32, true);
  ok = ok && encode_map(&m[MAP_A_K], A, s, s, ns, lds, BK, 128, true);
  ok = ok && encode_map(&m[MAP_A_IO], A, s, s, ns, lds, 64, 32, true);
  ok = ok && encode_map(&m[MAP_B_K], B, s, s, ns, lds, BK, 128, true);
  ok = ok && encode_map(&m[MAP_B_IO], B, s, s, ns, lds, 64, 32, true);
  // MN-major operands: one 4-D copy per slab when the column count is a multiple of 64 and the
  // driver accepts the layout, else two 64 x 64 boxes
  pl->wide_x = encode_map_mn2(&m[MAP_X0_MN], X0, l, s, chunk, ldx) && encode_map_mn2(&m[MAP_XA_MN], XA, l, s, ns, ldx) &&
               encode_map_mn2(&m[MAP_XB_MN], XB, l, s, ns, ldx);
  if (!pl->wide_x) {
    ok = ok && encode_map(&m[MAP_X0_MN], X0, l, s, chunk, ldx, 64, BK, true);
    ok = ok && encode_map(&m[MAP_XA_MN], XA, l, s, ns, ldx, 64, BK, true);
    ok = ok && encode_map(&m[MAP_XB_MN], XB, l, s, ns, ldx, 64, BK, true);
  }
  pl->wide_s = encode_map_mn2(&m[MAP_A_MN], A, s, s, ns, lds) && encode_map_mn2(&m[MAP_B_MN], B, s, s, ns, lds);
  if (!pl->wide_s) {
    ok = ok && encode_map(&m[MAP_A_MN], A, s, s, ns, lds, 64, BK, true);
    ok = ok && encode_map(&m[MAP_B_MN], B, s, s, ns, lds, 64, BK, true);
  }
  if (getenv("MULOCO_VERBOSE"))
    fprintf(stderr, "muloco: Newton-Schulz plan %lld x %lld, chunk %d, groups of %d (ring of %d slots): one-copy "
            "MN-major slabs for X %s, for A/B %s\n", (long long)s, (long long)l, chunk, group, ns,
            pl->wide_x ? "yes" : "no", pl->wide_s ? "yes" : "no");
  if (!ok) {
    snprintf(err, errlen, "cuTensorMapEncodeTiled failed for shape %lld x %lld", (long long)s, (long long)l);
    delete pl;
    return nullptr;
  }
  std::vector<int2> sym, full;
  const int64_t T = 128 * pl->cg;
  const int tm_n = (int)((s + T - 1) / T);
  for (int tm = 0; tm < tm_n; ++tm)
    for (int tn = tm; tn < tm_n; ++tn) sym.push_back(make_int2(tm, tn));
  const int tn_full = (int)((l + T - 1) / T);
  for (int tm = 0; tm < tm_n; ++tm)
    for (int tn = 0; tn < tn_full; ++tn) full.push_back(make_int2(tm, tn));
  pl->n_sym = (int)sym.size();
  pl->n_full = (int)full.size();
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
  for (auto& kv : pl->tables)
    if (kv.second.dev) cudaFree(kv.second.dev);
  delete pl;
}

namespace {

// The work list for the first n_mats matrices of the chunk.  The matrices are taken in groups of
// `group`; a group runs its products one after the other (Gram, polynomial, apply of iteration 0, 1,
// ...), one block per product, matrix by matrix inside a block.  Three groups are in flight, a third
// of the products apart: in step t of the list, group g is at product t - (n_ph / 3) g.  With five
// iterations (15 products) the three groups of a step are at a Gram, a polynomial and an apply,
// so between a product of a matrix and its next product always lie two blocks of other groups,
// one of them of a long kind, and the matrices in flight stay few (3 * group).
cudaError_t get_table(TcGroupPlan* pl, int n_mats, BlockTable* out) {
  auto it = pl->tables.find(n_mats);
  if (it != pl->tables.end()) { *out = it->second; return cudaSuccess; }
  std::vector<TcBlock> blocks;
  int64_t item = 0;
  const int n_ph = pl->cw;
  const int last_ph = n_ph - 1;
  const int n_groups = (n_mats + pl->group - 1) / pl->group;
  const int lag = (n_ph + 2) / 3;                            // steps between the starts of two groups
  const int n_steps = (n_groups - 1) * lag + n_ph;
  for (int t = 0; t < n_steps; ++t) {
    for (int g = 0; g < n_groups; ++g) {
      const int ph = t - g * lag;
      if (ph < 0) break;
      if (ph > last_ph) continue;
      const int g0 = g * pl->group;
      const int n = (n_mats - g0 < pl->group) ? (n_mats - g0) : pl->group;
      TcBlock b;
      memset(&b, 0, sizeof b);
      b.kind = (ph % 3 == 0) ? GEMM_GRAM : (ph % 3 == 1) ? GEMM_POLY : (ph == last_ph ? GEMM_FINAL : GEMM_APPLY);
      b.ph = ph;
      b.mat0 = g0; b.n_mats = n;
      b.first_item = (int)item;
      b.n_items = n * ((ph % 3 == 2) ? pl->n_full : pl->n_sym);
      item += b.n_items;
      blocks.push_back(b);
    }
  }
  if (item >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;
  BlockTable t;
  t.n_blocks = (int)blocks.size();
  t.total_items = (int)item;
  cudaError_t e = cudaMalloc(&t.dev, blocks.size() * sizeof(TcBlock));
  if (e != cudaSuccess) return e;
  e = cudaMemcpy(t.dev, blocks.data(), blocks.size() * sizeof(TcBlock), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) { cudaFree(t.dev); return e; }
  pl->tables[n_mats] = t;
  *out = t;
  return cudaSuccess;
}

}  // namespace

cudaError_t tc_launch(cudaStream_t st, TcGroupPlan* pl, int n_mats, const NsIterArgs& args) {
  if (n_mats <= 0) return cudaSuccess;
  if (n_mats > pl->chunk) return cudaErrorInvalidValue;
  BlockTable t;
  cudaError_t e = get_table(pl, n_mats, &t);
  if (e != cudaSuccess) return e;
  // tile counters and, behind them, the ticket counter
  e = cudaMemsetAsync(pl->counters, 0, ((size_t)n_mats * pl->cw + 1) * sizeof(int), st);
  if (e != cudaSuccess) return e;
  TcParams p;
  memset(&p, 0, sizeof(p));
  p.blocks = t.dev; p.n_blocks = t.n_blocks; p.total_items = t.total_items;
  p.n_mats = n_mats;
  p.tiles_sym = pl->tiles_sym; p.tiles_full = pl->tiles_full;
  p.n_sym = pl->n_sym; p.n_full = pl->n_full;
  p.s = (int)pl->s; p.l = (int)pl->l;
  p.last_ph = pl->cw - 1;
  p.a = args.a; p.b = args.b; p.c = args.c;
  p.scales = args.scales; p.mats = args.mats; p.sink_mode = args.sink_mode;
  p.x_wide = pl->wide_x; p.s_wide = pl->wide_s;
  p.n_slots = pl->n_slots;
  p.counters = pl->counters; p.cw = pl->cw;
  p.ticket = pl->counters + (size_t)n_mats * pl->cw;
  p.status = args.status;
  p.wait_limit_ns = args.wait_limit_ns ? args.wait_limit_ns : 2000000000ull;
  p.debug_withhold = args.debug_withhold;
  return pl->cg == 2 ? launch_one<2>(st, pl->maps, p, pl->n_sms) : launch_one<1>(st, pl->maps, p, pl->n_sms);
}

}  // namespace muloco
