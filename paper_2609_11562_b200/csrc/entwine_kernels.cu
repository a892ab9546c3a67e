// Fused GEMM-ReduceScatter for sm_100a: one persistent launch whose CTAs are split into
// producers (tcgen05/TMEM GEMM fed by TMA, one flag per finished 128x128 tile) and consumers
// (flag polling, scatter push, fp32-accumulated tile reduction).  See include/entwine.h for
// the contract and the paper sections each step follows.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "entwine_internal.h"

// Optional per-role wait-time counters (builds with -DENTWINE_PROFILE only; off in the product):
// cycles a role spent waiting at each of its synchronisation points, per CTA.
#ifdef ENTWINE_PROFILE
__device__ unsigned long long g_prof[256 * 16];
extern "C" int entwine_debug_read_profile(void* dst, int clear) {
  cudaError_t e = cudaMemcpyFromSymbol(dst, g_prof, sizeof(g_prof));
  if (e == cudaSuccess && clear) {
    static unsigned long long zeros[256 * 16];
    e = cudaMemcpyToSymbol(g_prof, zeros, sizeof(zeros));
  }
  return (int)e;
}
// a role accumulates in a register array and writes it out once, at its end
#define PROF_DECL() unsigned long long prof_acc_[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define PROF_T0() const long long prof_t0_ = clock64()
#define PROF_ADD(k) (prof_acc_[k] += (unsigned long long)(clock64() - prof_t0_))
#define PROF_FLUSH(cond)                                                        \
  do {                                                                          \
    if (cond) {                                                                 \
      for (int k_ = 0; k_ < 16; ++k_)                                           \
        if (prof_acc_[k_]) atomicAdd(&g_prof[blockIdx.x * 16 + k_], prof_acc_[k_]); \
    }                                                                           \
  } while (0)
#else
#define PROF_DECL() do { } while (0)
#define PROF_T0() do { } while (0)
#define PROF_ADD(k) do { } while (0)
#define PROF_FLUSH(cond) do { } while (0)
#endif

namespace entwine {

// ------------------------------------------------------------------------------------------
// compile-time shape of the kernel
// ------------------------------------------------------------------------------------------
constexpr int kBM = 128;          // producer block rows = reduction tile rows
constexpr int kBK = 64;           // K elements per k-block (128 bytes = one swizzle row); a pipeline
                                  // stage holds P.kpb k-blocks of both operands
constexpr int kUmmaK = 16;        // K per tcgen05.mma for 16-bit operands
// Warp roles of the 16 warps of a CTA.  Producer work (warps 0, 1, 4-7) and consumer work
// (warps 2, 3, 8-15) run side by side in a producer CTA: the tensor pipe is driven by one
// thread, so the SM's TMA and ALUs are free to move and reduce tiles meanwhile.
constexpr int kThreads = 576;
constexpr int kTmaWarp = 0;       // producer: TMA loads of A and B
constexpr int kMmaWarp = 1;       // producer: tcgen05.mma issue, TMEM owner
constexpr int kCommWarp = 2;      // consumer: claims tasks, polls flags, issues TMA loads
constexpr int kStoreWarp = 3;     // consumer: TMA stores of pushed tiles, recycles ring slots
constexpr int kEpiWarp0 = 4;      // producer: epilogue warps 4..7
constexpr int kEpiThreads = 128;
constexpr int kRedWarp0 = 8;      // consumer: reducing warps 8..15
constexpr int kRedThreads = 256;
constexpr int kSpareWarp = 16;    // (no role: keeps the flag warp on the sub-core it was measured on)
constexpr int kFlagWarp = 17;     // producer: releases the tile flags of stored blocks
constexpr int kGemmThreads = 256; // warps 0, 1, 4-7, 16, 17
constexpr uint32_t kSpinCheck = 128;  // spins between looks at the timer / abort flag
constexpr int kEpiWarpBytes = 4096;   // an epilogue warp's staging: its 32 rows x 64 columns of bf16, 128B-swizzled

// Shared-memory map (offsets from a 1024-byte aligned base).  The first 224 KiB are split at
// launch time between the producer's operand ring (S stages), the epilogue staging and the
// consumer's ring A, which a producer CTA's consumer warps use while it still produces:
//   [0, S*stage)                operand ring of the producer
//   [S*stage, S*stage + 16 KiB) epilogue staging (4 KiB per epilogue warp)
//   [.., 229376)                consumer ring A (32 KiB with 5 pair stages, 64 KiB with 4, ...)
//   [0, 196608)                 consumer ring B: 6 slots of 32 KiB, used once the CTA's producer
//                               work is over (and by dedicated consumer CTAs from the start)
//   [229376, 230016)            mbarriers, TMEM base slot
constexpr int kDataBytes = 229376;
constexpr int kStagingBytes = 4 * kEpiWarpBytes;
constexpr int kRingBOff = 0;
constexpr int kRingBBytes = 196608;
constexpr int kMaxSlots = 8;
#ifndef ENTWINE_NORM_LOADS
#define ENTWINE_NORM_LOADS 1
#endif
// Layer chain: 1: the reducing warps read the tile to normalise themselves (from L2, eight 16-byte loads per
// thread in flight; the ring slot carries the task only); 0: its rows come into the slot by TMA.
constexpr bool kNormLoads = ENTWINE_NORM_LOADS != 0;
constexpr int kRegSlots = 4;       // task descriptors in flight between the claiming and the reducing warps
constexpr int kMaxStages = 6;
constexpr int kBarOff = kDataBytes;
constexpr int kBarBytes = 640;
constexpr int kBarGemm = 0;        // full[6], empty[6], tfull[2], tempty[2]; 152..191 unused
constexpr int kBarTmemSlot = 136;
constexpr int kBarPair = 144;      // end-of-producer handshake of a CTA pair
constexpr int kBarRingA = 192;     // full[8], empty[8], reduced[8]
constexpr int kBarRingB = 192 + 192;
constexpr int kSmemBytes = kBarOff + kBarBytes + 1024;  // + alignment slack

// PAIR = two CTAs of a cluster compute a 256 x 256 pair tile with tcgen05 cta_group::2: each
// CTA loads its own 128 rows of A and half (128 rows) of the B panel, so a CTA moves 32 KiB
// per k-block instead of 48 KiB.
template <int BN, bool PAIR>
struct Cfg {
  static_assert(!PAIR || BN == 256, "pair tiles are 256 wide");
  static constexpr int kBRows = PAIR ? 128 : BN;  // rows of B this CTA loads per stage
  static constexpr int kABytes = kBM * kBK * 2;     // one k-block of A
  static constexpr int kBBytes = kBRows * kBK * 2;  // one k-block of this CTA's rows of B
  static constexpr int kKBlockBytes = kABytes + kBBytes;  // a stage is P.kpb of these: all of A, then all of B
  static constexpr int kTmemCols = 2 * BN;  // two accumulators: epilogue overlaps next mainloop
};

struct KParams {
  // geometry
  int M, N, K, W, r, order;
  int rowsT, nBn, nTn, Lb, P_blk, Q, cpb;
  long long R;
  // launch shape
  int G;          // CTAs [0, G) are producers (pairs of them in pair mode)
  int n_ded;      // CTAs [G, G + n_ded) are dedicated consumers
  int x;          // consumer lists
  int mode;       // Mode
  int help;       // CTAs take tasks from lists other than their own
  int colocate;   // a producer CTA's consumer warps work while it still produces
  int prefetch;   // pull the next reduce task's peer tiles into L2 ahead of its loads
  int l2_hints;   // consumer TMA traffic carries an evict-first L2 policy
  int stages;     // operand-ring stages of the producer
  int split;      // pair tiles: the last `split` pair tiles of the order are each done as two half-width
                  // units (256 x 128: one 128 x 128 tile per CTA), so that a last wave that fills at
                  // most half of the CTA pairs costs half a tile time; 0 = none
  int b_kn;       // 1: B is given as [K_local, N] (N contiguous); its stage share is one 3-D TMA box
                  // [N groups of 64][k rows][64] and the MMA reads it as an MN-major operand
  int kpb;        // k-blocks (64 elements of K) per stage
  int k3d;        // 1: a stage's k-blocks of one operand arrive as ONE 3-D TMA box (half the load instructions
                  // and barrier transactions of k-block-sized boxes)
  int ring_a_off, ring_a_bytes;  // consumer ring A (after the epilogue staging)
  int stage_area;                // bytes of the operand stages
  int early_b;                   // 1: a producer CTA's ring B is its operand stages, used as soon as its
                                 // last MMA has completed; 0: the full ring B once its producer work is over
  int ring_a_geom;               // which geometry ring A uses (0: 16 KiB steps, 1: 32 KiB steps)
  int reg_a;      // 1: while a producer CTA still produces, its consumer warps run whole-tile tasks from
                  // registers (plain loads and stores) instead of a shared-memory ring: ring A then holds
                  // task descriptors only, all shared memory goes to the operand stages, and the SM's TMA
                  // unit serves the operand loads alone
  int reg_only;   // 1 (with reg_a): the consumer never moves to the TMA ring: every tile, to the end of the
                  // call and in CTAs that do not produce, goes through registers with plain loads
  int skip_wait;  // treat every flag as published (consumer in isolation)
  int claim;      // most consecutive tasks taken from a list per claim
  int release_group;     // blocks released together (1 = each block by itself; -1, -2: see the header)
  unsigned* group_ctr;   // stored blocks per release group (counts modulo the group's size)
  // consumer ring geometry, [0] ring A (small, beside the producer's buffers), [1] ring B
  int rs[2];         // rows of a tile moved per reduce step (all W contributions of those rows)
  int prs[2];        // rows of a tile moved per push step
  int slot_bytes[2]; // bytes of one ring slot
  unsigned epoch;  // flag value of this producer run
  unsigned seq;    // launch counter: selects the status slot
  unsigned long long wait_budget_ns;
  // memory
  __nv_bfloat16* out;            // out_shard [R][N] (written by the reducing warps)
  const __nv_bfloat16* cws;      // the rank's partial C [M][N] as the consumer reads it (register path)
  __nv_bfloat16* cws_out;        // ... as the producer's epilogue writes it
  const __nv_bfloat16* peers;    // incoming partials [W-1][peer_rows][N] (register path; pull mode: see heap)
  int peer_row0;                 // row of the [M,N] numbering that is row 0 of a peer's plane: 0 for the
  int peer_rows;                 // full [W-1][M][N] layout (peer_rows = M), r * R for the compact staging
                                 // of the host-buffer calls, which holds partition r's rows only (= R)
  __nv_bfloat16* send;           // send_bufs [W-1][R][N] (register path)
  long long heap_buf_off;        // pull mode: offset of this call's partial-output buffer inside a segment
  unsigned* flags_own;           // [W][Q]
  const unsigned* flags_peer;    // [W-1][Q]
  const Task* tasks;
  const int* list_offs;          // [x+1]
  // layer chain (residual add + RMSNorm fused into the consumer), off unless norm != 0
  int norm;
  float eps;
  const __nv_bfloat16* residual;  // [R][N]
  const __nv_bfloat16* weight;    // [N]
  __nv_bfloat16* norm_out;        // [R][N]
  float* ssq_part;                // [R][nTn] sum of squares of a row's 128 elements inside one tile
  unsigned* band_ctr;             // [rowsT] reduced tiles per band of 128 rows (cleared per launch)
  // pull mode (ranks on GPUs of their own, Sec. 4.2): every rank's segment of the symmetric heap
  // lies heap_stride bytes after the previous rank's; flags_own and flags_peer both point at
  // this rank's flag array [W sources][Q] inside its segment
  char* heap;                    // rank 0's segment
  long long heap_stride;
  long long heap_flags_off;      // offset of the flag array inside a segment
  int* list_head;                // [x + 1] head counters of this launch; entry x: normalisation tasks
  int* list_head_next;           // [x] head counters of the next launch, rewound by this one (or null)
  StatusSlot* status_next;       // status slot of the next launch, cleared by this one (or null)
  StatusSlot* status;            // [2]
};

// Tensor maps of one launch.  Loads of A and B and the epilogue's stores of C use the
// 128-byte swizzle; the consumer's maps are plain row-major boxes of 128 columns x rs rows.
struct KMaps {
  CUtensorMap a, b;      // operands, one k-block per box
  CUtensorMap a3, b3;    // operands viewed as [K/64][rows][64]: one box brings kpb k-blocks (k3d)
  CUtensorMap bh, bh3;   // B with boxes of 64 rows: a CTA's share of a half-width pair tile
  CUtensorMap bkn, bknh; // B given as [K, N], viewed as [N/64][K][64]: box = kpb*64 k-rows x the CTA's
                         // groups of 64 columns (whole and half-width units)
  // consumer maps, one set per ring (the box height is the ring's rs)
  CUtensorMap c_ld[2];      // partial C, box 128 x rs: the local rows of a reduce step
  CUtensorMap p_ld[2];      // incoming partials as a 3-D tensor [W-1][M][N], box 128 x rs x (W-1):
                            // one load brings all peers' rows of a reduce step
  CUtensorMap res_ld[2];    // layer chain: residual [R, N], box 128 x prs (a tile's residual, ahead of its reduce steps)
  CUtensorMap c_push[2];    // partial C, box 128 x prs: one load per push step
  CUtensorMap send_st[2];   // send_bufs viewed as [(W-1)*R, N], box 128 x prs: one store per push step
  CUtensorMap p_pf;         // incoming partials, whole-tile box, for L2 prefetch
  CUtensorMap p_hi[2];      // pull mode: partials of the ranks above this one (p_ld: the ranks below)
  CUtensorMap h_ld[2];      // layer chain: hidden_out [R, N], box 128 x prs (rows of a tile to normalise)
};

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// L2 eviction-priority policies for the cache-hinted TMA forms
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, int x, int y,
                                                 uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                                 uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap* map, int x, int y, uint32_t src,
                                                  uint64_t policy) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%1, %2}], [%3], %4;"
               ::"l"(map), "r"(x), "r"(y), "r"(src), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* map, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {  // <= N groups still reading shared memory
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_done() {  // <= N groups not yet complete
  asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void fence_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load of a CTA pair: the bytes are counted on the barrier at `bar_cluster_addr`, which may
// live in the peer CTA (no multicast: each CTA fetches its own box).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair_hint(uint32_t dst, const CUtensorMap* map, int x, int y,
                                                      uint32_t bar_cluster_addr, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      ".L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_cluster_addr), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair_hint(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                                      uint32_t bar_cluster_addr, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      ".L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar_cluster_addr), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem),
               "r"(cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols)
               : "memory");
}
// commit of a CTA pair's MMAs, arriving on the barrier at the same offset in both CTAs
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((unsigned short)3)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                               uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem),
               "r"(cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
// D[tmem] (+)= A[smem] . B[smem]^T, bf16 operands, fp32 accumulate; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives lane (base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
        "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned ld_relaxed_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_cta_add(int* p, int v) {
  asm volatile("red.release.cta.shared::cta.add.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_cta(const int* p) {
  int v;
  asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
  return v;
}
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
__device__ __forceinline__ void st_relaxed_gpu(unsigned* p, unsigned v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// system scope: flags that another GPU writes or reads (pull mode)
__device__ __forceinline__ unsigned ld_relaxed_sys(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_acquire_sys(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_acq_rel_sys() { asm volatile("fence.acq_rel.sys;" ::: "memory"); }
__device__ __forceinline__ void st_relaxed_sys(unsigned* p, unsigned v) {
  asm volatile("st.relaxed.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
template <bool SYS>
__device__ __forceinline__ unsigned ld_relaxed_flag(const unsigned* p) {
  return SYS ? ld_relaxed_sys(p) : ld_relaxed_gpu(p);
}
template <bool SYS>
__device__ __forceinline__ unsigned ld_acquire_flag(const unsigned* p) {
  return SYS ? ld_acquire_sys(p) : ld_acquire_gpu(p);
}
template <bool SYS>
__device__ __forceinline__ void fence_acq_rel_flag() {
  if (SYS) fence_acq_rel_sys();
  else fence_acq_rel_gpu();
}

__device__ __forceinline__ void st_release_gpu(unsigned* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, const uint4& v) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64
// elements) written by TMA with 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= uint64_t((saddr & 0x3FFFF) >> 4);  // start address, 16-byte units
  d |= uint64_t(1) << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= uint64_t(1024 >> 4) << 32;         // stride byte offset between 8-row groups
  d |= uint64_t(1) << 46;                 // descriptor version of this architecture
  d |= uint64_t(2) << 61;                 // 128-byte swizzle
  return d;
}
// The same for an operand stored with its M/N index contiguous ("MN-major": B given as [K, N]):
// TMA boxes of 64 N-elements (128 bytes, swizzled) x k-rows; 8 k-rows form a 1024-byte swizzle atom,
// consecutive atoms along K follow each other (stride byte offset 1024), and the next group of 64
// N-elements lies `group_bytes` further (leading byte offset).
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t saddr, uint32_t group_bytes) {
  uint64_t d = 0;
  d |= uint64_t((saddr & 0x3FFFF) >> 4);
  d |= uint64_t((group_bytes >> 4) & 0x3FFF) << 16;  // leading byte offset: between 64-element groups of N
  d |= uint64_t(1024 >> 4) << 32;                    // stride byte offset: between 8-row atoms along K
  d |= uint64_t(1) << 46;
  d |= uint64_t(2) << 61;
  return d;
}
// Instruction descriptor: fp32 accumulator, bf16 x bf16, both operands K-major, M = 128.
// (bit 16 set: B is MN-major)
template <int BN, int MM>
__device__ __forceinline__ constexpr uint32_t instr_desc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(BN >> 3) << 17) | (uint32_t(MM >> 4) << 24);
}

// Producer block handled by CTA `rank` of the pair that works on pair index u.  Both blocks of
// a pair share the block column (the B panel).  Interleaved order (W even): positions 2u and
// 2u+1 of Eq. 1, i.e. two destinations at once.  Row-major order (even tile rows per
// partition): vertically adjacent blocks of one partition.
// Destination partition d and block index l inside the partition of position p of the tile
// order (Eq. 1 for the interleaved order).
__device__ __forceinline__ void position_to_block(const KParams& P, int p, int* d, int* l) {
  if (P.order == ENTWINE_ORDER_INTERLEAVED) {
    *d = p % P.W;
    *l = p / P.W;
  } else if (P.order == ENTWINE_ORDER_M_MAJOR) {
    const int rows_all = P.W * P.rowsT;
    const int row_all = p % rows_all, col_all = p / rows_all;
    *d = row_all / P.rowsT;
    *l = (row_all - *d * P.rowsT) * P.nBn + col_all;
  } else {
    *d = p / P.Lb;
    *l = p - *d * P.Lb;
  }
}
__device__ __forceinline__ int pair_position(const KParams& P, int u, int rank) {
  // interleaved and M-major: consecutive positions share a block column
  if (P.order != ENTWINE_ORDER_ROW_MAJOR) return 2 * u + rank;
  const int half = P.Lb / 2;
  const int d = u / half, rem = u - d * half;
  const int v = rem / P.nBn, nb = rem - v * P.nBn;
  return d * P.Lb + (2 * v + rank) * P.nBn + nb;
}

// ------------------------------------------------------------------------------------------
// status helpers
// ------------------------------------------------------------------------------------------
struct SlotMeta {
  int kind;      // 0 reduce step, 1 push step, 2 normalisation of a tile, 3 residual rows of the tile whose
                 // reduce steps follow, 4 / 5 whole reduce / push task done from registers (dst_y: first
                 // destination row, aux: first row in the [M,N] buffers), -1 end of work, -2 continue on ring B
  int dst_x;     // column of the destination box
  int dst_y;     // row of the destination box in the destination buffer
  int aux;       // layer chain: band (tile row) whose count the last step of a reduce task raises, else -1
};
struct CtaShared {
  volatile int abort;      // a role of this CTA (or another CTA) gave up
  volatile int gemm_done;  // this CTA's producer work is over; its shared memory is free
  volatile int stages_free;  // the CTA's last MMA has completed: its operand stages are free
  int ring_b_bytes;          // size of this CTA's ring B: the operand stages of a producer CTA (ring B
                             // then starts before the epilogue is over), 192 KiB of a consumer CTA
  int warps_stored;        // epilogue warps x blocks of this CTA whose partial-C stores have been issued
  float inv_rms[kTile];    // layer chain: 1 / RMS of the rows of the tile being normalised
  SlotMeta meta[2][kMaxSlots];
};

__device__ __forceinline__ void report(const KParams& P, int code, long long where) {
  StatusSlot* s = &P.status[P.seq & 1];
  unsigned long long v = (unsigned long long)(code & 0xff) | ((unsigned long long)blockIdx.x << 8) |
                         ((unsigned long long)(where & 0xffffffffLL) << 32);
  atomicCAS(&s->code_cta_task, 0ULL, v);
}
__device__ __forceinline__ bool global_abort(const KParams& P) {
  return *reinterpret_cast<volatile unsigned long long*>(&P.status[P.seq & 1].code_cta_task) != 0;
}

// Bounded mbarrier wait: false if the budget ran out or the CTA was told to abort.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const KParams& P,
                                          CtaShared* sh) {
  if (mbar_try_wait(bar, parity)) return true;
  unsigned long long t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spins % kSpinCheck) == 0) {
      if (sh->abort) return mbar_try_wait(bar, parity) != 0;
      unsigned long long now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > P.wait_budget_ns) return mbar_try_wait(bar, parity) != 0;
    }
  }
}

// Bounded acquire-poll of one flag (Sec. 4.2: acquire loads until the flag is published).
template <bool SYS = false>
__device__ __forceinline__ bool wait_flag(const unsigned* f, const KParams& P) {
  if (ld_acquire_flag<SYS>(f) >= P.epoch) return true;
  unsigned long long t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (ld_acquire_flag<SYS>(f) >= P.epoch) return true;
    if ((spins % 32) == 0) {
      if (global_abort(P)) return false;
      unsigned long long now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > P.wait_budget_ns) return false;
    }
    __nanosleep(64);  // longer, growing pauses (up to 4 us) were measured: no effect on the producer
  }
}

// Bounded acquire-poll of a counter until it reaches `target`.
__device__ __forceinline__ bool wait_count(const unsigned* f, unsigned target, const KParams& P) {
  unsigned long long t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (ld_acquire_gpu(f) >= target) return true;
    if ((spins % 32) == 0) {
      if (global_abort(P)) return false;
      unsigned long long now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > P.wait_budget_ns) return false;
    }
    __nanosleep(128);
  }
}

// ------------------------------------------------------------------------------------------
// consumer: flag polling, scatter push and ReduceTile (Sec. 4.2) as a TMA ring pipeline
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void acc_bf16x8(float (&a)[8], const uint4& v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    a[2 * i] += __uint_as_float(w[i] << 16);
    a[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint4 pack_bf16x8(const float (&a)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a[2 * i], a[2 * i + 1]);  // round to nearest even
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

struct CommCounters {
  unsigned reduced = 0, pushed = 0;
};

// A ring of shared-memory slots with its three barriers per slot.
struct Ring {
  uint32_t base;   // shared address of slot 0
  uint32_t bars;   // shared address of full[kMaxSlots], empty[kMaxSlots], reduced[kMaxSlots]
  int n_slots;
  int id;          // 0 = ring A, 1 = ring B
  int geom;        // index of the step geometry and of the tensor-map set
  int rs, prs, slot_bytes;
  int sub_bytes;   // one contribution's rows of one reduce step
  __device__ __forceinline__ uint32_t full(int s) const { return bars + 8u * s; }
  __device__ __forceinline__ uint32_t empty(int s) const { return bars + 8u * (kMaxSlots + s); }
  __device__ __forceinline__ uint32_t red(int s) const { return bars + 8u * (2 * kMaxSlots + s); }
};
template <bool REG>
__device__ __forceinline__ Ring make_ring(uint32_t smem_base, int id, const KParams& P, const CtaShared* sh) {
  Ring r;
  r.id = id;
  r.geom = id == 0 ? P.ring_a_geom : 1;
  r.base = smem_base + (id == 0 ? P.ring_a_off : kRingBOff);
  r.bars = smem_base + kBarOff + (id == 0 ? kBarRingA : kBarRingB);
  r.rs = P.rs[r.geom];
  r.prs = P.prs[r.geom];
  r.slot_bytes = P.slot_bytes[r.geom];
  r.sub_bytes = r.rs * kTile * 2;
  r.n_slots = min(kMaxSlots, (id == 0 ? P.ring_a_bytes : sh->ring_b_bytes) / r.slot_bytes);
  if (REG && id == 0) r.n_slots = kRegSlots;  // descriptors only
  return r;
}

// ------------------------------------------------------------------------------------------
// Whole-tile tasks from registers (the consumer warps of a CTA that still produces).  256 threads
// share a 128 x 128 tile: thread ctid takes the 16-byte chunks ctid, ctid + 256, ... (row c / 16,
// column chunk c % 16), so a warp's load covers two 256-byte row segments.  Up to 16 loads of 16
// bytes are in flight per thread.  The partial C was written through the async proxy by other
// SMs and is read at L2 (never from this SM's L1); the flags were acquired by the claiming warp,
// whose barrier arrival orders these loads after them.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_l2_v4(const __nv_bfloat16* p) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ld_stream_v4(const __nv_bfloat16* p) {
  uint4 v;
  asm volatile("ld.global.cs.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
// contribution of peer slot q (ascending rank order with the own rank left out), as [M][N]
template <bool PULL>
__device__ __forceinline__ const __nv_bfloat16* peer_base(const KParams& P, int q) {
  if (PULL) {
    const int w = q + (q >= P.r ? 1 : 0);
    return reinterpret_cast<const __nv_bfloat16*>(P.heap + (long long)w * P.heap_stride + P.heap_buf_off);
  }
  // (rows are numbered as in [M,N]: the offset of the plane's first row is taken out here)
  return P.peers + ((long long)q * P.peer_rows - P.peer_row0) * P.N;
}
// ReduceTile of Sec. 4.2 on a whole tile: local contribution first, then the peers in ascending rank
// order, fp32, one rounding.  A thread's 8 chunks go in batches of 16 / W chunks: all loads of a
// batch are issued before the first is used.  (A rolling window over the flat sequence of loads was
// measured too: no faster here, and it spills in the layer-chain kernels.)
template <int WW, bool PULL>
__device__ __forceinline__ void reg_reduce_tile(const KParams& P, int ctid, int col, int src_row, int dst_row) {
  constexpr int kChunks = kTile * (kTile * 2 / 16) / kRedThreads;  // 8 per thread
  constexpr int NB = (16 / WW) < 1 ? 1 : ((16 / WW) > kChunks ? kChunks : (16 / WW));
  const long long N = P.N;
#pragma unroll 1
  for (int i0 = 0; i0 < kChunks; i0 += NB) {
    uint4 v[NB][WW];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const int c = ctid + (i0 + b) * kRedThreads;
      const long long off = (long long)(src_row + (c >> 4)) * N + col + (c & 15) * 8;
      v[b][0] = ld_l2_v4(P.cws + off);
#pragma unroll
      for (int q = 1; q < WW; ++q) v[b][q] = ld_stream_v4(peer_base<PULL>(P, q - 1) + off);
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const int c = ctid + (i0 + b) * kRedThreads;
      float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int q = 0; q < WW; ++q) acc_bf16x8(a, v[b][q]);
      __stcs(reinterpret_cast<uint4*>(P.out + (long long)(dst_row + (c >> 4)) * N + col + (c & 15) * 8), pack_bf16x8(a));
    }
  }
}
// any W: chunk by chunk, the peers' loads of a chunk in flight four at a time
template <bool PULL>
__device__ __forceinline__ void reg_reduce_tile_any(const KParams& P, int ctid, int col, int src_row, int dst_row) {
  constexpr int kChunks = kTile * (kTile * 2 / 16) / kRedThreads;
  const long long N = P.N;
#pragma unroll 1
  for (int i = 0; i < kChunks; ++i) {
    const int c = ctid + i * kRedThreads;
    const long long off = (long long)(src_row + (c >> 4)) * N + col + (c & 15) * 8;
    float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    acc_bf16x8(a, ld_l2_v4(P.cws + off));
#pragma unroll 1
    for (int q0 = 0; q0 < P.W - 1; q0 += 4) {
      uint4 v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        v[j] = (q0 + j < P.W - 1) ? ld_stream_v4(peer_base<PULL>(P, q0 + j) + off) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (q0 + j < P.W - 1) acc_bf16x8(a, v[j]);
    }
    __stcs(reinterpret_cast<uint4*>(P.out + (long long)(dst_row + (c >> 4)) * N + col + (c & 15) * 8), pack_bf16x8(a));
  }
}
// Layer chain (Sec. 5.2.3) from registers: the rank-order fp32 sum, then the residual, one rounding;
// the bf16 result is the new residual stream (P.out), and the sum of squares of the 128 stored
// values of each row inside this tile goes to ssq_part (one writer each).  Same arithmetic, in the
// same order, as the ring path: the sixteen threads of a row add their partial sums by the same
// shuffles.  WW = 0: any W.
template <int WW>
__device__ __forceinline__ void reg_reduce_tile_norm(const KParams& P, int ctid, int lane, int col, int src_row,
                                                     int dst_row) {
  constexpr int kChunks = kTile * (kTile * 2 / 16) / kRedThreads;
  const long long N = P.N;
#pragma unroll 1
  for (int i = 0; i < kChunks; ++i) {
    const int c = ctid + i * kRedThreads;
    const long long off = (long long)(src_row + (c >> 4)) * N + col + (c & 15) * 8;
    const long long doff = (long long)(dst_row + (c >> 4)) * N + col + (c & 15) * 8;
    float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (WW > 0) {
      uint4 v[WW > 0 ? WW : 1];
      v[0] = ld_l2_v4(P.cws + off);
#pragma unroll
      for (int q = 1; q < WW; ++q) v[q] = ld_stream_v4(peer_base<false>(P, q - 1) + off);
      const uint4 rv = ld_stream_v4(P.residual + doff);
#pragma unroll
      for (int q = 0; q < WW; ++q) acc_bf16x8(a, v[q]);
      acc_bf16x8(a, rv);
    } else {
      acc_bf16x8(a, ld_l2_v4(P.cws + off));
      for (int q = 1; q < P.W; ++q) acc_bf16x8(a, ld_stream_v4(peer_base<false>(P, q - 1) + off));
      acc_bf16x8(a, ld_stream_v4(P.residual + doff));
    }
    const uint4 o = pack_bf16x8(a);
    __stcg(reinterpret_cast<uint4*>(P.out + doff), o);  // re-read from L2 by the normalisation
    float h[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    acc_bf16x8(h, o);
    float ssq = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) ssq = fmaf(h[e], h[e], ssq);
#pragma unroll
    for (int sft = 8; sft > 0; sft >>= 1) ssq += __shfl_xor_sync(0xffffffffu, ssq, sft);
    if ((lane & 15) == 0) __stcg(&P.ssq_part[(long long)(dst_row + (c >> 4)) * P.nTn + col / kTile], ssq);
  }
}
__device__ __forceinline__ void reg_push_tile(const KParams& P, int ctid, int col, int src_row, int dst_row) {
  constexpr int kChunks = kTile * (kTile * 2 / 16) / kRedThreads;
  const long long N = P.N;
  uint4 v[kChunks];
#pragma unroll
  for (int i = 0; i < kChunks; ++i) {
    const int c = ctid + i * kRedThreads;
    v[i] = ld_l2_v4(P.cws + (long long)(src_row + (c >> 4)) * N + col + (c & 15) * 8);
  }
#pragma unroll
  for (int i = 0; i < kChunks; ++i) {
    const int c = ctid + i * kRedThreads;
    __stcs(reinterpret_cast<uint4*>(P.send + (long long)(dst_row + (c >> 4)) * N + col + (c & 15) * 8), v[i]);
  }
}

// The reducing warps' loop (Sec. 4.2, ReduceTile).  NORM selects the layer-chain variant, which
// carries the tile's residual in registers and handles the residual and normalisation steps; the
// plain variant is compiled without any of that state.
template <bool NORM, bool PULL, bool REG>
__device__ __forceinline__ void reducer_role(const KParams& P, CtaShared* sh, uint32_t smem_base, Ring ring) {
  const int lane = threadIdx.x & 31;
  const int ctid = threadIdx.x - kRedWarp0 * 32;
  PROF_DECL();
  int slot = -1;
  uint32_t ph = 0;
  // layer chain: this thread's 8 chunks (16 bytes each) of the residual of the tile being
  // reduced: chunks ctid, ctid + 256, ... of the tile's 128 rows x 16 chunks
  constexpr int kResChunks = kTile * (kTile * 2 / 16) / kRedThreads;
  uint4 resv[kResChunks];
#pragma unroll
  for (int k = 0; k < kResChunks; ++k) resv[k] = make_uint4(0u, 0u, 0u, 0u);
  for (;;) {
    if (++slot == ring.n_slots) { slot = 0; ph ^= 1; }
    // one lane per warp polls; the warp-level vote carries the barrier's acquire to all lanes
    bool landed = true;
    if (lane == 0) {
      PROF_T0();
      landed = mbar_wait(ring.full(slot), ph, P, sh);
      if (ctid == 0) PROF_ADD(12);
    }
    if (!__all_sync(0xffffffffu, landed)) {
      sh->abort = 1;
      break;
    }
    const SlotMeta m = sh->meta[ring.id][slot];
    if (m.kind == -1) break;
    if (m.kind == -2) {
      ring = make_ring<REG>(smem_base, 1, P, sh);
      slot = -1;
      ph = 0;
      continue;
    }
    if (REG && !NORM && m.kind == 4) {
      // a whole reduce task from registers (ReduceTile of Sec. 4.2 on all 128 rows of the tile)
      PROF_T0();
      if (P.W == 2) reg_reduce_tile<2, PULL>(P, ctid, m.dst_x, m.aux, m.dst_y);
      else if (P.W == 4) reg_reduce_tile<4, PULL>(P, ctid, m.dst_x, m.aux, m.dst_y);
      else if (P.W == 8) reg_reduce_tile<8, PULL>(P, ctid, m.dst_x, m.aux, m.dst_y);
      else reg_reduce_tile_any<PULL>(P, ctid, m.dst_x, m.aux, m.dst_y);
      if (ctid == 0) PROF_ADD(10);
    } else if (REG && !PULL && m.kind == 5) {
      PROF_T0();
      reg_push_tile(P, ctid, m.dst_x, m.aux, m.dst_y);
      if (ctid == 0) PROF_ADD(11);
    } else if (REG && NORM && !PULL && m.kind == 4) {
      if (P.W == 2) reg_reduce_tile_norm<2>(P, ctid, lane, m.dst_x, m.aux, m.dst_y);
      else if (P.W == 4) reg_reduce_tile_norm<4>(P, ctid, lane, m.dst_x, m.aux, m.dst_y);
      else if (P.W == 8) reg_reduce_tile_norm<8>(P, ctid, lane, m.dst_x, m.aux, m.dst_y);
      else reg_reduce_tile_norm<0>(P, ctid, lane, m.dst_x, m.aux, m.dst_y);
    } else if (!NORM && m.kind == 0) {
      const uint32_t sbase = ring.base + slot * ring.slot_bytes;
      const int rs = ring.rs, sub_bytes = ring.sub_bytes;
      __nv_bfloat16* dst = P.out + (long long)m.dst_y * P.N + m.dst_x;
      // start from the local contribution, add the peers in ascending rank order, fp32; every
      // thread writes its own 16 bytes of the output (single writer, 256-byte row segments)
      for (int c = ctid; c < rs * (kTile * 2 / 16); c += kRedThreads) {
        float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        const uint32_t addr = sbase + c * 16;
        acc_bf16x8(a, ld_shared_v4(addr));
#pragma unroll 4
        for (int q = 1; q < P.W; ++q) acc_bf16x8(a, ld_shared_v4(addr + q * sub_bytes));
        __stcs(reinterpret_cast<uint4*>(dst + (long long)(c >> 4) * P.N + (c & 15) * 8), pack_bf16x8(a));
      }
    } else if (NORM && m.kind == 0) {
      // Layer chain (Sec. 5.2.3): the same rank-order fp32 sum, plus the residual; the bf16
      // result is the new residual stream (written to P.out), and the sum of squares of the
      // 128 stored values of each row inside this tile goes to ssq_part (one writer each).
      const uint32_t sbase = ring.base + slot * ring.slot_bytes;
      const int rs = ring.rs, sub_bytes = ring.sub_bytes;
      const int n_chunks = rs * (kTile * 2 / 16);
      for (int c0 = 0; c0 < n_chunks; c0 += kRedThreads) {
        const int c = c0 + ctid;
        const bool act = c < n_chunks;
        float ssq = 0.f;
        if (act) {
          const long long off = (long long)(m.dst_y + (c >> 4)) * P.N + m.dst_x + (c & 15) * 8;
          float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
          const uint32_t addr = sbase + c * 16;
          acc_bf16x8(a, ld_shared_v4(addr));
#pragma unroll 4
          for (int q = 1; q < P.W; ++q) acc_bf16x8(a, ld_shared_v4(addr + q * sub_bytes));
          // the residual, last: chunk (row of the tile) * 16 + (c & 15) of the tile, kept by this
          // thread (or, for steps of fewer than 16 rows, read from global memory)
          const int g = ((m.dst_y & (kTile - 1)) * (kTile * 2 / 16) + c) / kRedThreads;
          uint4 rv = make_uint4(0u, 0u, 0u, 0u);
          if (rs * (kTile * 2 / 16) >= kRedThreads) {
#pragma unroll
            for (int k = 0; k < kResChunks; ++k)
              if (k == g) rv = resv[k];
          } else {
            rv = __ldcs(reinterpret_cast<const uint4*>(P.residual + off));
          }
          acc_bf16x8(a, rv);
          const uint4 o = pack_bf16x8(a);
          __stcg(reinterpret_cast<uint4*>(P.out + off), o);  // re-read from L2 by the normalisation
          float h[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
          acc_bf16x8(h, o);
#pragma unroll
          for (int e = 0; e < 8; ++e) ssq = fmaf(h[e], h[e], ssq);
        }
        // the 16 threads of a row segment (half a warp) add up in a fixed order
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) ssq += __shfl_xor_sync(0xffffffffu, ssq, o);
        if (act && (lane & 15) == 0)
          __stcg(&P.ssq_part[(long long)(m.dst_y + (c >> 4)) * P.nTn + m.dst_x / kTile], ssq);
      }
    } else if (NORM && m.kind == 3) {
      // residual rows [dst_y, dst_y + prs) of the tile: every thread takes its chunks
      const uint32_t sbase = ring.base + slot * ring.slot_bytes;
      const int g0 = m.dst_y * (kTile * 2 / 16), g1 = g0 + ring.prs * (kTile * 2 / 16);
#pragma unroll
      for (int k = 0; k < kResChunks; ++k) {
        const int g = ctid + k * kRedThreads;
        if (g >= g0 && g < g1) resv[k] = ld_shared_v4(sbase + (g - g0) * 16);
      }
    } else if (NORM && (m.kind == 2 || m.kind == 6)) {
      // Normalisation of prs rows of one 128 x 128 tile of a complete band; the rows are in the
      // slot (loaded from hidden_out by TMA).  m.aux >= 0: the first step of a run of tiles of
      // band m.aux: 1/RMS of the band's 128 rows from the nTn partial sums of each row, kept in
      // shared memory for the following steps of the run.  Two threads per row, each adds its
      // half of the row's partial sums (all loads in flight together where the halves are
      // 16-byte aligned), one shuffle joins the halves; the order of the additions is fixed.
      if (m.aux >= 0) {
        named_bar_sync(2, kRedThreads);  // every thread is done with the previous run's values
        const int row = ctid >> 1, half = ctid & 1;
        const int n_half = (P.nTn + 1) / 2;
        const int first = half * n_half;
        const int cnt = min(n_half, P.nTn - first);
        const float* pr = P.ssq_part + (long long)(m.aux * kTile + row) * P.nTn + first;
        float sum = 0.f;
        if ((P.nTn & 7) == 0) {
          for (int q0 = 0; q0 < cnt; q0 += 32) {
            float4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
              v[j] = (q0 + 4 * j < cnt) ? __ldcg(reinterpret_cast<const float4*>(pr + q0 + 4 * j))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < 8; ++j) sum += (v[j].x + v[j].y) + (v[j].z + v[j].w);
          }
        } else {
          for (int q = 0; q < cnt; ++q) sum += __ldcg(pr + q);
        }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        if (half == 0) sh->inv_rms[row] = rsqrtf(sum / (float)P.N + P.eps);
        named_bar_sync(2, kRedThreads);
      }
      const uint32_t sbase = ring.base + slot * ring.slot_bytes;
      float w[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      acc_bf16x8(w, __ldg(reinterpret_cast<const uint4*>(P.weight + m.dst_x + (ctid & 15) * 8)));
      if (m.kind == 6) {
        // the whole 128 x 128 tile from L2 (hidden_out was stored there by the reduce tasks; the claiming
        // warp acquired the band's count before it handed this record over): this thread's eight
        // chunks, rows ctid / 16 + 16 k, all loads in flight before the first is used
        const __nv_bfloat16* src = P.out + (long long)m.dst_y * P.N + m.dst_x + (ctid & 15) * 8;
        __nv_bfloat16* dst = P.norm_out + (long long)m.dst_y * P.N + m.dst_x + (ctid & 15) * 8;
        // (the registers that hold a tile's residual during its reduce steps are free here: every reduce
        // task reloads them before it uses them)
        uint4 (&v)[kResChunks] = resv;
#pragma unroll
        for (int k = 0; k < kResChunks; ++k) v[k] = ld_l2_v4(src + (long long)((ctid >> 4) + k * (kRedThreads / 16)) * P.N);
#pragma unroll
        for (int k = 0; k < kResChunks; ++k) {
          const int row = (ctid >> 4) + k * (kRedThreads / 16);
          float h[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
          acc_bf16x8(h, v[k]);
          const float inv = sh->inv_rms[row];
#pragma unroll
          for (int e = 0; e < 8; ++e) h[e] = h[e] * inv * w[e];
          __stcs(reinterpret_cast<uint4*>(dst + (long long)row * P.N), pack_bf16x8(h));
        }
      }
      const int n_chunks = m.kind == 6 ? 0 : ring.prs * (kTile * 2 / 16);
      for (int c = ctid; c < n_chunks; c += kRedThreads) {
        const int row = m.dst_y + (c >> 4);  // row of hidden_out; its band row is row % 128
        float h[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        acc_bf16x8(h, ld_shared_v4(sbase + c * 16));
        const float inv = sh->inv_rms[row & (kTile - 1)];
#pragma unroll
        for (int e = 0; e < 8; ++e) h[e] = h[e] * inv * w[e];
        __stcs(reinterpret_cast<uint4*>(P.norm_out + (long long)row * P.N + m.dst_x + (c & 15) * 8), pack_bf16x8(h));
      }
    }
    // one arrival per warp returns the slot (a push step is forwarded by the store warp alone;
    // the arrival then only says that this warp has read the slot's header)
    __syncwarp();
    if (lane == 0) mbar_arrive(ring.red(slot));
  }
  PROF_FLUSH(ctid == 0);
}

// One CTA's consumer work, run by warps 2, 3 and 8-15.  Warp 2 claims tasks from `n_lists`
// consumer lists starting at `first_list` (each list is consumed in order through its head
// counter, Sec. 3.1), polls the tile flags with one lane per contributing rank, and streams
// the tiles through a ring of shared-memory slots with TMA; warps 8-15 reduce a slot in fp32
// and write the result; warp 3 forwards pushed tiles with TMA stores and recycles the slots.
// In a producer CTA the pipeline starts on the small ring A beside the producer's buffers and
// moves to ring B (the producer's buffers) once `gemm_done` is set.
template <bool NORM, bool PULL, bool REG>
__device__ __forceinline__ void consumer_pipeline(const KParams& P, const KMaps& maps, CtaShared* sh, uint32_t smem_base,
                                  int first_list, int n_lists, bool start_on_a, CommCounters* cnt) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (REG && !NORM && P.reg_only) start_on_a = true;
  Ring ring = make_ring<REG>(smem_base, start_on_a ? 0 : 1, P, sh);

  if (warp == kCommWarp) {
    // ---------------- claim, poll, load ----------------
    PROF_DECL();
    // tiles are read once: ask L2 to evict them first so that the producer's operand panels stay
    const uint64_t pol = (P.l2_hints & 1) ? l2_policy_evict_first() : l2_policy_evict_normal();
    int it = 0;
    bool ok = true;
    const long long MN = (long long)P.M * P.N, RN = P.R * (long long)P.N;
    // moves the pipeline to ring B once the producer's buffers are free
    auto maybe_switch = [&]() {
      if (ring.id != 0 || (REG && !NORM && P.reg_only)) return;
      int done = 0;
      if (lane == 0) done = P.early_b ? sh->stages_free : sh->gemm_done;
      done = __shfl_sync(0xffffffffu, done, 0);
      if (!done) return;
      bool free_slot = true;
      if (lane == 0) {
        // With early_b, ring B lies in the operand stages only, which neither ring A nor the
        // epilogue's staging overlaps: steps still in flight in ring A are not disturbed.
        // Otherwise ring B's last slots overlap ring A's memory, and every ring-A step in flight
        // must have returned its slot first: slot s has been used uses(s) times; its last use,
        // number uses(s) - 1, is over when its empty barrier completes the phase of that parity.
        // (In register mode ring A holds no data at all.)
        for (int sl = 0; !P.early_b && !REG && free_slot && sl < ring.n_slots; ++sl) {
          const int uses = (it - sl + ring.n_slots - 1) / ring.n_slots;
          if (uses > 0) free_slot = mbar_wait(ring.empty(sl), (uses - 1) & 1, P, sh);
        }
        // the marker travels through the next ring-A slot, which must be free
        const int slot = it % ring.n_slots;
        if (free_slot) free_slot = mbar_wait(ring.empty(slot), ((it / ring.n_slots) & 1) ^ 1, P, sh);
        if (free_slot) {
          sh->meta[0][slot].kind = -2;
          mbar_arrive(ring.full(slot));
        }
      }
      ok = __all_sync(0xffffffffu, free_slot);
      ring = make_ring<REG>(smem_base, 1, P, sh);
      it = 0;
    };
    // Layer chain: normalisation tasks (one per tile of the rank's partition, band by band) are
    // handed out through one counter in runs of kRun tiles; a run's steps bring the rows of
    // hidden_out into ring slots, and the band's 1/RMS values are computed once per run.
    constexpr int kRun = 4;
    int* const norm_head = &P.list_head[P.x];
    // issues the steps of the run of n tiles that starts at tile i (lane 0 does the work)
    auto issue_norm_run = [&](int i, int n) {
      bool run_ok = true;
      if (lane == 0) {
        int band_seen = -1;
        for (int t = i; run_ok && t < min(i + n, P.Q); ++t) {
          const int band = t / P.nTn, tc = t - band * P.nTn;
          if (band != band_seen) {
            // (the run may reach into the next band, which may not be complete yet)
            run_ok = wait_count(&P.band_ctr[band], (unsigned)P.nTn, P);
            if (!run_ok) break;
            fence_async_all();  // the TMA reads of hidden_out are ordered after the acquire
          }
          if (kNormLoads) {
            // one record per tile: the reducing warps fetch its rows themselves
            const int slot = it % ring.n_slots;
            run_ok = mbar_wait(ring.empty(slot), ((it / ring.n_slots) & 1) ^ 1, P, sh);
            if (!run_ok) break;
            SlotMeta& m = sh->meta[ring.id][slot];
            m.kind = 6;
            m.dst_x = tc * kTile;
            m.dst_y = band * kTile;
            m.aux = (band != band_seen) ? band : -1;
            band_seen = band;
            mbar_arrive(ring.full(slot));
            it += 1;
            continue;
          }
          for (int u = 0; run_ok && u < kTile / ring.prs; ++u) {
            const int slot = it % ring.n_slots;
            run_ok = mbar_wait(ring.empty(slot), ((it / ring.n_slots) & 1) ^ 1, P, sh);
            if (!run_ok) break;
            SlotMeta& m = sh->meta[ring.id][slot];
            m.kind = 2;
            m.dst_x = tc * kTile;
            m.dst_y = band * kTile + u * ring.prs;
            m.aux = (band != band_seen) ? band : -1;
            band_seen = band;
            mbar_arrive_expect_tx(ring.full(slot), ring.prs * kTile * 2);
            tma_load_2d_hint(ring.base + slot * ring.slot_bytes, &maps.h_ld[ring.geom], tc * kTile,
                             band * kTile + u * ring.prs, ring.full(slot), pol);
            it += 1;
          }
        }
        if (!run_ok) report(P, -ENTWINE_ERR_TIMEOUT, -7);
      }
      ok = __all_sync(0xffffffffu, run_ok);
      it = __shfl_sync(0xffffffffu, it, 0);
    };
    // Drains list j.  Claims go through the list's head counter in runs of up to P.claim
    // consecutive tasks, so the list is consumed in order whoever executes it (Sec. 3.1).  This
    // warp is the one serial stage of the pipeline and a push task is a single ring step, so the
    // per-task path is kept short:
    //   * nothing a task needs from global memory is waited for on that path: three claims are
    //     kept going (`cur` is executed, `nxt` has its flags in flight, `fut` its atomic), a
    //     window of 32 task records is loaded ahead of the first claim's return, and the flags
    //     of claim `nxt` are read early with relaxed loads (up to 64 flags, two per lane); when
    //     `nxt` becomes `cur`, flags seen as published are made an acquire by one fence for the
    //     whole claim, the others fall back to the acquire poll of Sec. 4.2;
    //   * the 32 lanes turn the 32 records of a window into load coordinates in parallel
    //     (checks, divisions), and one lane then runs a task's ring steps without warp votes.
    auto drain = [&](int j) {
      const int base = P.list_offs[j];
      const int len = P.list_offs[j + 1] - base;
      if (len <= 0) return;
      const int CH = P.claim;  // CH * W <= 64 (W <= 64): the flags of a claim fit the early look
      // Where several CTAs share a list, claims shrink towards its end (guided self-scheduling)
      // so that they finish together: a quarter of an even share of what is left, at most CH
      // tasks.  A list with one CTA of its own is claimed CH tasks at a time to the end: the
      // fence that turns a claim's early flag reads into an acquire waits for the claim atomic in
      // flight, and is paid once per claim.
      const int sharers = ((int)gridDim.x + P.x - 1) / P.x;
      auto claim_len = [&](int head) {
        // (longer claims on shared lists measured slower: the tiles in flight at one time then
        // lie further apart in memory)
        return sharers > 1 ? max(1, min(min(CH, 2), (len - head) / (4 * sharers))) : max(1, min(CH, len - head));
      };
      int cur = len, nxt = len, fut = len;
      int cur_n = claim_len(0), nxt_n = cur_n, fut_n = cur_n;
      if (lane == 0) {
        cur = atomicAdd(&P.list_head[j], cur_n);
        nxt = atomicAdd(&P.list_head[j], nxt_n);
        fut = atomicAdd(&P.list_head[j], fut_n);
      }
      // this lane's record of the window, as coordinates: kind (-3 = record out of range), tile
      // column, row of the tile in an [M,N] buffer, first destination row, flag indices
      int win = 0;
      int k_kind, k_col, k_row, k_dst, k_own, k_t;
      auto load_window = [&](int first) {
        win = first;
        const Task rec = P.tasks[base + min(first + lane, len - 1)];
        const bool bad = rec.src_off < 0 || rec.src_off + (long long)(kTile - 1) * P.N + kTile > MN ||
                         rec.dst_off < 0 || rec.dst_off + (long long)(kTile - 1) * P.N + kTile > RN ||
                         rec.t < 0 || rec.t >= P.Q || rec.d < 0 || rec.d >= P.W ||
                         (rec.kind == 1 && (rec.slot < 0 || rec.slot >= P.W - 1));
        const int trow = rec.t / P.nTn, tcol = rec.t - trow * P.nTn;
        k_kind = bad ? -3 : rec.kind;
        k_col = tcol * kTile;
        k_row = rec.d * (int)P.R + trow * kTile;
        k_dst = (rec.kind == 0 ? 0 : rec.slot * (int)P.R) + trow * kTile;
        k_own = rec.d * P.Q + rec.t;
        k_t = rec.t;
      };
      load_window(0);
      // row of peer slot q in the peers' flag array: the slot itself, or, in pull mode, the
      // peer's rank in this rank's array of all W sources
      auto peer_row = [&](int q) { return PULL ? q + (q >= P.r ? 1 : 0) : q; };
      unsigned pf[2] = {0u, 0u};
      int pf_start = -1;
      // relaxed look at the flags of the claim starting at s (if its records are in the window)
      auto peek_flags = [&](int s, int n_claim) {
        pf_start = -1;
        if (P.skip_wait || s >= len || s < win || s + n_claim > win + 32) return;
        pf_start = s;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int f = r * 32 + lane;
          const int c = f / P.W, q = f - c * P.W;
          const int src = min(s - win + c, 31);
          const int kind = __shfl_sync(0xffffffffu, k_kind, src);
          const int own = __shfl_sync(0xffffffffu, k_own, src);
          const int t = __shfl_sync(0xffffffffu, k_t, src);
          pf[r] = 0xffffffffu;
          if (c < n_claim && s + c < len && kind >= 0) {
            if (q == 0) pf[r] = ld_relaxed_gpu(&P.flags_own[own]);  // written by this GPU in every mode
            else if (kind == 0) pf[r] = ld_relaxed_flag<PULL>(&P.flags_peer[peer_row(q - 1) * P.Q + t]);
          }
        }
      };
      while (ok) {
        const int s = __shfl_sync(0xffffffffu, cur, 0);
        if (s >= len) break;
        const int n = min(cur_n, len - s);
        // tasks of this claim whose flags were all seen as published by the early look
        unsigned ready = 0;
        if (pf_start == s) {
          unsigned unset = 0;
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            const int c = (r * 32 + lane) / P.W;
            if (pf[r] < P.epoch) unset |= 1u << min(c, 31);
          }
          ready = ~__reduce_or_sync(0xffffffffu, unset) & ((1u << n) - 1u);
          if (ready) {
            fence_acq_rel_flag<PULL>();  // relaxed reads of published flags + this fence = acquire
            fence_async_all();    // and the TMA reads below are ordered after it
          }
        }
        // rotate the claims (after the fence, which waits for the atomics in flight)
        cur = nxt;
        nxt = fut;
        cur_n = nxt_n;
        nxt_n = fut_n;
        fut_n = claim_len(s + n);
        if (lane == 0) fut = atomicAdd(&P.list_head[j], fut_n);
        if (s < win || s + n > win + 32) load_window(s);
        peek_flags(__shfl_sync(0xffffffffu, cur, 0), cur_n);
        for (int c = 0; ok && c < n; ++c) {
          const int i = s + c;
          const int src = i - win;
          const int kind = __shfl_sync(0xffffffffu, k_kind, src);
          const int col = __shfl_sync(0xffffffffu, k_col, src);
          const int src_row = __shfl_sync(0xffffffffu, k_row, src);
          const int dst_row = __shfl_sync(0xffffffffu, k_dst, src);
          if (kind < 0) {
            // index check failed: record and skip instead of touching memory out of range
            if (lane == 0) report(P, -ENTWINE_ERR_INTERNAL, base + i);
            continue;
          }
          if (!PULL && P.prefetch && i + 1 < len && src + 1 < 32) {
            // Look-ahead: if the list's next task is a reduce task whose peer contributions are
            // already published, pull their tiles into L2 now (one lane per peer) so that the
            // ring's loads find them there while holding a slot.  (The task may end up with
            // another CTA; the tiles are in L2 for it all the same.)
            const int nkind = __shfl_sync(0xffffffffu, k_kind, src + 1);
            const int nt = __shfl_sync(0xffffffffu, k_t, src + 1);
            const int nrow = __shfl_sync(0xffffffffu, k_row, src + 1);
            const int ncol = __shfl_sync(0xffffffffu, k_col, src + 1);
            if (nkind == 0) {
              for (int q = lane - 1; q >= 0 && q < P.W - 1; q += 31) {
                if (P.skip_wait || ld_acquire_gpu(&P.flags_peer[q * P.Q + nt]) >= P.epoch)
                  tma_prefetch_l2_2d(&maps.p_pf, ncol, q * P.peer_rows + nrow - P.peer_row0);
              }
            }
          }
          if (!P.skip_wait && !((ready >> c) & 1u)) {
            // lane 0 polls the local flag, lanes 1.. the peers' flags in rank order (Sec. 4.2);
            // the warp proceeds when all W contributions of the tile are published
            const int own = __shfl_sync(0xffffffffu, k_own, src);
            const int t = __shfl_sync(0xffffffffu, k_t, src);
            bool mine_ok = true;
            PROF_T0();
            if (lane == 0) mine_ok = wait_flag<false>(&P.flags_own[own], P);
            else if (kind == 0) {
              for (int q = lane - 1; mine_ok && q < P.W - 1; q += 31)
                mine_ok = wait_flag<PULL>(&P.flags_peer[peer_row(q) * P.Q + t], P);
            }
            ok = __all_sync(0xffffffffu, mine_ok);
            if (lane == 0) PROF_ADD(13);
            if (!ok) {
              if (lane == 0) report(P, -ENTWINE_ERR_TIMEOUT, base + i);
              break;
            }
            fence_async_all();  // the TMA reads below are ordered after the acquires
          }
          maybe_switch();
          if (!ok) break;
          if (REG && ring.id == 0) {
            // register path: the reducing warps load the tile themselves; one descriptor per task
            bool slot_ok = true;
            if (lane == 0) {
              const int slot = it % ring.n_slots;
              {
                PROF_T0();
                slot_ok = mbar_wait(ring.empty(slot), ((it / ring.n_slots) & 1) ^ 1, P, sh);
                PROF_ADD(14);
              }
              if (slot_ok) {
                SlotMeta& m = sh->meta[0][slot];
                m.kind = 4 + kind;
                m.dst_x = col;
                m.dst_y = dst_row;
                m.aux = src_row;
                mbar_arrive(ring.full(slot));
                if (kind == 0) cnt->reduced++;
                else cnt->pushed++;
              } else {
                report(P, -ENTWINE_ERR_TIMEOUT, base + i);
              }
            }
            ok = __all_sync(0xffffffffu, slot_ok);
            it += 1;
            continue;
          }
          const int rows = kind == 0 ? ring.rs : ring.prs;  // rows of the tile per ring step
          const int n_steps = kTile / rows;
          bool steps_ok = true;
          if (lane == 0) {
            // one lane runs the task's steps: wait for the slot, describe it, issue its loads
            int slot = it % ring.n_slots;
            uint32_t ph = (it / ring.n_slots) & 1;
            const uint32_t tx = kind == 0 ? P.W * ring.sub_bytes : ring.prs * kTile * 2;
            if (NORM && kind == 0) {
              // layer chain: the tile's residual rows first (whole push-sized steps); the reducing
              // warps keep them in registers for the reduce steps that follow
              for (int u = 0; u < kTile / ring.prs; ++u) {
                if (!mbar_wait(ring.empty(slot), ph ^ 1, P, sh)) { steps_ok = false; break; }
                SlotMeta& m = sh->meta[ring.id][slot];
                m.kind = 3;
                m.dst_x = col;
                m.dst_y = u * ring.prs;  // first row of these residual rows inside the tile
                m.aux = -1;
                mbar_arrive_expect_tx(ring.full(slot), ring.prs * kTile * 2);
                tma_load_2d_hint(ring.base + slot * ring.slot_bytes, &maps.res_ld[ring.geom], col,
                                 dst_row + u * ring.prs, ring.full(slot), pol);
                if (++slot == ring.n_slots) { slot = 0; ph ^= 1; }
              }
            }
            for (int step = 0; steps_ok && step < n_steps; ++step) {
              if (!mbar_wait(ring.empty(slot), ph ^ 1, P, sh)) { steps_ok = false; break; }
              const uint32_t dst = ring.base + slot * ring.slot_bytes;
              SlotMeta& m = sh->meta[ring.id][slot];
              m.kind = kind;
              m.dst_x = col;
              m.dst_y = dst_row + step * rows;
              m.aux = (NORM && kind == 0 && step == n_steps - 1) ? dst_row / kTile : -1;
              mbar_arrive_expect_tx(ring.full(slot), tx);
              // Few, large TMA operations: the per-operation cost of the TMA unit, not bandwidth,
              // bounds a consumer that issues many small boxes.
              if (kind == 0) {
                // rs rows of the local contribution, then of all peers in ascending rank order
                // as one 3-D box
                tma_load_2d_hint(dst, &maps.c_ld[ring.geom], col, src_row + step * rows, ring.full(slot), pol);
                if (!PULL) {
                  tma_load_3d_hint(dst + ring.sub_bytes, &maps.p_ld[ring.geom], col,
                                   src_row + step * rows - P.peer_row0, 0, ring.full(slot), pol);
                } else {
                  // the peers' rows come straight from their segments of the heap: the ranks
                  // below this one, then the ranks above it, each group as one 3-D box
                  if (P.r > 0)
                    tma_load_3d_hint(dst + ring.sub_bytes, &maps.p_ld[ring.geom], col, src_row + step * rows, 0,
                                     ring.full(slot), pol);
                  if (P.r < P.W - 1)
                    tma_load_3d_hint(dst + (1 + P.r) * ring.sub_bytes, &maps.p_hi[ring.geom], col,
                                     src_row + step * rows, 0, ring.full(slot), pol);
                }

              } else {
                tma_load_2d_hint(dst, &maps.c_push[ring.geom], col, src_row + step * rows, ring.full(slot), pol);
              }
              if (++slot == ring.n_slots) { slot = 0; ph ^= 1; }
            }
            if (steps_ok) {
              if (kind == 0) cnt->reduced++;
              else cnt->pushed++;
            } else {
              report(P, -ENTWINE_ERR_TIMEOUT, base + i);
            }
          }
          ok = __all_sync(0xffffffffu, steps_ok);
          it += n_steps + ((NORM && kind == 0) ? kTile / ring.prs : 0);
        }
      }
    };
    // the CTA's own list first
    if (n_lists > 0) drain(first_list);
    // consumer alone on fewer CTAs than lists: the lists without a CTA of their own are dealt out
    // round-robin before anybody scans for leftovers (CTAs scanning in the same order would all
    // try the same list first)
    if (P.mode == MODE_COMM_ONLY && n_lists > 1) {
      for (int j = first_list + (int)gridDim.x; ok && j < P.x; j += (int)gridDim.x) drain(j);
    }
    // then the other lists: every lane looks at one list per round, lists with work are drained
    while (ok && n_lists > 1) {
      bool any = false;
      for (int j0 = 0; ok && j0 < P.x; j0 += 32) {
        int j = first_list + 1 + j0 + lane;  // walk starts after the own list
        const bool in = j0 + lane < P.x - 1;
        while (j >= P.x) j -= P.x;
        bool work = false;
        if (in) work = *reinterpret_cast<volatile int*>(&P.list_head[j]) < P.list_offs[j + 1] - P.list_offs[j];
        unsigned mask = __ballot_sync(0xffffffffu, work);
        while (ok && mask) {
          const int b = __ffs(mask) - 1;
          mask &= mask - 1;
          int jj = first_list + 1 + j0 + b;
          while (jj >= P.x) jj -= P.x;
          any = true;
          drain(jj);
        }
      }
      if (!any) break;
    }
    // Layer chain: when no reduce or push task is left to claim, the CTAs share the normalisation
    // tasks (one per tile of the rank's partition, band by band) through one counter.  A task
    // waits until all nTn tiles of its band are reduced; the reducing warps read the band from
    // L2 themselves, the ring slot only hands them the task.
    if (NORM && ok && n_lists > 0) {
      while (ok) {
        // Wait for the band at the head of the task counter BEFORE claiming: a CTA that waits
        // holds no task, so the tasks of a band that completes are shared by every CTA that is
        // free at that moment.
        int i = P.Q;
        bool band_ok = true;
        if (lane == 0) {
          const int peek = *reinterpret_cast<volatile int*>(norm_head);
          if (peek < P.Q) {
            band_ok = wait_count(&P.band_ctr[peek / P.nTn], (unsigned)P.nTn, P);
            if (band_ok) i = atomicAdd(norm_head, kRun);
          }
        }
        ok = __all_sync(0xffffffffu, band_ok);
        if (!ok) {
          if (lane == 0) report(P, -ENTWINE_ERR_TIMEOUT, -7);
          break;
        }
        i = __shfl_sync(0xffffffffu, i, 0);
        if (i >= P.Q) break;
        if (REG && ring.id == 0) {
          // the descriptor ring has no memory for the rows to normalise: wait (boundedly) until the
          // CTA's operand stages are free, then move to ring B
          bool open = true;
          if (lane == 0) {
            unsigned long long t0 = 0;
            for (uint32_t spins = 1; !(P.early_b ? sh->stages_free : sh->gemm_done); ++spins) {
              __nanosleep(128);
              if ((spins % kSpinCheck) == 0) {
                if (sh->abort) { open = false; break; }
                const unsigned long long now = globaltimer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > 64ULL * P.wait_budget_ns) { open = false; break; }
              }
            }
          }
          ok = __all_sync(0xffffffffu, open);
          if (!ok) {
            if (lane == 0) report(P, -ENTWINE_ERR_TIMEOUT, -7);
            break;
          }
        }
        maybe_switch();
        if (!ok) break;
        issue_norm_run(i, kRun);
      }
    }
    PROF_FLUSH(lane == 0);
    // end-of-work marker so that the other consumer warps leave their loops
    if (lane == 0) {
      const int slot = it % ring.n_slots;
      const bool free_slot = mbar_wait(ring.empty(slot), ((it / ring.n_slots) & 1) ^ 1, P, sh);
      if (!free_slot) sh->abort = 1;
      sh->meta[ring.id][slot].kind = -1;
      mbar_arrive(ring.full(slot));
    }
    __syncwarp();
  } else if (warp >= kRedWarp0 && warp < kRedWarp0 + kRedThreads / 32) {
    // ---------------- ReduceTile on the slots (Sec. 4.2) ----------------
    reducer_role<NORM, PULL, REG>(P, sh, smem_base, ring);
  } else if (warp == kStoreWarp && lane == 0) {
    // ---------------- forward push slots with TMA stores, recycle all slots ----------------
    // Push stores are kept in flight: a pushed slot is released once its store has read it,
    // which is awaited only when kPend younger stores exist or when this thread would idle.
    constexpr int kPend = 3;
    // pushed tiles are not read again on this GPU
    const uint64_t pol = (P.l2_hints & 1) ? l2_policy_evict_first() : l2_policy_evict_normal();
    unsigned long long pend = 0;  // queue of barrier addresses' slot/ring ids, 8 bits each
    int n_pend = 0;
    // returns the oldest pushed slot: its store has read it (awaited by the caller) and the reducing
    // warps have passed it (they only read a pushed slot's record, so the store does not wait for
    // them: the slot's return does)
    auto retire_one = [&]() {
      const Ring rr = make_ring<REG>(smem_base, int(pend >> 4) & 1, P, sh);
      const int sl = int(pend & 15u);
      if (!mbar_wait(rr.red(sl), uint32_t(pend >> 5) & 1u, P, sh)) sh->abort = 1;
      mbar_arrive(rr.empty(sl));
      pend >>= 8;
      --n_pend;
    };
    auto retire_all = [&]() {
      if (!n_pend) return;
      bulk_wait_read<0>();
      while (n_pend > 0) retire_one();
    };
    int slot = -1;
    uint32_t ph = 0;
    for (;;) {
      if (++slot == ring.n_slots) { slot = 0; ph ^= 1; }
      if (!mbar_try_wait(ring.full(slot), ph)) {
        retire_all();  // nothing to do yet: let the stores in flight return their slots
        if (!mbar_wait(ring.full(slot), ph, P, sh)) {
          sh->abort = 1;
          break;
        }
      }
      const SlotMeta m = sh->meta[ring.id][slot];
      if (m.kind == -1) break;
      if (m.kind == -2) {
        retire_all();
        ring = make_ring<REG>(smem_base, 1, P, sh);
        slot = -1;
        ph = 0;
        continue;
      }
      const uint32_t sbase = ring.base + slot * ring.slot_bytes;
      if (m.kind == 0 || (REG && m.kind >= 4) || (NORM && (m.kind == 2 || m.kind == 3 || m.kind == 6))) {
        if (!mbar_wait(ring.red(slot), ph, P, sh)) {
          sh->abort = 1;
          break;
        }
        if (NORM && ((m.kind == 0 && m.aux >= 0) || (REG && m.kind == 4))) {
          // layer chain: the last step of a reduce task (or a whole task done from registers,
          // whose first destination row is dst_y) counts its tile in the band
          fence_acq_rel_gpu();  // the reducing warps' stores (seen through the barrier) first
          atomicAdd(&P.band_ctr[(REG && m.kind == 4) ? m.dst_y / kTile : m.aux], 1u);
        }
        mbar_arrive(ring.empty(slot));  // reduced and written out by the reducing warps
      } else {
        tma_store_2d_hint(&maps.send_st[ring.geom], m.dst_x, m.dst_y, sbase, pol);
        bulk_commit();
        if (n_pend == kPend) {
          bulk_wait_read<kPend - 1>();  // the oldest store has read its slot
          retire_one();
          if (sh->abort) break;
        }
        pend |= (unsigned long long)(unsigned(slot) | (unsigned(ring.id) << 4) | (ph << 5)) << (8 * n_pend);
        ++n_pend;
      }
    }
    bulk_wait_done<0>();  // every store of this CTA is complete before it exits
  }
}

// ------------------------------------------------------------------------------------------
// Reset of a plan's launch state on the device.  A launch captured into a CUDA graph replays
// with the parameters of the capture, so its flag epoch cannot grow from replay to replay:
// this kernel, captured in front of it, clears the own flags, both sets of head counters and
// both status slots instead, and any epoch above zero then means "published by this run".
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
entwine_reset_kernel(unsigned* flags, int n_flags, int* heads, int n_heads, StatusSlot* status) {
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (int i = tid; i < n_flags; i += nth) flags[i] = 0;
  for (int i = tid; i < n_heads; i += nth) heads[i] = 0;
  if (tid < 2) {
    StatusSlot* s = &status[tid];
    s->code_cta_task = 0;
    s->flags_published = 0;
    s->tiles_reduced = 0;
    s->tiles_pushed = 0;
    s->t_start = ~0ULL;
    s->t_gemm_end = 0;
    s->t_end = 0;
  }
}

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------
// NORM: the layer-chain variant (residual add + RMSNorm in the consumer) is a kernel of its own,
// so that the plain kernel's code and register allocation are untouched by it.
template <int BN, bool PAIR, bool NORM, bool PULL, bool REG>
__global__ void __launch_bounds__(kThreads, 1)
entwine_fused_kernel(const __grid_constant__ KMaps maps, const KParams P) {
  using C = Cfg<BN, PAIR>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ CtaShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  PROF_DECL();
  StatusSlot* st = &P.status[P.seq & 1];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_base + kBarOff + kBarGemm;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kMaxStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * kMaxStages + 2 + a); };
  const int n_stages = P.stages;
  const int stage_bytes = P.kpb * C::kKBlockBytes;
  const uint32_t tmem_slot = smem_base + kBarOff + kBarTmemSlot;
  const uint32_t pair_bar = smem_base + kBarOff + kBarPair;
  const bool is_producer = (int)blockIdx.x < P.G && P.mode != MODE_COMM_ONLY;
  const int g = (int)blockIdx.x;                 // producer index
  const int cidx = (int)blockIdx.x - P.G;        // consumer index of a dedicated consumer CTA
  const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;
  const bool leader = cta_rank == 0;
  // work units of a producer: blocks p = g, g+G, ... or, for pairs, pair indices u = g/2, ...
  // (with a split last wave the last P.split pair tiles count as two units each)
  const int n_full = PAIR ? P.P_blk / 2 - P.split : P.P_blk;
  const int n_units = n_full + (PAIR ? 2 * P.split : 0);
  const int unit0 = PAIR ? g / 2 : g;
  const int stride = PAIR ? P.G / 2 : P.G;
  const int n_my = (is_producer && unit0 < n_units) ? (n_units - unit0 + stride - 1) / stride : 0;

  // Bookkeeping for the NEXT launch, done at the start of this one so that no CTA has anything to
  // do after its last task: head counters and status slots alternate between two sets, and the
  // set this launch does not use was last touched by the previous launch, which is complete.
  if (P.list_head_next) {
    for (int j = blockIdx.x * kThreads + threadIdx.x; j <= P.x; j += gridDim.x * kThreads) P.list_head_next[j] = 0;
  }
  if (P.status_next && blockIdx.x == 0 && threadIdx.x == 0) {
    StatusSlot* nx = P.status_next;
    nx->code_cta_task = 0;
    nx->flags_published = 0;
    nx->tiles_reduced = 0;
    nx->tiles_pushed = 0;
    nx->t_start = ~0ULL;
    nx->t_gemm_end = 0;
    nx->t_end = 0;
    nx->clock = 0;
  }
  // CTA 0 times itself with the SM's cycle counter and the global timer: their ratio is the SM
  // clock this launch really ran at
  long long clk0 = 0;
  unsigned long long ns0 = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    clk0 = clock64();
    ns0 = globaltimer_ns();
  }
  if (threadIdx.x == 0) {
    sh.abort = 0;
    sh.warps_stored = 0;
    sh.gemm_done = (is_producer && n_my > 0) ? 0 : 1;
    sh.stages_free = (is_producer && n_my > 0) ? 0 : 1;
    sh.ring_b_bytes = (is_producer && n_my > 0 && P.early_b) ? P.stage_area : kRingBBytes;
    atomicMin(&st->t_start, globaltimer_ns());
    if (is_producer) {
      for (int s = 0; s < n_stages; ++s) {
        mbar_init(full_bar(s), 1);
        mbar_init(empty_bar(s), 1);
      }
      for (int a = 0; a < 2; ++a) {
        mbar_init(tfull_bar(a), 1);
        mbar_init(tempty_bar(a), (PAIR ? 2 : 1) * (kEpiThreads / 32));
      }
      mbar_init(pair_bar, 1);
    }
    for (int ring = 0; ring < 2; ++ring) {  // consumer rings: full, empty, reduced
      const uint32_t rb = smem_base + kBarOff + (ring == 0 ? kBarRingA : kBarRingB);
      for (int s = 0; s < kMaxSlots; ++s) {
        mbar_init(rb + 8u * s, 1);
        mbar_init(rb + 8u * (kMaxSlots + s), 1);
        mbar_init(rb + 8u * (2 * kMaxSlots + s), kRedThreads / 32);
      }
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (is_producer && warp == kMmaWarp) {
    if (PAIR) tmem_alloc_pair(tmem_slot, C::kTmemCols);
    else tmem_alloc(tmem_slot, C::kTmemCols);
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR && is_producer) cluster_sync_all();  // both CTAs' barriers exist before either signals
  tc_fence_after();

  CommCounters cnt;
  unsigned published = 0;
  const bool gemm_warp = warp == kTmaWarp || warp == kMmaWarp || warp == kSpareWarp || warp == kFlagWarp ||
                         (warp >= kEpiWarp0 && warp < kEpiWarp0 + 4);
  const bool comm_warp = warp == kCommWarp || warp == kStoreWarp ||
                         (warp >= kRedWarp0 && warp < kRedWarp0 + kRedThreads / 32);

  if (is_producer && gemm_warp) {
    // ---------------- producer: tcgen05 GEMM ----------------
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(smem + kBarOff + kBarTmemSlot);
    const int KB = (P.K + kBK - 1) / kBK;
    // block i of this CTA: its position in the tile order (returned), its destination partition
    // d and its index l inside the partition
    // *half: -1 for a whole block; 0 / 1 when this unit is the left / right 128 columns of it
    auto block_of = [&](int i, int* d, int* l, int* half) {
      int unit = unit0 + i * stride;
      *half = -1;
      if (PAIR && unit >= n_full) {
        *half = (unit - n_full) & 1;
        unit = n_full + ((unit - n_full) >> 1);
      }
      const int p = PAIR ? pair_position(P, unit, (int)cta_rank) : unit;
      position_to_block(P, p, d, l);
      return p;
    };

    // The two single-thread loops of the producer, compiled once per (k-blocks per stage, layout of B):
    // with those as run-time values the issuing threads measured 8-10 % slower on long-K shapes.
    auto tma_loop = [&](auto kpb_c, auto bkn_c) -> bool {
      constexpr int KPB = decltype(kpb_c)::value;
      constexpr bool BKN = decltype(bkn_c)::value;
      constexpr int kStage = KPB * C::kKBlockBytes;
      // operand panels are re-read by many CTAs: ask L2 to keep them
      const uint64_t op_pol = (P.l2_hints & 2) ? l2_policy_evict_last() : l2_policy_evict_normal();
      const bool k3d = KPB > 1 && P.k3d;
      int stage = 0;
      uint32_t phase = 0;
      for (int i = 0; i < n_my; ++i) {
        int d, l, half;
        block_of(i, &d, &l, &half);
        const int mb = d * P.rowsT + l / P.nBn, nb = l % P.nBn;
        // rows of B this CTA loads: its half of the block's columns, or of the half block's
        const int b_rows = half < 0 ? C::kBRows : C::kBRows / 2;
        const int b_row = nb * BN + (half < 0 ? 0 : half * (BN / 2)) + (PAIR ? (int)cta_rank * b_rows : 0);
        const int b_bytes = b_rows * kBK * 2;  // one k-block of them
        const CUtensorMap* const mb2 = half < 0 ? &maps.b : &maps.bh;
        const CUtensorMap* const mb3 = BKN ? (half < 0 ? &maps.bkn : &maps.bknh) : (half < 0 ? &maps.b3 : &maps.bh3);
        for (int kb0 = 0; kb0 < KB; kb0 += KPB) {
          {
            PROF_T0();
            const bool got = mbar_wait(empty_bar(stage), phase ^ 1, P, &sh);
            PROF_ADD(0);
            if (!got) return false;
          }
          const uint32_t a_dst = smem_base + stage * kStage;
          const uint32_t b_dst = a_dst + KPB * C::kABytes;
          // k-blocks of this stage that exist (a ragged last stage is filled, and multiplied, in part)
          const int nkb = KPB == 1 ? 1 : min(KPB, KB - kb0);
          const uint32_t fbar = full_bar(stage);
          const uint32_t lead_bar = PAIR ? map_to_cta(fbar, 0) : fbar;
          // bytes this CTA brings: A as one 3-D box of KPB k-blocks (k-blocks past the end of K read
          // as zero and count) or k-block by k-block; B [K, N] always as one box of KPB * 64 k-rows
          const uint32_t a_tx = (k3d ? KPB : nkb) * C::kABytes;
          const uint32_t b_tx = ((BKN || k3d) ? KPB : nkb) * b_bytes;
          if (PAIR) {
            // both CTAs' bytes are counted on the leader's barrier, which the leader arms
            if (leader) mbar_arrive_expect_tx(fbar, 2 * (a_tx + b_tx));
          } else {
            mbar_arrive_expect_tx(fbar, a_tx + b_tx);
          }
          if (k3d) {
            if (PAIR) tma_load_3d_pair_hint(a_dst, &maps.a3, 0, mb * kBM, kb0, lead_bar, op_pol);
            else tma_load_3d_hint(a_dst, &maps.a3, 0, mb * kBM, kb0, fbar, op_pol);
          } else {
#pragma unroll
            for (int kk = 0; kk < KPB; ++kk) {
              if (kk < nkb) {
                if (PAIR) tma_load_2d_pair_hint(a_dst + kk * C::kABytes, &maps.a, (kb0 + kk) * kBK, mb * kBM, lead_bar, op_pol);
                else tma_load_2d_hint(a_dst + kk * C::kABytes, &maps.a, (kb0 + kk) * kBK, mb * kBM, fbar, op_pol);
              }
            }
          }
          if (BKN) {
            // B as [K, N]: one box [groups of 64 columns][KPB * 64 k-rows][64], rows past K read as zero
            if (PAIR) tma_load_3d_pair_hint(b_dst, mb3, 0, kb0 * kBK, b_row / 64, lead_bar, op_pol);
            else tma_load_3d_hint(b_dst, mb3, 0, kb0 * kBK, b_row / 64, fbar, op_pol);
          } else if (k3d) {
            // one box per operand: [KPB k-blocks][rows][64]
            if (PAIR) tma_load_3d_pair_hint(b_dst, mb3, 0, b_row, kb0, lead_bar, op_pol);
            else tma_load_3d_hint(b_dst, mb3, 0, b_row, kb0, fbar, op_pol);
          } else {
#pragma unroll
            for (int kk = 0; kk < KPB; ++kk) {
              if (kk < nkb) {
                if (PAIR) tma_load_2d_pair_hint(b_dst + kk * b_bytes, mb2, (kb0 + kk) * kBK, b_row, lead_bar, op_pol);
                else tma_load_2d_hint(b_dst + kk * b_bytes, mb2, (kb0 + kk) * kBK, b_row, fbar, op_pol);
              }
            }
          }
          if (++stage == n_stages) { stage = 0; phase ^= 1; }
        }
      }
      return true;
    };
    auto mma_loop = [&](auto kpb_c, auto bkn_c) -> bool {
      constexpr int KPB = decltype(kpb_c)::value;
      constexpr bool BKN = decltype(bkn_c)::value;
      constexpr int kStage = KPB * C::kKBlockBytes;
      constexpr uint32_t kBMajor = BKN ? (1u << 16) : 0u;  // B operand MN-major
      const uint32_t idesc_full = instr_desc<BN, PAIR ? 256 : 128>() | kBMajor;
      const uint32_t idesc_half = instr_desc<BN / 2, PAIR ? 256 : 128>() | kBMajor;
      // K advances by 16 elements per instruction: 32 bytes inside a row (K-major, 2 address units),
      // 16 rows of 128 bytes (MN-major B)
      constexpr uint32_t kBStep = BKN ? (kUmmaK * 128) >> 4 : 2;
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      for (int i = 0; i < n_my; ++i) {
        int d_, l_, half;
        block_of(i, &d_, &l_, &half);
        const uint32_t idesc = half < 0 ? idesc_full : idesc_half;
        const int b_bytes = (half < 0 ? C::kBRows : C::kBRows / 2) * kBK * 2;
        {
          PROF_T0();
          const bool got = mbar_wait(tempty_bar(acc), acc_phase ^ 1, P, &sh);
          PROF_ADD(1);
          if (!got) return false;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb0 = 0; kb0 < KB; kb0 += KPB) {
          {
            PROF_T0();
            const bool got = mbar_wait(full_bar(stage), phase, P, &sh);
            PROF_ADD(2);
            if (!got) return false;
          }
          tc_fence_after();
          const uint32_t a_s = smem_base + stage * kStage;
          const uint32_t b_s = a_s + KPB * C::kABytes;
          const int nkb = KPB == 1 ? 1 : min(KPB, KB - kb0);
#pragma unroll
          for (int kk = 0; kk < KPB; ++kk) {
            if (kk < nkb) {
              const uint64_t a_desc = smem_desc_sw128(a_s + kk * C::kABytes);
              // B K-major: k-block kk of this CTA's rows; B MN-major: k-rows [64 kk, 64 kk + 64) of
              // every 64-column group (groups KPB * 8 KiB apart)
              const uint64_t b_desc = BKN ? smem_desc_sw128_mn(b_s + kk * (kBK * 128), KPB * (kBK * 128))
                                          : smem_desc_sw128(b_s + kk * b_bytes);
#pragma unroll
              for (int k = 0; k < kBK / kUmmaK; ++k) {
                if (PAIR) umma_bf16_pair(d_tmem, a_desc + 2 * k, b_desc + kBStep * k, idesc, (kb0 | kk | k) != 0);
                else umma_bf16(d_tmem, a_desc + 2 * k, b_desc + kBStep * k, idesc, (kb0 | kk | k) != 0);
              }
            }
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if (PAIR) tc_commit_pair(empty_bar(stage));
          else tc_commit(empty_bar(stage));
          if (++stage == n_stages) { stage = 0; phase ^= 1; }
        }
        if (PAIR) tc_commit_pair(tfull_bar(acc));  // accumulator complete (both CTAs' halves)
        else tc_commit(tfull_bar(acc));
        if ((acc ^= 1) == 0) acc_phase ^= 1;
      }
      return true;
    };
    using Kpb1 = std::integral_constant<int, 1>;
    using Kpb2 = std::integral_constant<int, 2>;

    if (warp == kTmaWarp && lane == 0) {
      // ---- TMA producer (every CTA loads its own operands) ----
      bool ok;
      if (P.kpb == 2) ok = P.b_kn ? tma_loop(Kpb2{}, std::true_type{}) : tma_loop(Kpb2{}, std::false_type{});
      else ok = P.b_kn ? tma_loop(Kpb1{}, std::true_type{}) : tma_loop(Kpb1{}, std::false_type{});
      if (!ok) { sh.abort = 1; report(P, -ENTWINE_ERR_TIMEOUT, -1); }
    } else if (warp == kMmaWarp && lane == 0 && leader) {
      // ---- MMA issuer (the leader CTA issues for the pair) ----
#ifdef ENTWINE_PROFILE
      const long long prof_mma0 = clock64();
#endif
      bool ok;
      if (P.kpb == 2) ok = P.b_kn ? mma_loop(Kpb2{}, std::true_type{}) : mma_loop(Kpb2{}, std::false_type{});
      else ok = P.b_kn ? mma_loop(Kpb1{}, std::true_type{}) : mma_loop(Kpb1{}, std::false_type{});
#ifdef ENTWINE_PROFILE
      prof_acc_[8] += (unsigned long long)(clock64() - prof_mma0);
#endif
      if (!ok) { sh.abort = 1; report(P, -ENTWINE_ERR_TIMEOUT, -2); }
    } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + 4) {
      // ---- epilogue: TMEM -> bf16 -> global.  A warp owns 32 rows of the block (its TMEM lane
      //      quarter).  Its threads round their rows to bf16 into the warp's own swizzled staging
      //      (32 rows x 128 bytes), the warp reads that back row-wise and stores whole 128-byte
      //      lines of the partial C with plain 16-byte stores: no other warp, no copy engine and no
      //      buffer hand-over lies between the accumulator and memory.  After a block's stores
      //      the warp counts itself in warps_stored (release); the flag warp publishes the
      //      block's tiles when all four have (Sec. 4.2: flags after all of the block's stores) ----
      const int q = warp & 3;  // TMEM lane quarter this warp may read = its 32 rows of the block
      const uint32_t wstage = smem_base + n_stages * stage_bytes + q * kEpiWarpBytes;
      const uint32_t my_row = wstage + lane * 128;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
#ifdef ENTWINE_PROFILE
      const long long prof_epi0 = clock64();
#endif
      for (int i = 0; ok && i < n_my; ++i) {
        int d, l, half;
        block_of(i, &d, &l, &half);
        const int mb = d * P.rowsT + l / P.nBn, nb = l % P.nBn;
        const int n_cols64 = half < 0 ? BN / 64 : BN / 128;        // 64-column units of this unit
        const int col0 = nb * BN + (half < 0 ? 0 : half * (BN / 2));
        {
          PROF_T0();
          ok = mbar_wait(tfull_bar(acc), acc_phase, P, &sh);
          if (warp == kEpiWarp0 && lane == 0) PROF_ADD(3);
        }
        ok = __all_sync(0xffffffffu, ok);  // reconverge; the warp leaves the loop together
        if (!ok) break;
        tc_fence_after();
        if (i == n_my - 1 && warp == kEpiWarp0 && lane == 0) {
          // the CTA's (and, on a pair, the cluster's) last MMA has read the operand stages
          __threadfence_block();
          sh.stages_free = 1;
        }
        const uint32_t taddr = tmem_base + (uint32_t(q * 32) << 16) + acc * BN;
        // this lane's share of a read-back: row (lane / 8) + 4 * it of the warp's 32, 16-byte chunk lane % 8
        __nv_bfloat16* const cdst = P.cws_out + (long long)(mb * kBM + q * 32 + (lane >> 3)) * P.N + col0 + (lane & 7) * 8;
        // Two register sets: the TMEM load of the next 32 columns is in flight while the previous
        // 32 are rounded and staged (a tcgen05.ld takes a few hundred cycles).
        uint32_t va[32], vb[32];
        // rounds 32 fp32 values of this thread's row to bf16 (nearest even) and writes them as
        // four 16-byte chunks of the row's 128 swizzled bytes
        auto stage32 = [&](const uint32_t (&v)[32], int cc) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            uint4 o;
            uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(v[8 * e + 2 * u]),
                                                        __uint_as_float(v[8 * e + 2 * u + 1]));
              ow[u] = *reinterpret_cast<uint32_t*>(&hh);
            }
            const int chunk = cc * 4 + e;  // 16-byte chunk inside the 128-byte row
            st_shared_v4(my_row + ((chunk ^ (lane & 7)) << 4), o);
          }
        };
        tmem_ld32(taddr, va);
#pragma unroll 1
        for (int j = 0; j < n_cols64; ++j) {
          tmem_ld_wait();                                // columns [64 j, 64 j + 32) are in va
          tmem_ld32(taddr + j * 64 + 32, vb);
          stage32(va, 0);
          tmem_ld_wait();                                // columns [64 j + 32, 64 j + 64) are in vb
          if (j + 1 < n_cols64) {
            tmem_ld32(taddr + (j + 1) * 64, va);
          } else {
            // last read of this accumulator: the MMA warp may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              if (leader) mbar_arrive(tempty_bar(acc));
              else mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
            }
          }
          stage32(vb, 1);
          __syncwarp();
          // row-wise read-back: eight lanes carry one row's 128 bytes, four rows per instruction
          uint4 o[8];
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int row = it * 4 + (lane >> 3);
            o[it] = ld_shared_v4(wstage + row * 128 + (((lane & 7) ^ (row & 7)) << 4));
          }
          __syncwarp();  // the staging may be overwritten
#pragma unroll
          for (int it = 0; it < 8; ++it)
            __stcg(reinterpret_cast<uint4*>(cdst + (long long)(it * 4) * P.N + j * 64), o[it]);
        }
        // the block's stores of this warp are issued; the counter's release orders them before
        // whatever the flag warp does after it has read the count
        __syncwarp();
        if (lane == 0) red_release_cta_add(&sh.warps_stored, 1);
        if ((acc ^= 1) == 0) acc_phase ^= 1;
      }
#ifdef ENTWINE_PROFILE
      if (warp == kEpiWarp0 && lane == 0) prof_acc_[9] += (unsigned long long)(clock64() - prof_epi0);
#endif
      if (!ok && lane == 0) { sh.abort = 1; report(P, -ENTWINE_ERR_TIMEOUT, -3); }
    } else if (warp == kFlagWarp) {
      // ---- flag warp: releases the tile flags of every block whose stores are complete
      //      (Sec. 4.2).  The release fence takes about a microsecond when memory is busy; in a
      //      warp of its own it delays neither the epilogue nor the stores.  Lane 0 waits and
      //      counts; a group release (the granularity ablation) is spread over the lanes ----
      int seen = 0;
      unsigned long long t0 = 0;
      // half < 0: all tiles of the block; else the one tile a half-width unit covers
      auto release_block = [&](int dd, int ll, int half) {
        const int t_first = (ll / P.nBn) * P.nTn + (ll % P.nBn) * P.cpb + (half < 0 ? 0 : half);
        const int n_t = half < 0 ? P.cpb : 1;
        if (PULL && dd != P.r) {
          // the flag goes to its reader: row r of destination dd's flag array
          unsigned* f = reinterpret_cast<unsigned*>(P.heap + dd * P.heap_stride + P.heap_flags_off) + P.r * P.Q;
          for (int c = 0; c < n_t; ++c) st_relaxed_sys(&f[t_first + c], P.epoch);
        } else {
          for (int c = 0; c < n_t; ++c) st_relaxed_gpu(&P.flags_own[dd * P.Q + t_first + c], P.epoch);
        }
        published += n_t;
      };
      for (int i = 0; i < n_my; ++i) {
        int d, l, half;
        const int pos = block_of(i, &d, &l, &half);
        // what lane 0 finds: 0 = stop (abort / timeout), 1 = nothing to release for this block,
        // 2 = release the group [first, first + gsize) (or partition d)
        int verdict = 0, first = 0, gsize = 1;
        if (lane == 0) {
          for (uint32_t spins = 1; seen <= i; ++spins) {
            seen = ld_acquire_cta(&sh.warps_stored) / (kEpiThreads / 32);
            if (seen > i) break;
            __nanosleep(64);
            if ((spins % kSpinCheck) == 0) {
              if (sh.abort || global_abort(P)) break;
              const unsigned long long now = globaltimer_ns();
              if (t0 == 0) t0 = now;
              else if (now - t0 > 64ULL * P.wait_budget_ns) {
                sh.abort = 1;
                report(P, -ENTWINE_ERR_TIMEOUT, -6);
                break;
              }
            }
          }
          if (seen > i) {
            t0 = 0;
            // the epilogue warps' stores (generic-proxy writes, ordered before the count this thread
            // acquired), then the flags (a consumer that reads the tile with TMA orders its
            // async-proxy reads after its own acquire); system scope only where the flags go to
            // another GPU
            {
              PROF_T0();
              if (PULL && d != P.r) fence_acq_rel_sys();
              else fence_acq_rel_gpu();
              PROF_ADD(7);
            }
            if (P.release_group == 1) {
              release_block(d, l, half);
              verdict = 1;
            } else {
              // Coarser release: the block is counted in its group; whoever stores a group's
              // last block releases the flags of all its blocks.  Counts are taken modulo the
              // group's size: every launch adds exactly that much.
              int gid;
              if (P.release_group == ENTWINE_RELEASE_WHOLE) { gid = 0; gsize = P.P_blk; }
              else if (P.release_group == ENTWINE_RELEASE_PARTITION) { gid = d; gsize = P.Lb; }
              else {
                gid = pos / P.release_group;
                first = gid * P.release_group;
                gsize = min(P.release_group, P.P_blk - first);
              }
              const unsigned prev = atomicAdd(&P.group_ctr[gid], 1u);
              verdict = ((prev + 1u) % (unsigned)gsize == 0u) ? 2 : 1;
            }
          }
        }
        verdict = __shfl_sync(0xffffffffu, verdict, 0);
        if (verdict == 0) break;
        if (verdict == 1) continue;
        first = __shfl_sync(0xffffffffu, first, 0);
        gsize = __shfl_sync(0xffffffffu, gsize, 0);
        fence_acq_rel_gpu();  // the other blocks' stores, released by their CTAs' counts
        for (int j = lane; j < gsize; j += 32) {
          if (P.release_group == ENTWINE_RELEASE_PARTITION) {
            release_block(d, j, -1);
          } else {
            int dd, ll;
            position_to_block(P, first + j, &dd, &ll);
            release_block(dd, ll, -1);
          }
        }
      }
      // every lane's count of released flags, summed into lane 0
      for (int o = 16; o > 0; o >>= 1) published += __shfl_down_sync(0xffffffffu, published, o);
    }
    // ---- end of this CTA's producer work ----
    named_bar_sync(3, kGemmThreads);
    if (warp == kTmaWarp && lane == 0 && n_my > 0) atomicMax(&st->t_gemm_end, globaltimer_ns());
    if (sh.abort) {
      // give copies that may still be in flight time to land before the CTA's memory is reused
      const unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ULL) __nanosleep(1000);
    }
    if (PAIR) {
      // the peer may still signal this CTA's barriers until its producer warps are done too
      if (warp == kMmaWarp && lane == 0) {
        mbar_arrive_cluster(map_to_cta(pair_bar, cta_rank ^ 1));
        if (!mbar_wait(pair_bar, 0, P, &sh)) { sh.abort = 1; report(P, -ENTWINE_ERR_TIMEOUT, -4); }
      }
      named_bar_sync(3, kGemmThreads);
    }
    tc_fence_after();
    if (warp == kMmaWarp) {
      if (PAIR) tmem_dealloc_pair(tmem_base, C::kTmemCols);
      else tmem_dealloc(tmem_base, C::kTmemCols);
    }
    if (warp == kTmaWarp && lane == 0) {
      __threadfence_block();
      sh.gemm_done = 1;  // the consumer warps may take over the producer's shared memory
    }
    if (warp == kFlagWarp && lane == 0 && published)
      atomicAdd(&st->flags_published, (unsigned long long)published);
  } else if (comm_warp && P.mode != MODE_GEMM_ONLY) {
    // ---------------- consumer ----------------
    int first = 0, count = 0;
    bool on_a = false;
    if (!is_producer) {
      // dedicated consumer block j: its own list, then (shared-pool analogue) the others
      first = cidx % P.x;
      count = (cidx < P.x && !P.help) ? 1 : P.x;
    } else {
      if (P.n_ded == 0) {
        // no dedicated consumers: block g owns list g (and helps with the others)
        first = g % P.x;
        count = P.help ? P.x : (g < P.x ? 1 : 0);
      } else if (P.help) {
        first = g % P.x;
        count = P.x;
      }
      on_a = n_my > 0;
      if (count > 0 && on_a && !P.colocate) {
        // not co-located: wait for the CTA's producer work to end, then use ring B
        unsigned long long t0 = globaltimer_ns();
        while (!(P.early_b ? sh.stages_free : sh.gemm_done) && !sh.abort) {
          __nanosleep(256);
          if (globaltimer_ns() - t0 > 64ULL * P.wait_budget_ns) break;
        }
        on_a = false;
      }
    }
    if (count > 0 && !sh.abort) {
      consumer_pipeline<NORM, PULL, REG>(P, maps, &sh, smem_base, first, count, on_a, &cnt);
    }
    if (warp == kCommWarp && lane == 0) {
      if (cnt.reduced) atomicAdd(&st->tiles_reduced, (unsigned long long)cnt.reduced);
      if (cnt.pushed) atomicAdd(&st->tiles_pushed, (unsigned long long)cnt.pushed);
    }
  }

  // ---------------- exit bookkeeping ----------------
  PROF_FLUSH(true);
  __syncthreads();
  if (threadIdx.x == 0) atomicMax(&st->t_end, globaltimer_ns());
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    const unsigned long long cyc = (unsigned long long)(clock64() - clk0), ns = globaltimer_ns() - ns0;
    st->clock = (min(cyc, 0xffffffffULL) << 32) | min(ns, 0xffffffffULL);
  }
}

// ------------------------------------------------------------------------------------------
// host side: device resources and launches
// ------------------------------------------------------------------------------------------
struct DeviceState {
  int device = -1;
  __nv_bfloat16* C = nullptr;
  unsigned* flags_own = nullptr;
  unsigned* flags_peer = nullptr;
  Task* tasks = nullptr;
  int* list_offs = nullptr;
  int* list_head = nullptr;
  StatusSlot* status = nullptr;
  unsigned* group_ctr = nullptr;
  Task* tasks_pull = nullptr;     // pull mode: the reduce tasks alone, and their lists
  int* list_offs_pull = nullptr;
  float* ssq_part = nullptr;     // layer chain: [R][nTn]
  unsigned* band_ctr = nullptr;  // layer chain: [rowsT]
  unsigned epoch = 0;
  unsigned seq = 0;
  bool user_ws = false;   // the arrays below live in the caller's workspace (nothing of them is freed here)
  bool captured = false;  // a launch of this plan has been captured into a CUDA graph
  bool status_pending = false;
  cudaStream_t last_stream = nullptr;
  cudaEvent_t switch_event = nullptr;  // orders a new stream after the plan's last launch
  unsigned long long last_clock = 0;   // cycles << 32 | ns of CTA 0 in the launch entwine_last_status read
  int64_t withheld = -1;
  // staging for the host-buffer entry point
  cudaStream_t own_stream = nullptr;
  // pipelined host-buffer calls: two staging sets, copies up and down on streams of their own
  struct HostPipe {
    cudaStream_t up = nullptr, comp = nullptr, down = nullptr;
    cudaEvent_t up_done[2] = {nullptr, nullptr}, k_done[2] = {nullptr, nullptr}, d_done[2] = {nullptr, nullptr};
    __nv_bfloat16 *A[2] = {nullptr, nullptr}, *B[2] = {nullptr, nullptr}, *peers[2] = {nullptr, nullptr};
    __nv_bfloat16 *out[2] = {nullptr, nullptr}, *send[2] = {nullptr, nullptr};
    uint64_t issued = 0, waited = 0;
  };
  HostPipe* pipe = nullptr;
  __nv_bfloat16 *sA = nullptr, *sB = nullptr, *sPeers = nullptr, *sOut = nullptr, *sSend = nullptr;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// 2-D map over a row-major bf16 matrix [rows, cols] with a (box_rows x box_cols) box;
// out-of-range elements read as zero (K tails).  `swizzle128` selects the 128-byte swizzle
// (box_cols must then be 64 elements = 128 bytes).
static bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_cols,
                     int box_rows, bool swizzle128, int64_t pitch_elems = 0) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cuuint64_t(cols), cuuint64_t(rows)};
  cuuint64_t strides[1] = {cuuint64_t(pitch_elems > 0 ? pitch_elems : cols) * 2};
  cuuint32_t box[2] = {cuuint32_t(box_cols), cuuint32_t(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS;
}

// 3-D map over bf16 [planes][rows][cols] with a (box_planes x box_rows x box_cols) box, no swizzle.
static bool make_map3(CUtensorMap* map, const void* base, int64_t planes, int64_t rows, int64_t cols,
                      int box_cols, int box_rows, int box_planes, int64_t plane_stride_bytes = 0) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {cuuint64_t(cols), cuuint64_t(rows), cuuint64_t(planes)};
  cuuint64_t strides[2] = {cuuint64_t(cols) * 2, cuuint64_t(cols) * cuuint64_t(rows) * 2};
  if (plane_stride_bytes > 0) strides[1] = cuuint64_t(plane_stride_bytes);
  cuuint32_t box[3] = {cuuint32_t(box_cols), cuuint32_t(box_rows), cuuint32_t(box_planes)};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS;
}

// Operand maps of the producer.  a / b: one k-block (64 elements of K, 128-byte swizzle) per box.
// a3 / b3: the same matrix seen as [K/64][rows][64] (k-blocks 128 bytes apart inside a row), so that
// one box of kpb k-blocks fills a whole pipeline stage of that operand with one TMA instruction;
// only where K is a multiple of 64 (the view has no partial k-block).  Returns false on an
// encoding failure; *k3d tells whether the 3-D maps are usable.
static bool make_operand_maps(KMaps* maps, const void* A, const void* B, const Geometry& g, int b_rows, int kpb,
                              int64_t lda, int64_t ldb, int b_kn, int* k3d) {
  *k3d = 0;
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if ((lda > 0 && lda < g.K) || (ldb > 0 && ldb < (b_kn ? g.N : g.K))) return false;
  // (bh, bh3: half as many rows of B per box, for the half-width units of a split last wave)
  if (!make_map(&maps->a, A, g.M, g.K, kBK, kBM, true, lda)) return false;
  if (b_kn) {
    // B [K, N] seen as [N/64][K][64]: groups of 64 columns are 128 bytes apart inside a row of B
    for (int h = 0; h < 2; ++h) {
      const int groups = std::max(1, (h == 0 ? b_rows : b_rows / 2) / 64);
      cuuint64_t dims[3] = {64, cuuint64_t(g.K), cuuint64_t(g.N / 64)};
      cuuint64_t strides[2] = {cuuint64_t(ldb > 0 ? ldb : g.N) * 2, 128};
      cuuint32_t box[3] = {64, cuuint32_t(kBK * kpb), cuuint32_t(groups)};
      cuuint32_t estr[3] = {1, 1, 1};
      if (fn(h == 0 ? &maps->bkn : &maps->bknh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(B), dims, strides,
             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    }
  } else if (!make_map(&maps->b, B, g.N, g.K, kBK, b_rows, true, ldb) ||
             !make_map(&maps->bh, B, g.N, g.K, kBK, b_rows / 2, true, ldb)) {
    return false;
  }
  if (kpb < 2 || g.K % kBK != 0) return true;
  bool ok = true;
  for (int op = 0; op < (b_kn ? 1 : 3); ++op) {
    const int64_t rows = op == 0 ? g.M : g.N;
    const int64_t ld = op == 0 ? (lda > 0 ? lda : g.K) : (ldb > 0 ? ldb : g.K);
    cuuint64_t dims[3] = {cuuint64_t(kBK), cuuint64_t(rows), cuuint64_t(g.K / kBK)};
    cuuint64_t strides[2] = {cuuint64_t(ld) * 2, cuuint64_t(kBK) * 2};
    cuuint32_t box[3] = {cuuint32_t(kBK), cuuint32_t(op == 0 ? kBM : (op == 1 ? b_rows : b_rows / 2)), cuuint32_t(kpb)};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult rc = fn(op == 0 ? &maps->a3 : (op == 1 ? &maps->b3 : &maps->bh3), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                     const_cast<void*>(op == 0 ? A : B), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    ok = ok && rc == CUDA_SUCCESS;
  }
  *k3d = ok ? 1 : 0;  // without them a stage is filled k-block by k-block
  return true;
}

// Split last wave (CTA pairs only): if the pair tiles left over after the last full wave occupy at
// most half of the n_pairs CTA pairs, each of them is done as two half-width units on two pairs, and
// the last wave costs half a tile time.  Returns how many pair tiles are split.
static int split_last_wave(const Plan* p, int n_producer_ctas) {
  if (!p->pair || !p->split_opt || p->release_group != 1) return 0;
  const int n_pairs = n_producer_ctas / 2, n_tiles = p->g.P_blk / 2;
  if (n_pairs < 1) return 0;
  const int rest = n_tiles % n_pairs;
  return (rest > 0 && 2 * rest <= n_pairs) ? rest : 0;
}

// Tasks per claim: as many as have their flags (W per reduce task) in the 64 flag values the
// claiming warp reads ahead, at most four (two where several CTAs share a list).
#ifndef ENTWINE_CLAIM_MAX
#define ENTWINE_CLAIM_MAX 4
#endif
static int claim_size(int W) { return std::max(1, std::min(ENTWINE_CLAIM_MAX, 64 / W)); }

int device_sm_count() {
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return -1;
  }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
  return sms;
}

#define CK(call)                           \
  do {                                     \
    cudaError_t e_ = (call);               \
    if (e_ != cudaSuccess) {               \
      cudaGetLastError();                  \
      return ENTWINE_ERR_CUDA;             \
    }                                      \
  } while (0)

// Plan-owned device memory: one section per array, each starting on a 256-byte boundary.  The same
// layout serves cudaMalloc'ed arrays (one allocation each) and a caller-provided workspace (one
// block, entwine_plan_set_workspace), which also holds what the layer chain and the pull mode
// would otherwise allocate at their first call.
struct WorkspaceLayout {
  size_t c, flags_own, flags_peer, tasks, list_offs, list_head, status, group_ctr, ssq_part, band_ctr, tasks_pull,
      list_offs_pull, total;
};
static size_t align256(size_t v) { return (v + 255) / 256 * 256; }
static WorkspaceLayout workspace_layout(const Plan* p) {
  const Geometry& g = p->g;
  const HostTables& t = p->tables;
  WorkspaceLayout w;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off += align256(std::max<size_t>(bytes, 1)); return at; };
  w.c = take(size_t(g.M) * g.N * 2);
  w.flags_own = take(size_t(g.W) * g.Q * 4);
  w.flags_peer = take(size_t(g.W - 1) * g.Q * 4);
  w.tasks = take(t.dev_tasks.size() * sizeof(Task));
  w.list_offs = take(t.list_offs.size() * 4);
  w.list_head = take(size_t(p->x + 1) * 2 * 4);
  w.status = take(2 * sizeof(StatusSlot));
  w.group_ctr = take(size_t(g.P_blk) * 4);
  w.ssq_part = take(size_t(g.R) * g.nTn * 4);
  w.band_ctr = take(size_t(g.rowsT) * 4);
  w.tasks_pull = take(t.pull_tasks.size() * sizeof(Task));
  w.list_offs_pull = take(t.pull_list_offs.size() * 4);
  w.total = off;
  return w;
}

// The partial-output workspace C[M,N] of a plan that allocates its own memory is allocated when a
// call first needs it: pull mode keeps its partial in the heap and never does.
static int ensure_partial_c(Plan* p) {
  DeviceState* d = p->dev;
  if (d->C) return ENTWINE_OK;
  const size_t bytes = size_t(p->g.M) * p->g.N * 2;
  if (cudaMalloc(&d->C, bytes) != cudaSuccess || cudaMemset(d->C, 0, bytes) != cudaSuccess) {
    cudaGetLastError();
    return ENTWINE_ERR_CUDA;
  }
  return ENTWINE_OK;
}

static int ensure_device(Plan* p, bool need_c = true) {
  if (p->dev) return need_c ? ensure_partial_c(p) : ENTWINE_OK;
  int sms = device_sm_count();
  if (sms <= 0) return ENTWINE_ERR_CUDA;
  int dev = 0;
  CK(cudaGetDevice(&dev));
  int major = 0;
  CK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return ENTWINE_ERR_RESOURCES;  // tcgen05 / TMEM needed
  if (p->num_sms > sms) return ENTWINE_ERR_RESOURCES;
  const WorkspaceLayout w = workspace_layout(p);
  if (p->ws_ptr && p->ws_bytes < w.total) return ENTWINE_ERR_INVALID;  // the tables grew after set_workspace
  DeviceState* d = new DeviceState();
  d->device = dev;
  const Geometry& g = p->g;
  const size_t n_own = size_t(g.W) * g.Q, n_peer = size_t(g.W - 1) * g.Q;
  const HostTables& t = p->tables;
  bool ok;
  if (p->ws_ptr) {
    char* b = static_cast<char*>(p->ws_ptr);
    d->user_ws = true;
    d->C = reinterpret_cast<__nv_bfloat16*>(b + w.c);
    d->flags_own = reinterpret_cast<unsigned*>(b + w.flags_own);
    d->flags_peer = reinterpret_cast<unsigned*>(b + w.flags_peer);
    d->tasks = reinterpret_cast<Task*>(b + w.tasks);
    d->list_offs = reinterpret_cast<int*>(b + w.list_offs);
    d->list_head = reinterpret_cast<int*>(b + w.list_head);
    d->status = reinterpret_cast<StatusSlot*>(b + w.status);
    d->group_ctr = reinterpret_cast<unsigned*>(b + w.group_ctr);
    d->ssq_part = reinterpret_cast<float*>(b + w.ssq_part);
    d->band_ctr = reinterpret_cast<unsigned*>(b + w.band_ctr);
    d->tasks_pull = reinterpret_cast<Task*>(b + w.tasks_pull);
    d->list_offs_pull = reinterpret_cast<int*>(b + w.list_offs_pull);
    ok = cudaMemcpy(d->tasks_pull, t.pull_tasks.data(), t.pull_tasks.size() * sizeof(Task), cudaMemcpyHostToDevice) ==
             cudaSuccess &&
         cudaMemcpy(d->list_offs_pull, t.pull_list_offs.data(), t.pull_list_offs.size() * 4, cudaMemcpyHostToDevice) ==
             cudaSuccess;
  } else {
    ok = (!need_c || cudaMalloc(&d->C, size_t(g.M) * g.N * 2) == cudaSuccess) &&
         cudaMalloc(&d->flags_own, n_own * 4) == cudaSuccess &&
         cudaMalloc(&d->flags_peer, n_peer * 4) == cudaSuccess &&
         cudaMalloc(&d->tasks, t.dev_tasks.size() * sizeof(Task)) == cudaSuccess &&
         cudaMalloc(&d->list_offs, t.list_offs.size() * 4) == cudaSuccess &&
         cudaMalloc(&d->list_head, size_t(p->x + 1) * 2 * 4) == cudaSuccess &&
         cudaMalloc(&d->status, 2 * sizeof(StatusSlot)) == cudaSuccess &&
         cudaMalloc(&d->group_ctr, size_t(g.P_blk) * 4) == cudaSuccess;
  }
  if (ok) {
    StatusSlot init[2];
    std::memset(init, 0, sizeof(init));
    init[0].t_start = init[1].t_start = ~0ULL;
    ok = cudaMemset(d->flags_own, 0, n_own * 4) == cudaSuccess &&
         cudaMemset(d->flags_peer, 0xff, n_peer * 4) == cudaSuccess &&
         (!d->C || cudaMemset(d->C, 0, size_t(g.M) * g.N * 2) == cudaSuccess) &&
         cudaMemcpy(d->tasks, t.dev_tasks.data(), t.dev_tasks.size() * sizeof(Task),
                    cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(d->list_offs, t.list_offs.data(), t.list_offs.size() * 4, cudaMemcpyHostToDevice) ==
             cudaSuccess &&
         cudaMemset(d->list_head, 0, size_t(p->x + 1) * 2 * 4) == cudaSuccess &&
         cudaMemcpy(d->status, init, sizeof(init), cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemset(d->group_ctr, 0, size_t(g.P_blk) * 4) == cudaSuccess;
  }
  p->dev = d;
  if (!ok) {
    cudaGetLastError();
    device_release(p);
    return ENTWINE_ERR_CUDA;
  }
  return ENTWINE_OK;
}

void device_release(Plan* p) {
  DeviceState* d = p->dev;
  if (!d) return;
  if (d->last_stream || d->status_pending) cudaStreamSynchronize(d->last_stream);
  if (d->pipe) {
    DeviceState::HostPipe* hp = d->pipe;
    for (cudaStream_t st : {hp->up, hp->comp, hp->down}) {
      if (st) {
        cudaStreamSynchronize(st);
        cudaStreamDestroy(st);
      }
    }
    for (int i = 0; i < 2; ++i) {
      if (hp->up_done[i]) cudaEventDestroy(hp->up_done[i]);
      if (hp->k_done[i]) cudaEventDestroy(hp->k_done[i]);
      if (hp->d_done[i]) cudaEventDestroy(hp->d_done[i]);
      cudaFree(hp->A[i]);
      cudaFree(hp->B[i]);
      cudaFree(hp->peers[i]);
      cudaFree(hp->out[i]);
      cudaFree(hp->send[i]);
    }
    delete hp;
    d->pipe = nullptr;
  }
  if (d->own_stream) {
    cudaStreamSynchronize(d->own_stream);
    cudaStreamDestroy(d->own_stream);
  }
  if (d->switch_event) cudaEventDestroy(d->switch_event);
  if (!d->user_ws) {
    cudaFree(d->C);
    cudaFree(d->flags_own);
    cudaFree(d->flags_peer);
    cudaFree(d->tasks);
    cudaFree(d->list_offs);
    cudaFree(d->list_head);
    cudaFree(d->status);
    cudaFree(d->group_ctr);
    cudaFree(d->tasks_pull);
    cudaFree(d->list_offs_pull);
    cudaFree(d->ssq_part);
    cudaFree(d->band_ctr);
  }
  cudaFree(d->sA);
  cudaFree(d->sB);
  cudaFree(d->sPeers);
  cudaFree(d->sOut);
  cudaFree(d->sSend);
  cudaGetLastError();
  delete d;
  p->dev = nullptr;
}

// The caller moved the plan to another stream: the new stream waits, on the device, for what the
// old one still has to do for this plan (one workspace: calls of a plan never overlap).
static cudaError_t order_after_last_launch(DeviceState* d, cudaStream_t stream) {
  if (!d->switch_event) {
    cudaError_t e = cudaEventCreateWithFlags(&d->switch_event, cudaEventDisableTiming);
    if (e != cudaSuccess) return e;
  }
  cudaError_t e = cudaEventRecord(d->switch_event, d->last_stream);
  if (e != cudaSuccess) return e;
  return cudaStreamWaitEvent(stream, d->switch_event, 0);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// The register path of the consumer (KParams::reg_a) is a kernel of its own: with its code compiled
// into the same kernel, the TMA-ring consumer measured 4-10 us slower on the benchmark's shapes.
template <int BN, bool PAIR, bool NORM = false, bool PULL = false, bool REG = false>
static int launch_bn(Plan* p, const KParams& kp, const KMaps& maps, int grid, cudaStream_t stream,
                     bool config_only = false) {
  if (!NORM && !PULL && kp.norm) return launch_bn<BN, PAIR, true, false, REG>(p, kp, maps, grid, stream, config_only);
  if (!REG && kp.reg_a) return launch_bn<BN, PAIR, NORM, PULL, true>(p, kp, maps, grid, stream, config_only);
  // per device: the shared-memory opt-in has been set, and how many clusters fit at once (shared by
  // all plans, which may be used from different threads)
  static int max_clusters[64] = {0};
  static bool configured[64] = {false};
  static std::mutex config_mutex;
  int dev = 0;
  CK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return ENTWINE_ERR_RESOURCES;
  auto kern = entwine_fused_kernel<BN, PAIR, NORM, PULL, REG>;
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(unsigned(grid), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = PAIR ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  {
    std::lock_guard<std::mutex> lock(config_mutex);
    if (!configured[dev]) {
      CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
      int per_sm = 0;
      CK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, kSmemBytes));
      if (per_sm < 1) return ENTWINE_ERR_RESOURCES;
      if (PAIR) CK(cudaOccupancyMaxActiveClusters(&max_clusters[dev], kern, &cfg));
      configured[dev] = true;
    }
    clusters = max_clusters[dev];
  }
  // every cluster of the grid must be resident at once: producers and consumers wait on each
  // other inside one launch
  if (PAIR && clusters * 2 < grid) return ENTWINE_ERR_RESOURCES;
  if (config_only) return ENTWINE_OK;
  CK(cudaLaunchKernelEx(&cfg, kern, maps, kp));
  CK(cudaGetLastError());
  return ENTWINE_OK;
}

// Consumer ring geometry and the split of shared memory.  A reduce step moves rs rows of all W
// contributions (at most 16 KiB with geometry 0, 32 KiB with geometry 1), a push step moves as
// many rows of one tile as fit in a slot.  The producer's operand ring gets `stages` stages;
// what remains after the epilogue staging is the co-located consumer ring A.
static int ring_geometry(const Plan* p, KParams* kp, bool reg_a) {
  const Geometry& g = p->g;
  for (int id = 0; id < 2; ++id) {
    const int budget = id == 0 ? 16384 : 32768;
    int rs = 1;
    while (int64_t(g.W) * (rs * 2) * kTile * 2 <= budget && rs * 2 <= kTile) rs *= 2;
    // a slot is as large as the budget even when a reduce step fills less of it (W not a
    // power of two): push steps, most of the traffic, then keep their full size
    int slot_bytes = int(int64_t(g.W) * rs * kTile * 2);
    slot_bytes = std::max((slot_bytes + 1023) / 1024 * 1024, budget);
    int prs = rs;
    while (prs < kTile && int64_t(prs) * 2 * kTile * 2 <= slot_bytes) prs *= 2;
    kp->rs[id] = rs;
    kp->prs[id] = prs;
    kp->slot_bytes[id] = slot_bytes;
  }
  // k-blocks per stage: two where a k-block of both operands is 32 KiB (pair tiles, 128-wide blocks), so
  // that an operand's share of a stage is one 32 KiB TMA box
  const int kblock_bytes = kBM * kBK * 2 + (p->pair ? 128 : g.BN) * kBK * 2;
  int kpb = p->kpb;
  if (kpb <= 0) {
    // (only with the register consumer, which leaves all of shared memory to the operand ring: beside a
    // consumer ring, five single k-blocks in flight measured better than two pairs)
    kpb = (reg_a && kblock_bytes <= 32768 && g.K >= 2 * kBK) ? 2 : 1;
    // a requested number of stages that only fits with single k-blocks gets single k-blocks
    if (kpb == 2 && p->stages > 0 && p->stages * 2 * kblock_bytes + kStagingBytes > kDataBytes) kpb = 1;
  }
  if (kpb > 2 || kpb * kblock_bytes > 65536) return ENTWINE_ERR_INVALID;  // the kernel has loops for 1 and 2
  const int stage_bytes = kpb * kblock_bytes;
  int stages = p->stages;
  if (stages <= 0) {
    // default: as deep an operand ring as leaves two small slots to the co-located consumer ring;
    // shapes whose communication outweighs their tensor work give one stage to that ring
    stages = (kDataBytes - kStagingBytes - (reg_a ? 0 : 2 * kp->slot_bytes[0])) / stage_bytes;
    if (stages > (reg_a ? kMaxStages : 5)) stages = reg_a ? kMaxStages : 5;
    // rough peaks, only to rank the two kinds of work of a shape against each other
    const double t_tc = 2.0 * g.M * g.N * g.K / 1.6e15;
    const double t_hbm = double(g.M) * g.N * 2.0 * (3 * g.W - 1) / g.W / 6.5e12;
    if (!reg_a && p->colocate && t_hbm > 0.5 * t_tc && stages * kpb > 3) stages -= 1;
    // communication-bound shapes (K_local of a few hundred): one more stage goes to the ring
    if (!reg_a && p->colocate && t_hbm > t_tc && stages * kpb > 3) stages -= 1;
    if (stages < 2) stages = 2;
  }
  if (stages < 2 || stages > kMaxStages || stages * stage_bytes + kStagingBytes > kDataBytes) return ENTWINE_ERR_INVALID;
  const int ring_a_off = stages * stage_bytes + kStagingBytes;
  const int ring_a_bytes = kDataBytes - ring_a_off;
  kp->stages = stages;
  kp->kpb = kpb;
  kp->ring_a_off = ring_a_off;
  kp->stage_area = std::min(stages * stage_bytes, kRingBBytes);
  // ring B in the operand stages alone needs room for at least four slots to keep the tail's rate
  kp->early_b = kp->stage_area >= 4 * kp->slot_bytes[1] ? 1 : 0;
  kp->ring_a_bytes = ring_a_bytes;
  kp->ring_a_geom = ring_a_bytes >= 2 * kp->slot_bytes[1] ? 1 : 0;
  // no room for a ring beside the operand stages: the consumer warps of a producer CTA start when
  // its stages are free
  kp->colocate = (p->colocate && (reg_a || ring_a_bytes >= 2 * kp->slot_bytes[0])) ? 1 : 0;
  kp->reg_a = reg_a ? 1 : 0;
  kp->reg_only = (reg_a && !p->consumer_tma) ? 1 : 0;
  return ENTWINE_OK;
}

// Common launch path.  `partial` overrides the workspace in consumer-only mode.
// Arguments of the layer chain (residual add + RMSNorm after the reduction).
struct NormArgs {
  const void* residual;  // [R][N] bf16
  const void* weight;    // [N] bf16
  void* norm_out;        // [R][N] bf16
  float eps;
};

static int launch(Plan* p, int mode, const void* A, const void* B, const void* partial, const void* peers,
                  void* out, void* send, int n_ctas, cudaStream_t stream, const NormArgs* norm = nullptr) {
  if (!p->dev || !p->dev->C || !(p->launched || p->dev->user_ws)) {
    // the first launch allocates the workspace and configures the kernel: not inside a capture
    // (a plan with a caller-provided workspace did both in entwine_plan_set_workspace)
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess) {
      cudaGetLastError();
      return ENTWINE_ERR_CUDA;
    }
    if (cs != cudaStreamCaptureStatusNone) return ENTWINE_ERR_INVALID;
  }
  int rc = ensure_device(p);
  if (rc != ENTWINE_OK) return rc;
  DeviceState* d = p->dev;
  const Geometry& g = p->g;
  if (norm) {
    if (mode != MODE_FUSED || !norm->residual || !norm->weight || !norm->norm_out ||
        !aligned16(norm->residual) || !aligned16(norm->weight) || !aligned16(norm->norm_out) ||
        !(norm->eps >= 0.f))
      return ENTWINE_ERR_INVALID;
    // a CTA that waits for a band cannot drain lists: every list needs a consumer CTA of its own
    if (p->x > p->n_gemm_ctas + p->n_comm_ctas) return ENTWINE_ERR_INVALID;
    if (!d->ssq_part) {
      cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
      if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone)
        return ENTWINE_ERR_INVALID;  // the layer chain's scratch is allocated by an eager call
      if (cudaMalloc(&d->ssq_part, size_t(g.R) * g.nTn * 4) != cudaSuccess ||
          cudaMalloc(&d->band_ctr, size_t(g.rowsT) * 4) != cudaSuccess) {
        cudaGetLastError();
        return ENTWINE_ERR_CUDA;
      }
    }
  }
  if (mode != MODE_COMM_ONLY && (!A || !B || !aligned16(A) || !aligned16(B))) return ENTWINE_ERR_INVALID;
  if (mode != MODE_GEMM_ONLY &&
      (!peers || !out || !send || !aligned16(peers) || !aligned16(out) || !aligned16(send)))
    return ENTWINE_ERR_INVALID;
  if (partial && !aligned16(partial)) return ENTWINE_ERR_INVALID;

  // A launch may be captured into a CUDA graph once the plan has run eagerly (nothing is
  // allocated or configured during a capture).  From then on every launch of the plan, replayed
  // or not, starts with the reset kernel.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  CK(cudaStreamIsCapturing(stream, &cap));
  const bool capturing = cap != cudaStreamCaptureStatusNone;
  if (capturing) {
    if (!(p->launched || d->user_ws) || (norm && !d->ssq_part)) return ENTWINE_ERR_INVALID;
    d->captured = true;
  }

  // serialise with the plan's previous launch if the caller switched streams (a graph's
  // launches are ordered by whoever replays it)
  if (d->last_stream != stream && p->launched && !capturing) CK(order_after_last_launch(d, stream));

  if (mode != MODE_COMM_ONLY) {
    d->epoch += 1;
    if (d->epoch >= 0xfffffff0u) {  // epoch wrap: start over with cleared flags
      CK(cudaMemsetAsync(d->flags_own, 0, size_t(g.W) * g.Q * 4, stream));
      d->epoch = 1;
    }
    if (p->poison) CK(cudaMemsetAsync(d->C, 0xff, size_t(g.M) * g.N * 2, stream));
    // coarse release only: start the group counts from zero whatever an earlier launch left
    if (p->release_group != 1) CK(cudaMemsetAsync(d->group_ctr, 0, size_t(g.P_blk) * 4, stream));
  }
  if (d->withheld != p->withhold_peer) {
    // host-side fault injection: a peer flag that is never published
    if (d->withheld >= 0) {
      int64_t w = d->withheld >> 32, t = d->withheld & 0xffffffffLL;
      int64_t q = w < p->rank ? w : w - 1;
      CK(cudaMemsetAsync(d->flags_peer + q * g.Q + t, 0xff, 4, stream));
    }
    if (p->withhold_peer >= 0) {
      int64_t w = p->withhold_peer >> 32, t = p->withhold_peer & 0xffffffffLL;
      int64_t q = w < p->rank ? w : w - 1;
      CK(cudaMemsetAsync(d->flags_peer + q * g.Q + t, 0, 4, stream));
    }
    d->withheld = p->withhold_peer;
  }
  if (d->captured) {
    const int n_flags = g.W * int(g.Q), n_heads = 2 * (p->x + 1);
    const int blocks = std::min(64, (std::max(n_flags, n_heads) + 1023) / 1024);
    entwine_reset_kernel<<<blocks, 1024, 0, stream>>>(d->flags_own, n_flags, d->list_head, n_heads, d->status);
    CK(cudaGetLastError());
  }

  KParams kp;
  std::memset(&kp, 0, sizeof(kp));
  kp.M = int(g.M); kp.N = int(g.N); kp.K = int(g.K); kp.W = g.W; kp.r = p->rank; kp.order = p->order;
  kp.rowsT = g.rowsT; kp.nBn = g.nBn; kp.nTn = g.nTn; kp.Lb = g.Lb; kp.P_blk = g.P_blk; kp.Q = g.Q;
  kp.cpb = g.cpb; kp.R = g.R;
  kp.x = p->x;
  kp.mode = mode;
  kp.help = (p->tail_help || p->lists_opt > 0) ? 1 : 0;  // shared lists need every CTA to scan them
  kp.skip_wait = (mode == MODE_COMM_ONLY) ? 1 : 0;
  kp.release_group = p->release_group;
  kp.group_ctr = d->group_ctr;
  kp.norm = norm ? 1 : 0;
  if (norm) {
    kp.eps = norm->eps;
    kp.residual = static_cast<const __nv_bfloat16*>(norm->residual);
    kp.weight = static_cast<const __nv_bfloat16*>(norm->weight);
    kp.norm_out = static_cast<__nv_bfloat16*>(norm->norm_out);
    kp.ssq_part = d->ssq_part;
    kp.band_ctr = d->band_ctr;
    CK(cudaMemsetAsync(d->band_ctr, 0, size_t(g.rowsT) * 4, stream));
  }
  kp.claim = claim_size(g.W);
  kp.epoch = d->epoch;
  // the launch number is committed only when the launch has been enqueued
  const unsigned seq_next = d->seq + 1;
  kp.seq = seq_next;
  // two sets of head counters and status slots, used alternately; a launch rewinds the other set
  kp.list_head = d->list_head + size_t(seq_next & 1) * (p->x + 1);
  kp.list_head_next = d->list_head + size_t((seq_next & 1) ^ 1) * (p->x + 1);
  kp.status_next = &d->status[(seq_next & 1) ^ 1];
  kp.wait_budget_ns = (unsigned long long)p->wait_budget_ns;
  rc = ring_geometry(p, &kp, p->reg_consumer != 0 || p->consumer_tma == 0);
  if (rc != ENTWINE_OK) return rc;
  kp.prefetch = p->prefetch;
  kp.l2_hints = p->l2_hints;
  kp.out = static_cast<__nv_bfloat16*>(out);
  kp.cws = (mode == MODE_COMM_ONLY && partial) ? static_cast<const __nv_bfloat16*>(partial) : d->C;
  kp.cws_out = d->C;
  kp.peers = static_cast<const __nv_bfloat16*>(peers);
  kp.send = static_cast<__nv_bfloat16*>(send);
  kp.flags_own = d->flags_own;
  kp.flags_peer = d->flags_peer;
  kp.tasks = d->tasks;
  kp.list_offs = d->list_offs;
  kp.status = d->status;

  int grid;
  const bool pair = p->pair;
  if (mode == MODE_FUSED) {
    kp.n_ded = p->n_comm_ctas;
    kp.G = p->n_gemm_ctas;
    grid = p->n_comm_ctas + p->n_gemm_ctas;
  } else if (mode == MODE_GEMM_ONLY) {
    kp.n_ded = 0;
    kp.G = pair ? (p->num_sms & ~1) : p->num_sms;
    grid = kp.G;
  } else {
    grid = (n_ctas <= 0) ? p->num_sms : n_ctas;
    if (grid > p->num_sms) return ENTWINE_ERR_INVALID;
    kp.n_ded = grid;
    kp.G = 0;
    // with fewer CTAs than lists the CTAs must visit every list
    if (grid < p->x) kp.help = 1;
  }
  // a cluster launch needs whole clusters: an odd grid gets one more consumer CTA, which owns
  // no list and only helps
  if (pair && (grid & 1)) {
    if (grid + 1 > p->num_sms) grid -= 1, kp.n_ded -= 1;
    else grid += 1, kp.n_ded += 1;
    if (kp.n_ded < p->x) kp.help = 1;
  }
  kp.split = (mode != MODE_COMM_ONLY) ? split_last_wave(p, kp.G) : 0;

  KMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  const void* c_src = (mode == MODE_COMM_ONLY && partial) ? partial : d->C;
  // maps of buffers a mode does not touch point at the workspace so that they stay encodable
  const void* a_p = (mode != MODE_COMM_ONLY) ? A : d->C;
  const void* b_p = (mode != MODE_COMM_ONLY) ? B : d->C;
  const bool comm = mode != MODE_GEMM_ONLY;
  bool ok = (mode != MODE_COMM_ONLY)
                ? make_operand_maps(&maps, a_p, b_p, g, pair ? 128 : g.BN, kp.kpb, p->lda, p->ldb, kp.b_kn = p->b_kn, &kp.k3d)
                : (make_map(&maps.a, a_p, g.M, g.N, kBK, kBM, true) && make_map(&maps.b, b_p, g.M, g.N, kBK, kBM, true));
  // rows of one peer's plane: all M, or (compact staging of the host-buffer calls) partition r's R
  const int64_t prows = p->peers_compact ? g.R : g.M;
  kp.peer_rows = int(prows);
  kp.peer_row0 = p->peers_compact ? int(p->rank * g.R) : 0;
  ok = ok && make_map(&maps.p_pf, comm ? peers : d->C, comm ? int64_t(g.W - 1) * prows : g.M, g.N, kTile, kTile, false);
  for (int id = 0; ok && id < 2; ++id) {
    const int rs = kp.rs[id];
    const int prs = kp.prs[id];
    ok = make_map(&maps.c_ld[id], c_src, g.M, g.N, kTile, rs, false) &&
         make_map(&maps.c_push[id], c_src, g.M, g.N, kTile, prs, false) &&
         (comm ? make_map3(&maps.p_ld[id], peers, g.W - 1, prows, g.N, kTile, rs, g.W - 1)
               : make_map3(&maps.p_ld[id], d->C, 1, g.M, g.N, kTile, rs, 1)) &&
         make_map(&maps.send_st[id], comm ? send : d->C, comm ? int64_t(g.W - 1) * g.R : g.M, g.N, kTile, prs, false) &&
         make_map(&maps.res_ld[id], norm ? norm->residual : d->C, norm ? g.R : g.M, g.N, kTile, prs, false) &&
         make_map(&maps.h_ld[id], norm ? out : d->C, norm ? g.R : g.M, g.N, kTile, prs, false);
  }
  if (!ok) return ENTWINE_ERR_CUDA;
  if (pair) rc = launch_bn<256, true>(p, kp, maps, grid, stream);
  else if (g.BN == 256) rc = launch_bn<256, false>(p, kp, maps, grid, stream);
  else rc = launch_bn<128, false>(p, kp, maps, grid, stream);
  if (rc != ENTWINE_OK) return rc;
  d->seq = seq_next;
  p->launched = true;
  if (!capturing) d->last_stream = stream;
  d->status_pending = true;
  return ENTWINE_OK;
}


// ------------------------------------------------------------------------------------------
// Pull mode: the call of one rank of W ranks that run on GPUs of their own (Sec. 4.2, Sec. 4.1's
// symmetric heap).  Every rank owns one segment of a heap that all ranks map at the same
// stride; a segment holds two partial-output buffers [M][N] (used alternately, by the parity
// of the call number) and the rank's flag array [W sources][Q].  The producer stores its
// partial into its own segment and writes each tile's flag into the flag array of the tile's
// destination; the reducers poll their local flags and read the peers' rows of their own
// partition straight out of the peers' segments.  Nothing is pushed.
// ------------------------------------------------------------------------------------------
static int64_t heap_flags_offset(const Geometry& g) { return 2 * g.M * g.N * 2; }
static int64_t heap_segment_bytes(const Geometry& g) {
  return heap_flags_offset(g) + ((int64_t(g.W) * g.Q * 4 + 255) / 256) * 256;
}

static int launch_pull(Plan* p, const void* A, const void* B, void* heap, int64_t stride, uint32_t epoch,
                       int produce_only, void* out, cudaStream_t stream) {
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) {
    cudaGetLastError();
    return ENTWINE_ERR_CUDA;
  }
  if (cap != cudaStreamCaptureStatusNone) return ENTWINE_ERR_INVALID;  // the epoch is a launch parameter
  int rc = ensure_device(p, /*need_c=*/false);  // the partial output lives in the heap
  if (rc != ENTWINE_OK) return rc;
  DeviceState* d = p->dev;
  const Geometry& g = p->g;
  const HostTables& t = p->tables;
  if (!A || !B || !heap || !aligned16(A) || !aligned16(B) || (!produce_only && (!out || !aligned16(out))))
    return ENTWINE_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(heap) & 255) || (stride & 255) || stride < heap_segment_bytes(g) ||
      epoch == 0 || epoch >= 0xfffffff0u)
    return ENTWINE_ERR_INVALID;
  if (p->release_group != 1 || p->poison || p->withhold_peer >= 0) return ENTWINE_ERR_INVALID;
  if (!d->tasks_pull) {
    bool ok = cudaMalloc(&d->tasks_pull, std::max<size_t>(1, t.pull_tasks.size()) * sizeof(Task)) == cudaSuccess &&
              cudaMalloc(&d->list_offs_pull, t.pull_list_offs.size() * 4) == cudaSuccess &&
              cudaMemcpy(d->tasks_pull, t.pull_tasks.data(), t.pull_tasks.size() * sizeof(Task),
                         cudaMemcpyHostToDevice) == cudaSuccess &&
              cudaMemcpy(d->list_offs_pull, t.pull_list_offs.data(), t.pull_list_offs.size() * 4,
                         cudaMemcpyHostToDevice) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      cudaFree(d->tasks_pull);
      cudaFree(d->list_offs_pull);
      d->tasks_pull = nullptr;
      d->list_offs_pull = nullptr;
      return ENTWINE_ERR_CUDA;
    }
  }
  if (d->last_stream != stream && p->launched) CK(order_after_last_launch(d, stream));
  if (d->captured) {
    // (the plan's own flags are not used here; heads and status are)
    const int n_heads = 2 * (p->x + 1);
    entwine_reset_kernel<<<1, 1024, 0, stream>>>(d->flags_own, 0, d->list_head, n_heads, d->status);
    CK(cudaGetLastError());
  }

  char* seg0 = static_cast<char*>(heap);
  char* own_seg = seg0 + int64_t(p->rank) * stride;
  const int64_t buf_off = int64_t(epoch & 1u) * g.M * g.N * 2;

  KParams kp;
  std::memset(&kp, 0, sizeof(kp));
  kp.M = int(g.M); kp.N = int(g.N); kp.K = int(g.K); kp.W = g.W; kp.r = p->rank; kp.order = p->order;
  kp.rowsT = g.rowsT; kp.nBn = g.nBn; kp.nTn = g.nTn; kp.Lb = g.Lb; kp.P_blk = g.P_blk; kp.Q = g.Q;
  kp.cpb = g.cpb; kp.R = g.R;
  kp.x = p->x;
  kp.mode = produce_only ? MODE_GEMM_ONLY : MODE_FUSED;
  kp.help = (p->tail_help || p->lists_opt > 0) ? 1 : 0;
  kp.release_group = 1;
  kp.claim = claim_size(g.W);
  kp.epoch = epoch;
  const unsigned seq_next = d->seq + 1;
  kp.seq = seq_next;
  kp.list_head = d->list_head + size_t(seq_next & 1) * (p->x + 1);
  kp.list_head_next = d->list_head + size_t((seq_next & 1) ^ 1) * (p->x + 1);
  kp.status_next = &d->status[(seq_next & 1) ^ 1];
  kp.wait_budget_ns = (unsigned long long)p->wait_budget_ns;
  rc = ring_geometry(p, &kp, p->reg_consumer != 0 || p->consumer_tma == 0);
  if (rc != ENTWINE_OK) return rc;
  kp.prefetch = 0;
  kp.l2_hints = p->l2_hints;
  kp.out = static_cast<__nv_bfloat16*>(out);
  kp.cws = reinterpret_cast<const __nv_bfloat16*>(own_seg + buf_off);
  kp.cws_out = reinterpret_cast<__nv_bfloat16*>(own_seg + buf_off);
  kp.heap_buf_off = buf_off;
  kp.heap = seg0;
  kp.heap_stride = stride;
  kp.heap_flags_off = heap_flags_offset(g);
  kp.flags_own = reinterpret_cast<unsigned*>(own_seg + kp.heap_flags_off);
  kp.flags_peer = kp.flags_own;
  kp.tasks = d->tasks_pull;
  kp.list_offs = d->list_offs_pull;
  kp.status = d->status;

  int grid;
  const bool pair = p->pair;
  if (!produce_only) {
    kp.n_ded = p->n_comm_ctas;
    kp.G = p->n_gemm_ctas;
    grid = p->n_comm_ctas + p->n_gemm_ctas;
  } else {
    kp.n_ded = 0;
    kp.G = pair ? (p->num_sms & ~1) : p->num_sms;
    grid = kp.G;
  }
  if (pair && (grid & 1)) {
    if (grid + 1 > p->num_sms) grid -= 1, kp.n_ded -= 1;
    else grid += 1, kp.n_ded += 1;
    if (kp.n_ded < p->x) kp.help = 1;
  }
  kp.split = split_last_wave(p, kp.G);

  KMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  void* own_buf = own_seg + buf_off;
  const int r = p->rank, W = g.W;
  bool ok = make_operand_maps(&maps, A, B, g, pair ? 128 : g.BN, kp.kpb, p->lda, p->ldb, kp.b_kn = p->b_kn, &kp.k3d) &&
            make_map(&maps.p_pf, own_buf, g.M, g.N, kTile, kTile, false);
  for (int id = 0; ok && id < 2; ++id) {
    const int rs = kp.rs[id];
    const int prs = kp.prs[id];
    // the ranks below this one start at rank 0's segment, the ranks above it at rank r+1's; an
    // empty group gets a map of this rank's buffer, which no load uses
    const void* lo = r > 0 ? seg0 + buf_off : own_buf;
    const void* hi = r < W - 1 ? seg0 + int64_t(r + 1) * stride + buf_off : own_buf;
    ok = make_map(&maps.c_ld[id], own_buf, g.M, g.N, kTile, rs, false) &&
         make_map(&maps.c_push[id], own_buf, g.M, g.N, kTile, prs, false) &&
         make_map3(&maps.p_ld[id], lo, std::max(r, 1), g.M, g.N, kTile, rs, std::max(r, 1), stride) &&
         make_map3(&maps.p_hi[id], hi, std::max(W - 1 - r, 1), g.M, g.N, kTile, rs, std::max(W - 1 - r, 1),
                   stride) &&
         make_map(&maps.send_st[id], own_buf, g.M, g.N, kTile, prs, false) &&
         make_map(&maps.res_ld[id], own_buf, g.M, g.N, kTile, prs, false) &&
         make_map(&maps.h_ld[id], own_buf, g.M, g.N, kTile, prs, false);
  }
  if (!ok) return ENTWINE_ERR_CUDA;
  if (pair) rc = launch_bn<256, true, false, true>(p, kp, maps, grid, stream);
  else if (g.BN == 256) rc = launch_bn<256, false, false, true>(p, kp, maps, grid, stream);
  else rc = launch_bn<128, false, false, true>(p, kp, maps, grid, stream);
  if (rc != ENTWINE_OK) return rc;
  d->seq = seq_next;
  p->launched = true;
  d->last_stream = stream;
  d->status_pending = true;
  return ENTWINE_OK;
}

}  // namespace entwine

using namespace entwine;

extern "C" {

int entwine_gemm_rs(entwine_plan_t plan, const void* A, const void* B, const void* peer_partials,
                    void* out_shard, void* send_bufs, void* stream) {
  if (!plan) return ENTWINE_ERR_INVALID;
  return launch(plan, MODE_FUSED, A, B, nullptr, peer_partials, out_shard, send_bufs, 0,
                static_cast<cudaStream_t>(stream));
}

int entwine_gemm_rs_norm(entwine_plan_t plan, const void* A, const void* B, const void* peer_partials,
                         const void* residual, const void* weight, float eps, void* hidden_out,
                         void* norm_out, void* send_bufs, void* stream) {
  if (!plan) return ENTWINE_ERR_INVALID;
  NormArgs na;
  na.residual = residual;
  na.weight = weight;
  na.norm_out = norm_out;
  na.eps = eps;
  return launch(plan, MODE_FUSED, A, B, nullptr, peer_partials, hidden_out, send_bufs, 0,
                static_cast<cudaStream_t>(stream), &na);
}

int entwine_gemm_only(entwine_plan_t plan, const void* A, const void* B, void* stream) {
  if (!plan) return ENTWINE_ERR_INVALID;
  return launch(plan, MODE_GEMM_ONLY, A, B, nullptr, nullptr, nullptr, nullptr, 0,
                static_cast<cudaStream_t>(stream));
}

int entwine_heap_bytes(entwine_plan_t plan, int64_t* segment_bytes, int64_t* flags_offset) {
  if (!plan || !segment_bytes) return ENTWINE_ERR_INVALID;
  *segment_bytes = heap_segment_bytes(plan->g);
  if (flags_offset) *flags_offset = heap_flags_offset(plan->g);
  return ENTWINE_OK;
}

int entwine_gemm_rs_pull(entwine_plan_t plan, const void* A, const void* B, void* heap, int64_t heap_stride,
                         uint32_t epoch, int produce_only, void* out_shard, void* stream) {
  if (!plan) return ENTWINE_ERR_INVALID;
  return launch_pull(plan, A, B, heap, heap_stride, epoch, produce_only, out_shard,
                     static_cast<cudaStream_t>(stream));
}

int entwine_comm_only(entwine_plan_t plan, const void* partial, const void* peer_partials, void* out_shard,
                      void* send_bufs, int n_ctas, void* stream) {
  if (!plan || n_ctas < 0) return ENTWINE_ERR_INVALID;
  return launch(plan, MODE_COMM_ONLY, nullptr, nullptr, partial, peer_partials, out_shard, send_bufs, n_ctas,
                static_cast<cudaStream_t>(stream));
}

int entwine_read_partial(entwine_plan_t plan, void* dst, void* stream) {
  if (!plan || !dst) return ENTWINE_ERR_INVALID;
  int rc = ensure_device(plan);
  if (rc != ENTWINE_OK) return rc;
  const Geometry& g = plan->g;
  CK(cudaMemcpyAsync(dst, plan->dev->C, size_t(g.M) * g.N * 2, cudaMemcpyDeviceToDevice,
                     static_cast<cudaStream_t>(stream)));
  return ENTWINE_OK;
}

int entwine_last_status(entwine_plan_t plan, int64_t out[8]) {
  if (!plan || !out) return ENTWINE_ERR_INVALID;
  for (int i = 0; i < 8; ++i) out[i] = 0;
  DeviceState* d = plan->dev;
  if (!d || !plan->launched) return ENTWINE_OK;
  CK(cudaStreamSynchronize(d->last_stream));
  StatusSlot s;
  CK(cudaMemcpy(&s, &d->status[d->seq & 1], sizeof(s), cudaMemcpyDeviceToHost));
  d->status_pending = false;
  const int code = int(s.code_cta_task & 0xff);
  out[0] = code ? -code : 0;
  out[1] = int64_t((s.code_cta_task >> 8) & 0xffffff);
  out[2] = int64_t(int32_t(s.code_cta_task >> 32));
  out[3] = int64_t(s.flags_published);
  out[4] = int64_t(s.tiles_reduced);
  out[5] = int64_t(s.tiles_pushed);
  out[6] = (s.t_gemm_end > s.t_start) ? int64_t(s.t_gemm_end - s.t_start) : 0;
  out[7] = (s.t_end > s.t_start) ? int64_t(s.t_end - s.t_start) : 0;
  d->last_clock = s.clock;
  if (code) {
    // the launch gave up part-way: rewind what its last CTA would have rewound
    cudaMemset(d->list_head, 0, size_t(plan->x + 1) * 2 * 4);
    StatusSlot init[2];
    std::memset(init, 0, sizeof(init));
    init[0].t_start = init[1].t_start = ~0ULL;
    cudaMemcpy(d->status, init, sizeof(init), cudaMemcpyHostToDevice);
  }
  return int(out[0]);
}

int entwine_plan_workspace_bytes(entwine_plan_t plan, size_t* bytes) {
  if (!plan || !bytes) return ENTWINE_ERR_INVALID;
  *bytes = workspace_layout(plan).total;
  return ENTWINE_OK;
}

int entwine_plan_set_workspace(entwine_plan_t plan, void* workspace, size_t bytes) {
  if (!plan || plan->launched) return ENTWINE_ERR_INVALID;
  Plan* p = plan;
  if (p->dev) device_release(p);
  p->ws_ptr = nullptr;
  p->ws_bytes = 0;
  if (!workspace) return ENTWINE_OK;  // back to memory of the library's own
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) || bytes < workspace_layout(p).total) return ENTWINE_ERR_INVALID;
  p->ws_ptr = workspace;
  p->ws_bytes = bytes;
  int rc = ensure_device(p);  // carves the block and fills tables, flags and status (synchronous copies)
  if (rc == ENTWINE_OK) {
    // everything else a first launch would do once per device: the kernels' shared-memory opt-in
    // and the residency check, for every variant this plan can launch
    KParams kp;
    std::memset(&kp, 0, sizeof(kp));
    KMaps maps;
    std::memset(&maps, 0, sizeof(maps));
    const int grid = std::min(p->num_sms, p->n_gemm_ctas + p->n_comm_ctas);
    for (int v6 = 0; rc == ENTWINE_OK && v6 < 6; ++v6) {
      const int variant = v6 % 3;
      kp.reg_a = v6 / 3;  // both consumer kernels: options may still change which one a call launches
      kp.norm = variant == 1;
      if (variant == 2) {
        if (p->pair) rc = launch_bn<256, true, false, true>(p, kp, maps, grid, nullptr, true);
        else if (p->g.BN == 256) rc = launch_bn<256, false, false, true>(p, kp, maps, grid, nullptr, true);
        else rc = launch_bn<128, false, false, true>(p, kp, maps, grid, nullptr, true);
      } else {
        if (p->pair) rc = launch_bn<256, true>(p, kp, maps, grid, nullptr, true);
        else if (p->g.BN == 256) rc = launch_bn<256, false>(p, kp, maps, grid, nullptr, true);
        else rc = launch_bn<128, false>(p, kp, maps, grid, nullptr, true);
      }
    }
  }
  if (rc != ENTWINE_OK) {
    if (p->dev) device_release(p);
    p->ws_ptr = nullptr;
    p->ws_bytes = 0;
  }
  return rc;
}

int entwine_last_sm_clock(entwine_plan_t plan, int64_t out[2]) {
  if (!plan || !out) return ENTWINE_ERR_INVALID;
  out[0] = out[1] = 0;
  if (!plan->dev) return ENTWINE_OK;
  out[0] = int64_t(plan->dev->last_clock >> 32);
  out[1] = int64_t(plan->dev->last_clock & 0xffffffffULL);
  return ENTWINE_OK;
}

int entwine_gemm_rs_host(entwine_plan_t plan, const void* A, const void* B, const void* peer_partials,
                         void* out_shard, void* send_bufs) {
  if (!plan || !A || !B || !peer_partials || !out_shard || !send_bufs) return ENTWINE_ERR_INVALID;
  int rc = ensure_device(plan);
  if (rc != ENTWINE_OK) return rc;
  DeviceState* d = plan->dev;
  const Geometry& g = plan->g;
  const size_t szA = size_t(g.M) * g.K * 2, szB = size_t(g.N) * g.K * 2;
  // staging of the incoming partials is compact: [W-1][R][N], the rows of partition r that the call reads
  const size_t szP = size_t(g.W - 1) * g.R * g.N * 2, szO = size_t(g.R) * g.N * 2;
  const size_t szS = size_t(g.W - 1) * g.R * g.N * 2;
  if (!d->own_stream) {
    CK(cudaStreamCreateWithFlags(&d->own_stream, cudaStreamNonBlocking));
    bool ok = cudaMalloc(&d->sA, szA) == cudaSuccess && cudaMalloc(&d->sB, szB) == cudaSuccess &&
              cudaMalloc(&d->sPeers, szP) == cudaSuccess && cudaMalloc(&d->sOut, szO) == cudaSuccess &&
              cudaMalloc(&d->sSend, szS) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      return ENTWINE_ERR_CUDA;
    }
  }
  cudaStream_t s = d->own_stream;
  CK(cudaMemcpyAsync(d->sA, A, szA, cudaMemcpyHostToDevice, s));
  CK(cudaMemcpyAsync(d->sB, B, szB, cudaMemcpyHostToDevice, s));
  // only the rows of partition r of every incoming partial are consumed
  const size_t part = size_t(g.R) * g.N * 2, full = size_t(g.M) * g.N * 2;
  for (int q = 0; q < g.W - 1; ++q) {
    const size_t off = size_t(q) * full + size_t(plan->rank) * part;
    CK(cudaMemcpyAsync(reinterpret_cast<char*>(d->sPeers) + size_t(q) * part, static_cast<const char*>(peer_partials) + off,
                       part, cudaMemcpyHostToDevice, s));
  }
  {
    // the staging copies are contiguous whatever the leading dimensions of device operands are
    const int64_t lda = plan->lda, ldb = plan->ldb;
    plan->lda = plan->ldb = 0;
    plan->peers_compact = 1;
    rc = launch(plan, MODE_FUSED, d->sA, d->sB, nullptr, d->sPeers, d->sOut, d->sSend, 0, s);
    plan->peers_compact = 0;
    plan->lda = lda;
    plan->ldb = ldb;
  }
  if (rc != ENTWINE_OK) return rc;
  CK(cudaMemcpyAsync(out_shard, d->sOut, szO, cudaMemcpyDeviceToHost, s));
  CK(cudaMemcpyAsync(send_bufs, d->sSend, szS, cudaMemcpyDeviceToHost, s));
  CK(cudaStreamSynchronize(s));
  int64_t stw[8];
  return entwine_last_status(plan, stw);
}

int entwine_gemm_rs_host_begin(entwine_plan_t plan, const void* A, const void* B, const void* peer_partials,
                               void* out_shard, void* send_bufs) {
  if (!plan || !A || !B || !peer_partials || !out_shard || !send_bufs) return ENTWINE_ERR_INVALID;
  int rc = ensure_device(plan);
  if (rc != ENTWINE_OK) return rc;
  DeviceState* d = plan->dev;
  const Geometry& g = plan->g;
  const size_t szA = size_t(g.M) * g.K * 2, szB = size_t(g.N) * g.K * 2;
  // staging of the incoming partials is compact: [W-1][R][N], the rows of partition r that the call reads
  const size_t szP = size_t(g.W - 1) * g.R * g.N * 2, szO = size_t(g.R) * g.N * 2;
  const size_t szS = size_t(g.W - 1) * g.R * g.N * 2;
  if (!d->pipe) {
    DeviceState::HostPipe* hp = new DeviceState::HostPipe();
    d->pipe = hp;  // released with the plan, whatever was allocated
    bool ok = cudaStreamCreateWithFlags(&hp->up, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp->comp, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp->down, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < 2; ++i) {
      ok = cudaEventCreateWithFlags(&hp->up_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp->k_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp->d_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaMalloc(&hp->A[i], szA) == cudaSuccess && cudaMalloc(&hp->B[i], szB) == cudaSuccess &&
           cudaMalloc(&hp->peers[i], szP) == cudaSuccess && cudaMalloc(&hp->out[i], szO) == cudaSuccess &&
           cudaMalloc(&hp->send[i], szS) == cudaSuccess;
    }
    if (!ok) {
      cudaGetLastError();
      return ENTWINE_ERR_CUDA;
    }
  }
  DeviceState::HostPipe* hp = d->pipe;
  if (!hp->send[1]) return ENTWINE_ERR_CUDA;             // an earlier set-up failed part-way
  if (hp->issued - hp->waited >= 2) return ENTWINE_ERR_INVALID;  // both staging sets are in use
  const int s = int(hp->issued & 1);
  // copies up: after the kernel that last read this staging set
  CK(cudaStreamWaitEvent(hp->up, hp->k_done[s], 0));
  CK(cudaMemcpyAsync(hp->A[s], A, szA, cudaMemcpyHostToDevice, hp->up));
  CK(cudaMemcpyAsync(hp->B[s], B, szB, cudaMemcpyHostToDevice, hp->up));
  const size_t part = size_t(g.R) * g.N * 2, full = size_t(g.M) * g.N * 2;
  for (int q = 0; q < g.W - 1; ++q) {
    const size_t off = size_t(q) * full + size_t(plan->rank) * part;
    CK(cudaMemcpyAsync(reinterpret_cast<char*>(hp->peers[s]) + size_t(q) * part, static_cast<const char*>(peer_partials) + off,
                       part, cudaMemcpyHostToDevice, hp->up));
  }
  CK(cudaEventRecord(hp->up_done[s], hp->up));
  // the kernel: after its inputs are up and the copies down that last read this set's results
  CK(cudaStreamWaitEvent(hp->comp, hp->up_done[s], 0));
  CK(cudaStreamWaitEvent(hp->comp, hp->d_done[s], 0));
  {
    const int64_t lda = plan->lda, ldb = plan->ldb;
    plan->lda = plan->ldb = 0;
    plan->peers_compact = 1;
    rc = launch(plan, MODE_FUSED, hp->A[s], hp->B[s], nullptr, hp->peers[s], hp->out[s], hp->send[s], 0, hp->comp);
    plan->peers_compact = 0;
    plan->lda = lda;
    plan->ldb = ldb;
  }
  if (rc != ENTWINE_OK) return rc;
  CK(cudaEventRecord(hp->k_done[s], hp->comp));
  CK(cudaStreamWaitEvent(hp->down, hp->k_done[s], 0));
  CK(cudaMemcpyAsync(out_shard, hp->out[s], szO, cudaMemcpyDeviceToHost, hp->down));
  CK(cudaMemcpyAsync(send_bufs, hp->send[s], szS, cudaMemcpyDeviceToHost, hp->down));
  CK(cudaEventRecord(hp->d_done[s], hp->down));
  hp->issued += 1;
  return ENTWINE_OK;
}

int entwine_gemm_rs_host_wait(entwine_plan_t plan) {
  if (!plan) return ENTWINE_ERR_INVALID;
  DeviceState* d = plan->dev;
  if (!d || !d->pipe || d->pipe->waited == d->pipe->issued) return ENTWINE_OK;
  DeviceState::HostPipe* hp = d->pipe;
  CK(cudaEventSynchronize(hp->d_done[hp->waited & 1]));
  hp->waited += 1;
  return ENTWINE_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// entwine_gemm_rs_static: the fused call for callers that must not allocate
// ------------------------------------------------------------------------------------------
namespace entwine {

// Scratch of the no-allocation entry point.  It lives in the library image: every device that
// loads the library holds these 9 MiB until the process exits.  The first kStaticPartialMax
// bytes hold the partial output C[M,N]; the rest holds the status block, the completion
// counter, the list heads and offsets, the flag arrays and the task table.
constexpr size_t kStaticPartialMax = size_t(8) << 20;
constexpr size_t kStaticControlMax = size_t(1) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticPartialMax + kStaticControlMax];

// Device address of g_static_scratch per device.  In host code the array's name is only a
// stand-in for the symbol; the address a kernel can use comes from cudaGetSymbolAddress.
constexpr int kMaxDevices = 64;
static unsigned char* g_static_scratch_addr[kMaxDevices] = {nullptr};

}  // namespace entwine

extern "C" int entwine_gemm_rs_static(entwine_plan_t plan, const void* A, const void* B,
                                      const void* peer_partials, void* out_shard, void* send_bufs,
                                      void* stream_v, int64_t* status_out) {
  using namespace entwine;
  if (!plan || !A || !B || !peer_partials || !out_shard || !send_bufs) return ENTWINE_ERR_INVALID;
  if (!aligned16(A) || !aligned16(B) || !aligned16(peer_partials) || !aligned16(out_shard) ||
      !aligned16(send_bufs))
    return ENTWINE_ERR_INVALID;
  Plan* p = plan;
  const Geometry& g = p->g;
  const HostTables& t = p->tables;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  // options this entry point does not implement are refused, not ignored
  if (p->release_group != 1 || p->withhold_peer >= 0) return ENTWINE_ERR_INVALID;
  {
    // every call uploads the plan's tables from the plan's host vectors: captured into a graph,
    // those copies would keep host addresses that a later option change frees
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess) {
      cudaGetLastError();
      return ENTWINE_ERR_CUDA;
    }
    if (cs != cudaStreamCaptureStatusNone) return ENTWINE_ERR_INVALID;
  }

  // ---- sizes against the static maximum ----
  const size_t c_bytes = size_t(g.M) * g.N * 2;
  const size_t n_own = size_t(g.W) * g.Q, n_peer = size_t(g.W - 1) * g.Q;
  const size_t off_status = 0;
  const size_t off_done = off_status + align256(2 * sizeof(StatusSlot));
  const size_t off_heads = off_done + 256;
  const size_t off_offs = off_heads + align256(size_t(p->x) * 4);
  const size_t off_fown = off_offs + align256(t.list_offs.size() * 4);
  const size_t off_fpeer = off_fown + align256(n_own * 4);
  const size_t off_tasks = off_fpeer + align256(n_peer * 4);
  const size_t ctrl_bytes = off_tasks + align256(t.dev_tasks.size() * sizeof(Task));
  if (c_bytes > kStaticPartialMax || ctrl_bytes > kStaticControlMax) return ENTWINE_ERR_TOO_LARGE;

  // ---- once per device: the device address of the scratch symbol ----
  int dev = 0;
  CK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ENTWINE_ERR_RESOURCES;
  if (!g_static_scratch_addr[dev]) {
    int major = 0, sms = 0;
    CK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (major != 10) return ENTWINE_ERR_RESOURCES;
    void* addr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&addr, g_static_scratch);
    if (e != cudaSuccess || !addr) {
      cudaGetLastError();
      return ENTWINE_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = static_cast<unsigned char*>(addr);
  }
  {
    int sms = 0;
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (p->num_sms > sms) return ENTWINE_ERR_RESOURCES;
  }
  unsigned char* base = g_static_scratch_addr[dev];
  unsigned char* ctrl = base + kStaticPartialMax;

  // ---- the array keeps the previous call's contents: reset what must start clean ----
  static const StatusSlot kInit[2] = {{0, 0, 0, 0, ~0ULL, 0, 0, 0}, {0, 0, 0, 0, ~0ULL, 0, 0, 0}};
  CK(cudaMemsetAsync(ctrl, 0, off_fpeer, stream));                      // status .. own flags
  CK(cudaMemcpyAsync(ctrl + off_status, kInit, sizeof(kInit), cudaMemcpyHostToDevice, stream));
  CK(cudaMemsetAsync(ctrl + off_fpeer, 0xff, n_peer * 4, stream));      // peers: pre-published
  CK(cudaMemcpyAsync(ctrl + off_offs, t.list_offs.data(), t.list_offs.size() * 4, cudaMemcpyHostToDevice,
                     stream));
  CK(cudaMemcpyAsync(ctrl + off_tasks, t.dev_tasks.data(), t.dev_tasks.size() * sizeof(Task),
                     cudaMemcpyHostToDevice, stream));
  if (p->poison) CK(cudaMemsetAsync(base, 0xff, c_bytes, stream));

  // ---- kernel arguments (same kernel as entwine_gemm_rs) ----
  KParams kp;
  std::memset(&kp, 0, sizeof(kp));
  kp.M = int(g.M); kp.N = int(g.N); kp.K = int(g.K); kp.W = g.W; kp.r = p->rank; kp.order = p->order;
  kp.rowsT = g.rowsT; kp.nBn = g.nBn; kp.nTn = g.nTn; kp.Lb = g.Lb; kp.P_blk = g.P_blk; kp.Q = g.Q;
  kp.cpb = g.cpb; kp.R = g.R;
  kp.x = p->x;
  kp.mode = MODE_FUSED;
  kp.help = (p->tail_help || p->lists_opt > 0) ? 1 : 0;  // shared lists need every CTA to scan them
  kp.skip_wait = 0;
  kp.release_group = 1;  // this entry point keeps the per-block release
  kp.group_ctr = nullptr;
  kp.norm = 0;
  kp.claim = claim_size(g.W);
  kp.epoch = 1;  // the flags were cleared above
  kp.seq = 0;
  kp.wait_budget_ns = (unsigned long long)p->wait_budget_ns;
  {
    const int grc = ring_geometry(p, &kp, p->reg_consumer != 0 || p->consumer_tma == 0);
    if (grc != ENTWINE_OK) return grc;
  }
  kp.cws = reinterpret_cast<const __nv_bfloat16*>(base);
  kp.cws_out = reinterpret_cast<__nv_bfloat16*>(base);
  kp.peers = static_cast<const __nv_bfloat16*>(peer_partials);
  kp.peer_rows = g.M;
  kp.peer_row0 = 0;
  kp.send = static_cast<__nv_bfloat16*>(send_bufs);
  kp.prefetch = p->prefetch;
  kp.l2_hints = p->l2_hints;
  kp.out = static_cast<__nv_bfloat16*>(out_shard);
  kp.status = reinterpret_cast<StatusSlot*>(ctrl + off_status);
  kp.list_head = reinterpret_cast<int*>(ctrl + off_heads);
  kp.list_head_next = nullptr;  // this entry point clears its control block before every launch
  kp.status_next = nullptr;
  kp.list_offs = reinterpret_cast<const int*>(ctrl + off_offs);
  kp.flags_own = reinterpret_cast<unsigned*>(ctrl + off_fown);
  kp.flags_peer = reinterpret_cast<const unsigned*>(ctrl + off_fpeer);
  kp.tasks = reinterpret_cast<const Task*>(ctrl + off_tasks);
  kp.G = p->n_gemm_ctas;
  kp.n_ded = p->n_comm_ctas;
  int grid = p->n_gemm_ctas + p->n_comm_ctas;
  const bool pair = p->pair;
  if (pair && (grid & 1)) {
    if (grid + 1 > p->num_sms) grid -= 1, kp.n_ded -= 1;
    else grid += 1, kp.n_ded += 1;
    if (kp.n_ded < p->x) kp.help = 1;
  }
  kp.split = split_last_wave(p, kp.G);
  KMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  bool ok = make_operand_maps(&maps, A, B, g, pair ? 128 : g.BN, kp.kpb, p->lda, p->ldb, kp.b_kn = p->b_kn, &kp.k3d) &&
            make_map(&maps.p_pf, peer_partials, int64_t(g.W - 1) * g.M, g.N, kTile, kTile, false);
  for (int id = 0; ok && id < 2; ++id) {
    const int rs = kp.rs[id];
    const int prs = kp.prs[id];
    ok = make_map(&maps.c_ld[id], base, g.M, g.N, kTile, rs, false) &&
         make_map(&maps.c_push[id], base, g.M, g.N, kTile, prs, false) &&
         make_map3(&maps.p_ld[id], peer_partials, g.W - 1, g.M, g.N, kTile, rs, g.W - 1) &&
         make_map(&maps.send_st[id], send_bufs, int64_t(g.W - 1) * g.R, g.N, kTile, prs, false);
  }
  if (!ok) return ENTWINE_ERR_CUDA;
  int rc;
  if (pair) rc = launch_bn<256, true>(p, kp, maps, grid, stream);
  else if (g.BN == 256) rc = launch_bn<256, false>(p, kp, maps, grid, stream);
  else rc = launch_bn<128, false>(p, kp, maps, grid, stream);
  if (rc != ENTWINE_OK) return rc;

  if (status_out) {
    StatusSlot s;
    CK(cudaStreamSynchronize(stream));
    CK(cudaMemcpy(&s, ctrl + off_status, sizeof(s), cudaMemcpyDeviceToHost));
    const int code = int(s.code_cta_task & 0xff);
    status_out[0] = code ? -code : 0;
    status_out[1] = int64_t((s.code_cta_task >> 8) & 0xffffff);
    status_out[2] = int64_t(int32_t(s.code_cta_task >> 32));
    status_out[3] = int64_t(s.flags_published);
    status_out[4] = int64_t(s.tiles_reduced);
    status_out[5] = int64_t(s.tiles_pushed);
    status_out[6] = (s.t_gemm_end > s.t_start) ? int64_t(s.t_gemm_end - s.t_start) : 0;
    status_out[7] = (s.t_end > s.t_start) ? int64_t(s.t_end - s.t_start) : 0;
    return int(status_out[0]);
  }
  return ENTWINE_OK;
}
