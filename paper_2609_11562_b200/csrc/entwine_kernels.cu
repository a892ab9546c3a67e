// Fused GEMM-ReduceScatter for sm_100a: one persistent launch whose CTAs are split into
// producers (tcgen05/TMEM GEMM fed by TMA, one flag per finished 128x128 tile) and consumers
// (flag polling, scatter push, fp32-accumulated tile reduction).  See include/entwine.h for
// the contract and the paper sections each step follows.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>

#include "entwine_internal.h"

namespace entwine {

// ------------------------------------------------------------------------------------------
// compile-time shape of the producer
// ------------------------------------------------------------------------------------------
constexpr int kBM = 128;          // producer block rows = reduction tile rows
constexpr int kBK = 64;           // K elements per pipeline stage (128 bytes = one swizzle row)
constexpr int kUmmaK = 16;        // K per tcgen05.mma for 16-bit operands
constexpr int kThreads = 256;     // warp 0: TMA, warp 1: MMA + TMEM owner, warps 4-7: epilogue
constexpr int kEpiWarp0 = 4;
constexpr int kEpiThreads = 128;
constexpr uint32_t kSpinCheck = 128;  // spins between looks at the timer / abort flag

template <int BN>
struct Cfg {
  static constexpr int kStages = (BN == 256) ? 4 : 6;
  static constexpr int kABytes = kBM * kBK * 2;
  static constexpr int kBBytes = BN * kBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kTmemCols = 2 * BN;  // two accumulators: epilogue overlaps next mainloop
  static constexpr int kBarBytes = 256;
  static constexpr int kSmemBytes = kStages * kStageBytes + kBarBytes + 1024;  // + align slack
};

struct KParams {
  // geometry
  int M, N, K, W, r, order;
  int rowsT, nBn, nTn, Lb, P_blk, Q, cpb;
  long long R;
  // launch shape
  int n_ded;      // CTAs [0, n_ded) are dedicated consumers
  int G;          // CTAs [n_ded, n_ded+G) are producers
  int x;          // consumer lists
  int mode;       // Mode
  int help;       // producers / finished consumers take tasks from other lists
  int skip_wait;  // treat every flag as published (consumer in isolation)
  unsigned epoch;  // flag value of this producer run
  unsigned seq;    // launch counter: selects the status slot
  unsigned long long wait_budget_ns;
  // memory
  __nv_bfloat16* C;              // partial output workspace [M,N] (or caller's partial)
  const __nv_bfloat16* peers;    // [W-1][M][N]
  __nv_bfloat16* out;            // [R][N]
  __nv_bfloat16* send;           // [W-1][R][N]
  unsigned* flags_own;           // [W][Q]
  const unsigned* flags_peer;    // [W-1][Q]
  const Task* tasks;
  const int* list_offs;          // [x+1]
  int* list_head;                // [x]
  StatusSlot* status;            // [2]
  unsigned* done_ctr;
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
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_gpu(unsigned* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
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
// Instruction descriptor: fp32 accumulator, bf16 x bf16, both operands K-major, M = 128.
template <int BN>
__device__ __forceinline__ constexpr uint32_t instr_desc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(BN >> 3) << 17) | (uint32_t(kBM >> 4) << 24);
}

// ------------------------------------------------------------------------------------------
// status helpers
// ------------------------------------------------------------------------------------------
struct CtaShared {
  volatile int abort;   // another role of this CTA (or a peer CTA) gave up
  int claim;            // broadcast of the claimed task index
  int wait_ok;          // broadcast of the flag wait's result
  uint32_t tmem_base;
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

// Bounded acquire-poll of one flag (Sec. 4.2: thread 0 polls with acquire loads).
__device__ __forceinline__ bool wait_flag(const unsigned* f, const KParams& P) {
  if (ld_acquire_gpu(f) >= P.epoch) return true;
  unsigned long long t0 = 0;
  for (uint32_t spins = 1;; ++spins) {
    if (ld_acquire_gpu(f) >= P.epoch) return true;
    if ((spins % 32) == 0) {
      if (global_abort(P)) return false;
      unsigned long long now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > P.wait_budget_ns) return false;
    }
    __nanosleep(40);
  }
}

// ------------------------------------------------------------------------------------------
// consumer: ReduceTile and the scatter push (Sec. 4.2)
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

constexpr int kChunksPerTile = kTile * kTile * 2 / 16;  // 16-byte chunks in a 128x128 bf16 tile

// out = bf16( fp32(own) + sum over peers in ascending rank order ), one writer per element.
template <int NP>
__device__ __forceinline__ void reduce_tile(const __nv_bfloat16* own, const __nv_bfloat16* peer0,
                                            long long peer_stride, __nv_bfloat16* dst, long long N,
                                            int n_peers_rt) {
  constexpr int U = (NP > 0 && NP <= 3) ? 4 : 2;
  const int n_peers = NP > 0 ? NP : n_peers_rt;
  for (int it = 0; it < kChunksPerTile / kThreads; it += U) {
    uint4 o[U];
    uint4 pv[U][NP > 0 ? NP : 1];
    long long off[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int idx = threadIdx.x + (it + u) * kThreads;
      off[u] = (long long)(idx >> 4) * N + (idx & 15) * 8;
      o[u] = __ldcg(reinterpret_cast<const uint4*>(own + off[u]));
      if (NP > 0) {
#pragma unroll
        for (int q = 0; q < (NP > 0 ? NP : 1); ++q)
          pv[u][q] = __ldcs(reinterpret_cast<const uint4*>(peer0 + q * peer_stride + off[u]));
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      acc_bf16x8(a, o[u]);  // start from the local contribution
      if (NP > 0) {
#pragma unroll
        for (int q = 0; q < (NP > 0 ? NP : 1); ++q) acc_bf16x8(a, pv[u][q]);
      } else {
        for (int q = 0; q < n_peers; ++q)
          acc_bf16x8(a, __ldcs(reinterpret_cast<const uint4*>(peer0 + q * peer_stride + off[u])));
      }
      __stcs(reinterpret_cast<uint4*>(dst + off[u]), pack_bf16x8(a));
    }
  }
}

__device__ __forceinline__ void push_tile(const __nv_bfloat16* src, __nv_bfloat16* dst, long long N) {
  constexpr int U = 8;
  static_assert(kChunksPerTile / kThreads == U, "one pass");
  uint4 v[U];
  long long off[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int idx = threadIdx.x + u * kThreads;
    off[u] = (long long)(idx >> 4) * N + (idx & 15) * 8;
    v[u] = __ldcg(reinterpret_cast<const uint4*>(src + off[u]));
  }
#pragma unroll
  for (int u = 0; u < U; ++u) __stcs(reinterpret_cast<uint4*>(dst + off[u]), v[u]);
}

struct CommCounters {
  unsigned reduced = 0, pushed = 0;
};

// Walk consumer lists starting at `first_list`; every task is claimed through its list's
// head counter, so a list is always consumed in order (Sec. 3.1) whoever executes it.
__device__ void consumer_walk(const KParams& P, CtaShared* sh, int first_list, int n_lists_to_visit,
                              CommCounters* cnt) {
  const long long MN = (long long)P.M * P.N;
  const long long RN = P.R * (long long)P.N;
  for (int li = 0; li < n_lists_to_visit; ++li) {
    int j = first_list + li;
    if (j >= P.x) j -= P.x;
    const int base = P.list_offs[j];
    const int len = P.list_offs[j + 1] - base;
    for (;;) {
      if (threadIdx.x == 0) {
        // cheap look before the atomic so that exhausted lists cost one load
        int head = *reinterpret_cast<volatile int*>(&P.list_head[j]);
        sh->claim = (head >= len) ? len : atomicAdd(&P.list_head[j], 1);
      }
      __syncthreads();
      const int i = sh->claim;
      __syncthreads();
      if (i >= len) break;
      const Task task = P.tasks[base + i];
      // index check: record and skip instead of touching memory out of range
      bool bad = task.src_off < 0 || task.src_off + (long long)(kTile - 1) * P.N + kTile > MN ||
                 task.dst_off < 0 || task.dst_off + (long long)(kTile - 1) * P.N + kTile > RN ||
                 task.t < 0 || task.t >= P.Q || task.d < 0 || task.d >= P.W ||
                 (task.kind == 1 && (task.slot < 0 || task.slot >= P.W - 1));
      if (bad) {
        if (threadIdx.x == 0) report(P, -ENTWINE_ERR_INTERNAL, base + i);
        continue;
      }
      if (!P.skip_wait) {
        if (threadIdx.x == 0) {
          // local flag first, then the peers in ascending rank order (Sec. 4.2)
          bool ok = wait_flag(&P.flags_own[task.d * P.Q + task.t], P);
          if (ok && task.kind == 0) {
            for (int q = 0; ok && q < P.W - 1; ++q) ok = wait_flag(&P.flags_peer[q * P.Q + task.t], P);
          }
          if (!ok) report(P, -ENTWINE_ERR_TIMEOUT, base + i);
          sh->wait_ok = ok ? 1 : 0;
        }
        __syncthreads();  // extends thread 0's acquire to the whole CTA (Sec. 4.2)
        const int ok = sh->wait_ok;
        __syncthreads();
        if (!ok) return;
      }
      const __nv_bfloat16* src = P.C + task.src_off;
      if (task.kind == 0) {
        const __nv_bfloat16* peer0 = P.peers + task.src_off;
        __nv_bfloat16* dst = P.out + task.dst_off;
        switch (P.W - 1) {
          case 1: reduce_tile<1>(src, peer0, MN, dst, P.N, 1); break;
          case 3: reduce_tile<3>(src, peer0, MN, dst, P.N, 3); break;
          case 7: reduce_tile<7>(src, peer0, MN, dst, P.N, 7); break;
          default: reduce_tile<0>(src, peer0, MN, dst, P.N, P.W - 1); break;
        }
        if (threadIdx.x == 0) cnt->reduced++;
      } else {
        push_tile(src, P.send + (long long)task.slot * RN + task.dst_off, P.N);
        if (threadIdx.x == 0) cnt->pushed++;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
entwine_fused_kernel(const __grid_constant__ CUtensorMap tmap_a,
                     const __grid_constant__ CUtensorMap tmap_b, const KParams P) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ CtaShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  StatusSlot* st = &P.status[P.seq & 1];

  if (threadIdx.x == 0) {
    sh.abort = 0;
    sh.claim = 0;
    sh.wait_ok = 0;
    sh.tmem_base = 0;
    atomicMin(&st->t_start, globaltimer_ns());
  }
  CommCounters cnt;
  unsigned published = 0;
  const bool is_producer = (int)blockIdx.x >= P.n_ded && P.mode != MODE_COMM_ONLY;
  const int g = (int)blockIdx.x - P.n_ded;

  if (is_producer) {
    // ---------------- producer: tcgen05 GEMM over blocks p = g, g+G, ... ----------------
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~uintptr_t(1023));
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_base = smem_base + C::kStages * C::kStageBytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (C::kStages + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * C::kStages + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * C::kStages + 2 + a); };
    const uint32_t tmem_slot = bar_base + 8u * (2 * C::kStages + 4);

    if (threadIdx.x == 0) {
      for (int s = 0; s < C::kStages; ++s) {
        mbar_init(full_bar(s), 1);
        mbar_init(empty_bar(s), 1);
      }
      for (int a = 0; a < 2; ++a) {
        mbar_init(tfull_bar(a), 1);
        mbar_init(tempty_bar(a), kEpiThreads / 32);
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base =
        *reinterpret_cast<volatile uint32_t*>(smem + C::kStages * C::kStageBytes + 8 * (2 * C::kStages + 4));
    const int KB = (P.K + kBK - 1) / kBK;
    const int n_my = (g < P.P_blk) ? (P.P_blk - g + P.G - 1) / P.G : 0;

    if (warp == 0 && lane == 0) {
      // ---- TMA producer ----
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int i = 0; ok && i < n_my; ++i) {
        const int p = g + i * P.G;
        int d, l;
        if (P.order == ENTWINE_ORDER_INTERLEAVED) { d = p % P.W; l = p / P.W; }
        else { d = p / P.Lb; l = p - d * P.Lb; }
        const int mb = d * P.rowsT + l / P.nBn, nb = l % P.nBn;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1, P, &sh)) { ok = false; break; }
          mbar_arrive_expect_tx(full_bar(stage), C::kStageBytes);
          const uint32_t a_dst = smem_base + stage * C::kStageBytes;
          tma_load_2d(a_dst, &tmap_a, kb * kBK, mb * kBM, full_bar(stage));
          tma_load_2d(a_dst + C::kABytes, &tmap_b, kb * kBK, nb * BN, full_bar(stage));
          if (++stage == C::kStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) { sh.abort = 1; report(P, -ENTWINE_ERR_TIMEOUT, -1); }
    } else if (warp == 1 && lane == 0) {
      // ---- MMA issuer ----
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      constexpr uint32_t idesc = instr_desc<BN>();
      bool ok = true;
      for (int i = 0; ok && i < n_my; ++i) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1, P, &sh)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < KB; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, P, &sh)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_s = smem_base + stage * C::kStageBytes;
          const uint64_t a_desc = smem_desc_sw128(a_s);
          const uint64_t b_desc = smem_desc_sw128(a_s + C::kABytes);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            // advancing K by 16 elements = 32 bytes = 2 descriptor address units
            umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
          }
          tc_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
          if (++stage == C::kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc_commit(tfull_bar(acc));  // accumulator complete
        if ((acc ^= 1) == 0) acc_phase ^= 1;
      }
      if (!ok) { sh.abort = 1; report(P, -ENTWINE_ERR_TIMEOUT, -2); }
    } else if (warp >= kEpiWarp0) {
      // ---- epilogue: TMEM -> bf16 -> partial C, then publish the block's tile flags ----
      const int q = warp & 3;  // TMEM lane quarter this warp may read
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int i = 0; ok && i < n_my; ++i) {
        const int p = g + i * P.G;
        int d, l;
        if (P.order == ENTWINE_ORDER_INTERLEAVED) { d = p % P.W; l = p / P.W; }
        else { d = p / P.Lb; l = p - d * P.Lb; }
        const int trow = l / P.nBn, nb = l % P.nBn;
        const int mb = d * P.rowsT + trow;
        ok = mbar_wait(tfull_bar(acc), acc_phase, P, &sh);
        ok = __all_sync(0xffffffffu, ok);  // reconverge; the warp leaves the loop together
        if (!ok) break;
        tc_fence_after();
        const long long row = (long long)mb * kBM + q * 32 + lane;
        __nv_bfloat16* crow = P.C + row * P.N + (long long)nb * BN;
        const uint32_t taddr = tmem_base + (uint32_t(q * 32) << 16) + acc * BN;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(taddr + c * 32, v);
          tmem_ld_wait();
          uint4 o[4];
          uint32_t* ow = reinterpret_cast<uint32_t*>(o);
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
            ow[e] = *reinterpret_cast<uint32_t*>(&h);
          }
          uint4* dstp = reinterpret_cast<uint4*>(crow + c * 32);
#pragma unroll
          for (int e = 0; e < 4; ++e) dstp[e] = o[e];
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));  // accumulator may be overwritten
        // all of the block's stores, then the flags (Sec. 4.2)
        named_bar_sync(1, kEpiThreads);
        if (warp == kEpiWarp0 && lane == 0) {
          for (int c = 0; c < P.cpb; ++c) {
            const int t = trow * P.nTn + nb * P.cpb + c;
            st_release_gpu(&P.flags_own[d * P.Q + t], P.epoch);
          }
          published += P.cpb;
        }
        if ((acc ^= 1) == 0) acc_phase ^= 1;
      }
      if (!ok && lane == 0) { sh.abort = 1; report(P, -ENTWINE_ERR_TIMEOUT, -3); }
    }
    __syncthreads();
    if (threadIdx.x == 0 && n_my > 0) atomicMax(&st->t_gemm_end, globaltimer_ns());
    if (sh.abort) {
      // give copies that may still be in flight time to land before the CTA's memory is reused
      const unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ULL) __nanosleep(1000);
    }
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
    __syncthreads();
  }

  // ---------------- consumer ----------------
  if (P.mode != MODE_GEMM_ONLY && !sh.abort) {
    if (!is_producer) {
      // dedicated consumer block j: its own list, then (shared-pool analogue) the others
      const int j = (int)blockIdx.x % P.x;
      const bool owns = (int)blockIdx.x < P.x;
      if (owns) consumer_walk(P, &sh, j, 1, &cnt);
      if (P.help || !owns) consumer_walk(P, &sh, owns ? (j + 1) % P.x : j, owns ? P.x - 1 : P.x, &cnt);
    } else if (P.n_ded == 0) {
      // non-overlapped use of all SMs: block g consumes list g (then helps)
      if (g < P.x) consumer_walk(P, &sh, g, 1, &cnt);
      if (P.help) consumer_walk(P, &sh, (g + 1) % P.x, P.x - 1, &cnt);
    } else if (P.help) {
      consumer_walk(P, &sh, g % P.x, P.x, &cnt);
    }
  }

  // ---------------- exit bookkeeping ----------------
  __syncthreads();
  // the epilogue's publishing thread adds its own count
  if (is_producer && warp == kEpiWarp0 && lane == 0 && published)
    atomicAdd(&st->flags_published, (unsigned long long)published);
  __syncthreads();
  if (threadIdx.x == 0) {
    if (cnt.reduced) atomicAdd(&st->tiles_reduced, (unsigned long long)cnt.reduced);
    if (cnt.pushed) atomicAdd(&st->tiles_pushed, (unsigned long long)cnt.pushed);
    atomicMax(&st->t_end, globaltimer_ns());
    __threadfence();
    const unsigned prev = atomicAdd(P.done_ctr, 1u);
    if (prev == gridDim.x - 1) {
      // last CTA out: rewind the list heads and prepare the other status slot
      for (int j = 0; j < P.x; ++j) P.list_head[j] = 0;
      StatusSlot* nx = &P.status[(P.seq & 1) ^ 1];
      nx->code_cta_task = 0;
      nx->flags_published = 0;
      nx->tiles_reduced = 0;
      nx->tiles_pushed = 0;
      nx->t_start = ~0ULL;
      nx->t_gemm_end = 0;
      nx->t_end = 0;
      *P.done_ctr = 0;
      __threadfence();
    }
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
  unsigned* done_ctr = nullptr;
  unsigned epoch = 0;
  unsigned seq = 0;
  bool status_pending = false;
  cudaStream_t last_stream = nullptr;
  int64_t withheld = -1;
  // staging for the host-buffer entry point
  cudaStream_t own_stream = nullptr;
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

// 2-D map over a row-major bf16 matrix [rows, cols] with a (box_rows x 64-column) box and
// 128-byte swizzle; out-of-range elements read as zero (K tails).
static bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cuuint64_t(cols), cuuint64_t(rows)};
  cuuint64_t strides[1] = {cuuint64_t(cols) * 2};
  cuuint32_t box[2] = {cuuint32_t(kBK), cuuint32_t(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS;
}

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

static int ensure_device(Plan* p) {
  if (p->dev) return ENTWINE_OK;
  int sms = device_sm_count();
  if (sms <= 0) return ENTWINE_ERR_CUDA;
  int dev = 0;
  CK(cudaGetDevice(&dev));
  int major = 0;
  CK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return ENTWINE_ERR_RESOURCES;  // tcgen05 / TMEM needed
  if (p->num_sms > sms) return ENTWINE_ERR_RESOURCES;
  DeviceState* d = new DeviceState();
  d->device = dev;
  const Geometry& g = p->g;
  const size_t n_own = size_t(g.W) * g.Q, n_peer = size_t(g.W - 1) * g.Q;
  const HostTables& t = p->tables;
  bool ok = cudaMalloc(&d->C, size_t(g.M) * g.N * 2) == cudaSuccess &&
            cudaMalloc(&d->flags_own, n_own * 4) == cudaSuccess &&
            cudaMalloc(&d->flags_peer, n_peer * 4) == cudaSuccess &&
            cudaMalloc(&d->tasks, t.dev_tasks.size() * sizeof(Task)) == cudaSuccess &&
            cudaMalloc(&d->list_offs, t.list_offs.size() * 4) == cudaSuccess &&
            cudaMalloc(&d->list_head, size_t(p->x) * 4) == cudaSuccess &&
            cudaMalloc(&d->status, 2 * sizeof(StatusSlot)) == cudaSuccess &&
            cudaMalloc(&d->done_ctr, 4) == cudaSuccess;
  if (ok) {
    StatusSlot init[2];
    std::memset(init, 0, sizeof(init));
    init[0].t_start = init[1].t_start = ~0ULL;
    ok = cudaMemset(d->flags_own, 0, n_own * 4) == cudaSuccess &&
         cudaMemset(d->flags_peer, 0xff, n_peer * 4) == cudaSuccess &&
         cudaMemset(d->C, 0, size_t(g.M) * g.N * 2) == cudaSuccess &&
         cudaMemcpy(d->tasks, t.dev_tasks.data(), t.dev_tasks.size() * sizeof(Task),
                    cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(d->list_offs, t.list_offs.data(), t.list_offs.size() * 4, cudaMemcpyHostToDevice) ==
             cudaSuccess &&
         cudaMemset(d->list_head, 0, size_t(p->x) * 4) == cudaSuccess &&
         cudaMemcpy(d->status, init, sizeof(init), cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemset(d->done_ctr, 0, 4) == cudaSuccess;
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
  if (d->own_stream) {
    cudaStreamSynchronize(d->own_stream);
    cudaStreamDestroy(d->own_stream);
  }
  cudaFree(d->C);
  cudaFree(d->flags_own);
  cudaFree(d->flags_peer);
  cudaFree(d->tasks);
  cudaFree(d->list_offs);
  cudaFree(d->list_head);
  cudaFree(d->status);
  cudaFree(d->done_ctr);
  cudaFree(d->sA);
  cudaFree(d->sB);
  cudaFree(d->sPeers);
  cudaFree(d->sOut);
  cudaFree(d->sSend);
  cudaGetLastError();
  delete d;
  p->dev = nullptr;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

template <int BN>
static int launch_bn(Plan* p, const KParams& kp, const CUtensorMap& ma, const CUtensorMap& mb, int grid,
                     cudaStream_t stream) {
  using C = Cfg<BN>;
  static bool configured = false;
  auto kern = entwine_fused_kernel<BN>;
  if (!configured) {
    CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes));
    int per_sm = 0;
    CK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, C::kSmemBytes));
    if (per_sm < 1) return ENTWINE_ERR_RESOURCES;
    configured = true;
  }
  kern<<<grid, kThreads, C::kSmemBytes, stream>>>(ma, mb, kp);
  CK(cudaGetLastError());
  return ENTWINE_OK;
}

// Common launch path.  `partial` overrides the workspace in consumer-only mode.
static int launch(Plan* p, int mode, const void* A, const void* B, const void* partial, const void* peers,
                  void* out, void* send, int n_ctas, cudaStream_t stream) {
  int rc = ensure_device(p);
  if (rc != ENTWINE_OK) return rc;
  DeviceState* d = p->dev;
  const Geometry& g = p->g;
  if (mode != MODE_COMM_ONLY && (!A || !B || !aligned16(A) || !aligned16(B))) return ENTWINE_ERR_INVALID;
  if (mode != MODE_GEMM_ONLY &&
      (!peers || !out || !send || !aligned16(peers) || !aligned16(out) || !aligned16(send)))
    return ENTWINE_ERR_INVALID;
  if (partial && !aligned16(partial)) return ENTWINE_ERR_INVALID;

  // serialise with the plan's previous launch if the caller switched streams
  if (d->last_stream != stream && p->launched) CK(cudaStreamSynchronize(d->last_stream));

  if (mode != MODE_COMM_ONLY) {
    d->epoch += 1;
    if (d->epoch >= 0xfffffff0u) {  // epoch wrap: start over with cleared flags
      CK(cudaMemsetAsync(d->flags_own, 0, size_t(g.W) * g.Q * 4, stream));
      d->epoch = 1;
    }
    if (p->poison) CK(cudaMemsetAsync(d->C, 0xff, size_t(g.M) * g.N * 2, stream));
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

  KParams kp;
  std::memset(&kp, 0, sizeof(kp));
  kp.M = int(g.M); kp.N = int(g.N); kp.K = int(g.K); kp.W = g.W; kp.r = p->rank; kp.order = p->order;
  kp.rowsT = g.rowsT; kp.nBn = g.nBn; kp.nTn = g.nTn; kp.Lb = g.Lb; kp.P_blk = g.P_blk; kp.Q = g.Q;
  kp.cpb = g.cpb; kp.R = g.R;
  kp.x = p->x;
  kp.mode = mode;
  kp.help = p->tail_help;
  kp.skip_wait = (mode == MODE_COMM_ONLY) ? 1 : 0;
  kp.epoch = d->epoch;
  d->seq += 1;
  kp.seq = d->seq;
  kp.wait_budget_ns = (unsigned long long)p->wait_budget_ns;
  kp.C = (mode == MODE_COMM_ONLY && partial) ? const_cast<__nv_bfloat16*>(static_cast<const __nv_bfloat16*>(partial))
                                             : d->C;
  kp.peers = static_cast<const __nv_bfloat16*>(peers);
  kp.out = static_cast<__nv_bfloat16*>(out);
  kp.send = static_cast<__nv_bfloat16*>(send);
  kp.flags_own = d->flags_own;
  kp.flags_peer = d->flags_peer;
  kp.tasks = d->tasks;
  kp.list_offs = d->list_offs;
  kp.list_head = d->list_head;
  kp.status = d->status;
  kp.done_ctr = d->done_ctr;

  int grid;
  if (mode == MODE_FUSED) {
    kp.n_ded = p->n_comm_ctas;
    kp.G = p->n_gemm_ctas;
    grid = p->n_comm_ctas + p->n_gemm_ctas;
  } else if (mode == MODE_GEMM_ONLY) {
    kp.n_ded = 0;
    kp.G = p->num_sms;
    grid = p->num_sms;
  } else {
    grid = (n_ctas <= 0) ? p->num_sms : n_ctas;
    if (grid > p->num_sms) return ENTWINE_ERR_INVALID;
    kp.n_ded = grid;
    kp.G = 0;
    // with fewer CTAs than lists the CTAs must visit every list
    if (grid < p->x) kp.help = 1;
  }

  CUtensorMap ma, mb;
  std::memset(&ma, 0, sizeof(ma));
  std::memset(&mb, 0, sizeof(mb));
  if (mode != MODE_COMM_ONLY) {
    if (!make_map(&ma, A, g.M, g.K, kBM) || !make_map(&mb, B, g.N, g.K, g.BN)) return ENTWINE_ERR_CUDA;
  }
  rc = (g.BN == 256) ? launch_bn<256>(p, kp, ma, mb, grid, stream) : launch_bn<128>(p, kp, ma, mb, grid, stream);
  if (rc != ENTWINE_OK) return rc;
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

int entwine_gemm_only(entwine_plan_t plan, const void* A, const void* B, void* stream) {
  if (!plan) return ENTWINE_ERR_INVALID;
  return launch(plan, MODE_GEMM_ONLY, A, B, nullptr, nullptr, nullptr, nullptr, 0,
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
  if (code) {
    // the launch gave up part-way: rewind what its last CTA would have rewound
    cudaMemset(d->list_head, 0, size_t(plan->x) * 4);
    cudaMemset(d->done_ctr, 0, 4);
    StatusSlot init[2];
    std::memset(init, 0, sizeof(init));
    init[0].t_start = init[1].t_start = ~0ULL;
    cudaMemcpy(d->status, init, sizeof(init), cudaMemcpyHostToDevice);
  }
  return int(out[0]);
}

int entwine_gemm_rs_host(entwine_plan_t plan, const void* A, const void* B, const void* peer_partials,
                         void* out_shard, void* send_bufs) {
  if (!plan || !A || !B || !peer_partials || !out_shard || !send_bufs) return ENTWINE_ERR_INVALID;
  int rc = ensure_device(plan);
  if (rc != ENTWINE_OK) return rc;
  DeviceState* d = plan->dev;
  const Geometry& g = plan->g;
  const size_t szA = size_t(g.M) * g.K * 2, szB = size_t(g.N) * g.K * 2;
  const size_t szP = size_t(g.W - 1) * g.M * g.N * 2, szO = size_t(g.R) * g.N * 2;
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
    CK(cudaMemcpyAsync(reinterpret_cast<char*>(d->sPeers) + off, static_cast<const char*>(peer_partials) + off,
                       part, cudaMemcpyHostToDevice, s));
  }
  rc = launch(plan, MODE_FUSED, d->sA, d->sB, nullptr, d->sPeers, d->sOut, d->sSend, 0, s);
  if (rc != ENTWINE_OK) return rc;
  CK(cudaMemcpyAsync(out_shard, d->sOut, szO, cudaMemcpyDeviceToHost, s));
  CK(cudaMemcpyAsync(send_bufs, d->sSend, szS, cudaMemcpyDeviceToHost, s));
  CK(cudaStreamSynchronize(s));
  int64_t stw[8];
  return entwine_last_status(plan, stw);
}

}  // extern "C"
