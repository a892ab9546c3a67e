/*
 * entwine.h - C ABI of the B200 (sm_100a) fused GEMM-ReduceScatter of a tensor-parallel
 * row-parallel linear layer, run on one GPU as a one-rank emulation of W logical ranks
 * (Entwine: interleaved tile production + tile-level flags + SM-based communication).
 *
 * Conventions
 *   - Every function returns an int: ENTWINE_OK (0) or a negative ENTWINE_ERR_* code.
 *     Nothing throws across this boundary; nothing traps or hangs the device: every
 *     device-side wait is bounded and reports through the plan's status word.
 *   - "device pointer" = global memory of the current CUDA device, 16-byte aligned,
 *     valid until the stream has finished the call.  "host pointer" = ordinary host
 *     memory.  The library never takes ownership of caller buffers.
 *   - No function synchronises the device unless its comment says so.
 *   - A plan is not thread-safe; calls on one plan must be issued from one thread and are
 *     serialised on the device by stream order (use one stream per plan; if the stream changes
 *     between two calls, the new stream is made to wait for the plan's previous call).
 *   - Launches of DIFFERENT plans must not overlap on the device either: a launch fills the
 *     GPU with one CTA per SM whose producers and consumers wait on each other, and two
 *     half-resident launches would each wait (boundedly: both end in ENTWINE_ERR_TIMEOUT) for
 *     CTAs that cannot start.  Put them on one stream or order them with events.
 *
 * Notation (paper Sec. 3.1 / 4.2): R = M/W rows per output partition; reduction tile
 * 128x128; producer block 128 x BN with BN in {128,256}; cpb = BN/128; nTn = N/128;
 * Q = (R/128)*nTn tiles per partition; P_blk = (M/128)*(N/BN) producer blocks; r = the
 * emulated rank; x = number of consumer (communication) task lists.
 *
 * Data layout (all bf16, row-major, contiguous)
 *   A             [M, K_local]   rows lda elements apart (ENTWINE_OPT_LDA, default K_local)
 *   B             [N, K_local]   rows ldb elements apart (ENTWINE_OPT_LDB, default K_local): the rank's shard
 *                                (or [K_local, N] with ENTWINE_OPT_B_LAYOUT = ENTWINE_B_LAYOUT_KN) of the layer weight (K contiguous), so the
 *                                rank's partial output is C = A . B^T, [M, N]
 *   peer_partials [W-1, M, N]    incoming partial outputs of the other ranks in ascending
 *                                rank order (slot q(w) = w < r ? w : w-1).  Only rows
 *                                [r*R, (r+1)*R) of each are read (Sec. 4.1: contributions
 *                                sit at matching offsets in every rank's buffer).
 *   out_shard     [R, N]         the reduced output partition of rank r
 *   send_bufs     [W-1, R, N]    slot q(d) receives rows [d*R,(d+1)*R) of C: what rank r
 *                                contributes to destination d (stands in for peer memory)
 */
#ifndef ENTWINE_H_
#define ENTWINE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct entwine_plan_s* entwine_plan_t;

/* Producer tile orders (Sec. 3.1 and Fig. 1). */
enum {
  ENTWINE_ORDER_ROW_MAJOR   = 0, /* partition-grouped: all blocks of partition 0, then 1, ... */
  ENTWINE_ORDER_INTERLEAVED = 1, /* Eq. 1: d = p mod W, l = floor(p / W)                      */
  ENTWINE_ORDER_M_MAJOR     = 2  /* ablation baseline (Sec. 5, "Computation Order"): the block
                                    grid of the whole output walked down the rows first, one
                                    block column after another, regardless of partitions      */
};

enum {
  ENTWINE_OK            =  0,
  ENTWINE_ERR_INVALID   = -1, /* bad shape, argument, option or call order                  */
  ENTWINE_ERR_RESOURCES = -2, /* not enough SMs / shared memory for a co-resident launch     */
  ENTWINE_ERR_CUDA      = -3, /* a CUDA call failed, or there is no CUDA device              */
  ENTWINE_ERR_TIMEOUT   = -4, /* a device-side wait ran out of its budget                    */
  ENTWINE_ERR_INTERNAL  = -5, /* a device-side index check failed                            */
  ENTWINE_ERR_TOO_LARGE = -6  /* the problem does not fit entwine_gemm_rs_static's fixed scratch */
};

/* Values of ENTWINE_OPT_B_LAYOUT. */
enum { ENTWINE_B_LAYOUT_NK = 0, ENTWINE_B_LAYOUT_KN = 1 };

/* Values of ENTWINE_OPT_RELEASE_GROUP besides a block count. */
enum { ENTWINE_RELEASE_PARTITION = -1, ENTWINE_RELEASE_WHOLE = -2 };

/* Option keys for entwine_set_option. Options marked [pre] must be set before the first
 * launch of the plan; the others may change between launches. */
enum {
  ENTWINE_OPT_RANK            = 1, /* [pre] emulated rank r, 0 <= r < W (default 0)             */
  ENTWINE_OPT_BLOCK_N         = 2, /* [pre] producer block width BN: 128 or 256 (default 256)   */
  ENTWINE_OPT_WAIT_BUDGET_NS  = 3, /* budget of every device-side flag wait (default 2e9 ns)    */
  ENTWINE_OPT_TAIL_HELP       = 4, /* 1 (default): producer CTAs that have finished their last
                                      block take tasks from the consumer lists (the one-launch
                                      analogue of the shared SM pool, Sec. 3.2 "Resource reuse");
                                      0: strict static partition (Sec. 5.3.3's other arm)        */
  ENTWINE_OPT_WITHHOLD_PEER   = 5, /* host-side fault injection: value = w*2^32 + t withholds the
                                      pre-published flag of peer rank w for tile t; -1 restores
                                      all peer flags (default)                                   */
  ENTWINE_OPT_NUM_SMS         = 6, /* [pre] override the SM count used for planning (testing
                                      without a device; default: the device's SM count, 148 if
                                      there is no device)                                        */
  ENTWINE_OPT_POISON_PARTIAL  = 7, /* 1: fill the partial-output workspace with NaN patterns
                                      before each launch (ordering stress test; default 0)       */
  ENTWINE_OPT_PAIR_CTAS       = 8, /* [pre] 1 (default): where the order allows it, two CTAs of a
                                      cluster compute a 256x256 pair tile (tcgen05 cta_group::2:
                                      two producer blocks that share a block column, each CTA
                                      loading half of the B panel); 0: every CTA works alone     */
  ENTWINE_OPT_PREFETCH        = 10, /* 1: the consumer's polling warp prefetches the next reduce
                                      task's published peer tiles into L2; 0 (default): off      */
  ENTWINE_OPT_L2_HINTS        = 12, /* L2 eviction policies on TMA traffic, bit mask (default 3):
                                      bit 0: the consumer's tile loads and pushed-tile stores are
                                      evict-first (touched once); bit 1: the producer's operand
                                      loads are evict-last (panels are re-read by many CTAs)     */
  ENTWINE_OPT_LISTS           = 13, /* [pre] number of consumer task lists x (Sec. 3.1: tile t of the
                                      own partition goes to list t mod x); 0 (default): one list
                                      per consumer CTA.  With fewer lists than CTAs the CTAs share
                                      lists through the lists' head counters                     */
  ENTWINE_OPT_RELEASE_GROUP   = 14, /* release granularity of the tile flags (the ablation of Sec. 5,
                                      "Release Granularity"; each reduction task stays one tile):
                                      1 (default): a producer block's tiles are released when the
                                      block is stored; g > 1: g consecutive blocks of the tile order
                                      are released together, when the last of them is stored;
                                      ENTWINE_RELEASE_PARTITION (-1): all tiles of a destination
                                      partition together; ENTWINE_RELEASE_WHOLE (-2): the whole
                                      output together.  Results are identical for every value      */
  ENTWINE_OPT_STAGES          = 11, /* stages of the producer's operand ring (2..6); the shared
                                      memory they leave goes to the co-located consumer ring;
                                      0 (default): chosen from the shape                         */
  ENTWINE_OPT_KBLOCKS_PER_STAGE = 15, /* k-blocks (64 elements of K_local) per stage of the operand
                                      ring: 1 or 2; 0 (default): 1 beside the consumer's TMA ring; 2
                                      with the register consumer where a k-block of both operands
                                      is 32 KiB (CTA pairs, BN = 128).  With 2 and K_local a
                                      multiple of 64 an operand's share of a stage arrives as one
                                      32 KiB TMA box                                                */
  ENTWINE_OPT_LDA             = 16, /* leading dimension of A in elements (row pitch), a multiple of 8
                                      and >= K_local; 0 (default) = K_local.  May change between
                                      launches                                                     */
  ENTWINE_OPT_LDB             = 17, /* the same for B                                              */
  ENTWINE_OPT_CONSUMER_TMA    = 21, /* 1 (default): once a CTA's producer work is over (and in CTAs
                                      that do not produce) the consumer streams tiles through a
                                      shared-memory ring filled by TMA: in pull mode one 3-D box
                                      whose planes are the peers' heap segments.  0 (implies the
                                      register path of REG_CONSUMER): plain 128-bit loads and stores
                                      for the whole call, nothing but ordinary loads ever touches
                                      peer memory: the conservative data path for a first run over
                                      NVLink                                                       */
  ENTWINE_OPT_B_LAYOUT        = 20, /* layout of B.  ENTWINE_B_LAYOUT_NK (default): [N, K_local], K
                                      contiguous (the shard of an nn.Linear weight); ENTWINE_B_LAYOUT_KN:
                                      [K_local, N], N contiguous (the C = A . B of Sec. 3.3 as
                                      written), read by the tensor core as an MN-major operand.  LDB
                                      is the row pitch of the layout in force; changing the layout
                                      resets it to contiguous (set LDB after B_LAYOUT).  May change
                                      between launches                                             */
  ENTWINE_OPT_SPLIT_LAST_WAVE = 19, /* CTA pairs only.  1 (default): when the pair tiles left for the
                                      last wave occupy at most half of the CTA pairs, each of them is
                                      computed as two half-width units (256 x 128: one 128 x 128 tile
                                      per CTA, its flag published by itself) on two pairs, so that
                                      the last wave costs half a tile time (the producer block may
                                      be any multiple of the reduction tile, Sec. 4.2); 0: whole
                                      pair tiles only.  Off with a release group other than 1      */
  ENTWINE_OPT_REG_CONSUMER    = 18, /* how the consumer warps of a CTA that still produces move their
                                      tiles.  0 (default): through a small shared-memory ring filled
                                      by TMA beside the operand stages; 1: whole tiles through
                                      registers with plain 128-bit loads and stores, so that all
                                      shared memory and the SM's TMA unit serve the operand ring
                                      (measured slower on the benchmark's shapes: the loads of eight
                                      warps stretch the producer more than the ring does; a kernel
                                      of its own, so that neither path's code weighs on the other).
                                      Once a CTA's producer work is over (and in dedicated consumer
                                      CTAs) tiles go through the large TMA ring either way          */
  ENTWINE_OPT_COLOCATE        = 9  /* 1 (default): with TAIL_HELP (or n_comm_sms = 0) a producer
                                      CTA's consumer warps take tasks while its tensor-core work
                                      is still running, through a small shared-memory ring beside
                                      the producer's buffers (computation and communication share
                                      the SM, Sec. 3.2); 0: they start when its last block is done */
};

/* What entwine_plan_export can write.  Integer tables, host memory, for bit-exact diffs. */
enum {
  ENTWINE_EXPORT_COUNTS      = 0, /* int64[16]: P_blk, Q, cpb, x, n_tasks, n_reduce, n_push,
                                     flags_published, peer_flags_prepublished, min_flag_reads,
                                     bytes_peer_read, bytes_own_read, bytes_push_write,
                                     bytes_out_write, n_gemm_ctas, n_comm_ctas               */
  ENTWINE_EXPORT_ORDER       = 1, /* int32[P_blk][4]: mb, nb, d, l per logical position p     */
  ENTWINE_EXPORT_TILES       = 2, /* int32[P_blk][cpb]: tile indices covered by block p       */
  ENTWINE_EXPORT_FLAG_SEQ    = 3, /* int32[P_blk*cpb][3]: (src=r, d, t) at k = p*cpb + c      */
  ENTWINE_EXPORT_LIST_OFFS   = 4, /* int32[x+1]: rows of TASKS that belong to list j          */
  ENTWINE_EXPORT_TASKS       = 5, /* int64[n_tasks][8]: kind(0 reduce,1 push), d, t, k, list,
                                     src_off, dst_slot(-1 for reduce), dst_off  (elements)    */
  ENTWINE_EXPORT_PEER_OFFS   = 6  /* int64[n_reduce][W-1]: element offsets into peer_partials */
};

/*
 * entwine_plan - validate a problem and build its schedule (Sec. 3.1 Eq. 1, Sec. 3.2).
 *   M, N, K_local  GEMM extents of the emulated rank (C[M,N] = A[M,K_local] . B[N,K_local]^T)
 *   W              number of logical ranks, >= 2
 *   tile_order     ENTWINE_ORDER_*
 *   n_comm_sms     SMs dedicated to communication CTAs (the communication budget x,
 *                  Sec. 3.2); 0 = non-overlapped use of all SMs: every CTA first produces,
 *                  then consumes (Sec. 5.3.2's baseline)
 * Requirements (Sec. 4.1): M % (128*W) == 0, N % 128 == 0 (and N % BN == 0 at launch),
 * K_local % 16 == 0, 0 <= n_comm_sms < number of SMs.
 * The plan owns the partial-output workspace C[M,N] (bf16), the flag arrays, the device
 * copies of the task tables and a status block; they are allocated with cudaMalloc at the
 * first launch (so do the first launch outside stream capture) and reused by every later
 * launch (Sec. 4.1).  Without a CUDA device the plan is host-only: tables can be exported,
 * launches return ENTWINE_ERR_CUDA.
 * Writes the handle to *plan.  Errors: ENTWINE_ERR_INVALID.
 */
int entwine_plan(entwine_plan_t* plan, int64_t M, int64_t N, int64_t K_local, int W,
                 int tile_order, int n_comm_sms);

/*
 * entwine_plan_workspace_bytes / entwine_plan_set_workspace - let the caller's allocator own the
 * plan's device memory.  Without these calls the plan allocates its arrays with cudaMalloc at the
 * first call that needs the device; with them, everything the plan (and its layer-chain and
 * pull-mode calls) would allocate lives in one caller-provided block.
 *   _workspace_bytes  writes the size of that block for the plan as it is now ([pre] options
 *                     that change the tables change the size: query after setting them).
 *   _set_workspace    workspace: device pointer, 256-byte aligned, at least that size, valid until
 *                     entwine_destroy (the library never frees it); NULL returns the plan to
 *                     memory of its own.  The call initialises the block (synchronous copies of
 *                     the task tables, cleared flags and status) and performs the per-device
 *                     kernel set-up, so the plan's first launch neither allocates nor
 *                     synchronises and may already be captured into a CUDA graph.
 * Call before the plan's first launch.  Errors: ENTWINE_ERR_INVALID (after a launch, misaligned
 * or too small), ENTWINE_ERR_RESOURCES, ENTWINE_ERR_CUDA.  A [pre] option set afterwards keeps
 * the block; the next call fails with ENTWINE_ERR_INVALID if the rebuilt tables no longer fit it.
 */
int entwine_plan_workspace_bytes(entwine_plan_t plan, size_t* bytes);
int entwine_plan_set_workspace(entwine_plan_t plan, void* workspace, size_t bytes);

/* entwine_set_option - see ENTWINE_OPT_*.  Errors: ENTWINE_ERR_INVALID (unknown key, bad
 * value, or a [pre] option after the first launch). */
int entwine_set_option(entwine_plan_t plan, int key, int64_t value);

/*
 * entwine_gemm_rs - one fused GEMM-ReduceScatter call of the emulated rank, enqueued on
 * `stream` (a cudaStream_t passed as void*; NULL = the default stream).  One kernel launch:
 * producer CTAs run the tcgen05 GEMM over the plan's block order and publish one flag per
 * finished 128x128 tile (Sec. 3.1, Sec. 4.2); consumer CTAs on the dedicated SMs poll the
 * flags, copy non-owned tiles to send_bufs and reduce owned tiles with the W-1 incoming
 * partials into out_shard (ReduceTile, Sec. 4.2: start from the local contribution, add the
 * peers in ascending rank order in fp32, single writer).
 * All five pointers are device pointers (layouts above).  Returns after enqueueing.
 * Errors: ENTWINE_ERR_INVALID (null / misaligned pointer), ENTWINE_ERR_RESOURCES,
 * ENTWINE_ERR_CUDA; a timeout or index failure of an earlier launch that
 * entwine_last_status has not yet collected is returned as ENTWINE_ERR_TIMEOUT /
 * ENTWINE_ERR_INTERNAL by that later query, never by a trap.
 * CUDA graphs: entwine_gemm_rs, entwine_gemm_rs_norm, entwine_gemm_only and
 * entwine_comm_only may be called on a capturing stream once the plan has made one launch of
 * that kind outside a capture (the first launch allocates; a capture before it returns
 * ENTWINE_ERR_INVALID).  A replay runs with the pointers and the flag value of the capture,
 * so a captured call is preceded by a small kernel that clears the plan's flags, list heads
 * and status, and so is every later call of that plan.  Replays of one plan must not overlap
 * each other or its other launches; entwine_last_status after a replay reports that replay
 * if the captured call was the plan's latest call.
 */
int entwine_gemm_rs(entwine_plan_t plan, const void* A, const void* B,
                    const void* peer_partials, void* out_shard, void* send_bufs,
                    void* stream);

/*
 * entwine_gemm_rs_host - the same call for HOST buffers (same layouts, always contiguous: the
 * leading-dimension options apply to device operands only): copies A, B and
 * rows [r*R,(r+1)*R) of each peer partial to plan-owned device staging buffers, runs the
 * fused kernel, copies out_shard and send_bufs back and synchronises the plan's internal
 * stream before returning.  Pinned host memory makes the copies asynchronous with each
 * other but is not required.  Errors as entwine_gemm_rs, plus a pending device status.
 */
int entwine_gemm_rs_host(entwine_plan_t plan, const void* A, const void* B,
                         const void* peer_partials, void* out_shard, void* send_bufs);

/*
 * entwine_gemm_rs_host_begin / entwine_gemm_rs_host_wait - the host-buffer call as a pipeline
 * of depth two.  _begin enqueues the copies up, the fused call and the copies down of one call
 * on streams of the library (two staging sets on the device, used alternately) and returns;
 * _wait blocks until the oldest call that has not been waited for has delivered out_shard and
 * send_bufs (and returns at once if there is none).  With pinned host buffers the copies up
 * of one call overlap the copies down of the call before it.  At most two calls may be
 * outstanding: a third _begin without a _wait returns ENTWINE_ERR_INVALID.  The host buffers
 * of a call must stay untouched until its _wait.  Device-side failures are reported by
 * entwine_last_status, as for entwine_gemm_rs.
 */
int entwine_gemm_rs_host_begin(entwine_plan_t plan, const void* A, const void* B,
                               const void* peer_partials, void* out_shard, void* send_bufs);
int entwine_gemm_rs_host_wait(entwine_plan_t plan);

/*
 * entwine_gemm_rs_norm - the fused call followed, inside the same launch, by the rest of the
 * attention-output layer's chain (Sec. 5.2.3: GEMM + ReduceScatter, then residual addition and
 * RMSNorm).  The reduction of an owned tile adds residual[R][N] to the rank-order fp32 sum and
 * rounds once: hidden_out[R][N] (bf16) is the new residual stream and takes the place of
 * out_shard.  When all tiles of a band of 128 rows are reduced the band's rows are complete,
 * and its tiles are normalised by whichever CTAs are free:
 *   norm_out[i][j] = bf16( hidden_out[i][j] * rsqrt(mean_j(hidden_out[i][:]^2) + eps) * weight[j] ),
 * computed in fp32 from the stored bf16 hidden values (row sums of squares are accumulated in a
 * fixed order: results are bitwise reproducible).  send_bufs as in entwine_gemm_rs.
 * residual, weight[N], hidden_out, norm_out: device pointers, bf16, 16-byte aligned; eps >= 0.
 * Errors as entwine_gemm_rs; ENTWINE_ERR_INVALID also if the plan has more consumer lists than
 * consumer CTAs (ENTWINE_OPT_LISTS).  Not available through the host-buffer or the
 * no-allocation entry points.
 */
int entwine_gemm_rs_norm(entwine_plan_t plan, const void* A, const void* B,
                         const void* peer_partials, const void* residual, const void* weight,
                         float eps, void* hidden_out, void* norm_out, void* send_bufs,
                         void* stream);

/*
 * entwine_gemm_only - the producer alone on all SMs (no consumer work): fills the plan's
 * partial-output workspace and publishes the flags.  Gives the uncontended GEMM time of the
 * overlap-efficiency ratio (Sec. 5.2.1, App. C).  A, B device pointers.
 */
int entwine_gemm_only(entwine_plan_t plan, const void* A, const void* B, void* stream);

/*
 * entwine_comm_only - the consumer alone with every input already available (App. A):
 * all flags are treated as published and n_ctas communication CTAs (0 = one per SM) walk
 * the task lists.  partial = device pointer to a bf16 C[M,N] to consume, or NULL for the
 * plan's own workspace (as left by the last producer run).  With partial produced by a
 * library GEMM this is the second half of the unfused GEMM-then-ReduceScatter sequence.
 */
int entwine_comm_only(entwine_plan_t plan, const void* partial, const void* peer_partials,
                      void* out_shard, void* send_bufs, int n_ctas, void* stream);

/*
 * entwine_read_partial - copy the plan's partial-output workspace C[M,N] (bf16) to a
 * device buffer `dst` on `stream` (for checking the producer by itself).
 */
int entwine_read_partial(entwine_plan_t plan, void* dst, void* stream);

/*
 * entwine_plan_export - write one of the plan's integer tables to host memory.
 *   what      ENTWINE_EXPORT_*
 *   host_buf  host pointer, or NULL to query the size only
 *   bytes     in: capacity of host_buf; out: bytes needed / written
 * Errors: ENTWINE_ERR_INVALID (unknown table, or capacity too small: *bytes is still set).
 */
int entwine_plan_export(entwine_plan_t plan, int what, void* host_buf, size_t* bytes);

/*
 * entwine_last_status - synchronise the stream of the plan's last launch and read its
 * status block into out[8]:
 *   0 code (ENTWINE_OK / ENTWINE_ERR_TIMEOUT / ENTWINE_ERR_INTERNAL), 1 CTA that reported,
 *   2 task or block it was on, 3 flags published, 4 tiles reduced, 5 tiles pushed,
 *   6 T_G: ns from the first CTA's start to the last producer block's completion (Eq. 3),
 *   7 T_end: ns from the first CTA's start to the last CTA's exit (end-to-end, Sec. 3.2).
 * Returns out[0].  Clears the pending status.
 */
int entwine_last_status(entwine_plan_t plan, int64_t out[8]);

/*
 * entwine_last_sm_clock - how fast the SMs really ran during the launch that the last
 * entwine_last_status call reported: out[0] = SM cycles and out[1] = nanoseconds that CTA 0
 * spent in the kernel (cycle counter against the global timer).  cycles / ns = GHz.  Times
 * measured on a power-limited part are read against this clock, not the nominal one.  Host
 * only (no synchronisation); zeros before the first status read.
 */
int entwine_last_sm_clock(entwine_plan_t plan, int64_t out[2]);

/*
 * entwine_gemm_rs_static - entwine_gemm_rs for callers that must not allocate.  (The paper
 * has no counterpart; this entry point exists for the library's users only.)
 *
 * Who needs it: code that runs where device allocation is forbidden or unaffordable - inside
 * a region that an application has declared allocation-free (a serving loop with a frozen
 * memory plan, a real-time path where cudaMalloc's implicit device synchronisation or its
 * latency is unacceptable), or a host that has handed all device memory to another
 * allocator and has nothing left for cudaMalloc to give.  entwine_gemm_rs allocates its
 * workspace with cudaMalloc at a plan's first launch; this variant never calls cudaMalloc,
 * cudaFree or any allocating routine.
 *
 * Instead of plan-owned memory it uses one fixed array inside the library image (9 MiB of
 * device memory, present on every GPU that loads the library until the process exits) for
 * the partial output C[M,N], the tile flags, the task table and the status block.  Limits:
 * M*N*2 bytes <= 8 MiB (for example 2048 x 2048) and control tables <= 1 MiB; a larger
 * problem is rejected with ENTWINE_ERR_TOO_LARGE before anything is enqueued.
 *
 * Arguments as entwine_gemm_rs (all device pointers; `stream` a cudaStream_t), plus
 *   status_out  NULL, or a host array of 8 values: the call then synchronises `stream` and
 *               writes what entwine_last_status would (code, CTA, where, flags published,
 *               tiles reduced, tiles pushed, T_G ns, T_end ns) and returns the code.
 * The plan supplies the shape, order, budget and options; its own workspace is not touched
 * and entwine_last_status does not report this call.  With status_out == NULL nothing reports it:
 * a device-side timeout or index failure of that call then goes unnoticed (its outputs are
 * incomplete), so pass status_out wherever the result matters.  Options that this entry point
 * does not implement (a release group other than 1, a withheld peer flag) make it return
 * ENTWINE_ERR_INVALID, and so does a `stream` that is being captured into a CUDA graph (every call
 * uploads the plan's tables from host memory; for graphs use entwine_plan_set_workspace and
 * entwine_gemm_rs).
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) and
 * caches it per device: make that first call outside any stream capture.  All calls on a
 * device share the one array, which keeps whatever the previous call left: every call first
 * clears the flags, list heads and status on `stream`.  Two calls whose execution overlaps
 * on the GPU (different streams, or different plans at once) therefore race; serialise them.
 * Errors: ENTWINE_ERR_INVALID, ENTWINE_ERR_TOO_LARGE, ENTWINE_ERR_RESOURCES, ENTWINE_ERR_CUDA;
 * with status_out also ENTWINE_ERR_TIMEOUT / ENTWINE_ERR_INTERNAL from the device.
 */
int entwine_gemm_rs_static(entwine_plan_t plan, const void* A, const void* B,
                           const void* peer_partials, void* out_shard, void* send_bufs,
                           void* stream, int64_t* status_out);

/*
 * entwine_heap_bytes / entwine_gemm_rs_pull - the call of one rank when the W ranks run on GPUs
 * of their own (Sec. 4.1: partial outputs and flags live in a symmetric heap; Sec. 4.2: the
 * reducer waits for the flags of all W contributions and reads the peers' tiles itself).
 *
 * The heap is W segments, segment w belonging to rank w, mapped by every rank so that segment
 * w starts at heap + w * heap_stride (device pointer valid on the calling rank's GPU: its own
 * memory for w = rank, peer-mapped memory otherwise).  entwine_heap_bytes gives the least
 * size of a segment and, optionally, where its flag array starts; heap and heap_stride must
 * be multiples of 256 bytes, and the whole heap must be zero before the first call.
 * A segment holds two partial-output buffers [M][N] (bf16), used alternately by the parity of
 * `epoch`, and the flags [W sources][Q] (uint32) that the W ranks write for this rank's tiles.
 *
 * entwine_gemm_rs_pull(plan, A, B, heap, heap_stride, epoch, produce_only, out_shard, stream):
 * the producer stores the rank's partial into its own segment and, per finished tile, writes
 * `epoch` into the flag array of the tile's destination rank (a store into that rank's
 * segment, system scope); the consumer warps reduce the tiles of the rank's own partition:
 * they poll the rank's local flags until all W sources show a value >= epoch and read the W
 * contributions (own segment first, then the peers' in ascending rank order) into
 * out_shard[R][N].  There are no push tasks and no send buffers: the peers' reads are the
 * communication of Eq. 2.  `epoch` is the call's sequence number: the same on every rank,
 * 1, 2, 3, ... without gaps.  Two buffers suffice because a rank can finish call n+1 only
 * after every peer has started it, i.e. finished reading the buffers of call n.
 * produce_only != 0 runs the producer alone (out_shard may be NULL).
 * Not available: coarse release groups, the layer chain, capture into a CUDA graph (the
 * epoch is a launch parameter).  Errors as entwine_gemm_rs.
 * On one GPU the call is exercised rank by rank: a rank's consumer never waits for a kernel
 * that has not been launched if the other ranks' producers have run before it.
 */
int entwine_heap_bytes(entwine_plan_t plan, int64_t* segment_bytes, int64_t* flags_offset);
int entwine_gemm_rs_pull(entwine_plan_t plan, const void* A, const void* B, void* heap,
                         int64_t heap_stride, uint32_t epoch, int produce_only, void* out_shard,
                         void* stream);

/* entwine_destroy - free the plan and everything it owns (synchronises its last stream). */
int entwine_destroy(entwine_plan_t plan);

/* entwine_strerror - static, human-readable text for a return code. */
const char* entwine_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* ENTWINE_H_ */
