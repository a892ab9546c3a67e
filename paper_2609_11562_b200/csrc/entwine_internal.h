// Internal declarations shared by the host planner and the CUDA launch code.
#pragma once

#include <cstddef>
#include <cstdint>
#include <vector>

#include "entwine.h"

namespace entwine {

constexpr int kTile = 128;  // edge of the square reduction tile (Sec. 4.2)

// One consumer task as the device reads it (32 bytes).  Offsets are in elements.
struct Task {
  int32_t kind;      // 0 reduce, 1 push
  int32_t d;         // destination partition of the tile
  int32_t t;         // tile index inside the partition
  int32_t slot;      // push: send_bufs slot q(d); reduce: -1
  int64_t src_off;   // first element of the tile in the partial C[M,N]
  int64_t dst_off;   // first element in out_shard[R,N] or send_bufs[slot][R,N]
};
static_assert(sizeof(Task) == 32, "Task layout");

// Sizes that follow from (M, N, W, BN).
struct Geometry {
  int64_t M = 0, N = 0, K = 0;
  int W = 0, BN = 256;
  int64_t R = 0;
  int cpb = 0, nTn = 0, nBn = 0, rowsT = 0, Lb = 0, P_blk = 0, Q = 0;
};

// Host-side schedule of one plan: everything entwine_plan_export can return.
struct HostTables {
  std::vector<int32_t> order;      // [P_blk][4] mb, nb, d, l
  std::vector<int32_t> tiles;      // [P_blk][cpb]
  std::vector<int32_t> flag_seq;   // [P_blk*cpb][3]
  std::vector<int32_t> list_offs;  // [x+1]
  std::vector<int64_t> tasks;      // [n_tasks][8]
  std::vector<int64_t> peer_offs;  // [n_reduce][W-1]
  std::vector<Task> dev_tasks;     // [n_tasks], same rows as `tasks`
  std::vector<Task> pull_tasks;          // pull mode: the reduce tasks of dev_tasks, list by list
  std::vector<int32_t> pull_list_offs;   // [x+1]
  int64_t counts[16] = {0};
};

// Device status block, two slots used alternately by successive launches.
struct StatusSlot {
  unsigned long long code_cta_task;  // 0 = ok; else (code & 0xff) | cta << 8 | task << 32
  unsigned long long flags_published;
  unsigned long long tiles_reduced;
  unsigned long long tiles_pushed;
  unsigned long long t_start;     // min globaltimer at CTA entry
  unsigned long long t_gemm_end;  // max globaltimer after a producer CTA's last block
  unsigned long long t_end;       // max globaltimer at CTA exit
  unsigned long long clock;       // CTA 0: SM cycles << 32 | ns between its start and its exit
};
static_assert(sizeof(StatusSlot) == 64, "StatusSlot layout");

bool make_geometry(int64_t M, int64_t N, int64_t K, int W, int BN, Geometry* g);
// Block p of the logical order -> block row, block column, destination, within-partition index.
void block_of_position(const Geometry& g, int order, int p, int* mb, int* nb, int* d, int* l);
void build_tables(const Geometry& g, int order, int r, int x, int n_gemm_ctas, int n_comm_ctas,
                  HostTables* out);

// Launch modes of the one kernel.
enum Mode { MODE_FUSED = 0, MODE_GEMM_ONLY = 1, MODE_COMM_ONLY = 2 };

struct DeviceState;  // owned by the CUDA side

struct Plan {
  Geometry g;
  int order = ENTWINE_ORDER_INTERLEAVED;
  int n_comm_sms = 0;
  int rank = 0;
  int num_sms = 148;
  bool num_sms_overridden = false;
  int tail_help = 1;
  int prefetch = 0;         // look-ahead L2 prefetch of peer tiles (measured: no gain)
  int l2_hints = 3;         // bit 0: evict-first on the consumer's TMA traffic, bit 1: evict-last on operands
  int lists_opt = 0;        // number of consumer lists x, 0 = one per consumer CTA
  int release_group = 1;    // blocks released together; -1 per destination partition, -2 whole output
  int stages = 0;           // operand-ring stages of the producer, 0 = choose
  int kpb = 0;              // k-blocks (64 elements of K) per stage, 0 = choose
  int split_opt = 1;        // a last wave that fills at most half of the CTA pairs runs as half-width units
  int64_t lda = 0, ldb = 0; // leading dimensions of A and B in elements, 0 = contiguous
  int peers_compact = 0;    // (set around a launch by the host-buffer calls) peers are staged as [W-1][R][N]
  int b_kn = 0;             // 1: B is [K_local, N] (N contiguous) instead of [N, K_local]
  int colocate = 1;         // consumer warps of a producer CTA work while it produces
  int reg_consumer = 0;     // 1: ... from registers (plain loads and stores) instead of a shared-memory TMA ring
  int consumer_tma = 1;     // 0: the consumer uses plain loads and stores only, to the end (implies the register path)
  int pair_opt = 1;         // allow CTA-pair (256 x 256) producer tiles
  bool pair = false;        // pair tiles in use for this plan
  int poison = 0;
  int64_t wait_budget_ns = 2000000000LL;
  int64_t withhold_peer = -1;
  bool launched = false;
  bool tables_built = false;
  int x = 0;            // number of consumer lists
  int n_gemm_ctas = 0;  // producer CTAs of the fused launch
  int n_comm_ctas = 0;  // dedicated consumer CTAs of the fused launch
  HostTables tables;
  void* ws_ptr = nullptr;   // caller-provided device workspace (entwine_plan_set_workspace), or null
  size_t ws_bytes = 0;
  DeviceState* dev = nullptr;
};

// Resolve SM-dependent sizes and (re)build host tables.  Returns an ENTWINE_* code.
int finalize_plan(Plan* p);

// CUDA side (entwine_kernels.cu).
int device_sm_count();  // -1 if there is no usable device
void device_release(Plan* p);

}  // namespace entwine

struct entwine_plan_s : public entwine::Plan {};
