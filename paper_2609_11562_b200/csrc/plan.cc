// Host planner: shape validation, the logical block order (Sec. 3.1, Eq. 1), consumer task
// lists (Sec. 3.1 "Matching task order", Sec. 3.2 "Communication budget"), index maps and
// the integer tables that entwine_plan_export returns.  No CUDA calls in this file.
#include <algorithm>
#include <cstring>
#include <new>

#include "entwine_internal.h"

namespace entwine {

bool make_geometry(int64_t M, int64_t N, int64_t K, int W, int BN, Geometry* g) {
  if (W < 2 || W > 64) return false;
  if (BN != 128 && BN != 256) return false;
  if (M <= 0 || N <= 0 || K <= 0) return false;
  if (M % (int64_t(kTile) * W) != 0) return false;  // equal partitions of whole tile rows
  if (N % kTile != 0 || N % BN != 0) return false;
  if (K % 16 != 0) return false;
  if (M > (int64_t(1) << 30) || N > (int64_t(1) << 30) || K > (int64_t(1) << 30)) return false;
  g->M = M; g->N = N; g->K = K; g->W = W; g->BN = BN;
  g->R = M / W;
  g->cpb = BN / kTile;
  g->nTn = int(N / kTile);
  g->nBn = int(N / BN);
  g->rowsT = int(g->R / kTile);
  int64_t Lb = int64_t(g->rowsT) * g->nBn;
  int64_t Q = int64_t(g->rowsT) * g->nTn;
  if (Lb * W > (int64_t(1) << 24) || Q * W > (int64_t(1) << 26)) return false;
  g->Lb = int(Lb);
  g->P_blk = int(Lb * W);
  g->Q = int(Q);
  return true;
}

void block_of_position(const Geometry& g, int order, int p, int* mb, int* nb, int* d, int* l) {
  int dest, ell;
  if (order == ENTWINE_ORDER_INTERLEAVED) {  // Eq. 1
    dest = p % g.W;
    ell = p / g.W;
  } else if (order == ENTWINE_ORDER_M_MAJOR) {  // rows of the whole output first
    const int rows_all = g.W * g.rowsT;
    const int row_all = p % rows_all, col_all = p / rows_all;
    dest = row_all / g.rowsT;
    ell = (row_all - dest * g.rowsT) * g.nBn + col_all;
  } else {  // partition-grouped traversal (Fig. 1, top)
    dest = p / g.Lb;
    ell = p - dest * g.Lb;
  }
  // inside a partition the block column runs fastest
  *d = dest;
  *l = ell;
  *mb = dest * g.rowsT + ell / g.nBn;
  *nb = ell % g.nBn;
}

namespace {
struct Pending {
  int32_t kind, d, t, k;
};
}  // namespace

void build_tables(const Geometry& g, int order, int r, int x, int n_gemm_ctas, int n_comm_ctas,
                  HostTables* out) {
  const int P = g.P_blk, cpb = g.cpb, W = g.W, Q = g.Q;
  out->order.assign(size_t(P) * 4, 0);
  out->tiles.assign(size_t(P) * cpb, 0);
  out->flag_seq.assign(size_t(P) * cpb * 3, 0);

  // Consumer lists.  Reduce tasks: tile t of the own partition goes to list t mod min(x, Q).
  // Push tasks: the u-th non-owned tile in publication order goes to list u mod
  // min(x, (W-1)Q).  Each list is kept sorted by publication index k.
  std::vector<std::vector<Pending>> lists(static_cast<size_t>(x));
  const int64_t n_push_total = int64_t(W - 1) * Q;
  const int x_r = int(std::min<int64_t>(x, Q));
  const int x_p = int(std::min<int64_t>(x, n_push_total));
  int64_t u = 0;
  for (int p = 0; p < P; ++p) {
    int mb, nb, d, l;
    block_of_position(g, order, p, &mb, &nb, &d, &l);
    int32_t* o = &out->order[size_t(p) * 4];
    o[0] = mb; o[1] = nb; o[2] = d; o[3] = l;
    const int tile_row = mb - d * g.rowsT;
    for (int c = 0; c < cpb; ++c) {
      const int t = tile_row * g.nTn + nb * cpb + c;  // row-major over the partition's tiles
      const int k = p * cpb + c;
      out->tiles[size_t(p) * cpb + c] = t;
      int32_t* f = &out->flag_seq[size_t(k) * 3];
      f[0] = r; f[1] = d; f[2] = t;
      if (d == r) {
        lists[size_t(t % x_r)].push_back({0, d, t, k});
      } else {
        lists[size_t(u % x_p)].push_back({1, d, t, k});
        ++u;
      }
    }
  }

  out->pull_list_offs.assign(size_t(x) + 1, 0);
  out->pull_tasks.clear();
  out->list_offs.assign(size_t(x) + 1, 0);
  out->tasks.clear();
  out->peer_offs.clear();
  out->dev_tasks.clear();
  int64_t n_reduce = 0, n_push = 0;
  for (int j = 0; j < x; ++j) {
    auto& lst = lists[size_t(j)];
    std::stable_sort(lst.begin(), lst.end(),
                     [](const Pending& a, const Pending& b) { return a.k < b.k; });
    for (const Pending& e : lst) {
      const int64_t trow = e.t / g.nTn, tcol = e.t % g.nTn;
      const int64_t src = (int64_t(e.d) * g.R + trow * kTile) * g.N + tcol * kTile;
      const int64_t dst = (trow * kTile) * g.N + tcol * kTile;
      const int slot = (e.kind == 1) ? (e.d < r ? e.d : e.d - 1) : -1;
      const int64_t row[8] = {e.kind, e.d, e.t, e.k, j, src, slot, dst};
      out->tasks.insert(out->tasks.end(), row, row + 8);
      Task dt;
      dt.kind = e.kind; dt.d = e.d; dt.t = e.t; dt.slot = slot;
      dt.src_off = src; dt.dst_off = dst;
      out->dev_tasks.push_back(dt);
      if (e.kind == 0) out->pull_tasks.push_back(dt);
      if (e.kind == 0) {
        for (int w = 0; w < W; ++w) {
          if (w == r) continue;
          const int64_t q = (w < r) ? w : w - 1;
          out->peer_offs.push_back(q * g.M * g.N + src);
        }
        ++n_reduce;
      } else {
        ++n_push;
      }
    }
    out->list_offs[size_t(j) + 1] = int32_t(out->dev_tasks.size());
    out->pull_list_offs[size_t(j) + 1] = int32_t(out->pull_tasks.size());
  }

  const int64_t tile_bytes = int64_t(kTile) * kTile * 2;
  int64_t* c = out->counts;
  c[0] = P; c[1] = Q; c[2] = cpb; c[3] = x;
  c[4] = n_reduce + n_push; c[5] = n_reduce; c[6] = n_push;
  c[7] = int64_t(P) * cpb;            // flags published by rank r per call
  c[8] = int64_t(W - 1) * Q;          // peer flags pre-published
  c[9] = int64_t(W) * n_reduce + n_push;  // minimum flag reads
  c[10] = n_reduce * (W - 1) * tile_bytes;
  c[11] = (n_reduce + n_push) * tile_bytes;
  c[12] = n_push * tile_bytes;
  c[13] = n_reduce * tile_bytes;
  c[14] = n_gemm_ctas;
  c[15] = n_comm_ctas;
}

int finalize_plan(Plan* p) {
  // The device copies of the tables (made by the first call that needs the device, which may be
  // entwine_read_partial or a launch that failed later on) describe the plan as it was: drop them,
  // the next call uploads the rebuilt tables.
  if (p->dev) device_release(p);
  if (!p->num_sms_overridden) {
    int sms = device_sm_count();
    p->num_sms = sms > 0 ? sms : 148;
  }
  if (p->n_comm_sms < 0 || p->n_comm_sms >= p->num_sms) return ENTWINE_ERR_INVALID;
  if (p->rank < 0 || p->rank >= p->g.W) return ENTWINE_ERR_INVALID;
  // CTA-pair producer tiles need two blocks that share a block column: positions 2u, 2u+1 of
  // the interleaved order (W even) or vertically adjacent blocks of a partition (row-major,
  // even number of tile rows per partition).
  const Geometry& g = p->g;
  p->pair = p->pair_opt && g.BN == 256 && p->num_sms >= 2 &&
            ((p->order == ENTWINE_ORDER_INTERLEAVED && g.W % 2 == 0) ||
             (p->order == ENTWINE_ORDER_ROW_MAJOR && g.rowsT % 2 == 0) ||
             (p->order == ENTWINE_ORDER_M_MAJOR && (g.W * g.rowsT) % 2 == 0));
  if (p->n_comm_sms == 0) {
    // non-overlapped use of all SMs: every CTA produces, then consumes
    p->n_comm_ctas = 0;
    p->n_gemm_ctas = p->pair ? (p->num_sms & ~1) : p->num_sms;
    p->x = p->n_gemm_ctas;
  } else {
    p->n_comm_ctas = p->n_comm_sms;
    p->n_gemm_ctas = p->num_sms - p->n_comm_sms;
    if (p->pair) p->n_gemm_ctas &= ~1;
    if (p->n_gemm_ctas < 1) return ENTWINE_ERR_INVALID;
    p->x = p->n_comm_sms;
  }
  if (p->lists_opt > 0) p->x = p->lists_opt;
  build_tables(p->g, p->order, p->rank, p->x, p->n_gemm_ctas, p->n_comm_ctas, &p->tables);
  p->tables_built = true;
  return ENTWINE_OK;
}

}  // namespace entwine

using entwine::Plan;

extern "C" {

int entwine_plan(entwine_plan_t* plan, int64_t M, int64_t N, int64_t K_local, int W,
                 int tile_order, int n_comm_sms) {
  if (!plan) return ENTWINE_ERR_INVALID;
  *plan = nullptr;
  if (tile_order != ENTWINE_ORDER_ROW_MAJOR && tile_order != ENTWINE_ORDER_INTERLEAVED &&
      tile_order != ENTWINE_ORDER_M_MAJOR)
    return ENTWINE_ERR_INVALID;
  entwine::Geometry g;
  if (!entwine::make_geometry(M, N, K_local, W, 256, &g)) {
    // BN = 256 is only the default; a shape that needs BN = 128 is still plannable
    if (!entwine::make_geometry(M, N, K_local, W, 128, &g)) return ENTWINE_ERR_INVALID;
  }
  entwine_plan_s* p = new (std::nothrow) entwine_plan_s();
  if (!p) return ENTWINE_ERR_RESOURCES;
  p->g = g;
  p->order = tile_order;
  p->n_comm_sms = n_comm_sms;
  int rc = entwine::finalize_plan(p);
  if (rc != ENTWINE_OK) {
    delete p;
    return rc;
  }
  *plan = p;
  return ENTWINE_OK;
}

int entwine_set_option(entwine_plan_t plan, int key, int64_t value) {
  if (!plan) return ENTWINE_ERR_INVALID;
  Plan* p = plan;
  switch (key) {
    case ENTWINE_OPT_RANK:
      if (p->launched || value < 0 || value >= p->g.W) return ENTWINE_ERR_INVALID;
      p->rank = int(value);
      return entwine::finalize_plan(p);
    case ENTWINE_OPT_BLOCK_N: {
      if (p->launched) return ENTWINE_ERR_INVALID;
      entwine::Geometry g;
      if (!entwine::make_geometry(p->g.M, p->g.N, p->g.K, p->g.W, int(value), &g))
        return ENTWINE_ERR_INVALID;
      p->g = g;
      return entwine::finalize_plan(p);
    }
    case ENTWINE_OPT_WAIT_BUDGET_NS:
      if (value <= 0) return ENTWINE_ERR_INVALID;
      p->wait_budget_ns = value;
      return ENTWINE_OK;
    case ENTWINE_OPT_TAIL_HELP:
      if (value != 0 && value != 1) return ENTWINE_ERR_INVALID;
      p->tail_help = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_WITHHOLD_PEER:
      if (value >= 0) {
        int64_t w = value >> 32, t = value & 0xffffffffLL;
        if (w >= p->g.W || w == p->rank || t >= p->g.Q) return ENTWINE_ERR_INVALID;
      } else if (value != -1) {
        return ENTWINE_ERR_INVALID;
      }
      p->withhold_peer = value;
      return ENTWINE_OK;
    case ENTWINE_OPT_NUM_SMS: {
      if (p->launched || value < 1 || value > 4096) return ENTWINE_ERR_INVALID;
      int old = p->num_sms;
      bool old_over = p->num_sms_overridden;
      p->num_sms = int(value);
      p->num_sms_overridden = true;
      int rc = entwine::finalize_plan(p);
      if (rc != ENTWINE_OK) {
        p->num_sms = old;
        p->num_sms_overridden = old_over;
        entwine::finalize_plan(p);
      }
      return rc;
    }
    case ENTWINE_OPT_L2_HINTS:
      if (value < 0 || value > 3) return ENTWINE_ERR_INVALID;
      p->l2_hints = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_LISTS:
      if (p->launched || value < 0 || value > 4096) return ENTWINE_ERR_INVALID;
      p->lists_opt = int(value);
      return entwine::finalize_plan(p);
    case ENTWINE_OPT_RELEASE_GROUP:
      if (value == 0 || value < ENTWINE_RELEASE_WHOLE || value > (int64_t(1) << 24)) return ENTWINE_ERR_INVALID;
      p->release_group = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_STAGES:
      if (value < 0 || value > 6 || value == 1) return ENTWINE_ERR_INVALID;
      p->stages = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_CONSUMER_TMA:
      if (value != 0 && value != 1) return ENTWINE_ERR_INVALID;
      p->consumer_tma = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_B_LAYOUT:
      if (value != ENTWINE_B_LAYOUT_NK && value != ENTWINE_B_LAYOUT_KN) return ENTWINE_ERR_INVALID;
      if (p->b_kn != (value == ENTWINE_B_LAYOUT_KN ? 1 : 0)) p->ldb = 0;  // the pitch belonged to the other layout
      p->b_kn = value == ENTWINE_B_LAYOUT_KN ? 1 : 0;
      return ENTWINE_OK;
    case ENTWINE_OPT_SPLIT_LAST_WAVE:
      if (value != 0 && value != 1) return ENTWINE_ERR_INVALID;
      p->split_opt = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_REG_CONSUMER:
      if (value != 0 && value != 1) return ENTWINE_ERR_INVALID;
      p->reg_consumer = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_KBLOCKS_PER_STAGE:
      if (value < 0 || value > 2) return ENTWINE_ERR_INVALID;
      p->kpb = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_LDA:
    case ENTWINE_OPT_LDB:
      // rows start on 16-byte boundaries (that they do not overlap is checked at the launch, against
      // the layout in force then)
      if (value != 0 && (value < 8 || value % 8 != 0 || value > (int64_t(1) << 36))) return ENTWINE_ERR_INVALID;
      if (value != 0 && key == ENTWINE_OPT_LDA && value < p->g.K) return ENTWINE_ERR_INVALID;
      if (value != 0 && key == ENTWINE_OPT_LDB && value < (p->b_kn ? p->g.N : p->g.K)) return ENTWINE_ERR_INVALID;
      (key == ENTWINE_OPT_LDA ? p->lda : p->ldb) = value;
      return ENTWINE_OK;
    case ENTWINE_OPT_PREFETCH:
      if (value != 0 && value != 1) return ENTWINE_ERR_INVALID;
      p->prefetch = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_COLOCATE:
      if (value != 0 && value != 1) return ENTWINE_ERR_INVALID;
      p->colocate = int(value);
      return ENTWINE_OK;
    case ENTWINE_OPT_PAIR_CTAS:
      if (p->launched || (value != 0 && value != 1)) return ENTWINE_ERR_INVALID;
      p->pair_opt = int(value);
      return entwine::finalize_plan(p);
    case ENTWINE_OPT_POISON_PARTIAL:
      if (value != 0 && value != 1) return ENTWINE_ERR_INVALID;
      p->poison = int(value);
      return ENTWINE_OK;
    default:
      return ENTWINE_ERR_INVALID;
  }
}

int entwine_plan_export(entwine_plan_t plan, int what, void* host_buf, size_t* bytes) {
  if (!plan || !bytes) return ENTWINE_ERR_INVALID;
  const entwine::HostTables& t = plan->tables;
  const void* src = nullptr;
  size_t n = 0;
  switch (what) {
    case ENTWINE_EXPORT_COUNTS:    src = t.counts;           n = sizeof(t.counts); break;
    case ENTWINE_EXPORT_ORDER:     src = t.order.data();     n = t.order.size() * 4; break;
    case ENTWINE_EXPORT_TILES:     src = t.tiles.data();     n = t.tiles.size() * 4; break;
    case ENTWINE_EXPORT_FLAG_SEQ:  src = t.flag_seq.data();  n = t.flag_seq.size() * 4; break;
    case ENTWINE_EXPORT_LIST_OFFS: src = t.list_offs.data(); n = t.list_offs.size() * 4; break;
    case ENTWINE_EXPORT_TASKS:     src = t.tasks.data();     n = t.tasks.size() * 8; break;
    case ENTWINE_EXPORT_PEER_OFFS: src = t.peer_offs.data(); n = t.peer_offs.size() * 8; break;
    default: return ENTWINE_ERR_INVALID;
  }
  size_t cap = *bytes;
  *bytes = n;
  if (!host_buf) return ENTWINE_OK;
  if (cap < n) return ENTWINE_ERR_INVALID;
  if (n) std::memcpy(host_buf, src, n);
  return ENTWINE_OK;
}

int entwine_destroy(entwine_plan_t plan) {
  if (!plan) return ENTWINE_ERR_INVALID;
  entwine::device_release(plan);
  delete plan;
  return ENTWINE_OK;
}

const char* entwine_strerror(int code) {
  switch (code) {
    case ENTWINE_OK: return "ok";
    case ENTWINE_ERR_INVALID: return "invalid shape, argument, option or call order";
    case ENTWINE_ERR_RESOURCES: return "not enough SMs or shared memory for a co-resident launch";
    case ENTWINE_ERR_CUDA: return "CUDA call failed or no CUDA device";
    case ENTWINE_ERR_TIMEOUT: return "a device-side wait ran out of its budget";
    case ENTWINE_ERR_INTERNAL: return "a device-side index check failed";
    case ENTWINE_ERR_TOO_LARGE:
      return "problem exceeds the fixed scratch of entwine_gemm_rs_static (M*N*2 <= 8 MiB, tables <= 1 MiB)";
    default: return "unknown entwine error code";
  }
}

}  // extern "C"
