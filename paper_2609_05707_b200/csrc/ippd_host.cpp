// Host-only part of the IPPD library: integer layout tables and the per-step split-KV scheduler.
// No CUDA call is made from this file.
#include <algorithm>
#include <climits>
#include <cstring>

#include "ippd_internal.h"

static thread_local std::string g_last_error;
void ippd_set_error(const std::string& msg) { g_last_error = msg; }
extern "C" const char* ippd_last_error(void) { return g_last_error.c_str(); }

static const int kTargetCtas = 148 * 2 * 4;  // CTAs wanted per launch: SMs x resident CTAs x waves
static const int kMinTilesPerSplit = 4;

int IppdHostLayout::kernel_path() const { return opt_kernel == 0 ? IPPD_DEFAULT_KERNEL : opt_kernel; }
int IppdHostLayout::rows_per_block() const { return kernel_path() >= 2 ? 128 : 64; }
// questions per row block: the tensor-core path keeps at most 64 questions per block
static int questions_per_block(const IppdHostLayout& L) {
  int qpr = L.rows_per_block() / L.G;
  return L.kernel_path() >= 2 ? std::min(qpr, 64) : qpr;
}

static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

int ippd_host_build(const ippd_geometry_t* g, int32_t shared_len, int32_t B, const int32_t* ctx_len,
                    const int32_t* q_count, const int32_t* q_len, const int32_t* max_new, IppdHostLayout* L) {
  if (!g || !ctx_len || !q_count || !q_len || !max_new || !L) {
    ippd_set_error("ippd_build_layout: NULL argument");
    return IPPD_ERR_INVALID_ARG;
  }
  if (B < 1) { ippd_set_error("ippd_build_layout: n_prompts must be >= 1"); return IPPD_ERR_INVALID_ARG; }
  if (shared_len < 0) { ippd_set_error("ippd_build_layout: shared_len < 0"); return IPPD_ERR_INVALID_ARG; }
  if (g->n_layers < 1 || g->n_kv_heads < 1 || g->n_q_heads < 1 || g->n_q_heads % g->n_kv_heads != 0) {
    ippd_set_error("ippd_build_layout: bad head counts / layers");
    return IPPD_ERR_INVALID_ARG;
  }
  int G = g->n_q_heads / g->n_kv_heads;
  if (!(G == 1 || G == 2 || G == 4 || G == 8 || G == 16)) {
    ippd_set_error("ippd_build_layout: group size Hq/Hkv must be 1, 2, 4, 8 or 16");
    return IPPD_ERR_INVALID_ARG;
  }
  if (g->head_dim != 64 && g->head_dim != 128) {
    ippd_set_error("ippd_build_layout: head_dim must be 64 or 128");
    return IPPD_ERR_INVALID_ARG;
  }
  if (!(g->rope_theta > 1.0)) { ippd_set_error("ippd_build_layout: rope_theta must be > 1"); return IPPD_ERR_INVALID_ARG; }
  if (g->branch_align < IPPD_TILE_TOKENS || g->branch_align % IPPD_TILE_TOKENS != 0) {
    ippd_set_error("ippd_build_layout: branch_align must be a positive multiple of IPPD_TILE_TOKENS");
    return IPPD_ERR_INVALID_ARG;
  }
  if (g->out_dtype != IPPD_BF16 && g->out_dtype != IPPD_F32) {
    ippd_set_error("ippd_build_layout: out_dtype must be IPPD_BF16 or IPPD_F32");
    return IPPD_ERR_INVALID_ARG;
  }
  try {
    L->geom = *g;
    L->shared_len = shared_len;
    L->n_shared_tiles = (int32_t)ceil_div(shared_len, IPPD_TILE_TOKENS);
    L->B = B;
    L->G = G;
    L->ctx_len.assign(ctx_len, ctx_len + B);
    L->q_count.assign(q_count, q_count + B);
    L->q_begin.assign(B + 1, 0);
    int64_t nq = 0;
    for (int b = 0; b < B; ++b) {
      if (ctx_len[b] < 0) { ippd_set_error("ippd_build_layout: ctx_len < 0"); return IPPD_ERR_INVALID_ARG; }
      if (q_count[b] < 1) { ippd_set_error("ippd_build_layout: q_count < 1"); return IPPD_ERR_INVALID_ARG; }
      nq += q_count[b];
      if (nq > (1 << 24)) { ippd_set_error("ippd_build_layout: too many questions"); return IPPD_ERR_INVALID_ARG; }
      L->q_begin[b + 1] = (int32_t)nq;
    }
    L->NQ = (int32_t)nq;
    L->q_len.assign(q_len, q_len + nq);
    L->max_new.assign(max_new, max_new + nq);
    L->prompt_of.resize(nq);
    L->branch_off.assign(nq + 1, 0);
    L->branch_tile_off.assign(nq + 1, 0);
    L->hdr_begin.assign(B + 1, 0);
    L->ctx_tile_off.assign(B + 1, L->n_shared_tiles);  // the shared instruction owns the first tiles of the cache
    int64_t max_pos = 0, hdr = shared_len;
    L->hdr_begin[0] = shared_len;
    for (int b = 0; b < B; ++b) {
      L->ctx_tile_off[b + 1] = L->ctx_tile_off[b] + (int32_t)ceil_div(ctx_len[b], IPPD_TILE_TOKENS);
      hdr += ctx_len[b];
      for (int k = L->q_begin[b]; k < L->q_begin[b + 1]; ++k) {
        if (q_len[k] < 1 || max_new[k] < 1) {
          ippd_set_error("ippd_build_layout: q_len and max_new must be >= 1");
          return IPPD_ERR_INVALID_ARG;
        }
        int64_t last = (int64_t)shared_len + ctx_len[b] + q_len[k] + max_new[k];
        if (last >= INT32_MAX) { ippd_set_error("ippd_build_layout: position overflows int32"); return IPPD_ERR_INVALID_ARG; }
        max_pos = std::max(max_pos, last - 1);
        L->prompt_of[k] = b;
        int64_t cap = ceil_div((int64_t)q_len[k] + max_new[k], g->branch_align) * g->branch_align;
        L->branch_off[k + 1] = L->branch_off[k] + cap;
        hdr += q_len[k];
      }
      L->hdr_begin[b + 1] = hdr;
    }
    L->max_pos = (int32_t)max_pos;
    L->n_ctx_tiles = L->ctx_tile_off[B];
    int64_t n_tiles = L->n_ctx_tiles + L->branch_off[nq] / IPPD_TILE_TOKENS;
    if (n_tiles >= INT32_MAX) { ippd_set_error("ippd_build_layout: cache too large"); return IPPD_ERR_INVALID_ARG; }
    L->n_tiles = n_tiles;
    for (int64_t k = 0; k <= nq; ++k)
      L->branch_tile_off[k] = (int32_t)(L->n_ctx_tiles + L->branch_off[k] / IPPD_TILE_TOKENS);
    // stacked-header metadata: the shared instruction (context id 0: everybody's), then per prompt its context
    // tokens and question blocks
    L->hdr_pos.resize(hdr); L->hdr_ctx.resize(hdr); L->hdr_qtn.resize(hdr);
    int64_t h = 0;
    for (int i = 0; i < shared_len; ++i, ++h) { L->hdr_pos[h] = i; L->hdr_ctx[h] = 0; L->hdr_qtn[h] = 0; }
    for (int b = 0; b < B; ++b) {
      for (int i = 0; i < ctx_len[b]; ++i, ++h) { L->hdr_pos[h] = shared_len + i; L->hdr_ctx[h] = b + 1; L->hdr_qtn[h] = 0; }
      for (int k = L->q_begin[b]; k < L->q_begin[b + 1]; ++k)
        for (int j = 0; j < q_len[k]; ++j, ++h) {
          L->hdr_pos[h] = shared_len + ctx_len[b] + j; L->hdr_ctx[h] = b + 1; L->hdr_qtn[h] = k + 1;
        }
    }
  } catch (const std::bad_alloc&) {
    ippd_set_error("ippd_build_layout: out of host memory");
    return IPPD_ERR_OOM;
  }
  return IPPD_OK;
}

int64_t ippd_host_max_rowblocks(const IppdHostLayout& L) {
  int qpr = questions_per_block(L);
  int64_t n = 0;
  for (int b = 0; b < L.B; ++b) n += ceil_div(L.q_count[b], qpr);
  return n;
}

int64_t ippd_host_max_units(const IppdHostLayout& L, int32_t layer_count) {
  int64_t nrb = ippd_host_max_rowblocks(L);
  if (L.opt_tiles_per_split > 0) {
    // every row block may stream its prompt's context plus all of its questions' branches
    int64_t tiles = 0;
    int qpr = questions_per_block(L);
    for (int b = 0; b < L.B; ++b) {
      tiles += ceil_div(L.q_count[b], qpr) * (L.n_shared_tiles + L.ctx_tile_off[b + 1] - L.ctx_tile_off[b]);
      tiles += L.branch_tile_off[L.q_begin[b + 1]] - L.branch_tile_off[L.q_begin[b]];
    }
    return nrb + ceil_div(tiles, L.opt_tiles_per_split);
  }
  int64_t per = std::max<int64_t>(1, (int64_t)L.geom.n_kv_heads * std::max(1, layer_count));
  return nrb + ceil_div(kTargetCtas, per) + 1;
}

int ippd_host_plan_step(const IppdHostLayout& L, const int32_t* active_q, const int32_t* answer_idx,
                        int32_t A, int32_t layer_count, IppdStepPlan* plan) {
  if (A < 0 || (A > 0 && (!active_q || !answer_idx))) {
    ippd_set_error("ippd_begin_step: bad active list");
    return IPPD_ERR_INVALID_ARG;
  }
  static thread_local std::vector<IppdPlanEntry> ent;
  static thread_local std::vector<int32_t> pos;
  ent.resize(A);
  pos.resize(A);
  int32_t prev = -1;
  for (int a = 0; a < A; ++a) {
    const int32_t k = active_q[a];
    if (k < 0 || k >= L.NQ) { ippd_set_error("ippd_begin_step: question id out of range"); return IPPD_ERR_INVALID_ARG; }
    if (k <= prev) { ippd_set_error("ippd_begin_step: active_q must be strictly increasing"); return IPPD_ERR_INVALID_ARG; }
    if (answer_idx[a] < 0) { ippd_set_error("ippd_begin_step: answer_idx < 0"); return IPPD_ERR_INVALID_ARG; }
    if (answer_idx[a] >= L.max_new[k]) { ippd_set_error("ippd_begin_step: answer_idx >= max_new (branch capacity)"); return IPPD_ERR_CAPACITY; }
    prev = k;
    const int b = L.prompt_of[k];
    ent[a] = {b, k, L.q_len[k] + answer_idx[a] + 1, 0};
    // virtual position of the query (Sec. 4.1): instruction + context + question length + answer index
    pos[a] = L.shared_len + L.ctx_len[b] + L.q_len[k] + answer_idx[a];
  }
  int rc = ippd_host_plan_entries(L, ent.data(), pos.data(), A, layer_count, true, plan);
  if (rc != IPPD_OK) return rc;
  plan->act_q.assign(active_q, active_q + A);
  plan->act_s.assign(answer_idx, answer_idx + A);
  return IPPD_OK;
}

int ippd_host_plan_entries(const IppdHostLayout& L, const IppdPlanEntry* ent, const int32_t* pos, int32_t A,
                           int32_t layer_count, bool mark_new, IppdStepPlan* plan) {
  const int RB = L.rows_per_block();
  const int qpr = questions_per_block(L);
  plan->act_q.assign(A, 0);
  plan->act_s.assign(A, 0);
  plan->act_pos.assign(pos, pos + A);
  plan->rbs.clear();
  plan->units.clear();
  plan->tc_tiles.clear();
  plan->tc_pieces.clear();
  const bool tc_path = L.kernel_path() >= 2;
  if (!tc_path && L.shared_len > 0) {
    ippd_set_error("ippd_begin_step: a shared instruction needs the tensor-core path (IPPD_OPT_KERNEL 0 or 2)");
    return IPPD_ERR_INVALID_ARG;
  }
  int64_t total = 0;
  int i = 0;
  while (i < A) {
    const int b = ent[i].prompt;
    const int causal = ent[i].causal;
    int j = i;
    while (j < A && ent[j].prompt == b && ent[j].causal == causal) ++j;
    if (!tc_path && (causal || b < 0)) {
      ippd_set_error("prefill needs the tensor-core path (IPPD_OPT_KERNEL 0 or 2)");
      return IPPD_ERR_INVALID_ARG;
    }
    const int nct_own = b >= 0 ? L.ctx_tile_off[b + 1] - L.ctx_tile_off[b] : 0;
    for (int a0 = i; a0 < j; a0 += qpr) {
      IppdRowBlock rb;
      memset(&rb, 0, sizeof(rb));
      rb.prompt = b;
      rb.act_begin = a0;
      rb.n_act = std::min(qpr, j - a0);
      // every query row sees the shared instruction, then its own context; a causal row only up to its own position
      int n_sh = L.n_shared_tiles, n_own = nct_own;
      int pos_min = 0;
      if (causal) {
        int pos_max = 0;
        pos_min = INT_MAX;
        for (int a = a0; a < a0 + rb.n_act; ++a) { pos_max = std::max(pos_max, pos[a]); pos_min = std::min(pos_min, pos[a]); }
        if (pos_max < L.shared_len) {
          n_sh = pos_max / IPPD_TILE_TOKENS + 1;
          n_own = 0;
        } else {
          n_own = std::min(nct_own, (pos_max - L.shared_len) / IPPD_TILE_TOKENS + 1);
        }
      }
      const int nct = n_sh + n_own;
      rb.n_ctx_tiles = nct;
      int64_t tiles = nct;
      if (tc_path) {
        for (int t = 0; t < n_sh; ++t) {
          IppdTcTile ti = {t, std::min(IPPD_TILE_TOKENS, L.shared_len - t * IPPD_TILE_TOKENS), 0, 0};
          if (causal && t * IPPD_TILE_TOKENS + ti.rows - 1 >= pos_min) { ti.n_pieces = -1; ti.piece_begin = t * IPPD_TILE_TOKENS; }
          plan->tc_tiles.push_back(ti);
        }
        for (int t = 0; t < n_own; ++t) {
          IppdTcTile ti = {L.ctx_tile_off[b] + t, std::min(IPPD_TILE_TOKENS, L.ctx_len[b] - t * IPPD_TILE_TOKENS), 0, 0};
          const int tok0 = L.shared_len + t * IPPD_TILE_TOKENS;  // virtual position of the tile's first token
          if (causal && tok0 + ti.rows - 1 >= pos_min) { ti.n_pieces = -1; ti.piece_begin = tok0; }
          plan->tc_tiles.push_back(ti);
        }
        // Pack the branches of the block's questions, 8-token group by group, into 128-row tiles.  Every tile takes
        // an equal share of its 16 groups from each quarter of the block's rows that still has groups left (32 rows =
        // 32 / G questions; the softmax warps that own a quarter's TMEM lanes do the work for its pieces), so that each
        // tile spreads its work over all those warps instead of queueing on the four of one quarter.
        const int G = L.geom.n_q_heads / L.geom.n_kv_heads;
        const int q_per_quarter = std::max(1, 32 / G);
        const int n_quarters = (rb.n_act + q_per_quarter - 1) / q_per_quarter;
        // 8-token groups [off, off+groups) of one cache tile; `last`: the tile that holds the branch's newest token
        struct Run { int a, cache_tile, off, groups, valid, last; };
        static thread_local std::vector<Run> runs[4];
        size_t next[4] = {0, 0, 0, 0};
        int rem[4] = {0, 0, 0, 0};  // groups each quarter still has to place
        int left_q = 0;
        for (int qu = 0; qu < n_quarters; ++qu) {
          runs[qu].clear();
          const int a_end = std::min(a0 + rb.n_act, a0 + (qu + 1) * q_per_quarter);
          for (int a = a0 + qu * q_per_quarter; a < a_end; ++a) {
            const int k = ent[a].branch;
            const int len = k >= 0 ? ent[a].branch_len : 0;
            for (int jt = 0; jt * IPPD_TILE_TOKENS < len; ++jt) {
              const int valid_j = std::min(IPPD_TILE_TOKENS, len - jt * IPPD_TILE_TOKENS);
              runs[qu].push_back({a - a0, L.branch_tile_off[k] + jt, 0, (valid_j + 7) / 8, valid_j,
                                  mark_new && (jt + 1) * IPPD_TILE_TOKENS >= len});
              rem[qu] += (valid_j + 7) / 8;
            }
          }
          left_q += rem[qu] > 0;
        }
        while (left_q > 0) {
          // this tile's allotment: an equal share for every quarter that has groups left, the room that short quarters
          // leave goes to the others; each quarter's allotment is laid out as one contiguous run of rows (the kernel
          // takes the union of a question's pieces in a tile as its window, so they must be adjacent)
          int alloc[4] = {0, 0, 0, 0};
          int room = 16;
          const int share = std::max(1, 16 / left_q);
          for (int qu = 0; qu < n_quarters; ++qu) {
            alloc[qu] = std::min(rem[qu], std::min(share, room));
            room -= alloc[qu];
          }
          for (int qu = 0; qu < n_quarters && room > 0; ++qu) {
            const int more = std::min(rem[qu] - alloc[qu], room);
            alloc[qu] += more;
            room -= more;
          }
          IppdTcTile ti = {-1, 0, (int32_t)plan->tc_pieces.size(), 0};
          int used = 0;
          for (int qu = 0; qu < n_quarters; ++qu) {
            int want = alloc[qu];
            rem[qu] -= want;
            if (alloc[qu] > 0 && rem[qu] == 0) --left_q;
            while (want > 0) {
              Run& r = runs[qu][next[qu]];
              const int take = std::min(want, r.groups);
              IppdTcPiece pc = {r.a, r.cache_tile, r.off, take, used * 8, std::min(take * 8, r.valid - r.off * 8), 0, 0};
              // the token fed at this step is the branch's last valid token: exactly one piece of the step holds it
              const int newest = r.valid - 1 - r.off * 8;
              if (r.last && newest >= 0 && newest < take * 8) pc.new_tok = 1 + newest;
              plan->tc_pieces.push_back(pc);
              ti.n_pieces++;
              used += take;
              want -= take;
              r.off += take;
              r.groups -= take;
              if (r.groups == 0) ++next[qu];
            }
          }
          ti.rows = used * 8;
          plan->tc_tiles.push_back(ti);
          ++tiles;
        }
      } else {
        for (int a = a0; a < a0 + rb.n_act; ++a)
          tiles += ceil_div((int64_t)ent[a].branch_len, IPPD_TILE_TOKENS);
      }
      rb.n_tiles = (int32_t)tiles;
      rb.tile_begin = (int32_t)total;
      total += tiles;
      if (total >= INT32_MAX) { ippd_set_error("ippd_begin_step: too many key tiles"); return IPPD_ERR_INVALID_ARG; }
      plan->rbs.push_back(rb);
    }
    i = j;
  }
  plan->rb_tile_begin.clear();
  for (const IppdRowBlock& rb : plan->rbs) plan->rb_tile_begin.push_back(rb.tile_begin);
  plan->rb_tile_begin.push_back((int32_t)total);
  plan->total_tiles = total;
  plan->hdr.n_active = A;
  plan->hdr.n_rowblocks = (int32_t)plan->rbs.size();
  plan->hdr.rows_per_block = RB;
  if (L.kernel_path() >= 2) {  // the persistent kernel cuts the tile sequence itself: no unit list
    plan->hdr.n_units = 0;
    return IPPD_OK;
  }
  int64_t tps;
  if (L.opt_tiles_per_split > 0) {
    tps = L.opt_tiles_per_split;
  } else {
    int64_t all = total * L.geom.n_kv_heads * std::max(1, layer_count);
    tps = std::max<int64_t>(kMinTilesPerSplit, ceil_div(all, kTargetCtas));
  }
  for (size_t r = 0; r < plan->rbs.size(); ++r) {
    IppdRowBlock& rb = plan->rbs[r];
    int n_seg = (int)ceil_div(rb.n_tiles, tps);
    rb.unit_begin = (int32_t)plan->units.size();
    rb.n_seg = n_seg;
    for (int sgm = 0; sgm < n_seg; ++sgm) {
      IppdUnit u;
      u.rowblock = (int32_t)r;
      u.tile_begin = (int32_t)((int64_t)rb.n_tiles * sgm / n_seg);
      u.tile_end = (int32_t)((int64_t)rb.n_tiles * (sgm + 1) / n_seg);
      u.seg = sgm;
      plan->units.push_back(u);
    }
  }
  plan->hdr.n_units = (int32_t)plan->units.size();
  return IPPD_OK;
}
