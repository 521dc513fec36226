// Internal structures shared by the host scheduler and the CUDA kernels of the IPPD library.
#pragma once
#include <stddef.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/ippd.h"

#define IPPD_MAX_ROWS_PER_BLOCK 128
#define IPPD_DEFAULT_KERNEL 2  // what IPPD_OPT_KERNEL = 0 selects

// ---- per-step work description (layer- and head-independent; the grid adds those axes) ----
struct IppdStepHeader {
  int32_t n_active;    // A
  int32_t n_rowblocks;
  int32_t n_units;
  int32_t rows_per_block;  // RB: query rows (questions x G) one CTA holds
};
// A row block: up to RB/G consecutive active questions of one prompt.
struct IppdRowBlock {
  int32_t prompt;
  int32_t act_begin;   // index of its first question in the step's active list
  int32_t n_act;       // questions in the block
  int32_t n_ctx_tiles; // ceil(L_b / 128)
  int32_t n_tiles;     // context tiles + branch tiles of its questions
  int32_t unit_begin;  // first split-KV unit of this block
  int32_t n_seg;       // number of units (segments of its key-tile sequence)
  int32_t tile_begin;  // first tile of this block inside one (layer, KV head) tile sequence
};
// A split-KV unit: key tiles [tile_begin, tile_end) of a row block's sequence
// (context tiles first, then the branch tiles of its questions in order).
struct IppdUnit {
  int32_t rowblock;
  int32_t tile_begin;
  int32_t tile_end;
  int32_t seg;
};

// Key tile of the tensor-core path.  A context tile (n_pieces == 0) is pool tile `pool_tile` with `rows` valid tokens.
// A packed branch tile (n_pieces > 0) is the concatenation of pieces; `rows` = 8 x the groups it holds.
// A causal context tile (n_pieces == -1, prefill only) is a context tile of which a query row sees only the tokens up
// to its own position; piece_begin then holds the virtual position of the tile's first token.
struct IppdTcTile {
  int32_t pool_tile;
  int32_t rows;
  int32_t piece_begin;
  int32_t n_pieces;
};
// A run of 8-token groups of one question's branch placed at row `row0` of a packed tile.
struct IppdTcPiece {
  int32_t a_local;    // question index inside its row block
  int32_t src_tile;   // pool tile the groups come from
  int32_t src_group;  // first group inside that pool tile
  int32_t n_groups;
  int32_t row0;       // first row in the packed tile (multiple of 8)
  int32_t valid;      // valid tokens in the piece (<= 8 * n_groups)
  int32_t new_tok;    // 1 + index inside the piece of the token fed at this step, 0 if the piece does not hold it
  int32_t pad1;
};

// One query of a planned pass: a decode step's token, or a header token of the prefill.
struct IppdPlanEntry {
  int32_t prompt;      // -1: a token of the shared instruction
  int32_t branch;      // question whose branch the query sees, -1: none
  int32_t branch_len;  // how many of the branch's tokens it sees (from slot 0)
  int32_t causal;      // 1: of the (instruction, context) key stream it sees only the tokens up to its own position
};

struct IppdStepPlan {
  IppdStepHeader hdr;
  std::vector<int32_t> act_q, act_s, act_pos;
  std::vector<IppdRowBlock> rbs;
  std::vector<IppdUnit> units;
  std::vector<int32_t> rb_tile_begin;  // [n_rb+1] prefix sums of n_tiles
  std::vector<IppdTcTile> tc_tiles;    // tensor-core path: tiles of one (layer, KV head) sequence
  std::vector<IppdTcPiece> tc_pieces;
  int64_t total_tiles = 0;
};

// ---- host-side layout object ----
struct IppdHostLayout {
  ippd_geometry_t geom;
  int32_t B = 0, NQ = 0, G = 1;
  std::vector<int32_t> ctx_len, q_count, q_len, max_new, q_begin, prompt_of, ctx_tile_off;
  std::vector<int64_t> branch_off, hdr_begin;
  std::vector<int32_t> branch_tile_off;  // [NQ+1] global tile index (context tiles come first)
  std::vector<int32_t> hdr_pos, hdr_ctx, hdr_qtn;
  int64_t n_ctx_tiles = 0, n_tiles = 0;  // n_ctx_tiles counts the shared instruction's tiles too
  int32_t shared_len = 0, n_shared_tiles = 0;  // instruction shared by every prompt of the batch: tiles [0, n_shared_tiles)
  int32_t max_pos = 0;
  // options
  int32_t opt_kernel = 0, opt_layers_per_call = 0, opt_tiles_per_split = 0;
  int32_t opt_kv_dtype = IPPD_KV_BF16;
  int64_t opt_wait_limit_us = 2000000;

  // K (or V) half of a 128-token cache tile
  size_t tile_bytes() const { return (size_t)IPPD_TILE_TOKENS * geom.head_dim * (opt_kv_dtype == IPPD_KV_E4M3 ? 1 : 2); }
  size_t cache_bytes() const {
    return (size_t)geom.n_layers * geom.n_kv_heads * (size_t)n_tiles * 2 * tile_bytes();
  }
  int rows_per_block() const;  // depends on the kernel path
  int kernel_path() const;     // 1 = mma.sync, 2 = tcgen05
};

void ippd_set_error(const std::string& msg);
int ippd_host_build(const ippd_geometry_t* geom, int32_t shared_len, int32_t n_prompts, const int32_t* ctx_len,
                    const int32_t* q_count, const int32_t* q_len, const int32_t* max_new,
                    IppdHostLayout* out);
// Builds the work list of one step.  Returns IPPD_OK or an error code.
int ippd_host_plan_step(const IppdHostLayout& L, const int32_t* active_q, const int32_t* answer_idx,
                        int32_t n_active, int32_t layer_count, IppdStepPlan* plan);
// The same for an arbitrary list of queries (consecutive entries of one prompt and one kind form row blocks);
// pos[i] = virtual position of entry i; mark_new: the last visible branch token of every entry is the step's new token.
int ippd_host_plan_entries(const IppdHostLayout& L, const IppdPlanEntry* ent, const int32_t* pos, int32_t n,
                           int32_t layer_count, bool mark_new, IppdStepPlan* plan);
// Upper bound of plan.units.size() over all possible steps.
int64_t ippd_host_max_units(const IppdHostLayout& L, int32_t layer_count);
int64_t ippd_host_max_rowblocks(const IppdHostLayout& L);
