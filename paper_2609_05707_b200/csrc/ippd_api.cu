// C ABI of the IPPD library: device state, uploads, kernel launches.
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "ippd_aux_kernels.cuh"
#include "ippd_attn_mma.cuh"
#include "ippd_attn_tc.cuh"
#include "ippd_read_probe.cuh"
#include "ippd_device.cuh"
#include "ippd_internal.h"

#define CUDA_TRY(expr)                                                                   \
  do {                                                                                   \
    cudaError_t _e = (expr);                                                             \
    if (_e != cudaSuccess) {                                                             \
      ippd_set_error(std::string(#expr) + ": " + cudaGetErrorString(_e));                \
      return IPPD_ERR_CUDA;                                                              \
    }                                                                                    \
  } while (0)

static const int kRingSlots = 16;
static const int kMaxCtas = IPPD_TC_MAX_CTAS;  // upper bound of the persistent kernel's grid (SM count)

struct ippd_layout {
  IppdHostLayout h;
  bool bound = false;
  int device = -1;
  // device mirrors
  int32_t *d_ctx_len = nullptr, *d_ctx_tile_off = nullptr, *d_q_len = nullptr, *d_prompt_of = nullptr,
          *d_branch_tile_off = nullptr, *d_error = nullptr, *d_hdr_begin = nullptr, *d_q_hdr_begin = nullptr,
          *d_q_first = nullptr;
  char* prefill_dev = nullptr;  // device copy of the prefill's work list
  size_t prefill_cap = 0;
  float2* d_rope = nullptr;
  char* cache = nullptr;
  // ring of pinned host / device slots for the small per-call descriptors
  char* ring_host[kRingSlots] = {};
  char* ring_host_dev[kRingSlots] = {};  // device mapping of ring_host
  char* ring_dev[kRingSlots] = {};
  cudaEvent_t ring_ev[kRingSlots] = {};
  bool ring_used[kRingSlots] = {};
  size_t ring_cap = 0;
  int ring_next = 0;
  int pending_slot = -1;  // ring slot staged on the host whose upload has not been enqueued yet
  unsigned pending_n16 = 0;
  // current step
  bool have_step = false;
  IppdStepPlan plan;
  IppdStepDev step_dev = {};
  bool step_needs_merge = false;
  const int32_t* d_rb_tile_begin = nullptr;  // inside the step blob
  const IppdTcTile* d_tc_tiles = nullptr;
  const IppdTcPiece* d_tc_pieces = nullptr;
  int sm_count = 0;
  cudaStream_t last_stream = nullptr;
  int64_t launches = 0;
  double host_plan_us = 0.0;  // host time spent in ippd_begin_step (planning, packing, staging) since the last read
  double host_wait_us = 0.0;  // part of it spent waiting for a free staging slot (the device is behind)
  int64_t host_plan_steps = 0;
  // optional event record: (kind, start, stop) per bracketed kernel; kind 0 attention, 1 merge, 2 append
  bool profile = false;        // the current step is bracketed
  int64_t profile_stride = 0;  // 0 off; N: every N-th step declared by ippd_begin_step is bracketed
  int64_t profile_steps = 0;   // steps declared since the option was set
  std::vector<cudaEvent_t> ev_pool;
  std::vector<int> ev_kind;
  size_t ev_used = 0;
  // pipelined host steps (ippd_decode_step_host_async): copy streams and per-slot events, created on first use
  bool hs_init = false;
  cudaStream_t hs_in = nullptr, hs_out = nullptr;
  cudaEvent_t hs_ev_in[2] = {}, hs_ev_done[2] = {}, hs_ev_out[2] = {};
  int64_t hs_count = 0;
};

static size_t ceil_div_sz(size_t a, size_t b) { return (a + b - 1) / b; }

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Offsets of the parts of a step descriptor (each 16-byte aligned) and its total size.
struct StepBlobLayout {
  size_t off_q, off_s, off_rb, off_u, off_tb, off_tt, off_tp, off_pos, total;
};
static StepBlobLayout step_blob_layout(size_t A, size_t n_rb, size_t n_units, size_t n_tiles, size_t n_pieces) {
  StepBlobLayout b;
  b.off_q = 0;
  b.off_s = align_up(b.off_q + A * 4, 16);
  b.off_rb = align_up(b.off_s + A * 4, 16);
  b.off_u = align_up(b.off_rb + n_rb * sizeof(IppdRowBlock), 16);
  b.off_tb = align_up(b.off_u + n_units * sizeof(IppdUnit), 16);
  b.off_tt = align_up(b.off_tb + (n_rb + 1) * 4, 16);
  b.off_tp = align_up(b.off_tt + n_tiles * sizeof(IppdTcTile), 16);
  b.off_pos = align_up(b.off_tp + n_pieces * sizeof(IppdTcPiece), 16);
  b.total = align_up(b.off_pos + A * 4, 16) + 16;
  return b;
}

// Capacity of a descriptor staging slot: a bound of the descriptor size over every step the layout admits (every
// question active, every branch full), and of the id list of a CONTEXT / QUESTION append.
//   row blocks  <= nrb; unit list (mma.sync path) <= max over the split settings of its unit count;
//   key tiles   <= every row block's context tiles + packed branch tiles; 16 groups of 8 tokens per packed tile and
//                  at most 16 groups per cache tile of a branch give packed tiles <= branch cache tiles + nrb;
//   pieces      <= one per (question, cache tile) run + one more wherever a packed tile's per-quarter allotment ends
//                  inside a run: runs + 4 * packed tiles <= 5 * branch cache tiles + 4 * nrb.
static size_t ring_capacity(const IppdHostLayout& h) {
  const size_t nrb = (size_t)ippd_host_max_rowblocks(h);
  const size_t branch_tiles = (size_t)(h.n_tiles - h.n_ctx_tiles);
  const int qpr_tc = std::max(1, std::min(IPPD_MAX_ROWS_PER_BLOCK / h.G, 64));
  const int qpr_mma = std::max(1, 64 / h.G);
  size_t ctx_tiles_all_blocks = 0;  // whichever kernel path is selected later
  for (int b = 0; b < h.B; ++b) {
    const size_t blocks = (size_t)(h.q_count[b] + std::min(qpr_tc, qpr_mma) - 1) / std::min(qpr_tc, qpr_mma);
    ctx_tiles_all_blocks += (size_t)(h.n_shared_tiles + h.ctx_tile_off[b + 1] - h.ctx_tile_off[b]) * blocks;
  }
  const size_t nrb_any = std::max(nrb, (size_t)ceil_div_sz(h.NQ, 1));  // row blocks never outnumber questions
  const size_t units = ctx_tiles_all_blocks + branch_tiles + nrb_any + 2048;  // one unit per tile at worst
  const StepBlobLayout b = step_blob_layout((size_t)h.NQ, nrb_any, units, ctx_tiles_all_blocks + branch_tiles + nrb_any,
                                            5 * branch_tiles + 4 * nrb_any);
  const size_t ids = ((size_t)2 * std::max(h.NQ, h.B) + 4) * 4;
  return align_up(std::max(b.total, ids) + 256, 256);  // the upload kernel moves 16-byte words
}

// Launch with the programmatic-serialisation attribute: the kernel may be scheduled while its predecessor in the
// stream still runs and calls pdl_wait() before it touches global memory.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Records an event on `stream` when profiling is on (start when `start`, else stop) for a kernel of `kind`.
static void prof_mark(ippd_layout* L, int kind, bool start, cudaStream_t stream) {
  if (!L->profile) return;
  if (L->ev_used == L->ev_pool.size()) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    L->ev_pool.push_back(e);
  }
  if (start) L->ev_kind.push_back(kind);
  cudaEventRecord(L->ev_pool[L->ev_used++], stream);
}

static IppdDev make_dev(const ippd_layout* L) {
  IppdDev d;
  d.ctx_len = L->d_ctx_len;
  d.ctx_tile_off = L->d_ctx_tile_off;
  d.q_len = L->d_q_len;
  d.prompt_of = L->d_prompt_of;
  d.branch_tile_off = L->d_branch_tile_off;
  d.hdr_begin = L->d_hdr_begin;
  d.q_hdr_begin = L->d_q_hdr_begin;
  d.rope = L->d_rope;
  d.cache = L->cache;
  d.error_word = L->d_error;
  d.n_tiles = L->h.n_tiles;
  d.wait_limit_ns = L->h.opt_wait_limit_us * 1000;
  d.n_layers = L->h.geom.n_layers;
  d.Hq = L->h.geom.n_q_heads;
  d.Hkv = L->h.geom.n_kv_heads;
  d.G = L->h.G;
  d.D = L->h.geom.head_dim;
  d.max_pos = L->h.max_pos;
  d.shared_len = L->h.shared_len;
  d.kv8 = L->h.opt_kv_dtype == IPPD_KV_E4M3;
  return d;
}

extern "C" int ippd_build_layout_shared(const ippd_geometry_t* geom, int32_t shared_len, int32_t n_prompts,
                                        const int32_t* ctx_len, const int32_t* q_count, const int32_t* q_len,
                                        const int32_t* max_new, ippd_layout_t** out) {
  if (!out) { ippd_set_error("ippd_build_layout: out is NULL"); return IPPD_ERR_INVALID_ARG; }
  *out = nullptr;
  ippd_layout* L = new (std::nothrow) ippd_layout();
  if (!L) { ippd_set_error("ippd_build_layout: out of host memory"); return IPPD_ERR_OOM; }
  int rc = ippd_host_build(geom, shared_len, n_prompts, ctx_len, q_count, q_len, max_new, &L->h);
  if (rc != IPPD_OK) { delete L; return rc; }
  *out = L;
  return IPPD_OK;
}

extern "C" int ippd_build_layout(const ippd_geometry_t* geom, int32_t n_prompts, const int32_t* ctx_len,
                                 const int32_t* q_count, const int32_t* q_len, const int32_t* max_new,
                                 ippd_layout_t** out) {
  return ippd_build_layout_shared(geom, 0, n_prompts, ctx_len, q_count, q_len, max_new, out);
}

extern "C" int ippd_layout_tables(const ippd_layout_t* L, ippd_tables_t* t) {
  if (!L || !t) { ippd_set_error("ippd_layout_tables: NULL argument"); return IPPD_ERR_INVALID_ARG; }
  const IppdHostLayout& h = L->h;
  t->q_begin = h.q_begin.data();
  t->prompt_of = h.prompt_of.data();
  t->q_len = h.q_len.data();
  t->ctx_len = h.ctx_len.data();
  t->branch_off = h.branch_off.data();
  t->ctx_tile_off = h.ctx_tile_off.data();
  t->hdr_begin = h.hdr_begin.data();
  t->hdr_pos_virt = h.hdr_pos.data();
  t->hdr_ctx_id = h.hdr_ctx.data();
  t->hdr_qtn_id = h.hdr_qtn.data();
  t->n_prompts = h.B;
  t->n_questions = h.NQ;
  t->n_header_tokens = (int64_t)h.hdr_pos.size();
  t->n_branch_slots = h.branch_off[h.NQ];
  t->n_tiles = h.n_tiles;
  t->n_shared_tokens = h.shared_len;
  return IPPD_OK;
}

extern "C" int ippd_cache_bytes(const ippd_layout_t* L, size_t* bytes, size_t* align) {
  if (!L || !bytes) { ippd_set_error("ippd_cache_bytes: NULL argument"); return IPPD_ERR_INVALID_ARG; }
  *bytes = L->h.cache_bytes();
  if (align) *align = 256;
  return IPPD_OK;
}

extern "C" int ippd_set_option(ippd_layout_t* L, int32_t key, int64_t value) {
  if (!L) { ippd_set_error("ippd_set_option: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  switch (key) {
    case IPPD_OPT_KERNEL:
      if (value < 0 || value > 2) { ippd_set_error("ippd_set_option: kernel path not available"); return IPPD_ERR_INVALID_ARG; }
      if (value == 1 && L->h.opt_kv_dtype == IPPD_KV_E4M3) { ippd_set_error("ippd_set_option: the 8-bit cache needs the tensor-core path"); return IPPD_ERR_INVALID_ARG; }
      L->h.opt_kernel = (int32_t)value;
      break;
    case IPPD_OPT_LAYERS_PER_CALL:
      if (value < 0 || value > L->h.geom.n_layers) { ippd_set_error("ippd_set_option: bad layer count"); return IPPD_ERR_INVALID_ARG; }
      L->h.opt_layers_per_call = (int32_t)value;
      break;
    case IPPD_OPT_TILES_PER_SPLIT:
      if (value < 0 || value > (1 << 20)) { ippd_set_error("ippd_set_option: bad tiles per split"); return IPPD_ERR_INVALID_ARG; }
      L->h.opt_tiles_per_split = (int32_t)value;
      break;
    case IPPD_OPT_PROFILE:
      if (value < 0) { ippd_set_error("ippd_set_option: bad profile stride"); return IPPD_ERR_INVALID_ARG; }
      L->profile_stride = value;
      L->profile_steps = 0;
      L->profile = false;
      return IPPD_OK;
    case IPPD_OPT_KV_DTYPE:
      if (value != IPPD_KV_BF16 && value != IPPD_KV_E4M3) { ippd_set_error("ippd_set_option: unknown cache element type"); return IPPD_ERR_INVALID_ARG; }
      if (L->bound) { ippd_set_error("ippd_set_option: the cache element type is fixed once a cache is bound"); return IPPD_ERR_INVALID_ARG; }
      if (value == IPPD_KV_E4M3 && L->h.kernel_path() < 2) { ippd_set_error("ippd_set_option: the 8-bit cache needs the tensor-core path"); return IPPD_ERR_INVALID_ARG; }
      L->h.opt_kv_dtype = (int32_t)value;
      break;
    case IPPD_OPT_WAIT_LIMIT_US:
      if (value < 0 || value > 60000000) { ippd_set_error("ippd_set_option: bad wait limit"); return IPPD_ERR_INVALID_ARG; }
      L->h.opt_wait_limit_us = value;
      break;
    default:
      ippd_set_error("ippd_set_option: unknown key");
      return IPPD_ERR_INVALID_ARG;
  }
  L->have_step = false;  // the work list depends on the options
  return IPPD_OK;
}

static int plan_layers(const ippd_layout* L) {
  return L->h.opt_layers_per_call > 0 ? L->h.opt_layers_per_call : L->h.geom.n_layers;
}

template <typename T>
static int upload_vec(T** dst, const std::vector<T>& v) {
  CUDA_TRY(cudaMalloc((void**)dst, std::max<size_t>(1, v.size()) * sizeof(T)));
  if (!v.empty()) CUDA_TRY(cudaMemcpy(*dst, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice));
  return IPPD_OK;
}

static void free_device(ippd_layout* L) {
  cudaFree(L->d_ctx_len); cudaFree(L->d_ctx_tile_off); cudaFree(L->d_q_len); cudaFree(L->d_prompt_of);
  cudaFree(L->d_branch_tile_off); cudaFree(L->d_error); cudaFree(L->d_rope);
  cudaFree(L->d_hdr_begin); cudaFree(L->d_q_hdr_begin); cudaFree(L->d_q_first); cudaFree(L->prefill_dev);
  L->d_hdr_begin = L->d_q_hdr_begin = L->d_q_first = nullptr;
  L->prefill_dev = nullptr;
  L->prefill_cap = 0;
  L->d_ctx_len = L->d_ctx_tile_off = L->d_q_len = L->d_prompt_of = L->d_branch_tile_off = L->d_error = nullptr;
  L->d_rope = nullptr;
  for (int i = 0; i < kRingSlots; ++i) {
    if (L->ring_host[i]) cudaFreeHost(L->ring_host[i]);
    if (L->ring_dev[i]) cudaFree(L->ring_dev[i]);
    if (L->ring_ev[i]) cudaEventDestroy(L->ring_ev[i]);
    L->ring_host[i] = L->ring_dev[i] = nullptr;
    L->ring_ev[i] = nullptr;
    L->ring_used[i] = false;
  }
  L->bound = false;
}

extern "C" int ippd_bind_cache(ippd_layout_t* L, void* dev_cache, size_t bytes, void* stream_) {
  if (!L || !dev_cache) { ippd_set_error("ippd_bind_cache: NULL argument"); return IPPD_ERR_INVALID_ARG; }
  if (bytes < L->h.cache_bytes()) { ippd_set_error("ippd_bind_cache: cache too small"); return IPPD_ERR_INVALID_ARG; }
  if ((uintptr_t)dev_cache % 256 != 0) { ippd_set_error("ippd_bind_cache: cache must be 256-byte aligned"); return IPPD_ERR_INVALID_ARG; }
  cudaStream_t stream = (cudaStream_t)stream_;
  if (L->bound) free_device(L);
  CUDA_TRY(cudaGetDevice(&L->device));
  CUDA_TRY(cudaDeviceGetAttribute(&L->sm_count, cudaDevAttrMultiProcessorCount, L->device));
  const IppdHostLayout& h = L->h;
  int rc;
  if ((rc = upload_vec(&L->d_ctx_len, h.ctx_len)) != IPPD_OK) return rc;
  if ((rc = upload_vec(&L->d_ctx_tile_off, h.ctx_tile_off)) != IPPD_OK) return rc;
  if ((rc = upload_vec(&L->d_q_len, h.q_len)) != IPPD_OK) return rc;
  if ((rc = upload_vec(&L->d_prompt_of, h.prompt_of)) != IPPD_OK) return rc;
  if ((rc = upload_vec(&L->d_branch_tile_off, h.branch_tile_off)) != IPPD_OK) return rc;
  {
    // header offsets: first header token of each prompt and of each question (the hdr_* order)
    std::vector<int32_t> hb(h.hdr_begin.begin(), h.hdr_begin.end()), qb((size_t)h.NQ + 1, 0);
    for (int b = 0; b < h.B; ++b) {
      int64_t t = h.hdr_begin[b] + h.ctx_len[b];
      for (int k = h.q_begin[b]; k < h.q_begin[b + 1]; ++k) { qb[k] = (int32_t)t; t += h.q_len[k]; }
    }
    qb[h.NQ] = (int32_t)h.hdr_begin[h.B];
    if ((rc = upload_vec(&L->d_hdr_begin, hb)) != IPPD_OK) return rc;
    if ((rc = upload_vec(&L->d_q_hdr_begin, qb)) != IPPD_OK) return rc;
    if ((rc = upload_vec(&L->d_q_first, h.q_begin)) != IPPD_OK) return rc;
  }
  CUDA_TRY(cudaMalloc((void**)&L->d_error, sizeof(int32_t)));
  CUDA_TRY(cudaMemset(L->d_error, 0, sizeof(int32_t)));
  size_t n_rope = (size_t)(h.max_pos + 1) * (h.geom.head_dim / 2);
  CUDA_TRY(cudaMalloc((void**)&L->d_rope, n_rope * sizeof(float2)));
  ippd_rope_table_kernel<<<(unsigned)((n_rope + 255) / 256), 256, 0, stream>>>(L->d_rope, h.max_pos,
                                                                                h.geom.head_dim, h.geom.rope_theta);
  CUDA_TRY(cudaGetLastError());
  L->launches++;
  L->ring_cap = ring_capacity(h);
  const size_t cap = L->ring_cap;
  for (int i = 0; i < kRingSlots; ++i) {
    CUDA_TRY(cudaHostAlloc((void**)&L->ring_host[i], cap, cudaHostAllocMapped));
    CUDA_TRY(cudaHostGetDevicePointer((void**)&L->ring_host_dev[i], L->ring_host[i], 0));
    CUDA_TRY(cudaMalloc((void**)&L->ring_dev[i], cap));
    CUDA_TRY(cudaEventCreateWithFlags(&L->ring_ev[i], cudaEventDisableTiming));
  }
  L->cache = (char*)dev_cache;
  // Every slot of the cache must hold a finite number before it is ever streamed (a 128-row tile is multiplied as a
  // whole; rows past the valid tokens get probability zero, and 0 * NaN would still be NaN).
  CUDA_TRY(cudaMemsetAsync(dev_cache, 0, h.cache_bytes(), stream));
  CUDA_TRY(cudaStreamSynchronize(stream));
  L->bound = true;
  L->have_step = false;
  L->last_stream = stream;
  return IPPD_OK;
}

// Copies a host blob into the next pinned ring slot; returns the device address it will have once uploaded.
// The upload itself is launched by ring_flush (or folded into the next STEP append).
static int ring_stage(ippd_layout* L, const void* blob, size_t bytes, char** dev) {
  if (bytes > L->ring_cap) { ippd_set_error("descriptor larger than the staging slot"); return IPPD_ERR_CAPACITY; }
  int slot = L->ring_next;
  L->ring_next = (L->ring_next + 1) % kRingSlots;
  if (L->ring_used[slot]) {
    // back-pressure, not work: the host may run at most kRingSlots descriptors ahead of the device
    const auto w0 = std::chrono::steady_clock::now();
    CUDA_TRY(cudaEventSynchronize(L->ring_ev[slot]));
    L->host_wait_us += std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - w0).count();
  }
  memcpy(L->ring_host[slot], blob, bytes);
  L->pending_slot = slot;
  L->pending_n16 = (unsigned)((bytes + 15) / 16);
  *dev = L->ring_dev[slot];
  return IPPD_OK;
}

// Marks the staged slot as read by the work enqueued so far on `stream`.
static int ring_uploaded(ippd_layout* L, cudaStream_t stream) {
  const int slot = L->pending_slot;
  L->pending_slot = -1;
  CUDA_TRY(cudaEventRecord(L->ring_ev[slot], stream));
  L->ring_used[slot] = true;
  return IPPD_OK;
}

// Uploads the staged descriptor, if any.  A kernel reads the pinned slot through its device mapping instead of a
// copy-engine transfer: it depends only on the stream, so it neither waits behind nor holds up the bulk host<->device
// copies other streams have queued on the copy engines, and a kernel-to-kernel dependency is cheaper than
// copy-to-kernel.
static int ring_flush(ippd_layout* L, cudaStream_t stream) {
  if (L->pending_slot < 0) return IPPD_OK;
  const int slot = L->pending_slot;
  // Programmatic launch: the copy touches only its own slot, so it runs while the kernel before it in the stream is
  // still busy; the kernel waits for that predecessor only at its end, which keeps the stream's order for whatever
  // comes next.
  CUDA_TRY(launch_pdl(ippd_upload_kernel, dim3((L->pending_n16 + 255) / 256), dim3(256), 0, stream,
                      (const uint4*)L->ring_host_dev[slot], (uint4*)L->ring_dev[slot], L->pending_n16));
  CUDA_TRY(cudaGetLastError());
  L->launches++;
  return ring_uploaded(L, stream);
}

static int ring_upload(ippd_layout* L, const void* blob, size_t bytes, cudaStream_t stream, char** dev) {
  int rc = ring_flush(L, stream);  // a descriptor staged earlier goes first
  if (rc != IPPD_OK) return rc;
  rc = ring_stage(L, blob, bytes, dev);
  if (rc != IPPD_OK) return rc;
  return ring_flush(L, stream);
}

extern "C" int ippd_begin_step(ippd_layout_t* L, const int32_t* active_q, const int32_t* answer_idx,
                               int32_t A, void* stream_) {
  if (!L) { ippd_set_error("ippd_begin_step: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  if (!L->bound) { ippd_set_error("ippd_begin_step: no cache bound"); return IPPD_ERR_NOT_BOUND; }
  cudaStream_t stream = (cudaStream_t)stream_;
  const auto host_t0 = std::chrono::steady_clock::now();
  L->have_step = false;
  L->profile = L->profile_stride > 0 && (L->profile_steps++ % L->profile_stride) == 0;
  int rc = ippd_host_plan_step(L->h, active_q, answer_idx, A, plan_layers(L), &L->plan);
  if (rc != IPPD_OK) return rc;
  const IppdStepPlan& P = L->plan;
  // blob: [act_q | act_s | row blocks | units | tile prefix | tiles | pieces | positions], each 16-byte aligned
  const StepBlobLayout bl = step_blob_layout((size_t)A, P.rbs.size(), P.units.size(), P.tc_tiles.size(), P.tc_pieces.size());
  const size_t off_q = bl.off_q, off_s = bl.off_s, off_rb = bl.off_rb, off_u = bl.off_u, off_tb = bl.off_tb,
               off_tt = bl.off_tt, off_tp = bl.off_tp, off_pos = bl.off_pos, total = bl.total;
  std::vector<char> blob(total, 0);
  if (A) {
    memcpy(blob.data() + off_q, P.act_q.data(), (size_t)A * 4);
    memcpy(blob.data() + off_s, P.act_s.data(), (size_t)A * 4);
    memcpy(blob.data() + off_rb, P.rbs.data(), P.rbs.size() * sizeof(IppdRowBlock));
    memcpy(blob.data() + off_u, P.units.data(), P.units.size() * sizeof(IppdUnit));
    memcpy(blob.data() + off_tb, P.rb_tile_begin.data(), P.rb_tile_begin.size() * 4);
    if (!P.tc_tiles.empty()) memcpy(blob.data() + off_tt, P.tc_tiles.data(), P.tc_tiles.size() * sizeof(IppdTcTile));
    if (!P.tc_pieces.empty()) memcpy(blob.data() + off_tp, P.tc_pieces.data(), P.tc_pieces.size() * sizeof(IppdTcPiece));
    // virtual position of every query (Sec. 4.1), kept in the descriptor so that the kernels' Q~ staging does not
    // chase it through three tables
    memcpy(blob.data() + off_pos, P.act_pos.data(), (size_t)A * 4);
  }
  char* dev = nullptr;
  L->pending_slot = -1;  // a step that was declared but never used is dropped
  rc = ring_stage(L, blob.data(), total, &dev);
  if (rc != IPPD_OK) return rc;
  L->step_dev.act_q = (const int32_t*)(dev + off_q);
  L->step_dev.act_s = (const int32_t*)(dev + off_s);
  L->step_dev.rbs = (const IppdRowBlock*)(dev + off_rb);
  L->step_dev.act_pos = (const int32_t*)(dev + off_pos);
  L->step_dev.units = (const IppdUnit*)(dev + off_u);
  L->d_rb_tile_begin = (const int32_t*)(dev + off_tb);
  L->d_tc_tiles = (const IppdTcTile*)(dev + off_tt);
  L->d_tc_pieces = (const IppdTcPiece*)(dev + off_tp);
  L->step_dev.A = A;
  L->step_dev.n_rb = P.hdr.n_rowblocks;
  L->step_dev.n_units = P.hdr.n_units;
  L->step_dev.RB = P.hdr.rows_per_block;
  L->step_needs_merge = false;
  for (const IppdRowBlock& rb : P.rbs) L->step_needs_merge |= rb.n_seg > 1;
  L->have_step = true;
  L->last_stream = stream;
  L->host_plan_us += std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - host_t0).count();
  L->host_plan_steps++;
  return IPPD_OK;
}

extern "C" int ippd_host_time_read(ippd_layout_t* L, double* begin_step_us, int64_t* n_steps) {
  if (!L) { ippd_set_error("ippd_host_time_read: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  if (begin_step_us) *begin_step_us = L->host_plan_us - L->host_wait_us;
  L->host_wait_us = 0.0;
  if (n_steps) *n_steps = L->host_plan_steps;
  L->host_plan_us = 0.0;
  L->host_plan_steps = 0;
  return IPPD_OK;
}

extern "C" int ippd_step_descriptor_bytes(const ippd_layout_t* L, const int32_t* active_q, const int32_t* answer_idx,
                                          int32_t A, size_t* bytes, size_t* capacity) {
  if (!L || !bytes || !capacity) { ippd_set_error("ippd_step_descriptor_bytes: NULL argument"); return IPPD_ERR_INVALID_ARG; }
  IppdStepPlan plan;
  int rc = ippd_host_plan_step(L->h, active_q, answer_idx, A, plan_layers(L), &plan);
  if (rc != IPPD_OK) return rc;
  *bytes = step_blob_layout((size_t)A, plan.rbs.size(), plan.units.size(), plan.tc_tiles.size(), plan.tc_pieces.size()).total;
  *capacity = ring_capacity(L->h);
  return IPPD_OK;
}

extern "C" int ippd_append_kv(ippd_layout_t* L, int32_t layer_begin, int32_t layer_count, int32_t kind,
                              const int32_t* ids, int32_t n_ids, const void* k_raw, const void* v_raw,
                              void* stream_) {
  if (!L) { ippd_set_error("ippd_append_kv: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  if (!L->bound) { ippd_set_error("ippd_append_kv: no cache bound"); return IPPD_ERR_NOT_BOUND; }
  const IppdHostLayout& h = L->h;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > h.geom.n_layers) {
    ippd_set_error("ippd_append_kv: layer range out of bounds");
    return IPPD_ERR_INVALID_ARG;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  IppdAppendArgs a;
  memset(&a, 0, sizeof(a));
  a.kind = kind;
  if (kind == IPPD_APPEND_STEP) {
    if (!L->have_step) { ippd_set_error("ippd_append_kv(STEP): call ippd_begin_step first"); return IPPD_ERR_INVALID_ARG; }
    a.n_tokens = L->step_dev.A;
    if (L->pending_slot >= 0 && a.n_tokens > 0 && a.n_tokens <= IPPD_APPEND_INLINE && k_raw && v_raw) {
      a.inline_acts = 1;
      memcpy(a.act_q, L->plan.act_q.data(), (size_t)a.n_tokens * 4);
      memcpy(a.act_s, L->plan.act_s.data(), (size_t)a.n_tokens * 4);
      a.up_n16 = L->pending_n16;
      a.up_src = (const uint4*)L->ring_host_dev[L->pending_slot];
      a.up_dst = (uint4*)L->ring_dev[L->pending_slot];
    } else {
      int rc = ring_flush(L, stream);
      if (rc != IPPD_OK) return rc;
    }
  } else if (kind == IPPD_APPEND_SHARED || kind == IPPD_APPEND_HEADER) {
    a.n_tokens = kind == IPPD_APPEND_SHARED ? h.shared_len : (int)h.hdr_pos.size();
    a.n_ids = h.B;
    a.q_first = L->d_q_first;
    int rc = ring_flush(L, stream);  // keeps the descriptor ring in stream order
    if (rc != IPPD_OK) return rc;
  } else if (kind == IPPD_APPEND_CONTEXT || kind == IPPD_APPEND_QUESTION) {
    if (n_ids < 1 || !ids) { ippd_set_error("ippd_append_kv: ids missing"); return IPPD_ERR_INVALID_ARG; }
    std::vector<int32_t> blob((size_t)2 * n_ids + 4, 0);
    int64_t tok = 0;
    for (int i = 0; i < n_ids; ++i) {
      int id = ids[i];
      int lim = kind == IPPD_APPEND_CONTEXT ? h.B : h.NQ;
      if (id < 0 || id >= lim) { ippd_set_error("ippd_append_kv: id out of range"); return IPPD_ERR_INVALID_ARG; }
      blob[i] = id;
      blob[n_ids + i] = (int32_t)tok;
      tok += kind == IPPD_APPEND_CONTEXT ? h.ctx_len[id] : h.q_len[id];
      if (tok >= INT32_MAX) { ippd_set_error("ippd_append_kv: too many tokens in one call"); return IPPD_ERR_INVALID_ARG; }
    }
    blob[2 * n_ids] = (int32_t)tok;
    a.n_tokens = (int)tok;
    a.n_ids = n_ids;
    if (tok > 0) {
      char* dev = nullptr;
      int rc = ring_upload(L, blob.data(), blob.size() * 4, stream, &dev);
      if (rc != IPPD_OK) return rc;
      a.ids = (const int32_t*)dev;
      a.tok_begin = (const int32_t*)dev + n_ids;
    }
  } else {
    ippd_set_error("ippd_append_kv: unknown kind");
    return IPPD_ERR_INVALID_ARG;
  }
  L->last_stream = stream;
  if (a.n_tokens == 0) return IPPD_OK;
  if (!k_raw || !v_raw) { ippd_set_error("ippd_append_kv: NULL k_raw / v_raw"); return IPPD_ERR_INVALID_ARG; }
  IppdDev d = make_dev(L);
  int D = h.geom.head_dim;
  long long items = (long long)a.n_tokens * h.geom.n_kv_heads * (D / 16);
  dim3 grid((unsigned)((items + 255) / 256), (unsigned)layer_count);
  if (a.inline_acts) {
    a.n_append_blocks = (int)grid.x;
    grid.x += (a.up_n16 + 255) / 256;
  }
  const bool prof = kind == IPPD_APPEND_STEP;
  if (prof) prof_mark(L, 2, true, stream);
  const bool kv8 = h.opt_kv_dtype == IPPD_KV_E4M3;
  if (D == 128)
    CUDA_TRY(launch_pdl(kv8 ? ippd_append_kernel<128, true> : ippd_append_kernel<128, false>, grid, dim3(256), 0, stream,
                        d, L->step_dev, a, layer_begin, (const __nv_bfloat16*)k_raw, (const __nv_bfloat16*)v_raw));
  else
    CUDA_TRY(launch_pdl(kv8 ? ippd_append_kernel<64, true> : ippd_append_kernel<64, false>, grid, dim3(256), 0, stream,
                        d, L->step_dev, a, layer_begin, (const __nv_bfloat16*)k_raw, (const __nv_bfloat16*)v_raw));
  if (prof) prof_mark(L, 2, false, stream);
  CUDA_TRY(cudaGetLastError());
  L->launches++;
  if (a.inline_acts) return ring_uploaded(L, stream);
  return IPPD_OK;
}

extern "C" int ippd_workspace_bytes(const ippd_layout_t* L, int32_t layer_count, size_t* bytes) {
  if (!L || !bytes || layer_count < 1 || layer_count > L->h.geom.n_layers) {
    ippd_set_error("ippd_workspace_bytes: bad argument");
    return IPPD_ERR_INVALID_ARG;
  }
  const IppdHostLayout& h = L->h;
  if (h.kernel_path() >= 2) {
    // two partial slots per CTA of the persistent kernel, whatever the step
    size_t per_slot = (size_t)IPPD_TC_ROWS * (h.geom.head_dim + 2) * sizeof(float);
    *bytes = align_up((size_t)kMaxCtas * 2 * per_slot, 256) + 512;
    return IPPD_OK;
  }
  int64_t units = ippd_host_max_units(h, plan_layers(L));
  size_t per_unit = (size_t)h.rows_per_block() * (h.geom.head_dim + 2) * sizeof(float);
  *bytes = align_up((size_t)layer_count * h.geom.n_kv_heads * (size_t)units * per_unit, 256) + 256;
  return IPPD_OK;
}

// Slices of the persistent tensor-core kernel for `layer_count` layers of the current step: fills a->total_tiles,
// a->n_cta and a->cut; *any_partial tells whether a cut falls inside a row block's key sequence (then partials are
// written and the merge kernel runs).
static int tc_partition(const ippd_layout* L, int layer_count, IppdTcArgs* a, bool* any_partial) {
  const long long t1 = L->plan.total_tiles;
  const long long total = t1 * L->h.geom.n_kv_heads * layer_count;
  if (total >= INT32_MAX) { ippd_set_error("too many key tiles in one launch: pass fewer layers per call"); return IPPD_ERR_INVALID_ARG; }
  int n_cta = L->sm_count > 0 ? L->sm_count : 148;
  if (n_cta > kMaxCtas) n_cta = kMaxCtas;
  long long ch = (total + n_cta - 1) / n_cta;
  const bool forced = L->h.opt_tiles_per_split > 0;  // test knob: cuts every `ch` tiles, wherever they fall
  if (forced) ch = L->h.opt_tiles_per_split;
  if (ch < 1) ch = 1;
  long long g = (total + ch - 1) / ch;
  if (g > n_cta) {  // more pieces than CTAs: grow the pieces
    ch = (total + n_cta - 1) / n_cta;
    g = (total + ch - 1) / ch;
  }
  const std::vector<int32_t>& rbt = L->plan.rb_tile_begin;  // [n_rb + 1], rbt[n_rb] = t1
  const long long slack = forced ? 0 : ch / 32;
  *any_partial = false;
  a->cut[0] = 0;
  int n = 0;
  for (long long c = 1; c <= g; ++c) {
    long long x = std::min(total, c * ch);
    if (x < total) {
      const long long seq = x / t1, within = x - seq * t1;
      size_t rb = std::upper_bound(rbt.begin(), rbt.end(), (int32_t)within) - rbt.begin() - 1;
      const long long lower = seq * t1 + rbt[rb], upper = seq * t1 + rbt[rb + 1];
      long long snapped = (x - lower <= upper - x) ? lower : upper;
      if (std::llabs(snapped - x) <= slack && snapped > a->cut[n] && snapped < total) x = snapped;
      if (x != lower && x != upper) *any_partial = true;
    }
    if (x <= a->cut[n]) continue;
    a->cut[++n] = (int32_t)x;
  }
  a->total_tiles = (int)total;
  a->n_cta = n;
  return IPPD_OK;
}

// Bytes of scratch the current step needs for `layer_count` layers; *o_bytes = offset of the (m, l) part.
static size_t scratch_need(const ippd_layout* L, int layer_count, size_t* o_bytes, bool* needed) {
  const IppdHostLayout& h = L->h;
  size_t n_part;
  if (h.kernel_path() >= 2) {
    IppdTcArgs a;
    bool any_partial = false;
    if (tc_partition(L, layer_count, &a, &any_partial) != IPPD_OK) { a.n_cta = kMaxCtas; any_partial = true; }
    n_part = (size_t)a.n_cta * 2 * IPPD_TC_ROWS;
    *needed = any_partial;
  } else {
    n_part = (size_t)layer_count * h.geom.n_kv_heads * (size_t)L->step_dev.n_units * L->step_dev.RB;
    *needed = L->step_needs_merge;
  }
  *o_bytes = align_up(n_part * h.geom.head_dim * sizeof(float), 256);
  return *o_bytes + n_part * 2 * sizeof(float);
}

template <int D>
static int launch_attention(ippd_layout* L, const IppdDev& d, int layer_begin, int layer_count, const void* q_raw,
                            void* out, float* part_o, float* part_ml, cudaStream_t stream, bool marks,
                            const void* k_step = nullptr, const void* v_step = nullptr) {
  {
    // once per device and head size; host threads making their first calls at the same time take turns
    static std::mutex mu;
    static bool attr_set[64] = {};
    std::lock_guard<std::mutex> lock(mu);
    int dev = L->device >= 0 && L->device < 64 ? L->device : 0;
    if (!attr_set[dev]) {
      CUDA_TRY(cudaFuncSetAttribute(ippd_attn_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    MmaCfg<D>::SMEM));
      CUDA_TRY(cudaFuncSetAttribute(ippd_attn_tc_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    tc_smem_bytes<D, false>()));
      CUDA_TRY(cudaFuncSetAttribute(ippd_attn_tc_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    tc_smem_bytes<D, true>()));
      attr_set[dev] = true;
    }
  }
  const IppdStepDev& S = L->step_dev;
  const int Hkv = L->h.geom.n_kv_heads;
  int out_f32 = L->h.geom.out_dtype == IPPD_F32;
  if (L->h.kernel_path() >= 2) {
    IppdTcArgs a;
    bool any_partial = false;
    {
      int rc = tc_partition(L, layer_count, &a, &any_partial);
      if (rc != IPPD_OK) return rc;
    }
    const int grid = a.n_cta;
    a.rb_tile_begin = L->d_rb_tile_begin;
    a.tiles = L->d_tc_tiles;
    a.pieces = L->d_tc_pieces;
    a.T1 = (int)L->plan.total_tiles;
    a.layer_begin = layer_begin;
    a.layer_count = layer_count;
    a.out_f32 = out_f32;
    a.k_step = (const __nv_bfloat16*)k_step;
    a.v_step = (const __nv_bfloat16*)v_step;
    if (marks) prof_mark(L, 0, true, stream);
    const bool kv8 = L->h.opt_kv_dtype == IPPD_KV_E4M3;
    CUDA_TRY(launch_pdl(kv8 ? ippd_attn_tc_kernel<D, true> : ippd_attn_tc_kernel<D, false>, dim3(grid),
                        dim3(IPPD_TC_THREADS), (size_t)(kv8 ? tc_smem_bytes<D, true>() : tc_smem_bytes<D, false>()),
                        stream, d, S, a, (const __nv_bfloat16*)q_raw, out, part_o, part_ml));
    if (marks) prof_mark(L, 0, false, stream);
    CUDA_TRY(cudaGetLastError());
    L->launches++;
    if (any_partial) {
      dim3 mg((unsigned)(grid - 1) * IPPD_TC_MERGE_SPLIT);
      if (marks) prof_mark(L, 1, true, stream);
      CUDA_TRY(launch_pdl(ippd_merge_tc_kernel<D>, mg, dim3(128), 0, stream, d, S, a, (const float*)part_o,
                          (const float*)part_ml, out));
      if (marks) prof_mark(L, 1, false, stream);
      CUDA_TRY(cudaGetLastError());
      L->launches++;
    }
    return IPPD_OK;
  }
  using C = MmaCfg<D>;
  dim3 grid((unsigned)S.n_units, (unsigned)Hkv, (unsigned)layer_count);
  if (marks) prof_mark(L, 0, true, stream);
  ippd_attn_mma_kernel<D><<<grid, C::THREADS, C::SMEM, stream>>>(d, S, layer_begin, (const __nv_bfloat16*)q_raw, out,
                                                                 out_f32, part_o, part_ml);
  if (marks) prof_mark(L, 0, false, stream);
  CUDA_TRY(cudaGetLastError());
  L->launches++;
  if (L->step_needs_merge) {
    dim3 mg((unsigned)S.n_rb, (unsigned)Hkv, (unsigned)layer_count);
    if (marks) prof_mark(L, 1, true, stream);
    ippd_merge_kernel<D><<<mg, 128, 0, stream>>>(d, S, S.RB, part_o, part_ml, out, out_f32);
    if (marks) prof_mark(L, 1, false, stream);
    CUDA_TRY(cudaGetLastError());
    L->launches++;
  }
  return IPPD_OK;
}

// Common body of ippd_decode_attention (k_step == NULL) and ippd_decode_step.
static int decode_attention_impl(ippd_layout_t* L, const char* who, int32_t layer_begin, int32_t layer_count,
                                 const void* q_raw, const void* k_step, const void* v_step, void* out, void* workspace,
                                 size_t workspace_bytes, void* stream_) {
  const std::string name(who);
  if (!L) { ippd_set_error(name + ": NULL layout"); return IPPD_ERR_INVALID_ARG; }
  if (!L->bound) { ippd_set_error(name + ": no cache bound"); return IPPD_ERR_NOT_BOUND; }
  if (!L->have_step) { ippd_set_error(name + ": call ippd_begin_step first"); return IPPD_ERR_INVALID_ARG; }
  const IppdHostLayout& h = L->h;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > h.geom.n_layers) {
    ippd_set_error(name + ": layer range out of bounds");
    return IPPD_ERR_INVALID_ARG;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  L->last_stream = stream;
  const IppdStepDev& S = L->step_dev;
  if (S.A == 0) return IPPD_OK;
  if (!q_raw || !out) { ippd_set_error(name + ": NULL q_raw / out"); return IPPD_ERR_INVALID_ARG; }
  size_t o_bytes = 0;
  bool needed = false;
  size_t need = scratch_need(L, layer_count, &o_bytes, &needed);
  float *part_o = nullptr, *part_ml = nullptr;
  if (needed) {
    if (!workspace || workspace_bytes < need || (uintptr_t)workspace % 256 != 0) {
      ippd_set_error(name + ": workspace missing, misaligned or too small");
      return IPPD_ERR_INVALID_ARG;
    }
    part_o = (float*)workspace;
    part_ml = (float*)((char*)workspace + o_bytes);
  }
  if (k_step && h.kernel_path() < 2) {
    // the warp-level path has no append role: the step's tokens go through the append kernel first
    int rc = ippd_append_kv(L, layer_begin, layer_count, IPPD_APPEND_STEP, nullptr, 0, k_step, v_step, stream_);
    if (rc != IPPD_OK) return rc;
    k_step = v_step = nullptr;
  }
  {
    int rc = ring_flush(L, stream);  // the step's descriptor, unless a STEP append carried it along
    if (rc != IPPD_OK) return rc;
  }
  IppdDev d = make_dev(L);
  if (h.geom.head_dim == 128)
    return launch_attention<128>(L, d, layer_begin, layer_count, q_raw, out, part_o, part_ml, stream, true, k_step, v_step);
  return launch_attention<64>(L, d, layer_begin, layer_count, q_raw, out, part_o, part_ml, stream, true, k_step, v_step);
}

extern "C" int ippd_decode_attention(ippd_layout_t* L, int32_t layer_begin, int32_t layer_count, const void* q_raw,
                                     void* out, void* workspace, size_t workspace_bytes, void* stream_) {
  return decode_attention_impl(L, "ippd_decode_attention", layer_begin, layer_count, q_raw, nullptr, nullptr, out,
                               workspace, workspace_bytes, stream_);
}

extern "C" int ippd_decode_step(ippd_layout_t* L, int32_t layer_begin, int32_t layer_count, const void* q_raw,
                                const void* k_raw, const void* v_raw, void* out, void* workspace,
                                size_t workspace_bytes, void* stream_) {
  if (L && L->have_step && L->step_dev.A > 0 && (!k_raw || !v_raw)) {
    ippd_set_error("ippd_decode_step: NULL k_raw / v_raw");
    return IPPD_ERR_INVALID_ARG;
  }
  return decode_attention_impl(L, "ippd_decode_step", layer_begin, layer_count, q_raw, k_raw, v_raw, out, workspace,
                               workspace_bytes, stream_);
}

// ---------------------------------------------------------------------------------------------
// Attention without any allocation: the split-KV partials live in a fixed array of the device image.
// In host code `g_ippd_static_scratch` is only a handle for the symbol, not a device address; the
// address a kernel may use comes from cudaGetSymbolAddress, looked up once per device below.
static __device__ __align__(256) unsigned char g_ippd_static_scratch[IPPD_STATIC_SCRATCH_BYTES];
static void* g_static_scratch_addr[64] = {};
static std::mutex g_static_scratch_mu;  // guards the table above: first calls may come from several host threads

extern "C" int ippd_decode_attention_static(ippd_layout_t* L, int32_t layer_begin, int32_t layer_count,
                                            const void* q_raw, void* out, void* stream_) {
  if (!L) { ippd_set_error("ippd_decode_attention_static: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  if (!L->bound) { ippd_set_error("ippd_decode_attention_static: no cache bound"); return IPPD_ERR_NOT_BOUND; }
  if (!L->have_step) { ippd_set_error("ippd_decode_attention_static: call ippd_begin_step first"); return IPPD_ERR_INVALID_ARG; }
  const IppdHostLayout& h = L->h;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > h.geom.n_layers) {
    ippd_set_error("ippd_decode_attention_static: layer range out of bounds");
    return IPPD_ERR_INVALID_ARG;
  }
  int dev = -1;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev != L->device || dev < 0 || dev >= 64) {
    ippd_set_error("ippd_decode_attention_static: the current device is not the one the cache was bound on");
    return IPPD_ERR_INVALID_ARG;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  L->last_stream = stream;
  const IppdStepDev& S = L->step_dev;
  if (S.A == 0) return IPPD_OK;
  if (!q_raw || !out) { ippd_set_error("ippd_decode_attention_static: NULL q_raw / out"); return IPPD_ERR_INVALID_ARG; }
  size_t o_bytes = 0;
  bool needed = false;
  size_t need = scratch_need(L, layer_count, &o_bytes, &needed);
  float *part_o = nullptr, *part_ml = nullptr;
  if (needed) {
    if (need > (size_t)IPPD_STATIC_SCRATCH_BYTES) {
      ippd_set_error("ippd_decode_attention_static: this step needs " + std::to_string(need) +
                     " bytes of scratch for " + std::to_string(layer_count) + " layers, the built-in array holds " +
                     std::to_string((size_t)IPPD_STATIC_SCRATCH_BYTES) +
                     "; pass fewer layers per call or raise IPPD_OPT_TILES_PER_SPLIT");
      return IPPD_ERR_CAPACITY;
    }
    void* base = nullptr;
    {
      std::lock_guard<std::mutex> lock(g_static_scratch_mu);
      if (!g_static_scratch_addr[dev]) {
        // first call on this device (it is the current one): resolve the symbol to its device address
        void* p = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&p, g_ippd_static_scratch));
        if (!p) { ippd_set_error("ippd_decode_attention_static: scratch symbol has no device address"); return IPPD_ERR_CUDA; }
        g_static_scratch_addr[dev] = p;
      }
      base = g_static_scratch_addr[dev];
    }
    part_o = (float*)base;
    part_ml = (float*)((char*)base + o_bytes);
  }
  {
    int rc = ring_flush(L, stream);  // the step's descriptor, unless a STEP append carried it along
    if (rc != IPPD_OK) return rc;
  }
  IppdDev d = make_dev(L);
  if (h.geom.head_dim == 128)
    return launch_attention<128>(L, d, layer_begin, layer_count, q_raw, out, part_o, part_ml, stream, false);
  return launch_attention<64>(L, d, layer_begin, layer_count, q_raw, out, part_o, part_ml, stream, false);
}

extern "C" int ippd_prefill_attention(ippd_layout_t* L, int32_t layer_begin, int32_t layer_count, const void* q_raw,
                                      const void* k_raw, const void* v_raw, void* out, void* workspace,
                                      size_t workspace_bytes, void* stream_) {
  if (!L) { ippd_set_error("ippd_prefill_attention: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  if (!L->bound) { ippd_set_error("ippd_prefill_attention: no cache bound"); return IPPD_ERR_NOT_BOUND; }
  const IppdHostLayout& h = L->h;
  if (h.kernel_path() < 2) { ippd_set_error("ippd_prefill_attention: tensor-core path only"); return IPPD_ERR_INVALID_ARG; }
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > h.geom.n_layers) {
    ippd_set_error("ippd_prefill_attention: layer range out of bounds");
    return IPPD_ERR_INVALID_ARG;
  }
  if (!q_raw || !k_raw || !v_raw || !out) { ippd_set_error("ippd_prefill_attention: NULL tensor"); return IPPD_ERR_INVALID_ARG; }
  cudaStream_t stream = (cudaStream_t)stream_;
  const int n_hdr = (int)h.hdr_pos.size();
  if (n_hdr == 0) return IPPD_OK;
  // 1. the header's K/V into the cache
  int rc = ippd_append_kv(L, layer_begin, layer_count, IPPD_APPEND_HEADER, nullptr, 0, k_raw, v_raw, stream_);
  if (rc != IPPD_OK) return rc;
  // 2. one query per header token, in header order
  std::vector<IppdPlanEntry> ent((size_t)n_hdr);
  int t = 0;
  for (; t < h.shared_len; ++t) ent[t] = {-1, -1, 0, 1};
  for (int b = 0; b < h.B; ++b) {
    for (int i = 0; i < h.ctx_len[b]; ++i, ++t) ent[t] = {b, -1, 0, 1};
    for (int k = h.q_begin[b]; k < h.q_begin[b + 1]; ++k)
      for (int j = 0; j < h.q_len[k]; ++j, ++t) ent[t] = {b, k, j + 1, 0};
  }
  L->have_step = false;
  L->pending_slot = -1;
  L->profile = L->profile_stride > 0;
  rc = ippd_host_plan_entries(h, ent.data(), h.hdr_pos.data(), n_hdr, layer_count, false, &L->plan);
  if (rc != IPPD_OK) return rc;
  const IppdStepPlan& P = L->plan;
  const StepBlobLayout bl = step_blob_layout((size_t)n_hdr, P.rbs.size(), P.units.size(), P.tc_tiles.size(), P.tc_pieces.size());
  std::vector<char> blob(bl.total, 0);
  memcpy(blob.data() + bl.off_rb, P.rbs.data(), P.rbs.size() * sizeof(IppdRowBlock));
  memcpy(blob.data() + bl.off_tb, P.rb_tile_begin.data(), P.rb_tile_begin.size() * 4);
  memcpy(blob.data() + bl.off_tt, P.tc_tiles.data(), P.tc_tiles.size() * sizeof(IppdTcTile));
  if (!P.tc_pieces.empty()) memcpy(blob.data() + bl.off_tp, P.tc_pieces.data(), P.tc_pieces.size() * sizeof(IppdTcPiece));
  memcpy(blob.data() + bl.off_pos, P.act_pos.data(), (size_t)n_hdr * 4);
  if (bl.total > L->prefill_cap) {
    CUDA_TRY(cudaStreamSynchronize(stream));  // an earlier prefill may still read the old buffer
    cudaFree(L->prefill_dev);
    L->prefill_dev = nullptr;
    L->prefill_cap = 0;
    if (cudaMalloc((void**)&L->prefill_dev, bl.total) != cudaSuccess) { ippd_set_error("ippd_prefill_attention: out of device memory"); return IPPD_ERR_OOM; }
    L->prefill_cap = bl.total;
  }
  CUDA_TRY(cudaMemcpyAsync(L->prefill_dev, blob.data(), bl.total, cudaMemcpyHostToDevice, stream));
  CUDA_TRY(cudaStreamSynchronize(stream));  // `blob` is pageable host memory of this call
  char* dev = L->prefill_dev;
  L->step_dev.act_q = (const int32_t*)(dev + bl.off_q);
  L->step_dev.act_s = (const int32_t*)(dev + bl.off_s);
  L->step_dev.rbs = (const IppdRowBlock*)(dev + bl.off_rb);
  L->step_dev.act_pos = (const int32_t*)(dev + bl.off_pos);
  L->step_dev.units = (const IppdUnit*)(dev + bl.off_u);
  L->d_rb_tile_begin = (const int32_t*)(dev + bl.off_tb);
  L->d_tc_tiles = (const IppdTcTile*)(dev + bl.off_tt);
  L->d_tc_pieces = (const IppdTcPiece*)(dev + bl.off_tp);
  L->step_dev.A = n_hdr;
  L->step_dev.n_rb = P.hdr.n_rowblocks;
  L->step_dev.n_units = 0;
  L->step_dev.RB = P.hdr.rows_per_block;
  L->last_stream = stream;
  // 3. the attention pass
  L->have_step = true;
  size_t o_bytes = 0;
  bool needed = false;
  const size_t need = scratch_need(L, layer_count, &o_bytes, &needed);
  float *part_o = nullptr, *part_ml = nullptr;
  if (needed) {
    if (!workspace || workspace_bytes < need || (uintptr_t)workspace % 256 != 0) {
      L->have_step = false;
      ippd_set_error("ippd_prefill_attention: workspace missing, misaligned or too small");
      return IPPD_ERR_INVALID_ARG;
    }
    part_o = (float*)workspace;
    part_ml = (float*)((char*)workspace + o_bytes);
  }
  IppdDev d = make_dev(L);
  rc = h.geom.head_dim == 128
           ? launch_attention<128>(L, d, layer_begin, layer_count, q_raw, out, part_o, part_ml, stream, true)
           : launch_attention<64>(L, d, layer_begin, layer_count, q_raw, out, part_o, part_ml, stream, true);
  L->have_step = false;  // the work list in force is the prefill's: a decode step must be declared anew
  L->profile = false;
  return rc;
}

extern "C" int ippd_decode_step_grouped(ippd_layout_t* L, int32_t layers_per_call, const void* q_raw, const void* k_raw,
                                        const void* v_raw, void* out, void* workspace, size_t workspace_bytes,
                                        void* stream_) {
  if (!L) { ippd_set_error("ippd_decode_step_grouped: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  const ippd_geometry_t& g = L->h.geom;
  if (layers_per_call < 1 || layers_per_call > g.n_layers) {
    ippd_set_error("ippd_decode_step_grouped: bad layers_per_call");
    return IPPD_ERR_INVALID_ARG;
  }
  const size_t A = L->have_step ? (size_t)L->step_dev.A : 0;
  const size_t q_layer = A * g.n_q_heads * g.head_dim * 2, kv_layer = A * g.n_kv_heads * g.head_dim * 2;
  const size_t o_layer = A * g.n_q_heads * g.head_dim * (g.out_dtype == IPPD_F32 ? 4 : 2);
  for (int l0 = 0; l0 < g.n_layers; l0 += layers_per_call) {
    const int n = std::min(layers_per_call, g.n_layers - l0);
    int rc = ippd_decode_step(L, l0, n, (const char*)q_raw + l0 * q_layer, (const char*)k_raw + l0 * kv_layer,
                              (const char*)v_raw + l0 * kv_layer, (char*)out + l0 * o_layer, workspace,
                              workspace_bytes, stream_);
    if (rc != IPPD_OK) return rc;
  }
  return IPPD_OK;
}

extern "C" int ippd_read_probe(ippd_layout_t* L, int32_t layer_begin, int32_t layer_count, void* stream_) {
  if (!L) { ippd_set_error("ippd_read_probe: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  if (!L->bound) { ippd_set_error("ippd_read_probe: no cache bound"); return IPPD_ERR_NOT_BOUND; }
  if (!L->have_step || L->h.kernel_path() < 2) {
    ippd_set_error("ippd_read_probe: needs a step declared for the tensor-core path");
    return IPPD_ERR_INVALID_ARG;
  }
  const IppdHostLayout& h = L->h;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > h.geom.n_layers) {
    ippd_set_error("ippd_read_probe: layer range out of bounds");
    return IPPD_ERR_INVALID_ARG;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  L->last_stream = stream;
  if (L->step_dev.A == 0) return IPPD_OK;
  int rc = ring_flush(L, stream);
  if (rc != IPPD_OK) return rc;
  IppdTcArgs a = {};
  bool any_partial = false;
  rc = tc_partition(L, layer_count, &a, &any_partial);
  if (rc != IPPD_OK) return rc;
  const int grid = a.n_cta;
  a.rb_tile_begin = L->d_rb_tile_begin;
  a.tiles = L->d_tc_tiles;
  a.pieces = L->d_tc_pieces;
  a.T1 = (int)L->plan.total_tiles;
  a.layer_begin = layer_begin;
  a.layer_count = layer_count;
  IppdDev d = make_dev(L);
  const int D = h.geom.head_dim;
  const bool kv8 = h.opt_kv_dtype == IPPD_KV_E4M3;
  auto kern = D == 128 ? (kv8 ? ippd_read_probe_kernel<128, true> : ippd_read_probe_kernel<128, false>)
                       : (kv8 ? ippd_read_probe_kernel<64, true> : ippd_read_probe_kernel<64, false>);
  const size_t nbuf = kv8 ? TcCfg<128, true>::NBUF : TcCfg<128, false>::NBUF;
  const size_t smem = nbuf * h.tile_bytes() + nbuf * sizeof(uint64_t);
  CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<grid, 64, smem, stream>>>(d, L->step_dev, a);
  CUDA_TRY(cudaGetLastError());
  L->launches++;
  return IPPD_OK;
}

extern "C" int ippd_step_stage_bytes(const ippd_layout_t* L, int32_t A, size_t* bytes) {
  if (!L || !bytes || A < 0) { ippd_set_error("ippd_step_stage_bytes: bad argument"); return IPPD_ERR_INVALID_ARG; }
  const ippd_geometry_t& g = L->h.geom;
  size_t q = align_up((size_t)g.n_layers * A * g.n_q_heads * g.head_dim * 2, 256);
  size_t kv = align_up((size_t)g.n_layers * A * g.n_kv_heads * g.head_dim * 2, 256);
  size_t o = align_up((size_t)g.n_layers * A * g.n_q_heads * g.head_dim * (g.out_dtype == IPPD_F32 ? 4 : 2), 256);
  *bytes = q + 2 * kv + o;
  return IPPD_OK;
}

extern "C" int ippd_decode_step_host(ippd_layout_t* L, const int32_t* active_q, const int32_t* answer_idx, int32_t A,
                                     const void* host_q, const void* host_k, const void* host_v, void* host_out,
                                     void* dev_stage, size_t dev_stage_bytes, void* workspace, size_t workspace_bytes,
                                     void* stream_) {
  if (!L) { ippd_set_error("ippd_decode_step_host: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  size_t need = 0;
  int rc = ippd_step_stage_bytes(L, A, &need);
  if (rc != IPPD_OK) return rc;
  if (A > 0 && (!host_q || !host_k || !host_v || !host_out || !dev_stage || dev_stage_bytes < need ||
                (uintptr_t)dev_stage % 256 != 0)) {
    ippd_set_error("ippd_decode_step_host: bad buffers");
    return IPPD_ERR_INVALID_ARG;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  const ippd_geometry_t& g = L->h.geom;
  size_t qb = (size_t)g.n_layers * A * g.n_q_heads * g.head_dim * 2;
  size_t kvb = (size_t)g.n_layers * A * g.n_kv_heads * g.head_dim * 2;
  size_t ob = (size_t)g.n_layers * A * g.n_q_heads * g.head_dim * (g.out_dtype == IPPD_F32 ? 4 : 2);
  char* dq = (char*)dev_stage;
  char* dk = dq + align_up(qb, 256);
  char* dv = dk + align_up(kvb, 256);
  char* dout = dv + align_up(kvb, 256);
  rc = ippd_begin_step(L, active_q, answer_idx, A, stream_);
  if (rc != IPPD_OK) return rc;
  if (A == 0) return IPPD_OK;
  CUDA_TRY(cudaMemcpyAsync(dq, host_q, qb, cudaMemcpyHostToDevice, stream));
  CUDA_TRY(cudaMemcpyAsync(dk, host_k, kvb, cudaMemcpyHostToDevice, stream));
  CUDA_TRY(cudaMemcpyAsync(dv, host_v, kvb, cudaMemcpyHostToDevice, stream));
  rc = ippd_decode_step(L, 0, g.n_layers, dq, dk, dv, dout, workspace, workspace_bytes, stream_);
  if (rc != IPPD_OK) return rc;
  CUDA_TRY(cudaMemcpyAsync(host_out, dout, ob, cudaMemcpyDeviceToHost, stream));
  CUDA_TRY(cudaStreamSynchronize(stream));
  return IPPD_OK;
}

// Pipelined form of ippd_decode_step_host.  Slot (n & 1) of the staging buffer serves the n-th call:
//   copy-in stream : waits until the kernels that last read the slot's inputs are done, then copies q, k, v in;
//   caller's stream: waits for that copy and for the copy-out that last read the slot's output, runs the step;
//   copy-out stream: waits for the step, copies the output to the host.
// Nothing here waits on the host, so the copies of neighbouring steps overlap this step's kernels.
extern "C" int ippd_decode_step_host_async(ippd_layout_t* L, const int32_t* active_q, const int32_t* answer_idx,
                                           int32_t A, const void* host_q, const void* host_k, const void* host_v,
                                           void* host_out, void* dev_stage, size_t dev_stage_bytes, void* workspace,
                                           size_t workspace_bytes, void* stream_) {
  if (!L) { ippd_set_error("ippd_decode_step_host_async: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  size_t need = 0;
  int rc = ippd_step_stage_bytes(L, A, &need);
  if (rc != IPPD_OK) return rc;
  const size_t slot_bytes = (dev_stage_bytes / 2) & ~(size_t)255;
  if (A > 0 && (!host_q || !host_k || !host_v || !host_out || !dev_stage || slot_bytes < need ||
                (uintptr_t)dev_stage % 256 != 0)) {
    ippd_set_error("ippd_decode_step_host_async: bad buffers (the staging buffer holds two slots of ippd_step_stage_bytes)");
    return IPPD_ERR_INVALID_ARG;
  }
  if (!L->hs_init) {
    CUDA_TRY(cudaStreamCreateWithFlags(&L->hs_in, cudaStreamNonBlocking));
    CUDA_TRY(cudaStreamCreateWithFlags(&L->hs_out, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i) {
      CUDA_TRY(cudaEventCreateWithFlags(&L->hs_ev_in[i], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&L->hs_ev_done[i], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&L->hs_ev_out[i], cudaEventDisableTiming));
    }
    L->hs_init = true;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  const ippd_geometry_t& g = L->h.geom;
  size_t qb = (size_t)g.n_layers * A * g.n_q_heads * g.head_dim * 2;
  size_t kvb = (size_t)g.n_layers * A * g.n_kv_heads * g.head_dim * 2;
  size_t ob = (size_t)g.n_layers * A * g.n_q_heads * g.head_dim * (g.out_dtype == IPPD_F32 ? 4 : 2);
  if (A == 0) return ippd_begin_step(L, active_q, answer_idx, A, stream_);
  const int slot = (int)(L->hs_count & 1);
  const bool reused = L->hs_count >= 2;
  L->hs_count++;
  char* dq = (char*)dev_stage + (size_t)slot * slot_bytes;
  char* dk = dq + align_up(qb, 256);
  char* dv = dk + align_up(kvb, 256);
  char* dout = dv + align_up(kvb, 256);
  if (reused) CUDA_TRY(cudaStreamWaitEvent(L->hs_in, L->hs_ev_done[slot], 0));
  CUDA_TRY(cudaMemcpyAsync(dq, host_q, qb, cudaMemcpyHostToDevice, L->hs_in));
  CUDA_TRY(cudaMemcpyAsync(dk, host_k, kvb, cudaMemcpyHostToDevice, L->hs_in));
  CUDA_TRY(cudaMemcpyAsync(dv, host_v, kvb, cudaMemcpyHostToDevice, L->hs_in));
  CUDA_TRY(cudaEventRecord(L->hs_ev_in[slot], L->hs_in));
  // The step's descriptor is copied on the caller's stream, behind the previous step's kernels; the copy engine
  // takes copies in the order they were issued, so the input copies above go first: issued after it they would
  // wait for those kernels too instead of overlapping them.
  rc = ippd_begin_step(L, active_q, answer_idx, A, stream_);
  if (rc != IPPD_OK) return rc;
  CUDA_TRY(cudaStreamWaitEvent(stream, L->hs_ev_in[slot], 0));
  if (reused) CUDA_TRY(cudaStreamWaitEvent(stream, L->hs_ev_out[slot], 0));
  rc = ippd_decode_step(L, 0, g.n_layers, dq, dk, dv, dout, workspace, workspace_bytes, stream_);
  if (rc != IPPD_OK) return rc;
  CUDA_TRY(cudaEventRecord(L->hs_ev_done[slot], stream));
  CUDA_TRY(cudaStreamWaitEvent(L->hs_out, L->hs_ev_done[slot], 0));
  CUDA_TRY(cudaMemcpyAsync(host_out, dout, ob, cudaMemcpyDeviceToHost, L->hs_out));
  CUDA_TRY(cudaEventRecord(L->hs_ev_out[slot], L->hs_out));
  return IPPD_OK;
}

extern "C" int ippd_host_steps_wait(ippd_layout_t* L, void* stream_) {
  if (!L) { ippd_set_error("ippd_host_steps_wait: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream_));
  if (L->hs_init) {
    CUDA_TRY(cudaStreamSynchronize(L->hs_in));
    CUDA_TRY(cudaStreamSynchronize(L->hs_out));
  }
  return IPPD_OK;
}

extern "C" int ippd_export_mask(ippd_layout_t* L, int32_t prompt, const int32_t* n_answer, uint8_t* host_out,
                                int64_t* n_tokens) {
  if (!L || !n_answer || !n_tokens) { ippd_set_error("ippd_export_mask: NULL argument"); return IPPD_ERR_INVALID_ARG; }
  const IppdHostLayout& h = L->h;
  if (prompt < 0 || prompt >= h.B) { ippd_set_error("ippd_export_mask: prompt out of range"); return IPPD_ERR_INVALID_ARG; }
  std::vector<IppdMaskTok> toks;  // shared instruction and context tokens: kind 0, idx = virtual position
  for (int i = 0; i < h.shared_len + h.ctx_len[prompt]; ++i) toks.push_back({0, -1, i, 0});
  int k0 = h.q_begin[prompt], k1 = h.q_begin[prompt + 1];
  int max_t = 0;
  for (int k = k0; k < k1; ++k) {
    for (int j = 0; j < h.q_len[k]; ++j) toks.push_back({1, k, j, 0});
    if (n_answer[k - k0] < 0 || n_answer[k - k0] > h.max_new[k]) {
      ippd_set_error("ippd_export_mask: n_answer out of range");
      return IPPD_ERR_INVALID_ARG;
    }
    max_t = std::max(max_t, n_answer[k - k0]);
  }
  for (int t = 0; t < max_t; ++t)
    for (int k = k0; k < k1; ++k)
      if (n_answer[k - k0] > t) toks.push_back({2, k, t, 0});
  int64_t n = (int64_t)toks.size();
  *n_tokens = n;
  if (!host_out) return IPPD_OK;
  if (!L->bound) { ippd_set_error("ippd_export_mask: no cache bound"); return IPPD_ERR_NOT_BOUND; }
  if (n == 0) return IPPD_OK;
  if (n > 8192) { ippd_set_error("ippd_export_mask: sequence too long for a dense mask"); return IPPD_ERR_INVALID_ARG; }
  IppdMaskTok* d_toks = nullptr;
  uint8_t* d_out = nullptr;
  CUDA_TRY(cudaMalloc((void**)&d_toks, n * sizeof(IppdMaskTok)));
  if (cudaMalloc((void**)&d_out, n * n) != cudaSuccess) { cudaFree(d_toks); ippd_set_error("ippd_export_mask: cudaMalloc"); return IPPD_ERR_CUDA; }
  cudaMemcpy(d_toks, toks.data(), n * sizeof(IppdMaskTok), cudaMemcpyHostToDevice);
  ippd_export_mask_kernel<<<(unsigned)((n * n + 255) / 256), 256>>>(make_dev(L), d_toks, (int)n, d_out);
  L->launches++;
  cudaError_t e = cudaMemcpy(host_out, d_out, n * n, cudaMemcpyDeviceToHost);
  cudaFree(d_toks);
  cudaFree(d_out);
  if (e != cudaSuccess) { ippd_set_error(std::string("ippd_export_mask: ") + cudaGetErrorString(e)); return IPPD_ERR_CUDA; }
  return IPPD_OK;
}

extern "C" int ippd_poll_status(ippd_layout_t* L, int32_t* word) {
  if (!L || !word) { ippd_set_error("ippd_poll_status: NULL argument"); return IPPD_ERR_INVALID_ARG; }
  if (!L->bound) { ippd_set_error("ippd_poll_status: no cache bound"); return IPPD_ERR_NOT_BOUND; }
  CUDA_TRY(cudaStreamSynchronize(L->last_stream));
  CUDA_TRY(cudaMemcpy(word, L->d_error, sizeof(int32_t), cudaMemcpyDeviceToHost));
  if (*word) CUDA_TRY(cudaMemset(L->d_error, 0, sizeof(int32_t)));  // reported once; the layout stays usable
  if (*word & IPPD_ERRBIT_TIMEOUT) { ippd_set_error("a bounded device-side wait ran out"); return IPPD_ERR_TIMEOUT; }
  if (*word & IPPD_ERRBIT_RANGE) { ippd_set_error("an id or slot was out of range on the device"); return IPPD_ERR_INVALID_ARG; }
  if (*word & IPPD_ERRBIT_NONFINITE) { ippd_set_error("ippd_append_kv was handed a NaN or an infinity"); return IPPD_ERR_INVALID_ARG; }
  return IPPD_OK;
}

extern "C" int ippd_profile_read(ippd_layout_t* L, double* attention_ms, double* merge_ms, double* append_ms,
                                 int64_t* n_attention) {
  if (!L) { ippd_set_error("ippd_profile_read: NULL layout"); return IPPD_ERR_INVALID_ARG; }
  double sum[3] = {0, 0, 0};
  int64_t n_att = 0;
  if (L->ev_used) CUDA_TRY(cudaEventSynchronize(L->ev_pool[L->ev_used - 1]));
  for (size_t i = 0; i + 1 < L->ev_used && i / 2 < L->ev_kind.size(); i += 2) {
    float ms = 0.f;
    CUDA_TRY(cudaEventElapsedTime(&ms, L->ev_pool[i], L->ev_pool[i + 1]));
    int kind = L->ev_kind[i / 2];
    sum[kind] += ms;
    n_att += kind == 0;
  }
  L->ev_used = 0;
  L->ev_kind.clear();
  if (attention_ms) *attention_ms = sum[0];
  if (merge_ms) *merge_ms = sum[1];
  if (append_ms) *append_ms = sum[2];
  if (n_attention) *n_attention = n_att;
  return IPPD_OK;
}

extern "C" int64_t ippd_launch_count(const ippd_layout_t* L) { return L ? L->launches : 0; }

extern "C" void ippd_destroy_layout(ippd_layout_t* L) {
  if (!L) return;
  if (L->bound) {
    cudaStreamSynchronize(L->last_stream);
    free_device(L);
  }
  for (cudaEvent_t e : L->ev_pool) cudaEventDestroy(e);
  if (L->hs_init) {
    cudaStreamSynchronize(L->hs_in);
    cudaStreamSynchronize(L->hs_out);
    for (int i = 0; i < 2; ++i) {
      cudaEventDestroy(L->hs_ev_in[i]);
      cudaEventDestroy(L->hs_ev_done[i]);
      cudaEventDestroy(L->hs_ev_out[i]);
    }
    cudaStreamDestroy(L->hs_in);
    cudaStreamDestroy(L->hs_out);
  }
  delete L;
}
