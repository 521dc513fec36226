// Small kernels around the attention: RoPE table, RoPE + append into the tiled cache, dense mask export.
#pragma once
#include "ippd_device.cuh"

// cos/sin of pos * theta^(-2i/D), angle and functions evaluated in fp64, stored as fp32 pairs.
__global__ void ippd_rope_table_kernel(float2* table, int max_pos, int D, double theta) {
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  int half = D / 2;
  if (idx >= (long long)(max_pos + 1) * half) return;
  int pos = (int)(idx / half), i = (int)(idx % half);
  double inv_freq = pow(theta, -2.0 * (double)i / (double)D);
  double s, c;
  sincos((double)pos * inv_freq, &s, &c);
  table[idx] = make_float2((float)c, (float)s);
}

// RoPE + store of one (token, KV head, pair of 16-byte chunks c and c + D/16): the two halves of 8 rotation pairs of K,
// and the same two chunks of V.  k_src / v_src point at chunk c of the token's raw row; `k_tile` is the byte offset of
// the K half of the destination cache tile (its V half follows it), `u` the token's row inside the tile.  Cache tile
// layout (K and V alike): [token/8][d/8][token%8][d%8] bf16, i.e. 8x8 blocks of 128 contiguous bytes.
// KV8: the rotated key and the value are stored as e4m3 bytes, [token/8][d/16][token%8][d%16] (8x16 blocks of 128
// bytes); a thread's 8 values are half of a block row.
template <int D, bool KV8 = false>
__device__ __forceinline__ void ippd_rope_store_pair(const IppdDev& L, const __nv_bfloat16* __restrict__ k_src,
                                                     const __nv_bfloat16* __restrict__ v_src, int pos, int c,
                                                     size_t k_tile, int u) {
  constexpr int CP = D / 16;
  constexpr int GB = (D / 8) * 128;
  uint4 klo = *reinterpret_cast<const uint4*>(k_src);
  uint4 khi = *reinterpret_cast<const uint4*>(k_src + D / 2);
  uint4 vlo = *reinterpret_cast<const uint4*>(v_src);
  uint4 vhi = *reinterpret_cast<const uint4*>(v_src + D / 2);
  {
    // A NaN or an infinity (bf16: all exponent bits set) is stored like any value but reported: a cache row shares
    // its 128-row tile with rows of other questions, and 0 x NaN would reach their outputs too.
    const uint32_t* w[4] = {reinterpret_cast<const uint32_t*>(&klo), reinterpret_cast<const uint32_t*>(&khi),
                            reinterpret_cast<const uint32_t*>(&vlo), reinterpret_cast<const uint32_t*>(&vhi)};
    bool bad = false;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        bad |= (w[i][e] & 0x7F800000u) == 0x7F800000u || (w[i][e] & 0x00007F80u) == 0x00007F80u;
    if (bad) atomicOr(L.error_word, IPPD_ERRBIT_NONFINITE);
  }
  const float2* cs = L.rope + (size_t)pos * (D / 2) + c * 8;
  const __nv_bfloat162* pl = reinterpret_cast<const __nv_bfloat162*>(&klo);
  const __nv_bfloat162* ph = reinterpret_cast<const __nv_bfloat162*>(&khi);
  if constexpr (KV8) {
    constexpr int GB8 = (D / 16) * 128;
    float kl[8], kh[8];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float2 c0 = cs[2 * e], c1 = cs[2 * e + 1];
      float l0 = __bfloat162float(pl[e].x), l1 = __bfloat162float(pl[e].y);
      float h0 = __bfloat162float(ph[e].x), h1 = __bfloat162float(ph[e].y);
      kl[2 * e] = l0 * c0.x - h0 * c0.y;
      kl[2 * e + 1] = l1 * c1.x - h1 * c1.y;
      kh[2 * e] = h0 * c0.x + l0 * c0.y;
      kh[2 * e + 1] = h1 * c1.x + l1 * c1.y;
    }
    const __nv_bfloat16* vl = reinterpret_cast<const __nv_bfloat16*>(&vlo);
    const __nv_bfloat16* vh = reinterpret_cast<const __nv_bfloat16*>(&vhi);
    auto f = [](__nv_bfloat16 x) { return __bfloat162float(x); };
    const uint2 k_lo8 = make_uint2(pack_e4m3x4(kl[0], kl[1], kl[2], kl[3]), pack_e4m3x4(kl[4], kl[5], kl[6], kl[7]));
    const uint2 k_hi8 = make_uint2(pack_e4m3x4(kh[0], kh[1], kh[2], kh[3]), pack_e4m3x4(kh[4], kh[5], kh[6], kh[7]));
    const uint2 v_lo8 = make_uint2(pack_e4m3x4(f(vl[0]), f(vl[1]), f(vl[2]), f(vl[3])),
                                   pack_e4m3x4(f(vl[4]), f(vl[5]), f(vl[6]), f(vl[7])));
    const uint2 v_hi8 = make_uint2(pack_e4m3x4(f(vh[0]), f(vh[1]), f(vh[2]), f(vh[3])),
                                   pack_e4m3x4(f(vh[4]), f(vh[5]), f(vh[6]), f(vh[7])));
    // values d = 8c.. sit in 16-value block c/2, half c%2; the rotation partners D/2 further in block D/32 + c/2
    const size_t in_tile = (size_t)(u >> 3) * GB8 + (size_t)(u & 7) * 16 + (size_t)(c & 1) * 8;
    char* kdst = L.cache + k_tile + in_tile;
    char* vdst = kdst + (size_t)IPPD_TILE_TOKENS * D;  // the V half of the tile follows its K half
    *reinterpret_cast<uint2*>(kdst + (c >> 1) * 128) = k_lo8;
    *reinterpret_cast<uint2*>(kdst + (D / 32 + (c >> 1)) * 128) = k_hi8;
    *reinterpret_cast<uint2*>(vdst + (c >> 1) * 128) = v_lo8;
    *reinterpret_cast<uint2*>(vdst + (D / 32 + (c >> 1)) * 128) = v_hi8;
  } else {
    uint4 olo, ohi;
    uint32_t* wl = reinterpret_cast<uint32_t*>(&olo);
    uint32_t* wh = reinterpret_cast<uint32_t*>(&ohi);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float2 c0 = cs[2 * e], c1 = cs[2 * e + 1];
      float l0 = __bfloat162float(pl[e].x), l1 = __bfloat162float(pl[e].y);
      float h0 = __bfloat162float(ph[e].x), h1 = __bfloat162float(ph[e].y);
      wl[e] = pack_bf16(l0 * c0.x - h0 * c0.y, l1 * c1.x - h1 * c1.y);
      wh[e] = pack_bf16(h0 * c0.x + l0 * c0.y, h1 * c1.x + l1 * c1.y);
    }
    const size_t in_tile = (size_t)(u >> 3) * GB + (size_t)(u & 7) * 16;
    char* kdst = L.cache + k_tile + in_tile;
    char* vdst = kdst + (size_t)IPPD_TILE_TOKENS * D * 2;  // the V half of the tile follows its K half
    *reinterpret_cast<uint4*>(kdst + c * 128) = olo;
    *reinterpret_cast<uint4*>(kdst + (c + CP) * 128) = ohi;
    *reinterpret_cast<uint4*>(vdst + c * 128) = vlo;
    *reinterpret_cast<uint4*>(vdst + (c + CP) * 128) = vhi;
  }
}

#define IPPD_APPEND_INLINE 64

struct IppdAppendArgs {
  int kind;                  // IPPD_APPEND_*
  int n_tokens;              // tokens per layer
  int n_ids;
  const int32_t* ids;        // device: prompt or question ids (CONTEXT / QUESTION)
  const int32_t* tok_begin;  // device: [n_ids+1] first token of each id
  const int32_t* q_first;    // device: [B+1] first question of each prompt (HEADER)
  // STEP appends of at most IPPD_APPEND_INLINE tokens carry the step's active list in the kernel parameters and also
  // move the step's descriptor from its pinned slot to the device (blocks past the first n_append_blocks of row 0):
  // the append does not have to wait for a separate upload kernel, and the upload's PCIe latency hides behind it.
  int inline_acts;
  int n_append_blocks;
  unsigned up_n16;
  const uint4* up_src;
  uint4* up_dst;
  int32_t act_q[IPPD_APPEND_INLINE], act_s[IPPD_APPEND_INLINE];
};

// One thread moves one (token, KV head, pair of 16-byte chunks c and c + D/16), see ippd_rope_store_pair.
template <int D, bool KV8 = false>
__global__ void __launch_bounds__(256)
ippd_append_kernel(IppdDev L, IppdStepDev S, IppdAppendArgs a, int layer_begin,
                   const __nv_bfloat16* __restrict__ k_raw, const __nv_bfloat16* __restrict__ v_raw) {
  constexpr int CP = D / 16;  // chunk pairs per row
  pdl_trigger();
  pdl_wait();
  if (a.n_append_blocks > 0 && (int)blockIdx.x >= a.n_append_blocks) {
    if (blockIdx.y == 0) {
      const unsigned i = (blockIdx.x - a.n_append_blocks) * blockDim.x + threadIdx.x;
      if (i < a.up_n16) a.up_dst[i] = a.up_src[i];
    }
    return;
  }
  long long item = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  long long total = (long long)a.n_tokens * L.Hkv * CP;
  if (item >= total) return;
  int c = (int)(item % CP);
  int head = (int)((item / CP) % L.Hkv);
  int tok = (int)(item / ((long long)CP * L.Hkv));
  int ll = blockIdx.y, layer = layer_begin + ll;

  int pos;
  long long tile;
  int u;
  if (a.kind == IPPD_APPEND_STEP) {
    int qid = a.inline_acts ? a.act_q[tok] : S.act_q[tok];
    int slot = L.q_len[qid] + (a.inline_acts ? a.act_s[tok] : S.act_s[tok]);
    pos = L.shared_len + L.ctx_len[L.prompt_of[qid]] + slot;
    tile = L.branch_tile_off[qid] + slot / IPPD_TILE_TOKENS;
    u = slot % IPPD_TILE_TOKENS;
  } else if (a.kind == IPPD_APPEND_SHARED || (a.kind == IPPD_APPEND_HEADER && tok < L.shared_len)) {
    pos = tok;
    tile = tok / IPPD_TILE_TOKENS;
    u = tok % IPPD_TILE_TOKENS;
  } else if (a.kind == IPPD_APPEND_HEADER) {
    // token `tok` of the stacked header: find its prompt, then whether it is a context or a question token
    int lo = 0, hi = a.n_ids - 1;  // n_ids = number of prompts
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (L.hdr_begin[mid] <= tok) lo = mid; else hi = mid - 1;
    }
    const int b = lo, i = tok - L.hdr_begin[b];
    if (i < L.ctx_len[b]) {
      pos = L.shared_len + i;
      tile = L.ctx_tile_off[b] + i / IPPD_TILE_TOKENS;
      u = i % IPPD_TILE_TOKENS;
    } else {
      int qlo = a.q_first[b], qhi = a.q_first[b + 1] - 1;  // questions of prompt b
      while (qlo < qhi) {
        int mid = (qlo + qhi + 1) >> 1;
        if (L.q_hdr_begin[mid] <= tok) qlo = mid; else qhi = mid - 1;
      }
      const int j = tok - L.q_hdr_begin[qlo];
      pos = L.shared_len + L.ctx_len[b] + j;
      tile = L.branch_tile_off[qlo] + j / IPPD_TILE_TOKENS;
      u = j % IPPD_TILE_TOKENS;
    }
  } else {
    int lo = 0, hi = a.n_ids - 1;  // last id whose first token is <= tok
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (a.tok_begin[mid] <= tok) lo = mid; else hi = mid - 1;
    }
    int id = a.ids[lo], i = tok - a.tok_begin[lo];
    if (a.kind == IPPD_APPEND_CONTEXT) {
      pos = L.shared_len + i;
      tile = L.ctx_tile_off[id] + i / IPPD_TILE_TOKENS;
    } else {
      pos = L.shared_len + L.ctx_len[L.prompt_of[id]] + i;
      tile = L.branch_tile_off[id] + i / IPPD_TILE_TOKENS;
    }
    u = i % IPPD_TILE_TOKENS;
  }
  if (pos < 0 || pos > L.max_pos || tile < 0 || tile >= L.n_tiles) {
    atomicOr(L.error_word, IPPD_ERRBIT_RANGE);
    return;
  }
  size_t src = (((size_t)ll * a.n_tokens + tok) * L.Hkv + head) * D + c * 8;
  ippd_rope_store_pair<D, KV8>(L, k_raw + src, v_raw + src, pos, c, ippd_tile_addr<KV8>(L, layer, head, tile, 0), u);
}

// Token descriptor of the mask export: kind 0 = context token, 1 = question token, 2 = answer token.
struct IppdMaskTok {
  int32_t kind;
  int32_t q;    // global question id (kinds 1, 2)
  int32_t idx;  // index inside its block (context index, question-token index, answer index t)
  int32_t pad;
};

// Row r attends column c iff c lies in the key set the attention kernels stream for r: the prompt's
// context (for context rows: up to r itself) and the row's own branch slots up to its own slot.
__global__ void ippd_export_mask_kernel(IppdDev L, const IppdMaskTok* toks, int n, uint8_t* out) {
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n * n) return;
  int r = (int)(idx / n), c = (int)(idx % n);
  IppdMaskTok tr = toks[r], tc = toks[c];
  bool ok;
  if (tc.kind == 0) {
    ok = (tr.kind != 0) || (tc.idx <= tr.idx);
  } else if (tr.kind == 0 || tr.q != tc.q) {
    ok = false;
  } else {
    int slot_r = (tr.kind == 1) ? tr.idx : L.q_len[tr.q] + tr.idx;
    int slot_c = (tc.kind == 1) ? tc.idx : L.q_len[tc.q] + tc.idx;
    ok = slot_c <= slot_r;
  }
  out[idx] = ok ? 1 : 0;
}

// Copies a step descriptor from pinned host memory (read through its device mapping) to device memory.  Launched
// programmatically: nothing it touches depends on the kernel before it in the stream (the host wrote the pinned slot
// before the launch, and the device slot's previous readers finished long ago), so the copy runs first and the wait
// for that kernel comes last -- it only keeps the stream's order for the kernels that follow.
__global__ void __launch_bounds__(256) ippd_upload_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                          unsigned n16) {
  pdl_trigger();
  const unsigned i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n16) dst[i] = src[i];
  pdl_wait();
}
