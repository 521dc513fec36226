// Split-KV IPPD decode attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM).
//
// Persistent kernel, one CTA per SM.  The key tiles of the whole launch form one sequence
//   for layer, for KV head, for row block: [context tiles of its prompt | packed branch tiles of its questions]
// and CTA c owns the contiguous slice [c*chunk, (c+1)*chunk) of it, cut wherever the slice ends (split-KV
// happens only at those cuts).  A row block is up to 128 query rows (questions x G heads), row r <-> TMEM lane r.
// A context tile is 128 consecutive context tokens.  A packed branch tile holds PIECES: runs of 8-token groups taken
// from the branches of several questions of the row block, laid one after the other (the host packs them per step);
// a row may look only at the columns of its own question's piece -- the IPPD mask, realised structurally.
//
// Warp roles (640 threads):
//   warp 0      producer: bulk async copies (TMA engine) of K and V into a 7-deep ring of 128-row buffers, mbarrier
//               completion; only the 8-token groups that hold valid tokens are fetched.
//   warp 1      P V issuer (one lane): O += P V with P read from TMEM (it overwrites the S buffer it came from) and V
//               from shared memory (MN-major).
//   warps 2..17 softmax (four warpgroups): thread (wg, row) handles S columns [32 wg, 32 wg + 32) of TMEM lane `row`:
//               TMEM -> registers, masked running max in the exp2 domain, lazy rescale of the O row in TMEM,
//               P (bf16) -> TMEM; they also stage Q~ (RoPE in fp32) into TMEM and run the epilogue
//               (normalise and store, or store the partial).
//   warp 18     S issuer (one lane): S = Q~ K~^T with Q~ read from TMEM and K from shared memory (K-major
//               core-matrix layout) into one of two S buffers in TMEM, once the P V product that read the buffer's
//               previous contents has completed.  Two issuers, because a tcgen05.mma holds its issuing thread about
//               as long as it executes: one thread for both made a late K tile delay the P V products and a late P
//               delay the S products.
//   warp 19     append (only when the call carries the step's raw K/V): walks the CTA's slice ahead of the producer and,
//               for every packed branch piece that holds the token fed at this step, rotates its key (RoPE) and writes
//               K~ and V into the piece's cache slot; the producer fetches a packed tile only after its slots are in
//               place.  A step's token belongs to exactly one piece of one (layer, KV head) sequence, so exactly one
//               CTA writes it and only that CTA reads it in this launch.
// Every wait is bounded; on expiry the error word is raised and all roles drain out.
#pragma once
#include "ippd_aux_kernels.cuh"
#include "ippd_device.cuh"

#define IPPD_TC_THREADS 640
#define IPPD_TC_WARP_S_ISSUER 18
#define IPPD_TC_WARP_APPEND 19
#define IPPD_TC_NBUF 7
#define IPPD_TC_ROWS 128
#define IPPD_TC_MERGE_SPLIT 8  // merge blocks per cut key sequence
#define IPPD_TC_MAX_CTAS 192   // upper bound of the persistent grid (one CTA per SM)
#define IPPD_TC_RESCALE_THRESHOLD 8.0f  // log2 units: the reference maximum may lag by up to 2^8

// Sizes that depend on the cache's element type.  KV8: keys and values are e4m3 bytes (half the bytes per token, so
// almost twice as many buffers of half the size); the products then run on the 8-bit tensor-core kind, with the query
// rows and the probabilities each split into two e4m3 terms (value = hi + lo) so that they keep bf16-like precision.
template <int D, bool KV8>
struct TcCfg {
  static constexpr int GB = (KV8 ? D / 16 : D / 8) * 128;  // bytes of an 8-token group (one row of core matrices)
  static constexpr int TILE_BYTES = 16 * GB;               // 128 tokens
  static constexpr int NBUF = KV8 ? 13 : IPPD_TC_NBUF;
  static constexpr int NMETA = KV8 ? 8 : 5;
  static constexpr int PV_TOKENS = KV8 ? 32 : 16;          // tokens one P V product consumes
};

struct IppdTcArgs {
  const int32_t* rb_tile_begin;  // [n_rb+1] first tile of each row block inside one (layer, head) sequence
  const IppdTcTile* tiles;       // [T1] tiles of one (layer, head) sequence
  const IppdTcPiece* pieces;     // pieces of the packed branch tiles
  int total_tiles;               // T1 * Hkv * layer_count
  int n_cta;                     // CTAs of the launch
  // CTA c owns tiles [cut[c], cut[c+1]) of the launch's tile sequence.  The host cuts it into equal parts and moves a
  // cut to the nearest boundary between two row blocks' key sequences when that is close: a sequence that is not cut
  // needs no partial and no merge.
  int32_t cut[IPPD_TC_MAX_CTAS + 1];
  int T1;                        // tiles of one (layer, head) sequence
  int layer_begin, layer_count;
  int out_f32;
  // raw K and V of the step's tokens, [layer_count, A, Hkv, D] (pre-RoPE), when the call appends them itself; else NULL
  const __nv_bfloat16* k_step;
  const __nv_bfloat16* v_step;
};

// ---- tcgen05 wrappers ----
// No-swizzle shared-memory matrix descriptor, split in two words: lo = address and leading byte offset,
// hi = stride byte offset and the descriptor version (all in 16-byte units).
__device__ __forceinline__ uint32_t tc_desc_lo(uint32_t addr, uint32_t lbo_bytes) {
  return ((addr >> 4) & 0x3FFF) | (((lbo_bytes >> 4) & 0x3FFF) << 16);
}
__device__ __forceinline__ uint32_t tc_desc_hi(uint32_t sbo_bytes) { return ((sbo_bytes >> 4) & 0x3FFF) | (1u << 14); }
__device__ __forceinline__ uint32_t tc_idesc(int M, int N, int b_mn_major) {
  // fp32 accumulate, bf16 x bf16, A K-major, B K- or MN-major
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                          uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\tsetp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                          uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc)
      : "memory");
}
// The 8-bit kind: fp32 accumulate, e4m3 x e4m3 (format code 0), A K-major in TMEM (four values per 32-bit column),
// B K- or MN-major in shared memory.
__device__ __forceinline__ uint32_t tc_idesc8(int M, int N, int b_mn_major) {
  return (1u << 4) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma_ts8(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                           uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

#define TC_LD32(taddr, r)                                                                                          \
  asm volatile(                                                                                                    \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                                    \
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28," \
      "%29,%30,%31}, [%32];"                                                                                       \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), \
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),     \
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),    \
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])                  \
      : "r"(taddr)                                                                                                 \
      : "memory")
#define TC_ST32(taddr, r)                                                                                          \
  asm volatile(                                                                                                    \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                                                             \
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28," \
      "%29,%30,%31};" ::"r"(r[0]),                                                                                 \
      "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),           \
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),  \
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),  \
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)                                                   \
      : "memory")

#define TC_ST16(taddr, r)                                                                                     \
  asm volatile(                                                                                               \
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};" \
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),     \
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(taddr)           \
      : "memory")

#define TC_LD16(taddr, r)                                                                                        \
  asm volatile(                                                                                                  \
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"     \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),         \
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])     \
      : "r"(taddr)                                                                                               \
      : "memory")
#define TC_ST2(taddr, r) \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%2], {%0,%1};" ::"r"(r[0]), "r"(r[1]), "r"(taddr) : "memory")
#define TC_ST4(taddr, r)                                                                                       \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%4], {%0,%1,%2,%3};" ::"r"(r[0]), "r"(r[1]), "r"(r[2]), \
               "r"(r[3]), "r"(taddr)                                                                            \
               : "memory")
#define TC_ST8(taddr, r)                                                                             \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};" ::"r"(r[0]), \
               "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(taddr) \
               : "memory")

// One split-KV segment: tiles [t_begin, t_end) (indices into IppdTcArgs::tiles) of row block `rb`, layer ll, KV head.
struct TcSegment {
  int rb, ll, head, t_begin, t_end;
  bool complete;  // covers the whole key sequence of the row block: write the final output
  int slot;       // else: partial slot of this CTA (0 = its first segment, 1 = a later one)
};

// Walks the CTA's slice of the global tile sequence.  All roles call it with the same arguments.
__device__ __forceinline__ bool tc_next_segment(const IppdTcArgs& a, const IppdStepDev& S, int Hkv, long long g0,
                                                long long g1, long long& g, TcSegment& sg) {
  if (g >= g1) return false;
  long long seq = g / a.T1;
  int within = (int)(g - seq * a.T1);
  int lo = 0, hi = S.n_rb - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (a.rb_tile_begin[mid] <= within) lo = mid; else hi = mid - 1;
  }
  sg.rb = lo;
  sg.ll = (int)(seq / Hkv);
  sg.head = (int)(seq % Hkv);
  const int rb0 = a.rb_tile_begin[lo], rb1 = a.rb_tile_begin[lo + 1];
  sg.t_begin = within;
  long long room = g1 - g;
  sg.t_end = (int)min((long long)rb1, (long long)within + room);
  sg.complete = sg.t_begin == rb0 && sg.t_end == rb1;
  sg.slot = (g == g0) ? 0 : 1;
  g += sg.t_end - sg.t_begin;
  return true;
}

#define IPPD_TC_NMETA 5  // (bf16 cache; the 8-bit variant has its own count in TcCfg)
// Per-tile description staged in shared memory by the producer warp.  The producer starts tile t + 5 only after the
// P V product of tile t has released its V buffer (7 ring buffers, two per tile), and every reader of tile t's entry
// is done by then, so five entries suffice.  For a packed branch tile, [c0[a], c1[a]) are the columns question `a` of
// the row block owns in it (the union of its adjacent pieces; empty when it has none).
struct TcMeta {
  int32_t rows;
  int32_t n_pieces;
  uint8_t c0[64], c1[64];
};

template <int NBUF, int NMETA>
struct TcSharedT {
  static constexpr int kNMeta = NMETA;
  uint64_t kv_full[NBUF], kv_empty[NBUF];
  uint64_t s_full[2], p_full[2];
  uint64_t pv_done[2];
  uint64_t o_free, q_full;
  uint64_t drain[2];     // completion of each issuer's MMAs in flight when it stops
  uint32_t tmem_base;
  volatile int abort_flag;
  uint32_t app_done;     // the append warp has finished the packed tiles with index (in the CTA's slice) below this
  unsigned short xmax[2][4][IPPD_TC_ROWS];  // [tile parity][warpgroup][row]: bf16 bits of the quarter-row maxima
  TcMeta meta[NMETA];
};
using TcShared = TcSharedT<IPPD_TC_NBUF, IPPD_TC_NMETA>;

template <int D, bool KV8 = false>
constexpr int tc_smem_bytes() {
  using C = TcCfg<D, KV8>;
  return C::NBUF * C::TILE_BYTES + (int)sizeof(TcSharedT<C::NBUF, C::NMETA>);
}


// Bounded wait that also gives up when another role has raised the abort flag.  (SH: the kernel's shared block.)
template <class SH>
__device__ __forceinline__ bool tc_wait(uint64_t* bar, uint32_t parity, const IppdDev& L, SH* sh) {
  if (mbar_try_wait(bar, parity)) return true;
  if (L.wait_limit_ns == 0) {  // "never wait": a phase still incomplete after one (briefly suspending) probe fails
    sh->abort_flag = 1;
    atomicOr(L.error_word, IPPD_ERRBIT_TIMEOUT);
    return false;
  }
  unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 127u) == 0) {
      if (sh->abort_flag) return false;
      if (globaltimer_ns() - t0 > (unsigned long long)L.wait_limit_ns) {
        sh->abort_flag = 1;
        atomicOr(L.error_word, IPPD_ERRBIT_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Bounded wait until the append warp's progress counter has passed `need`.
template <class SH>
__device__ __forceinline__ bool tc_wait_appended(const uint32_t* counter, uint32_t need, const IppdDev& L, SH* sh) {
  auto load = [&]() {
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(counter)) : "memory");
    return v;
  };
  if (load() >= need) return true;
  unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (load() < need) {
    if ((++spins & 63u) == 0) {
      if (sh->abort_flag) return false;
      if (globaltimer_ns() - t0 > (unsigned long long)L.wait_limit_ns) {
        sh->abort_flag = 1;
        atomicOr(L.error_word, IPPD_ERRBIT_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Producer role (one warp): walks the CTA's slice of the tile sequence and keeps the ring of NBUF 128-row buffers
// full.  Lane 0 owns the barriers and the context copies, lane i < n_pieces fetches piece i of a packed tile; the
// tile's description is left in shared memory for the other roles (published by the K buffer's mbarrier, which this
// warp arrives on afterwards).  SH needs kv_full[], kv_empty[], meta[], app_done and abort_flag.
template <int D, int NBUF, class SH, bool KV8 = false>
__device__ __forceinline__ void tc_producer_role(const IppdDev& L, const IppdStepDev& S, const IppdTcArgs& A, SH* sh,
                                                 uint8_t* ring, long long g0, long long g1, int lane) {
  constexpr int GB = TcCfg<D, KV8>::GB;
  constexpr int TILE_BYTES = 16 * GB;
  constexpr int PVG = TcCfg<D, KV8>::PV_TOKENS / 8;  // 8-token groups one P V product consumes
  const int Hkv = L.Hkv;
  long long g = g0;
  TcSegment sg;
  uint32_t n = 0;   // buffers filled so far
  uint32_t tc = 0;  // tiles issued so far
  bool ok = true;
  while (ok && tc_next_segment(A, S, Hkv, g0, g1, g, sg)) {
    const int layer = A.layer_begin + sg.ll;
    const int seg_act_begin = S.rbs[sg.rb].act_begin, seg_n_act = S.rbs[sg.rb].n_act;
    // the description of tile t + 1 (and its pieces) is fetched while tile t is being issued: two dependent loads
    // from global memory that would otherwise sit between the copies of consecutive tiles
    IppdTcTile ti = A.tiles[sg.t_begin];
    IppdTcPiece pc;
    pc.n_groups = 0;
    if (lane < ti.n_pieces) pc = A.pieces[ti.piece_begin + lane];
    for (int t = sg.t_begin; t < sg.t_end && ok; ++t, ++tc) {
      IppdTcTile ti_next = ti;
      IppdTcPiece pc_next;
      pc_next.n_groups = 0;
      if (t + 1 < sg.t_end) {
        ti_next = A.tiles[t + 1];
        if (lane < ti_next.n_pieces) pc_next = A.pieces[ti_next.piece_begin + lane];
      }
      TcMeta& mt = sh->meta[tc % SH::kNMeta];
      if (lane == 0) { mt.rows = ti.rows; mt.n_pieces = ti.n_pieces; }
      if (ti.n_pieces > 0) {
        // column window of every question in this tile: its pieces sit on adjacent lanes, the first gives c0 and
        // the last c1 (only the last piece of a question can be partly valid)
        reinterpret_cast<uint32_t*>(mt.c0)[lane & 15] = 0u;  // 64 + 64 bytes: lanes 0..15 clear c0, 16..31 clear c1
        if (lane >= 16) reinterpret_cast<uint32_t*>(mt.c1)[lane & 15] = 0u;
        __syncwarp();
        const int a_me = lane < ti.n_pieces ? pc.a_local : -1;
        const int a_prev = __shfl_up_sync(0xffffffffu, a_me, 1), a_next = __shfl_down_sync(0xffffffffu, a_me, 1);
        if (lane < ti.n_pieces) {
          if (lane == 0 || a_prev != a_me) mt.c0[a_me] = (uint8_t)pc.row0;
          if (lane == ti.n_pieces - 1 || a_next != a_me) mt.c1[a_me] = (uint8_t)(pc.row0 + pc.valid);
        }
      } else if (ti.n_pieces < 0) {
        // causal context tile (prefill): query a of the row block sits at virtual position pos_a and sees the
        // tile's tokens up to itself, columns [0, pos_a + 1 - first position of the tile)
        for (int a = lane; a < 64; a += 32) {
          int c1 = 0;
          if (a < seg_n_act) c1 = max(0, min(ti.rows, S.act_pos[seg_act_begin + a] + 1 - ti.piece_begin));
          mt.c0[a] = 0;
          mt.c1[a] = (uint8_t)c1;
        }
      }
      __syncwarp();
      const int groups = (ti.rows + 7) >> 3;
      if (A.k_step != nullptr && ti.n_pieces > 0) {
        // the step's own tokens are written by the append warp of this CTA: fetch the tile after them
        if (lane == 0) ok = tc_wait_appended(&sh->app_done, tc + 1, L, sh);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
      }
      for (int kv = 0; kv < 2 && ok; ++kv, ++n) {
        uint32_t buf = n % NBUF, ph = (n / NBUF) & 1;
        if (lane == 0) ok = tc_wait(&sh->kv_empty[buf], ph ^ 1, L, sh);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        uint8_t* dst = ring + buf * TILE_BYTES;
        if (kv == 1 && (groups % PVG) != 0) {
          // The P V product works in steps of 16 (8-bit cache: 32) rows: the rows between the fetched groups and the
          // end of the last step are not written by the copies below and would be stale shared memory; P is zero
          // there, but 0 * NaN = NaN.
          uint4* z = reinterpret_cast<uint4*>(dst + groups * GB);
          const int n16 = (PVG - groups % PVG) * (GB / 16);
          for (int idx = lane; idx < n16; idx += 32) z[idx] = make_uint4(0, 0, 0, 0);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
        }
        if (lane == 0) mbar_arrive_expect_tx(&sh->kv_full[buf], (uint32_t)groups * GB);
        __syncwarp();
        if (ti.n_pieces <= 0) {
          if (lane == 0)
            bulk_g2s(dst, L.cache + ippd_tile_addr<KV8>(L, layer, sg.head, ti.pool_tile, kv), (uint32_t)groups * GB,
                     &sh->kv_full[buf]);
        } else if (lane < ti.n_pieces) {
          bulk_g2s(dst + (pc.row0 >> 3) * GB,
                   L.cache + ippd_tile_addr<KV8>(L, layer, sg.head, pc.src_tile, kv) + (size_t)pc.src_group * GB,
                   (uint32_t)pc.n_groups * GB, &sh->kv_full[buf]);
        }
      }
      ti = ti_next;
      pc = pc_next;
    }
  }
  if (lane == 0) {
    // copies already issued must land before the CTA's shared memory is released (they normally have: the MMA lane
    // consumed them; this matters when the other roles gave up early)
    uint32_t first = n > NBUF ? n - NBUF : 0;
    for (uint32_t i = first; i < n; ++i)
      mbar_wait_ns(&sh->kv_full[i % NBUF], (i / NBUF) & 1, L, IPPD_DRAIN_LIMIT_NS);
  }
}

// Append role (one warp, only when the call carries the step's raw K/V): walks the CTA's slice ahead of the producer
// and, for every packed branch piece that holds the token fed at this step, rotates its key (RoPE) and writes K~ and V
// into the piece's cache slot; the producer fetches a packed tile only after its slots are in place.
template <int D, class SH, bool KV8 = false>
__device__ __forceinline__ void tc_append_role(const IppdDev& L, const IppdStepDev& S, const IppdTcArgs& A, SH* sh,
                                               long long g0, long long g1, int lane) {
  const int Hkv = L.Hkv;
  if (A.k_step != nullptr) {
    constexpr int CP = D / 16;    // lanes per token: one per pair of 16-byte chunks (c, c + D/16)
    constexpr int TPP = 32 / CP;  // tokens per pass of the warp
    long long g = g0;
    TcSegment sg;
    uint32_t tc = 0;  // tiles of the slice passed so far (the producer counts the same way)
    bool stop = false;
    while (!stop && tc_next_segment(A, S, Hkv, g0, g1, g, sg)) {
      const IppdRowBlock rb = S.rbs[sg.rb];
      const int first_packed = A.rb_tile_begin[sg.rb] + rb.n_ctx_tiles;
      const int layer = A.layer_begin + sg.ll;
      for (int t = sg.t_begin; t < sg.t_end; ++t, ++tc) {
        if (t < first_packed) continue;  // context tiles hold no token of this step
        if (sh->abort_flag) { stop = true; break; }
        const IppdTcTile ti = A.tiles[t];
        IppdTcPiece pc;
        pc.new_tok = 0;
        if (lane < ti.n_pieces) pc = A.pieces[ti.piece_begin + lane];
        unsigned todo = __ballot_sync(0xffffffffu, pc.new_tok != 0);
        while (todo) {
          // lane group gi takes the gi-th piece still to do
          const int gi = lane / CP, c = lane % CP;
          unsigned m = todo;
          int src = 0;
          for (int i = 0; i <= gi && m; ++i) { src = __ffs(m) - 1; m &= m - 1; }
          const bool have = __popc(todo) > gi;
          const int a_local = __shfl_sync(0xffffffffu, pc.a_local, src);
          const int src_tile = __shfl_sync(0xffffffffu, pc.src_tile, src);
          const int src_group = __shfl_sync(0xffffffffu, pc.src_group, src);
          const int new_tok = __shfl_sync(0xffffffffu, pc.new_tok, src);
          if (have) {
            const int a = rb.act_begin + a_local;
            const size_t row = (((size_t)sg.ll * S.A + a) * Hkv + sg.head) * D + c * 8;
            ippd_rope_store_pair<D, KV8>(L, A.k_step + row, A.v_step + row, S.act_pos[a], c,
                                         ippd_tile_addr<KV8>(L, layer, sg.head, src_tile, 0),
                                         src_group * 8 + new_tok - 1);
          }
          for (int i = 0; i < TPP && todo; ++i) todo &= todo - 1;
        }
        // the stores above (generic proxy) are read by the producer's bulk copies (async proxy)
        asm volatile("fence.proxy.async;" ::: "memory");
        __syncwarp();
        if (lane == 0)
          asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(smem_u32(&sh->app_done)), "r"(tc + 1) : "memory");
      }
    }
    if (lane == 0)
      asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(smem_u32(&sh->app_done)), "r"(0xFFFFFFFFu) : "memory");
  }
}

#include "ippd_attn_tc_softmax.cuh"

template <int D, bool KV8 = false>
__global__ void __launch_bounds__(IPPD_TC_THREADS, 1)
ippd_attn_tc_kernel(IppdDev L, IppdStepDev S, IppdTcArgs A, const __nv_bfloat16* __restrict__ q_raw,
                    void* __restrict__ out, float* __restrict__ part_o, float* __restrict__ part_ml) {
  using Cfg = TcCfg<D, KV8>;
  using SH = TcSharedT<Cfg::NBUF, Cfg::NMETA>;
  constexpr int NBUF = Cfg::NBUF;
  constexpr int GB = Cfg::GB;                  // bytes of an 8-row group
  constexpr int TILE_BYTES = Cfg::TILE_BYTES;  // 128 rows
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* ring = smem_raw;  // NBUF buffers of 128 rows
  SH* sh = reinterpret_cast<SH*>(ring + NBUF * TILE_BYTES);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Hkv = L.Hkv;
  pdl_trigger();  // the merge kernel may be scheduled as soon as SMs become free
  const long long g0 = A.cut[blockIdx.x], g1 = A.cut[blockIdx.x + 1];

  if (tid == 0) {
    for (int i = 0; i < NBUF; ++i) { mbar_init(&sh->kv_full[i], 1); mbar_init(&sh->kv_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh->s_full[i], 1); mbar_init(&sh->p_full[i], 16); }
    for (int i = 0; i < 2; ++i) mbar_init(&sh->pv_done[i], 1);
    mbar_init(&sh->drain[0], 1);
    mbar_init(&sh->drain[1], 1);
    mbar_init(&sh->o_free, 16);
    mbar_init(&sh->q_full, 16);
    sh->abort_flag = 0;
    sh->app_done = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sh->tmem_base))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // the set-up above overlaps the tail of the kernel before this one in the stream; global memory only from here on
  pdl_wait();
  // TMEM columns: S buffers at +0 / +128 (the bf16 P row of a tile overwrites the first 64 columns of its S buffer),
  // O at +256, two Q~ buffers (bf16 pairs, the A operand of S = Q~ K^T; segment n uses buffer n & 1) at +384 / +448.
  const uint32_t tmem = sh->tmem_base;
  const uint32_t tS0 = tmem, tO = tmem + 256, tQ = tmem + 384;

  if (warp == 0) {
    tc_producer_role<D, NBUF, SH, KV8>(L, S, A, sh, ring, g0, g1, lane);
  } else if (warp == 1) {
    // =========================== P V issuer (one lane) ===========================
    // O += P(j) V(j): P from TMEM (the head of S buffer j & 1), V from ring slot 2j+1 (MN-major).
    if (lane == 0) {
      const uint32_t ring_lo_v = tc_desc_lo(smem_u32(ring), GB);  // d chunks 128 B apart, 8-token groups GB apart
      const uint32_t hi_v = tc_desc_hi(128);
      const uint32_t idesc_pv = KV8 ? tc_idesc8(128, D, 1) : tc_idesc(128, D, 1);
      long long g = g0;
      TcSegment sg;
      uint32_t jt = 0;  // tiles processed so far by this CTA
      uint32_t nseg = 0;
      bool ok = true;
      while (ok && tc_next_segment(A, S, Hkv, g0, g1, g, sg)) {
        const int nt = sg.t_end - sg.t_begin;
        for (int i = 0; i < nt; ++i, ++jt) {
          const uint32_t nb = 2 * jt + 1, buf = nb % NBUF, ph = (nb / NBUF) & 1;
          if (!tc_wait(&sh->kv_full[buf], ph, L, sh)) { ok = false; break; }
          if (!tc_wait(&sh->p_full[jt & 1], (jt >> 1) & 1, L, sh)) { ok = false; break; }
          if (i == 0 && nseg > 0) {
            // the epilogue of the previous segment has read O
            if (!tc_wait(&sh->o_free, (nseg - 1) & 1, L, sh)) { ok = false; break; }
          }
          tc_fence_after();
          const uint32_t v_lo = ring_lo_v + buf * (TILE_BYTES >> 4);
          const uint32_t a_tmem = tS0 + (jt & 1) * 128;
          if constexpr (KV8) {
            // P = P_hi + P_lo, two e4m3 rows (columns +0 and +32 of the S buffer, four tokens per column), each
            // against the same V tile, 32 tokens per product
            // (unrolled: the products' operands are then constants of the instruction stream, which shortens the time
            // the thread spends per product; on the bf16 path the same change made no difference)
            const int ksteps = (sh->meta[jt % SH::kNMeta].rows + 31) >> 5;
#pragma unroll
            for (int half = 0; half < 2; ++half)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                if (k < ksteps)
                  tc_mma_ts8(tO, a_tmem + half * 32 + k * 8, v_lo + k * (4 * GB >> 4), hi_v, idesc_pv,
                             (i > 0 || half > 0 || k > 0) ? 1u : 0u);
          } else {
            const int ksteps = (sh->meta[jt % SH::kNMeta].rows + 15) >> 4;
            for (int k = 0; k < ksteps; ++k)
              tc_mma_ts(tO, a_tmem + k * 8, v_lo + k * (2 * GB >> 4), hi_v, idesc_pv, (i > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit(&sh->kv_empty[buf]);
          tc_commit(&sh->pv_done[jt & 1]);
        }
        ++nseg;
      }
      // tensor-core operations already issued must finish before TMEM is released (they normally have)
      tc_commit(&sh->drain[0]);
      mbar_wait_ns(&sh->drain[0], 0, L, IPPD_DRAIN_LIMIT_NS);
    }
  } else if (warp == IPPD_TC_WARP_APPEND) {
    tc_append_role<D, SH, KV8>(L, S, A, sh, g0, g1, lane);
  } else if (warp == IPPD_TC_WARP_S_ISSUER) {
    // =========================== S issuer (one lane) ===========================
    // S(j) = Q~ K(j)^T: Q~ from TMEM, K from ring slot 2j (K-major), into S buffer j & 1.  That buffer held P(j-2),
    // so PV(j-2) must have completed (pv_done): the two issuers' operations are not ordered by the tensor pipe.
    // A separate issuer, because a tcgen05.mma holds the issuing thread about as long as it executes and this
    // thread's waits (for K tiles) must not delay the P V products, nor theirs (for P) the S products.
    if (lane == 0) {
      const uint32_t ring_lo = tc_desc_lo(smem_u32(ring), 128);  // d chunks 128 B apart, 8-token groups GB apart
      const uint32_t hi_k = tc_desc_hi(GB);
      long long g = g0;
      TcSegment sg;
      uint32_t jt = 0;
      uint32_t nseg = 0;
      bool ok = true;
      while (ok && tc_next_segment(A, S, Hkv, g0, g1, g, sg)) {
        const int nt = sg.t_end - sg.t_begin;
        if (nseg == 0 && L.wait_limit_ns == 0 && !mbar_test_wait(&sh->q_full, 0)) {
          // "never wait", taken literally at the kernel's first wait (a non-suspending probe of a phase that cannot be
          // complete yet), so that a zero limit reports IPPD_ERRBIT_TIMEOUT whatever the probe's suspend time is
          sh->abort_flag = 1;
          atomicOr(L.error_word, IPPD_ERRBIT_TIMEOUT);
          break;
        }
        if (!tc_wait(&sh->q_full, nseg & 1, L, sh)) break;
        const uint32_t a_tmem = tQ + (nseg & 1) * 64;
        for (int i = 0; i < nt; ++i, ++jt) {
          const uint32_t nb = 2 * jt, buf = nb % NBUF, ph = (nb / NBUF) & 1;
          if (!tc_wait(&sh->kv_full[buf], ph, L, sh)) { ok = false; break; }
          if (jt >= 2 && !tc_wait(&sh->pv_done[jt & 1], ((jt - 2) >> 1) & 1, L, sh)) { ok = false; break; }
          tc_fence_after();
          const int rows_i = sh->meta[jt % SH::kNMeta].rows;  // published by the K buffer's barrier
          const uint32_t k_lo = ring_lo + buf * (TILE_BYTES >> 4);
          const uint32_t d_tmem = tS0 + (jt & 1) * 128;
          if constexpr (KV8) {
            // Q~ = Q~_hi + Q~_lo, two e4m3 rows (columns +0 and +D/4 of the Q~ buffer), each against the same K tile,
            // 32 values of d per product
            const uint32_t idesc = tc_idesc8(128, (rows_i + 15) & ~15, 0);
#pragma unroll
            for (int half = 0; half < 2; ++half)
#pragma unroll
              for (int k = 0; k < D / 32; ++k)
                tc_mma_ts8(d_tmem, a_tmem + half * (D / 4) + k * 8, k_lo + k * 16, hi_k, idesc, (half > 0 || k > 0));
          } else {
            const uint32_t idesc = tc_idesc(128, (rows_i + 15) & ~15, 0);
#pragma unroll
            for (int k = 0; k < D / 16; ++k) tc_mma_ts(d_tmem, a_tmem + k * 8, k_lo + k * 16, hi_k, idesc, k > 0);
          }
          tc_commit(&sh->kv_empty[buf]);
          tc_commit(&sh->s_full[jt & 1]);
        }
        ++nseg;
      }
      tc_commit(&sh->drain[1]);
      mbar_wait_ns(&sh->drain[1], 0, L, IPPD_DRAIN_LIMIT_NS);
    }
  } else {
    // =========================== softmax / correction / epilogue (warps 2..17) ===========================
    tc_softmax_role<D, SH, KV8>(L, S, A, sh, tmem, g0, g1, q_raw, out, part_o, part_ml);
  }

  // ---- teardown: every role gets here (all waits are bounded) ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// Log-sum-exp merge for the persistent kernel: a row block whose key sequence was cut across CTAs has one partial
// per CTA that touched it (slot 0 if the piece is that CTA's first segment, else slot 1).  Blocks [c * SPLIT,
// (c + 1) * SPLIT) look at interior cut c + 1: if it falls strictly inside a key sequence and is the first cut to do so,
// they merge that sequence's partials; otherwise they have nothing to do.
template <int D>
__global__ void __launch_bounds__(128)
ippd_merge_tc_kernel(IppdDev L, IppdStepDev S, IppdTcArgs A, const float* __restrict__ part_o,
                     const float* __restrict__ part_ml, void* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  const int ci = blockIdx.x / IPPD_TC_MERGE_SPLIT + 1, part = blockIdx.x % IPPD_TC_MERGE_SPLIT;
  const int x = A.cut[ci];
  const int seq = x / A.T1, within = x - seq * A.T1;
  int rbi = 0;
  {
    int lo = 0, hi = S.n_rb - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (A.rb_tile_begin[mid] <= within) lo = mid; else hi = mid - 1;
    }
    rbi = lo;
  }
  const int a0 = seq * A.T1 + A.rb_tile_begin[rbi];
  if (x == a0) return;              // the cut sits between two key sequences
  if (A.cut[ci - 1] > a0) return;   // an earlier cut lies inside the same sequence: its blocks do the merge
  const IppdRowBlock rb = S.rbs[rbi];
  const int ll = seq / L.Hkv, head = seq - ll * L.Hkv, G = L.G;
  const int b0 = a0 + rb.n_tiles;
  const int c0 = ci - 1;  // the CTA that holds the sequence's first tiles
  int c1 = ci;            // ... and the one that holds its last tile
  while (c1 + 1 < A.n_cta && A.cut[c1 + 1] < b0) ++c1;
  const int nrows = rb.n_act * G;
  for (int item = part * blockDim.x + threadIdx.x; item < nrows * (D / 4); item += blockDim.x * IPPD_TC_MERGE_SPLIT) {
    int r = item / (D / 4), cc = item - r * (D / 4);
    // one pass over the partials with a running reference maximum (the loads of the next partial do not depend on
    // the arithmetic of this one)
    float M = -INFINITY, lsum = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
    for (int c = c0; c <= c1; ++c) {
      const size_t slot = (size_t)c * 2 + ((A.cut[c] >= a0) ? 0 : 1);
      const float2 ml = *reinterpret_cast<const float2*>(part_ml + (slot * IPPD_TC_ROWS + r) * 2);
      const float4 v = *reinterpret_cast<const float4*>(part_o + (slot * IPPD_TC_ROWS + r) * D + cc * 4);
      if (ml.x == -INFINITY) continue;  // this part of the key sequence held nothing the row may see
      const float mn = fmaxf(M, ml.x);
      const float so = fast_exp2(M - mn), w = fast_exp2(ml.x - mn);  // so = 0 on the first contributing partial
      lsum = lsum * so + w * ml.y;
      acc.x = acc.x * so + w * v.x; acc.y = acc.y * so + w * v.y;
      acc.z = acc.z * so + w * v.z; acc.w = acc.w * so + w * v.w;
      M = mn;
    }
    float inv = 1.f / lsum;
    int a = r / G, j = r - a * G;
    size_t base = (((size_t)ll * S.A + rb.act_begin + a) * L.Hq + head * G + j) * D + cc * 4;
    if (A.out_f32) {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + base) =
          make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    } else {
      uint2 pk;
      pk.x = pack_bf16(acc.x * inv, acc.y * inv);
      pk.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + base) = pk;
    }
  }
}
