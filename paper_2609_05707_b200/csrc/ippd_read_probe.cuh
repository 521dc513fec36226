// Read probe: streams the key/value tiles of the current step through the attention kernel's bulk-copy ring and does
// nothing with them.  Its time is the floor the attention kernel's memory side sets on its own: the same tile list,
// the same copies (cp.async.bulk into the same ring of buffers, one CTA per SM, the same slices), no tensor-core
// or softmax work.  A measuring aid; it reads the cache and writes nothing to global memory.
#pragma once
#include "ippd_attn_tc.cuh"

template <int D, bool KV8 = false>
__global__ void __launch_bounds__(64, 1)
ippd_read_probe_kernel(IppdDev L, IppdStepDev S, IppdTcArgs A) {
  constexpr int GB = TcCfg<D, KV8>::GB;
  constexpr int TILE_BYTES = 16 * GB;
  constexpr int NBUF = TcCfg<D, KV8>::NBUF;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* ring = smem_raw;
  uint64_t* full = reinterpret_cast<uint64_t*>(ring + NBUF * TILE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long g0 = A.cut[blockIdx.x], g1 = A.cut[blockIdx.x + 1];
  if (threadIdx.x == 0) {
    for (int i = 0; i < NBUF; ++i) mbar_init(&full[i], 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (warp != 0) return;
  // One warp is producer and consumer: it keeps NBUF copies in flight and waits for the oldest before reusing its
  // buffer.  Lane i fetches piece i of a packed tile, lane 0 the context tiles, as in the attention kernel.
  long long g = g0;
  TcSegment sg;
  uint32_t n = 0;
  bool ok = true;
  while (ok && tc_next_segment(A, S, L.Hkv, g0, g1, g, sg)) {
    const int layer = A.layer_begin + sg.ll;
    for (int t = sg.t_begin; t < sg.t_end && ok; ++t) {
      const IppdTcTile ti = A.tiles[t];
      IppdTcPiece pc;
      pc.n_groups = 0;
      if (lane < ti.n_pieces) pc = A.pieces[ti.piece_begin + lane];
      const int groups = (ti.rows + 7) >> 3;
      for (int kv = 0; kv < 2 && ok; ++kv, ++n) {
        const uint32_t buf = n % NBUF;
        if (n >= NBUF) {
          if (lane == 0) ok = mbar_wait(&full[buf], ((n / NBUF) - 1) & 1, L);
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) break;
        }
        uint8_t* dst = ring + buf * TILE_BYTES;
        if (lane == 0) mbar_arrive_expect_tx(&full[buf], (uint32_t)groups * GB);
        __syncwarp();
        if (ti.n_pieces <= 0) {
          if (lane == 0)
            bulk_g2s(dst, L.cache + ippd_tile_addr<KV8>(L, layer, sg.head, ti.pool_tile, kv), (uint32_t)groups * GB, &full[buf]);
        } else if (lane < ti.n_pieces) {
          bulk_g2s(dst + (pc.row0 >> 3) * GB,
                   L.cache + ippd_tile_addr<KV8>(L, layer, sg.head, pc.src_tile, kv) + (size_t)pc.src_group * GB,
                   (uint32_t)pc.n_groups * GB, &full[buf]);
        }
      }
    }
  }
  if (lane == 0) {
    // copies in flight must land before the CTA's shared memory is released
    const uint32_t first = n > NBUF ? n - NBUF : 0;
    for (uint32_t i = first; i < n; ++i) mbar_wait_ns(&full[i % NBUF], (i / NBUF) & 1, L, IPPD_DRAIN_LIMIT_NS);
  }
}
