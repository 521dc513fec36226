// Device-side primitives (inline PTX for sm_100a) and parameter structs of the IPPD kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ippd_internal.h"

#define IPPD_ERRBIT_TIMEOUT 1
#define IPPD_ERRBIT_RANGE 2
#define IPPD_ERRBIT_NONFINITE 4

// Everything a kernel needs to know about the cache and the ragged tables.
struct IppdDev {
  const int32_t* ctx_len;          // [B]
  const int32_t* ctx_tile_off;     // [B+1]
  const int32_t* q_len;            // [NQ]
  const int32_t* prompt_of;        // [NQ]
  const int32_t* branch_tile_off;  // [NQ+1]
  const int32_t* hdr_begin;        // [B+1] first header token of each prompt (the shared instruction comes first)
  const int32_t* q_hdr_begin;      // [NQ+1] first header token of each question
  const float2* rope;              // [max_pos+1][D/2] (cos, sin)
  char* cache;                     // [layer][kv head][tile][K|V][tile bytes]
  int32_t* error_word;
  long long n_tiles;
  long long wait_limit_ns;
  int n_layers, Hq, Hkv, G, D, max_pos;
  int shared_len;  // tokens of the instruction shared by all prompts (positions 0 .. shared_len-1, tiles from 0)
  int kv8;         // 1: the cache holds e4m3 bytes (IPPD_OPT_KV_DTYPE)
};

// Per-step arrays (device pointers into the step blob).
struct IppdStepDev {
  const int32_t* act_q;
  const int32_t* act_s;
  const int32_t* act_pos;  // virtual position of each active question's query at this step
  const IppdRowBlock* rbs;
  const IppdUnit* units;
  int A, n_rb, n_units, RB;
};

// Byte offset of the K (kv = 0) or V (kv = 1) half of a cache tile.  KV8: the cache holds e4m3 bytes, not bf16.
template <bool KV8 = false>
__device__ __forceinline__ size_t ippd_tile_addr(const IppdDev& L, int layer, int head, long long tile, int kv) {
  size_t tile_bytes = (size_t)IPPD_TILE_TOKENS * L.D * (KV8 ? 1 : 2);
  return ((((size_t)layer * L.Hkv + head) * (size_t)L.n_tiles + (size_t)tile) * 2 + kv) * tile_bytes;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// ---- programmatic dependent launch ----
// A kernel launched with the programmatic-serialisation attribute may be scheduled while the kernel before it in the
// stream still runs; pdl_wait() returns once that kernel has completed and its writes are visible (it returns at
// once after an ordinary launch).  pdl_trigger() lets the next kernel in the stream be scheduled from now on.  Every
// kernel launched with the attribute calls pdl_wait() before its first access to global memory.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- mbarrier ----
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking test of a phase.
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: returns false (and raises the device error word) when `limit_ns` runs out.
__device__ __forceinline__ bool mbar_wait_ns(uint64_t* bar, uint32_t parity, const IppdDev& L,
                                             unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  if (limit_ns == 0) {  // "never wait": a phase still incomplete after one (briefly suspending) probe fails
    atomicOr(L.error_word, IPPD_ERRBIT_TIMEOUT);
    return false;
  }
  unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (globaltimer_ns() - t0 > limit_ns) {
        atomicOr(L.error_word, IPPD_ERRBIT_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const IppdDev& L) {
  return mbar_wait_ns(bar, parity, L, (unsigned long long)L.wait_limit_ns);
}
// Waits that drain hardware work already in flight (bulk copies into shared memory, tensor-core operations on TMEM)
// before the resources are released get at least this long, whatever the configured limit of the other waits.
#define IPPD_DRAIN_LIMIT_NS 20000000ull

// ---- bulk async copy (TMA engine, untiled form): global -> shared, completes on an mbarrier ----
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// ---- warp-level matrix ops (legacy tensor path) ----
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                              uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Four floats -> four e4m3 bytes (round to nearest even, saturating at 448), a in the lowest byte.
__device__ __forceinline__ uint32_t pack_e4m3x4(float a, float b, float c, float d) {
  const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
  const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(c, d), __NV_SATFINITE, __NV_E4M3);
  return lo | (hi << 16);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
