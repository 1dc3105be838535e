// Shared device-side types of libbild (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bild.h"

namespace bild {

constexpr int MAXB = BILD_MAX_BLOCK;  // largest block of tokens one decoder pass takes

// What one decoder pass works on.  Written on the device by the policy code (or by a
// tiny set-up kernel for the single-step entry points), read by every kernel of the
// pass, so that a captured launch sequence can be replayed with new values.
constexpr int SUB_CHUNK = 8;   // rows of a chunk when a block of 9 to 16 rows runs on the fused sub-layer kernels

struct CallDesc {
  int k;              // rows in this pass (1 for a small-model step)
  int pos0;           // position of row 0 = number of rows already in the self cache
  int run_policy;     // 1: the LM head's last block also advances the decode loop
  int pad;
  int tokens[MAXB];   // input token of each row
  int targets[MAXB];  // token judged by row i (the next input token), -1 = none
};

// Per-row results of the fused LM head and the policy tests derived from them.
struct HeadOut {
  int argmax[MAXB];
  float zmax[MAXB];
  float lse[MAXB];
  float gather[MAXB];  // logit of targets[i]
  float d[MAXB];       // lse - gather = -ln p(target)   (rollback distance)
  float pmax;          // row 0: 1 / sum exp(z - zmax)   (fallback confidence)
  int fallback;        // pmax < alpha_fb
  int first_violation; // smallest i < k-1 with d[i] > alpha_rb, else -1
  int next_token;
};

// Decode-loop state (Algorithm 1) kept on the device.
struct DevState {
  int n;        // index of the last token of y
  int S_len;    // rows in the small model's self cache
  int L_len;    // rows in the large model's self cache
  int drafts;   // small-model tokens written since the last large pass
  int fallback; // the step just taken asks for a large pass
  int done;
  int mode;
  int err;
  int max_len, max_draft, eos_id, start_id;
  float alpha_fb, alpha_rb;
  int n_trace, trace_cap;
  bild_stats stats;
  int passes;   // decoder passes taken by the running loop (guards against a runaway loop)
  int pad0;
  float top_p;  // > 0: the sampling variant, tokens are drawn from the nucleus of this mass
  int pad1;
  long long cum_draws;       // token-drawing kernels run from the loop graphs since create
  long long cum_passes[4];   // passes run from the loop graphs since create: small, large block, large single row, large up to 8 rows
};

struct Partial {  // running soft-max statistics of a slice of the vocabulary
  float m;        // max logit
  float s;        // sum exp(z - m)
  int idx;        // arg max (lowest index on ties)
};

__device__ __forceinline__ Partial combine(Partial a, Partial b) {
  // fixed tie rule: the lower index wins among equal maxima
  Partial r;
  if (b.m > a.m || (b.m == a.m && b.idx < a.idx)) { Partial t = a; a = b; b = t; }
  r.m = a.m;
  r.idx = a.idx;
  r.s = a.s + (b.s == 0.f ? 0.f : b.s * expf(b.m - a.m));
  return r;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// 8 consecutive weights as fp32, one 128-bit (bf16) or two 128-bit (fp32) streaming loads.
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&w)[8]) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  w[0] = __uint_as_float(v.x << 16); w[1] = __uint_as_float(v.x & 0xffff0000u);
  w[2] = __uint_as_float(v.y << 16); w[3] = __uint_as_float(v.y & 0xffff0000u);
  w[4] = __uint_as_float(v.z << 16); w[5] = __uint_as_float(v.z & 0xffff0000u);
  w[6] = __uint_as_float(v.w << 16); w[7] = __uint_as_float(v.w & 0xffff0000u);
}
__device__ __forceinline__ void load8(const float* p, float (&w)[8]) {
  float4 a, b;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w) : "l"(p));
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w) : "l"(p + 4));
  w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
  w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
}

// Programmatic dependent launch: let the next kernel in the stream start its prologue,
// and wait until everything the previous kernel wrote is visible.  Both are no-ops in a
// kernel that was launched without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- thread-block clusters: rank, barrier, stores into a peer's shared memory ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f4(uint32_t local_addr, uint32_t rank, float4 v) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(remote), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void st_cluster_f1(uint32_t local_addr, uint32_t rank, float v) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// ---- mbarrier, bulk (TMA) copies, bounded polling ------------------------------------------
constexpr unsigned SPIN_LIMIT = 1u << 20;   // polls of a barrier before a kernel gives up and reports BILD_ERR_TIMEOUT
constexpr int MAX_GRID_SM = 256;            // per-block record areas are sized for this many blocks (one per SM)

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// global -> shared bulk copy (16-byte aligned addresses, size a multiple of 16) that reports to an mbarrier
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// barrier of the first 256 threads of a block (the computing warps of kernels with a copy-issuing extra warp)
__device__ __forceinline__ void csync256() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// ---- sum of NP register values across the warp, one shuffle per halving ------------------
// Returns in every lane the warp-wide sum of v[lane >> (5 - log2 NP)].
template <int NP>
__device__ __forceinline__ float treduce(float (&v)[NP], int lane) {
  int s = 16;
#pragma unroll
  for (int n = NP; n > 1; n >>= 1) {
    const bool up = (lane & s) != 0;
#pragma unroll
    for (int j = 0; j < n / 2; ++j) {
      const float send = up ? v[j] : v[j + n / 2];
      const float keep = up ? v[j + n / 2] : v[j];
      v[j] = keep + __shfl_xor_sync(0xffffffffu, send, s);
    }
    s >>= 1;
  }
  float r = v[0];
  for (; s >= 1; s >>= 1) r += __shfl_xor_sync(0xffffffffu, r, s);
  return r;
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ float gelu_tanh(float u) {
  return 0.5f * u * (1.f + tanhf(0.7978845608028654f * (u + 0.044715f * u * u * u)));
}

}  // namespace bild
