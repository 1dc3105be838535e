// Self-attention of the encoder (set-up step) for d_kv = 64: softmax(Q K^T + bias) V per head over
// all encoder positions, bias by signed relative position.
// One block per (head, 64 query rows); a group of 4 warps (16 rows each) visits keys and values in tiles
// of 64 with a running soft-max (no score matrix in memory); G such groups share a block, group i taking the
// tiles i, i + G, ... with staging areas of its own, and their (maximum, sum, weighted values) are merged at the end.  Both products run on mma.sync
// m16n8k16 with every fp32 operand split into a bf16 head and a bf16 remainder and three products
// kept (head x head, head x remainder, remainder x head), i.e. ~16 mantissa bits per operand:
//   * the key tile is staged as [key][d] (the "col" operand of Q K^T), the value tile transposed as
//     [d][key] (the "col" operand of P V), both as head and remainder, rows padded against bank
//     conflicts;
//   * the next tile's keys and values are on their way (asynchronous 16-byte copies into a raw fp32 area) while the
//     current tile is multiplied; staging then converts from shared memory;
//   * the score fragment of a warp (16 rows x 64 keys) stays in registers, is turned into
//     probabilities and re-used as the left operand of P V (accumulator fragment of two 8-key
//     tiles = operand fragment of one 16-key step).
#pragma once
#include "decode_kernels.cuh"

namespace bild {

constexpr int EA_THREADS = 128;
constexpr int EA_ROWS = 64;    // query rows per block
constexpr int EA_KEYS = 64;    // keys per tile
constexpr int EA_D = 64;       // d_kv
constexpr int EA_PAD = 8;      // bf16 elements of padding per staged row
constexpr int EA_RVS = EA_D + 4;   // row stride (floats) of the raw value tile: two keys 2 rows apart fall into different banks

__device__ __forceinline__ uint32_t ea_pack(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ void ea_split(float a, float b, uint32_t& hi, uint32_t& lo) {
  hi = ea_pack(a, b);
  lo = ea_pack(a - __uint_as_float(hi << 16), b - __uint_as_float(hi & 0xffff0000u));
}
__device__ __forceinline__ void ea_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr size_t EA_GROUP_BYTES = (size_t)4 * EA_KEYS * (EA_D + EA_PAD) * 2 + (size_t)EA_KEYS * (EA_D + EA_RVS) * 4;   // one group's areas
constexpr int EA_MAX_GROUPS = 3;   // what fits the shared memory of an SM
inline size_t enc_attn_smem_bytes(int max_keys, int groups) {
  return groups * EA_GROUP_BYTES + (size_t)((max_keys + EA_ROWS + 3) & ~3) * 4;
}
inline int enc_attn_groups(int max_keys) { return std::max(1, std::min(EA_MAX_GROUPS, (max_keys + EA_KEYS - 1) / EA_KEYS)); }
__device__ __forceinline__ void ea_group_sync(int grp) { asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "n"(EA_THREADS) : "memory"); }

// q [E][ldq], kc / vc [H][cap][64], out [E][ldo]; bias [H][bias_ld] indexed by bias_off + key - query
// oh / ol != nullptr: the output is written as its bf16 head and remainder [E][H * 64] (what the
// output projection reads) instead of fp32
template <int G>
__global__ void __launch_bounds__(EA_THREADS * G) enc_attn_kernel(BAttnArgs a, __nv_bfloat16* oh, __nv_bfloat16* ol) {
  extern __shared__ __align__(16) unsigned char ea_smem[];
  constexpr int ST = EA_D + EA_PAD;   // staged row length (bf16 elements)
  const int grp = threadIdx.x / EA_THREADS;   // key group of this warp
  __nv_bfloat16* sKh = reinterpret_cast<__nv_bfloat16*>(ea_smem + grp * EA_GROUP_BYTES);   // [key][d]
  __nv_bfloat16* sKl = sKh + EA_KEYS * ST;
  __nv_bfloat16* sVh = sKl + EA_KEYS * ST;                          // [d][key]
  __nv_bfloat16* sVl = sVh + EA_D * ST;
  float* sRawK = reinterpret_cast<float*>(sVl + EA_D * ST);        // [key][64] fp32 as it lies in the cache
  float* sRawV = sRawK + EA_KEYS * EA_D;                            // [key][EA_RVS]
  float* sBias = reinterpret_cast<float*>(ea_smem + G * EA_GROUP_BYTES);   // [E + 63]: entry (key - query + r0 + 63)
  const int h = blockIdx.x, r0 = blockIdx.y * EA_ROWS;
  const int tid = threadIdx.x % EA_THREADS, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;   // (within the group)
  pdl_launch_dependents();
  pdl_wait();
  const int E = min(min(a.M, *a.n_keys_dev), a.cap);
  for (int i = threadIdx.x; i < E + EA_ROWS - 1; i += EA_THREADS * G) {
    // key - query for query r0 + 63 - ... : entry i stands for key - query = i - (r0 + 63)
    const int rel = i - (r0 + EA_ROWS - 1);
    const int idx = a.bias_off + rel;
    sBias[i] = (idx >= 0 && idx < a.bias_ld) ? __ldg(a.bias + (size_t)h * a.bias_ld + idx) : 0.f;
  }
  // this warp's queries as left-operand fragments (head and remainder), kept for the whole kernel
  const int row_a = min(r0 + warp * 16 + g, E - 1), row_b = min(r0 + warp * 16 + g + 8, E - 1);
  uint32_t qh[4][4], ql[4][4];
  {
    const float* qa = a.q + (size_t)row_a * a.ldq + h * EA_D;
    const float* qb = a.q + (size_t)row_b * a.ldq + h * EA_D;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      const float2 x0 = *reinterpret_cast<const float2*>(qa + ks * 16 + 2 * t);
      const float2 x1 = *reinterpret_cast<const float2*>(qb + ks * 16 + 2 * t);
      const float2 x2 = *reinterpret_cast<const float2*>(qa + ks * 16 + 8 + 2 * t);
      const float2 x3 = *reinterpret_cast<const float2*>(qb + ks * 16 + 8 + 2 * t);
      ea_split(x0.x, x0.y, qh[ks][0], ql[ks][0]);
      ea_split(x1.x, x1.y, qh[ks][1], ql[ks][1]);
      ea_split(x2.x, x2.y, qh[ks][2], ql[ks][2]);
      ea_split(x3.x, x3.y, qh[ks][3], ql[ks][3]);
    }
  }
  float o[8][4];   // 16 rows x 64 channels of weighted values (unnormalised)
#pragma unroll
  for (int dt = 0; dt < 8; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;
  float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;   // rows g and g + 8 of the warp
  const float* Kg = a.kc + (size_t)h * a.cap * EA_D;
  const float* Vg = a.vc + (size_t)h * a.cap * EA_D;
  const int qa_pos = r0 + warp * 16 + g, qb_pos = qa_pos + 8;
  auto fetch = [&](int k0) {   // the raw tile: 16-byte asynchronous copies, keys past the end repeat the last one
    for (int idx = tid; idx < EA_KEYS * (EA_D / 4); idx += EA_THREADS) {
      const int key = idx >> 4, c4 = (idx & 15) << 2;
      const int kg = min(k0 + key, E - 1);
      cp_async16(sRawK + key * EA_D + c4, Kg + (size_t)kg * EA_D + c4);
      cp_async16(sRawV + key * EA_RVS + c4, Vg + (size_t)kg * EA_D + c4);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  if (grp * EA_KEYS < E) fetch(grp * EA_KEYS);
  __syncthreads();   // the bias table is complete
#pragma unroll 1
  for (int k0 = grp * EA_KEYS; k0 < E; k0 += EA_KEYS * G) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    ea_group_sync(grp);   // the raw tile has arrived for the whole group; the previous tile is no longer read
    // stage the tile.  Keys: thread -> (key, 4 channels), rows written 8 bytes at a time.
    for (int idx = tid; idx < EA_KEYS * (EA_D / 4); idx += EA_THREADS) {
      const int key = idx >> 4, c4 = (idx & 15) << 2;
      const float4 kv = *reinterpret_cast<const float4*>(sRawK + key * EA_D + c4);
      uint32_t h0, l0, h1, l1;
      ea_split(kv.x, kv.y, h0, l0);
      ea_split(kv.z, kv.w, h1, l1);
      *reinterpret_cast<uint2*>(sKh + key * ST + c4) = make_uint2(h0, h1);
      *reinterpret_cast<uint2*>(sKl + key * ST + c4) = make_uint2(l0, l1);
    }
    // Values, transposed: thread -> (pair of keys, 4 channels) with the key pair varying fastest, so that a
    // warp writes 32 consecutive words of one transposed row
    for (int idx = tid; idx < (EA_KEYS / 2) * (EA_D / 4); idx += EA_THREADS) {
      const int kp = idx & 31, c4 = (idx >> 5) << 2;
      const float4 va = *reinterpret_cast<const float4*>(sRawV + (2 * kp) * EA_RVS + c4);
      const float4 vb = *reinterpret_cast<const float4*>(sRawV + (2 * kp + 1) * EA_RVS + c4);
      const float ea[4] = {va.x, va.y, va.z, va.w}, eb[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        uint32_t hv, lv;
        ea_split(ea[e], eb[e], hv, lv);
        *reinterpret_cast<uint32_t*>(sVh + (c4 + e) * ST + 2 * kp) = hv;
        *reinterpret_cast<uint32_t*>(sVl + (c4 + e) * ST + 2 * kp) = lv;
      }
    }
    ea_group_sync(grp);
    if (k0 + EA_KEYS * G < E) fetch(k0 + EA_KEYS * G);   // (the raw area is free again: everybody has converted its share)
    // scores of 16 rows x 64 keys
    // (consecutive instructions go to different accumulators, four key tiles side by side: an instruction that adds to the
    // accumulator of the one in front waits for its result)
    float s[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
#pragma unroll
      for (int n4 = 0; n4 < 8; n4 += 4) {
        uint32_t bh[4][2], bl[4][2];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const __nv_bfloat16* kh = sKh + ((n4 + i) * 8 + g) * ST + 2 * t + ks * 16;
          const __nv_bfloat16* kl = sKl + ((n4 + i) * 8 + g) * ST + 2 * t + ks * 16;
          bh[i][0] = *reinterpret_cast<const uint32_t*>(kh); bh[i][1] = *reinterpret_cast<const uint32_t*>(kh + 8);
          bl[i][0] = *reinterpret_cast<const uint32_t*>(kl); bl[i][1] = *reinterpret_cast<const uint32_t*>(kl + 8);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) ea_mma(s[n4 + i], qh[ks][0], qh[ks][1], qh[ks][2], qh[ks][3], bh[i][0], bh[i][1]);
#pragma unroll
        for (int i = 0; i < 4; ++i) ea_mma(s[n4 + i], qh[ks][0], qh[ks][1], qh[ks][2], qh[ks][3], bl[i][0], bl[i][1]);
#pragma unroll
        for (int i = 0; i < 4; ++i) ea_mma(s[n4 + i], ql[ks][0], ql[ks][1], ql[ks][2], ql[ks][3], bh[i][0], bh[i][1]);
      }
    // bias, mask of the keys past the end, tile maxima
    float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int key = k0 + nt * 8 + 2 * t + e;
        const bool ok = key < E;
        // entry (key - query + r0 + 63)
        s[nt][e] = ok ? s[nt][e] + sBias[key - qa_pos + r0 + EA_ROWS - 1] : -INFINITY;
        s[nt][2 + e] = ok ? s[nt][2 + e] + sBias[key - qb_pos + r0 + EA_ROWS - 1] : -INFINITY;
        mx_a = fmaxf(mx_a, s[nt][e]);
        mx_b = fmaxf(mx_b, s[nt][2 + e]);
      }
    }
    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1)); mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1)); mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
    const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
    const float sc_a = m_a == -INFINITY ? 0.f : __expf(m_a - mn_a), sc_b = m_b == -INFINITY ? 0.f : __expf(m_b - mn_b);
    m_a = mn_a; m_b = mn_b;
    float sum_a = 0.f, sum_b = 0.f;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float pa = s[nt][e] == -INFINITY ? 0.f : __expf(s[nt][e] - mn_a);
        const float pb = s[nt][2 + e] == -INFINITY ? 0.f : __expf(s[nt][2 + e] - mn_b);
        s[nt][e] = pa; s[nt][2 + e] = pb;
        sum_a += pa; sum_b += pb;
      }
    }
    l_a = l_a * sc_a + sum_a;   // (this thread's share of the row; the quad is added at the end)
    l_b = l_b * sc_b + sum_b;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) { o[dt][0] *= sc_a; o[dt][1] *= sc_a; o[dt][2] *= sc_b; o[dt][3] *= sc_b; }
    // weighted values: probabilities of two 8-key tiles are the operand of one 16-key step
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t ph[4], pl[4];
      ea_split(s[2 * j][0], s[2 * j][1], ph[0], pl[0]);
      ea_split(s[2 * j][2], s[2 * j][3], ph[1], pl[1]);
      ea_split(s[2 * j + 1][0], s[2 * j + 1][1], ph[2], pl[2]);
      ea_split(s[2 * j + 1][2], s[2 * j + 1][3], ph[3], pl[3]);
#pragma unroll
      for (int d4 = 0; d4 < 8; d4 += 4) {   // four channel tiles side by side, as above
        uint32_t bh[4][2], bl[4][2];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const __nv_bfloat16* vh = sVh + ((d4 + i) * 8 + g) * ST + j * 16 + 2 * t;
          const __nv_bfloat16* vl = sVl + ((d4 + i) * 8 + g) * ST + j * 16 + 2 * t;
          bh[i][0] = *reinterpret_cast<const uint32_t*>(vh); bh[i][1] = *reinterpret_cast<const uint32_t*>(vh + 8);
          bl[i][0] = *reinterpret_cast<const uint32_t*>(vl); bl[i][1] = *reinterpret_cast<const uint32_t*>(vl + 8);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) ea_mma(o[d4 + i], ph[0], ph[1], ph[2], ph[3], bh[i][0], bh[i][1]);
#pragma unroll
        for (int i = 0; i < 4; ++i) ea_mma(o[d4 + i], ph[0], ph[1], ph[2], ph[3], bl[i][0], bl[i][1]);
#pragma unroll
        for (int i = 0; i < 4; ++i) ea_mma(o[d4 + i], pl[0], pl[1], pl[2], pl[3], bh[i][0], bh[i][1]);
      }
    }
  }
  if (G > 1) {   // the groups' partial results meet in group 0 (thread to thread: the same rows and channels), in group order
    float* sM = reinterpret_cast<float*>(sKh);   // [36][EA_THREADS] in the group's own staging area
    ea_group_sync(grp);                          // the last tile is no longer read
    if (grp > 0) {
#pragma unroll
      for (int dt = 0; dt < 8; ++dt)
#pragma unroll
        for (int e = 0; e < 4; ++e) sM[(dt * 4 + e) * EA_THREADS + tid] = o[dt][e];
      sM[32 * EA_THREADS + tid] = m_a; sM[33 * EA_THREADS + tid] = m_b;
      sM[34 * EA_THREADS + tid] = l_a; sM[35 * EA_THREADS + tid] = l_b;
    }
    __syncthreads();
    if (grp > 0) return;
    float gm_a = m_a, gm_b = m_b;
#pragma unroll
    for (int j = 1; j < G; ++j) {
      const float* sJ = reinterpret_cast<const float*>(ea_smem + j * EA_GROUP_BYTES);
      gm_a = fmaxf(gm_a, sJ[32 * EA_THREADS + tid]); gm_b = fmaxf(gm_b, sJ[33 * EA_THREADS + tid]);
    }
    const float w_a = m_a == -INFINITY ? 0.f : __expf(m_a - gm_a), w_b = m_b == -INFINITY ? 0.f : __expf(m_b - gm_b);
    l_a *= w_a; l_b *= w_b;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) { o[dt][0] *= w_a; o[dt][1] *= w_a; o[dt][2] *= w_b; o[dt][3] *= w_b; }
#pragma unroll
    for (int j = 1; j < G; ++j) {
      const float* sJ = reinterpret_cast<const float*>(ea_smem + j * EA_GROUP_BYTES);
      const float mj_a = sJ[32 * EA_THREADS + tid], mj_b = sJ[33 * EA_THREADS + tid];
      const float v_a = mj_a == -INFINITY ? 0.f : __expf(mj_a - gm_a), v_b = mj_b == -INFINITY ? 0.f : __expf(mj_b - gm_b);
      l_a += sJ[34 * EA_THREADS + tid] * v_a; l_b += sJ[35 * EA_THREADS + tid] * v_b;
#pragma unroll
      for (int dt = 0; dt < 8; ++dt) {
        o[dt][0] += sJ[(dt * 4 + 0) * EA_THREADS + tid] * v_a; o[dt][1] += sJ[(dt * 4 + 1) * EA_THREADS + tid] * v_a;
        o[dt][2] += sJ[(dt * 4 + 2) * EA_THREADS + tid] * v_b; o[dt][3] += sJ[(dt * 4 + 3) * EA_THREADS + tid] * v_b;
      }
    }
  }
  l_a += __shfl_xor_sync(0xffffffffu, l_a, 1); l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
  l_b += __shfl_xor_sync(0xffffffffu, l_b, 1); l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
  const float ia = l_a > 0.f ? 1.f / l_a : 0.f, ib = l_b > 0.f ? 1.f / l_b : 0.f;
  const int ldh = a.H * EA_D;
#pragma unroll
  for (int dt = 0; dt < 8; ++dt) {
    const int col = h * EA_D + dt * 8 + 2 * t;
    if (oh) {
      uint32_t hv, lv;
      if (qa_pos < E) {
        ea_split(o[dt][0] * ia, o[dt][1] * ia, hv, lv);
        *reinterpret_cast<uint32_t*>(oh + (size_t)qa_pos * ldh + col) = hv;
        *reinterpret_cast<uint32_t*>(ol + (size_t)qa_pos * ldh + col) = lv;
      }
      if (qb_pos < E) {
        ea_split(o[dt][2] * ib, o[dt][3] * ib, hv, lv);
        *reinterpret_cast<uint32_t*>(oh + (size_t)qb_pos * ldh + col) = hv;
        *reinterpret_cast<uint32_t*>(ol + (size_t)qb_pos * ldh + col) = lv;
      }
    } else {
      if (qa_pos < E) *reinterpret_cast<float2*>(a.out + (size_t)qa_pos * a.ldo + col) = make_float2(o[dt][0] * ia, o[dt][1] * ia);
      if (qb_pos < E) *reinterpret_cast<float2*>(a.out + (size_t)qb_pos * a.ldo + col) = make_float2(o[dt][2] * ib, o[dt][3] * ib);
    }
  }
}

}  // namespace bild
