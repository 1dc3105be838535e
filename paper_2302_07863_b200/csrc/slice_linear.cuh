// Linear layer of a decoder pass for up to MAXB token rows, bf16 weights (steps S1, S3, S4, S6,
// S7, S8 and L1, L3, L4, L6, L7, L8), one block per SM:
//   * block b owns output rows [b N / G, (b + 1) N / G) of the weight matrix, a contiguous piece
//     of memory that one bulk (TMA) copy brings into shared memory.  The copy is issued BEFORE
//     the dependency wait of the programmatic launch, so the weights of a layer stream in while
//     the kernel before it is still running;
//   * after the wait the token rows (a few KB) follow: bulk copies for three rows and more, plain
//     128-bit loads for one or two; every block needs all of them, so they are read 148 times
//     from L2 instead of once per pair of rows.  The fused T5 norm takes one column group per
//     thread and row after row for one or two rows, one warp per row from three rows on;
//   * one or two token rows: a work item is 4 weight rows x 256 columns for all token rows of
//     the group; warp w takes items w, w + 8, ...; the partial sums of a quad are added in warp
//     order (fixed);
//   * more token rows: the block's 16-row tiles of the slice times 8-token tiles go through
//     mma.sync m16n8k16 (bf16 weights straight from shared memory, each activation split into
//     a bf16 head and a bf16 remainder, fp32 accumulation), the K range split over the warps of
//     a tile and added in warp order.  Rows in shared memory are padded so that the fragment
//     loads do not collide on banks;
//   * the epilogues are those of the other linear kernels (store, ReLU, GELU gate, residual add,
//     scatter to q / the KV cache); a thread owns one output row of the slice and every 4th, 8th
//     or 16th token row, the shorter the slice the more token rows per turn (a slice has 7 to 28
//     rows for the T5-large shapes, so five to sixteen token rows finish in one turn).
#pragma once
#include "decode_kernels.cuh"

namespace bild {

constexpr int SL_THREADS = 256;
constexpr int SL_QUADS = 12;                         // weight-row quads per block (48 rows)
constexpr int SL_PSUM = SL_QUADS * 8 * 32 * 4;
constexpr int SL_MISC = 1024;
constexpr int SL_PLAIN_ROWS = 2;      // groups of at most this many token rows are fetched with plain loads
constexpr int SL_NORM_ROWS_MIN = 3;   // groups of at least this many token rows: one warp per row in the fused norm

struct SliceShared {
  unsigned long long wbar, xbar;
  float inv[MAXB];
  float ssq[8][MAXB];
  int failed;
};

struct SliceArgs {
  LinArgs lin;
  int* err;
  int w_bytes;     // shared memory reserved for the weight slice
  int x_rows;      // token rows per group
  int mma_min;     // groups of at least this many token rows go through the tensor cores
};

constexpr int SL_WPAD = 16;   // bytes added to every weight row in shared memory
constexpr int SL_XPAD = 8;    // floats added to every token row in shared memory
inline size_t slice_w_bytes(int rows, int K) { return ((size_t)rows * (K * 2 + SL_WPAD) + 1023) / 1024 * 1024; }
inline size_t slice_smem_bytes(int w_bytes, int x_rows, int K) {
  return (size_t)w_bytes + (size_t)x_rows * (K + SL_XPAD) * 4 + SL_PSUM + SL_MISC + (size_t)K * 4;   // ... + norm gains
}

__device__ __forceinline__ void sl_wait(SliceShared* sh, int* err, unsigned long long* bar, uint32_t parity) {
  const uint32_t b = smem_u32(bar);
  if (mbar_try(b, parity)) return;
  if (*(volatile int*)&sh->failed) return;
  for (unsigned it = 0; it < SPIN_LIMIT; ++it)
    if (mbar_try(b, parity)) return;
  sh->failed = 1;
  atomicExch(err, (int)BILD_ERR_TIMEOUT);
}

// Item it belongs to quad it / nkb and column block it % nkb (rows past the end of the slice repeat
// its last row; nobody reads their sums).
template <int MG>
__device__ __forceinline__ void sl_items(const unsigned char* sW, int rowbytes, int nrows, int K, const float* Xs, int xst,
                                         float* psum, int warp, int lane) {
  constexpr int NA = 4 * MG;
  constexpr int NP = NA <= 4 ? 4 : NA <= 8 ? 8 : NA <= 16 ? 16 : 32;
  constexpr int SH = NP == 32 ? 0 : NP == 16 ? 1 : NP == 8 ? 2 : 3;
  const int nkb = (K + 255) >> 8, nq = (nrows + 3) >> 2;
#pragma unroll 1
  for (int qd = 0; qd < nq; ++qd) {
    int kb = (warp - qd * nkb) & 7;   // first column block of this quad that falls to this warp
    if (kb >= nkb) continue;
    float acc[NP];
#pragma unroll
    for (int i = 0; i < NP; ++i) acc[i] = 0.f;
    const unsigned char* rowp[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) rowp[r] = sW + (size_t)min(qd * 4 + r, nrows - 1) * rowbytes;
#pragma unroll 1
    for (; kb < nkb; kb += 8) {
      const int kofs = (kb << 8) + lane * 8;
      if (kofs < K) {
        uint4 w[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) w[r] = *reinterpret_cast<const uint4*>(rowp[r] + (size_t)kofs * 2);
#pragma unroll
        for (int m = 0; m < MG; ++m) {
          const float4 x0 = *reinterpret_cast<const float4*>(Xs + (size_t)m * xst + kofs);
          const float4 x1 = *reinterpret_cast<const float4*>(Xs + (size_t)m * xst + kofs + 4);
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            float s = acc[r * MG + m];
            s += __uint_as_float(w[r].x << 16) * x0.x;
            s += __uint_as_float(w[r].x & 0xffff0000u) * x0.y;
            s += __uint_as_float(w[r].y << 16) * x0.z;
            s += __uint_as_float(w[r].y & 0xffff0000u) * x0.w;
            s += __uint_as_float(w[r].z << 16) * x1.x;
            s += __uint_as_float(w[r].z & 0xffff0000u) * x1.y;
            s += __uint_as_float(w[r].w << 16) * x1.z;
            s += __uint_as_float(w[r].w & 0xffff0000u) * x1.w;
            acc[r * MG + m] = s;
          }
        }
      }
    }
    const float r = treduce<NP>(acc, lane);
    if ((lane & (32 / NP - 1)) == 0) psum[(qd * 8 + warp) * 32 + (lane >> SH)] = r;
  }
}

// Tensor-core variant for NT tiles of 8 token rows.  Warp w works on row tile w / KS and on
// the w % KS-th part of K (KS = 8, 4 or 2 for 1, 2 or 3 row tiles); its 16 x 8 accumulators go to
// psum[(w * NT + nt) * 128 + lane * 4 ..] in the fragment layout of the instruction.
__device__ __forceinline__ uint32_t sl_pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
template <int NT>
__device__ __forceinline__ void sl_mma(const unsigned char* sW, int rowst, int nrows, int K, const float* Xs, int xst, int mg,
                                       float* psum, int warp, int lane) {
  const int MT = (nrows + 15) >> 4, ks_sh = MT == 1 ? 3 : MT == 2 ? 2 : 1, KS = 1 << ks_sh;
  if (warp >= MT * KS) return;
  const int mt = warp >> ks_sh, ks = warp & (KS - 1);
  const int steps = (K + 15) >> 4, per = (steps + KS - 1) >> ks_sh;
  const int s0 = ks * per, s1 = min(steps, s0 + per);
  const int g = lane >> 2, t = lane & 3;
  const unsigned char* pa0 = sW + (size_t)min(mt * 16 + g, nrows - 1) * rowst + t * 4;
  const unsigned char* pa1 = sW + (size_t)min(mt * 16 + g + 8, nrows - 1) * rowst + t * 4;
  const float* xb[NT];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) xb[nt] = Xs + (size_t)min(nt * 8 + g, mg - 1) * xst + 2 * t;
  float c[NT][4], e[NT][4];   // products with the heads and with the remainders of the activations: two independent chains
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
    e[nt][0] = e[nt][1] = e[nt][2] = e[nt][3] = 0.f;
  }
#pragma unroll 4
  for (int st = s0; st < s1; ++st) {
    const int k0 = st << 4;
    const bool tail = k0 + 8 >= K;   // K is a multiple of 8: the second half of the last step may not exist
    const uint32_t a0 = *reinterpret_cast<const uint32_t*>(pa0 + k0 * 2);
    const uint32_t a1 = *reinterpret_cast<const uint32_t*>(pa1 + k0 * 2);
    const uint32_t a2 = tail ? 0u : *reinterpret_cast<const uint32_t*>(pa0 + k0 * 2 + 16);
    const uint32_t a3 = tail ? 0u : *reinterpret_cast<const uint32_t*>(pa1 + k0 * 2 + 16);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float2 x0 = *reinterpret_cast<const float2*>(xb[nt] + k0);
      const float2 x1 = tail ? make_float2(0.f, 0.f) : *reinterpret_cast<const float2*>(xb[nt] + k0 + 8);
      const uint32_t h0 = sl_pack_bf16(x0.x, x0.y), h1 = sl_pack_bf16(x1.x, x1.y);
      const uint32_t l0 = sl_pack_bf16(x0.x - __uint_as_float(h0 << 16), x0.y - __uint_as_float(h0 & 0xffff0000u));
      const uint32_t l1 = sl_pack_bf16(x1.x - __uint_as_float(h1 << 16), x1.y - __uint_as_float(h1 & 0xffff0000u));
      asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                   : "+f"(c[nt][0]), "+f"(c[nt][1]), "+f"(c[nt][2]), "+f"(c[nt][3])
                   : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(h0), "r"(h1));
      asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                   : "+f"(e[nt][0]), "+f"(e[nt][1]), "+f"(e[nt][2]), "+f"(e[nt][3])
                   : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(l0), "r"(l1));
    }
  }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
    *reinterpret_cast<float4*>(psum + ((size_t)(warp * NT + nt) * 32 + lane) * 4) = make_float4(c[nt][0] + e[nt][0], c[nt][1] + e[nt][1], c[nt][2] + e[nt][2], c[nt][3] + e[nt][3]);
}

// Products of a weight tile in shared memory (rows `rowst` bytes apart) with token rows whose operand fragments were built
// once (a caller that multiplies many tiles with the same rows: the LM head).  A thread loads 16 bytes of a weight row -- the columns
// 8 t .. 8 t + 7 of a 32-column chunk -- and uses them as the left operands of two m16n8k16 instructions: within a chunk
// the instruction's column positions are dealt to the threads' columns (position 2 t, 2 t + 1 | 2 t + 8, 2 t + 9 of
// instruction m <-> columns 8 t + 4 m + 0, 1 | 2, 3), and the fragments of the token rows follow the same order, so every
// product meets its partner.
constexpr int SL_PERM_CHUNKS = 4;   // 32-column chunks of a warp's K range (K / 8 or K / 4 columns: K <= 1024 or 512)
template <int NT>
struct SlPermFrags { uint32_t h[NT][SL_PERM_CHUNKS][2][2], l[NT][SL_PERM_CHUNKS][2][2]; };
__host__ __device__ inline bool sl_perm_fits(int nrows, int K) {
  const int MT = (nrows + 15) >> 4, ks_sh = MT == 1 ? 3 : MT == 2 ? 2 : 1;
  return (nrows == 16 || nrows == 32) && K % (32 << ks_sh) == 0 && (K >> ks_sh) / 32 <= SL_PERM_CHUNKS;
}
template <int NT>
__device__ __forceinline__ void sl_perm_frags(int nrows, int K, const float* Xs, int xst, int mg, int warp, int lane, SlPermFrags<NT>& f) {
  const int MT = (nrows + 15) >> 4, ks_sh = MT == 1 ? 3 : MT == 2 ? 2 : 1, KS = 1 << ks_sh;
  const int ks = warp & (KS - 1), cols = K >> ks_sh, chunks = cols >> 5;
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const float* xb = Xs + (size_t)min(nt * 8 + g, mg - 1) * xst + ks * cols + 8 * t;
#pragma unroll
    for (int ch = 0; ch < SL_PERM_CHUNKS; ++ch)
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ch < chunks) x = *reinterpret_cast<const float4*>(xb + ch * 32 + 4 * m);
        const uint32_t h0 = sl_pack_bf16(x.x, x.y), h1 = sl_pack_bf16(x.z, x.w);
        f.h[nt][ch][m][0] = h0; f.h[nt][ch][m][1] = h1;
        f.l[nt][ch][m][0] = sl_pack_bf16(x.x - __uint_as_float(h0 << 16), x.y - __uint_as_float(h0 & 0xffff0000u));
        f.l[nt][ch][m][1] = sl_pack_bf16(x.z - __uint_as_float(h1 << 16), x.w - __uint_as_float(h1 & 0xffff0000u));
      }
  }
}
template <int NT>
__device__ __forceinline__ void sl_mma_perm(const unsigned char* sW, int rowst, int nrows, int K, const SlPermFrags<NT>& f, float* psum, int warp,
                                            int lane) {
  const int MT = (nrows + 15) >> 4, ks_sh = MT == 1 ? 3 : MT == 2 ? 2 : 1, KS = 1 << ks_sh;
  if (warp >= MT * KS) return;
  const int mt = warp >> ks_sh, ks = warp & (KS - 1), cols = K >> ks_sh, chunks = cols >> 5;
  const int g = lane >> 2, t = lane & 3;
  const unsigned char* pa0 = sW + (size_t)(mt * 16 + g) * rowst + (size_t)(ks * cols + 8 * t) * 2;
  const unsigned char* pa1 = pa0 + (size_t)8 * rowst;
  float c[NT][4], e[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
    e[nt][0] = e[nt][1] = e[nt][2] = e[nt][3] = 0.f;
  }
#pragma unroll
  for (int ch = 0; ch < SL_PERM_CHUNKS; ++ch)
    if (ch < chunks) {
      const uint4 a0 = *reinterpret_cast<const uint4*>(pa0 + ch * 64), a1 = *reinterpret_cast<const uint4*>(pa1 + ch * 64);
#define SL_MMA_P(ACC, A0, A1, A2, A3, B0, B1)                                                                                    \
      asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"   \
                   : "+f"(ACC[0]), "+f"(ACC[1]), "+f"(ACC[2]), "+f"(ACC[3]) : "r"(A0), "r"(A1), "r"(A2), "r"(A3), "r"(B0), "r"(B1))
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        SL_MMA_P(c[nt], a0.x, a1.x, a0.y, a1.y, f.h[nt][ch][0][0], f.h[nt][ch][0][1]);
        SL_MMA_P(e[nt], a0.x, a1.x, a0.y, a1.y, f.l[nt][ch][0][0], f.l[nt][ch][0][1]);
        SL_MMA_P(c[nt], a0.z, a1.z, a0.w, a1.w, f.h[nt][ch][1][0], f.h[nt][ch][1][1]);
        SL_MMA_P(e[nt], a0.z, a1.z, a0.w, a1.w, f.l[nt][ch][1][0], f.l[nt][ch][1][1]);
      }
#undef SL_MMA_P
    }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
    *reinterpret_cast<float4*>(psum + ((size_t)(warp * NT + nt) * 32 + lane) * 4) = make_float4(c[nt][0] + e[nt][0], c[nt][1] + e[nt][1], c[nt][2] + e[nt][2], c[nt][3] + e[nt][3]);
}

__global__ void __launch_bounds__(SL_THREADS) slice_linear_kernel(SliceArgs s) {
  extern __shared__ __align__(1024) unsigned char sl_smem[];
  const LinArgs& a = s.lin;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, K = a.K;
  const int r0 = (int)(((long long)blockIdx.x * a.N) / G), r1 = (int)(((long long)(blockIdx.x + 1) * a.N) / G);
  const int n = r1 - r0, nmat = a.epi == EPI_GATED ? 2 : 1, nrows = n * nmat, rowbytes = K * 2 + SL_WPAD, xst = K + SL_XPAD;
  if (n == 0) {   // more blocks than rows
    pdl_launch_dependents();
    return;
  }
  unsigned char* sW = sl_smem;
  float* Xs = reinterpret_cast<float*>(sl_smem + s.w_bytes);
  float* psum = Xs + (size_t)s.x_rows * xst;
  SliceShared* sh = reinterpret_cast<SliceShared*>(psum + SL_PSUM / 4);
  float* sG = psum + SL_PSUM / 4 + SL_MISC / 4;   // [K] norm gains
  if (tid == 0) {
    mbar_init(smem_u32(&sh->wbar), 1);
    mbar_init(smem_u32(&sh->xbar), 1);
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect(smem_u32(&sh->wbar), (uint32_t)(nrows * K * 2));
  }
  __syncthreads();
  // the weights depend on nothing: request them before waiting for the kernel in front, one copy per
  // row (the rows are padded in shared memory)
  if (tid < nrows) {
    const int r = tid < n ? tid : tid - n;
    const __nv_bfloat16* W = (const __nv_bfloat16*)(tid < n ? a.W0 : a.W1);
    bulk_g2s(smem_u32(sW + (size_t)tid * rowbytes), W + (size_t)(r0 + r) * K, (uint32_t)(K * 2), smem_u32(&sh->wbar));
  }
  float4 gv[2];   // gains of the columns this thread scales (K <= 2048 where a norm precedes)
  if (a.gain) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int c = tid * 4 + j * 1024;
      gv[j] = c < K ? __ldg(reinterpret_cast<const float4*>(a.gain + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
      if (c < K) *reinterpret_cast<float4*>(sG + c) = gv[j];   // (read after the barriers below)
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  const int M = min(a.desc->k, MAXB), pos0 = a.desc->pos0;
  const int nkb = (K + 255) >> 8, rgl = s.x_rows;
  // epilogue: thread <-> (output row ep_r of the slice, token rows ep_m, ep_m + ep_step, ...); short slices take
  // more token rows per turn (16 / 8 / 4 for slices of up to 16 / 32 / 64 rows)
  const int ep_sh = n <= 16 ? 4 : n <= 32 ? 5 : 6;
  const int ep_r = tid & ((1 << ep_sh) - 1), ep_m = tid >> ep_sh, ep_step = SL_THREADS >> ep_sh;
  unsigned xuse = 0;
#pragma unroll 1
  for (int m0 = 0; m0 < M; m0 += rgl, ++xuse) {
    const int mg = min(rgl, M - m0);
    // the values a residual epilogue adds to are requested now, not when the sums are ready
    float y_old[4] = {0.f, 0.f, 0.f, 0.f};
    if (a.epi == EPI_RESID && ep_r < n) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int m = ep_m + ep_step * i;
        if (m < mg) y_old[i] = __ldcg(a.Y + (size_t)(m0 + m) * a.ldy + r0 + ep_r);
      }
    }
    if (mg <= SL_PLAIN_ROWS) {
      // one or two token rows: plain 128-bit loads, eight in flight per thread (one round trip to L2 and no
      // proxy fence, copy engine or mbarrier between the dependency wait and the first product; measured
      // 2.5 % faster per pass for one row, slower than the bulk copies from five rows on)
      const int K4 = K >> 2, per_row = (K4 + SL_THREADS - 1) / SL_THREADS, nitems = mg * per_row;
#pragma unroll 1
      for (int it0 = 0; it0 < nitems; it0 += 8) {
        float4 r[8];
        int dst[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int it = it0 + j, m = it / per_row, c4 = (it - m * per_row) * SL_THREADS + tid;
          dst[j] = -1;
          if (it < nitems && c4 < K4) {
            r[j] = __ldcg(reinterpret_cast<const float4*>(a.X + (size_t)(m0 + m) * a.ldx) + c4);
            dst[j] = m * xst + c4 * 4;
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (dst[j] >= 0) *reinterpret_cast<float4*>(Xs + dst[j]) = r[j];
      }
      __syncthreads();
    } else {
    if (tid == 0) mbar_expect(smem_u32(&sh->xbar), (uint32_t)(mg * K * 4));
    __syncthreads();   // the barrier expects the bytes (and the group before is done with the rows)
    if (tid < mg) {
      asm volatile("fence.proxy.async;" ::: "memory");   // rows written by the kernel in front, read by the copy engine
      bulk_g2s(smem_u32(Xs + (size_t)tid * xst), a.X + (size_t)(m0 + tid) * a.ldx, (uint32_t)(K * 4), smem_u32(&sh->xbar));
    }
    sl_wait(sh, s.err, &sh->xbar, xuse & 1);
    }
    if (a.gain && mg >= SL_NORM_ROWS_MIN) {   // T5 norm, one warp per token row: all rows of the group at once (faster from three rows on)
#pragma unroll 1
      for (int m = warp; m < mg; m += SL_THREADS / 32) {
        float* xr = Xs + (size_t)m * xst;
        float ss0 = 0.f, ss1 = 0.f;
#pragma unroll 2
        for (int c = lane * 4; c < K; c += 128) {
          float4 v = *reinterpret_cast<float4*>(xr + c);
          const float4 g = *reinterpret_cast<const float4*>(sG + c);
          ss0 += v.x * v.x + v.y * v.y;
          ss1 += v.z * v.z + v.w * v.w;
          v.x *= g.x; v.y *= g.y; v.z *= g.z; v.w *= g.w;
          *reinterpret_cast<float4*>(xr + c) = v;
        }
        const float ss = warp_sum(ss0 + ss1);
        if (lane == 0) sh->inv[m] = rsqrtf(ss / (float)K + a.eps);
      }
      __syncthreads();   // scaled rows and 1 / rms are visible to every warp
    } else if (a.gain) {   // T5 norm: x * g / sqrt(mean(x^2) + eps); the division is applied to the dot products
      for (int m = 0; m < mg; ++m) {
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int c = tid * 4 + j * 1024;
          if (c < K) {
            float4 v = *reinterpret_cast<float4*>(Xs + (size_t)m * xst + c);
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
            v.x *= gv[j].x; v.y *= gv[j].y; v.z *= gv[j].z; v.w *= gv[j].w;
            *reinterpret_cast<float4*>(Xs + (size_t)m * xst + c) = v;
          }
        }
        ss = warp_sum(ss);
        if (lane == 0) sh->ssq[warp][m] = ss;
      }
      __syncthreads();
      if (tid < mg) {
        float ss = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv) ss += sh->ssq[wv][tid];
        sh->inv[tid] = rsqrtf(ss / (float)K + a.eps);
      }
    }
    if (m0 == 0) sl_wait(sh, s.err, &sh->wbar, 0);
    const bool tc = mg >= s.mma_min;   // tensor cores for the larger groups
    const int mgr = mg;
    if (tc) {
      if (!a.gain) __syncthreads();   // (with a norm the rows were synchronised above)
      if (mg <= 8) sl_mma<1>(sW, rowbytes, nrows, K, Xs, xst, mg, psum, warp, lane);
      else sl_mma<2>(sW, rowbytes, nrows, K, Xs, xst, mg, psum, warp, lane);
    } else {
      switch (mgr) {
        case 1: sl_items<1>(sW, rowbytes, nrows, K, Xs, xst, psum, warp, lane); break;
        case 2: sl_items<2>(sW, rowbytes, nrows, K, Xs, xst, psum, warp, lane); break;
        case 3: sl_items<3>(sW, rowbytes, nrows, K, Xs, xst, psum, warp, lane); break;
        default: sl_items<4>(sW, rowbytes, nrows, K, Xs, xst, psum, warp, lane); break;
      }
    }
    __syncthreads();
    // epilogue: (output row r, token row m); partial sums are added in warp order
    const int MT = (nrows + 15) >> 4, ks_sh = MT == 1 ? 3 : MT == 2 ? 2 : 1, NT = mg <= 8 ? 1 : 2;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = ep_m + ep_step * i;
      if (m >= mg) break;
      const int r = ep_r;
      if (r >= n) continue;
      auto total = [&](int row) {
        float t = 0.f;
        if (tc) {   // fragment layout: row = group (+ 8), token = 2 * (lane & 3) (+ 1)
          const int mt = row >> 4, rr = row & 15, col = m & 7;
          const float* p = psum + ((size_t)((mt << ks_sh) * NT + (m >> 3)) * 32 + (rr & 7) * 4 + (col >> 1)) * 4 + (rr >> 3) * 2 + (col & 1);
          for (int ks = 0; ks < (1 << ks_sh); ++ks) t += p[(size_t)ks * NT * 128];
        } else {
          const int qd = row >> 2, first = qd * nkb;
          const float* p = psum + (size_t)(qd * 8) * 32 + (row & 3) * mgr + m;
#pragma unroll
          for (int wv = 0; wv < 8; ++wv)
            if (((wv - first) & 7) < nkb) t += p[wv * 32];   // warp wv took part in this quad
        }
        return t;
      };
      float v = total(r);
      if (a.gain) v *= sh->inv[m];
      const int nn = r0 + r, mm = m0 + m;
      if (a.epi == EPI_RESID) a.Y[(size_t)mm * a.ldy + nn] = y_old[i] + v;
      else if (a.epi == EPI_STORE) a.Y[(size_t)mm * a.ldy + nn] = v;
      else if (a.epi == EPI_RELU) a.Y[(size_t)mm * a.ldy + nn] = fmaxf(v, 0.f);
      else if (a.epi == EPI_GATED) a.Y[(size_t)mm * a.ldy + nn] = gelu_tanh(v) * (total(n + r) * (a.gain ? sh->inv[m] : 1.f));
      else heads_store(a, nn, mm, pos0, v);
    }
    if (m0 + rgl < M) __syncthreads();   // another group of token rows: staged rows and partial sums are reused
  }
}

}  // namespace bild
