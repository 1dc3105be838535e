// Decoder sub-layers as ONE kernel each (bf16 weights, up to 8 token rows a launch), so that a layer
// of a decoder pass is three dependent kernels instead of eight:
//   * attn_sub_kernel: x_out = x_in + W_o * Attention(W_q|k|v * rms_norm(x_in))   (steps S1-S3 / L1-L3
//     for self-attention, S4-S6 / L4-L6 for cross-attention).  A cluster of C blocks owns one head:
//     rank r multiplies its share of the head's q|k|v rows (weights fetched by bulk copies BEFORE
//     the dependency wait of the programmatic launch), the cluster exchanges the k x 3 x d_kv results
//     through distributed shared memory, rank r then attends over its share of the keys, the
//     per-rank (max, sum, weighted values) records are exchanged the same way, and every rank
//     multiplies the merged head output with its share of the rows of W_o's column slice; while a head has few keys
//     (they fit one staged chunk) every rank attends over all of them instead and the second exchange falls away;
//     the first kernel of a pass takes its rows from the embedding table (S0 / L0);
//   * ffn_sub_kernel: x_out = x_in + W_fo * act(W_i * rms_norm(x_in))   (S7-S8 / L7-L8).  Block b owns a
//     slice of d_ff (a multiple of 8 rows): the rows of W_i (and of the gate matrix) in shared memory and the
//     matching columns of W_fo in registers (from a copy laid out in load order), so the hidden activations never
//     leave the block.
// Both kernels produce partial sums over heads / slices of d_ff of the d_model outputs.  They are added
// into x_out with vector reductions at the L2 (red.global.add); x_out was zeroed by the kernel before the
// previous one, one designated block adds x_in (the residual term), and every kernel zeroes the buffer
// the next kernel accumulates into: three buffers rotate through the pass.  The order of the floating-
// point additions at the L2 is not fixed, so logits may differ in the last bits from run to run.
#pragma once
#include "slice_linear.cuh"

namespace bild {

constexpr int SUB_THREADS = 256;
constexpr int SUB_PSUM = SL_PSUM;   // bytes of partial sums of sl_items / sl_mma
constexpr int SUB_RECPAD = 4;       // record of a rank and row = [max, sum, -, -, values[d_kv]]
constexpr int SUB_MAX_ROWS = 4 * SL_QUADS;   // weight rows of one block and phase (limit of sl_items / sl_mma)
constexpr int SUB_FO_REGS = 32;              // most rows of d_ff a block takes: its columns of W_fo fill 64 registers of a thread
constexpr int SUB_HALF_SM = 113 * 1024;      // shared memory of a block that leaves room for a second one on the SM
constexpr int SUB_MB = 8;                    // token rows of the block variant (one 8-token tile of the tensor-core instruction)

struct SubShared {
  unsigned long long wbar;
  float inv[MAXB];
  float ssq[8][MAXB];
  float rmax[MAXB], rsum[MAXB], rscale[MAXB];
  int failed;
};

// Optional cycle stamps (build with -DBILD_STAMPS), summed per kernel kind and phase boundary: [0] block 0, [1] every
// block, [2] the longest a block took ([..][23]: how many blocks were added).
#ifdef BILD_STAMPS
__device__ unsigned long long g_sub_stamps[3][4][24];
#define SUB_STAMP_BEGIN() long long st_t[20]; int st_n = 0; st_t[st_n++] = clock64()
#define SUB_STAMP() st_t[st_n++] = clock64()
#define SUB_STAMP_END(kind)                                                                                \
  if (threadIdx.x == 0) {                                                                                 \
    for (int i_ = 1; i_ < st_n; ++i_) {                                                                   \
      const unsigned long long dt_ = (unsigned long long)(st_t[i_] - st_t[i_ - 1]);                      \
      if (blockIdx.x == 0) atomicAdd(&g_sub_stamps[0][kind][i_ - 1], dt_);                                \
      atomicAdd(&g_sub_stamps[1][kind][i_ - 1], dt_);                                                     \
      atomicMax(&g_sub_stamps[2][kind][i_ - 1], dt_);                                                     \
    }                                                                                                     \
    if (blockIdx.x == 0) atomicAdd(&g_sub_stamps[0][kind][23], 1ull);                                     \
    atomicAdd(&g_sub_stamps[1][kind][23], 1ull);                                                          \
  }
#else
#define SUB_STAMP_BEGIN()
#define SUB_STAMP()
#define SUB_STAMP_END(kind)
#endif

__host__ __device__ inline int sub_up16(int v) { return (v + 15) & ~15; }
// row stride (floats) of staged keys / values: 16 mod 32, so the four channel quarters of two keys hit 32 distinct banks
__host__ __device__ inline int sub_kv_stride(int dkv) { return ((dkv + 15) / 32) * 32 + 16; }

// Bounded wait for the weight copies: after `spin` unsuccessful polls the block records BILD_ERR_TIMEOUT for the host
// and goes on (with whatever the shared memory holds), so that every block of the kernel still leaves.
__device__ __forceinline__ void sub_wait(SubShared* sh, int* err, unsigned long long* bar, uint32_t parity, unsigned spin) {
  const uint32_t b = smem_u32(bar);
  if (mbar_try(b, parity)) return;
  if (*(volatile int*)&sh->failed) return;
  for (unsigned it = 0; it < spin; ++it)
    if (mbar_try(b, parity)) return;
  sh->failed = 1;
  atomicExch(err, (int)BILD_ERR_TIMEOUT);
}

__device__ __forceinline__ void sub_cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
// (nothing to publish: does not wait for the loads in flight)
__device__ __forceinline__ void sub_cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void sub_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void sub_cp16(void* dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void sub_cp_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// dot product (weight row `row`, token row m) from the partial sums of sl_items<1> (ONE) or sl_mma<1>, added in warp order
template <bool ONE>
__device__ __forceinline__ float sub_total(const float* psum, int row, int m, int nrows, int K) {
  float t = 0.f;
  if (ONE) {
    const int nkb = (K + 255) >> 8, qd = row >> 2, first = qd * nkb;
    const float* p = psum + (size_t)(qd * 8) * 32 + (row & 3);
#pragma unroll
    for (int wv = 0; wv < 8; ++wv)
      if (((wv - first) & 7) < nkb) t += p[wv * 32];   // warp wv took part in this quad
  } else {   // fragment layout of the instruction: row = group (+ 8), token = 2 * (lane & 3) (+ 1); one tile of 8 tokens
    const int MT = (nrows + 15) >> 4, ks_sh = MT == 1 ? 3 : MT == 2 ? 2 : 1;
    const int mt = row >> 4, rr = row & 15;
    const float* p = psum + ((size_t)(mt << ks_sh) * 32 + (rr & 7) * 4 + (m >> 1)) * 4 + (rr >> 3) * 2 + (m & 1);
    float v[8];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) v[ks] = ks < (1 << ks_sh) ? p[(size_t)ks * 128] : 0.f;   // loads side by side
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) t += v[ks];
  }
  return t;
}

// Token rows, after the dependency wait (d <= 1024: one 128-bit load per thread and row).  The loads are issued first
// thing after the wait, for the rows of the pass (the row count is read before the wait); sub_rows_finish then writes
// x * gain into Xs and 1 / rms into
// sh->inv (returned for the single row of ONE).  The raw values of the columns [seed0, seed1) (multiples of 4) also go
// to sSeed[m][column - seed0]: the residual term the block adds.
// Block variant: the normalised token rows wait in shared memory as bf16 heads [SUB_MB][d / 2 + 4] (two values a word)
// followed by their bf16 remainders in the same layout: d + 8 words a row in all, as for the fp32 rows of the single-row
// variant.  The row stride of d / 2 + 4 words is 4 times an odd number for d a multiple of 32: the eight rows a warp
// reads side by side fall into different banks.
__host__ __device__ inline int sub_split_stride(int d) { return (d >> 1) + 4; }

// Products of up to 48 weight rows (shared memory, row stride rowst bytes) with the token rows on mma.sync m16n8k16, one tile
// of 8 token rows: warp w works on row tile w / KS and on the w % KS-th part of K (KS = 8, 4 or 2 for 1, 2 or 3 row tiles),
// as sl_mma<1>, with the right operand read ready-made; partial sums in the same place and layout (sub_total<false>).
__device__ __forceinline__ void sub_mma_split(const unsigned char* sW, int rowst, int nrows, int K, const float* Xs, int mg, float* psum,
                                              int warp, int lane) {
  const int MT = (nrows + 15) >> 4, ks_sh = MT == 1 ? 3 : MT == 2 ? 2 : 1, KS = 1 << ks_sh;
  if (warp >= MT * KS) return;
  const int mt = warp >> ks_sh, ks = warp & (KS - 1);
  const int steps = K >> 4, per = (steps + KS - 1) >> ks_sh;   // K is a multiple of 16 here
  const int s0 = ks * per, s1 = min(steps, s0 + per);
  const int g = lane >> 2, t = lane & 3, hw = sub_split_stride(K);
  const unsigned char* pa0 = sW + (size_t)min(mt * 16 + g, nrows - 1) * rowst + t * 4;
  const unsigned char* pa1 = sW + (size_t)min(mt * 16 + g + 8, nrows - 1) * rowst + t * 4;
  const uint32_t* xh = reinterpret_cast<const uint32_t*>(Xs) + (size_t)min(g, mg - 1) * hw + t;
  const uint32_t* xl = xh + (size_t)SUB_MB * hw;
  float c[4] = {0.f, 0.f, 0.f, 0.f}, e[4] = {0.f, 0.f, 0.f, 0.f};   // heads and remainders: two independent chains
#pragma unroll 4
  for (int st = s0; st < s1; ++st) {
    const int k0 = st << 4;
    const uint32_t a0 = *reinterpret_cast<const uint32_t*>(pa0 + k0 * 2), a1 = *reinterpret_cast<const uint32_t*>(pa1 + k0 * 2);
    const uint32_t a2 = *reinterpret_cast<const uint32_t*>(pa0 + k0 * 2 + 16), a3 = *reinterpret_cast<const uint32_t*>(pa1 + k0 * 2 + 16);
    const uint32_t h0 = xh[k0 >> 1], h1 = xh[(k0 >> 1) + 4], l0 = xl[k0 >> 1], l1 = xl[(k0 >> 1) + 4];
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(h0), "r"(h1));
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(e[0]), "+f"(e[1]), "+f"(e[2]), "+f"(e[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(l0), "r"(l1));
  }
  *reinterpret_cast<float4*>(psum + ((size_t)warp * 32 + lane) * 4) = make_float4(c[0] + e[0], c[1] + e[1], c[2] + e[2], c[3] + e[3]);
}

template <bool ONE>
struct SubRows { float4 v[ONE ? 1 : SUB_MB]; };

template <bool ONE>
__device__ __forceinline__ void sub_rows_issue(const float* __restrict__ x_in, int rows, int d, int tid, SubRows<ONE>& rw) {
  if (tid * 4 < d) {   // rows: the rows of the pass
#pragma unroll
    for (int i = 0; i < (ONE ? 1 : SUB_MB); ++i)
      if (i < rows) rw.v[i] = __ldcg(reinterpret_cast<const float4*>(x_in + (size_t)i * d) + tid);
  }
}

// The first sub-layer of a pass takes its rows from the embedding table (S0 / L0): row i = E[token_i], bf16.
template <bool ONE>
__device__ __forceinline__ void sub_rows_embed(const __nv_bfloat16* __restrict__ E, const int* __restrict__ tokens, int vocab, int rows,
                                               int d, int tid, SubRows<ONE>& rw) {
  if (tid * 4 < d) {
#pragma unroll
    for (int i = 0; i < (ONE ? 1 : SUB_MB); ++i)
      if (i < rows) {
        int t = tokens[i];
        t = t < 0 ? 0 : (t >= vocab ? vocab - 1 : t);
        const uint2 w = __ldg(reinterpret_cast<const uint2*>(E + (size_t)t * d) + tid);
        rw.v[i] = make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u), __uint_as_float(w.y << 16),
                              __uint_as_float(w.y & 0xffff0000u));
      }
  }
}

template <bool ONE>
__device__ __forceinline__ float sub_rows_finish(const SubRows<ONE>& rw, int k, int d, float4 g, float eps, float* Xs, int xst,
                                                 SubShared* sh, float* sSeed, int seed0, int seed1, int tid, int lane, int warp) {
  const int d4 = d >> 2, c = tid * 4;
  const bool on = tid < d4, sd = c >= seed0 && c < seed1;
  if (ONE) {
    float ss = 0.f;
    if (on) {
      float4 w = rw.v[0];
      ss = w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
      if (sd) *reinterpret_cast<float4*>(sSeed + (c - seed0)) = w;
      w.x *= g.x; w.y *= g.y; w.z *= g.z; w.w *= g.w;
      *reinterpret_cast<float4*>(Xs + c) = w;
    }
    ss = warp_sum(ss);
    if (lane == 0) sh->ssq[warp][0] = ss;
    __syncthreads();
    ss = 0.f;
#pragma unroll
    for (int wv = 0; wv < 8; ++wv) ss += sh->ssq[wv][0];
    return rsqrtf(ss / (float)d + eps);
  } else {
    float q[SUB_MB];
#pragma unroll
    for (int i = 0; i < SUB_MB; ++i) {
      q[i] = 0.f;
      if (on && i < k) {
        float4 w = rw.v[i];
        q[i] = w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
        if (sd) *reinterpret_cast<float4*>(sSeed + (size_t)i * (seed1 - seed0) + (c - seed0)) = w;
        w.x *= g.x; w.y *= g.y; w.z *= g.z; w.w *= g.w;
        // stored as bf16 heads and bf16 remainders, the form the tensor-core products read (sub_mma_split)
        const uint32_t h0 = sl_pack_bf16(w.x, w.y), h1 = sl_pack_bf16(w.z, w.w);
        const uint32_t l0 = sl_pack_bf16(w.x - __uint_as_float(h0 << 16), w.y - __uint_as_float(h0 & 0xffff0000u));
        const uint32_t l1 = sl_pack_bf16(w.z - __uint_as_float(h1 << 16), w.w - __uint_as_float(h1 & 0xffff0000u));
        uint32_t* xh = reinterpret_cast<uint32_t*>(Xs);
        const int hw = sub_split_stride(d);
        *reinterpret_cast<uint2*>(xh + (size_t)i * hw + 2 * tid) = make_uint2(h0, h1);
        *reinterpret_cast<uint2*>(xh + (size_t)(SUB_MB + i) * hw + 2 * tid) = make_uint2(l0, l1);
      }
    }
    const float r8 = treduce<8>(q, lane);   // lanes 4 i hold the warp's sum of row i
    if ((lane & 3) == 0) sh->ssq[warp][lane >> 2] = r8;
    __syncthreads();
    if (tid < k) {
      float ss = 0.f;
#pragma unroll
      for (int wv = 0; wv < 8; ++wv) ss += sh->ssq[wv][tid];
      sh->inv[tid] = rsqrtf(ss / (float)d + eps);
    }
    __syncthreads();
    return 0.f;
  }
}

// ------------------------------------------------------------------------------------------------
// Attention sub-layer
// ------------------------------------------------------------------------------------------------
struct AttnSubLayout { int wq, xs, kv, kv_late, qkv, psum, probs, bias, seed, sa, red, recloc, loc, out, sh, total; };

struct AttnSubArgs {
  const CallDesc* desc;
  const float* x_in;    // [rows of the pass][d] residual stream (complete)
  const __nv_bfloat16* emb;  // not null: the first sub-layer of a pass, its rows are E[tokens[i]] instead of x_in (S0 / L0)
  const int* tokens;
  int vocab;
  float* x_out;         // [MAXB][d] zero on entry; receives x_in + the sub-layer's output
  float* x_zero;        // [MAXB][d] cleared for the kernel after this one
  const float* gain;
  float eps;
  const __nv_bfloat16* Wp;   // self: [3 I][d] (q rows, then k, then v); cross: [I][d]
  const __nv_bfloat16* Wo;   // [d][I]
  float* kc;                 // [H][cap][dkv] keys of this layer (self: rows pos0.. are appended; cross: read only)
  float* vc;
  int cap;
  const float* bias;         // self: [H][bias_ld] relative-position bias by distance; cross: unused
  int bias_ld;
  const int* n_keys_dev;     // cross: encoder positions
  int self;
  int d, I, H, dkv, dkv_shift, C, c_shift;
  int kc_keys;               // keys per staged chunk
  int red_keys;              // up to this many keys every rank attends over ALL keys of the head (no second exchange)
  int bias_len;              // floats reserved for the staged bias
  int mb;                    // token rows the shared memory is sized for
  unsigned spin;             // polls of the weight barrier before the kernel gives up
  int skip_copies;           // test of the time-out path: the weight copies are announced but not issued
  int* err;
  AttnSubLayout L;
};

// Shared memory is kept under half an SM's (113 KB) where possible, so that the next kernel's blocks can sit beside
// this kernel's and run their prologue and weight fetch in its shadow (and so that 16 clusters of 8 are resident at
// once: above that size an SM takes one block, and a B200 then holds only 15 such clusters).
inline AttnSubLayout attn_sub_layout(int d, int dkv, int P, int C, int mb, int kc, int bias_len) {
  AttnSubLayout L;
  const int npr = (P * dkv + C - 1) / C, no = (d + C - 1) / C;
  const int wq_b = sub_up16(npr * (d * 2 + SL_WPAD)), kv_b = sub_up16(kc * (sub_kv_stride(dkv) + dkv + 4) * 4);
  int off = 0;
  // block variant, self-attention: the keys / values of the rank are staged where the projection rows were, once the
  // products are done (they depend on the cache position anyway); otherwise they have an area of their own and the
  // encoder keys are requested in the prologue
  L.kv_late = (mb > 1 && P == 3 && kv_b <= wq_b) ? 1 : 0;
  L.wq = off; off += wq_b;
  const int xs_b = mb * (d + SL_XPAD) * 4, rec_b = C * mb * (dkv + SUB_RECPAD) * 4;
  L.xs = off; off += sub_up16(xs_b > rec_b ? xs_b : rec_b);   // the records of the merge reuse the token rows
  if (L.kv_late) L.kv = L.wq;
  else { L.kv = off; off += kv_b; }
  L.qkv = off; off += sub_up16(mb * P * dkv * 4);
  // partial sums of the products; afterwards the merged head output and this rank's record
  const int ps_b = mb == 1 ? ((npr + 3) / 4) * 8 * 32 * 4 : 8 * 128 * 4, after_b = sub_up16(mb * dkv * 4) + sub_up16(mb * (dkv + SUB_RECPAD) * 4);
  L.psum = off; L.sa = off; L.recloc = off + sub_up16(mb * dkv * 4);
  off += sub_up16(ps_b > after_b ? ps_b : after_b);
  L.probs = off; off += sub_up16(mb * (kc + 4) * 4);
  L.bias = off; off += sub_up16(bias_len * 4);
  L.seed = off; off += sub_up16(mb * no * 4);
  L.red = off; off += sub_up16(SUB_THREADS * 16 + 64 * 4);   // single row: [key part][d_kv] weighted values, then the parts' sums
  L.loc = off; off += sub_up16(mb * npr * 4);
  L.out = off; off += mb == 1 ? 0 : sub_up16(SUB_MB * (no + 4) * 4);
  L.sh = off; off += sub_up16((int)sizeof(SubShared));
  L.total = off;
  return L;
}

// Chunk size, bias room and the key count up to which the ranks attend redundantly, for a cache of keys_cap keys.
// `all_keys` > 0 asks for a chunk that holds up to that many keys so that short caches need no second exchange; the
// chunk shrinks until the layout for passes of `mb` rows (1: the single-row kernel, SUB_MB: the block kernel; each has a plan
// of its own) stays under `prefer` bytes (half an SM), else under `limit`.
struct AttnSubPlan { int kc, bias_len, red_keys; bool ok; };
inline AttnSubPlan attn_sub_plan(int d, int dkv, int P, int C, int keys_cap, int all_keys, int prefer, int limit, int mb) {
  AttnSubPlan pl;
  const int per_rank = (keys_cap + C - 1) / C;
  const int need = std::min(64, sub_up16(per_rank)), want = std::min(128, sub_up16(std::min(all_keys, keys_cap)));
  auto blen = [&](int kc) { return P == 3 ? (std::max(per_rank, kc) + MAXB + 8 + 3) / 4 * 4 : 4; };
  auto fits = [&](int kc, int lim) {
    return attn_sub_layout(d, dkv, P, C, mb, kc, blen(kc)).total <= lim;
  };
  int kc = std::max(need, want);
  while (kc > need && !fits(kc, prefer)) kc -= 16;
  while (kc > 16 && !fits(kc, limit)) kc -= 16;
  pl.kc = kc; pl.bias_len = blen(kc); pl.ok = fits(kc, limit);
  pl.red_keys = all_keys > 0 ? kc : 0;
  return pl;
}

// ONE: a single token row (the small model's step, the large model's single-row pass): SIMT products, no loops over rows.
template <bool ONE>
__global__ void __launch_bounds__(SUB_THREADS) attn_sub_kernel(const AttnSubArgs a) {
  extern __shared__ __align__(1024) unsigned char sub_smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int C = a.C, d = a.d, dkv = a.dkv, P = a.self ? 3 : 1, R = P * dkv;
  const int h = blockIdx.x >> a.c_shift, r = (int)cluster_rank();
  const int pr0 = (r * R) >> a.c_shift, npr = (((r + 1) * R) >> a.c_shift) - pr0;   // rows of the head's q|k|v projection
  const int no = d >> a.c_shift, o0 = r * no;                                         // output rows of W_o
  const int rowbytes = d * 2 + SL_WPAD, xst = d + SL_XPAD, kvst = sub_kv_stride(dkv);
  const int vst = dkv + 4;   // row stride of the staged values: rows 2 t and channels g of a tensor-core tile hit 32 banks
  unsigned char* sWq = sub_smem + a.L.wq;
  float* Xs = reinterpret_cast<float*>(sub_smem + a.L.xs);
  float* rec = Xs;
  float* sK = reinterpret_cast<float*>(sub_smem + a.L.kv);
  float* sV = sK + (size_t)a.kc_keys * kvst;
  float* sQKV = reinterpret_cast<float*>(sub_smem + a.L.qkv);
  float* psum = reinterpret_cast<float*>(sub_smem + a.L.psum);
  float* sP = reinterpret_cast<float*>(sub_smem + a.L.probs);
  float* sBias = reinterpret_cast<float*>(sub_smem + a.L.bias);
  float* sSeed = reinterpret_cast<float*>(sub_smem + a.L.seed);
  float* sA = reinterpret_cast<float*>(sub_smem + a.L.sa);
  float* sRed = reinterpret_cast<float*>(sub_smem + a.L.red);
  float* recLoc = reinterpret_cast<float*>(sub_smem + a.L.recloc);
  float* sLoc = reinterpret_cast<float*>(sub_smem + a.L.loc);
  SubShared* sh = reinterpret_cast<SubShared*>(sub_smem + a.L.sh);
  const int pst = a.kc_keys + 4, recst = dkv + SUB_RECPAD;
  SUB_STAMP_BEGIN();

  if (tid == 0) {
    mbar_init(smem_u32(&sh->wbar), 1);
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect(smem_u32(&sh->wbar), (uint32_t)(npr * d * 2));
  }
  __syncthreads();
  SUB_STAMP();            // P0: barrier initialised
  pdl_launch_dependents();
  // weights depend on nothing: requested before the dependency wait.  Row i is copied by lane i / 8 of warp i % 8:
  // the copies a warp issues go out one after the other (about 25 ns each), the warps issue side by side
  {
    const int i = ((tid & 31) << 3) | (tid >> 5);
    if (i < npr && !a.skip_copies) {
      const int j = pr0 + i, part = j >> a.dkv_shift, ch = j & (dkv - 1);
      bulk_g2s(smem_u32(sWq + (size_t)i * rowbytes), a.Wp + ((size_t)part * a.I + h * dkv + ch) * d, (uint32_t)(d * 2), smem_u32(&sh->wbar));
    }
  }
  SUB_STAMP();            // P1: copies issued
  // output projection: warp w owns rows 16 w .. 16 w + 15 of this rank's share of W_o's column slice.  Thread (g, t) of the
  // warp keeps, of rows g and g + 8, the channels [t d_kv / 4, (t + 1) d_kv / 4), two per register: as it stands the left
  // operand of mma.sync m16n8k16 with the channels of a 16-channel step dealt out four to a thread
  const int og = lane >> 2, ot = lane & 3, cpt = dkv >> 2;
  uint32_t wr[2][8];
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
#pragma unroll
    for (int i = 0; i < 8; ++i) wr[rr][i] = 0u;
    if (warp * 16 < no) {
      const __nv_bfloat16* p = a.Wo + (size_t)(o0 + min(warp * 16 + og + 8 * rr, no - 1)) * a.I + h * dkv + ot * cpt;
      if (cpt == 4) {
        asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(wr[rr][0]), "=r"(wr[rr][1]) : "l"(p));
      } else {
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(wr[rr][0]), "=r"(wr[rr][1]), "=r"(wr[rr][2]), "=r"(wr[rr][3]) : "l"(p));
        if (cpt == 16)
          asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(wr[rr][4]), "=r"(wr[rr][5]), "=r"(wr[rr][6]), "=r"(wr[rr][7]) : "l"(p + 8));
      }
    }
  }
  float4 g4 = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid * 4 < d) g4 = __ldg(reinterpret_cast<const float4*>(a.gain) + tid);
  const float* Kh = a.kc + (size_t)h * a.cap * dkv;
  const float* Vh = a.vc + (size_t)h * a.cap * dkv;
  // stages keys / values [c0, c1) of the cache into sK / sV rows 0.. (asynchronous 16-byte copies)
  auto stage_cached = [&](int c0, int c1) {
    const int up_sh = a.dkv_shift - 2, units = (c1 - c0) << up_sh;
#pragma unroll 1
    for (int i = tid; i < units; i += SUB_THREADS) {
      const int jj = i >> up_sh, u = (i & ((1 << up_sh) - 1)) * 4;
      sub_cp16(sK + (size_t)jj * kvst + u, Kh + (size_t)(c0 + jj) * dkv + u);
      sub_cp16(sV + (size_t)jj * vst + u, Vh + (size_t)(c0 + jj) * dkv + u);
    }
  };
  // Few keys: every rank attends over all of them (the keys of the cache come from the L2, those of this pass from the
  // first exchange anyway), which costs a fraction of a microsecond and saves the exchange of the records and their merge.
  int n_keys = 0, j0 = 0, j1 = 0;
  bool red = false;
  if (!a.self) {   // the encoder keys are static: the first chunk is requested before the wait as well
    n_keys = min(*a.n_keys_dev, a.cap);
    red = n_keys <= a.red_keys;
    j0 = red ? 0 : (r * n_keys) >> a.c_shift; j1 = red ? n_keys : ((r + 1) * n_keys) >> a.c_shift;
    stage_cached(j0, min(j1, j0 + a.kc_keys));
    // a share of more than one chunk: the later chunks are asked into the L2 now (they are staged when the first is used up)
    const int later = (j1 - j0 - a.kc_keys) * (dkv >> 5);   // 128-byte lines of keys (as many again of values)
#pragma unroll 1
    for (int i = tid; i < later; i += SUB_THREADS) {
      const size_t o = (size_t)(j0 + a.kc_keys) * dkv + (size_t)i * 32;
      asm volatile("prefetch.global.L2 [%0];" ::"l"(Kh + o));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(Vh + o));
    }
  }
  // The call descriptor (row count, cache position) is written by kernels that have finished before the first kernel of a
  // pass starts -- the head of the pass before, or a set-up kernel in front of the embedding -- never by the kernel in
  // front of this one: it is read before the dependency wait, and with it the cached keys and values (rows below the
  // cache position, written by earlier passes; a second chunk of a block is launched only when the first chunk's rows
  // of this layer are complete) and the bias by distance.
  const int k = ONE ? 1 : min(a.desc->k, a.mb), pos0 = a.desc->pos0;
  if (a.self) {
    n_keys = min(pos0 + k, a.cap);
    red = n_keys <= a.red_keys;
    j0 = red ? 0 : (r * n_keys) >> a.c_shift; j1 = red ? n_keys : ((r + 1) * n_keys) >> a.c_shift;
    if (!a.L.kv_late) stage_cached(j0, min(min(j1, pos0), j0 + a.kc_keys));
  }
  // relative-position bias of the distances this rank meets
  const int dist_lo = max(0, pos0 - (j1 - 1));
  const int bias_cnt = a.self ? min(pos0 + k - j0 - dist_lo, a.bias_len) : 0;
#pragma unroll 1
  for (int i = tid; i < bias_cnt; i += SUB_THREADS) sBias[i] = __ldg(a.bias + (size_t)h * a.bias_ld + dist_lo + i);
  SubRows<ONE> rw;
  if (a.emb) sub_rows_embed<ONE>(a.emb, a.tokens, a.vocab, k, d, tid, rw);   // (tokens: part of the descriptor; the table: weights)
  SUB_STAMP();            // P2: loads issued, keys requested
  sub_cluster_arrive_relaxed();   // (0) this block is up: its shared memory may be written by the cluster
  SUB_STAMP();            // 0: prologue
  pdl_wait();
  SUB_STAMP();            // 1: dependency wait
  if (!a.emb) sub_rows_issue<ONE>(a.x_in, k, d, tid, rw);
  {   // clear the buffer the next kernel accumulates into
    const int n4 = k * (d >> 2);
#pragma unroll 1
    for (int i = blockIdx.x * SUB_THREADS + tid; i < n4; i += gridDim.x * SUB_THREADS)
      reinterpret_cast<float4*>(a.x_zero)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float inv1 = sub_rows_finish<ONE>(rw, k, d, g4, a.eps, Xs, xst, sh, sSeed, h == 0 ? o0 : 0, h == 0 ? o0 + no : 0, tid, lane, warp);
  SUB_STAMP();            // 2: token rows + norm
  sub_wait(sh, a.err, &sh->wbar, 0, a.spin);
  SUB_STAMP();            // 3: wait for the weights
  // ---- phase A: this rank's q|k|v rows for all token rows -----------------------------------
  if (ONE) sl_items<1>(sWq, rowbytes, npr, d, Xs, xst, psum, warp, lane);
  else sub_mma_split(sWq, rowbytes, npr, d, Xs, k, psum, warp, lane);
  __syncthreads();
  if (a.L.kv_late) stage_cached(j0, min(min(j1, pos0), j0 + a.kc_keys));   // the projection rows are done with: their place takes the keys
  SUB_STAMP();            // 4: q|k|v products
  sub_cluster_wait();     // (0) every block of the cluster is up
  if (ONE || (npr & 3) || (pr0 & 3)) {   // one (value, destination rank) pair per thread and turn
    const int tot = (npr * k) << a.c_shift;
#pragma unroll 1
    for (int idx = tid; idx < tot; idx += SUB_THREADS) {
      const int rk = idx & (C - 1), rest = idx >> a.c_shift, m = ONE ? 0 : rest / npr, i = rest - m * npr;
      const float v = sub_total<ONE>(psum, i, m, npr, d) * (ONE ? inv1 : sh->inv[m]);
      const int j = pr0 + i;
      st_cluster_f1(smem_u32(sQKV + (size_t)m * R + j), (uint32_t)rk, v);
      if (a.self && rk == r && j >= dkv && pos0 + m < a.cap)
        (j < 2 * dkv ? a.kc : a.vc)[((size_t)h * a.cap + pos0 + m) * dkv + (j & (dkv - 1))] = v;
    }
  } else {   // values first, then one 16-byte store per thread and turn
#pragma unroll 1
    for (int idx = tid; idx < npr * k; idx += SUB_THREADS) {
      const int m = idx / npr, i = idx - m * npr;
      const float v = sub_total<ONE>(psum, i, m, npr, d) * sh->inv[m];
      const int j = pr0 + i;
      sLoc[idx] = v;
      if (a.self && j >= dkv && pos0 + m < a.cap)
        (j < 2 * dkv ? a.kc : a.vc)[((size_t)h * a.cap + pos0 + m) * dkv + (j & (dkv - 1))] = v;
    }
    __syncthreads();
    const int n4 = npr >> 2, tot = (n4 * k) << a.c_shift;
#pragma unroll 1
    for (int idx = tid; idx < tot; idx += SUB_THREADS) {
      const int rk = idx & (C - 1), rest = idx >> a.c_shift, m = rest / n4, q = rest - m * n4;
      st_cluster_f4(smem_u32(sQKV + (size_t)m * R + pr0 + q * 4), (uint32_t)rk, *reinterpret_cast<const float4*>(sLoc + (size_t)m * npr + q * 4));
    }
  }
  SUB_STAMP();            // 5: exchange stores
  sub_cluster_arrive();   // (1) q, new keys and new values of the head are complete in every block
  sub_cluster_wait();
  SUB_STAMP();            // 6: cluster barrier 1
  // ---- phase B: attention of the k rows over the keys [j0, j1) ---------------------------------
  // single row, value phase: thread = (group of four channels, key part)
  const int cg4 = tid & ((dkv >> 2) - 1), part4 = tid >> (a.dkv_shift - 2), nparts4 = SUB_THREADS >> (a.dkv_shift - 2);
  float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
  const int dq4 = dkv >> 4;   // 16-byte units per channel quarter (d_kv <= 64)
  constexpr int RPP = ONE ? 1 : 2;   // rows per thread in the value phase (up to 8 rows over at least 4 parts)
  float acc[RPP], run1 = -INFINITY, lsum1 = 0.f;
#pragma unroll
  for (int i = 0; i < RPP; ++i) acc[i] = 0.f;
  if (!ONE && tid < MAXB) { sh->rmax[tid] = -INFINITY; sh->rsum[tid] = 0.f; sh->rscale[tid] = 1.f; }
#pragma unroll 1
  for (int c0 = j0; c0 < j1; c0 += a.kc_keys) {
    const int c1 = min(j1, c0 + a.kc_keys), nk = c1 - c0;
    if (c0 > j0) {   // later chunks: staged now (the first one is on its way since the prologue)
      __syncthreads();
      stage_cached(c0, a.self ? min(c1, pos0) : c1);
    }
    if (a.self) {   // keys of this pass come from the exchange buffer
      const int n0 = max(c0, pos0), cnt = (c1 - n0) << a.dkv_shift;
#pragma unroll 1
      for (int i = tid; i < cnt; i += SUB_THREADS) {
        const int jj = i >> a.dkv_shift, cc = i & (dkv - 1), mm = n0 + jj - pos0;
        sK[(size_t)(n0 + jj - c0) * kvst + cc] = sQKV[(size_t)mm * R + dkv + cc];
        sV[(size_t)(n0 + jj - c0) * vst + cc] = sQKV[(size_t)mm * R + 2 * dkv + cc];
      }
    }
    sub_cp_wait();
    __syncthreads();
    SUB_STAMP();          // B1: keys / values staged
    if (ONE) {   // scores: four threads per key, one channel quarter each (16-byte units interleaved over the quarters);
                 // two keys (64 apart) per thread and turn so that their loads are in flight together
      const int qt = tid & 3;
      const float* qp = sQKV;
#pragma unroll 1
      for (int j0b = 0; j0b < nk; j0b += SUB_THREADS / 2) {   // (the same trip count for every thread: the quads shuffle)
        const int jb = j0b + (tid >> 2), jc = jb + SUB_THREADS / 4;
        const bool va = jb < nk, vb = jc < nk;
        const float* pa = sK + (size_t)(va ? jb : 0) * kvst;
        const float* pb = sK + (size_t)(vb ? jc : 0) * kvst;
        float sa = 0.f, sb = 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (u < dq4) {
            const float4 q4 = *reinterpret_cast<const float4*>(qp + (u * 4 + qt) * 4);
            const float4 ka = *reinterpret_cast<const float4*>(pa + (u * 4 + qt) * 4);
            const float4 kb = *reinterpret_cast<const float4*>(pb + (u * 4 + qt) * 4);
            sa += q4.x * ka.x + q4.y * ka.y + q4.z * ka.z + q4.w * ka.w;
            sb += q4.x * kb.x + q4.y * kb.y + q4.z * kb.z + q4.w * kb.w;
          }
        sa += __shfl_xor_sync(0xffffffffu, sa, 1); sb += __shfl_xor_sync(0xffffffffu, sb, 1);
        sa += __shfl_xor_sync(0xffffffffu, sa, 2); sb += __shfl_xor_sync(0xffffffffu, sb, 2);
        if (qt == 0) {
          if (a.self) {   // (a single row sees every key up to its own position: all of them)
            if (va) sa += sBias[min(pos0 - (c0 + jb) - dist_lo, a.bias_len - 1)];
            if (vb) sb += sBias[min(pos0 - (c0 + jc) - dist_lo, a.bias_len - 1)];
          }
          if (va) sP[jb] = sa;
          if (vb) sP[jc] = sb;
        }
      }
    } else {
      // scores on mma.sync m16n8k16: 16 keys of the chunk are the rows of the left operand, the token rows the columns of
      // the right one, 16 channels per step; keys and queries each as a bf16 head and a bf16 remainder, three products kept.
      // Warp w takes the key tiles w, w + 8, ...
      const int g = lane >> 2, t = lane & 3;
#pragma unroll 1
      for (int t0 = warp * 16; t0 < nk; t0 += 16 * (SUB_THREADS / 32)) {
        float c0a = 0.f, c1a = 0.f, c2a = 0.f, c3a = 0.f, c0b = 0.f, c1b = 0.f, c2b = 0.f, c3b = 0.f, c0c = 0.f, c1c = 0.f, c2c = 0.f, c3c = 0.f;
        const float* ka = sK + (size_t)min(t0 + g, nk - 1) * kvst + 2 * t;
        const float* kb = sK + (size_t)min(t0 + g + 8, nk - 1) * kvst + 2 * t;
        const float* qp = sQKV + (size_t)min(g, k - 1) * R + 2 * t;
#pragma unroll
        for (int st = 0; st < 4; ++st)
          if (st * 16 < dkv) {
            const float2 a0 = *reinterpret_cast<const float2*>(ka + st * 16), a1 = *reinterpret_cast<const float2*>(kb + st * 16);
            const float2 a2 = *reinterpret_cast<const float2*>(ka + st * 16 + 8), a3 = *reinterpret_cast<const float2*>(kb + st * 16 + 8);
            float2 b0 = *reinterpret_cast<const float2*>(qp + st * 16), b1 = *reinterpret_cast<const float2*>(qp + st * 16 + 8);
            if (g >= k) { b0 = make_float2(0.f, 0.f); b1 = b0; }
            const uint32_t ah0 = sl_pack_bf16(a0.x, a0.y), ah1 = sl_pack_bf16(a1.x, a1.y), ah2 = sl_pack_bf16(a2.x, a2.y), ah3 = sl_pack_bf16(a3.x, a3.y);
            const uint32_t al0 = sl_pack_bf16(a0.x - __uint_as_float(ah0 << 16), a0.y - __uint_as_float(ah0 & 0xffff0000u));
            const uint32_t al1 = sl_pack_bf16(a1.x - __uint_as_float(ah1 << 16), a1.y - __uint_as_float(ah1 & 0xffff0000u));
            const uint32_t al2 = sl_pack_bf16(a2.x - __uint_as_float(ah2 << 16), a2.y - __uint_as_float(ah2 & 0xffff0000u));
            const uint32_t al3 = sl_pack_bf16(a3.x - __uint_as_float(ah3 << 16), a3.y - __uint_as_float(ah3 & 0xffff0000u));
            const uint32_t bh0 = sl_pack_bf16(b0.x, b0.y), bh1 = sl_pack_bf16(b1.x, b1.y);
            const uint32_t bl0 = sl_pack_bf16(b0.x - __uint_as_float(bh0 << 16), b0.y - __uint_as_float(bh0 & 0xffff0000u));
            const uint32_t bl1 = sl_pack_bf16(b1.x - __uint_as_float(bh1 << 16), b1.y - __uint_as_float(bh1 & 0xffff0000u));
#define SUB_MMA_S(C0, C1, C2, C3, A0, A1, A2, A3, B0, B1)                                                                        \
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};" \
                         : "+f"(C0), "+f"(C1), "+f"(C2), "+f"(C3) : "r"(A0), "r"(A1), "r"(A2), "r"(A3), "r"(B0), "r"(B1))
            SUB_MMA_S(c0a, c1a, c2a, c3a, ah0, ah1, ah2, ah3, bh0, bh1);
            SUB_MMA_S(c0b, c1b, c2b, c3b, al0, al1, al2, al3, bh0, bh1);
            SUB_MMA_S(c0c, c1c, c2c, c3c, ah0, ah1, ah2, ah3, bl0, bl1);
#undef SUB_MMA_S
          }
        // accumulators: keys t0 + g and t0 + g + 8, token rows 2 t and 2 t + 1
        const float cv[4] = {c0a + (c0b + c0c), c1a + (c1b + c1c), c2a + (c2b + c2c), c3a + (c3b + c3c)};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int jj = t0 + g + 8 * (i >> 1), m = 2 * t + (i & 1);
          if (jj < nk && m < k) {
            float sc = cv[i];
            if (a.self) {
              const int dist = pos0 + m - (c0 + jj);   // causal inside the block: row m sees keys up to its own position
              sc = dist >= 0 ? sc + sBias[min(dist - dist_lo, a.bias_len - 1)] : -INFINITY;
            }
            sP[(size_t)m * pst + jj] = sc;
          }
        }
      }
    }
    __syncthreads();
    SUB_STAMP();          // B2: scores
    if (ONE) {
      // every warp finds the chunk's maximum; thread (group of four channels, key part) then exponentiates and weighs its keys
      float mx = -INFINITY;
#pragma unroll 4
      for (int jj = lane; jj < nk; jj += 32) mx = fmaxf(mx, sP[jj]);   // (unrolled: the loads of a thread side by side)
      mx = warp_max(mx);
      const float nw = fmaxf(run1, mx), sc = run1 == -INFINITY ? 0.f : __expf(run1 - nw);
      float4 t4 = make_float4(acc4.x * sc, acc4.y * sc, acc4.z * sc, acc4.w * sc);
      float l = lsum1 * sc;
#pragma unroll 4
      for (int jj = part4; jj < nk; jj += nparts4) {
        const float p = __expf(sP[jj] - nw);
        const float4 v = *reinterpret_cast<const float4*>(sV + (size_t)jj * vst + cg4 * 4);
        l += p;
        t4.x += p * v.x; t4.y += p * v.y; t4.z += p * v.z; t4.w += p * v.w;
      }
      acc4 = t4; lsum1 = l; run1 = nw;
    } else {
      // running soft-max, one warp per row
#pragma unroll 1
      for (int m = warp; m < k; m += SUB_THREADS / 32) {
        float mx = -INFINITY;
        for (int jj = lane; jj < nk; jj += 32) mx = fmaxf(mx, sP[(size_t)m * pst + jj]);
        mx = warp_max(mx);
        const float old = sh->rmax[m], nw = fmaxf(old, mx);
        float sum = 0.f;
        for (int jj = lane; jj < ((nk + 15) & ~15); jj += 32) {   // (zeros up to the end of the last 16-key step)
          const float p = (jj >= nk || nw == -INFINITY) ? 0.f : __expf(sP[(size_t)m * pst + jj] - nw);
          sP[(size_t)m * pst + jj] = p;
          sum += p;
        }
        sum = warp_sum(sum);
        if (lane == 0) {
          const float sc = nw == -INFINITY ? 1.f : __expf(old - nw);
          sh->rscale[m] = sc;
          sh->rsum[m] = sh->rsum[m] * sc + sum;
          sh->rmax[m] = nw;
        }
      }
      __syncthreads();
      SUB_STAMP();        // B3: soft-max (block variant)
      // weighted values on mma.sync m16n8k16: out[row][channel] = sum_j p[row][j] v[j][channel]; the token rows are the
      // rows of the left operand (8..15 zero), warp w owns the channels 8 w .. 8 w + 7, 16 keys per step; probabilities
      // and values each as a bf16 head and a bf16 remainder, three products kept
      if (warp * 8 < dkv) {
        const int g = lane >> 2, t = lane & 3, n0 = warp * 8;
        const float rs = g < k ? sh->rscale[g] : 1.f;
        acc[0] *= rs; acc[1] *= rs;
        float c2 = 0.f, c3 = 0.f, d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;   // (d: the products with the remainders, a chain of their own)
        const uint32_t zero = 0u;
#pragma unroll 2
        for (int k0 = 0; k0 < nk; k0 += 16) {
          float2 p0 = make_float2(0.f, 0.f), p1 = p0;
          if (g < k) {
            p0 = *reinterpret_cast<const float2*>(sP + (size_t)g * pst + k0 + 2 * t);
            p1 = *reinterpret_cast<const float2*>(sP + (size_t)g * pst + k0 + 2 * t + 8);
          }
          const int ja = k0 + 2 * t;
          const float v00 = ja < nk ? sV[(size_t)ja * vst + n0 + g] : 0.f, v01 = ja + 1 < nk ? sV[(size_t)(ja + 1) * vst + n0 + g] : 0.f;
          const float v10 = ja + 8 < nk ? sV[(size_t)(ja + 8) * vst + n0 + g] : 0.f, v11 = ja + 9 < nk ? sV[(size_t)(ja + 9) * vst + n0 + g] : 0.f;
          const uint32_t ah0 = sl_pack_bf16(p0.x, p0.y), ah2 = sl_pack_bf16(p1.x, p1.y);
          const uint32_t al0 = sl_pack_bf16(p0.x - __uint_as_float(ah0 << 16), p0.y - __uint_as_float(ah0 & 0xffff0000u));
          const uint32_t al2 = sl_pack_bf16(p1.x - __uint_as_float(ah2 << 16), p1.y - __uint_as_float(ah2 & 0xffff0000u));
          const uint32_t bh0 = sl_pack_bf16(v00, v01), bh1 = sl_pack_bf16(v10, v11);
          const uint32_t bl0 = sl_pack_bf16(v00 - __uint_as_float(bh0 << 16), v01 - __uint_as_float(bh0 & 0xffff0000u));
          const uint32_t bl1 = sl_pack_bf16(v10 - __uint_as_float(bh1 << 16), v11 - __uint_as_float(bh1 & 0xffff0000u));
#define SUB_MMA(A0, A2, B0, B1)                                                                                                  \
          asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};" \
                       : "+f"(acc[0]), "+f"(acc[1]), "+f"(c2), "+f"(c3) : "r"(A0), "r"(zero), "r"(A2), "r"(zero), "r"(B0), "r"(B1))
          SUB_MMA(ah0, ah2, bh0, bh1);
          asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                       : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3) : "r"(al0), "r"(zero), "r"(al2), "r"(zero), "r"(bh0), "r"(bh1));
          asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                       : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3) : "r"(ah0), "r"(zero), "r"(ah2), "r"(zero), "r"(bl0), "r"(bl1));
#undef SUB_MMA
        }
        acc[0] += d0; acc[1] += d1;
      }
    }
  }
  // this rank's record (max, sum, weighted values per row), assembled locally
  if (ONE) {
    *reinterpret_cast<float4*>(sRed + (size_t)part4 * dkv + cg4 * 4) = acc4;
    if (cg4 == 0) sRed[SUB_THREADS * 4 + part4] = lsum1;
    __syncthreads();
    if (tid < dkv) {
      float t = 0.f;
#pragma unroll 16
      for (int p2 = 0; p2 < nparts4; ++p2) t += sRed[p2 * dkv + tid];
      recLoc[SUB_RECPAD + tid] = t;
    } else if (warp == SUB_THREADS / 32 - 1) {   // the parts' sums, added by one warp
      float l = 0.f;
      for (int p2 = lane; p2 < nparts4; p2 += 32) l += sRed[SUB_THREADS * 4 + p2];
      l = warp_sum(l);
      if (lane == 0) { recLoc[0] = run1; recLoc[1] = l; recLoc[2] = 0.f; recLoc[3] = 0.f; }
    }
  } else {
    if (warp * 8 < dkv && (lane >> 2) < k)   // accumulators of the tile: row lane / 4, channels 8 warp + 2 (lane % 4) (+ 1)
      *reinterpret_cast<float2*>(recLoc + (size_t)(lane >> 2) * recst + SUB_RECPAD + warp * 8 + 2 * (lane & 3)) = make_float2(acc[0], acc[1]);
    if (tid < k) { recLoc[(size_t)tid * recst] = sh->rmax[tid]; recLoc[(size_t)tid * recst + 1] = sh->rsum[tid]; }
  }
  __syncthreads();
  SUB_STAMP();            // 7: attention over this rank's keys
  if (red) {   // this rank's record covers every key: the head output is its values over its sum
#pragma unroll 1
    for (int o = tid; o < k * dkv; o += SUB_THREADS) {
      const int m = o >> a.dkv_shift, cc = o & (dkv - 1);
      sA[(size_t)m * dkv + cc] = recLoc[(size_t)m * recst + SUB_RECPAD + cc] / recLoc[(size_t)m * recst + 1];
    }
    SUB_STAMP(); SUB_STAMP(); SUB_STAMP();
  } else {
  {   // the record goes to every block of the cluster: one 16-byte store per thread and turn
    const int q4 = (k * recst) >> 2, tot = q4 << a.c_shift;
#pragma unroll 1
    for (int idx = tid; idx < tot; idx += SUB_THREADS) {
      const int rk = idx & (C - 1), q = idx >> a.c_shift;
      st_cluster_f4(smem_u32(rec + (size_t)r * a.mb * recst + q * 4), (uint32_t)rk, *reinterpret_cast<const float4*>(recLoc + q * 4));
    }
  }
  SUB_STAMP();            // 8: record stores
  sub_cluster_arrive();   // (2) all records are in place
  sub_cluster_wait();
  SUB_STAMP();            // 9: cluster barrier 2
  // ---- phase C: merge in rank order, then this rank's rows of the output projection ---------------
#pragma unroll 1
  for (int o = tid; o < k * dkv; o += SUB_THREADS) {
    const int m = o >> a.dkv_shift, cc = o & (dkv - 1);
    float mx[8], ls[8], av[8], gm = -INFINITY;   // the ranks' records are loaded side by side (C <= 8)
#pragma unroll
    for (int rk = 0; rk < 8; ++rk) {
      const float* rp = rec + ((size_t)min(rk, C - 1) * a.mb + m) * recst;
      const float2 ml = *reinterpret_cast<const float2*>(rp);
      mx[rk] = ml.x; ls[rk] = rk < C ? ml.y : 0.f; av[rk] = rp[SUB_RECPAD + cc];
    }
#pragma unroll
    for (int rk = 0; rk < 8; ++rk) gm = fmaxf(gm, mx[rk]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int rk = 0; rk < 8; ++rk) {   // fixed rank order
      const float w = ls[rk] > 0.f ? __expf(mx[rk] - gm) : 0.f;
      den += ls[rk] * w;
      num += (ls[rk] > 0.f ? av[rk] : 0.f) * w;
    }
    sA[(size_t)m * dkv + cc] = num / den;
  }
  SUB_STAMP();            // 10: merge
  }
  __syncthreads();
  if (ONE) {   // output projection, one row: the thread's channels of rows g and g + 8, then the four threads of a row add up
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const float* ap = sA + ot * cpt;
      float o = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (2 * i < cpt) o += __uint_as_float(wr[rr][i] << 16) * ap[2 * i] + __uint_as_float(wr[rr][i] & 0xffff0000u) * ap[2 * i + 1];
      o += __shfl_xor_sync(0xffffffffu, o, 1);
      o += __shfl_xor_sync(0xffffffffu, o, 2);
      const int row = warp * 16 + og + 8 * rr;
      if (ot == 0 && row < no) atomicAdd(a.x_out + o0 + row, h == 0 ? o + sSeed[row] : o);   // residual term once per column
    }
  } else {
    // output projection on mma.sync m16n8k16: rows of W_o x token rows (the right operand: the merged head output, each value
    // as a bf16 head and a bf16 remainder), 16 channels per step
    float* sOut = reinterpret_cast<float*>(sub_smem + a.L.out);
    const int ost = no + 4;
    if (warp * 16 < no) {
      float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f, e0 = 0.f, e1 = 0.f, e2 = 0.f, e3 = 0.f;   // (heads | remainders: two chains)
#pragma unroll
      for (int st = 0; st < 4; ++st)
        if (st * 16 < dkv) {
          float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
          if (og < k) b4 = *reinterpret_cast<const float4*>(sA + (size_t)og * dkv + ot * cpt + 4 * st);
          const uint32_t bh0 = sl_pack_bf16(b4.x, b4.y), bh1 = sl_pack_bf16(b4.z, b4.w);
          const uint32_t bl0 = sl_pack_bf16(b4.x - __uint_as_float(bh0 << 16), b4.y - __uint_as_float(bh0 & 0xffff0000u));
          const uint32_t bl1 = sl_pack_bf16(b4.z - __uint_as_float(bh1 << 16), b4.w - __uint_as_float(bh1 & 0xffff0000u));
          asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                       : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3)
                       : "r"(wr[0][2 * st]), "r"(wr[1][2 * st]), "r"(wr[0][2 * st + 1]), "r"(wr[1][2 * st + 1]), "r"(bh0), "r"(bh1));
          asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                       : "+f"(e0), "+f"(e1), "+f"(e2), "+f"(e3)
                       : "r"(wr[0][2 * st]), "r"(wr[1][2 * st]), "r"(wr[0][2 * st + 1]), "r"(wr[1][2 * st + 1]), "r"(bl0), "r"(bl1));
        }
      c0 += e0; c1 += e1; c2 += e2; c3 += e3;
      // accumulators: rows g and g + 8 of the tile, token rows 2 t and 2 t + 1
      const int row = warp * 16 + og;
      if (row < no) { sOut[(size_t)(2 * ot) * ost + row] = c0; sOut[(size_t)(2 * ot + 1) * ost + row] = c1; }
      if (row + 8 < no) { sOut[(size_t)(2 * ot) * ost + row + 8] = c2; sOut[(size_t)(2 * ot + 1) * ost + row + 8] = c3; }
    }
    __syncthreads();
    const int n4 = no >> 2;
#pragma unroll 1
    for (int idx = tid; idx < k * n4; idx += SUB_THREADS) {   // added four columns at a time
      const int m = idx / n4, q = idx - m * n4;
      float4 v = *reinterpret_cast<const float4*>(sOut + (size_t)m * ost + q * 4);
      if (h == 0) {   // residual term once per column
        const float4 xr = *reinterpret_cast<const float4*>(sSeed + (size_t)m * no + q * 4);
        v.x += xr.x; v.y += xr.y; v.z += xr.z; v.w += xr.w;
      }
      asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(a.x_out + (size_t)m * d + o0 + q * 4), "f"(v.x), "f"(v.y), "f"(v.z),
                   "f"(v.w) : "memory");
    }
  }
  SUB_STAMP();            // 11: output projection + reductions issued
  SUB_STAMP_END(a.self ? 0 : 1);
}

// ------------------------------------------------------------------------------------------------
// Feed-forward sub-layer
// ------------------------------------------------------------------------------------------------
// W_fo [d][F] in the order the feed-forward kernels load it, in units of 8 columns (16 bytes of a row).  Unit u holds
//   one: [i < 4][tid < d / 4]            the piece of row 4 tid + i                  (d pieces)
//   blk: [i][rr < 2][w < 8][g < 8]       the piece of row (w + 8 i) 16 + g + 8 rr    (pack_wfo_dpad(d) pieces, zero past d)
// so that the threads of a warp read neighbouring pieces.  Built once, when the context is created.
__host__ __device__ inline int pack_wfo_dpad(int d) { return (d + 127) / 128 * 128; }
__global__ void pack_wfo_kernel(const __nv_bfloat16* __restrict__ W, uint4* __restrict__ one, uint4* __restrict__ blk, int d, int F) {
  const int u = blockIdx.x, d4 = d >> 2, dpad = pack_wfo_dpad(d);
  for (int p = threadIdx.x; p < d; p += blockDim.x) {
    const int i = p / d4, tt = p - i * d4;
    one[(size_t)u * d + p] = *reinterpret_cast<const uint4*>(W + (size_t)(4 * tt + i) * F + 8 * u);
  }
  for (int p = threadIdx.x; p < dpad; p += blockDim.x) {
    const int g = p & 7, w = (p >> 3) & 7, rr = (p >> 6) & 1, i = p >> 7, n = (w + 8 * i) * 16 + g + 8 * rr;
    blk[(size_t)u * dpad + p] = n < d ? *reinterpret_cast<const uint4*>(W + (size_t)n * F + 8 * u) : make_uint4(0u, 0u, 0u, 0u);
  }
}

struct FfnSubLayout { int wi, xs, psum, u, seed, sh, total; };

struct FfnSubArgs {
  const CallDesc* desc;
  const float* x_in;
  float* x_out;
  float* x_zero;             // nullptr: nothing to clear (second part of a split launch)
  const float* gain;
  float eps;
  const __nv_bfloat16* Wi0;  // [F][d]
  const __nv_bfloat16* Wi1;  // [F][d] gate matrix (gated GELU) or nullptr
  const uint4* Wfo1;         // W_fo in the load order of the single-row variant (pack_wfo_kernel)
  const uint4* Wfo8;         // ... and of the block variant
  int d, F, gated;
  int part, nparts;          // this launch covers the slices blockIdx.x * nparts + part of gridDim.x * nparts
  int seed;                  // 1: the blocks add x_in for their share of the columns
  int mb;
  unsigned spin;             // polls of the weight barrier before the kernel gives up
  int* err;
  FfnSubLayout L;
};

// most rows of a slice when F (a multiple of 8) is dealt out in units of 8 rows
inline int ffn_sub_rows(int F, int slices) { return 8 * ((F / 8 + slices - 1) / slices); }
inline FfnSubLayout ffn_sub_layout(int d, int F, int gated, int slices, int grid, int mb) {
  FfnSubLayout L;
  const int nf = ffn_sub_rows(F, slices), nmat = gated ? 2 : 1;
  int off = 0;
  L.wi = off; off += sub_up16(nf * nmat * (d * 2 + SL_WPAD));
  L.xs = off; off += sub_up16(mb * (d + SL_XPAD) * 4);   // token rows; the block variant later collects its output tile here
  L.psum = off; off += mb == 1 ? SUB_PSUM : 8 * 128 * 4;
  L.u = off; off += sub_up16(mb * (SUB_FO_REGS + 4) * 4);
  L.seed = off; off += sub_up16(mb * 4 * ((d / 4 + grid - 1) / grid + 1) * 4);
  L.sh = off; off += sub_up16((int)sizeof(SubShared));
  L.total = off;
  return L;
}

template <bool ONE>
__global__ void __launch_bounds__(SUB_THREADS) ffn_sub_kernel(const FfnSubArgs a) {
  extern __shared__ __align__(1024) unsigned char sub_smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = a.d, F = a.F, G = gridDim.x, S = G * a.nparts, s = blockIdx.x * a.nparts + a.part;
  const int f0 = 8 * (int)(((long long)s * (F >> 3)) / S), f1 = 8 * (int)(((long long)(s + 1) * (F >> 3)) / S), nf = f1 - f0;
  const int nmat = a.gated ? 2 : 1, nrows = nf * nmat;
  const int rowbytes = d * 2 + SL_WPAD, xst = d + SL_XPAD;
  unsigned char* sWi = sub_smem + a.L.wi;
  float* Xs = reinterpret_cast<float*>(sub_smem + a.L.xs);
  float* psum = reinterpret_cast<float*>(sub_smem + a.L.psum);
  float* sU = reinterpret_cast<float*>(sub_smem + a.L.u);
  float* sSeed = reinterpret_cast<float*>(sub_smem + a.L.seed);
  SubShared* sh = reinterpret_cast<SubShared*>(sub_smem + a.L.sh);
  constexpr int ust = SUB_FO_REGS + 4;
  // columns whose residual term this block adds: units of four columns, spread over the grid
  const int d4 = d >> 2;
  const int su0 = a.seed ? (int)(((long long)blockIdx.x * d4) / G) : 0, su1 = a.seed ? (int)(((long long)(blockIdx.x + 1) * d4) / G) : 0;
  SUB_STAMP_BEGIN();

  if (tid == 0) {
    mbar_init(smem_u32(&sh->wbar), 1);
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect(smem_u32(&sh->wbar), (uint32_t)(nrows * d * 2));
  }
  __syncthreads();
  pdl_launch_dependents();
  {   // row i is copied by lane i / 8 of warp i % 8 (the copies of one warp are issued one after the other)
    const int i = ((tid & 31) << 3) | (tid >> 5);
    if (i < nrows) {
      const __nv_bfloat16* W = i < nf ? a.Wi0 : a.Wi1;
      const int rr = i < nf ? i : i - nf;
      bulk_g2s(smem_u32(sWi + (size_t)i * rowbytes), W + (size_t)(f0 + rr) * d, (uint32_t)(d * 2), smem_u32(&sh->wbar));
    }
  }
  // The block's columns [f0, f1) of W_fo stay in registers, 16 bytes (8 columns of a row) per load, from the copies of
  // W_fo that pack_wfo_kernel lays out so that the loads of a warp are contiguous (8 columns of a row in place are 16
  // bytes every 2 F bytes: a fraction of the memory's rate).  ONE: thread <-> the four output rows 4 tid .. 4 tid + 3,
  // chunk q = columns 8 q .. 8 q + 7.  Block variant: warp w owns the output tiles w, w + 8, ... (16 rows each); thread
  // (g, t) keeps, of rows g and g + 8 of a tile, the columns 8 t .. 8 t + 7: read as the left operand of mma.sync m16n8k16
  // they are two steps of 16 slice rows, with the slice rows dealt to the steps' positions so that one 16-byte load
  // fills them (the right operand, the hidden activations, follows the same order).
  uint4 wf[8][2];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 2; ++j) wf[i][j] = make_uint4(0u, 0u, 0u, 0u);
  if (ONE) {
    if (tid * 4 < d) {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (8 * q < nf) {
          const uint4* p = a.Wfo1 + (size_t)((f0 >> 3) + q) * d + tid;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4& w = wf[i * 2 + (q >> 1)][q & 1];
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "l"(p + i * (d >> 2)));
          }
        }
    }
  } else {
    const int g = lane >> 2, t = lane & 3;
    if (8 * t < nf) {
      const uint4* p = a.Wfo8 + (size_t)((f0 >> 3) + t) * pack_wfo_dpad(d) + warp * 8 + g;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if ((warp + 8 * i) * 16 < d) {
#pragma unroll
          for (int rr = 0; rr < 2; ++rr) {
            uint4& w = wf[i][rr];
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "l"(p + (i * 2 + rr) * 64));
          }
        }
    }
  }
  float4 g4 = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid * 4 < d) g4 = __ldg(reinterpret_cast<const float4*>(a.gain) + tid);
  const int k = ONE ? 1 : min(a.desc->k, a.mb);   // (written before the pass began: see the attention kernel)
  SUB_STAMP();            // 0: prologue
  pdl_wait();
  SUB_STAMP();            // 1: dependency wait
  SubRows<ONE> rw;
  sub_rows_issue<ONE>(a.x_in, k, d, tid, rw);
  if (a.x_zero) {
    const int n4 = k * d4;
#pragma unroll 1
    for (int i = blockIdx.x * SUB_THREADS + tid; i < n4; i += G * SUB_THREADS)
      reinterpret_cast<float4*>(a.x_zero)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float inv1 = sub_rows_finish<ONE>(rw, k, d, g4, a.eps, Xs, xst, sh, sSeed, su0 * 4, su1 * 4, tid, lane, warp);
  SUB_STAMP();            // 2: token rows + norm
  {
    if (nf > 0) sub_wait(sh, a.err, &sh->wbar, 0, a.spin);
    SUB_STAMP();          // 3: wait for the weights
    // hidden activations of the slice
    if (ONE) sl_items<1>(sWi, rowbytes, nrows, d, Xs, xst, psum, warp, lane);
    else sub_mma_split(sWi, rowbytes, nrows, d, Xs, k, psum, warp, lane);
    __syncthreads();   // (both product routines do nothing for a block without rows)
    if (ONE) {
      if (tid < nf) {
        const float v0 = sub_total<true>(psum, tid, 0, nrows, d) * inv1;
        sU[tid] = a.gated ? gelu_tanh(v0) * (sub_total<true>(psum, nf + tid, 0, nrows, d) * inv1) : fmaxf(v0, 0.f);
      }
    } else {   // thread <-> (token row, slice row) of the 8 x 32 tile the output products read; what lies outside is zero
      const int m = tid >> 5, i = tid & 31;
      float uv = 0.f;
      if (m < k && i < nf) {
        const float sc = sh->inv[m], v0 = sub_total<false>(psum, i, m, nrows, d) * sc;
        uv = a.gated ? gelu_tanh(v0) * (sub_total<false>(psum, nf + i, m, nrows, d) * sc) : fmaxf(v0, 0.f);
      }
      sU[(size_t)m * ust + i] = uv;
    }
    __syncthreads();
    SUB_STAMP();          // 4: hidden activations
  }
  if (ONE) {
    // this slice's share of all d outputs: thread <-> four output rows, their columns of W_fo from its registers
    if (tid < d4) {
      const bool seeds = tid >= su0 && tid < su1;
      float o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (8 * q < nf) {
          const float4 u0 = *reinterpret_cast<const float4*>(sU + 8 * q), u1 = *reinterpret_cast<const float4*>(sU + 8 * q + 4);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 w = wf[i * 2 + (q >> 1)][q & 1];
            o[i] += __uint_as_float(w.x << 16) * u0.x + __uint_as_float(w.x & 0xffff0000u) * u0.y + __uint_as_float(w.y << 16) * u0.z +
                    __uint_as_float(w.y & 0xffff0000u) * u0.w + __uint_as_float(w.z << 16) * u1.x + __uint_as_float(w.z & 0xffff0000u) * u1.y +
                    __uint_as_float(w.w << 16) * u1.z + __uint_as_float(w.w & 0xffff0000u) * u1.w;
          }
        }
      if (seeds) {
        const float4 xr = *reinterpret_cast<const float4*>(sSeed + (tid - su0) * 4);
        o[0] += xr.x; o[1] += xr.y; o[2] += xr.z; o[3] += xr.w;
      }
      if (nf > 0 || seeds)
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(a.x_out + tid * 4), "f"(o[0]), "f"(o[1]), "f"(o[2]), "f"(o[3]) : "memory");
    }
  } else {
    // out[column][token] = sum_i W_fo[column][f0 + i] * u[token][i] on mma.sync m16n8k16: 16 output columns are the rows of
    // the left operand (from the registers), the token rows the columns of the right one, each activation as a bf16 head and
    // a bf16 remainder.  Step s of thread (g, t) covers the slice rows 8 t + 4 s .. 8 t + 4 s + 3.
    const int g = lane >> 2, t = lane & 3;
    uint32_t bh[2][2], bl[2][2];
#pragma unroll
    for (int st = 0; st < 2; ++st) {
      const float4 u4 = *reinterpret_cast<const float4*>(sU + (size_t)g * ust + 8 * t + 4 * st);
      bh[st][0] = sl_pack_bf16(u4.x, u4.y); bh[st][1] = sl_pack_bf16(u4.z, u4.w);
      bl[st][0] = sl_pack_bf16(u4.x - __uint_as_float(bh[st][0] << 16), u4.y - __uint_as_float(bh[st][0] & 0xffff0000u));
      bl[st][1] = sl_pack_bf16(u4.z - __uint_as_float(bh[st][1] << 16), u4.w - __uint_as_float(bh[st][1] & 0xffff0000u));
    }
    float* sOut = Xs;   // [token][column], row stride xst: the token rows are done with
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int n0 = (warp + 8 * i) * 16;
      if (n0 < d) {
        float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
#define SUB_MMA(A0, A1, A2, A3, B0, B1)                                                                                          \
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};" \
                     : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3) : "r"(A0), "r"(A1), "r"(A2), "r"(A3), "r"(B0), "r"(B1))
        SUB_MMA(wf[i][0].x, wf[i][1].x, wf[i][0].y, wf[i][1].y, bh[0][0], bh[0][1]);
        SUB_MMA(wf[i][0].x, wf[i][1].x, wf[i][0].y, wf[i][1].y, bl[0][0], bl[0][1]);
        SUB_MMA(wf[i][0].z, wf[i][1].z, wf[i][0].w, wf[i][1].w, bh[1][0], bh[1][1]);
        SUB_MMA(wf[i][0].z, wf[i][1].z, wf[i][0].w, wf[i][1].w, bl[1][0], bl[1][1]);
#undef SUB_MMA
        // accumulators: columns n0 + g and n0 + g + 8, token rows 2 t and 2 t + 1
        sOut[(size_t)(2 * t) * xst + n0 + g] = c0; sOut[(size_t)(2 * t + 1) * xst + n0 + g] = c1;
        sOut[(size_t)(2 * t) * xst + n0 + g + 8] = c2; sOut[(size_t)(2 * t + 1) * xst + n0 + g + 8] = c3;
      }
    }
    __syncthreads();
#pragma unroll 1
    for (int idx = tid; idx < k * d4; idx += SUB_THREADS) {   // added four columns at a time
      const int m = idx / d4, un = idx - m * d4;
      const bool seeds = un >= su0 && un < su1;
      if (nf > 0 || seeds) {
        float4 v = *reinterpret_cast<const float4*>(sOut + (size_t)m * xst + un * 4);
        if (seeds) {
          const float4 xr = *reinterpret_cast<const float4*>(sSeed + (size_t)m * (su1 - su0) * 4 + (un - su0) * 4);
          v.x += xr.x; v.y += xr.y; v.z += xr.z; v.w += xr.w;
        }
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(a.x_out + (size_t)m * d + un * 4), "f"(v.x), "f"(v.y), "f"(v.z),
                     "f"(v.w) : "memory");
      }
    }
  }
  SUB_STAMP();            // 5: output products + reductions issued
  SUB_STAMP_END(2);
}

}  // namespace bild
