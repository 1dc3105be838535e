// Decoder sub-layers as ONE kernel each (bf16 weights, up to MAXB token rows), so that a layer
// of a decoder pass is three or four dependent kernels instead of eight:
//   * attn_sub_kernel: x_out = x_in + W_o * Attention(W_q|k|v * rms_norm(x_in))   (steps S1-S3 / L1-L3
//     for self-attention, S4-S6 / L4-L6 for cross-attention).  A cluster of C blocks owns one head:
//     rank r multiplies its share of the head's q|k|v rows (weights fetched by bulk copies BEFORE
//     the dependency wait of the programmatic launch), the cluster exchanges the k x 3 x d_kv results
//     through distributed shared memory, rank r then attends over its share of the keys, the
//     per-rank (max, sum, weighted values) records are exchanged the same way, and every rank
//     multiplies the merged head output with its share of the rows of W_o's column slice;
//   * ffn_sub_kernel: x_out = x_in + W_fo * act(W_i * rms_norm(x_in))   (S7-S8 / L7-L8).  Block b owns a
//     slice of d_ff: the rows of W_i (and of the gate matrix) and the matching rows of the transposed
//     W_fo, so the hidden activations never leave the block.
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
constexpr int SUB_FO_REGS = 32;              // rows of the transposed W_fo a single-row block keeps in registers

struct SubShared {
  unsigned long long wbar;
  float inv[MAXB];
  float ssq[8][MAXB];
  float rmax[MAXB], rsum[MAXB], rscale[MAXB];
  int failed;
};

// Optional cycle stamps of block 0 (build with -DBILD_STAMPS): summed per kernel kind and phase boundary.
#ifdef BILD_STAMPS
__device__ unsigned long long g_sub_stamps[4][24];
#define SUB_STAMP_BEGIN() long long st_t[20]; int st_n = 0; st_t[st_n++] = clock64()
#define SUB_STAMP() st_t[st_n++] = clock64()
#define SUB_STAMP_END(kind)                                                                                \
  if (blockIdx.x == 0 && threadIdx.x == 0) {                                                              \
    for (int i_ = 1; i_ < st_n; ++i_) atomicAdd(&g_sub_stamps[kind][i_ - 1], (unsigned long long)(st_t[i_] - st_t[i_ - 1])); \
    atomicAdd(&g_sub_stamps[kind][23], 1ull);                                                              \
  }
#else
#define SUB_STAMP_BEGIN()
#define SUB_STAMP()
#define SUB_STAMP_END(kind)
#endif

__host__ __device__ inline int sub_up16(int v) { return (v + 15) & ~15; }
// row stride (floats) of staged keys / values: 16 mod 32, so the four channel quarters of two keys hit 32 distinct banks
__host__ __device__ inline int sub_kv_stride(int dkv) { return ((dkv + 15) / 32) * 32 + 16; }

__device__ __forceinline__ void sub_wait(SubShared* sh, int* err, unsigned long long* bar, uint32_t parity) {
  const uint32_t b = smem_u32(bar);
  if (mbar_try(b, parity)) return;
  if (*(volatile int*)&sh->failed) return;
  for (unsigned it = 0; it < SPIN_LIMIT; ++it)
    if (mbar_try(b, parity)) return;
  sh->failed = 1;
  atomicExch(err, (int)BILD_ERR_TIMEOUT);
}

__device__ __forceinline__ void sub_cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void sub_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void sub_cp16(void* dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void sub_cp_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// dot product (weight row `row`, token row m) from the partial sums of sl_items<1> (ONE) or sl_mma<2>, added in warp order
template <bool ONE>
__device__ __forceinline__ float sub_total(const float* psum, int row, int m, int nrows, int K) {
  float t = 0.f;
  if (ONE) {
    const int nkb = (K + 255) >> 8, qd = row >> 2, first = qd * nkb;
    const float* p = psum + (size_t)(qd * 8) * 32 + (row & 3);
#pragma unroll
    for (int wv = 0; wv < 8; ++wv)
      if (((wv - first) & 7) < nkb) t += p[wv * 32];   // warp wv took part in this quad
  } else {   // fragment layout of the instruction: row = group (+ 8), token = 2 * (lane & 3) (+ 1); two tiles of 8 tokens
    const int MT = (nrows + 15) >> 4, ks_sh = MT == 1 ? 3 : MT == 2 ? 2 : 1;
    const int mt = row >> 4, rr = row & 15, col = m & 7;
    const float* p = psum + ((size_t)((mt << ks_sh) * 2 + (m >> 3)) * 32 + (rr & 7) * 4 + (col >> 1)) * 4 + (rr >> 3) * 2 + (col & 1);
#pragma unroll 1
    for (int ks = 0; ks < (1 << ks_sh); ++ks) t += p[(size_t)ks * 256];
  }
  return t;
}

// Token rows, after the dependency wait (d <= 1024: one 128-bit load per thread and row, all rows of a turn in
// flight together): x * gain into Xs, 1 / rms into sh->inv (returned for the single row of ONE).  The raw values of the
// columns [seed0, seed1) (multiples of 4) also go to sSeed[m][column - seed0]: the residual term the block adds.
template <bool ONE>
__device__ __forceinline__ float sub_load_rows(const float* __restrict__ x_in, int k, int d, float4 g, float eps, float* Xs, int xst,
                                               SubShared* sh, float* sSeed, int seed0, int seed1, int tid, int lane, int warp) {
  const int d4 = d >> 2, c = tid * 4;
  const bool on = tid < d4, sd = c >= seed0 && c < seed1;
  if (ONE) {
    float ss = 0.f;
    if (on) {
      float4 w = __ldcg(reinterpret_cast<const float4*>(x_in) + tid);
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
  }
#pragma unroll 1
  for (int m0 = 0; m0 < k; m0 += 8) {
    float4 v[8];
    float q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (on && m0 + i < k) v[i] = __ldcg(reinterpret_cast<const float4*>(x_in + (size_t)(m0 + i) * d) + tid);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      q[i] = 0.f;
      if (on && m0 + i < k) {
        float4 w = v[i];
        q[i] = w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
        if (sd) *reinterpret_cast<float4*>(sSeed + (size_t)(m0 + i) * (seed1 - seed0) + (c - seed0)) = w;
        w.x *= g.x; w.y *= g.y; w.z *= g.z; w.w *= g.w;
        *reinterpret_cast<float4*>(Xs + (size_t)(m0 + i) * xst + c) = w;
      }
    }
    const float r8 = treduce<8>(q, lane);   // lanes 4 i hold the warp's sum of row m0 + i
    if ((lane & 3) == 0) sh->ssq[warp][m0 + (lane >> 2)] = r8;
  }
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

// ------------------------------------------------------------------------------------------------
// Attention sub-layer
// ------------------------------------------------------------------------------------------------
struct AttnSubLayout { int wq, wo, xs, kv, qkv, psum, probs, bias, seed, sa, red, recloc, sh, total; };

struct AttnSubArgs {
  const CallDesc* desc;
  const float* x_in;    // [MAXB][d] residual stream (complete)
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
  int kc_keys;               // keys per staged chunk (<= 64)
  int bias_len;              // floats reserved for the staged bias
  int mb;                    // token rows the shared memory is sized for
  int* err;
  AttnSubLayout L;
};

inline AttnSubLayout attn_sub_layout(int d, int dkv, int P, int C, int mb, int kc, int bias_len) {
  AttnSubLayout L;
  const int npr = (P * dkv + C - 1) / C, no = (d + C - 1) / C;
  int off = 0;
  L.wq = off; off += sub_up16(npr * (d * 2 + SL_WPAD));
  L.wo = off;   // (the rows of W_o live in registers)
  (void)no;
  const int xs_b = mb * (d + SL_XPAD) * 4, rec_b = C * mb * (dkv + SUB_RECPAD) * 4;
  L.xs = off; off += sub_up16(xs_b > rec_b ? xs_b : rec_b);   // the records of the merge reuse the token rows
  L.kv = off; off += sub_up16(2 * kc * sub_kv_stride(dkv) * 4);
  L.qkv = off; off += sub_up16(mb * P * dkv * 4);
  L.psum = off; off += SUB_PSUM;
  L.probs = off; off += sub_up16(mb * (kc + 4) * 4);
  L.bias = off; off += sub_up16(bias_len * 4);
  L.seed = off; off += sub_up16(mb * no * 4);
  L.sa = off; off += sub_up16(mb * dkv * 4);
  L.red = off; off += sub_up16(SUB_THREADS * 4 + 64);
  L.recloc = off; off += sub_up16(mb * (dkv + SUB_RECPAD) * 4);
  L.sh = off; off += sub_up16((int)sizeof(SubShared));
  L.total = off;
  return L;
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
    if (i < npr) {
      const int j = pr0 + i, part = j >> a.dkv_shift, ch = j & (dkv - 1);
      bulk_g2s(smem_u32(sWq + (size_t)i * rowbytes), a.Wp + ((size_t)part * a.I + h * dkv + ch) * d, (uint32_t)(d * 2), smem_u32(&sh->wbar));
    }
  }
  SUB_STAMP();            // P1: copies issued
  // output projection: two threads per row of this rank's share of W_o's column slice, half of the channels each, in registers
  const int oi = tid >> 1, ohf = tid & 1, hc = dkv >> 1;
  uint4 wo[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    wo[u] = make_uint4(0u, 0u, 0u, 0u);
    if (oi < no && u * 8 < hc) {
      const __nv_bfloat16* p = a.Wo + (size_t)(o0 + oi) * a.I + h * dkv + ohf * hc + u * 8;
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(wo[u].x), "=r"(wo[u].y), "=r"(wo[u].z), "=r"(wo[u].w) : "l"(p));
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
      sub_cp16(sV + (size_t)jj * kvst + u, Vh + (size_t)(c0 + jj) * dkv + u);
    }
  };
  int n_keys = 0, j0 = 0, j1 = 0;
  if (!a.self) {   // the encoder keys are static: the first chunk is requested before the wait as well
    n_keys = min(*a.n_keys_dev, a.cap);
    j0 = (r * n_keys) >> a.c_shift; j1 = ((r + 1) * n_keys) >> a.c_shift;
    stage_cached(j0, min(j1, j0 + a.kc_keys));
  }
  SUB_STAMP();            // P2: loads issued, cross keys requested
  sub_cluster_arrive();   // (0) this block is up: its shared memory may be written by the cluster
  SUB_STAMP();            // 0: prologue
  pdl_wait();
  SUB_STAMP();            // 1: dependency wait
  const int k = ONE ? 1 : min(a.desc->k, a.mb), pos0 = a.desc->pos0;
  if (a.self) {
    n_keys = min(pos0 + k, a.cap);
    j0 = (r * n_keys) >> a.c_shift; j1 = ((r + 1) * n_keys) >> a.c_shift;
    stage_cached(j0, min(min(j1, pos0), j0 + a.kc_keys));
  }
  // relative-position bias of the distances this rank meets
  const int dist_lo = max(0, pos0 - (j1 - 1));
  if (a.self) {
    const int cnt = min(pos0 + k - j0 - dist_lo, a.bias_len);
#pragma unroll 1
    for (int i = tid; i < cnt; i += SUB_THREADS) sBias[i] = __ldg(a.bias + (size_t)h * a.bias_ld + dist_lo + i);
  }
  {   // clear the buffer the next kernel accumulates into
    const int n4 = k * (d >> 2);
#pragma unroll 1
    for (int i = blockIdx.x * SUB_THREADS + tid; i < n4; i += gridDim.x * SUB_THREADS)
      reinterpret_cast<float4*>(a.x_zero)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float inv1 = sub_load_rows<ONE>(a.x_in, k, d, g4, a.eps, Xs, xst, sh, sSeed, h == 0 ? o0 : 0, h == 0 ? o0 + no : 0, tid, lane, warp);
  SUB_STAMP();            // 2: token rows + norm
  sub_wait(sh, a.err, &sh->wbar, 0);
  SUB_STAMP();            // 3: wait for the weights
  // ---- phase A: this rank's q|k|v rows for all token rows -----------------------------------
  if (ONE) sl_items<1>(sWq, rowbytes, npr, d, Xs, xst, psum, warp, lane);
  else sl_mma<2>(sWq, rowbytes, npr, d, Xs, xst, k, psum, warp, lane);
  __syncthreads();
  SUB_STAMP();            // 4: q|k|v products
  sub_cluster_wait();     // (0) every block of the cluster is up
  {   // one (value, destination rank) pair per thread and turn
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
  }
  SUB_STAMP();            // 5: exchange stores
  sub_cluster_arrive();   // (1) q, new keys and new values of the head are complete in every block
  sub_cluster_wait();
  SUB_STAMP();            // 6: cluster barrier 1
  // ---- phase B: attention of the k rows over the keys [j0, j1) ---------------------------------
  const int ch = tid & (dkv - 1), part = tid >> a.dkv_shift, nparts = SUB_THREADS >> a.dkv_shift;
  const int dq4 = dkv >> 4;   // 16-byte units per channel quarter (d_kv <= 64)
  constexpr int RPP = ONE ? 1 : 8;   // rows per thread in the value phase
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
        sV[(size_t)(n0 + jj - c0) * kvst + cc] = sQKV[(size_t)mm * R + 2 * dkv + cc];
      }
    }
    sub_cp_wait();
    __syncthreads();
    {   // scores: four threads per key, one channel quarter each (16-byte units interleaved over the quarters); the
        // quarter of the key stays in registers while the rows go by
      const int jj = tid >> 2, qt = tid & 3;
      const bool valid = jj < nk;
      float4 kq[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (valid && u < dq4) kq[u] = *reinterpret_cast<const float4*>(sK + (size_t)jj * kvst + (u * 4 + qt) * 4);
#pragma unroll 1
      for (int m = 0; m < k; ++m) {
        float s = 0.f;
        if (valid) {
          const float* qp = sQKV + (size_t)m * R;
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (u < dq4) {
              const float4 q4 = *reinterpret_cast<const float4*>(qp + (u * 4 + qt) * 4);
              s += q4.x * kq[u].x + q4.y * kq[u].y + q4.z * kq[u].z + q4.w * kq[u].w;
            }
        }
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        if (valid && qt == 0) {
          if (a.self) {
            const int dist = pos0 + m - (c0 + jj);   // causal inside the block: row m sees keys up to its own position
            s = dist >= 0 ? s + sBias[min(dist - dist_lo, a.bias_len - 1)] : -INFINITY;
          }
          sP[(size_t)m * pst + jj] = s;
        }
      }
    }
    __syncthreads();
    if (ONE) {
      // every warp finds the chunk's maximum; thread (channel, key part) then exponentiates and weighs its keys
      float mx = -INFINITY;
      for (int jj = lane; jj < nk; jj += 32) mx = fmaxf(mx, sP[jj]);
      mx = warp_max(mx);
      const float nw = fmaxf(run1, mx), sc = run1 == -INFINITY ? 0.f : __expf(run1 - nw);
      float t = acc[0] * sc, l = lsum1 * sc;
#pragma unroll 4
      for (int jj = part; jj < nk; jj += nparts) {
        const float p = __expf(sP[jj] - nw);
        l += p;
        t += p * sV[(size_t)jj * kvst + ch];
      }
      acc[0] = t; lsum1 = l; run1 = nw;
    } else {
      // running soft-max, one warp per row
#pragma unroll 1
      for (int m = warp; m < k; m += SUB_THREADS / 32) {
        float mx = -INFINITY;
        for (int jj = lane; jj < nk; jj += 32) mx = fmaxf(mx, sP[(size_t)m * pst + jj]);
        mx = warp_max(mx);
        const float old = sh->rmax[m], nw = fmaxf(old, mx);
        float sum = 0.f;
        for (int jj = lane; jj < nk; jj += 32) {
          const float p = nw == -INFINITY ? 0.f : __expf(sP[(size_t)m * pst + jj] - nw);
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
      // weighted values: thread (channel, part) takes the rows part, part + nparts, ...; a value is read once for all of them
#pragma unroll
      for (int i = 0; i < RPP; ++i)
        if (part + i * nparts < k) acc[i] *= sh->rscale[part + i * nparts];
#pragma unroll 1
      for (int jj = 0; jj < nk; ++jj) {
        const float v = sV[(size_t)jj * kvst + ch];
#pragma unroll
        for (int i = 0; i < RPP; ++i)
          if (part + i * nparts < k) acc[i] += sP[(size_t)(part + i * nparts) * pst + jj] * v;
      }
    }
  }
  // this rank's record (max, sum, weighted values per row), assembled locally
  if (ONE) {
    sRed[part * dkv + ch] = acc[0];
    if (ch == 0) sRed[SUB_THREADS + part] = lsum1;
    __syncthreads();
    if (tid < dkv) {
      float t = 0.f;
      for (int p2 = 0; p2 < nparts; ++p2) t += sRed[p2 * dkv + tid];
      recLoc[SUB_RECPAD + tid] = t;
    }
    if (tid == 0) {
      float l = 0.f;
      for (int p2 = 0; p2 < nparts; ++p2) l += sRed[SUB_THREADS + p2];
      recLoc[0] = run1; recLoc[1] = l; recLoc[2] = 0.f; recLoc[3] = 0.f;
    }
  } else {
#pragma unroll
    for (int i = 0; i < RPP; ++i)
      if (part + i * nparts < k) recLoc[(size_t)(part + i * nparts) * recst + SUB_RECPAD + ch] = acc[i];
    if (tid < k) { recLoc[(size_t)tid * recst] = sh->rmax[tid]; recLoc[(size_t)tid * recst + 1] = sh->rsum[tid]; }
  }
  __syncthreads();
  SUB_STAMP();            // 7: attention over this rank's keys
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
  __syncthreads();
  SUB_STAMP();            // 10: merge
  {   // output projection: the row half in this thread's registers times the head's merged output, row after row
    float wf[32];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      wf[u * 8 + 0] = __uint_as_float(wo[u].x << 16); wf[u * 8 + 1] = __uint_as_float(wo[u].x & 0xffff0000u);
      wf[u * 8 + 2] = __uint_as_float(wo[u].y << 16); wf[u * 8 + 3] = __uint_as_float(wo[u].y & 0xffff0000u);
      wf[u * 8 + 4] = __uint_as_float(wo[u].z << 16); wf[u * 8 + 5] = __uint_as_float(wo[u].z & 0xffff0000u);
      wf[u * 8 + 6] = __uint_as_float(wo[u].w << 16); wf[u * 8 + 7] = __uint_as_float(wo[u].w & 0xffff0000u);
    }
#pragma unroll 1
    for (int m = 0; m < k; ++m) {
      const float* ap = sA + (size_t)m * dkv + ohf * hc;
      float o = 0.f;
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (u * 8 < hc) {
          const float4 a0 = *reinterpret_cast<const float4*>(ap + u * 8), a1 = *reinterpret_cast<const float4*>(ap + u * 8 + 4);
          o += wf[u * 8] * a0.x + wf[u * 8 + 1] * a0.y + wf[u * 8 + 2] * a0.z + wf[u * 8 + 3] * a0.w + wf[u * 8 + 4] * a1.x +
               wf[u * 8 + 5] * a1.y + wf[u * 8 + 6] * a1.z + wf[u * 8 + 7] * a1.w;
        }
      o += __shfl_xor_sync(0xffffffffu, o, 1);
      if (oi < no && ohf == 0) atomicAdd(a.x_out + (size_t)m * d + o0 + oi, h == 0 ? o + sSeed[(size_t)m * no + oi] : o);   // residual term once per column
    }
  }
  SUB_STAMP();            // 11: output projection + reductions issued
  SUB_STAMP_END(a.self ? 0 : 1);
}

// ------------------------------------------------------------------------------------------------
// Feed-forward sub-layer
// ------------------------------------------------------------------------------------------------
struct FfnSubLayout { int wi, wfo, xs, psum, u, seed, sh, total; };

struct FfnSubArgs {
  const CallDesc* desc;
  const float* x_in;
  float* x_out;
  float* x_zero;             // nullptr: nothing to clear (second part of a split launch)
  const float* gain;
  float eps;
  const __nv_bfloat16* Wi0;  // [F][d]
  const __nv_bfloat16* Wi1;  // [F][d] gate matrix (gated GELU) or nullptr
  const __nv_bfloat16* WfoT; // [F][d]: W_fo transposed
  int d, F, gated;
  int part, nparts;          // this launch covers the slices blockIdx.x * nparts + part of gridDim.x * nparts
  int seed;                  // 1: the blocks add x_in for their share of the columns
  int mb;
  int* err;
  FfnSubLayout L;
};

inline int ffn_sub_rows(int F, int slices) { return (F + slices - 1) / slices; }
inline FfnSubLayout ffn_sub_layout(int d, int F, int gated, int slices, int grid, int mb) {
  FfnSubLayout L;
  const int nf = ffn_sub_rows(F, slices), nmat = gated ? 2 : 1;
  int off = 0;
  L.wi = off; off += sub_up16(nf * nmat * (d * 2 + SL_WPAD));
  L.wfo = off; off += mb == 1 ? 0 : sub_up16(nf * d * 2);   // (a single-row block keeps these rows in registers)
  L.xs = off; off += sub_up16(mb * (d + SL_XPAD) * 4);
  L.psum = off; off += SUB_PSUM;
  L.u = off; off += sub_up16(mb * (nf + 1) * 4);
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
  const int f0 = (int)(((long long)s * F) / S), f1 = (int)(((long long)(s + 1) * F) / S), nf = f1 - f0;
  const int nmat = a.gated ? 2 : 1, nrows = nf * nmat;
  const int rowbytes = d * 2 + SL_WPAD, xst = d + SL_XPAD;
  unsigned char* sWi = sub_smem + a.L.wi;
  const unsigned char* sWfo = sub_smem + a.L.wfo;
  float* Xs = reinterpret_cast<float*>(sub_smem + a.L.xs);
  float* psum = reinterpret_cast<float*>(sub_smem + a.L.psum);
  float* sU = reinterpret_cast<float*>(sub_smem + a.L.u);
  float* sSeed = reinterpret_cast<float*>(sub_smem + a.L.seed);
  SubShared* sh = reinterpret_cast<SubShared*>(sub_smem + a.L.sh);
  const int ust = (F + S - 1) / S + 1;
  // columns whose residual term this block adds: units of four columns, spread over the grid
  const int d4 = d >> 2;
  const int su0 = a.seed ? (int)(((long long)blockIdx.x * d4) / G) : 0, su1 = a.seed ? (int)(((long long)(blockIdx.x + 1) * d4) / G) : 0;
  SUB_STAMP_BEGIN();

  if (tid == 0) {
    mbar_init(smem_u32(&sh->wbar), 1);
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect(smem_u32(&sh->wbar), (uint32_t)((nrows + (ONE ? 0 : nf)) * d * 2));
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
  // the slice of the transposed W_fo: ONE keeps it in registers (thread <-> four columns of every row), else one bulk copy
  constexpr int NFR = ONE ? SUB_FO_REGS : 1;
  uint2 wfr[NFR];
  if (ONE) {
#pragma unroll
    for (int i = 0; i < NFR; ++i) {
      wfr[i] = make_uint2(0u, 0u);
      if (i < nf && tid * 4 < d) {
        const __nv_bfloat16* p = a.WfoT + (size_t)(f0 + i) * d + tid * 4;
        asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(wfr[i].x), "=r"(wfr[i].y) : "l"(p));
      }
    }
  } else if (tid == SUB_THREADS - 1 && nf > 0) {
    bulk_g2s(smem_u32(sWfo), a.WfoT + (size_t)f0 * d, (uint32_t)(nf * d * 2), smem_u32(&sh->wbar));
  }
  float4 g4 = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid * 4 < d) g4 = __ldg(reinterpret_cast<const float4*>(a.gain) + tid);
  SUB_STAMP();            // 0: prologue
  pdl_wait();
  SUB_STAMP();            // 1: dependency wait
  const int k = ONE ? 1 : min(a.desc->k, a.mb);
  if (a.x_zero) {
    const int n4 = k * d4;
#pragma unroll 1
    for (int i = blockIdx.x * SUB_THREADS + tid; i < n4; i += G * SUB_THREADS)
      reinterpret_cast<float4*>(a.x_zero)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float inv1 = sub_load_rows<ONE>(a.x_in, k, d, g4, a.eps, Xs, xst, sh, sSeed, su0 * 4, su1 * 4, tid, lane, warp);
  SUB_STAMP();            // 2: token rows + norm
  if (nf > 0) {
    sub_wait(sh, a.err, &sh->wbar, 0);
    SUB_STAMP();          // 3: wait for the weights
    // hidden activations of the slice
    if (ONE) sl_items<1>(sWi, rowbytes, nrows, d, Xs, xst, psum, warp, lane);
    else sl_mma<2>(sWi, rowbytes, nrows, d, Xs, xst, k, psum, warp, lane);
    __syncthreads();
#pragma unroll 1
    for (int idx = tid; idx < nf * k; idx += SUB_THREADS) {
      const int m = ONE ? 0 : idx / nf, i = idx - m * nf;
      const float sc = ONE ? inv1 : sh->inv[m];
      const float v0 = sub_total<ONE>(psum, i, m, nrows, d) * sc;
      sU[(size_t)m * ust + i] = a.gated ? gelu_tanh(v0) * (sub_total<ONE>(psum, nf + i, m, nrows, d) * sc) : fmaxf(v0, 0.f);
    }
    __syncthreads();
    SUB_STAMP();          // 4: hidden activations
  }
  // this slice's share of all d outputs: thread <-> four columns, up to eight token rows per turn
  constexpr int TB = ONE ? 1 : 8;
  if (tid < d4) {
    const bool seeds = tid >= su0 && tid < su1;
#pragma unroll 1
    for (int m0 = 0; m0 < k; m0 += TB) {
      float o[TB][4];
#pragma unroll
      for (int j = 0; j < TB; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
      if (ONE) {
#pragma unroll
        for (int i = 0; i < NFR; ++i) {   // (rows past the slice hold zeros)
          const float uv = i < nf ? sU[i] : 0.f;
          o[0][0] += __uint_as_float(wfr[i].x << 16) * uv; o[0][1] += __uint_as_float(wfr[i].x & 0xffff0000u) * uv;
          o[0][2] += __uint_as_float(wfr[i].y << 16) * uv; o[0][3] += __uint_as_float(wfr[i].y & 0xffff0000u) * uv;
        }
      } else
#pragma unroll 2
      for (int i = 0; i < nf; ++i) {
        const uint2 w = *reinterpret_cast<const uint2*>(sWfo + ((size_t)i * d + tid * 4) * 2);
        const float w0 = __uint_as_float(w.x << 16), w1 = __uint_as_float(w.x & 0xffff0000u);
        const float w2 = __uint_as_float(w.y << 16), w3 = __uint_as_float(w.y & 0xffff0000u);
#pragma unroll
        for (int j = 0; j < TB; ++j)
          if (m0 + j < k) {
            const float uv = sU[(size_t)(m0 + j) * ust + i];
            o[j][0] += w0 * uv; o[j][1] += w1 * uv; o[j][2] += w2 * uv; o[j][3] += w3 * uv;
          }
      }
#pragma unroll
      for (int j = 0; j < TB; ++j) {
        const int m = m0 + j;
        if (m < k) {
          if (seeds) {
            const float4 xr = *reinterpret_cast<const float4*>(sSeed + (size_t)m * (su1 - su0) * 4 + (tid - su0) * 4);
            o[j][0] += xr.x; o[j][1] += xr.y; o[j][2] += xr.z; o[j][3] += xr.w;
          }
          if (nf > 0 || seeds)
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(a.x_out + (size_t)m * d + tid * 4), "f"(o[j][0]), "f"(o[j][1]),
                         "f"(o[j][2]), "f"(o[j][3]) : "memory");
        }
      }
    }
  }
  SUB_STAMP();            // 5: output products + reductions issued
  SUB_STAMP_END(2);
}

// W_fo [d][F] -> [F][d] (once, when the context is created)
__global__ void transpose_bf16_kernel(const __nv_bfloat16* __restrict__ in, __nv_bfloat16* __restrict__ out, int rows, int cols) {
  __shared__ __nv_bfloat16 tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int r = r0 + i, c = c0 + threadIdx.x;
    if (r < rows && c < cols) tile[i][threadIdx.x] = in[(size_t)r * cols + c];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int c = c0 + i, r = r0 + threadIdx.x;
    if (r < rows && c < cols) out[(size_t)c * rows + r] = tile[threadIdx.x][i];
  }
}

}  // namespace bild
