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
constexpr int SUB_HALF_SM = 113 * 1024;      // shared memory of a block that leaves room for a second one on the SM
constexpr int SUB_MB = 8;                    // token rows of the block variant (one 8-token tile of the tensor-core instruction)

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
  {
    float4 v[SUB_MB];
    float q[SUB_MB];
#pragma unroll
    for (int i = 0; i < SUB_MB; ++i)
      if (on && i < k) v[i] = __ldcg(reinterpret_cast<const float4*>(x_in + (size_t)i * d) + tid);
#pragma unroll
    for (int i = 0; i < SUB_MB; ++i) {
      q[i] = 0.f;
      if (on && i < k) {
        float4 w = v[i];
        q[i] = w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
        if (sd) *reinterpret_cast<float4*>(sSeed + (size_t)i * (seed1 - seed0) + (c - seed0)) = w;
        w.x *= g.x; w.y *= g.y; w.z *= g.z; w.w *= g.w;
        *reinterpret_cast<float4*>(Xs + (size_t)i * xst + c) = w;
      }
    }
    const float r8 = treduce<8>(q, lane);   // lanes 4 i hold the warp's sum of row i
    if ((lane & 3) == 0) sh->ssq[warp][lane >> 2] = r8;
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
struct AttnSubLayout { int wq, xs, kv, kv_late, qkv, psum, probs, bias, seed, sa, red, recloc, loc, out, sh, total; };

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
  L.red = off; off += sub_up16(SUB_THREADS * 4 + 64);
  L.loc = off; off += sub_up16(mb * npr * 4);
  L.out = off; off += mb == 1 ? 0 : sub_up16(SUB_MB * (no + 4) * 4);
  L.sh = off; off += sub_up16((int)sizeof(SubShared));
  L.total = off;
  return L;
}

// Chunk size, bias room and the key count up to which the ranks attend redundantly, for a cache of keys_cap keys.
// `all_keys` > 0 asks for a chunk that holds up to that many keys so that short caches need no second exchange; the
// chunk shrinks until the single-row and the block layout both stay under `prefer` bytes (half an SM), else under `limit`.
struct AttnSubPlan { int kc, bias_len, red_keys; bool ok; };
inline AttnSubPlan attn_sub_plan(int d, int dkv, int P, int C, int keys_cap, int all_keys, int prefer, int limit) {
  AttnSubPlan pl;
  const int per_rank = (keys_cap + C - 1) / C;
  const int need = std::min(64, sub_up16(per_rank)), want = std::min(128, sub_up16(std::min(all_keys, keys_cap)));
  auto blen = [&](int kc) { return P == 3 ? (std::max(per_rank, kc) + MAXB + 8 + 3) / 4 * 4 : 4; };
  auto fits = [&](int kc, int lim) {
    return attn_sub_layout(d, dkv, P, C, 1, kc, blen(kc)).total <= lim && attn_sub_layout(d, dkv, P, C, SUB_MB, kc, blen(kc)).total <= lim;
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
  }
  SUB_STAMP();            // P2: loads issued, cross keys requested
  sub_cluster_arrive_relaxed();   // (0) this block is up: its shared memory may be written by the cluster
  SUB_STAMP();            // 0: prologue
  pdl_wait();
  SUB_STAMP();            // 1: dependency wait
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
  float bias0 = 0.f;   // requested now, stored once the token rows are requested too
  if (tid < bias_cnt) bias0 = __ldg(a.bias + (size_t)h * a.bias_ld + dist_lo + tid);
  {   // clear the buffer the next kernel accumulates into
    const int n4 = k * (d >> 2);
#pragma unroll 1
    for (int i = blockIdx.x * SUB_THREADS + tid; i < n4; i += gridDim.x * SUB_THREADS)
      reinterpret_cast<float4*>(a.x_zero)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float inv1 = sub_load_rows<ONE>(a.x_in, k, d, g4, a.eps, Xs, xst, sh, sSeed, h == 0 ? o0 : 0, h == 0 ? o0 + no : 0, tid, lane, warp);
  if (tid < bias_cnt) sBias[tid] = bias0;
#pragma unroll 1
  for (int i = tid + SUB_THREADS; i < bias_cnt; i += SUB_THREADS) sBias[i] = __ldg(a.bias + (size_t)h * a.bias_ld + dist_lo + i);
  SUB_STAMP();            // 2: token rows + norm
  sub_wait(sh, a.err, &sh->wbar, 0, a.spin);
  SUB_STAMP();            // 3: wait for the weights
  // ---- phase A: this rank's q|k|v rows for all token rows -----------------------------------
  if (ONE) sl_items<1>(sWq, rowbytes, npr, d, Xs, xst, psum, warp, lane);
  else sl_mma<1>(sWq, rowbytes, npr, d, Xs, xst, k, psum, warp, lane);
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
  const int ch = tid & (dkv - 1), part = tid >> a.dkv_shift, nparts = SUB_THREADS >> a.dkv_shift;
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
    {   // scores: four threads per key, one channel quarter each (16-byte units interleaved over the quarters); the
        // quarter of the key stays in registers while the rows go by; 64 keys per turn
      const int qt = tid & 3;
#pragma unroll 1
      for (int jj = tid >> 2; jj < ((nk + 63) & ~63); jj += SUB_THREADS / 4) {
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
    }
    __syncthreads();
    SUB_STAMP();          // B2: scores
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
        t += p * sV[(size_t)jj * vst + ch];
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
        float c2 = 0.f, c3 = 0.f;
        const uint32_t zero = 0u;
#pragma unroll 1
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
          SUB_MMA(al0, al2, bh0, bh1);
          SUB_MMA(ah0, ah2, bl0, bl1);
#undef SUB_MMA
        }
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
      float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
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
                       : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3)
                       : "r"(wr[0][2 * st]), "r"(wr[1][2 * st]), "r"(wr[0][2 * st + 1]), "r"(wr[1][2 * st + 1]), "r"(bl0), "r"(bl1));
        }
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
  unsigned spin;             // polls of the weight barrier before the kernel gives up
  int* err;
  FfnSubLayout L;
};

inline int ffn_sub_rows(int F, int slices) { return (F + slices - 1) / slices; }
inline FfnSubLayout ffn_sub_layout(int d, int F, int gated, int slices, int grid, int mb) {
  FfnSubLayout L;
  const int nf = ffn_sub_rows(F, slices), nmat = gated ? 2 : 1;
  int off = 0;
  L.wi = off; off += sub_up16(nf * nmat * (d * 2 + SL_WPAD));
  // a single-row block keeps the rows of the transposed W_fo in registers; the block variant stages SUB_FO_REGS padded
  // rows (those past the slice are zero) for the tensor-core tiles of the output products
  L.wfo = off; off += mb == 1 ? 0 : SUB_FO_REGS * (d * 2 + SL_WPAD);
  L.xs = off; off += sub_up16(mb * (d + SL_XPAD) * 4);
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
  constexpr int ust = SUB_FO_REGS + 4;
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
  } else {
    const int i = (((tid & 31) << 3) | (tid >> 5)) - nrows;   // the rows after those of W_i, spread over the warps in the same way
    if (i >= 0 && i < nf)
      bulk_g2s(smem_u32(sWfo + (size_t)i * rowbytes), a.WfoT + (size_t)(f0 + i) * d, (uint32_t)(d * 2), smem_u32(&sh->wbar));
    // rows past the slice take part in the tiles: they must be zero
    const int z16 = (SUB_FO_REGS - nf) * (rowbytes >> 4);
#pragma unroll 1
    for (int z = tid; z < z16; z += SUB_THREADS)
      *reinterpret_cast<uint4*>(sub_smem + a.L.wfo + (size_t)nf * rowbytes + (size_t)z * 16) = make_uint4(0u, 0u, 0u, 0u);
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
  {
    if (nf > 0) sub_wait(sh, a.err, &sh->wbar, 0, a.spin);
    SUB_STAMP();          // 3: wait for the weights
    // hidden activations of the slice
    if (ONE) sl_items<1>(sWi, rowbytes, nrows, d, Xs, xst, psum, warp, lane);
    else sl_mma<1>(sWi, rowbytes, nrows, d, Xs, xst, k, psum, warp, lane);
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
    // this slice's share of all d outputs: thread <-> four columns, the rows of the transposed W_fo from its registers
    if (tid < d4) {
      const bool seeds = tid >= su0 && tid < su1;
      float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
#pragma unroll
      for (int i = 0; i < NFR; ++i) {   // (registers past the slice hold zeros)
        const float uv = i < nf ? sU[i] : 0.f;
        o0 += __uint_as_float(wfr[i].x << 16) * uv; o1 += __uint_as_float(wfr[i].x & 0xffff0000u) * uv;
        o2 += __uint_as_float(wfr[i].y << 16) * uv; o3 += __uint_as_float(wfr[i].y & 0xffff0000u) * uv;
      }
      if (seeds) {
        const float4 xr = *reinterpret_cast<const float4*>(sSeed + (tid - su0) * 4);
        o0 += xr.x; o1 += xr.y; o2 += xr.z; o3 += xr.w;
      }
      if (nf > 0 || seeds)
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(a.x_out + tid * 4), "f"(o0), "f"(o1), "f"(o2), "f"(o3) : "memory");
    }
  } else {
    // out[token][column] = sum_i u[token][i] * WfoT[i][column] on mma.sync m16n8k16: the token rows are the 16 rows of
    // the left operand (rows 8..15 zero), each activation as a bf16 head and a bf16 remainder; the right operand
    // (32 slice rows x 8 columns, two steps of 16) comes out of the padded rows with one transposing matrix load
    const int g = lane >> 2, t = lane & 3;
    uint32_t ah[2][2], al[2][2];
#pragma unroll
    for (int st = 0; st < 2; ++st)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const float2 u2 = *reinterpret_cast<const float2*>(sU + (size_t)g * ust + 16 * st + 8 * hh + 2 * t);
        ah[st][hh] = sl_pack_bf16(u2.x, u2.y);
        al[st][hh] = sl_pack_bf16(u2.x - __uint_as_float(ah[st][hh] << 16), u2.y - __uint_as_float(ah[st][hh] & 0xffff0000u));
      }
    const uint32_t brow = smem_u32(sWfo + (size_t)lane * rowbytes);   // lane l addresses slice row l of each 8 x 8 piece
    const uint32_t zero = 0u;
#pragma unroll 1
    for (int nt = warp; nt < (d >> 3); nt += SUB_THREADS / 32) {
      uint32_t b0, b1, b2, b3;
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                   : "=r"(b0), "=r"(b1), "=r"(b2), "=r"(b3) : "r"(brow + (uint32_t)nt * 16u));
      float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
#define SUB_MMA(A0, A2, B0, B1)                                                                                              \
      asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};" \
                   : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3) : "r"(A0), "r"(zero), "r"(A2), "r"(zero), "r"(B0), "r"(B1))
      SUB_MMA(ah[0][0], ah[0][1], b0, b1);
      SUB_MMA(al[0][0], al[0][1], b0, b1);
      SUB_MMA(ah[1][0], ah[1][1], b2, b3);
      SUB_MMA(al[1][0], al[1][1], b2, b3);
#undef SUB_MMA
      // c0, c1: token row g, columns 8 nt + 2 t (+ 1)
      const int col = nt * 8 + 2 * t, un = col >> 2;
      const bool seeds = un >= su0 && un < su1;
      if (g < k && (nf > 0 || seeds)) {
        if (seeds) {
          const float2 xr = *reinterpret_cast<const float2*>(sSeed + (size_t)g * (su1 - su0) * 4 + (col - su0 * 4));
          c0 += xr.x; c1 += xr.y;
        }
        asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(a.x_out + (size_t)g * d + col), "f"(c0), "f"(c1) : "memory");
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
