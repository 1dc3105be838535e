// Latency-tuned kernels of the decode passes: the M = 1 weight-streaming GEMV of the
// small-model step and the block attention that reads each cached key/value once for all
// rows of the block.  All of them support programmatic dependent launch: what does not
// depend on the previous kernel (the weight loads) is issued before the dependency wait.
#pragma once
#include "kernels.cuh"

namespace bild {

// ---------------------------------------------------------------------------------
// GEMV for one activation row (steps S1, S3, S4, S6, S7, S8 of the small-model step):
//   v[n] = inv_rms * sum_j W[n][j] * x[j] * g[j]        (inv_rms = 1, g = 1 without norm)
// One warp owns RW weight rows.  Its first PRE*256 columns are loaded into registers
// before the dependency wait; x, g and the sum of squares are taken in the same pass, so
// there is no shared memory and no block-wide barrier.  Same epilogues as linear_kernel.
// ---------------------------------------------------------------------------------
// Kernel code is kept small on purpose: the kernels of a layer alternate every few
// microseconds and their instructions have to stay in the SMs' instruction caches.
constexpr int GEMV_PRE = 4;   // (block GEMV) column chunks of 256 whose weights are fetched ahead

// Where output row n of a packed q|k|v (or k|v) projection goes: part 0 = q, 1 = k, 2 = v.
__device__ __forceinline__ void heads_store(const LinArgs& a, int n, int m, int pos0, float v) {
  int part = a.first_part, rr = n;
  if (rr >= a.inner) { rr -= a.inner; ++part; }
  if (rr >= a.inner) { rr -= a.inner; ++part; }
  if (part == 0) {
    a.q_out[(size_t)m * a.ldq + rr] = v;
  } else {
    const int h = rr >> a.dkv_shift, c = rr & (a.dkv - 1);
    const int row = pos0 + m;
    if (row < a.cap) (part == 1 ? a.kc : a.vc)[((size_t)h * a.cap + row) * a.dkv + c] = v;
  }
}

// One group of 2 weight rows is shared by a.ksplit warps, each taking K / ksplit (<= 256 when
// K <= 4096) contiguous columns, so every weight byte is requested before the dependency
// wait with one 128-bit load per lane and row.  Partial sums are added in warp order.
template <typename WT, bool GATED>
__global__ void __launch_bounds__(512) gemv_kernel(LinArgs a) {
  __shared__ float s_part[16][5];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ks = a.ksplit;
  // more than one group per block only for ksplit 1 or 2 (host: groups = max(1, 4 / ksplit))
  const int group = a.groups == 1 ? 0 : (ks == 1 ? warp : warp >> 1);
  const int kw = a.groups == 1 ? warp : (ks == 1 ? 0 : warp & 1);
  const int n0 = (blockIdx.x * a.groups + group) * 2;
  const int K = a.K, kl = a.kl, kbeg = kw * kl;
  const int c0 = lane * 8;
  const int r0 = min(n0, a.N - 1), r1 = min(n0 + 1, a.N - 1);
  const WT* W0 = (const WT*)a.W0 + kbeg;
  const WT* W1 = (const WT*)a.W1 + kbeg;
  float w00[8], w01[8], w10[8], w11[8];
  if (c0 < kl) {
    load8(W0 + (size_t)r0 * K + c0, w00);
    load8(W0 + (size_t)r1 * K + c0, w01);
    if (GATED) { load8(W1 + (size_t)r0 * K + c0, w10); load8(W1 + (size_t)r1 * K + c0, w11); }
  }
  // the norm gains are weights too: fetched before the dependency wait
  float gpre[8] = {1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f};
  if (a.gain && c0 < kl) {
    const float4 g0 = __ldg(reinterpret_cast<const float4*>(a.gain + kbeg + c0));
    const float4 g1 = __ldg(reinterpret_cast<const float4*>(a.gain + kbeg + c0 + 4));
    gpre[0] = g0.x; gpre[1] = g0.y; gpre[2] = g0.z; gpre[3] = g0.w; gpre[4] = g1.x; gpre[5] = g1.y; gpre[6] = g1.z; gpre[7] = g1.w;
  }
  pdl_launch_dependents();
  pdl_wait();
  // the value a residual epilogue adds to is requested now, not when the sums are ready
  float y_old = 0.f;
  if (a.epi == EPI_RESID && lane < 2 && n0 + lane < a.N) y_old = __ldcg(a.Y + n0 + lane);
  const float* X = a.X + kbeg;
  const float* G = a.gain ? a.gain + kbeg : nullptr;
  float a00 = 0.f, a01 = 0.f, a10 = 0.f, a11 = 0.f, ss = 0.f;
#pragma unroll 1
  for (int c = c0; c < kl; c += 256) {
    if (c != c0) {   // columns beyond the first 256 of this warp (K > 4096 only)
      load8(W0 + (size_t)r0 * K + c, w00);
      load8(W0 + (size_t)r1 * K + c, w01);
      if (GATED) { load8(W1 + (size_t)r0 * K + c, w10); load8(W1 + (size_t)r1 * K + c, w11); }
    }
    const float4 x0 = *reinterpret_cast<const float4*>(X + c);
    const float4 x1 = *reinterpret_cast<const float4*>(X + c + 4);
    float h[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
    if (G) {
      if (c != c0) {
        const float4 g0 = *reinterpret_cast<const float4*>(G + c);
        const float4 g1 = *reinterpret_cast<const float4*>(G + c + 4);
        gpre[0] = g0.x; gpre[1] = g0.y; gpre[2] = g0.z; gpre[3] = g0.w; gpre[4] = g1.x; gpre[5] = g1.y; gpre[6] = g1.z; gpre[7] = g1.w;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) { ss += h[i] * h[i]; h[i] *= gpre[i]; }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      a00 += w00[i] * h[i];
      a01 += w01[i] * h[i];
      if (GATED) { a10 += w10[i] * h[i]; a11 += w11[i] * h[i]; }
    }
  }
  a00 = warp_sum(a00); a01 = warp_sum(a01); ss = warp_sum(ss);
  if (GATED) { a10 = warp_sum(a10); a11 = warp_sum(a11); }
  if (ks > 1) {
    if (lane == 0) { s_part[warp][0] = a00; s_part[warp][1] = a01; s_part[warp][2] = a10; s_part[warp][3] = a11; s_part[warp][4] = ss; }
    __syncthreads();
    if (kw != 0) return;
    a00 = a01 = a10 = a11 = ss = 0.f;
    for (int w2 = group * ks; w2 < group * ks + ks; ++w2) {   // fixed order
      a00 += s_part[w2][0]; a01 += s_part[w2][1]; a10 += s_part[w2][2]; a11 += s_part[w2][3]; ss += s_part[w2][4];
    }
  }
  if (lane > 1) return;
  const int n = n0 + lane;
  if (n >= a.N) return;
  const float inv = a.gain ? rsqrtf(ss * a.inv_k + a.eps) : 1.f;
  const float v0 = (lane ? a01 : a00) * inv;
  if (a.epi == EPI_RESID) a.Y[n] = y_old + v0;
  else if (a.epi == EPI_STORE) a.Y[n] = v0;
  else if (a.epi == EPI_RELU) a.Y[n] = fmaxf(v0, 0.f);
  else if (a.epi == EPI_GATED) { if (GATED) a.Y[n] = gelu_tanh(v0) * ((lane ? a11 : a10) * inv); }
  else heads_store(a, n, 0, a.desc ? a.desc->pos0 : a.pos0_host, v0);
}

// ---------------------------------------------------------------------------------
// Block GEMV, compact: the GEMV above with a loop over the token rows of the block (steps L1,
// L3, L4, L6, L7, L8).  The weights of the warp stay in registers (fetched before the
// dependency wait); token rows are taken four at a time, all four loads in flight at once.
// The first four rows are requested before the row count is known: all MAXB rows of the
// activation buffers exist.  Requires K <= 4096 (one 256-column chunk per warp).
// ---------------------------------------------------------------------------------
template <typename WT, bool GATED>
__global__ void __launch_bounds__(512) gemvb_kernel(LinArgs a) {
  __shared__ float s_part[MAXB][16][5];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ks = a.ksplit;                 // all warps of the block share one group of 2 rows
  const int n0 = blockIdx.x * 2;
  const int K = a.K, kl = a.kl, kbeg = warp * kl;
  const int c0 = lane * 8;
  const bool act = c0 < kl;
  const int r0 = min(n0, a.N - 1), r1 = min(n0 + 1, a.N - 1);
  const WT* W0 = (const WT*)a.W0 + kbeg;
  const WT* W1 = (const WT*)a.W1 + kbeg;
  float w00[8], w01[8], w10[8], w11[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { w00[i] = w01[i] = 0.f; if (GATED) w10[i] = w11[i] = 0.f; }
  if (act) {
    load8(W0 + (size_t)r0 * K + c0, w00);
    load8(W0 + (size_t)r1 * K + c0, w01);
    if (GATED) { load8(W1 + (size_t)r0 * K + c0, w10); load8(W1 + (size_t)r1 * K + c0, w11); }
  }
  pdl_launch_dependents();
  pdl_wait();
  const int out_m = threadIdx.x >> 1, out_r = threadIdx.x & 1;   // writer threads: tid < 2 * M
  float old = 0.f;
  if (threadIdx.x < 2 * MAXB && a.epi == EPI_RESID && n0 + out_r < a.N) old = a.Y[(size_t)out_m * a.ldy + n0 + out_r];
  float g[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) g[i] = 1.f;
  if (a.gain && act) {
    const float4 g0 = *reinterpret_cast<const float4*>(a.gain + kbeg + c0);
    const float4 g1 = *reinterpret_cast<const float4*>(a.gain + kbeg + c0 + 4);
    g[0] = g0.x; g[1] = g0.y; g[2] = g0.z; g[3] = g0.w; g[4] = g1.x; g[5] = g1.y; g[6] = g1.z; g[7] = g1.w;
  }
  const float* X = a.X + kbeg + c0;
  int M = 4;   // rows 0..3 first; the true count arrives with them
#pragma unroll 1
  for (int m0 = 0; m0 < M; m0 += 4) {
    float4 xa[4], xb[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      xa[t] = xb[t] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (act) {
        xa[t] = *reinterpret_cast<const float4*>(X + (size_t)(m0 + t) * a.ldx);
        xb[t] = *reinterpret_cast<const float4*>(X + (size_t)(m0 + t) * a.ldx + 4);
      }
    }
    if (m0 == 0) M = min(a.desc ? a.desc->k : a.M, MAXB);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      float h[8] = {xa[t].x, xa[t].y, xa[t].z, xa[t].w, xb[t].x, xb[t].y, xb[t].z, xb[t].w};
      float a00 = 0.f, a01 = 0.f, a10 = 0.f, a11 = 0.f, ss = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        ss += h[i] * h[i];
        h[i] *= g[i];
        a00 += w00[i] * h[i];
        a01 += w01[i] * h[i];
        if (GATED) { a10 += w10[i] * h[i]; a11 += w11[i] * h[i]; }
      }
      a00 = warp_sum(a00); a01 = warp_sum(a01); ss = warp_sum(ss);
      if (GATED) { a10 = warp_sum(a10); a11 = warp_sum(a11); }
      if (lane == 0) {
        float* sp = s_part[m0 + t][warp];
        sp[0] = a00; sp[1] = a01; sp[2] = a10; sp[3] = a11; sp[4] = ss;
      }
    }
  }
  __syncthreads();
  if (threadIdx.x >= 2 * M) return;
  const int n = n0 + out_r;
  if (n >= a.N) return;
  float v0 = 0.f, v1 = 0.f, sq = 0.f;
#pragma unroll 1
  for (int w2 = 0; w2 < ks; ++w2) {   // fixed order
    const float* sp = s_part[out_m][w2];
    v0 += sp[out_r]; v1 += sp[2 + out_r]; sq += sp[4];
  }
  const float inv = a.gain ? rsqrtf(sq * a.inv_k + a.eps) : 1.f;
  v0 *= inv;
  if (a.epi == EPI_RESID) a.Y[(size_t)out_m * a.ldy + n] = old + v0;
  else if (a.epi == EPI_STORE) a.Y[(size_t)out_m * a.ldy + n] = v0;
  else if (a.epi == EPI_RELU) a.Y[(size_t)out_m * a.ldy + n] = fmaxf(v0, 0.f);
  else if (a.epi == EPI_GATED) { if (GATED) a.Y[(size_t)out_m * a.ldy + n] = gelu_tanh(v0) * (v1 * inv); }
  else heads_store(a, n, out_m, a.desc ? a.desc->pos0 : a.pos0_host, v0);
}

// ---------------------------------------------------------------------------------
// The same GEMV for a block of up to MAXB token rows (steps L1, L3, L4, L6, L7, L8 when the
// block pass is latency-bound): one block owns RW weight rows, its warps split K so that each
// warp's weights (<= GEMV_PRE chunks of 256 columns) sit in registers before the dependency
// wait.  Token rows are then taken four at a time against those registers; the loads of the
// next four rows are in flight while the current four are reduced.  Partial sums of the
// warps are added in warp order through shared memory.
// ---------------------------------------------------------------------------------
constexpr int GEMVK_TG = 4;   // token rows per step

template <typename WT, int RW, int PC, bool GATED>   // PC: chunks of 256 columns per warp
__global__ void __launch_bounds__(512) gemvk_kernel(LinArgs a) {
  constexpr int NV = RW * (GATED ? 2 : 1) * GEMVK_TG + GEMVK_TG;   // values per warp and step: sums + squares
  __shared__ float s_part[2][16][NV];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ks = blockDim.x >> 5;
  const int n0 = blockIdx.x * RW;
  const int K = a.K, kl = K / ks, kbeg = warp * kl;
  const WT* W0 = (const WT*)a.W0;
  const WT* W1 = (const WT*)a.W1;
  float pre0[RW][PC][8], pre1[GATED ? RW : 1][GATED ? PC : 1][8];
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    const size_t row = (size_t)min(n0 + r, a.N - 1) * K + kbeg;
#pragma unroll
    for (int p = 0; p < PC; ++p) {
      const int c = p * 256 + lane * 8;
      if (c < kl) {
        load8(W0 + row + c, pre0[r][p]);
        if (GATED) load8(W1 + row + c, pre1[r][p]);
      }
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  // requested together: the row count, the gains, the first four activation rows, and (for the
  // threads that write results) the residual values they will update
  const int M = a.desc ? a.desc->k : a.M;
  const int pos0 = a.desc ? a.desc->pos0 : a.pos0_host;
  const int out_r = threadIdx.x / GEMVK_TG, out_m = threadIdx.x % GEMVK_TG;   // writer threads: tid < RW * TG
  const bool writer = threadIdx.x < RW * GEMVK_TG && n0 + out_r < a.N;
  float old[MAXB / GEMVK_TG];
  if (writer && a.epi == EPI_RESID) {
#pragma unroll
    for (int g = 0; g < MAXB / GEMVK_TG; ++g) old[g] = a.Y[(size_t)(g * GEMVK_TG + out_m) * a.ldy + n0 + out_r];
  }
  float gn[PC][8];
#pragma unroll
  for (int p = 0; p < PC; ++p) {
    const int c = p * 256 + lane * 8;
#pragma unroll
    for (int i = 0; i < 8; ++i) gn[p][i] = 1.f;
    if (a.gain && c < kl) {
      const float4 g0 = *reinterpret_cast<const float4*>(a.gain + kbeg + c);
      const float4 g1 = *reinterpret_cast<const float4*>(a.gain + kbeg + c + 4);
      gn[p][0] = g0.x; gn[p][1] = g0.y; gn[p][2] = g0.z; gn[p][3] = g0.w;
      gn[p][4] = g1.x; gn[p][5] = g1.y; gn[p][6] = g1.z; gn[p][7] = g1.w;
    }
  }
  float4 xa[GEMVK_TG][PC], xb[GEMVK_TG][PC];
  auto load_rows = [&](int m_first) {   // all MAXB rows of the activation buffer exist
#pragma unroll
    for (int t = 0; t < GEMVK_TG; ++t)
#pragma unroll
      for (int p = 0; p < PC; ++p) {
        const int c = p * 256 + lane * 8;
        if (c < kl) {
          const float* xp = a.X + (size_t)(m_first + t) * a.ldx + kbeg + c;
          xa[t][p] = *reinterpret_cast<const float4*>(xp);
          xb[t][p] = *reinterpret_cast<const float4*>(xp + 4);
        }
      }
  };
  load_rows(0);
  const int groups = (min(M, MAXB) + GEMVK_TG - 1) / GEMVK_TG;
#pragma unroll
  for (int g = 0; g < MAXB / GEMVK_TG; ++g) {
    if (g >= groups) break;   // uniform over the block
    float acc0[RW][GEMVK_TG], acc1[GATED ? RW : 1][GEMVK_TG], ss[GEMVK_TG];
#pragma unroll
    for (int t = 0; t < GEMVK_TG; ++t) {
      ss[t] = 0.f;
#pragma unroll
      for (int r = 0; r < RW; ++r) { acc0[r][t] = 0.f; if (GATED) acc1[r][t] = 0.f; }
#pragma unroll
      for (int p = 0; p < PC; ++p) {
        const int c = p * 256 + lane * 8;
        if (c < kl) {
          float h[8] = {xa[t][p].x, xa[t][p].y, xa[t][p].z, xa[t][p].w, xb[t][p].x, xb[t][p].y, xb[t][p].z, xb[t][p].w};
#pragma unroll
          for (int i = 0; i < 8; ++i) { ss[t] += h[i] * h[i]; h[i] *= gn[p][i]; }
#pragma unroll
          for (int r = 0; r < RW; ++r) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              acc0[r][t] += pre0[r][p][i] * h[i];
              if (GATED) acc1[r][t] += pre1[r][p][i] * h[i];
            }
          }
        }
      }
    }
    if (g + 1 < groups) load_rows((g + 1) * GEMVK_TG);   // in flight during the reduction below
    float* sp = s_part[g & 1][warp];
#pragma unroll
    for (int t = 0; t < GEMVK_TG; ++t) {
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        const float v = warp_sum(acc0[r][t]);
        if (lane == 0) sp[r * GEMVK_TG + t] = v;
        if (GATED) {
          const float v1 = warp_sum(acc1[r][t]);
          if (lane == 0) sp[(RW + r) * GEMVK_TG + t] = v1;
        }
      }
      const float sv = warp_sum(ss[t]);
      if (lane == 0) sp[NV - GEMVK_TG + t] = sv;
    }
    __syncthreads();
    const int m = g * GEMVK_TG + out_m;
    if (writer && m < M) {
      float v0 = 0.f, v1 = 0.f, sq = 0.f;
      for (int w2 = 0; w2 < ks; ++w2) {   // fixed order
        const float* q = s_part[g & 1][w2];
        v0 += q[out_r * GEMVK_TG + out_m];
        if (GATED) v1 += q[(RW + out_r) * GEMVK_TG + out_m];
        sq += q[NV - GEMVK_TG + out_m];
      }
      if (a.gain) {
        const float inv = rsqrtf(sq / (float)K + a.eps);
        v0 *= inv;
        v1 *= inv;
      }
      const int n = n0 + out_r;
      switch (a.epi) {
        case EPI_STORE: a.Y[(size_t)m * a.ldy + n] = v0; break;
        case EPI_RELU: a.Y[(size_t)m * a.ldy + n] = fmaxf(v0, 0.f); break;
        case EPI_GATED: a.Y[(size_t)m * a.ldy + n] = gelu_tanh(v0) * v1; break;
        case EPI_RESID: a.Y[(size_t)m * a.ldy + n] = old[g] + v0; break;
        default: heads_store(a, n, m, pos0, v0);
      }
    }
  }
}

// ---------------------------------------------------------------------------------
// Block attention (steps S2, S5, L2, L5 and the encoder's self-attention): one block per
// (head, key split, block of MB query rows) reads every key and value of its split ONCE
// and serves all MB rows from it.
//   scores : one thread per key, the key row in registers, MB dot products
//   softmax: one warp per row (max, exp, sum) in a fixed order
//   values : thread (channel c, group g) accumulates keys j = g mod ng for all MB rows
// Splits write (max, sum, weighted values) per row to scratch; the split that takes the
// last ticket of its (head, row block) merges them in split order.
// mode 0 cross (all E keys), 1 decoder self (row i sees keys 0..pos0+i, bias by distance),
// mode 2 encoder self (all E keys, bias by signed distance).
// ---------------------------------------------------------------------------------
struct BAttnArgs {
  const float* q;
  int ldq;
  const float* kc;
  const float* vc;
  int cap;
  float* out;
  int ldo;
  const float* bias;
  int bias_ld, bias_off;
  int mode, dkv, H;
  const int* n_keys_dev;
  int M;                 // rows when desc == nullptr
  const CallDesc* desc;
  float* part;           // [row block][H][nsplit][MB][2 + dkv]
  unsigned* counters;    // [row block][H]
  int nsplit, smem_keys;
  int* err;
};

constexpr int BATT_THREADS = 128;

// STAGE: the block's keys and values are first copied to shared memory with cp.async (for
// cross-attention before the dependency wait, since the encoder K/V never change during
// decoding), and scores and weighted values are then computed from shared memory.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}

template <int MB, bool STAGE>
__global__ void __launch_bounds__(BATT_THREADS) battn_kernel(BAttnArgs a) {
  extern __shared__ float s_dyn[];          // scores [MB][sk] | keys [sk][dkv + 4] | values [sk][dkv]
  __shared__ float s_q[MB][128];
  __shared__ float s_m[MB], s_l[MB];
  __shared__ float s_red[BATT_THREADS / 16][MB][16 + 1];   // value partials of the key groups (dkv = 16 chunks)
  __shared__ int s_last;
  const int h = blockIdx.x, sp = blockIdx.y, rb = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int dkv = a.dkv;
  const int sk = a.smem_keys;
  float* sK = s_dyn + MB * sk;
  float* sV = sK + sk * (dkv + 4);
  auto stage_kv = [&](int first, int count) {
    const float* Kg = a.kc + ((size_t)h * a.cap + first) * dkv;
    const float* Vg = a.vc + ((size_t)h * a.cap + first) * dkv;
    const int q4 = dkv / 4;
    for (int idx = tid; idx < count * q4; idx += BATT_THREADS) {
      const int jj = idx / q4, e = idx - jj * q4;
      cp_async16(sK + jj * (dkv + 4) + 4 * e, Kg + (size_t)jj * dkv + 4 * e);
      cp_async16(sV + jj * dkv + 4 * e, Vg + (size_t)jj * dkv + 4 * e);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  if (STAGE && a.mode == 0) {   // static data: fetch before waiting for the previous kernel
    const int n_all = min(*a.n_keys_dev, a.cap);
    const int ch = (n_all + a.nsplit - 1) / a.nsplit;
    if (ch <= sk) stage_kv(sp * ch, max(0, min(n_all, sp * ch + ch) - sp * ch));
  }
  pdl_launch_dependents();
  pdl_wait();
  const int M = a.desc ? a.desc->k : a.M;
  const int m0 = rb * MB;
  const int mrows = min(MB, M - m0);
  if (mrows <= 0) return;
  const int pos0 = a.desc ? a.desc->pos0 : 0;
  // keys any row of this block may see
  int n = (a.mode == 1) ? pos0 + m0 + mrows : *a.n_keys_dev;
  n = min(n, a.cap);
  const int chunk = (n + a.nsplit - 1) / a.nsplit;
  const int j0 = sp * chunk, j1 = min(n, j0 + chunk);
  const int nk = max(0, j1 - j0);
  if (chunk > a.smem_keys) {
    if (tid == 0) *a.err = BILD_ERR_CAPACITY;
    return;
  }
  const float* K = a.kc + (size_t)h * a.cap * dkv;
  const float* V = a.vc + (size_t)h * a.cap * dkv;
  if (STAGE && a.mode != 0) stage_kv(j0, nk);
  for (int idx = tid; idx < mrows * dkv; idx += BATT_THREADS) {
    const int i = idx / dkv, e = idx - i * dkv;
    s_q[i][e] = a.q[(size_t)(m0 + i) * a.ldq + h * dkv + e];
  }
  if (STAGE) asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  // ---- scores ----
  for (int jj = tid; jj < nk; jj += BATT_THREADS) {
    const int j = j0 + jj;
    float acc[MB];
#pragma unroll
    for (int i = 0; i < MB; ++i) acc[i] = 0.f;
    const float4* kr = STAGE ? reinterpret_cast<const float4*>(sK + jj * (dkv + 4))
                             : reinterpret_cast<const float4*>(K + (size_t)j * dkv);
    const int nq4 = dkv / 4;
    for (int e0 = 0; e0 < nq4; e0 += 8) {   // eight independent 16-byte loads in flight
      float4 kv[8];
#pragma unroll
      for (int u2 = 0; u2 < 8; ++u2) kv[u2] = (e0 + u2 < nq4) ? kr[e0 + u2] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u2 = 0; u2 < 8; ++u2) {
        if (e0 + u2 < nq4) {
#pragma unroll
          for (int i = 0; i < MB; ++i) {
            const float4 qv = *reinterpret_cast<const float4*>(&s_q[i][4 * (e0 + u2)]);
            acc[i] += kv[u2].x * qv.x + kv[u2].y * qv.y + kv[u2].z * qv.z + kv[u2].w * qv.w;
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < MB; ++i) {
      if (i < mrows) {
        float sc = acc[i];
        const int qi = m0 + i;
        if (a.mode == 1) sc = (j <= pos0 + qi) ? sc + a.bias[(size_t)h * a.bias_ld + (pos0 + qi - j)] : -INFINITY;
        else if (a.mode == 2) sc += a.bias[(size_t)h * a.bias_ld + (j - qi + a.bias_off)];
        s_dyn[i * sk + jj] = sc;
      }
    }
  }
  __syncthreads();
  // ---- softmax statistics, one warp per row ----
  for (int i = warp; i < mrows; i += BATT_THREADS / 32) {
    float mx = -INFINITY;
    for (int jj = lane; jj < nk; jj += 32) mx = fmaxf(mx, s_dyn[i * sk + jj]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int jj = lane; jj < nk; jj += 32) {
      const float sc = s_dyn[i * sk + jj];
      const float p = (sc == -INFINITY) ? 0.f : expf(sc - mx);
      s_dyn[i * sk + jj] = p;
      sum += p;
    }
    sum = warp_sum(sum);
    if (lane == 0) { s_m[i] = mx; s_l[i] = sum; }
  }
  __syncthreads();
  // ---- weighted values ----
  const int ng = BATT_THREADS / dkv;
  const int c = tid % dkv, g = tid / dkv;
  float acc[MB];
#pragma unroll
  for (int i = 0; i < MB; ++i) acc[i] = 0.f;
  for (int jj = g; jj < nk; jj += 4 * ng) {   // four values in flight per thread
    float v[4];
#pragma unroll
    for (int u2 = 0; u2 < 4; ++u2)
      v[u2] = (jj + u2 * ng < nk) ? (STAGE ? sV[(jj + u2 * ng) * dkv + c] : V[(size_t)(j0 + jj + u2 * ng) * dkv + c]) : 0.f;
#pragma unroll
    for (int u2 = 0; u2 < 4; ++u2) {
      if (jj + u2 * ng < nk) {
#pragma unroll
        for (int i = 0; i < MB; ++i) acc[i] += s_dyn[i * sk + jj + u2 * ng] * v[u2];
      }
    }
  }
  // reduce the ng key groups in group order through shared memory (reusing s_dyn is not
  // possible: other threads may still read it), 16 channels at a time
  float* P = a.part + ((((size_t)rb * a.H + h) * a.nsplit + sp) * MB) * (dkv + 2);
  for (int c0 = 0; c0 < dkv; c0 += 16) {
    __syncthreads();
    if (c >= c0 && c < c0 + 16)
#pragma unroll
      for (int i = 0; i < MB; ++i) s_red[g][i][c - c0] = acc[i];
    __syncthreads();
    for (int idx = tid; idx < mrows * 16; idx += BATT_THREADS) {
      const int i = idx / 16, cc = idx % 16;
      float t = 0.f;
      for (int gg = 0; gg < ng; ++gg) t += s_red[gg][i][cc];
      if (a.nsplit == 1) a.out[(size_t)(m0 + i) * a.ldo + h * dkv + c0 + cc] = t / s_l[i];
      else P[(size_t)i * (dkv + 2) + 2 + c0 + cc] = t;
    }
  }
  if (a.nsplit == 1) return;
  if (tid < mrows) { P[(size_t)tid * (dkv + 2)] = s_m[tid]; P[(size_t)tid * (dkv + 2) + 1] = s_l[tid]; }
  __threadfence();
  __syncthreads();
  const int slot = rb * a.H + h;
  if (tid == 0) {
    const unsigned t = atomicAdd(&a.counters[slot], 1u);
    s_last = (t == (unsigned)a.nsplit - 1);
    if (s_last) a.counters[slot] = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float* P0 = a.part + (((size_t)rb * a.H + h) * a.nsplit * MB) * (dkv + 2);
  for (int idx = tid; idx < mrows * dkv; idx += BATT_THREADS) {
    const int i = idx / dkv, cc = idx - i * dkv;
    float gm = -INFINITY;
    for (int s = 0; s < a.nsplit; ++s) gm = fmaxf(gm, __ldcg(&P0[((size_t)s * MB + i) * (dkv + 2)]));
    float num = 0.f, den = 0.f;
    for (int s = 0; s < a.nsplit; ++s) {
      const float* Ps = P0 + ((size_t)s * MB + i) * (dkv + 2);
      const float l = __ldcg(&Ps[1]);
      if (l > 0.f) {
        const float w = expf(__ldcg(&Ps[0]) - gm);
        den += l * w;
        num += __ldcg(&Ps[2 + cc]) * w;
      }
    }
    a.out[(size_t)(m0 + i) * a.ldo + h * dkv + cc] = num / den;
  }
}

// ---------------------------------------------------------------------------------
// LM head for one row (steps S9 + S10, and the large model at k = 1): a GEMV over the
// vocabulary fused with the online max / arg-max / sum-exp.  Every warp owns RPW consecutive
// vocabulary rows whose weights are all requested before the dependency wait (the head is
// the largest matrix of the step, so its load overlaps the last layers of the pass).  The
// block writes one partial; the block with the last ticket merges all partials (each thread
// loads its share at once, then a fixed-order tree) and runs the policy code.
// ---------------------------------------------------------------------------------
constexpr int HEAD1_THREADS = 256;

template <typename WT, int NCH, int RPW>   // NCH chunks of 256 columns per row, RPW rows per warp
__global__ void __launch_bounds__(HEAD1_THREADS) head1_kernel(HeadArgs a) {
  constexpr int NW = HEAD1_THREADS / 32;
  __shared__ Partial s_p[HEAD1_THREADS];
  __shared__ int s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int K = a.K, V = a.V;
  const int n0 = (blockIdx.x * NW + warp) * RPW;
  const WT* W = (const WT*)a.W;
  float w[RPW][NCH][8];
#pragma unroll
  for (int r = 0; r < RPW; ++r)
#pragma unroll
    for (int p = 0; p < NCH; ++p) {
      const int c = p * 256 + lane * 8;
      if (c < K) load8(W + (size_t)min(n0 + r, V - 1) * K + c, w[r][p]);
    }
  float gn[NCH][8];   // the norm gains are weights too
  if (a.gain) {
#pragma unroll
    for (int p = 0; p < NCH; ++p) {
      const int c = p * 256 + lane * 8;
      if (c < K) {
        const float4 g0 = __ldg(reinterpret_cast<const float4*>(a.gain + c)), g1 = __ldg(reinterpret_cast<const float4*>(a.gain + c + 4));
        gn[p][0] = g0.x; gn[p][1] = g0.y; gn[p][2] = g0.z; gn[p][3] = g0.w; gn[p][4] = g1.x; gn[p][5] = g1.y; gn[p][6] = g1.z; gn[p][7] = g1.w;
      }
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  const int target = a.desc ? a.desc->targets[0] : (a.target ? a.target[0] : -1);
  float acc[RPW], ss = 0.f;
#pragma unroll
  for (int r = 0; r < RPW; ++r) acc[r] = 0.f;
#pragma unroll
  for (int p = 0; p < NCH; ++p) {
    const int c = p * 256 + lane * 8;
    if (c < K) {
      const float4 x0 = *reinterpret_cast<const float4*>(a.X + c), x1 = *reinterpret_cast<const float4*>(a.X + c + 4);
      float h[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
      if (a.gain) {
#pragma unroll
        for (int i = 0; i < 8; ++i) { ss += h[i] * h[i]; h[i] *= gn[p][i]; }
      }
#pragma unroll
      for (int r = 0; r < RPW; ++r)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[r] += w[r][p][i] * h[i];
    }
  }
  ss = warp_sum(ss);
  const float mul = (a.gain ? rsqrtf(ss / (float)K + a.eps) : 1.f) * a.scale;
  Partial run;
  run.m = -INFINITY; run.s = 0.f; run.idx = 0x7fffffff;
#pragma unroll
  for (int r = 0; r < RPW; ++r) {
    const float z = warp_sum(acc[r]) * mul;
    const int n = n0 + r;
    if (n < V) {
      if (z > run.m) { run.s = run.s * __expf(run.m - z) + 1.f; run.m = z; run.idx = n; }
      else run.s += __expf(z - run.m);
      if (lane == 0) {
        if (n == target) a.out->gather[0] = z;
        if (a.logits_dbg) a.logits_dbg[n] = z;
      }
    }
  }
  if (lane == 0) s_p[warp] = run;
  __syncthreads();
  if (threadIdx.x == 0) {
    Partial p = s_p[0];
    for (int w2 = 1; w2 < NW; ++w2) p = combine(p, s_p[w2]);
    a.partials[blockIdx.x] = p;
    __threadfence();
    const unsigned t = atomicAdd(a.counter, 1u);
    s_last = (t == gridDim.x - 1);
    if (s_last) *a.counter = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // merge: every thread requests its partials together, then combines them in index order
  {
    Partial q[8];
    const int nb = (int)gridDim.x;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int b = threadIdx.x + j * HEAD1_THREADS;
      q[j].m = -INFINITY; q[j].s = 0.f; q[j].idx = 0x7fffffff;
      if (b < nb) { q[j].m = __ldcg(&a.partials[b].m); q[j].s = __ldcg(&a.partials[b].s); q[j].idx = __ldcg(&a.partials[b].idx); }
    }
    Partial p = q[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) p = combine(p, q[j]);
    for (int b = threadIdx.x + 8 * HEAD1_THREADS; b < nb; b += HEAD1_THREADS) {   // very large vocabularies
      Partial t2;
      t2.m = __ldcg(&a.partials[b].m); t2.s = __ldcg(&a.partials[b].s); t2.idx = __ldcg(&a.partials[b].idx);
      p = combine(p, t2);
    }
    s_p[threadIdx.x] = p;
  }
  __syncthreads();
  for (int stride = HEAD1_THREADS / 2; stride > 0; stride >>= 1) {
    if (threadIdx.x < stride) s_p[threadIdx.x] = combine(s_p[threadIdx.x], s_p[threadIdx.x + stride]);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const Partial p = s_p[0];
    HeadOut* o = a.out;
    o->argmax[0] = p.idx;
    o->zmax[0] = p.m;
    o->lse[0] = p.m + logf(p.s);
    o->pmax = 1.f / p.s;
    o->gather[0] = __ldcg(&o->gather[0]);
    policy_tail(a, o);
  }
}

// ---------------------------------------------------------------------------------
// LM head for one row, bf16 weights, streaming variant: two blocks per SM stay for the whole vocabulary; every warp
// owns a contiguous range of vocabulary rows and walks it R rows at a time, each batch requested with 16-byte loads
// (R x NCH per lane, all issued before any is used; the first batch before the dependency wait), reduced R rows at
// once (one shuffle per halving), with the running (max, arg, sum-exp) kept by the lane that ends up with a row's
// total.  Sixteen warps an SM with 8 KB in flight each keep the memory busy without a ring in shared memory and
// without the per-wave launch and load latency of the register-resident head above (one wave of 296 blocks holds a
// third of a 32 MB head; a 256 MB head would take 26 waves).
// ---------------------------------------------------------------------------------
template <int NCH, int R>   // NCH chunks of 256 columns per row, R rows per batch
__global__ void __launch_bounds__(HEAD1_THREADS, 2) head_stream_kernel(HeadArgs a) {
  constexpr int NW = HEAD1_THREADS / 32, SH = R == 8 ? 2 : R == 4 ? 3 : 4;   // lane >> SH: the row of the batch this lane ends up with
  __shared__ Partial s_p[HEAD1_THREADS];
  __shared__ int s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int K = a.K, V = a.V;
  const int tw = gridDim.x * NW, gw = blockIdx.x * NW + warp;
  const int per = ((V + tw - 1) / tw + R - 1) / R * R;   // rows per warp, whole batches
  const int w0 = min(V, gw * per), w1 = min(V, w0 + per);
  const __nv_bfloat16* W = (const __nv_bfloat16*)a.W;
  uint4 w[R][NCH];
  auto request = [&](int b) {
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int p = 0; p < NCH; ++p) {
        const int c = p * 256 + lane * 8;
        if (c < K) {
          const __nv_bfloat16* src = W + (size_t)min(b + r, V - 1) * K + c;
          asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w[r][p].x), "=r"(w[r][p].y), "=r"(w[r][p].z), "=r"(w[r][p].w) : "l"(src));
        }
      }
  };
  if (w0 < w1) request(w0);
  float gn[NCH][8];   // the norm gains are weights too
  if (a.gain) {
#pragma unroll
    for (int p = 0; p < NCH; ++p) {
      const int c = p * 256 + lane * 8;
      if (c < K) {
        const float4 g0 = __ldg(reinterpret_cast<const float4*>(a.gain + c)), g1 = __ldg(reinterpret_cast<const float4*>(a.gain + c + 4));
        gn[p][0] = g0.x; gn[p][1] = g0.y; gn[p][2] = g0.z; gn[p][3] = g0.w; gn[p][4] = g1.x; gn[p][5] = g1.y; gn[p][6] = g1.z; gn[p][7] = g1.w;
      }
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  const int target = a.desc ? a.desc->targets[0] : (a.target ? a.target[0] : -1);
  float h[NCH][8], ss = 0.f;
#pragma unroll
  for (int p = 0; p < NCH; ++p) {
    const int c = p * 256 + lane * 8;
#pragma unroll
    for (int i = 0; i < 8; ++i) h[p][i] = 0.f;
    if (c < K) {
      const float4 x0 = __ldcg(reinterpret_cast<const float4*>(a.X + c)), x1 = __ldcg(reinterpret_cast<const float4*>(a.X + c + 4));
      h[p][0] = x0.x; h[p][1] = x0.y; h[p][2] = x0.z; h[p][3] = x0.w; h[p][4] = x1.x; h[p][5] = x1.y; h[p][6] = x1.z; h[p][7] = x1.w;
      if (a.gain) {
#pragma unroll
        for (int i = 0; i < 8; ++i) { ss += h[p][i] * h[p][i]; h[p][i] *= gn[p][i]; }
      }
    }
  }
  ss = warp_sum(ss);
  const float mul = (a.gain ? rsqrtf(ss / (float)K + a.eps) : 1.f) * a.scale;
  Partial run;
  run.m = -INFINITY; run.s = 0.f; run.idx = 0x7fffffff;
#pragma unroll 1
  for (int b = w0; b < w1; b += R) {
    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float t = 0.f;
#pragma unroll
      for (int p = 0; p < NCH; ++p) {
        if (p * 256 + lane * 8 < K) {
          const uint4 q = w[r][p];
          t += __uint_as_float(q.x << 16) * h[p][0] + __uint_as_float(q.x & 0xffff0000u) * h[p][1] + __uint_as_float(q.y << 16) * h[p][2] +
               __uint_as_float(q.y & 0xffff0000u) * h[p][3] + __uint_as_float(q.z << 16) * h[p][4] + __uint_as_float(q.z & 0xffff0000u) * h[p][5] +
               __uint_as_float(q.w << 16) * h[p][6] + __uint_as_float(q.w & 0xffff0000u) * h[p][7];
        }
      }
      acc[r] = t;
    }
    if (b + R < w1) request(b + R);   // the next batch is on its way while this one is reduced
    const float z = treduce<R>(acc, lane) * mul;
    const int n = b + (lane >> SH);
    if ((lane & ((1 << SH) - 1)) == 0 && n < w1) {
      if (z > run.m) { run.s = run.s * __expf(run.m - z) + 1.f; run.m = z; run.idx = n; }
      else run.s += __expf(z - run.m);
      if (n == target) a.out->gather[0] = z;
      if (a.logits_dbg) a.logits_dbg[n] = z;
    }
  }
  // rows of a batch are in index order over the lanes, batches in index order over time: combining the lanes in lane
  // order keeps the lowest index among equal maxima
#pragma unroll
  for (int o = 1 << SH; o < 32; o <<= 1) {
    Partial q;
    q.m = __shfl_xor_sync(0xffffffffu, run.m, o);
    q.s = __shfl_xor_sync(0xffffffffu, run.s, o);
    q.idx = __shfl_xor_sync(0xffffffffu, run.idx, o);
    run = ((lane & o) == 0) ? combine(run, q) : combine(q, run);
  }
  if (lane == 0) s_p[warp] = run;
  __syncthreads();
  if (threadIdx.x == 0) {
    Partial p = s_p[0];
    for (int w2 = 1; w2 < NW; ++w2) p = combine(p, s_p[w2]);
    a.partials[blockIdx.x] = p;
    __threadfence();
    const unsigned t = atomicAdd(a.counter, 1u);
    s_last = (t == gridDim.x - 1);
    if (s_last) *a.counter = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  {   // merge: the grid has at most two blocks per SM, one partial each
    Partial p;
    p.m = -INFINITY; p.s = 0.f; p.idx = 0x7fffffff;
    for (int b = threadIdx.x; b < (int)gridDim.x; b += HEAD1_THREADS) {
      Partial t2;
      t2.m = __ldcg(&a.partials[b].m); t2.s = __ldcg(&a.partials[b].s); t2.idx = __ldcg(&a.partials[b].idx);
      p = combine(p, t2);
    }
    s_p[threadIdx.x] = p;
  }
  __syncthreads();
  for (int stride = HEAD1_THREADS / 2; stride > 0; stride >>= 1) {
    if (threadIdx.x < stride) s_p[threadIdx.x] = combine(s_p[threadIdx.x], s_p[threadIdx.x + stride]);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const Partial p = s_p[0];
    HeadOut* o = a.out;
    o->argmax[0] = p.idx;
    o->zmax[0] = p.m;
    o->lse[0] = p.m + logf(p.s);
    o->pmax = 1.f / p.s;
    o->gather[0] = __ldcg(&o->gather[0]);
    policy_tail(a, o);
  }
}

// ---------------------------------------------------------------------------------
// Decode attention, compact version of the block attention above for the decoder passes
// (modes 0 and 1 only).  Keys and values of the block's split are staged in shared memory
// (cross-attention: before the dependency wait), scores are taken one (row, key) pair per
// thread, soft-max one warp per row, values one (row, channel) pair per thread.  Loops are
// kept rolled: the kernel runs for a few microseconds and its instructions must stay cached.
// ---------------------------------------------------------------------------------
constexpr int DATT_THREADS = 128;

struct DAttnArgs {
  BAttnArgs b;
  int MB;          // rows of the q / out buffers and of the scratch layout (1 or MAXB)
  int dkv_shift;   // log2(dkv)
};

__device__ __forceinline__ void dattn_stage(const BAttnArgs& a, int h, int j0, int nk, int dshift, float* sK, float* sV) {
  const int dkv = a.dkv, kst = dkv + 4, q4s = dshift - 2;
  const float* Kg = a.kc + ((size_t)h * a.cap + j0) * dkv;
  const float* Vg = a.vc + ((size_t)h * a.cap + j0) * dkv;
#pragma unroll 1
  for (int idx = threadIdx.x; idx < (nk << q4s); idx += blockDim.x) {
    const int jj = idx >> q4s, e4 = (idx & ((1 << q4s) - 1)) << 2;
    cp_async16(sK + jj * kst + e4, Kg + jj * dkv + e4);
    cp_async16(sV + jj * dkv + e4, Vg + jj * dkv + e4);
  }
}

// grid (heads, splits); the splits of a head form one thread-block cluster, whose blocks hand
// their partial results to the first block through distributed shared memory.  Inside a block
// warp w owns rows w, w+nw, ...; for a single row (MB == 1) the block's warps instead share the
// row, each taking every nw-th key and writing its own slot of the merge area.
__global__ void __launch_bounds__(256) dattn_kernel(DAttnArgs d) {
  extern __shared__ float s_dyn[];   // q [MB][dkv] | scores [MB][sk] | keys [sk][dkv+4] | values [sk][dkv] | merge [slots][MB][dkv+2]
  const BAttnArgs& a = d.b;
  const int MB = d.MB, dshift = d.dkv_shift;
  const int h = blockIdx.x, sp = blockIdx.y, ns = a.nsplit;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
  const int dkv = a.dkv, sk = a.smem_keys, kst = dkv + 4, pst = dkv + 2;
  const int wsplit = 1;   // warps sharing one row (sharing did not pay: the merge grows with the slots)
  float* sQ = s_dyn;
  float* sS = sQ + MB * dkv;
  float* sK = sS + MB * sk;
  float* sV = sK + sk * kst;
  float* sM = sV + sk * dkv;
  if (ns > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  int j0 = 0, nk = 0;
  if (a.mode == 0) {   // encoder keys never change while decoding: fetch before the dependency wait
    const int n_all = min(*a.n_keys_dev, a.cap);
    const int ch = (n_all + ns - 1) / ns;
    j0 = sp * ch;
    nk = min(max(0, min(n_all, j0 + ch) - j0), sk);
    dattn_stage(a, h, j0, nk, dshift, sK, sV);
  }
  pdl_launch_dependents();
  pdl_wait();
  // all MB rows of the query buffer exist: stage them without waiting for the row count
#pragma unroll 1
  for (int idx = tid; idx < (MB << (dshift - 2)); idx += blockDim.x) {
    const int i = idx >> (dshift - 2), e4 = (idx & ((dkv >> 2) - 1)) << 2;
    cp_async16(sQ + i * dkv + e4, a.q + (size_t)i * a.ldq + h * dkv + e4);
  }
  const int M = min(a.desc->k, MB), pos0 = a.desc->pos0;
  if (a.mode == 1) {
    const int n_all = min(pos0 + M, a.cap);
    const int ch = (n_all + ns - 1) / ns;
    j0 = sp * ch;
    nk = min(max(0, min(n_all, j0 + ch) - j0), sk);
    dattn_stage(a, h, j0, nk, dshift, sK, sV);
  }
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_all;" ::: "memory");
  __syncthreads();
  if (ns > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  const int slots = ns * wsplit;
  const int i_first = wsplit > 1 ? 0 : warp, i_step = wsplit > 1 ? 1 : nw;
  // this warp's keys: a contiguous range [k_lo, k_hi)
  const int k_lo = wsplit > 1 ? (nk * warp) / nw : 0, k_hi = wsplit > 1 ? (nk * (warp + 1)) / nw : nk;
#pragma unroll 1
  for (int i = i_first; i < M; i += i_step) {
    const float4* qr = reinterpret_cast<const float4*>(sQ + i * dkv);
    float mx = -INFINITY;
#pragma unroll 1
    for (int jj = k_lo + lane; jj < k_hi; jj += 32) {
      const float4* kr = reinterpret_cast<const float4*>(sK + jj * kst);
      float acc = 0.f;
#pragma unroll 4
      for (int e = 0; e < (dkv >> 2); ++e) {
        const float4 kv = kr[e], qv = qr[e];
        acc += kv.x * qv.x + kv.y * qv.y + kv.z * qv.z + kv.w * qv.w;
      }
      const int j = j0 + jj;
      if (a.mode == 1) acc = (j <= pos0 + i) ? acc + a.bias[(size_t)h * a.bias_ld + (pos0 + i - j)] : -INFINITY;
      sS[i * sk + jj] = acc;
      mx = fmaxf(mx, acc);
    }
    mx = warp_max(mx);
    float sum = 0.f;
#pragma unroll 1
    for (int jj = k_lo + lane; jj < k_hi; jj += 32) {
      const float sc = sS[i * sk + jj];
      const float pr = (sc == -INFINITY) ? 0.f : __expf(sc - mx);
      sS[i * sk + jj] = pr;
      sum += pr;
    }
    sum = warp_sum(sum);
    __syncwarp();
    const bool direct = slots == 1;
    const float rl = direct ? __frcp_rn(sum) : 1.f;
    float* mrow = sM + ((size_t)(sp * wsplit + (wsplit > 1 ? warp : 0)) * MB + i) * pst;   // slot in the first block
#pragma unroll 1
    for (int c = lane; c < dkv; c += 32) {
      float acc0 = 0.f, acc1 = 0.f;   // two chains, added in a fixed order
      int jj = k_lo;
#pragma unroll 2
      for (; jj + 1 < k_hi; jj += 2) {
        acc0 += sS[i * sk + jj] * sV[jj * dkv + c];
        acc1 += sS[i * sk + jj + 1] * sV[(jj + 1) * dkv + c];
      }
      if (jj < k_hi) acc0 += sS[i * sk + jj] * sV[jj * dkv + c];
      const float acc = acc0 + acc1;
      if (direct) a.out[(size_t)i * a.ldo + h * dkv + c] = acc * rl;
      else if (ns > 1) st_cluster_f1(smem_u32(mrow + 2 + c), 0, acc);
      else mrow[2 + c] = acc;
    }
    if (!direct && lane == 0) {
      if (ns > 1) { st_cluster_f1(smem_u32(mrow), 0, mx); st_cluster_f1(smem_u32(mrow + 1), 0, sum); }
      else { mrow[0] = mx; mrow[1] = sum; }
    }
  }
  if (slots == 1) return;
  if (ns > 1) cluster_sync_all(); else __syncthreads();
  if (sp != 0) return;
#pragma unroll 1
  for (int i = warp; i < M; i += nw) {
    float gm = -INFINITY;
#pragma unroll 1
    for (int s2 = 0; s2 < slots; ++s2) gm = fmaxf(gm, sM[((size_t)s2 * MB + i) * pst]);
#pragma unroll 1
    for (int c = lane; c < dkv; c += 32) {
      float num = 0.f, den = 0.f;
#pragma unroll 1
      for (int s2 = 0; s2 < slots; ++s2) {   // slot order
        const float* Ps = sM + ((size_t)s2 * MB + i) * pst;
        const float l = Ps[1];
        const float w = l > 0.f ? __expf(Ps[0] - gm) : 0.f;
        den += l * w;
        num += Ps[2 + c] * w;
      }
      a.out[(size_t)i * a.ldo + h * dkv + c] = num * __frcp_rn(den);
    }
  }
}

}  // namespace bild
