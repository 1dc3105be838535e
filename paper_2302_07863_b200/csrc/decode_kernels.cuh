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
constexpr int GEMV_THREADS = 128;
constexpr int GEMV_PRE = 4;  // column chunks (of 256) whose weights are fetched ahead

// a.ksplit (1, 2 or 4) warps share one group of RW rows, each taking a contiguous K / ksplit
// columns, so that for K up to 4096 every weight byte of the block is requested in one batch
// before the dependency wait; their partial sums are added in warp order through shared memory.
template <typename WT, int RW, bool GATED>
__global__ void __launch_bounds__(GEMV_THREADS) gemv_kernel(LinArgs a) {
  constexpr int NW = GEMV_THREADS / 32;
  __shared__ float s_part[NW][2 * RW + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ks = a.ksplit > 1 ? a.ksplit : 1;
  const int group = warp / ks, kw = warp - group * ks;
  const int n0 = (blockIdx.x * (NW / ks) + group) * RW;
  const int K = a.K, kl = K / ks, kbeg = kw * kl;
  const WT* W0 = (const WT*)a.W0;
  const WT* W1 = (const WT*)a.W1;
  const bool active = n0 < a.N;
  float pre0[RW][GEMV_PRE][8], pre1[GATED ? RW : 1][GATED ? GEMV_PRE : 1][8];
  if (active) {
#pragma unroll
    for (int r = 0; r < RW; ++r) {
      const size_t row = (size_t)min(n0 + r, a.N - 1) * K + kbeg;
#pragma unroll
      for (int p = 0; p < GEMV_PRE; ++p) {
        const int c = p * 256 + lane * 8;
        if (c < kl) {
          load8(W0 + row + c, pre0[r][p]);
          if (GATED) load8(W1 + row + c, pre1[r][p]);
        }
      }
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  const float* X = a.X + kbeg;
  const float* G = a.gain ? a.gain + kbeg : nullptr;
  float acc0[RW], acc1[GATED ? RW : 1], ss = 0.f;
#pragma unroll
  for (int r = 0; r < RW; ++r) { acc0[r] = 0.f; if (GATED) acc1[r] = 0.f; }

  auto fma8 = [&](const float (&w)[8], const float (&h)[8]) {
    return w[0] * h[0] + w[1] * h[1] + w[2] * h[2] + w[3] * h[3] + w[4] * h[4] + w[5] * h[5] + w[6] * h[6] + w[7] * h[7];
  };
  auto load_h = [&](int c, float (&h)[8]) {
    const float4 x0 = *reinterpret_cast<const float4*>(X + c);
    const float4 x1 = *reinterpret_cast<const float4*>(X + c + 4);
    h[0] = x0.x; h[1] = x0.y; h[2] = x0.z; h[3] = x0.w; h[4] = x1.x; h[5] = x1.y; h[6] = x1.z; h[7] = x1.w;
    if (G) {
#pragma unroll
      for (int i = 0; i < 8; ++i) ss += h[i] * h[i];
      const float4 g0 = *reinterpret_cast<const float4*>(G + c);
      const float4 g1 = *reinterpret_cast<const float4*>(G + c + 4);
      h[0] *= g0.x; h[1] *= g0.y; h[2] *= g0.z; h[3] *= g0.w; h[4] *= g1.x; h[5] *= g1.y; h[6] *= g1.z; h[7] *= g1.w;
    }
  };
  if (active) {
    float hp[GEMV_PRE][8];
#pragma unroll
    for (int p = 0; p < GEMV_PRE; ++p) {
      const int c = p * 256 + lane * 8;
      if (c < kl) load_h(c, hp[p]);
    }
#pragma unroll
    for (int p = 0; p < GEMV_PRE; ++p) {
      const int c = p * 256 + lane * 8;
      if (c < kl) {
#pragma unroll
        for (int r = 0; r < RW; ++r) {
          acc0[r] += fma8(pre0[r][p], hp[p]);
          if (GATED) acc1[r] += fma8(pre1[r][p], hp[p]);
        }
      }
    }
    for (int c = GEMV_PRE * 256 + lane * 8; c < kl; c += 256) {   // only for K / ksplit > 1024
      float h[8];
      load_h(c, h);
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        float w[8];
        const size_t row = (size_t)min(n0 + r, a.N - 1) * K + kbeg;
        load8(W0 + row + c, w);
        acc0[r] += fma8(w, h);
        if (GATED) { load8(W1 + row + c, w); acc1[r] += fma8(w, h); }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    acc0[r] = warp_sum(acc0[r]);
    if (GATED) acc1[r] = warp_sum(acc1[r]);
  }
  ss = warp_sum(ss);
  if (ks > 1) {
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < RW; ++r) { s_part[warp][r] = acc0[r]; s_part[warp][RW + r] = GATED ? acc1[r] : 0.f; }
      s_part[warp][2 * RW] = ss;
    }
    __syncthreads();
    if (kw != 0) return;
    ss = 0.f;
#pragma unroll
    for (int r = 0; r < RW; ++r) { acc0[r] = 0.f; if (GATED) acc1[r] = 0.f; }
    for (int w2 = 0; w2 < ks; ++w2) {   // fixed order
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        acc0[r] += s_part[group * ks + w2][r];
        if (GATED) acc1[r] += s_part[group * ks + w2][RW + r];
      }
      ss += s_part[group * ks + w2][2 * RW];
    }
  }
  if (!active) return;
  float inv = 1.f;
  if (a.gain) inv = 1.f / sqrtf(ss / (float)K + a.eps);
  float v0 = 0.f, v1 = 0.f;
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    if (lane == r) { v0 = acc0[r] * inv; if (GATED) v1 = acc1[r] * inv; }
  }
  if (lane >= RW) return;
  const int n = n0 + lane;
  if (n >= a.N) return;
  const int pos0 = a.desc ? a.desc->pos0 : a.pos0_host;
  switch (a.epi) {
    case EPI_STORE: a.Y[n] = v0; break;
    case EPI_RELU: a.Y[n] = fmaxf(v0, 0.f); break;
    case EPI_GATED: a.Y[n] = gelu_tanh(v0) * v1; break;
    case EPI_RESID: a.Y[n] += v0; break;
    default: {
      const int part = a.first_part + n / a.inner;
      const int rr = n % a.inner;
      if (part == 0) {
        a.q_out[rr] = v0;
      } else {
        const int h = rr / a.dkv, c = rr % a.dkv;
        if (pos0 < a.cap) (part == 1 ? a.kc : a.vc)[((size_t)h * a.cap + pos0) * a.dkv + c] = v0;
      }
    }
  }
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
        const float inv = 1.f / sqrtf(sq / (float)K + a.eps);
        v0 *= inv;
        v1 *= inv;
      }
      const int n = n0 + out_r;
      switch (a.epi) {
        case EPI_STORE: a.Y[(size_t)m * a.ldy + n] = v0; break;
        case EPI_RELU: a.Y[(size_t)m * a.ldy + n] = fmaxf(v0, 0.f); break;
        case EPI_GATED: a.Y[(size_t)m * a.ldy + n] = gelu_tanh(v0) * v1; break;
        case EPI_RESID: a.Y[(size_t)m * a.ldy + n] = old[g] + v0; break;
        default: {
          const int part = a.first_part + n / a.inner;
          const int rr = n % a.inner;
          if (part == 0) {
            a.q_out[(size_t)m * a.ldq + rr] = v0;
          } else {
            const int h = rr / a.dkv, c = rr % a.dkv;
            if (pos0 + m < a.cap) (part == 1 ? a.kc : a.vc)[((size_t)h * a.cap + pos0 + m) * a.dkv + c] = v0;
          }
        }
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

}  // namespace bild
