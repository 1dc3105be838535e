// Decode-path kernels of libbild, SIMT versions: embedding gather, RMS-norm-fused
// weight-streaming GEMV / small-M GEMM, attention over the KV caches, the fused LM head
// with online max / log-sum-exp, and the policy bookkeeping of Algorithm 1.
#pragma once
#include "common.cuh"

namespace bild {

// ---------------------------------------------------------------------------------
// Embedding gather: x[m][:] = E[token_m][:]
// ---------------------------------------------------------------------------------
template <typename WT>
__global__ void embed_kernel(const WT* __restrict__ E, const int* __restrict__ tokens,
                             const int* __restrict__ count_dev, int count_host, int d,
                             int vocab, float* __restrict__ x, float* __restrict__ x_zero) {
  const int m = blockIdx.x;
  pdl_launch_dependents();
  pdl_wait();
  const int M = count_dev ? *count_dev : count_host;
  if (m >= M) return;
  int t = tokens[m];
  t = t < 0 ? 0 : (t >= vocab ? vocab - 1 : t);
  const WT* row = E + (size_t)t * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)m * d + c] = to_float(row[c]);
  // the buffer the first fused sub-layer accumulates into starts at zero
  if (x_zero) for (int c = threadIdx.x; c < d; c += blockDim.x) x_zero[(size_t)m * d + c] = 0.f;
}

// ---------------------------------------------------------------------------------
// Linear layer for up to MB rows with one pass over the weights.
//   H = X            (gain == nullptr)
//   H = rms_norm(X)  (gain != nullptr; T5 norm: x * g / sqrt(mean(x^2) + eps))
//   v[m][n] = sum_j W0[n][j] H[m][j]      (and v1 with W1 for the gated FFN)
// Each warp owns RW consecutive weight rows and streams them with 128-bit loads;
// the MB activation rows sit in shared memory, chunked along K.
// ---------------------------------------------------------------------------------
enum { EPI_STORE = 0, EPI_RELU = 1, EPI_GATED = 2, EPI_RESID = 3, EPI_HEADS = 4 };

struct LinArgs {
  const void* W0;
  const void* W1;
  const float* X;
  int ldx;
  const float* gain;
  float eps;
  float* Y;
  int ldy;
  int N, K;
  int M;                 // rows when desc == nullptr
  const CallDesc* desc;  // rows = desc->k, cache position = desc->pos0
  int epi;
  // EPI_HEADS: output row n belongs to part first_part + n / inner (0 = q, 1 = k, 2 = v),
  // head (n % inner) / dkv, channel n % dkv; k and v go to [H][cap][dkv] caches at
  // row pos0 + m, q goes to q_out[m][n % inner].
  int inner, dkv, first_part;
  float* q_out;
  int ldq;
  float* kc;
  float* vc;
  int cap;
  int pos0_host;
  int ksplit;             // gemv_kernel only: warps sharing one row group along K
  int dkv_shift;          // log2(dkv)
  int groups, kl;         // gemv_kernel only: row groups per block, columns per warp
  float inv_k;            // 1 / K
};

constexpr int LIN_THREADS = 256;
constexpr int LIN_KC = 1024;  // K chunk held in shared memory (MB > 1)

template <typename WT, int MB, int RW, bool GATED>
__global__ void __launch_bounds__(LIN_THREADS) linear_kernel(LinArgs a) {
  extern __shared__ float sH[];  // [MB][kc]
  __shared__ float s_scale[MB];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = LIN_THREADS / 32;
  pdl_launch_dependents();
  pdl_wait();
  const int M = a.desc ? a.desc->k : a.M;
  const int m0 = blockIdx.y * MB;
  const int mrows = min(MB, M - m0);
  if (mrows <= 0) return;
  const float* X = a.X + (size_t)m0 * a.ldx;
  const int K = a.K;

  for (int m = warp; m < MB; m += nwarps) {
    float sc = 1.f;
    if (a.gain && m < mrows) {
      float ss = 0.f;
      for (int j = lane; j < K; j += 32) { float v = X[(size_t)m * a.ldx + j]; ss += v * v; }
      ss = warp_sum(ss);
      sc = 1.f / sqrtf(ss / (float)K + a.eps);
    }
    if (lane == 0) s_scale[m] = sc;
  }
  __syncthreads();

  const int kc = (MB == 1) ? K : min(K, LIN_KC);
  const int n0 = (blockIdx.x * nwarps + warp) * RW;
  const WT* W0 = (const WT*)a.W0;
  const WT* W1 = (const WT*)a.W1;

  float acc0[RW][MB], acc1[GATED ? RW : 1][GATED ? MB : 1];
#pragma unroll
  for (int r = 0; r < RW; ++r)
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      acc0[r][m] = 0.f;
      if (GATED) acc1[r][m] = 0.f;
    }

  for (int k0 = 0; k0 < K; k0 += kc) {
    const int kl = min(kc, K - k0);
    if (k0 > 0) __syncthreads();
    for (int idx = threadIdx.x; idx < mrows * kl; idx += LIN_THREADS) {
      const int m = idx / kl, j = idx - m * kl;
      float v = X[(size_t)m * a.ldx + k0 + j] * s_scale[m];
      if (a.gain) v *= a.gain[k0 + j];
      sH[m * kc + j] = v;
    }
    __syncthreads();
    if (n0 < a.N) {
      for (int c = lane * 8; c < kl; c += 256) {
        float w0[RW][8], w1[GATED ? RW : 1][8];
#pragma unroll
        for (int r = 0; r < RW; ++r) {
          const int n = min(n0 + r, a.N - 1);
          load8(W0 + (size_t)n * K + k0 + c, w0[r]);
          if (GATED) load8(W1 + (size_t)n * K + k0 + c, w1[r]);
        }
#pragma unroll
        for (int m = 0; m < MB; ++m) {
          if (m < mrows) {
            const float4 h0 = *reinterpret_cast<const float4*>(&sH[m * kc + c]);
            const float4 h1 = *reinterpret_cast<const float4*>(&sH[m * kc + c + 4]);
#pragma unroll
            for (int r = 0; r < RW; ++r) {
              acc0[r][m] += w0[r][0] * h0.x + w0[r][1] * h0.y + w0[r][2] * h0.z + w0[r][3] * h0.w +
                            w0[r][4] * h1.x + w0[r][5] * h1.y + w0[r][6] * h1.z + w0[r][7] * h1.w;
              if (GATED)
                acc1[r][m] += w1[r][0] * h0.x + w1[r][1] * h0.y + w1[r][2] * h0.z + w1[r][3] * h0.w +
                              w1[r][4] * h1.x + w1[r][5] * h1.y + w1[r][6] * h1.z + w1[r][7] * h1.w;
            }
          }
        }
      }
    }
  }
  if (n0 >= a.N) return;

  // reduce over lanes; lane r*MB+m keeps (r, m)
  float v0 = 0.f, v1 = 0.f;
#pragma unroll
  for (int r = 0; r < RW; ++r)
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      const float s0 = warp_sum(acc0[r][m]);
      if (lane == r * MB + m) v0 = s0;
      if (GATED) {
        const float s1 = warp_sum(acc1[r][m]);
        if (lane == r * MB + m) v1 = s1;
      }
    }
  if (lane >= RW * MB) return;
  const int r = lane / MB, m = lane % MB;
  const int n = n0 + r;
  if (n >= a.N || m >= mrows) return;
  const int pos0 = a.desc ? a.desc->pos0 : a.pos0_host;
  switch (a.epi) {
    case EPI_STORE: a.Y[(size_t)(m0 + m) * a.ldy + n] = v0; break;
    case EPI_RELU: a.Y[(size_t)(m0 + m) * a.ldy + n] = fmaxf(v0, 0.f); break;
    case EPI_GATED: a.Y[(size_t)(m0 + m) * a.ldy + n] = gelu_tanh(v0) * v1; break;
    case EPI_RESID: a.Y[(size_t)(m0 + m) * a.ldy + n] += v0; break;
    default: {
      const int part = a.first_part + n / a.inner;
      const int rr = n % a.inner;
      if (part == 0) {
        a.q_out[(size_t)(m0 + m) * a.ldq + rr] = v0;
      } else {
        const int h = rr / a.dkv, c = rr % a.dkv;
        const int row = pos0 + m0 + m;
        if (row < a.cap) (part == 1 ? a.kc : a.vc)[((size_t)h * a.cap + row) * a.dkv + c] = v0;
      }
    }
  }
}

// ---------------------------------------------------------------------------------
// Attention of one query over a range of cached keys; grid (head, query, split).
// mode 0: cross-attention (no bias, all E keys)
// mode 1: decoder self-attention (query i sees keys 0 .. pos0+i; bias by distance)
// mode 2: encoder self-attention (all E keys; bias by signed distance)
// With nsplit > 1 every split writes (max, sum, weighted V) to scratch and the split
// that arrives last (ticket counter) merges them in split order.
// ---------------------------------------------------------------------------------
struct AttnArgs {
  const float* q;
  int ldq;
  const float* kc;
  const float* vc;
  int cap;  // rows per head in kc / vc
  float* out;
  int ldo;
  const float* bias;  // mode 1: [H][bias_ld] by distance; mode 2: [H][bias_ld] by (j - i + bias_off)
  int bias_ld, bias_off;
  int mode, dkv, H;
  const int* n_keys_dev;  // modes 0 and 2
  int M;
  const CallDesc* desc;
  float* part;  // [(M*H)][nsplit][2 + dkv]
  unsigned* counters;
  int nsplit, smem_keys;
  int* err;
};

constexpr int ATT_THREADS = 128;

__global__ void __launch_bounds__(ATT_THREADS) attn_kernel(AttnArgs a) {
  extern __shared__ float s_sc[];  // [smem_keys] scores, then probabilities
  __shared__ float s_q[128];
  __shared__ float s_red[ATT_THREADS];
  __shared__ float s_stat[2];
  __shared__ int s_last;
  const int h = blockIdx.x, i = blockIdx.y, sp = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int M = a.desc ? a.desc->k : a.M;
  if (i >= M) return;
  const int pos0 = a.desc ? a.desc->pos0 : 0;
  const int dkv = a.dkv;
  int n = (a.mode == 1) ? pos0 + i + 1 : *a.n_keys_dev;
  n = min(n, a.cap);
  const int chunk = (n + a.nsplit - 1) / a.nsplit;
  const int j0 = sp * chunk, j1 = min(n, j0 + chunk);
  if (chunk > a.smem_keys) {  // host sizing error: report, do not touch memory
    if (tid == 0) *a.err = BILD_ERR_CAPACITY;
    return;
  }
  const float* K = a.kc + (size_t)h * a.cap * dkv;
  const float* V = a.vc + (size_t)h * a.cap * dkv;
  if (tid < dkv) s_q[tid] = a.q[(size_t)i * a.ldq + h * dkv + tid];
  __syncthreads();

  // scores
  for (int j = j0 + warp; j < j1; j += ATT_THREADS / 32) {
    float dot = 0.f;
    for (int e = lane; e < dkv; e += 32) dot += s_q[e] * K[(size_t)j * dkv + e];
    dot = warp_sum(dot);
    if (lane == 0) {
      if (a.mode == 1) dot += a.bias[(size_t)h * a.bias_ld + (pos0 + i - j)];
      else if (a.mode == 2) dot += a.bias[(size_t)h * a.bias_ld + (j - i + a.bias_off)];
      s_sc[j - j0] = dot;
    }
  }
  __syncthreads();
  // max
  float mx = -INFINITY;
  for (int j = tid; j < j1 - j0; j += ATT_THREADS) mx = fmaxf(mx, s_sc[j]);
  mx = warp_max(mx);
  if (lane == 0) s_red[warp] = mx;
  __syncthreads();
  if (tid == 0) s_stat[0] = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
  __syncthreads();
  mx = s_stat[0];
  // probabilities and their sum (fixed order: per thread, then lanes, then warps)
  float sum = 0.f;
  for (int j = tid; j < j1 - j0; j += ATT_THREADS) {
    const float p = expf(s_sc[j] - mx);
    s_sc[j] = p;
    sum += p;
  }
  sum = warp_sum(sum);
  __syncthreads();
  if (lane == 0) s_red[warp] = sum;
  __syncthreads();
  if (tid == 0) s_stat[1] = (s_red[0] + s_red[1]) + (s_red[2] + s_red[3]);
  __syncthreads();
  sum = s_stat[1];
  // weighted values: thread (g, c) takes keys j = g mod ng of channel c
  const int ng = ATT_THREADS / dkv;
  const int c = tid % dkv, g = tid / dkv;
  float acc = 0.f;
  if (g < ng)
    for (int j = j0 + g; j < j1; j += ng) acc += s_sc[j - j0] * V[(size_t)j * dkv + c];
  __syncthreads();
  s_red[tid] = acc;
  __syncthreads();
  if (tid < dkv) {
    acc = 0.f;
    for (int gg = 0; gg < ng; ++gg) acc += s_red[gg * dkv + tid];
  }
  if (a.nsplit == 1) {
    if (tid < dkv) a.out[(size_t)i * a.ldo + h * dkv + tid] = acc / sum;
    return;
  }
  const int slot = i * a.H + h;
  float* P = a.part + ((size_t)slot * a.nsplit + sp) * (dkv + 2);
  if (tid < dkv) P[2 + tid] = acc;
  if (tid == 0) { P[0] = mx; P[1] = sum; }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned t = atomicAdd(&a.counters[slot], 1u);
    s_last = (t == (unsigned)a.nsplit - 1);
    if (s_last) a.counters[slot] = 0;  // ready for the next launch
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid < dkv) {
    const float* P0 = a.part + (size_t)slot * a.nsplit * (dkv + 2);
    float gm = -INFINITY;
    for (int s = 0; s < a.nsplit; ++s) gm = fmaxf(gm, __ldcg(&P0[(size_t)s * (dkv + 2)]));
    float num = 0.f, den = 0.f;
    for (int s = 0; s < a.nsplit; ++s) {
      const float* Ps = P0 + (size_t)s * (dkv + 2);
      const float l = __ldcg(&Ps[1]);
      if (l > 0.f) {
        const float w = expf(__ldcg(&Ps[0]) - gm);
        den += l * w;
        num += __ldcg(&Ps[2 + tid]) * w;
      }
    }
    a.out[(size_t)i * a.ldo + h * dkv + tid] = num / den;
  }
}

// ---------------------------------------------------------------------------------
// Relative-position bias by distance: out[h][x] = table[bucket[x]][h]
// ---------------------------------------------------------------------------------
__global__ void bias_table_kernel(const float* __restrict__ table, const int* __restrict__ bucket,
                                  int n, int H, float* __restrict__ out) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= n) return;
  const int b = bucket[x];
  for (int h = 0; h < H; ++h) out[(size_t)h * n + x] = table[b * H + h];
}

// ---------------------------------------------------------------------------------
// Policy bookkeeping of Algorithm 1 (one thread).  `which`: 0 after a small-model
// step, 1 after a large-model block pass.
// ---------------------------------------------------------------------------------
struct LoopPtrs {
  DevState* st;
  int* y;
  bild_trace_rec* trace;
  CallDesc* descS;
  CallDesc* descL;
};

__device__ inline void trace_add(const LoopPtrs& L, int kind, int pos, int token, int k, int m, float v) {
  DevState* st = L.st;
  const int i = st->n_trace++;
  if (i < st->trace_cap) {
    bild_trace_rec r;
    r.kind = kind; r.pos = pos; r.token = token; r.k = k; r.m = m; r.value = v;
    L.trace[i] = r;
  }
}

__device__ inline void next_small(const LoopPtrs& L) {
  DevState* st = L.st;
  L.descS->k = 1;
  L.descS->pos0 = st->S_len;
  L.descS->run_policy = 1;
  L.descS->tokens[0] = L.y[st->n];
  L.descS->targets[0] = -1;
}

__device__ inline void next_large(const LoopPtrs& L) {
  DevState* st = L.st;
  const int k = st->n - st->L_len + 1;
  L.descL->k = k;
  L.descL->pos0 = st->L_len;
  L.descL->run_policy = 1;
  for (int i = 0; i < MAXB; ++i) {
    L.descL->tokens[i] = i < k ? L.y[st->L_len + i] : 0;
    L.descL->targets[i] = i < k - 1 ? L.y[st->L_len + i + 1] : -1;
  }
}

// Tests of Sections 3.3 / 3.4 on the head's per-row results (always run).
__device__ inline void policy_tests(HeadOut* o, const CallDesc* desc, const DevState* st, int which) {
  if (which == 0) {
    o->fallback = (o->pmax < st->alpha_fb) ? 1 : 0;   // fallback iff p_max < alpha_FB
    o->first_violation = -1;
    o->next_token = o->argmax[0];
  } else {
    const int k = desc->k;
    int mv = -1;
    for (int i = 0; i < k - 1; ++i) {
      o->d[i] = o->lse[i] - o->gather[i];             // -ln p_L(drafted token)
      if (mv < 0 && o->d[i] > st->alpha_rb) mv = i;   // first violation of Eq. 3
    }
    o->first_violation = mv;
    o->next_token = o->argmax[mv >= 0 ? mv : k - 1];
    o->fallback = 0;
  }
}

__device__ inline void policy_step(const LoopPtrs& L, const HeadOut* o, const CallDesc* desc, int which) {
  DevState* st = L.st;
  int* y = L.y;
  // Every pass adds a token or consumes a pending draft, so a run takes at most
  // (max_len + 1) * (max_draft + 2) passes; beyond that the loop is stopped with an error.
  if (++st->passes > (st->max_len + 1) * (st->max_draft + 2) + 8) {
    st->err = BILD_ERR_TIMEOUT;
    st->done = 1;
    st->fallback = 0;
    return;
  }
  if (which == 0) {
    const int t = o->argmax[0];
    st->stats.small_steps++;
    st->S_len = desc->pos0 + 1;
    const bool confident = !o->fallback;
    if (st->mode == BILD_MODE_SMALL_ONLY || (confident && st->drafts < st->max_draft)) {
      y[++st->n] = t;
      st->drafts++;
      trace_add(L, 0, st->n, t, 0, -1, o->pmax);
      st->fallback = 0;
      st->done = (st->n >= st->max_len || t == st->eos_id) ? 1 : 0;
      next_small(L);
    } else {
      if (confident) st->stats.forced++; else st->stats.fallbacks++;
      trace_add(L, confident ? 2 : 1, st->n + 1, t, 0, -1, o->pmax);
      st->fallback = 1;
      next_large(L);
    }
  } else {
    const int k = desc->k, base = desc->pos0;
    st->stats.large_calls++;
    st->stats.sum_k += k;
    const int mv = o->first_violation;
    if (mv >= 0) {            // rollback: drop y[j..], write the large model's token at j
      const int j = base + mv + 1;
      st->stats.rollbacks++;
      st->stats.discarded += st->n - j + 1;
      y[j] = o->argmax[mv];
      st->n = j;
      st->S_len = j;
      st->L_len = j;
      trace_add(L, 4, j, y[j], k, mv, o->d[mv]);
    } else {
      float dmax = 0.f;
      for (int i = 0; i < k - 1; ++i) dmax = fmaxf(dmax, o->d[i]);
      y[++st->n] = o->argmax[k - 1];
      st->L_len = st->n;
      trace_add(L, 3, st->n, y[st->n], k, -1, dmax);
    }
    st->drafts = 0;
    st->fallback = 0;
    st->done = (st->n >= st->max_len || y[st->n] == st->eos_id) ? 1 : 0;
    if (st->mode == BILD_MODE_LARGE_ONLY) next_large(L); else next_small(L);
  }
}

// ---------------------------------------------------------------------------------
// Fused LM head: z = scale * W rms_norm(X) for up to MB rows, reduced on the fly to
// arg-max / max / sum-exp per row (the logits never reach memory unless a debug
// buffer is given) plus the logit of each row's target token.  Every block covers a
// contiguous slice of the vocabulary and writes one partial per row; the block that
// arrives last merges the partials in a fixed order, applies the policy tests and,
// if asked, advances the decode loop.
// ---------------------------------------------------------------------------------
struct HeadArgs {
  const void* W;
  const float* X;
  int ldx;
  const float* gain;
  float eps, scale;
  int V, K;
  int M;
  const CallDesc* desc;
  const int* target;  // used when desc == nullptr (may be nullptr)
  Partial* partials;  // [gridDim.x][MB]
  unsigned* counter;
  HeadOut* out;
  float* logits_dbg;
  int which;  // 0 small, 1 large
  LoopPtrs loop;  // loop.st may be nullptr (single-operation entry point)
  // handles of the graph's WHILE (loop goes on) and IF (large pass wanted) nodes; 0 = not in a graph
  unsigned long long cond_while, cond_if;
  unsigned long long cond_if1;   // IF node of the single-row large pass (0: the block branch takes every large pass)
  unsigned long long cond_if8;   // IF node of the large pass over 2 to 8 rows (0: the block branch takes them)
  // one SWITCH node instead of the IF nodes: body 0 the block pass, body 1 the single-row pass, body 2 (if sw_bodies is 3)
  // the pass over 2 to 8 rows; the value sw_bodies runs none
  unsigned long long cond_switch;
  int sw_bodies;
  int pass_kind;                 // which pass counter the kernel bumps inside a loop graph: 0 small, 1 block, 2 single row, 3 up to 8 rows
  int defer_policy;              // sampling: the head leaves policy and loop control to the kernel that draws the token
};

// What the last block of every LM-head kernel does once the per-row results are complete: the policy tests, the
// bookkeeping of Algorithm 1, and (inside a loop graph) the choice of what runs next.
__device__ inline void policy_tail(const HeadArgs& a, HeadOut* o) {
  if (!a.loop.st || a.defer_policy) return;
  policy_tests(o, a.desc, a.loop.st, a.which);
  if (a.desc->run_policy) policy_step(a.loop, o, a.desc, a.which);
  else if (a.which == 0) a.loop.st->S_len = a.desc->pos0 + 1;
  else a.loop.st->L_len = a.desc->pos0 + a.desc->k;
  if (a.cond_while) {
    a.loop.st->cum_passes[a.pass_kind]++;
    cudaGraphSetConditional(a.cond_while, a.loop.st->done ? 0u : 1u);
  }
  // the large pass wanted next: the graph branch for its row count where that branch exists, else the block branch
  const bool fb = a.loop.st->fallback != 0;
  const int kn = a.loop.descL->k;
  const bool one_row = a.cond_if1 && fb && kn == 1;
  const bool upto8 = a.cond_if8 && fb && !one_row && kn <= 8;
  if (a.cond_if) cudaGraphSetConditional(a.cond_if, (fb && !one_row && !upto8) ? 1u : 0u);
  if (a.cond_if1) cudaGraphSetConditional(a.cond_if1, one_row ? 1u : 0u);
  if (a.cond_if8) cudaGraphSetConditional(a.cond_if8, upto8 ? 1u : 0u);
  if (a.cond_switch)
    cudaGraphSetConditional(a.cond_switch, !fb ? (unsigned)a.sw_bodies : kn == 1 ? 1u : (a.sw_bodies == 3 && kn <= 8) ? 2u : 0u);
}

constexpr int HEAD_THREADS = 256;

template <typename WT, int MB, int RW>
__global__ void __launch_bounds__(HEAD_THREADS) lm_head_kernel(HeadArgs a) {
  extern __shared__ float sH[];  // [MB][K]
  __shared__ float s_scale[MB];
  __shared__ Partial s_part[HEAD_THREADS / 32][32];
  __shared__ int s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = HEAD_THREADS / 32;
  pdl_launch_dependents();
  pdl_wait();
  const int M = a.desc ? a.desc->k : a.M;
  const int mrows = min(MB, M);
  const int K = a.K, V = a.V;
  const int* target = a.desc ? a.desc->targets : a.target;

  for (int m = warp; m < MB; m += nwarps) {
    float sc = 1.f;
    if (a.gain && m < mrows) {
      float ss = 0.f;
      for (int j = lane; j < K; j += 32) { float v = a.X[(size_t)m * a.ldx + j]; ss += v * v; }
      ss = warp_sum(ss);
      sc = 1.f / sqrtf(ss / (float)K + a.eps);
    }
    if (lane == 0) s_scale[m] = sc;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < mrows * K; idx += HEAD_THREADS) {
    const int m = idx / K, j = idx - m * K;
    float v = a.X[(size_t)m * a.ldx + j] * s_scale[m];
    if (a.gain) v *= a.gain[j];
    sH[m * K + j] = v;
  }
  __syncthreads();

  const int rpc = (V + gridDim.x - 1) / gridDim.x;
  const int nb = blockIdx.x * rpc, ne = min(V, nb + rpc);
  const WT* W = (const WT*)a.W;
  // lane r*MB+m keeps the running statistics of (row parity r, token row m)
  const int my_r = lane / MB, my_m = lane % MB;
  const int my_target = (lane < RW * MB && my_m < mrows && target) ? target[my_m] : -1;
  Partial run;
  run.m = -INFINITY; run.s = 0.f; run.idx = 0x7fffffff;

  for (int n0 = nb + warp * RW; n0 < ne; n0 += nwarps * RW) {
    float acc[RW][MB];
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
      for (int m = 0; m < MB; ++m) acc[r][m] = 0.f;
    for (int c = lane * 8; c < K; c += 256) {
      float w[RW][8];
#pragma unroll
      for (int r = 0; r < RW; ++r) load8(W + (size_t)min(n0 + r, V - 1) * K + c, w[r]);
#pragma unroll
      for (int m = 0; m < MB; ++m) {
        if (m < mrows) {
          const float4 h0 = *reinterpret_cast<const float4*>(&sH[m * K + c]);
          const float4 h1 = *reinterpret_cast<const float4*>(&sH[m * K + c + 4]);
#pragma unroll
          for (int r = 0; r < RW; ++r)
            acc[r][m] += w[r][0] * h0.x + w[r][1] * h0.y + w[r][2] * h0.z + w[r][3] * h0.w +
                         w[r][4] * h1.x + w[r][5] * h1.y + w[r][6] * h1.z + w[r][7] * h1.w;
        }
      }
    }
    float z = 0.f;
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
      for (int m = 0; m < MB; ++m) {
        const float s = warp_sum(acc[r][m]);
        if (lane == r * MB + m) z = s;
      }
    const int n = n0 + my_r;
    if (lane < RW * MB && my_m < mrows && n < ne) {
      z *= a.scale;
      if (z > run.m) { run.s = run.s * expf(run.m - z) + 1.f; run.m = z; run.idx = n; }
      else run.s += expf(z - run.m);
      if (n == my_target) a.out->gather[my_m] = z;
      if (a.logits_dbg) a.logits_dbg[(size_t)my_m * V + n] = z;
    }
  }
  s_part[warp][lane] = run;
  __syncthreads();
  if (threadIdx.x < mrows) {
    Partial p;
    p.m = -INFINITY; p.s = 0.f; p.idx = 0x7fffffff;
    for (int w = 0; w < nwarps; ++w)
      for (int r = 0; r < RW; ++r) p = combine(p, s_part[w][r * MB + threadIdx.x]);
    a.partials[(size_t)blockIdx.x * MB + threadIdx.x] = p;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned t = atomicAdd(a.counter, 1u);
    s_last = (t == gridDim.x - 1);
    if (s_last) *a.counter = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int m = warp; m < mrows; m += nwarps) {
    Partial p;
    p.m = -INFINITY; p.s = 0.f; p.idx = 0x7fffffff;
    for (int b = lane; b < (int)gridDim.x; b += 32) {
      Partial q;
      const Partial* src = &a.partials[(size_t)b * MB + m];
      q.m = __ldcg(&src->m); q.s = __ldcg(&src->s); q.idx = __ldcg(&src->idx);
      p = combine(p, q);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      Partial q;
      q.m = __shfl_xor_sync(0xffffffffu, p.m, o);
      q.s = __shfl_xor_sync(0xffffffffu, p.s, o);
      q.idx = __shfl_xor_sync(0xffffffffu, p.idx, o);
      // both lanes of a pair must end with the same value: order the operands by lane
      p = ((lane & o) == 0) ? combine(p, q) : combine(q, p);
    }
    if (lane == 0) {
      a.out->argmax[m] = p.idx;
      a.out->zmax[m] = p.m;
      a.out->lse[m] = p.m + logf(p.s);
      if (m == 0) a.out->pmax = 1.f / p.s;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    HeadOut* o = a.out;
    // gather[] was written by other blocks before their tickets: read around L1
    for (int m = 0; m < mrows; ++m) o->gather[m] = __ldcg(&o->gather[m]);
    policy_tail(a, o);
  }
}

// ---------------------------------------------------------------------------------
// Small set-up kernels (one thread)
// ---------------------------------------------------------------------------------
struct TokList { int t[MAXB]; };

__global__ void set_desc_kernel(CallDesc* d, const DevState* st, int which, int k, TokList toks) {
  d->k = k;
  d->pos0 = which == 0 ? st->S_len : st->L_len;
  d->run_policy = 0;
  for (int i = 0; i < MAXB; ++i) {
    d->tokens[i] = i < k ? toks.t[i] : 0;
    d->targets[i] = i < k - 1 ? toks.t[i + 1] : -1;
  }
}

__global__ void set_desc_at_kernel(CallDesc* d, int k, int pos0, TokList toks) {
  d->k = k;
  d->pos0 = pos0;
  d->run_policy = 0;
  for (int i = 0; i < MAXB; ++i) {
    d->tokens[i] = i < k ? toks.t[i] : 0;
    d->targets[i] = i < k - 1 ? toks.t[i + 1] : -1;
  }
}

// A block of 9 to 16 rows as two chunks for the fused sub-layer kernels: rows 0..7 and the rest, the second chunk at
// the cache position right after the first.
__global__ void split_desc_kernel(const CallDesc* d, CallDesc* lo, CallDesc* hi) {
  const int k = d->k, klo = k < SUB_CHUNK ? k : SUB_CHUNK;
  lo->k = klo; lo->pos0 = d->pos0; lo->run_policy = 0;
  hi->k = k - klo; hi->pos0 = d->pos0 + klo; hi->run_policy = 0;
}

__global__ void set_alpha_kernel(DevState* st, float alpha_fb, float alpha_rb) {
  st->alpha_fb = alpha_fb;
  st->alpha_rb = alpha_rb;
}

__global__ void rewind_kernel(DevState* st, int which, int new_len) {
  if (which == 0) st->S_len = new_len; else st->L_len = new_len;
}

__global__ void reset_state_kernel(LoopPtrs L, int mode, float alpha_fb, float alpha_rb, int max_len,
                                   int max_draft, int eos_id, int start_id, int trace_cap, float top_p) {
  DevState* st = L.st;
  st->top_p = top_p;
  st->n = 0; st->S_len = 0; st->L_len = 0; st->drafts = 0;
  st->fallback = 0; st->mode = mode; st->err = 0;
  st->max_len = max_len; st->max_draft = max_draft; st->eos_id = eos_id; st->start_id = start_id;
  st->alpha_fb = alpha_fb; st->alpha_rb = alpha_rb;
  st->n_trace = 0; st->trace_cap = trace_cap;
  st->stats = bild_stats{0, 0, 0, 0, 0, 0, 0};
  st->passes = 0;
  L.y[0] = start_id;
  st->done = (max_len <= 0 || start_id == eos_id) ? 1 : 0;
  if (mode == BILD_MODE_LARGE_ONLY) next_large(L); else next_small(L);
}

}  // namespace bild
