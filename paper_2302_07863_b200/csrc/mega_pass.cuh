// One decoder pass (steps S0..S8 / L0..L8 of every layer) as ONE persistent kernel, bf16 weights.
//
// A decoder pass at batch 1 is a chain of 8 dependent stages per layer, each of which moves far
// less data than it takes to hide the memory latency, so a chain of separate kernels is bound
// by launch and memory latency.  Here one block per SM stays resident for the whole pass:
//   * a producer warp streams the block's slice of every weight matrix, in program order,
//     through a ring of shared-memory slots with bulk (TMA) copies.  The weights do not depend
//     on the activations, so the stream runs ahead of the dependency chain and a stage finds
//     its weights already on chip;
//   * eight consumer warps run the stages.  There is no grid-wide barrier: every activation
//     that crosses blocks travels as an 8-byte (value, epoch) pair written with one store, and
//     a reader polls the pairs it needs until they carry the epoch of the stage it is in
//     (one epoch per stage and launch).  A stage therefore starts in a block as soon as that
//     block's own inputs have arrived, one L2 round trip after they were written;
//   * a linear stage splits the output rows over the blocks (no cross-block reduction); inside
//     a block a work item is 4 weight rows x 256 columns for all token rows, partial sums are
//     added in a fixed order.  The block that owns a slice of the model dimension keeps the
//     residual stream of that slice in shared memory;
//   * attention splits (head, row group, key range) over the blocks; cached keys / values are
//     staged in 64-key chunks (bulk copies, double buffered, issued before the queries arrive)
//     with a running soft-max, the rows of the current block of tokens arrive as pairs; the
//     first split of a (head, row group) merges the others' (max, sum, weighted values).
// Every wait gives up after a fixed number of polls: the block then records BILD_ERR_TIMEOUT,
// stops waiting anywhere, and runs to the end.
#pragma once
#include "common.cuh"

namespace bild {

constexpr int MG_CONSUMERS = 256;                   // 8 consumer warps
constexpr int MG_THREADS = MG_CONSUMERS;
constexpr int MG_FEEDER = MG_CONSUMERS - 1;        // the thread that issues the weight copies
constexpr int MG_SLOT = 8192;                       // bytes per ring slot
constexpr int MG_ACT = 80 * 1024;                   // activation staging
constexpr int MG_QUADS = 12;                        // weight-row quads per stage and block (48 rows)
constexpr int MG_PSUM = MG_QUADS * 8 * 32 * 4;      // partial sums [quad][warp][32]; attention scratch
constexpr int MG_MAX_SLOTS = 20;
constexpr int MG_MAX_BLOCKS = 256;                 // record areas are sized for this many blocks
constexpr int MG_MISC = 7168;
constexpr int MG_MAX_LAYERS = 56;                  // the per-layer pointer table is copied to shared memory
constexpr int MG_PST_PAD = 4;                       // record = [max, sum, 0, 0, values[dkv]]
constexpr int MG_XRES = 16;                         // columns of the model dimension one block may own
constexpr unsigned MG_SPIN = 1u << 20;
constexpr int MG_EPOCHS_PER_LAUNCH = 1024;          // > 8 * layers

struct MegaLayer {
  const __nv_bfloat16 *wqkv, *wo, *wcq, *wco, *wi0, *wi1, *wfo;
  const float *ln1, *ln2, *ln3;
};

// (value, epoch) pairs of the eight stage outputs, each for MAXB token rows
struct MegaLL {
  uint2 *qkv1;  // [H][MAXB][3][dkv]  query | key | value of the rows of this pass, by head
  uint2 *a2;    // [MAXB][I]      self-attention output
  uint2 *r2;    // records of the key splits, self-attention
  uint2 *x3;    // [MAXB][d]
  uint2 *q4;    // [H][MAXB][dkv]  cross-attention queries, by head
  uint2 *a5;    // [MAXB][I]
  uint2 *r5;
  uint2 *x6;    // [MAXB][d]
  uint2 *u7;    // [MAXB][F]
  uint2 *x8;    // [MAXB][d]
};

struct MegaArgs {
  const MegaLayer* layers;
  int n_layers;
  int d, I, F, H, dkv, dkv_shift, gated, vocab;
  float eps;
  const CallDesc* desc;
  const __nv_bfloat16* emb;
  float* x;                   // [MAXB][d] residual stream after the last layer (input of the LM head)
  float *selfK, *selfV;
  const float *crossK, *crossV;
  int cap, ecap;
  const float* dec_bias;      // [H][cap] by distance
  const int* enc_len;
  unsigned* sync;             // [0]: launches so far (epoch base)
  int* err;
  int nslots;
  MegaLL ll;
};

inline size_t mega_smem_bytes(int nslots) { return (size_t)nslots * MG_SLOT + MG_ACT + MG_PSUM + MG_MISC; }
// pairs in one record area: per (head, row group) up to 7 later splits x 4 rows
inline size_t mega_record_pairs(int blocks, int dkv) { return (size_t)blocks * 32 * (dkv + MG_PST_PAD); }

// ---- small PTX helpers ----------------------------------------------------------------
__device__ __forceinline__ void mg_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mg_mbar_expect(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mg_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mg_mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void mg_bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void mg_csync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }   // consumer warps only
__device__ __forceinline__ void mg_ll_store(uint2* p, float v, uint32_t ep) {
  asm volatile("st.volatile.global.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(__float_as_uint(v)), "r"(ep) : "memory");
}
__device__ __forceinline__ uint4 mg_ll_load2(const uint2* p) {   // two pairs, 16-byte aligned
  uint4 v;
  asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}

// Block-wide state in shared memory.
struct MegaShared {
  unsigned long long full[MG_MAX_SLOTS], kvbar[2];   // full[i]: all slices of the i-th (mod) linear stage have landed
  MegaLayer layers[MG_MAX_LAYERS];
  int slice[6][2];                      // rows of the six matrices that belong to this block
  float inv[MAXB];                      // 1 / rms of the staged rows
  float ssq[8][MAXB];                   // sum of squares of the staged rows, per warp
  float amax[4], asum[4], ascale[4];    // running soft-max of the unit's rows
  unsigned rowoff[4 * MG_QUADS];        // byte offset of every slice row in the ring
  float xres[MAXB][MG_XRES];            // residual stream of the columns this block owns
  int failed;
};

__device__ __forceinline__ void mg_fail(MegaShared* sh, int* err) {
  sh->failed = 1;
  atomicExch(err, (int)BILD_ERR_TIMEOUT);
}
// bounded mbarrier wait; after a failure nothing waits any more
__device__ __forceinline__ void mg_wait(MegaShared* sh, int* err, unsigned long long* bar, uint32_t parity) {
  const uint32_t b = smem_u32(bar);
  if (mg_mbar_try(b, parity)) return;
  if (*(volatile int*)&sh->failed) return;
  for (unsigned it = 0; it < MG_SPIN; ++it)
    if (mg_mbar_try(b, parity)) return;
  mg_fail(sh, err);
}

// Polls the n2 16-byte units (two pairs each) at src until they carry epoch ep and writes the
// 2 * n2 values to dst (shared memory, same order).  All consumer threads call it; at most 8
// units per thread are in flight at a time.
__device__ __noinline__ void mg_ll_fetch(const uint2* src, int n2, float* dst, uint32_t ep, MegaShared* sh, int* err) {
  const int tid = threadIdx.x;
#pragma unroll 1
  for (int b0 = tid; b0 < n2; b0 += MG_CONSUMERS * 8) {
    unsigned pend = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (b0 + j * MG_CONSUMERS < n2) pend |= 1u << j;
    unsigned it = 0;
    while (pend) {
      uint4 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (pend & (1u << j)) v[j] = mg_ll_load2(src + 2 * (size_t)(b0 + j * MG_CONSUMERS));
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if ((pend & (1u << j)) && v[j].y == ep && v[j].w == ep) {
          *reinterpret_cast<float2*>(dst + 2 * (size_t)(b0 + j * MG_CONSUMERS)) =
              make_float2(__uint_as_float(v[j].x), __uint_as_float(v[j].z));
          pend &= ~(1u << j);
        }
      if (pend && (++it > MG_SPIN || *(volatile int*)&sh->failed)) {
        if (it > MG_SPIN) mg_fail(sh, err);
        break;
      }
    }
  }
}

// The six weight matrices of a layer in the order the stages use them.
struct MegaLin {
  const __nv_bfloat16 *W0, *W1;   // W1: second matrix of the gated FFN
  int N, K;
};
__device__ __forceinline__ MegaLin mg_lin(const MegaArgs& a, const MegaLayer& L, int p) {
  MegaLin r;
  r.W1 = nullptr;
  switch (p) {
    case 0: r.W0 = L.wqkv; r.N = 3 * a.I; r.K = a.d; break;
    case 1: r.W0 = L.wo; r.N = a.d; r.K = a.I; break;
    case 2: r.W0 = L.wcq; r.N = a.I; r.K = a.d; break;
    case 3: r.W0 = L.wco; r.N = a.d; r.K = a.I; break;
    case 4: r.W0 = L.wi0; r.W1 = a.gated ? L.wi1 : nullptr; r.N = a.F; r.K = a.d; break;
    default: r.W0 = L.wfo; r.N = a.d; r.K = a.F; break;
  }
  return r;
}
// rows [r0, r1) of an N-row matrix that block b of G owns
__device__ __forceinline__ void mg_slice(int N, int b, int G, int* r0, int* r1) {
  *r0 = (int)(((long long)b * N) / G);
  *r1 = (int)(((long long)(b + 1) * N) / G);
}

// ---- the block's weight slices, in program order, through the ring ------------------------
// One thread owns the stream: it fills every slot at the start and refills the slots of a stage
// as soon as the stage has used them (it frees them itself, so it never waits).
struct MegaFeed {
  int l, p, mat, r, r1, rps, K;          // next copy: layer, matrix, row range of this block's slice
  const __nv_bfloat16* W;
  int slot;                              // next slot to fill
  int stage;                             // linear stages of this block fully issued so far (mod MG_MAX_SLOTS)
  bool second;                           // the matrix under way has a successor in the same stage
  bool done;
};
__device__ __forceinline__ void mg_feed_open(const MegaArgs& a, const MegaShared* sh, MegaFeed& f) {   // positions f at (f.l, f.p, f.mat)
  while (f.l < a.n_layers) {
    const MegaLin w = mg_lin(a, sh->layers[f.l], f.p);
    const int r0 = sh->slice[f.p][0];
    f.r1 = sh->slice[f.p][1];
    if (f.r1 > r0) {
      f.r = r0; f.K = w.K; f.rps = MG_SLOT / (w.K * 2); f.W = f.mat ? w.W1 : w.W0;
      f.second = w.W1 && f.mat == 0;
      return;
    }
    if (++f.p == 6) { f.p = 0; ++f.l; }   // no rows of this matrix belong to the block
  }
  f.done = true;
}
__device__ __forceinline__ void mg_feed_init(const MegaArgs& a, const MegaShared* sh, MegaFeed& f) {
  f.l = 0; f.p = 0; f.mat = 0; f.slot = 0; f.stage = 0; f.done = false;
  mg_feed_open(a, sh, f);
}
// fills `count` slots (fewer if the program ends); the last copy of a stage also arrives on its barrier
__device__ __noinline__ void mg_feed(const MegaArgs& a, MegaShared* sh, unsigned char* ring, MegaFeed& f, int count) {
  for (int i = 0; i < count && !f.done; ++i) {
    const int nr = min(f.rps, f.r1 - f.r);
    const uint32_t bytes = (uint32_t)(nr * f.K * 2);
    const uint32_t bar = smem_u32(&sh->full[f.stage]);
    const bool last = f.r + nr >= f.r1 && !f.second;
    if (last) mg_mbar_expect(bar, bytes);
    else asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    mg_bulk_g2s(smem_u32(ring + (size_t)f.slot * MG_SLOT), f.W + (size_t)f.r * f.K, bytes, bar);
    if (++f.slot == a.nslots) f.slot = 0;
    f.r += nr;
    if (f.r >= f.r1) {
      if (f.second) f.mat = 1;
      else {
        f.mat = 0;
        if (++f.p == 6) { f.p = 0; ++f.l; }
        if (++f.stage == MG_MAX_SLOTS) f.stage = 0;
      }
      mg_feed_open(a, sh, f);
    }
  }
}

// ---- sum of NP register values across the warp, one shuffle per halving ------------------
// Returns in every lane the warp-wide sum of v[lane >> (5 - log2 NP)].
template <int NP>
__device__ __forceinline__ float mg_treduce(float (&v)[NP], int lane) {
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

// Work items of a linear stage: (quad of weight rows, 256 columns) x MG token rows.  Item it
// belongs to quad it / nkb and column block it % nkb; warp w takes items w, w + 8, ...  (rows past
// the end of the slice repeat its last row; nobody reads their sums)
template <int MG>
__device__ __forceinline__ void mg_items(const unsigned char* ring, const unsigned* rowoff, int nrows, int K, const float* Xs,
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
    unsigned off[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) off[r] = rowoff[min(qd * 4 + r, nrows - 1)];
#pragma unroll 1
    for (; kb < nkb; kb += 8) {
      const int kofs = (kb << 8) + lane * 8;
      if (kofs < K) {
        uint4 w[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) w[r] = *reinterpret_cast<const uint4*>(ring + off[r] + (size_t)kofs * 2);
#pragma unroll
        for (int m = 0; m < MG; ++m) {
          const float4 x0 = *reinterpret_cast<const float4*>(Xs + (size_t)m * K + kofs);
          const float4 x1 = *reinterpret_cast<const float4*>(Xs + (size_t)m * K + kofs + 4);
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
    const float r = mg_treduce<NP>(acc, lane);
    if ((lane & (32 / NP - 1)) == 0) psum[(qd * 8 + warp) * 32 + (lane >> SH)] = r;
  }
}

// Token rows are taken 1, 2, 4 or 8 at a time (rows beyond mg hold stale values whose sums nobody reads).
__device__ __forceinline__ int mg_round_rows(int mg) { return mg <= 2 ? mg : mg <= 4 ? 4 : 8; }
__device__ __forceinline__ void mg_items_dyn(int mgr, const unsigned char* ring, const unsigned* rowoff, int nrows, int K,
                                             const float* Xs, float* psum, int warp, int lane) {
  switch (mgr) {
    case 1: mg_items<1>(ring, rowoff, nrows, K, Xs, psum, warp, lane); break;
    case 2: mg_items<2>(ring, rowoff, nrows, K, Xs, psum, warp, lane); break;
    case 4: mg_items<4>(ring, rowoff, nrows, K, Xs, psum, warp, lane); break;
    default: mg_items<8>(ring, rowoff, nrows, K, Xs, psum, warp, lane); break;
  }
}

// How attention over M rows and nkeys keys is split over the blocks.
struct MegaAttnPlan {
  int rg;      // rows per unit
  int nrg;     // row groups
  int ns;      // key splits
  int ck;      // keys per staged chunk
  int per;     // keys per split
};
__device__ __forceinline__ MegaAttnPlan mg_attn_plan(const MegaArgs& a, int M, int nkeys, int G) {
  MegaAttnPlan p;
  const int rgmax = max(1, min(4, 256 >> a.dkv_shift));
  p.nrg = (M + rgmax - 1) / rgmax;
  p.rg = (M + p.nrg - 1) / p.nrg;
  p.ck = a.dkv > 64 ? 16 : 64;   // chunk buffers (2 x keys + values) take at most 64 KB of the staging area
  int ns = max(1, G / (a.H * p.nrg));
  ns = min(ns, max(1, nkeys / 32));
  p.ns = min(ns, 8);
  p.per = (nkeys + p.ns - 1) / p.ns;
  return p;
}

// ---- attention stage ---------------------------------------------------------------------
// mode 0: cross (all encoder keys, no bias), mode 1: self (row i sees keys 0..pos0+i, bias by distance)
__device__ void mg_attention(const MegaArgs& a, MegaShared* sh, float* act, float* scratch, int layer, int mode, int M, int pos0,
                             int nkeys, const MegaAttnPlan& P, const uint2* llin, uint2* llout, uint2* llrec, uint32_t ep_in,
                             uint32_t ep_out, unsigned& kvfill, unsigned char* ring, MegaFeed& feed, int& pending) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, H = a.H, dkv = a.dkv, dsh = a.dkv_shift;
  const int units = H * P.nrg * P.ns;
  const int kcap = mode == 0 ? a.ecap : a.cap;
  const size_t kvoff = (size_t)layer * H * dkv * kcap;
  const int ck = P.ck, chunk_floats = ck * dkv, pst = dkv + MG_PST_PAD;
  float* sS = scratch;                    // [rg][ck] scores, then probabilities
  float* sBias = scratch + 4 * 64;        // bias by distance, the distances this unit meets
  const int ck_sh = 31 - __clz(ck);
  const int bias_cap = MG_PSUM / 4 - 4 * 64;
  float* sIn = act + 4 * chunk_floats;    // what arrives as pairs: self [M][q | k | v][dkv], cross [rows][dkv]
  float* sRec = act;                      // records of the other splits (after the chunks are done)
  const int in_st = mode == 1 ? 3 * dkv : dkv;   // floats between the rows of sIn
#pragma unroll 1
  for (int u = blockIdx.x; u < units; u += G) {
    mg_csync();   // the scratch area may still be read as the partial sums of the stage before
    if (tid == MG_FEEDER && pending) mg_feed(a, sh, ring, feed, pending);
    pending = 0;
    const int h = u % H, rest = u / H, g = rest % P.nrg, sp = rest / P.nrg;
    const int j0 = min(nkeys, sp * P.per), j1 = min(nkeys, j0 + P.per);
    const int jo1 = mode == 1 ? min(j1, pos0) : j1;                 // cached keys [j0, jo1)
    const int jn0 = mode == 1 ? max(j0, pos0) : j1;                 // keys of this pass [jn0, j1)
    const int nold = jo1 > j0 ? (jo1 - j0 + ck - 1) >> ck_sh : 0;
    const int nchunks = nold + (j1 > jn0 ? 1 : 0);
    const float* Kh = (mode == 0 ? a.crossK : a.selfK) + kvoff + (size_t)h * kcap * dkv;
    const float* Vh = (mode == 0 ? a.crossV : a.selfV) + kvoff + (size_t)h * kcap * dkv;
    const int i0 = g * P.rg, nr = min(P.rg, M - i0);
    // the cache does not change during the pass: its first chunks start before the queries arrive
    const unsigned fill0 = kvfill;
    int issued = 0;   // cached chunks requested so far
    auto issue_to = [&](int upto) {
#pragma unroll 1
      for (; issued < upto; ++issued, ++kvfill) {
        if (tid != 0) continue;
        const int jc = j0 + (issued << ck_sh), nk = min(ck, jo1 - jc);
        const unsigned buf = kvfill & 1;
        const uint32_t bar = smem_u32(&sh->kvbar[buf]), bytes = (uint32_t)(nk * dkv * 4);
        mg_mbar_expect(bar, 2 * bytes);
        mg_bulk_g2s(smem_u32(act + (size_t)buf * 2 * chunk_floats), Kh + (size_t)jc * dkv, bytes, bar);
        mg_bulk_g2s(smem_u32(act + (size_t)buf * 2 * chunk_floats + chunk_floats), Vh + (size_t)jc * dkv, bytes, bar);
      }
    };
    issue_to(min(nold, 2));
    // bias of the distances pos0 + i - j of this unit (a static table)
    const int dmin = max(0, pos0 + i0 - (j1 - 1)), dmax = pos0 + i0 + nr - 1 - j0;
    const bool bias_staged = mode == 1 && dmax - dmin + 1 <= bias_cap;
    if (bias_staged)
      for (int dd = dmin + tid; dd <= dmax; dd += MG_CONSUMERS) sBias[dd - dmin] = __ldg(a.dec_bias + (size_t)h * a.cap + dd);
    // what arrives as pairs: all rows of this head (self: the new keys / values are among them), or the unit's queries
    const float* sQ;
    if (mode == 1) {
      mg_ll_fetch(llin + (size_t)h * MAXB * 3 * dkv, (M * 3 * dkv) >> 1, sIn, ep_in, sh, a.err);
      sQ = sIn + (size_t)i0 * 3 * dkv;
    } else {
      mg_ll_fetch(llin + ((size_t)h * MAXB + i0) * dkv, (nr * dkv) >> 1, sIn, ep_in, sh, a.err);
      sQ = sIn;
    }
    if (tid < 4) { sh->amax[tid] = -INFINITY; sh->asum[tid] = 0.f; sh->ascale[tid] = 1.f; }
    // thread <-> (row, channel) of the weighted values
    const int pv_i = tid >> dsh, pv_c = tid & (dkv - 1);
    const bool pv_on = pv_i < nr;
    float pv_acc = 0.f;
    mg_csync();
    unsigned use = fill0;
#pragma unroll 1
    for (int c = 0; c < nchunks; ++c) {
      const bool cached = c < nold;
      const unsigned buf = use & 1;
      const float* sK = cached ? act + (size_t)buf * 2 * chunk_floats : sIn + (size_t)(jn0 - pos0) * 3 * dkv + dkv;
      const float* sV = cached ? sK + chunk_floats : sK + dkv;
      const int kst = cached ? dkv : 3 * dkv;
      const int jc = cached ? j0 + (c << ck_sh) : jn0, nk = cached ? min(ck, jo1 - jc) : j1 - jn0;
      if (cached) mg_wait(sh, a.err, &sh->kvbar[buf], (use >> 1) & 1);
      // scores: one (row, key) pair per thread; the columns are visited in a rotated order so that
      // the threads of a quarter warp hit different banks
#pragma unroll 1
      for (int idx = tid; idx < (nr << ck_sh); idx += MG_CONSUMERS) {
        const int i = idx >> ck_sh, jj = idx & (ck - 1);
        float sc = -INFINITY;
        const int j = jc + jj;
        if (jj < nk && (mode == 0 || j <= pos0 + i0 + i)) {
          float accs = 0.f;
          const int nq4 = dkv >> 2;
#pragma unroll 4
          for (int e = 0; e < nq4; ++e) {
            const int er = ((e + jj) & (nq4 - 1)) << 2;
            const float4 kv = *reinterpret_cast<const float4*>(sK + jj * kst + er);
            const float4 qv = *reinterpret_cast<const float4*>(sQ + i * in_st + er);
            accs += kv.x * qv.x + kv.y * qv.y + kv.z * qv.z + kv.w * qv.w;
          }
          if (mode == 1) {
            const int dd = pos0 + i0 + i - j;
            accs += bias_staged ? sBias[dd - dmin] : __ldg(a.dec_bias + (size_t)h * a.cap + dd);
          }
          sc = accs;
        }
        sS[idx] = sc;
      }
      mg_csync();
      if (warp < nr) {   // running soft-max of row `warp`
        float mx = -INFINITY;
#pragma unroll 1
        for (int jj = lane; jj < ck; jj += 32) mx = fmaxf(mx, sS[(warp << ck_sh) + jj]);
        mx = warp_max(mx);
        const float mo = sh->amax[warp], mn = fmaxf(mo, mx);
        float sum = 0.f;
#pragma unroll 1
        for (int jj = lane; jj < ck; jj += 32) {
          const float scv = sS[(warp << ck_sh) + jj];
          const float pr = scv == -INFINITY ? 0.f : __expf(scv - mn);
          sS[(warp << ck_sh) + jj] = pr;
          sum += pr;
        }
        sum = warp_sum(sum);
        if (lane == 0) {
          const float scale = mo == -INFINITY ? 0.f : __expf(mo - mn);
          sh->ascale[warp] = scale;
          sh->asum[warp] = sh->asum[warp] * scale + sum;
          sh->amax[warp] = mn;
        }
      }
      mg_csync();
      if (pv_on) {
        float a0 = 0.f, a1 = 0.f;
        const float* pr = sS + (pv_i << ck_sh);
        int jj = 0;
#pragma unroll 2
        for (; jj + 1 < nk; jj += 2) {
          a0 += pr[jj] * sV[jj * kst + pv_c];
          a1 += pr[jj + 1] * sV[(jj + 1) * kst + pv_c];
        }
        if (jj < nk) a0 += pr[jj] * sV[jj * kst + pv_c];
        pv_acc = pv_acc * sh->ascale[pv_i] + (a0 + a1);
      }
      mg_csync();   // the chunk's buffer and the probabilities are free again
      if (cached) {
        issue_to(min(nold, c + 3));
        ++use;
      }
    }
    // finish: a lone split writes the rows, later splits leave records, the first split merges them
    const int slot = (h * P.nrg + g) * 32 * pst;   // pairs: [split - 1][row < rg][pst], at most 7 x 4 rows
    if (sp > 0) {
      if (pv_i < P.rg) {
        uint2* rec = llrec + slot + ((size_t)(sp - 1) * P.rg + pv_i) * pst;
        mg_ll_store(rec + MG_PST_PAD + pv_c, pv_on ? pv_acc : 0.f, ep_out);
        if (pv_c < MG_PST_PAD)
          mg_ll_store(rec + pv_c, pv_c == 0 ? (pv_on ? sh->amax[pv_i] : -INFINITY) : pv_c == 1 ? (pv_on ? sh->asum[pv_i] : 0.f) : 0.f, ep_out);
      }
    } else {
      float mx = pv_on ? sh->amax[pv_i] : -INFINITY, l = pv_on ? sh->asum[pv_i] : 0.f;
      if (P.ns > 1) {
        mg_ll_fetch(llrec + slot, ((P.ns - 1) * P.rg * pst) >> 1, sRec, ep_out, sh, a.err);
        mg_csync();
        if (pv_on) {
          float gm = mx;
#pragma unroll 1
          for (int s2 = 1; s2 < P.ns; ++s2) gm = fmaxf(gm, sRec[((s2 - 1) * P.rg + pv_i) * pst]);
          const float w0 = mx == -INFINITY ? 0.f : __expf(mx - gm);
          float num = pv_acc * w0, den = l * w0;
#pragma unroll 1
          for (int s2 = 1; s2 < P.ns; ++s2) {
            const float* rec = sRec + ((s2 - 1) * P.rg + pv_i) * pst;
            const float wgt = rec[1] > 0.f ? __expf(rec[0] - gm) : 0.f;
            den += rec[1] * wgt;
            num += rec[MG_PST_PAD + pv_c] * wgt;
          }
          pv_acc = num;
          l = den;
        }
      }
      if (pv_on) mg_ll_store(llout + (size_t)(i0 + pv_i) * a.I + h * dkv + pv_c, l > 0.f ? pv_acc / l : 0.f, ep_out);
    }
    mg_csync();
  }
}

// ---- linear stage ------------------------------------------------------------------------
enum { MG_EPI_QKV = 0, MG_EPI_RESID, MG_EPI_Q, MG_EPI_FFN };

// src == nullptr: the input rows are the embeddings of the tokens (first stage of the pass)
__device__ void mg_linear(const MegaArgs& a, MegaShared* sh, unsigned char* ring, float* act, float* psum, const MegaLin& w,
                          int which, const uint2* src, uint32_t ep_in, const float* gain, int epi, uint2* dst, uint32_t ep_out, int layer,
                          int M, int pos0, bool write_x, int& slot, unsigned& stage, MegaFeed& feed, int& pending) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = w.K;
  const int r0 = sh->slice[which][0], r1 = sh->slice[which][1];
  const int n = r1 - r0, nmat = w.W1 ? 2 : 1;
  if (n == 0) return;   // nothing to produce: the block needs neither the input nor any weights
  const int rowbytes = K * 2, rps = MG_SLOT / rowbytes;
  const int slots_mat = (n + rps - 1) / rps, nslots_stage = slots_mat * nmat, nrows = n * nmat;
  if (tid < nrows) {   // where each slice row sits in the ring
    int r = tid, s = slot;
    if (r >= n) { r -= n; s += slots_mat; }
    s += r / rps;
    if (s >= a.nslots) s -= a.nslots;
    if (s >= a.nslots) s -= a.nslots;
    sh->rowoff[tid] = (unsigned)(s * MG_SLOT + (r % rps) * rowbytes);
  }
  // the slots the previous linear stage handed back take the next slices while the inputs arrive
  if (tid == MG_FEEDER && pending) mg_feed(a, sh, ring, feed, pending);
  pending = nslots_stage;
  const int nkb = (K + 255) >> 8;
  float4 gv[2];   // gains of the columns this thread scales (K <= 2048 where a norm precedes)
  if (gain) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int c = tid * 4 + j * 1024;
      gv[j] = c < K ? __ldg(reinterpret_cast<const float4*>(gain + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  // token rows in groups that fit the staging area
  const int cap_rows = MG_ACT / (K * 4);
  const int rgl = cap_rows >= 8 ? 8 : cap_rows >= 4 ? 4 : cap_rows >= 2 ? 2 : 1;
#pragma unroll 1
  for (int m0 = 0; m0 < M; m0 += rgl) {
    const int mg = min(rgl, M - m0);
    float* Xs = act;
    if (!src) {
      for (int idx = tid; idx < mg * (K >> 3); idx += MG_CONSUMERS) {
        const int m = idx / (K >> 3), c8 = (idx - m * (K >> 3)) << 3;
        int t = a.desc->tokens[m0 + m];
        t = t < 0 ? 0 : (t >= a.vocab ? a.vocab - 1 : t);
        float v[8];
        load8(a.emb + (size_t)t * K + c8, v);
        *reinterpret_cast<float4*>(Xs + (size_t)m * K + c8) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(Xs + (size_t)m * K + c8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
      }
    } else {
      mg_ll_fetch(src + (size_t)m0 * K, (mg * K) >> 1, Xs, ep_in, sh, a.err);
    }
    mg_csync();
    if (gain) {   // T5 norm: x * g / sqrt(mean(x^2) + eps); the division is applied to the dot products
      // thread t scales columns 4t .. 4t+3 (+ 1024, ...) of every row; the gains were requested before the rows arrived
      for (int m = 0; m < mg; ++m) {
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int c = tid * 4 + j * 1024;
          if (c < K) {
            float4 v = *reinterpret_cast<float4*>(Xs + (size_t)m * K + c);
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
            v.x *= gv[j].x; v.y *= gv[j].y; v.z *= gv[j].z; v.w *= gv[j].w;
            *reinterpret_cast<float4*>(Xs + (size_t)m * K + c) = v;
          }
        }
        ss = warp_sum(ss);
        if (lane == 0) sh->ssq[warp][m] = ss;
      }
      mg_csync();
      if (tid < mg) {
        float ss = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv) ss += sh->ssq[wv][tid];
        sh->inv[tid] = rsqrtf(ss / (float)K + a.eps);
      }
    }
    if (m0 == 0) mg_wait(sh, a.err, &sh->full[stage % MG_MAX_SLOTS], (stage / MG_MAX_SLOTS) & 1);
    const int mgr = mg_round_rows(mg);
    mg_items_dyn(mgr, ring, sh->rowoff, nrows, K, Xs, psum, warp, lane);
    mg_csync();
    // epilogue: (output row r, token row m); the partial sums of a quad are added in warp order
    for (int m = tid >> 6; m < mg; m += 4) {
      const int r = tid & 63;
      if (r >= n) continue;
      auto total = [&](int row) {
        const int qd = row >> 2, first = qd * nkb;
        const float* p = psum + (size_t)(qd * 8) * 32 + (row & 3) * mgr + m;
        float s = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv)
          if (((wv - first) & 7) < nkb) s += p[wv * 32];   // warp wv took part in this quad
        return s;
      };
      float v = total(r);
      if (gain) v *= sh->inv[m];
      const int nn = r0 + r, mm = m0 + m;
      if (epi == MG_EPI_QKV) {
        int part = 0, rr = nn;
        if (rr >= a.I) { rr -= a.I; ++part; }
        if (rr >= a.I) { rr -= a.I; ++part; }
        const int h = rr >> a.dkv_shift, c = rr & (a.dkv - 1), row = pos0 + mm;
        mg_ll_store(dst + (((size_t)h * MAXB + mm) * 3 + part) * a.dkv + c, v, ep_out);
        if (part > 0 && row < a.cap) (part == 1 ? a.selfK : a.selfV)[(((size_t)layer * a.H + h) * a.cap + row) * a.dkv + c] = v;
      } else if (epi == MG_EPI_RESID) {
        const float xn = sh->xres[mm][r] + v;
        sh->xres[mm][r] = xn;
        mg_ll_store(dst + (size_t)mm * a.d + nn, xn, ep_out);
        if (write_x) a.x[(size_t)mm * a.d + nn] = xn;
      } else if (epi == MG_EPI_Q) {
        mg_ll_store(dst + ((size_t)(nn >> a.dkv_shift) * MAXB + mm) * a.dkv + (nn & (a.dkv - 1)), v, ep_out);
      } else {
        float uo;
        if (nmat == 2) uo = gelu_tanh(v) * (total(n + r) * sh->inv[m]);
        else uo = fmaxf(v, 0.f);
        mg_ll_store(dst + (size_t)mm * a.F + nn, uo, ep_out);
      }
    }
    if (m0 + rgl < M) mg_csync();   // another group of token rows: staged rows and partial sums are reused
  }
  slot += nslots_stage;
  if (slot >= a.nslots) slot -= a.nslots;
  if (slot >= a.nslots) slot -= a.nslots;
  ++stage;
}

// ---- the pass ----------------------------------------------------------------------------
__global__ void __launch_bounds__(MG_THREADS, 1) mega_pass_kernel(MegaArgs a) {
  extern __shared__ __align__(1024) unsigned char mg_smem[];
  unsigned char* ring = mg_smem;
  float* act = reinterpret_cast<float*>(mg_smem + (size_t)a.nslots * MG_SLOT);
  float* psum = act + MG_ACT / 4;
  MegaShared* sh = reinterpret_cast<MegaShared*>(psum + MG_PSUM / 4);
  const int tid = threadIdx.x;
  if (tid == 0) {
    for (int i = 0; i < MG_MAX_SLOTS; ++i) mg_mbar_init(smem_u32(&sh->full[i]), 1);
    mg_mbar_init(smem_u32(&sh->kvbar[0]), 1);
    mg_mbar_init(smem_u32(&sh->kvbar[1]), 1);
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < 6) {
    const int Ns[6] = {3 * a.I, a.d, a.I, a.d, a.F, a.d};
    mg_slice(Ns[tid], blockIdx.x, gridDim.x, &sh->slice[tid][0], &sh->slice[tid][1]);
  }
  for (int i = tid; i < a.n_layers * (int)(sizeof(MegaLayer) / 8); i += MG_CONSUMERS)
    reinterpret_cast<unsigned long long*>(sh->layers)[i] = reinterpret_cast<const unsigned long long*>(a.layers)[i];
  __syncthreads();
  MegaFeed feed;
  feed.done = true; feed.slot = 0; feed.stage = 0;
  if (tid == MG_FEEDER) {   // the weights do not wait for anything: start the stream
    mg_feed_init(a, sh, feed);
    mg_feed(a, sh, ring, feed, a.nslots);
  }
  const int M = max(1, min(a.desc->k, MAXB)), pos0 = a.desc->pos0;
  const unsigned seq = *(volatile unsigned*)a.sync;
  const uint32_t ep0 = seq * MG_EPOCHS_PER_LAUNCH + 1;
  int slot = 0;
  unsigned stage = 0, kvfill = 0;
  int pending = 0;   // slots to refill at the next opportunity
  const int G = gridDim.x;
  const int ekeys = min(*a.enc_len, a.ecap), skeys = min(pos0 + M, a.cap);
  const MegaAttnPlan plan_self = mg_attn_plan(a, M, skeys, G), plan_cross = mg_attn_plan(a, M, ekeys, G);
  {   // the residual stream starts as the embedding: this block keeps the columns it owns
    const int c_lo = sh->slice[1][0], c_hi = sh->slice[1][1];
    for (int idx = tid; idx < M * MG_XRES; idx += MG_CONSUMERS) {
      const int m = idx / MG_XRES, c = idx - m * MG_XRES;
      if (c < c_hi - c_lo) {
        int t = a.desc->tokens[m];
        t = t < 0 ? 0 : (t >= a.vocab ? a.vocab - 1 : t);
        sh->xres[m][c] = __bfloat162float(a.emb[(size_t)t * a.d + c_lo + c]);
      }
    }
  }
  // stage s of layer l writes epoch ep0 + 8 l + s; stages 1 and 4 are the attentions
  const int n_stages = 8 * a.n_layers;
#pragma unroll 1
  for (int st = 0; st < n_stages; ++st) {
    const int l = st >> 3, sg = st & 7;
    const uint32_t ep_out = ep0 + st, ep_in = ep_out - 1;
    if (sg == 1 || sg == 4) {
      const bool self = sg == 1;
      mg_attention(a, sh, act, psum, l, self ? 1 : 0, M, pos0, self ? skeys : ekeys, self ? plan_self : plan_cross,
                   self ? a.ll.qkv1 : a.ll.q4, self ? a.ll.a2 : a.ll.a5, self ? a.ll.r2 : a.ll.r5, ep_in, ep_out, kvfill, ring, feed,
                   pending);
    } else {
      const MegaLayer& L = sh->layers[l];
      const int p = sg == 0 ? 0 : sg == 2 ? 1 : sg == 3 ? 2 : sg - 2;     // which of the six matrices
      const uint2* src = sg == 0 ? (l == 0 ? nullptr : a.ll.x8) : sg == 2 ? a.ll.a2 : sg == 3 ? a.ll.x3 : sg == 5 ? a.ll.a5
                         : sg == 6 ? a.ll.x6 : a.ll.u7;
      uint2* dst = sg == 0 ? a.ll.qkv1 : sg == 2 ? a.ll.x3 : sg == 3 ? a.ll.q4 : sg == 5 ? a.ll.x6 : sg == 6 ? a.ll.u7 : a.ll.x8;
      const float* gain = sg == 0 ? L.ln1 : sg == 3 ? L.ln2 : sg == 6 ? L.ln3 : nullptr;
      const int epi = sg == 0 ? MG_EPI_QKV : sg == 3 ? MG_EPI_Q : sg == 6 ? MG_EPI_FFN : MG_EPI_RESID;
      mg_linear(a, sh, ring, act, psum, mg_lin(a, L, p), p, src, ep_in, gain, epi, dst, ep_out, l, M, pos0,
                sg == 7 && l + 1 == a.n_layers, slot, stage, feed, pending);
    }
  }
  // Every slice that was issued has been waited for by its stage (the program ends with the last
  // stage), so nothing is in flight into this block's shared memory when it exits - unless a wait
  // gave up: then the stages' barriers are polled once more, each with a limit.
  if (tid == MG_FEEDER && *(volatile int*)&sh->failed) {
    for (unsigned st2 = stage > (unsigned)MG_MAX_SLOTS ? stage - MG_MAX_SLOTS : 0; st2 < stage; ++st2) {
      const uint32_t bar = smem_u32(&sh->full[st2 % MG_MAX_SLOTS]);
      for (unsigned it = 0; it < MG_SPIN; ++it)
        if (mg_mbar_try(bar, (st2 / MG_MAX_SLOTS) & 1)) break;
    }
  }
  // the launch counter moves on once every block has read it: block 0 gets here only after it has
  // consumed values that every working block produced
  if (blockIdx.x == 0 && tid == 0) *(volatile unsigned*)a.sync = seq + 1;
}

}  // namespace bild
