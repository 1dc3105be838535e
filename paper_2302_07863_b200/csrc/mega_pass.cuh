// One decoder pass (steps S0..S8 / L0..L8 of every layer) as ONE persistent kernel, bf16 weights.
//
// A decoder pass at batch 1 is a chain of ~8 dependent stages per layer, each of which moves
// far less data than it takes to hide the memory latency, so a chain of separate kernels is
// bound by launch and memory latency.  Here one block per SM stays resident for the whole
// pass:
//   * a producer warp streams the block's slice of every weight matrix, in program order,
//     through a ring of shared-memory slots with bulk (TMA) copies.  The weights do not
//     depend on the activations, so the stream runs ahead of the dependency chain and a
//     stage finds its weights already on chip;
//   * eight consumer warps run the stages.  Stages are separated by a grid-wide barrier (an
//     arrive counter in global memory); the k activation rows a stage needs are pulled into
//     shared memory with one bulk copy right after the barrier;
//   * a linear stage splits the output rows over the blocks (no cross-block reduction);
//     inside a block a work item is 4 weight rows x 256 columns for all token rows, partial
//     sums are added in a fixed order;
//   * attention splits (head, row group, key range) over the blocks, keys and values are
//     staged in 64-key chunks (double buffered) with a running soft-max; key splits leave
//     (max, sum, weighted values) records that the following output projection merges while
//     it loads its input.
// Every wait (grid barrier, mbarrier) gives up after a fixed number of polls: the block
// then records BILD_ERR_TIMEOUT, stops waiting anywhere, and runs to the end.
#pragma once
#include "common.cuh"

namespace bild {

constexpr int MG_CONSUMERS = 256;                   // 8 consumer warps
constexpr int MG_THREADS = MG_CONSUMERS + 32;       // + the producer warp
constexpr int MG_SLOT = 8192;                       // bytes per ring slot
constexpr int MG_ACT = 80 * 1024;                   // activation staging
constexpr int MG_QUADS = 16;                        // weight-row quads per stage and block (64 rows)
constexpr int MG_PSUM = MG_QUADS * 8 * 32 * 4;      // partial sums [quad][warp][32]
constexpr int MG_MAX_SLOTS = 20;
constexpr int MG_MISC = 1024;
constexpr int MG_PST_PAD = 4;                       // record = [max, sum, -, -, values[dkv]]
constexpr unsigned MG_SPIN = 1u << 20;

struct MegaLayer {
  const __nv_bfloat16 *wqkv, *wo, *wcq, *wco, *wi0, *wi1, *wfo;
  const float *ln1, *ln2, *ln3;
};

struct MegaArgs {
  const MegaLayer* layers;
  int n_layers;
  int d, I, F, H, dkv, dkv_shift, gated, vocab;
  float eps;
  const CallDesc* desc;
  const __nv_bfloat16* emb;
  float *x, *q, *att, *u, *part;
  float *selfK, *selfV;
  const float *crossK, *crossV;
  int cap, ecap;
  const float* dec_bias;      // [H][cap] by distance
  const int* enc_len;
  unsigned* sync;             // [0], [1]: arrive counters (alternating between launches); [2]: which one is next
  int* err;
  int nslots;
};

inline size_t mega_smem_bytes(int nslots) { return (size_t)nslots * MG_SLOT + MG_ACT + MG_PSUM + MG_MISC; }

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
__device__ __forceinline__ void mg_fence_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ unsigned mg_ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void mg_red_release(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void mg_csync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }   // consumer warps only

// Block-wide state in shared memory.
struct MegaShared {
  unsigned long long full[MG_MAX_SLOTS], empty[MG_MAX_SLOTS], actbar, kvbar[2];
  float inv[MAXB];                      // 1 / rms of the staged rows
  float amax[4], asum[4], ascale[4];    // running soft-max of the unit's rows
  int failed;
};

__device__ __forceinline__ void mg_fail(MegaShared* sh, int* err) {
  sh->failed = 1;
  atomicExch(err, (int)BILD_ERR_TIMEOUT);
}
// bounded mbarrier wait; after a failure nothing waits any more
__device__ __forceinline__ void mg_wait(MegaShared* sh, int* err, unsigned long long* bar, uint32_t parity) {
  if (*(volatile int*)&sh->failed) return;
  const uint32_t b = smem_u32(bar);
  for (unsigned it = 0; it < MG_SPIN; ++it)
    if (mg_mbar_try(b, parity)) return;
  mg_fail(sh, err);
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

// ---- producer: the block's weight slices, in program order, through the ring -----------
__device__ void mg_producer(const MegaArgs& a, MegaShared* sh, unsigned char* ring) {
  const int G = gridDim.x, b = blockIdx.x, ns = a.nslots;
  unsigned fill = 0;
  for (int l = 0; l < a.n_layers; ++l) {
    const MegaLayer L = a.layers[l];
    for (int p = 0; p < 6; ++p) {
      const MegaLin w = mg_lin(a, L, p);
      int r0, r1;
      mg_slice(w.N, b, G, &r0, &r1);
      const int rowbytes = w.K * 2, rps = MG_SLOT / rowbytes;
      for (int mat = 0; mat < (w.W1 ? 2 : 1); ++mat) {
        const __nv_bfloat16* W = mat ? w.W1 : w.W0;
        for (int r = r0; r < r1; r += rps) {
          const int nr = min(rps, r1 - r);
          const int slot = fill % ns;
          mg_wait(sh, a.err, &sh->empty[slot], ((fill / ns) & 1) ^ 1);
          const uint32_t bar = smem_u32(&sh->full[slot]);
          mg_mbar_expect(bar, (uint32_t)(nr * rowbytes));
          mg_bulk_g2s(smem_u32(ring + (size_t)slot * MG_SLOT), W + (size_t)r * w.K, (uint32_t)(nr * rowbytes), bar);
          ++fill;
        }
      }
    }
  }
  // nothing may still be in flight into this block's shared memory when it exits
  const unsigned first = fill > (unsigned)ns ? fill - ns : 0;
  for (unsigned f = first; f < fill; ++f) {
    const uint32_t bar = smem_u32(&sh->full[f % ns]);
    for (unsigned it = 0; it < MG_SPIN; ++it)
      if (mg_mbar_try(bar, (f / ns) & 1)) break;
  }
}

// ---- grid barrier ------------------------------------------------------------------------
struct MegaBarrier {
  unsigned* ctr;
  unsigned done;    // barriers passed so far
};
// all consumer threads call both; global writes made before arrive are visible after wait
__device__ __forceinline__ void mg_arrive(MegaBarrier& gb) {
  mg_fence_async();   // this thread's global stores, for bulk copies issued by other blocks
  mg_csync();
  if (threadIdx.x == 0) mg_red_release(gb.ctr, 1u);
}
__device__ __forceinline__ void mg_wait_grid(MegaBarrier& gb, MegaShared* sh, int* err) {
  ++gb.done;
  if (threadIdx.x == 0 && !*(volatile int*)&sh->failed) {
    const unsigned target = gb.done * gridDim.x;
    unsigned it = 0;
    while (mg_ld_acquire(gb.ctr) < target)
      if (++it > MG_SPIN) { mg_fail(sh, err); break; }
    mg_fence_async();
  }
  mg_csync();
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

// Where slice row r of the running stage sits in the ring.
struct MegaRows {
  unsigned char* ring;
  int ns, slot0, rps, rowbytes;
  int n0, slots0;     // gated: rows >= n0 belong to the second matrix, which starts slots0 slots later
  __device__ __forceinline__ const unsigned char* row(int r) const {
    int s = slot0;
    if (r >= n0) { r -= n0; s += slots0; }
    s += r / rps;
    return ring + (size_t)(s % ns) * MG_SLOT + (size_t)(r % rps) * rowbytes;
  }
};

// Work items of a linear stage: (quad of weight rows, 256 columns) x MG token rows.
template <int MG>
__device__ __forceinline__ void mg_items(const MegaRows& R, int nrows, int K, const float* Xs, float* psum, int warp, int lane) {
  constexpr int NA = 4 * MG;
  constexpr int NP = NA <= 4 ? 4 : NA <= 8 ? 8 : NA <= 16 ? 16 : 32;
  const int nkb = (K + 255) >> 8, nq = (nrows + 3) >> 2, nitems = nq * nkb;
  float acc[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) acc[i] = 0.f;
  int cur = -1;
#pragma unroll 1
  for (int it = warp; it < nitems; it += 8) {
    const int qd = it / nkb, kb = it - qd * nkb;
    if (qd != cur) {
      if (cur >= 0) {
        const float r = mg_treduce<NP>(acc, lane);
        if ((lane & (32 / NP - 1)) == 0) psum[(cur * 8 + warp) * 32 + (lane >> (NP == 32 ? 0 : NP == 16 ? 1 : NP == 8 ? 2 : 3))] = r;
#pragma unroll
        for (int i = 0; i < NP; ++i) acc[i] = 0.f;
      }
      cur = qd;
    }
    const int kofs = (kb << 8) + lane * 8;
    if (kofs < K) {
      uint4 w[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int row = qd * 4 + r;
        w[r] = row < nrows ? *reinterpret_cast<const uint4*>(R.row(row) + (size_t)kofs * 2) : make_uint4(0, 0, 0, 0);
      }
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
  if (cur >= 0) {
    const float r = mg_treduce<NP>(acc, lane);
    if ((lane & (32 / NP - 1)) == 0) psum[(cur * 8 + warp) * 32 + (lane >> (NP == 32 ? 0 : NP == 16 ? 1 : NP == 8 ? 2 : 3))] = r;
  }
}

__device__ __forceinline__ void mg_items_dyn(int mg, const MegaRows& R, int nrows, int K, const float* Xs, float* psum, int warp, int lane) {
  switch (mg) {
    case 1: mg_items<1>(R, nrows, K, Xs, psum, warp, lane); break;
    case 2: mg_items<2>(R, nrows, K, Xs, psum, warp, lane); break;
    case 3: mg_items<3>(R, nrows, K, Xs, psum, warp, lane); break;
    case 4: mg_items<4>(R, nrows, K, Xs, psum, warp, lane); break;
    case 5: mg_items<5>(R, nrows, K, Xs, psum, warp, lane); break;
    case 6: mg_items<6>(R, nrows, K, Xs, psum, warp, lane); break;
    case 7: mg_items<7>(R, nrows, K, Xs, psum, warp, lane); break;
    default: mg_items<8>(R, nrows, K, Xs, psum, warp, lane); break;
  }
}

// How attention over M rows and nkeys keys is split over the blocks.
struct MegaAttnPlan {
  int rg;      // rows per unit
  int nrg;     // row groups
  int ns;      // key splits (1: the unit writes the finished rows)
  int ck;      // keys per staged chunk
};
__device__ __forceinline__ MegaAttnPlan mg_attn_plan(const MegaArgs& a, int M, int nkeys, int G) {
  MegaAttnPlan p;
  const int rgmax = max(1, min(4, 256 >> a.dkv_shift));
  p.nrg = (M + rgmax - 1) / rgmax;
  p.rg = (M + p.nrg - 1) / p.nrg;
  p.ck = min(64, 4096 >> a.dkv_shift);
  const int pst = a.dkv + MG_PST_PAD;
  int ns = max(1, G / (a.H * p.nrg));
  ns = min(ns, max(1, nkeys / 32));
  const int room = MG_ACT - M * a.I * 4;
  ns = min(ns, max(1, room / (M * a.H * pst * 4)));
  if (M > 8) ns = 1;   // the merging projection stages all rows at once
  p.ns = max(1, ns);
  return p;
}

// ---- attention stage ---------------------------------------------------------------------
// mode 0: cross (all encoder keys, no bias), mode 1: self (row i sees keys 0..pos0+i, bias by distance)
__device__ void mg_attention(const MegaArgs& a, MegaShared* sh, float* act, float* scratch, MegaBarrier& gb, int layer,
                             int mode, int M, int pos0, unsigned& kvfill) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, H = a.H, dkv = a.dkv, dsh = a.dkv_shift;
  const int nkeys = mode == 0 ? min(*a.enc_len, a.ecap) : min(pos0 + M, a.cap);
  const MegaAttnPlan P = mg_attn_plan(a, M, nkeys, G);
  const int units = H * P.nrg * P.ns;
  const int kcap = mode == 0 ? a.ecap : a.cap;
  const size_t kvoff = (size_t)layer * H * dkv * kcap;
  const float* Kb = (mode == 0 ? a.crossK : a.selfK) + kvoff;
  const float* Vb = (mode == 0 ? a.crossV : a.selfV) + kvoff;
  const int ck = P.ck, chunk_floats = ck * dkv;
  float* sQ = scratch;                    // [rg][dkv]
  float* sS = scratch + 4 * 128;          // [rg][ck]
  const int pst = dkv + MG_PST_PAD;
  bool waited = false;
#pragma unroll 1
  for (int u = blockIdx.x; u < units || !waited; u += G) {
    const bool active = u < units;
    int h = 0, g = 0, sp = 0, j0 = 0, j1 = 0, nchunks = 0;
    if (active) {
      h = u % H;
      const int rest = u / H;
      g = rest % P.nrg;
      sp = rest / P.nrg;
      const int per = (nkeys + P.ns - 1) / P.ns;
      j0 = sp * per;
      j1 = min(nkeys, j0 + per);
      nchunks = j1 > j0 ? (j1 - j0 + ck - 1) / ck : 0;
    }
    const float* Kh = Kb + (size_t)h * kcap * dkv;
    const float* Vh = Vb + (size_t)h * kcap * dkv;
    auto issue = [&](int c) {   // thread 0: chunk c of this unit into buffer (kvfill & 1)
      const int nk = min(ck, j1 - (j0 + c * ck));
      const unsigned buf = kvfill & 1;
      const uint32_t bar = smem_u32(&sh->kvbar[buf]);
      const uint32_t bytes = (uint32_t)(nk * dkv * 4);
      mg_mbar_expect(bar, 2 * bytes);
      mg_bulk_g2s(smem_u32(act + (size_t)buf * 2 * chunk_floats), Kh + (size_t)(j0 + c * ck) * dkv, bytes, bar);
      mg_bulk_g2s(smem_u32(act + (size_t)buf * 2 * chunk_floats + chunk_floats), Vh + (size_t)(j0 + c * ck) * dkv, bytes, bar);
      ++kvfill;
    };
    // cross keys / values never change while decoding: the first chunks may start before the barrier
    const bool early = mode == 0 && !waited;
    unsigned fill0 = kvfill;
    if (early && tid == 0 && active) {
      if (nchunks > 0) issue(0);
      if (nchunks > 1) issue(1);
    }
    if (!waited) { mg_wait_grid(gb, sh, a.err); waited = true; }
    if (!active) break;
    if (tid == 0) {
      if (!early) {
        if (nchunks > 0) issue(0);
        if (nchunks > 1) issue(1);
      }
    }
    if (tid != 0) kvfill = fill0 + min(nchunks, 2);   // every thread tracks the fill count
    const int i0 = g * P.rg, nr = min(P.rg, M - i0);
    // queries of the unit's rows
    for (int idx = tid; idx < nr * (dkv >> 2); idx += MG_CONSUMERS) {
      const int i = idx / (dkv >> 2), e4 = (idx - i * (dkv >> 2)) << 2;
      *reinterpret_cast<float4*>(sQ + i * dkv + e4) =
          __ldcg(reinterpret_cast<const float4*>(a.q + (size_t)(i0 + i) * a.I + h * dkv + e4));
    }
    if (tid < 4) { sh->amax[tid] = -INFINITY; sh->asum[tid] = 0.f; sh->ascale[tid] = 1.f; }
    // thread <-> (row, channel) of the weighted values
    const int pv_i = tid >> dsh, pv_c = tid & (dkv - 1);
    const bool pv_on = pv_i < nr;
    float pv_acc = 0.f;
    mg_csync();
    unsigned use = fill0;
#pragma unroll 1
    for (int c = 0; c < nchunks; ++c, ++use) {
      const unsigned buf = use & 1;
      const float* sK = act + (size_t)buf * 2 * chunk_floats;
      const float* sV = sK + chunk_floats;
      const int jc = j0 + c * ck, nk = min(ck, j1 - jc);
      mg_wait(sh, a.err, &sh->kvbar[buf], (use >> 1) & 1);
      // scores: one (row, key) pair per thread; the columns are visited in a rotated order so that
      // the threads of a quarter warp hit different banks
      for (int idx = tid; idx < nr * ck; idx += MG_CONSUMERS) {
        const int i = idx / ck, jj = idx - i * ck;
        float s = -INFINITY;
        if (jj < nk) {
          const int j = jc + jj;
          const bool seen = mode == 0 || j <= pos0 + i0 + i;
          if (seen) {
            float accs = 0.f;
            const int nq4 = dkv >> 2;
#pragma unroll 4
            for (int e = 0; e < nq4; ++e) {
              const int er = ((e + jj) & (nq4 - 1)) << 2;
              const float4 kv = *reinterpret_cast<const float4*>(sK + jj * dkv + er);
              const float4 qv = *reinterpret_cast<const float4*>(sQ + i * dkv + er);
              accs += kv.x * qv.x + kv.y * qv.y + kv.z * qv.z + kv.w * qv.w;
            }
            if (mode == 1) accs += a.dec_bias[(size_t)h * a.cap + (pos0 + i0 + i - j)];
            s = accs;
          }
        }
        sS[i * ck + jj] = s;
      }
      mg_csync();
      if (warp < nr) {   // running soft-max of row `warp`
        float mx = -INFINITY;
        for (int jj = lane; jj < ck; jj += 32) mx = fmaxf(mx, sS[warp * ck + jj]);
        mx = warp_max(mx);
        const float mo = sh->amax[warp], mn = fmaxf(mo, mx);
        float sum = 0.f;
        for (int jj = lane; jj < ck; jj += 32) {
          const float sc = sS[warp * ck + jj];
          const float pr = sc == -INFINITY ? 0.f : __expf(sc - mn);
          sS[warp * ck + jj] = pr;
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
        const float* pr = sS + pv_i * ck;
        int jj = 0;
#pragma unroll 4
        for (; jj + 1 < nk; jj += 2) {
          a0 += pr[jj] * sV[jj * dkv + pv_c];
          a1 += pr[jj + 1] * sV[(jj + 1) * dkv + pv_c];
        }
        if (jj < nk) a0 += pr[jj] * sV[jj * dkv + pv_c];
        pv_acc = pv_acc * sh->ascale[pv_i] + (a0 + a1);
      }
      mg_csync();   // the chunk's buffer and the probabilities are free again
      if (tid == 0 && c + 2 < nchunks) issue(c + 2);
      if (tid != 0 && c + 2 < nchunks) ++kvfill;
    }
    if (pv_on) {
      const int i = i0 + pv_i;
      if (P.ns == 1) {
        const float l = sh->asum[pv_i];
        a.att[(size_t)i * a.I + h * dkv + pv_c] = l > 0.f ? pv_acc / l : 0.f;
      } else {
        float* rec = a.part + ((size_t)(i * H + h) * P.ns + sp) * pst;
        rec[MG_PST_PAD + pv_c] = pv_acc;
        if (pv_c == 0) { rec[0] = sh->amax[pv_i]; rec[1] = sh->asum[pv_i]; }
      }
    }
    mg_csync();
  }
  mg_arrive(gb);
}

// ---- linear stage ------------------------------------------------------------------------
enum { MG_SRC_EMB = 0, MG_SRC_X, MG_SRC_ATT, MG_SRC_ATT_PARTS, MG_SRC_U };
enum { MG_EPI_QKV = 0, MG_EPI_RESID, MG_EPI_Q, MG_EPI_FFN };

__device__ void mg_linear(const MegaArgs& a, MegaShared* sh, unsigned char* ring, float* act, float* psum, MegaBarrier& gb,
                          const MegaLin& w, int src, const float* gain, int epi, int layer, int M, int pos0,
                          const MegaAttnPlan& AP, bool wait_first, bool arrive_last, unsigned& fill, unsigned& actuse) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, K = w.K;
  int r0, r1;
  mg_slice(w.N, blockIdx.x, G, &r0, &r1);
  const int n = r1 - r0, nmat = w.W1 ? 2 : 1;
  MegaRows R;
  R.ring = ring; R.ns = a.nslots; R.slot0 = fill % a.nslots; R.rowbytes = K * 2; R.rps = MG_SLOT / R.rowbytes;
  const int slots_mat = (n + R.rps - 1) / R.rps;
  R.n0 = nmat == 2 ? n : 0x7fffffff; R.slots0 = slots_mat;
  const int nslots_stage = slots_mat * nmat, nrows = n * nmat;
  // before the barrier: clear the partial sums
  for (int i = tid; i < MG_PSUM / 4; i += MG_CONSUMERS) psum[i] = 0.f;
  if (wait_first) mg_wait_grid(gb, sh, a.err); else mg_csync();
  // token rows in groups that fit the staging area
  int rgl = min(8, MG_ACT / (K * 4));
  if (src == MG_SRC_ATT_PARTS) rgl = min(rgl, M);   // plan guarantees records + rows fit for all M rows
#pragma unroll 1
  for (int m0 = 0; m0 < M; m0 += rgl) {
    const int mg = min(rgl, M - m0);
    float* Xs = act;
    if (src == MG_SRC_EMB) {
      for (int idx = tid; idx < mg * (K >> 3); idx += MG_CONSUMERS) {
        const int m = idx / (K >> 3), c8 = (idx - m * (K >> 3)) << 3;
        int t = a.desc->tokens[m0 + m];
        t = t < 0 ? 0 : (t >= a.vocab ? a.vocab - 1 : t);
        float v[8];
        load8(a.emb + (size_t)t * K + c8, v);
        *reinterpret_cast<float4*>(Xs + (size_t)m * K + c8) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(Xs + (size_t)m * K + c8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
      }
      // the residual stream starts as the embedding: every block writes its share of the columns
      mg_csync();
      int c_lo, c_hi;
      mg_slice(K, blockIdx.x, G, &c_lo, &c_hi);
      for (int idx = tid; idx < mg * (c_hi - c_lo); idx += MG_CONSUMERS) {
        const int m = idx / (c_hi - c_lo), c = c_lo + idx - m * (c_hi - c_lo);
        a.x[(size_t)(m0 + m) * a.d + c] = Xs[(size_t)m * K + c];
      }
    } else if (src == MG_SRC_ATT_PARTS) {
      const int pst = a.dkv + MG_PST_PAD;
      const uint32_t bytes = (uint32_t)(M * a.H * AP.ns * pst * 4);
      float* stage = act + (size_t)M * K;     // K == I
      if (tid == 0) {
        const uint32_t bar = smem_u32(&sh->actbar);
        mg_mbar_expect(bar, bytes);
        mg_bulk_g2s(smem_u32(stage), a.part, bytes, bar);
      }
      mg_wait(sh, a.err, &sh->actbar, actuse & 1);
      ++actuse;
      for (int idx = tid; idx < M * K; idx += MG_CONSUMERS) {
        const int i = idx / K, nn = idx - i * K, h = nn >> a.dkv_shift, c = nn & (a.dkv - 1);
        const float* rec = stage + (size_t)(i * a.H + h) * AP.ns * pst;
        float gm = -INFINITY;
        for (int s = 0; s < AP.ns; ++s) gm = fmaxf(gm, rec[s * pst]);
        float num = 0.f, den = 0.f;
        for (int s = 0; s < AP.ns; ++s) {
          const float l = rec[s * pst + 1];
          const float wgt = l > 0.f ? __expf(rec[s * pst] - gm) : 0.f;
          den += l * wgt;
          num += rec[s * pst + MG_PST_PAD + c] * wgt;
        }
        Xs[idx] = den > 0.f ? num / den : 0.f;
      }
    } else {
      const float* srcp = src == MG_SRC_X ? a.x : src == MG_SRC_ATT ? a.att : a.u;
      const uint32_t bytes = (uint32_t)(mg * K * 4);
      if (tid == 0) {
        const uint32_t bar = smem_u32(&sh->actbar);
        mg_mbar_expect(bar, bytes);
        mg_bulk_g2s(smem_u32(Xs), srcp + (size_t)m0 * K, bytes, bar);
      }
      mg_wait(sh, a.err, &sh->actbar, actuse & 1);
      ++actuse;
    }
    if (src == MG_SRC_EMB || src == MG_SRC_ATT_PARTS) mg_csync();
    if (gain) {   // T5 norm: x * g / sqrt(mean(x^2) + eps); the division is applied to the dot products
      for (int m = warp; m < mg; m += 8) {
        float ss = 0.f;
        for (int c = lane * 4; c < K; c += 128) {
          float4 v = *reinterpret_cast<float4*>(Xs + (size_t)m * K + c);
          const float4 gv = __ldg(reinterpret_cast<const float4*>(gain + c));
          ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          v.x *= gv.x; v.y *= gv.y; v.z *= gv.z; v.w *= gv.w;
          *reinterpret_cast<float4*>(Xs + (size_t)m * K + c) = v;
        }
        ss = warp_sum(ss);
        if (lane == 0) sh->inv[m] = rsqrtf(ss / (float)K + a.eps);
      }
      mg_csync();
    }
    if (m0 == 0)
      for (int s = 0; s < nslots_stage; ++s) mg_wait(sh, a.err, &sh->full[(fill + s) % a.nslots], ((fill + s) / a.nslots) & 1);
    mg_items_dyn(mg, R, nrows, K, Xs, psum, warp, lane);
    mg_csync();
    // epilogue: one (output row, token row) pair per thread, partial sums added in warp order
    for (int idx = tid; idx < n * mg; idx += MG_CONSUMERS) {
      const int r = idx / mg, m = idx - r * mg;
      auto total = [&](int row) {
        const float* p = psum + (size_t)((row >> 2) * 8) * 32 + (row & 3) * mg + m;
        float s = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv) s += p[wv * 32];
        return s;
      };
      float v = total(r);
      if (gain) v *= sh->inv[m];
      const int nn = r0 + r, mm = m0 + m;
      if (epi == MG_EPI_QKV) {
        int part = 0, rr = nn;
        if (rr >= a.I) { rr -= a.I; ++part; }
        if (rr >= a.I) { rr -= a.I; ++part; }
        if (part == 0) a.q[(size_t)mm * a.I + rr] = v;
        else {
          const int h = rr >> a.dkv_shift, c = rr & (a.dkv - 1), row = pos0 + mm;
          if (row < a.cap) (part == 1 ? a.selfK : a.selfV)[(((size_t)layer * a.H + h) * a.cap + row) * a.dkv + c] = v;
        }
      } else if (epi == MG_EPI_RESID) {
        a.x[(size_t)mm * a.d + nn] += v;
      } else if (epi == MG_EPI_Q) {
        a.q[(size_t)mm * a.I + nn] = v;
      } else {
        if (nmat == 2) {
          const float v1 = total(n + r) * sh->inv[m];
          a.u[(size_t)mm * a.F + nn] = gelu_tanh(v) * v1;
        } else {
          a.u[(size_t)mm * a.F + nn] = fmaxf(v, 0.f);
        }
      }
    }
    if (m0 + rgl < M) {   // another group of token rows follows
      mg_csync();
      for (int i = tid; i < MG_PSUM / 4; i += MG_CONSUMERS) psum[i] = 0.f;
      mg_csync();
    }
  }
  mg_csync();   // all warps are done with the weights (and the staged rows)
  if (tid == 0)
    for (int s = 0; s < nslots_stage; ++s) mg_mbar_arrive(smem_u32(&sh->empty[(fill + s) % a.nslots]));
  fill += nslots_stage;
  if (arrive_last) mg_arrive(gb);
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
    for (int i = 0; i < a.nslots; ++i) { mg_mbar_init(smem_u32(&sh->full[i]), 1); mg_mbar_init(smem_u32(&sh->empty[i]), 1); }
    mg_mbar_init(smem_u32(&sh->actbar), 1);
    mg_mbar_init(smem_u32(&sh->kvbar[0]), 1);
    mg_mbar_init(smem_u32(&sh->kvbar[1]), 1);
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid >= MG_CONSUMERS) {
    if (tid == MG_CONSUMERS) mg_producer(a, sh, ring);
    return;
  }
  const int M = max(1, min(a.desc->k, MAXB)), pos0 = a.desc->pos0;
  const unsigned par = a.sync[2] & 1u;
  MegaBarrier gb;
  gb.ctr = a.sync + par;
  gb.done = 0;
  if (blockIdx.x == 0 && tid == 0) a.sync[par ^ 1u] = 0;   // the next launch counts from zero
  unsigned fill = 0, actuse = 0, kvfill = 0;
  const int G = gridDim.x;
  const int ekeys = min(*a.enc_len, a.ecap), skeys = min(pos0 + M, a.cap);
  const MegaAttnPlan plan_self = mg_attn_plan(a, M, skeys, G), plan_cross = mg_attn_plan(a, M, ekeys, G);
#pragma unroll 1
  for (int l = 0; l < a.n_layers; ++l) {
    const MegaLayer L = a.layers[l];
    const bool last = l + 1 == a.n_layers;
    // norm + QKV, K/V appended to the cache
    mg_linear(a, sh, ring, act, psum, gb, mg_lin(a, L, 0), l == 0 ? MG_SRC_EMB : MG_SRC_X, L.ln1, MG_EPI_QKV, l, M, pos0,
              plan_self, l != 0, true, fill, actuse);
    mg_attention(a, sh, act, psum, gb, l, 1, M, pos0, kvfill);
    mg_linear(a, sh, ring, act, psum, gb, mg_lin(a, L, 1), plan_self.ns > 1 ? MG_SRC_ATT_PARTS : MG_SRC_ATT, nullptr,
              MG_EPI_RESID, l, M, pos0, plan_self, true, true, fill, actuse);
    mg_linear(a, sh, ring, act, psum, gb, mg_lin(a, L, 2), MG_SRC_X, L.ln2, MG_EPI_Q, l, M, pos0, plan_self, true, true,
              fill, actuse);
    mg_attention(a, sh, act, psum, gb, l, 0, M, pos0, kvfill);
    mg_linear(a, sh, ring, act, psum, gb, mg_lin(a, L, 3), plan_cross.ns > 1 ? MG_SRC_ATT_PARTS : MG_SRC_ATT, nullptr,
              MG_EPI_RESID, l, M, pos0, plan_cross, true, true, fill, actuse);
    mg_linear(a, sh, ring, act, psum, gb, mg_lin(a, L, 4), MG_SRC_X, L.ln3, MG_EPI_FFN, l, M, pos0, plan_self, true, true,
              fill, actuse);
    mg_linear(a, sh, ring, act, psum, gb, mg_lin(a, L, 5), MG_SRC_U, nullptr, MG_EPI_RESID, l, M, pos0, plan_self, true,
              !last, fill, actuse);
  }
  if (blockIdx.x == 0 && tid == 0) a.sync[2] = par ^ 1u;
}

}  // namespace bild
