// Fused LM head (steps S9+S10 / L9+L10) for up to MAXB rows, bf16 weights, one block per SM.
//   z[m][n] = scale * sum_j W[n][j] * rms_norm(x_m)[j]
// Block b owns the vocabulary rows [b V / G, (b + 1) V / G).  They stream through a ring of
// 16-row tiles in shared memory (one bulk copy per tile where the width allows the products of sl_mma_perm,
// else one copy per row with the rows padded against bank conflicts; the
// first tiles are requested before the dependency wait of the programmatic launch) by a ninth warp
// that does nothing else (issuing a tile's copies costs about as much as multiplying it).  A tile
// times the (up to 16) normalised token rows goes through mma.sync m16n8k16 (each activation as
// a bf16 head and a bf16 remainder, fp32 accumulation), K split over the 8 warps and added in
// warp order.  Thread (row r, token m) then folds the logit into its running (max, arg max,
// sum exp), picks up the target token's logit, and at the end the 16 threads of a token combine
// in a fixed order.  The logits never reach memory unless a debug buffer is given.  The last
// block to finish merges the per-block partials, applies the policy tests and advances the
// decode loop, exactly as the other head kernels do.
#pragma once
#include "slice_linear.cuh"

namespace bild {

constexpr int SH_COMPUTE = 256;             // 8 warps multiply, reduce and fold
constexpr int SH_THREADS = SH_COMPUTE + 32;  // + one warp that only requests tiles
constexpr int SH_TILES = 3;   // ring depth

struct SliceHeadShared {
  unsigned long long full[SH_TILES], empty[SH_TILES];
  float scale[MAXB];
  int last, failed;
};

// tile_rows: 16, or 32 for short rows and at most 8 token rows (half as many barriers per byte)
__host__ __device__ inline size_t slice_head_tile_bytes(int K, int tile_rows) { return (size_t)tile_rows * (K * 2 + SL_WPAD); }
inline size_t slice_head_smem_bytes(int K, int tile_rows) {
  return SH_TILES * slice_head_tile_bytes(K, tile_rows) + (size_t)MAXB * (K + SL_XPAD) * 4 + 2 * 8 * 2 * 128 * 4 + 1024;
}

__global__ void __launch_bounds__(SH_THREADS) slice_head_kernel(HeadArgs a, int* err, int TR) {
  extern __shared__ __align__(1024) unsigned char shd_smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = a.K, V = a.V, G = gridDim.x;
  const int rowst = K * 2 + SL_WPAD, xst = K + SL_XPAD;
  const size_t tile_bytes = slice_head_tile_bytes(K, TR);
  const int tr_sh = TR == 32 ? 5 : 4;
  unsigned char* sW = shd_smem;
  float* Xs = reinterpret_cast<float*>(shd_smem + SH_TILES * tile_bytes);
  float* psum = Xs + (size_t)MAXB * xst;                 // [2][8 warps][2][32 lanes][4]
  SliceHeadShared* sh = reinterpret_cast<SliceHeadShared*>(psum + 2 * 8 * 2 * 128);
  const int nb = (int)(((long long)blockIdx.x * V) / G), ne = (int)(((long long)(blockIdx.x + 1) * V) / G);
  const int ntiles = (ne - nb + TR - 1) >> tr_sh;
  const __nv_bfloat16* W = (const __nv_bfloat16*)a.W;
  if (tid == 0) {
    for (int i = 0; i < SH_TILES; ++i) { mbar_init(smem_u32(&sh->full[i]), 1); mbar_init(smem_u32(&sh->empty[i]), 1); }
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // the last warp requests tile t: lane 0 announces the bytes, lanes 0..15 copy one row each (rows past
  // the end of the slice repeat its last row; their logits are masked).  Issuing the copies takes about
  // as long as multiplying a tile, which is why the eight computing warps do not do it themselves.
  // usual widths (K a multiple of 256 up to 1024, or of 128 up to 512 for 32-row tiles): ONE bulk copy brings a tile, which
  // then lies unpadded, and the products read it with 16-byte loads (sl_mma_perm); otherwise one copy per padded row
  const bool whole = sl_perm_fits(TR, K);
  const int wrow = whole ? K * 2 : rowst;   // bytes from one weight row of a tile to the next
  auto request = [&](int t) {
    if (t >= ntiles) return;
    const int slot = t % SH_TILES;
    if (whole) {
      if (lane == 0) {
        const int n0 = nb + t * TR;
        const uint32_t bytes = (uint32_t)(min(TR, ne - n0) * K * 2);   // (rows past the end of the slice keep what the slot held: masked)
        mbar_expect(smem_u32(&sh->full[slot]), bytes);
        bulk_g2s(smem_u32(sW + slot * tile_bytes), W + (size_t)n0 * K, bytes, smem_u32(&sh->full[slot]));
      }
      return;
    }
    if (lane == 0) mbar_expect(smem_u32(&sh->full[slot]), (uint32_t)(TR * K * 2));
    __syncwarp();
    if (lane < TR) {
      const int n = min(nb + t * TR + lane, ne - 1);
      bulk_g2s(smem_u32(sW + slot * tile_bytes + (size_t)lane * rowst), W + (size_t)n * K, (uint32_t)(K * 2),
                  smem_u32(&sh->full[slot]));
    }
  };
  pdl_launch_dependents();
  if (warp == SH_COMPUTE / 32) {   // producer: the weights depend on nothing, so it never waits for the kernel in front
    for (int t = 0; t < SH_TILES; ++t) request(t);
#pragma unroll 1
    for (int t = SH_TILES; t < ntiles; ++t) {
      const int slot = t % SH_TILES;
      const uint32_t bar = smem_u32(&sh->empty[slot]), par = ((t / SH_TILES) - 1) & 1;
      bool ok = mbar_try(bar, par);
      if (!ok && !*(volatile int*)&sh->failed) {
        for (unsigned it = 0; it < SPIN_LIMIT && !ok; ++it) ok = mbar_try(bar, par);
        if (!ok && lane == 0) { sh->failed = 1; atomicExch(err, (int)BILD_ERR_TIMEOUT); }
      }
      request(t);
    }
    return;
  }
  pdl_wait();
  const int M = min(a.desc ? a.desc->k : a.M, MAXB);
  const int* target = a.desc ? a.desc->targets : a.target;
  // normalised token rows: x * g / rms (the head's own norm), fp32 in shared memory
  for (int m = warp; m < M; m += SH_COMPUTE / 32) {
    float ss = 0.f;
    for (int j = lane * 4; j < K; j += 128) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(a.X + (size_t)m * a.ldx + j));
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
      *reinterpret_cast<float4*>(Xs + (size_t)m * xst + j) = v;
    }
    ss = warp_sum(ss);
    const float sc = a.gain ? rsqrtf(ss / (float)K + a.eps) : 1.f;
    __syncwarp();
    for (int j = lane * 4; j < K; j += 128) {
      float4 v = *reinterpret_cast<float4*>(Xs + (size_t)m * xst + j);
      float4 g = a.gain ? __ldg(reinterpret_cast<const float4*>(a.gain + j)) : make_float4(1.f, 1.f, 1.f, 1.f);
      v.x *= g.x * sc; v.y *= g.y * sc; v.z *= g.z * sc; v.w *= g.w * sc;
      *reinterpret_cast<float4*>(Xs + (size_t)m * xst + j) = v;
    }
  }
  csync256();
  // thread <-> (row r of the tile, token m)
  const int er = tid & (TR - 1), em = tid >> tr_sh;
  const int ks_sh = TR == 32 ? 2 : 3;   // the K range of a 16-row tile is split over 8 (4) warps
  const int my_target = (em < M && target) ? target[em] : -1;
  Partial run;
  run.m = -INFINITY; run.s = 0.f; run.idx = 0x7fffffff;
  const int NT = M <= 8 ? 1 : 2;
  SlPermFrags<1> f1;
  SlPermFrags<2> f2;
  if (whole) {   // the token rows as operand fragments of this warp's K range, built once for all tiles
    if (NT == 1) sl_perm_frags<1>(TR, K, Xs, xst, M, warp, lane, f1);
    else sl_perm_frags<2>(TR, K, Xs, xst, M, warp, lane, f2);
  }
#pragma unroll 1
  for (int t = 0; t < ntiles; ++t) {
    const int slot = t % SH_TILES;
    {   // bounded wait for the tile
      const uint32_t bar = smem_u32(&sh->full[slot]), par = (t / SH_TILES) & 1;
      bool ok = mbar_try(bar, par);
      if (!ok && !*(volatile int*)&sh->failed) {
        for (unsigned it = 0; it < SPIN_LIMIT && !ok; ++it) ok = mbar_try(bar, par);
        if (!ok) { sh->failed = 1; atomicExch(err, (int)BILD_ERR_TIMEOUT); }
      }
    }
    float* ps = psum + (t & 1) * (8 * 2 * 128);
    if (whole) {
      if (NT == 1) sl_mma_perm<1>(sW + slot * tile_bytes, wrow, TR, K, f1, ps, warp, lane);
      else sl_mma_perm<2>(sW + slot * tile_bytes, wrow, TR, K, f2, ps, warp, lane);
    } else if (NT == 1) sl_mma<1>(sW + slot * tile_bytes, rowst, TR, K, Xs, xst, M, ps, warp, lane);
    else sl_mma<2>(sW + slot * tile_bytes, rowst, TR, K, Xs, xst, M, ps, warp, lane);
    csync256();   // partial sums complete; every warp is done with the tile
    if (tid == 0) mbar_arrive(smem_u32(&sh->empty[slot]));   // the producer may refill it
    if (em < M) {
      // fragment layout of the accumulators: row = group (+ 8), token = 2 * (lane & 3) (+ 1)
      const int col = em & 7, mt = er >> 4, rr = er & 15;
      const float* p = ps + ((size_t)((mt << ks_sh) * NT + (em >> 3)) * 32 + (rr & 7) * 4 + (col >> 1)) * 4 + (rr >> 3) * 2 + (col & 1);
      float z = 0.f;
      if (ks_sh == 3) {   // the eight partial sums are requested together, then added in warp order
        float v[8];
#pragma unroll
        for (int w = 0; w < 8; ++w) v[w] = p[(size_t)w * NT * 128];
#pragma unroll
        for (int w = 0; w < 8; ++w) z += v[w];
      } else {
        for (int w = 0; w < (1 << ks_sh); ++w) z += p[(size_t)w * NT * 128];
      }
      const int n = nb + t * TR + er;
      if (n < ne) {
        z *= a.scale;
        const float dz = z - run.m, ez = expf(-fabsf(dz));   // one exponential for either case (the lanes of a warp take both)
        if (dz > 0.f) { run.s = run.s * ez + 1.f; run.m = z; run.idx = n; }
        else run.s += ez;
        if (n == my_target) a.out->gather[em] = z;
        if (a.logits_dbg) a.logits_dbg[(size_t)em * V + n] = z;
      }
    }
    // the other half of psum is written next; this half is reused two tiles later, after another barrier
  }
  // the 16 (32) threads of a token combine (half a warp or a warp), lower row index first
  for (int o = TR >> 1; o > 0; o >>= 1) {
    Partial q;
    q.m = __shfl_xor_sync(0xffffffffu, run.m, o);
    q.s = __shfl_xor_sync(0xffffffffu, run.s, o);
    q.idx = __shfl_xor_sync(0xffffffffu, run.idx, o);
    run = ((lane & o) == 0) ? combine(run, q) : combine(q, run);
  }
  if (er == 0 && em < M) a.partials[(size_t)blockIdx.x * MAXB + em] = run;
  __threadfence();
  csync256();
  if (tid == 0) {
    const unsigned tk = atomicAdd(a.counter, 1u);
    sh->last = (tk == gridDim.x - 1);
    if (sh->last) *a.counter = 0;
  }
  csync256();
  if (!sh->last) return;
  __threadfence();
  for (int m = warp; m < M; m += SH_COMPUTE / 32) {
    Partial p;
    p.m = -INFINITY; p.s = 0.f; p.idx = 0x7fffffff;
    // (the blocks' partial results of a lane are requested together, eight at a time, then combined in block order)
    for (int b0 = lane; b0 < (int)gridDim.x; b0 += 8 * 32) {
      Partial q[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int b = b0 + 32 * j;
        q[j].m = -INFINITY; q[j].s = 0.f; q[j].idx = 0x7fffffff;
        if (b < (int)gridDim.x) {
          const Partial* src = &a.partials[(size_t)b * MAXB + m];
          q[j].m = __ldcg(&src->m); q[j].s = __ldcg(&src->s); q[j].idx = __ldcg(&src->idx);
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) p = combine(p, q[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      Partial q;
      q.m = __shfl_xor_sync(0xffffffffu, p.m, o);
      q.s = __shfl_xor_sync(0xffffffffu, p.s, o);
      q.idx = __shfl_xor_sync(0xffffffffu, p.idx, o);
      p = ((lane & o) == 0) ? combine(p, q) : combine(q, p);
    }
    if (lane == 0) {
      a.out->argmax[m] = p.idx;
      a.out->zmax[m] = p.m;
      a.out->lse[m] = p.m + logf(p.s);
      if (m == 0) a.out->pmax = 1.f / p.s;
    }
  }
  csync256();
  if (tid == 0) {
    __threadfence();
    HeadOut* o = a.out;
    // gather[] was written by other blocks before their tickets: read around L1
    for (int m = 0; m < M; ++m) o->gather[m] = __ldcg(&o->gather[m]);
    policy_tail(a, o);
  }
}

}  // namespace bild
