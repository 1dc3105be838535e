// Linear layer of a decoder pass for up to MAXB token rows, bf16 weights (steps S1, S3, S4, S6,
// S7, S8 and L1, L3, L4, L6, L7, L8), one block per SM:
//   * block b owns output rows [b N / G, (b + 1) N / G) of the weight matrix, a contiguous piece
//     of memory that one bulk (TMA) copy brings into shared memory.  The copy is issued BEFORE
//     the dependency wait of the programmatic launch, so the weights of a layer stream in while
//     the kernel before it is still running;
//   * after the wait the token rows (a few KB) follow with a second bulk copy; every block needs
//     all of them, so they are read 148 times from L2 instead of once per pair of rows;
//   * a work item is 4 weight rows x 256 columns for all token rows of the group; warp w takes
//     items w, w + 8, ...; the partial sums of a quad are added in warp order (fixed);
//   * the epilogues are those of the other linear kernels (store, ReLU, GELU gate, residual add,
//     scatter to q / the KV cache).
#pragma once
#include "decode_kernels.cuh"
#include "mega_pass.cuh"

namespace bild {

constexpr int SL_THREADS = 256;
constexpr int SL_QUADS = 12;                         // weight-row quads per block (48 rows)
constexpr int SL_PSUM = SL_QUADS * 8 * 32 * 4;
constexpr int SL_MISC = 1024;

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
  int x_rows;      // token rows per group (1, 2, 4 or 8)
};

inline size_t slice_smem_bytes(int w_bytes, int x_rows, int K) { return (size_t)w_bytes + (size_t)x_rows * K * 4 + SL_PSUM + SL_MISC; }

__device__ __forceinline__ void sl_wait(SliceShared* sh, int* err, unsigned long long* bar, uint32_t parity) {
  const uint32_t b = smem_u32(bar);
  if (mg_mbar_try(b, parity)) return;
  if (*(volatile int*)&sh->failed) return;
  for (unsigned it = 0; it < MG_SPIN; ++it)
    if (mg_mbar_try(b, parity)) return;
  sh->failed = 1;
  atomicExch(err, (int)BILD_ERR_TIMEOUT);
}

// Item it belongs to quad it / nkb and column block it % nkb (rows past the end of the slice repeat
// its last row; nobody reads their sums).
template <int MG>
__device__ __forceinline__ void sl_items(const unsigned char* sW, int rowbytes, int nrows, int K, const float* Xs, float* psum,
                                         int warp, int lane) {
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

__global__ void __launch_bounds__(SL_THREADS) slice_linear_kernel(SliceArgs s) {
  extern __shared__ __align__(1024) unsigned char sl_smem[];
  const LinArgs& a = s.lin;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, K = a.K;
  const int r0 = (int)(((long long)blockIdx.x * a.N) / G), r1 = (int)(((long long)(blockIdx.x + 1) * a.N) / G);
  const int n = r1 - r0, nmat = a.epi == EPI_GATED ? 2 : 1, nrows = n * nmat, rowbytes = K * 2;
  if (n == 0) {   // more blocks than rows
    pdl_launch_dependents();
    return;
  }
  unsigned char* sW = sl_smem;
  float* Xs = reinterpret_cast<float*>(sl_smem + s.w_bytes);
  float* psum = Xs + (size_t)s.x_rows * K;
  SliceShared* sh = reinterpret_cast<SliceShared*>(psum + SL_PSUM / 4);
  if (tid == 0) {
    mg_mbar_init(smem_u32(&sh->wbar), 1);
    mg_mbar_init(smem_u32(&sh->xbar), 1);
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // the weights depend on nothing: request them before waiting for the kernel in front
    const uint32_t bytes = (uint32_t)(n * rowbytes);
    mg_mbar_expect(smem_u32(&sh->wbar), bytes * nmat);
    mg_bulk_g2s(smem_u32(sW), (const __nv_bfloat16*)a.W0 + (size_t)r0 * K, bytes, smem_u32(&sh->wbar));
    if (nmat == 2) mg_bulk_g2s(smem_u32(sW + bytes), (const __nv_bfloat16*)a.W1 + (size_t)r0 * K, bytes, smem_u32(&sh->wbar));
  }
  float4 gv[2];   // gains of the columns this thread scales (K <= 2048 where a norm precedes)
  if (a.gain) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int c = tid * 4 + j * 1024;
      gv[j] = c < K ? __ldg(reinterpret_cast<const float4*>(a.gain + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  __syncthreads();
  pdl_launch_dependents();
  pdl_wait();
  const int M = min(a.desc->k, MAXB), pos0 = a.desc->pos0;
  const int nkb = (K + 255) >> 8, rgl = s.x_rows;
  unsigned xuse = 0;
#pragma unroll 1
  for (int m0 = 0; m0 < M; m0 += rgl, ++xuse) {
    const int mg = min(rgl, M - m0);
    if (tid == 0) {
      asm volatile("fence.proxy.async;" ::: "memory");   // rows written by the kernel in front, read by the copy engine
      const uint32_t bytes = (uint32_t)(mg * K * 4);
      mg_mbar_expect(smem_u32(&sh->xbar), bytes);
      mg_bulk_g2s(smem_u32(Xs), a.X + (size_t)m0 * a.ldx, bytes, smem_u32(&sh->xbar));
    }
    sl_wait(sh, s.err, &sh->xbar, xuse & 1);
    if (a.gain) {   // T5 norm: x * g / sqrt(mean(x^2) + eps); the division is applied to the dot products
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
      __syncthreads();
      if (tid < mg) {
        float ss = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv) ss += sh->ssq[wv][tid];
        sh->inv[tid] = rsqrtf(ss / (float)K + a.eps);
      }
    }
    if (m0 == 0) sl_wait(sh, s.err, &sh->wbar, 0);
    const int mgr = mg_round_rows(mg);
    switch (mgr) {
      case 1: sl_items<1>(sW, rowbytes, nrows, K, Xs, psum, warp, lane); break;
      case 2: sl_items<2>(sW, rowbytes, nrows, K, Xs, psum, warp, lane); break;
      case 4: sl_items<4>(sW, rowbytes, nrows, K, Xs, psum, warp, lane); break;
      default: sl_items<8>(sW, rowbytes, nrows, K, Xs, psum, warp, lane); break;
    }
    __syncthreads();
    // epilogue: (output row r, token row m); the partial sums of a quad are added in warp order
    for (int m = tid >> 6; m < mg; m += 4) {
      const int r = tid & 63;
      if (r >= n) continue;
      auto total = [&](int row) {
        const int qd = row >> 2, first = qd * nkb;
        const float* p = psum + (size_t)(qd * 8) * 32 + (row & 3) * mgr + m;
        float t = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv)
          if (((wv - first) & 7) < nkb) t += p[wv * 32];   // warp wv took part in this quad
        return t;
      };
      float v = total(r);
      if (a.gain) v *= sh->inv[m];
      const int nn = r0 + r, mm = m0 + m;
      if (a.epi == EPI_RESID) a.Y[(size_t)mm * a.ldy + nn] += v;
      else if (a.epi == EPI_STORE) a.Y[(size_t)mm * a.ldy + nn] = v;
      else if (a.epi == EPI_RELU) a.Y[(size_t)mm * a.ldy + nn] = fmaxf(v, 0.f);
      else if (a.epi == EPI_GATED) a.Y[(size_t)mm * a.ldy + nn] = gelu_tanh(v) * (total(n + r) * (a.gain ? sh->inv[m] : 1.f));
      else heads_store(a, nn, mm, pos0, v);
    }
    if (m0 + rgl < M) __syncthreads();   // another group of token rows: staged rows and partial sums are reused
  }
}

}  // namespace bild
