// Attention for up to MAXB query rows per block, 256 threads (512 in a block pass): the decoder's self- and cross-attention
// (steps S2, S5 and L2, L5) and the encoder's self-attention (set-up).
// grid (heads, key splits, blocks of query rows); the splits of a head form one thread-block cluster
// whose blocks hand (max, sum, weighted values) to the first block through distributed shared memory.
// mode 0 cross (all encoder keys, no bias), 1 decoder self (row i sees keys 0..pos0+i, bias by
// distance), 2 encoder self (all keys, bias by signed distance; rows blockIdx.z * MB ...).
//   * keys and values of the block's key range are staged in 64-key chunks with bulk (TMA)
//     copies, double buffered; for cross-attention (the encoder K/V never change while decoding)
//     the first chunks are requested before the dependency wait of the programmatic launch;
//   * per chunk: scores one (row, key) pair per thread and turn (columns visited in a rotated
//     order, so that the threads of a quarter warp hit different banks), running soft-max one
//     warp per row, weighted values one (row, channel) pair per thread and group of rows.
#pragma once
#include "decode_kernels.cuh"

namespace bild {

constexpr int UA_THREADS = 256;       // threads of a single-row pass
constexpr int UA_THREADS_MAX = 512;   // block passes: twice the threads halve the turns of the score and value phases
                                      // (measured per pass of 24 layers: 5 rows -58 us, 8 rows -37 us, 2 to 4 rows +20 us)
constexpr int UA_CK = 64;   // keys per staged chunk

struct UAttnShared {
  unsigned long long kvbar[2];
  float amax[MAXB], asum[MAXB], ascale[MAXB];
  int failed;
};

// floats of dynamic shared memory
inline size_t uattn_smem_floats(int MB, int dkv, int nsplit, int bias_len) {
  return (size_t)4 * UA_CK * dkv + (size_t)MB * dkv + (size_t)MB * UA_CK + (size_t)bias_len + (size_t)nsplit * MB * (dkv + 2) +
         (sizeof(UAttnShared) + 3) / 4 + 8 + 4 * 64;   // ... + the single-row value phase's partial sums
}

// ONE: instantiation for single-row passes (its score and value phases use all 256 threads for the one row)
template <bool ONE>
__global__ void __launch_bounds__(UA_THREADS_MAX) uattn_kernel(DAttnArgs d, int bias_len) {
  extern __shared__ __align__(1024) float ua_smem[];
  const BAttnArgs& a = d.b;
  const int MB = d.MB, dsh = d.dkv_shift, dkv = a.dkv;
  const int h = blockIdx.x, sp = blockIdx.y, ns = a.nsplit;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NT = blockDim.x;
  const int chunk_floats = UA_CK * dkv, pst = dkv + 2;
  float* sKV = ua_smem;                               // [2 buffers][keys | values][UA_CK][dkv]
  float* sQ = sKV + 4 * chunk_floats;                 // [MB][dkv]
  float* sS = sQ + MB * dkv;                          // [MB][UA_CK]
  float* sBias = sS + MB * UA_CK;                      // [bias_len]
  float* sM = sBias + bias_len;                       // [ns][MB][pst] (used in the first block of the cluster)
  UAttnShared* sh = reinterpret_cast<UAttnShared*>(sM + (size_t)ns * MB * pst + ((ns * MB * pst) & 1));
  float* sP1 = reinterpret_cast<float*>(sh + 1);     // [4 key quarters][64 channels], single-row passes
  if (tid == 0) {
    mbar_init(smem_u32(&sh->kvbar[0]), 1);
    mbar_init(smem_u32(&sh->kvbar[1]), 1);
    sh->failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (ns > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  __syncthreads();
  const float* Kh = a.kc + (size_t)h * a.cap * dkv;
  const float* Vh = a.vc + (size_t)h * a.cap * dkv;
  int j0 = 0, j1 = 0, nchunks = 0, issued = 0;
  auto issue_to = [&](int upto) {   // thread 0: request chunks [issued, upto)
#pragma unroll 1
    for (; issued < upto; ++issued) {
      if (tid != 0) continue;
      const int jc = j0 + issued * UA_CK, nk = min(UA_CK, j1 - jc), buf = issued & 1;
      const uint32_t bar = smem_u32(&sh->kvbar[buf]), bytes = (uint32_t)(nk * dkv * 4);
      mbar_expect(bar, 2 * bytes);
      bulk_g2s(smem_u32(sKV + (size_t)buf * 2 * chunk_floats), Kh + (size_t)jc * dkv, bytes, bar);
      bulk_g2s(smem_u32(sKV + (size_t)buf * 2 * chunk_floats + chunk_floats), Vh + (size_t)jc * dkv, bytes, bar);
    }
  };
  auto set_range = [&](int n_all) {
    const int per = (n_all + ns - 1) / ns;
    j0 = min(n_all, sp * per);
    j1 = min(n_all, j0 + per);
    nchunks = (j1 - j0 + UA_CK - 1) / UA_CK;
  };
  if (a.mode == 0) {   // encoder keys: before the dependency wait
    set_range(min(*a.n_keys_dev, a.cap));
    issue_to(min(nchunks, 2));
  }
  pdl_launch_dependents();
  pdl_wait();
  const int row0 = blockIdx.z * MB;   // first query row of this block (encoder: many blocks of rows)
  const int M = min((a.desc ? a.desc->k : a.M) - row0, MB), pos0 = a.desc ? a.desc->pos0 : 0;
  if (a.mode != 0) {
    set_range(a.mode == 1 ? min(pos0 + M, a.cap) : min(*a.n_keys_dev, a.cap));
    if (tid == 0) asm volatile("fence.proxy.async;" ::: "memory");   // cache rows written by the kernel in front
    issue_to(min(nchunks, 2));
  }
  for (int idx = tid; idx < (M << (dsh - 2)); idx += NT) {
    const int i = idx >> (dsh - 2), e4 = (idx & ((dkv >> 2) - 1)) << 2;
    *reinterpret_cast<float4*>(sQ + i * dkv + e4) =
        __ldcg(reinterpret_cast<const float4*>(a.q + (size_t)(row0 + i) * a.ldq + h * dkv + e4));
  }
  // bias entries this block meets (a static table): decoder index pos0 + i - j, encoder index off + j - (row0 + i)
  const int dmin = a.mode == 1 ? max(0, pos0 - (j1 - 1)) : a.bias_off + j0 - (row0 + M - 1);
  const int dmax = a.mode == 1 ? pos0 + M - 1 - j0 : a.bias_off + (j1 - 1) - row0;
  const bool bias_staged = a.mode != 0 && dmax - dmin + 1 <= bias_len;
  if (bias_staged)
    for (int dd = dmin + tid; dd <= dmax; dd += NT) sBias[dd - dmin] = __ldg(a.bias + (size_t)h * a.bias_ld + dd);
  if (tid < MAXB) { sh->amax[tid] = -INFINITY; sh->asum[tid] = 0.f; sh->ascale[tid] = 1.f; }
  const int RG = min(8, NT >> dsh);           // query rows per group
  const int ngroups = (M + RG - 1) / RG;
  const int pv_i = tid >> dsh, pv_c = tid & (dkv - 1);   // thread <-> (row of the group, channel)
  float pv_acc[4] = {0.f, 0.f, 0.f, 0.f};               // one per group (MAXB / RG <= 4 when dkv <= 64)
  // a single query row over 64-channel heads: the score and value phases are laid out so that all 256 threads work
  const bool one_row = ONE && M == 1 && dkv == 64 && NT == UA_THREADS && row0 == 0;
  __syncthreads();
#pragma unroll 1
  for (int c = 0; c < nchunks; ++c) {
    const int buf = c & 1;
    const float* sK = sKV + (size_t)buf * 2 * chunk_floats;
    const float* sV = sK + chunk_floats;
    const int jc = j0 + c * UA_CK, nk = min(UA_CK, j1 - jc);
    {   // bounded wait for the chunk
      const uint32_t bar = smem_u32(&sh->kvbar[buf]);
      bool ok = mbar_try(bar, (c >> 1) & 1);
      if (!ok && !*(volatile int*)&sh->failed) {
        for (unsigned it = 0; it < SPIN_LIMIT && !ok; ++it) ok = mbar_try(bar, (c >> 1) & 1);
        if (!ok) { sh->failed = 1; atomicExch(a.err, (int)BILD_ERR_TIMEOUT); }
      }
    }
    if (one_row) {   // thread <-> (key, quarter of the channels); the quarters meet by shuffle
      const int jj = tid >> 2, qt = tid & 3, j = jc + jj;
      const int rot = ((qt >> 1) + 2 * (jj & 1)) & 3;   // rotated walk: the eight threads of a wavefront hit different banks
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int er = qt * 16 + (((e + rot) & 3) << 2);
        const float4 kv = *reinterpret_cast<const float4*>(sK + jj * 64 + er);
        const float4 qv = *reinterpret_cast<const float4*>(sQ + er);
        s0 += kv.x * qv.x + kv.y * qv.y;
        s1 += kv.z * qv.z + kv.w * qv.w;
      }
      float accs = s0 + s1;
      accs += __shfl_xor_sync(0xffffffffu, accs, 1);
      accs += __shfl_xor_sync(0xffffffffu, accs, 2);
      if (qt == 0) {
        float sc = -INFINITY;
        if (jj < nk && (a.mode != 1 || j <= pos0)) {
          if (a.mode != 0) {
            const int dd = pos0 - j;
            accs += bias_staged ? sBias[dd - dmin] : __ldg(a.bias + (size_t)h * a.bias_ld + dd);
          }
          sc = accs;
        }
        sS[jj] = sc;
      }
    } else
    // scores of all rows: one (row, key) pair per thread and turn
#pragma unroll 1
    for (int idx = tid; idx < M * UA_CK; idx += NT) {
      const int i = idx >> 6, jj = idx & (UA_CK - 1);
      float sc = -INFINITY;
      const int j = jc + jj;
      if (jj < nk && (a.mode != 1 || j <= pos0 + i)) {
        float accs = 0.f;
        const int nq4 = dkv >> 2;
#pragma unroll 4
        for (int e = 0; e < nq4; ++e) {
          const int er = ((e + jj) & (nq4 - 1)) << 2;
          const float4 kv = *reinterpret_cast<const float4*>(sK + jj * dkv + er);
          const float4 qv = *reinterpret_cast<const float4*>(sQ + i * dkv + er);
          accs += kv.x * qv.x + kv.y * qv.y + kv.z * qv.z + kv.w * qv.w;
        }
        if (a.mode != 0) {
          const int dd = a.mode == 1 ? pos0 + i - j : a.bias_off + j - (row0 + i);
          accs += bias_staged ? sBias[dd - dmin] : __ldg(a.bias + (size_t)h * a.bias_ld + dd);
        }
        sc = accs;
      }
      sS[idx] = sc;
    }
    __syncthreads();
#pragma unroll 1
    for (int row = warp; row < M; row += NT >> 5) {   // running soft-max, one warp per row
      const float s0 = sS[row * UA_CK + lane], s1 = sS[row * UA_CK + 32 + lane];
      const float mx = warp_max(fmaxf(s0, s1));
      const float mo = sh->amax[row], mn = fmaxf(mo, mx);
      const float p0 = s0 == -INFINITY ? 0.f : __expf(s0 - mn), p1 = s1 == -INFINITY ? 0.f : __expf(s1 - mn);
      sS[row * UA_CK + lane] = p0;
      sS[row * UA_CK + 32 + lane] = p1;
      const float sum = warp_sum(p0 + p1);
      if (lane == 0) {
        const float scale = mo == -INFINITY ? 0.f : __expf(mo - mn);
        sh->ascale[row] = scale;
        sh->asum[row] = sh->asum[row] * scale + sum;
        sh->amax[row] = mn;
      }
    }
    __syncthreads();
    if (one_row) {   // weighted values: thread <-> (quarter of the chunk's keys, channel); the quarters are added in order
      const int kq = tid >> 6, jb = kq * 16;
      float a0 = 0.f, a1 = 0.f;
#pragma unroll
      for (int t = 0; t < 16; t += 2) {
        if (jb + t < nk) a0 += sS[jb + t] * sV[(jb + t) * 64 + pv_c];
        if (jb + t + 1 < nk) a1 += sS[jb + t + 1] * sV[(jb + t + 1) * 64 + pv_c];
      }
      sP1[tid] = a0 + a1;
      __syncthreads();
      if (tid < 64) pv_acc[0] = pv_acc[0] * sh->ascale[0] + (((sP1[tid] + sP1[64 + tid]) + sP1[128 + tid]) + sP1[192 + tid]);
    } else
#pragma unroll
    for (int gp = 0; gp < 4; ++gp) {   // weighted values: thread <-> (row gp * RG + pv_i, channel pv_c)
      const int i = gp * RG + pv_i;
      if (gp >= ngroups || pv_i >= RG || i >= M) continue;
      float a0 = 0.f, a1 = 0.f;
      const float* pr = sS + i * UA_CK;
      int jj = 0;
#pragma unroll 4
      for (; jj + 1 < nk; jj += 2) {
        a0 += pr[jj] * sV[jj * dkv + pv_c];
        a1 += pr[jj + 1] * sV[(jj + 1) * dkv + pv_c];
      }
      if (jj < nk) a0 += pr[jj] * sV[jj * dkv + pv_c];
      pv_acc[gp] = pv_acc[gp] * sh->ascale[i] + (a0 + a1);
    }
    __syncthreads();   // probabilities and the chunk's buffer are free again
    issue_to(min(nchunks, c + 3));
  }
  // finish: a lone split writes the rows; otherwise every split hands its sums to the first block
  // (which is known to be running once the cluster barrier entered at the start completes)
  if (ns > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
#pragma unroll
  for (int gp = 0; gp < 4; ++gp) {
    if (gp >= ngroups) break;
    const int i = gp * RG + pv_i;
    if (pv_i >= RG || i >= M) continue;
    if (ns == 1) {
      const float l = sh->asum[i];
      a.out[(size_t)(row0 + i) * a.ldo + h * dkv + pv_c] = l > 0.f ? pv_acc[gp] / l : 0.f;
    } else {
      float* mrow = sM + ((size_t)sp * MB + i) * pst;
      st_cluster_f1(smem_u32(mrow + 2 + pv_c), 0, pv_acc[gp]);
      if (pv_c == 0) { st_cluster_f1(smem_u32(mrow), 0, sh->amax[i]); st_cluster_f1(smem_u32(mrow + 1), 0, sh->asum[i]); }
    }
  }
  if (ns == 1) return;
  cluster_sync_all();
  if (sp != 0) return;
#pragma unroll 1
  for (int idx = tid; idx < (M << dsh); idx += NT) {
    const int i = idx >> dsh, c = idx & (dkv - 1);
    // at most 8 splits: the loads and exponentials of the splits are independent of each other, only the sums run in order
    float pm[8], pl[8], pa[8];
#pragma unroll
    for (int s2 = 0; s2 < 8; ++s2) {
      const float* Ps = sM + ((size_t)min(s2, ns - 1) * MB + i) * pst;
      pm[s2] = s2 < ns ? Ps[0] : -INFINITY;
      pl[s2] = s2 < ns ? Ps[1] : 0.f;
      pa[s2] = Ps[2 + c];
    }
    float gm = -INFINITY;
#pragma unroll
    for (int s2 = 0; s2 < 8; ++s2) gm = fmaxf(gm, pm[s2]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int s2 = 0; s2 < 8; ++s2) {   // split order
      const float w = pl[s2] > 0.f ? __expf(pm[s2] - gm) : 0.f;
      den += pl[s2] * w;
      num += pa[s2] * w;
    }
    a.out[(size_t)(row0 + i) * a.ldo + h * dkv + c] = den > 0.f ? num / den : 0.f;
  }
}

}  // namespace bild
