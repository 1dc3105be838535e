// Block linear layer of the large-model pass on the 5th-generation tensor cores
// (steps L1, L3, L4, L6, L7, L8): Y^T = W X^T for up to 16 token rows ("swap-AB": the weight's
// output dimension rides the MMA's M = 128 axis, the tokens its N = 16 axis).
//   * the bf16 weight tile [128 rows][64 k] arrives by TMA (128-byte swizzle) into a ring of
//     shared-memory stages, the first stages before the dependency wait of the launch;
//   * the fp32 activations (times the norm gain) are split into bf16 hi + bf16 lo and both
//     are multiplied against the same weight tile, so the weights are read once and the
//     product carries ~16 mantissa bits of the activation;
//   * accumulators live in tensor memory (one 16-column block per weight matrix);
//   * K is split over the CTAs of a thread-block cluster; their partial tiles (and partial
//     sums of squares for the RMS norm) are summed in rank order in the leader's shared
//     memory, so the result does not depend on timing;
//   * every wait on an mbarrier is bounded: on expiry an error code is recorded and the
//     block carries on to its barriers and frees its tensor memory.
#pragma once
#include <cuda.h>

#include "kernels.cuh"

namespace bild {

constexpr int UM_THREADS = 128;
constexpr int UM_TILE_M = 128;   // weight rows per CTA
constexpr int UM_KB = 64;        // k per stage = one 128-byte swizzle atom of bf16
constexpr int UM_STAGES = 8;
constexpr int UM_MAX_KB = 24;    // k blocks per CTA (activation tiles are resident)
constexpr uint32_t UM_SPIN_LIMIT = 1u << 20;

struct UmmaArgs {
  LinArgs lin;       // same operands / epilogues as linear_kernel (W pointers unused here)
  int cs;            // cluster size along K
  int nkb;           // k blocks (of 64) per CTA
  int* err;
};

// ---- raw PTX helpers --------------------------------------------------------------

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait; returns false (and the caller records an error) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < UM_SPIN_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// K-major operand tile with 128-byte swizzle: rows are 128 bytes, 8-row atoms are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);   // start address
  d |= (uint64_t)1 << 16;                    // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row atoms
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                    // SWIZZLE_128B
  return d;
}
// bf16 x bf16 -> fp32, A and B K-major, M = 128, N = 32 (16 token rows of hi, then 16 of lo)
constexpr uint32_t UM_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((32u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(UM_IDESC), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// 32 columns of this warp's 32 lanes, requested only: tmem_ld_wait() before the registers are read
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,"
      "%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// ties the registers of an earlier issue-only load to this point of the instruction stream (no instruction of its own):
// nothing that reads them may move above the wait in front
template <int N>
__device__ __forceinline__ void tmem_ld_pin(uint32_t (&r)[N]) {
#pragma unroll
  for (int i = 0; i < N; ++i) asm volatile("" : "+r"(r[i])::"memory");
}
// Shared-memory plan (bytes) for a launch; the kernel carves the same layout.
__host__ __device__ inline size_t umma_smem_bytes(bool gated, int nkb, int cs) {
  const size_t a = (size_t)(gated ? 4 : 8) * (gated ? 2 : 1) * 16384;   // weight stages
  const size_t b = (size_t)nkb * 4096;                                  // activations hi + lo
  const size_t red = (size_t)(cs > 1 ? cs - 1 : 0) * UM_TILE_M * 16 * 4 * (gated ? 2 : 1);
  return 1024 /*alignment slack*/ + a + b + red + 1024 /*ss partials, barriers, tmem slot*/;
}

template <bool GATED>
__global__ void __launch_bounds__(UM_THREADS) umma_linear_kernel(UmmaArgs u, const __grid_constant__ CUtensorMap tm0,
                                                                 const __grid_constant__ CUtensorMap tm1) {
  constexpr int NST = GATED ? 4 : 8;
  constexpr int NMAT = GATED ? 2 : 1;
  constexpr int TCOLS = 32 * NMAT;   // accumulator columns in tensor memory: [hi 16 | lo 16] per matrix
  extern __shared__ unsigned char um_raw[];
  // blockIdx.y selects a block of MAXB token rows (encoder: many blocks; decoder passes: one)
  LinArgs a = u.lin;
  const int row0 = blockIdx.y * MAXB;
  a.X += (size_t)row0 * a.ldx;
  if (a.Y) a.Y += (size_t)row0 * a.ldy;
  if (a.q_out) a.q_out += (size_t)row0 * a.ldq;
  a.pos0_host += row0;
  a.M -= row0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cs = u.cs, nkb = u.nkb;
  const uint32_t rank = cs > 1 ? cluster_rank() : 0;
  const int tile = blockIdx.x / cs;
  const int n_base = tile * UM_TILE_M;
  const int k_base = (int)rank * nkb * UM_KB;

  unsigned char* base = (unsigned char*)(((uintptr_t)um_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* sA = base;                                      // [NST][NMAT][16 KB]
  unsigned char* sB = sA + (size_t)NST * NMAT * 16384;           // [nkb][hi 2 KB | lo 2 KB]
  float* sRed = (float*)(sB + (size_t)nkb * 4096);               // [cs-1][NMAT][128][16]
  float* sSS = sRed + (size_t)(cs > 1 ? cs - 1 : 0) * NMAT * UM_TILE_M * 16;   // [8][16]
  uint64_t* full = (uint64_t*)(sSS + 9 * 16);   // [8][16] sums of squares per rank, [16] 1/rms
  uint64_t* empty = full + NST;
  uint64_t* done = empty + NST;
  uint32_t* tmem_slot = (uint32_t*)(done + 1);

  if (tid == 0) {
    for (int i = 0; i < NST; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(done, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(TCOLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;
  // every block of the cluster must be running before anyone stores into a peer's shared memory
  if (cs > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

  // weights do not depend on the previous kernel: fill the ring before the dependency wait
  if (tid == 0) {
    for (int kb = 0; kb < nkb && kb < NST; ++kb) {
      mbar_expect_tx(&full[kb], NMAT * 16384);
      tma_load_2d(sA + (size_t)kb * NMAT * 16384, &tm0, k_base + kb * UM_KB, n_base, &full[kb]);
      if (GATED) tma_load_2d(sA + (size_t)kb * NMAT * 16384 + 16384, &tm1, k_base + kb * UM_KB, n_base, &full[kb]);
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  if (cs > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");

  // Everything that needs a round trip to memory is requested here at once: the descriptor,
  // the residual rows this block will update, and (below) the activations.  All MAXB rows of
  // the activation buffers exist, so they are loaded without waiting for the row count; rows
  // beyond it only feed accumulator columns that the epilogue ignores.
  const int M = a.desc ? a.desc->k : a.M;
  const int pos0 = a.desc ? a.desc->pos0 : a.pos0_host;
  float old[MAXB];
  if (rank == 0 && a.epi == EPI_RESID && n_base + tid < a.N) {
#pragma unroll
    for (int m = 0; m < MAXB; ++m) old[m] = a.Y[(size_t)m * a.ldy + n_base + tid];
  }
  const int kl = nkb * UM_KB;
  {  // warp w owns rows w, w+4, w+8, w+12.  Two column chunks (2 x 256) of all four rows are
     // requested before any of them is converted, so a block with up to 512 columns needs one
     // round trip to L2 for its activations.
    float ssr[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
    for (int cb = lane * 8; cb < kl; cb += 512) {
      float4 xa[2][4], xb[2][4], g0[2], g1[2];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int c = cb + 256 * j;
        g0[j] = g1[j] = make_float4(1.f, 1.f, 1.f, 1.f);
        if (c < kl) {
          if (a.gain) {
            g0[j] = *reinterpret_cast<const float4*>(a.gain + k_base + c);
            g1[j] = *reinterpret_cast<const float4*>(a.gain + k_base + c + 4);
          }
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const float* xp = a.X + (size_t)(warp + 4 * r) * a.ldx + k_base + c;
            xa[j][r] = *reinterpret_cast<const float4*>(xp);
            xb[j][r] = *reinterpret_cast<const float4*>(xp + 4);
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int c = cb + 256 * j;
        if (c < kl) {
          const int kb = c / UM_KB, chunk = (c % UM_KB) / 8;
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const int m = warp + 4 * r;
            float h[8] = {xa[j][r].x, xa[j][r].y, xa[j][r].z, xa[j][r].w, xb[j][r].x, xb[j][r].y, xb[j][r].z, xb[j][r].w};
            const float gg[8] = {g0[j].x, g0[j].y, g0[j].z, g0[j].w, g1[j].x, g1[j].y, g1[j].z, g1[j].w};
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              ssr[r] += h[2 * i] * h[2 * i] + h[2 * i + 1] * h[2 * i + 1];
              const float e0 = h[2 * i] * gg[2 * i], e1 = h[2 * i + 1] * gg[2 * i + 1];
              const __nv_bfloat16 h0 = __float2bfloat16_rn(e0), h1 = __float2bfloat16_rn(e1);
              const __nv_bfloat16 l0 = __float2bfloat16_rn(e0 - __bfloat162float(h0));
              const __nv_bfloat16 l1 = __float2bfloat16_rn(e1 - __bfloat162float(h1));
              hi[i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
              lo[i] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
            }
            const uint32_t off = (uint32_t)kb * 4096 + (m >> 3) * 1024 + (m & 7) * 128 + ((chunk ^ (m & 7)) << 4);
            *reinterpret_cast<uint4*>(sB + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4*>(sB + off + 2048) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int m = warp + 4 * r;
      const float ss = warp_sum(ssr[r]);
      if (lane == 0) {
        if (rank == 0) sSS[m] = ss;
        else st_cluster_f1(smem_u32(&sSS[rank * 16 + m]), 0, ss);
      }
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  // ---- producer (rest of the ring) and MMA issue ----
  if (tid == 0) {
    for (int kb = NST; kb < nkb; ++kb) {
      const int st = kb % NST;
      if (!mbar_wait(&empty[st], ((kb / NST) - 1) & 1)) *u.err = BILD_ERR_TIMEOUT;
      mbar_expect_tx(&full[st], NMAT * 16384);
      tma_load_2d(sA + (size_t)st * NMAT * 16384, &tm0, k_base + kb * UM_KB, n_base, &full[st]);
      if (GATED) tma_load_2d(sA + (size_t)st * NMAT * 16384 + 16384, &tm1, k_base + kb * UM_KB, n_base, &full[st]);
    }
  } else if (tid == 32) {
    for (int kb = 0; kb < nkb; ++kb) {
      const int st = kb % NST;
      if (!mbar_wait(&full[st], (kb / NST) & 1)) *u.err = BILD_ERR_TIMEOUT;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t a0 = smem_u32(sA + (size_t)st * NMAT * 16384);
      const uint32_t bh = smem_u32(sB + (size_t)kb * 4096);
#pragma unroll
      for (int kk = 0; kk < UM_KB / 16; ++kk) {
        // one MMA covers hi (token rows 0..15) and lo (rows 16..31) of the activation tile,
        // so each weight tile is read from shared memory once
        const uint64_t db = umma_desc_sw128(bh + kk * 32);
        umma_bf16(tmem, umma_desc_sw128(a0 + kk * 32), db, (kb | kk) ? 1u : 0u);
        if (GATED) umma_bf16(tmem + 32, umma_desc_sw128(a0 + 16384 + kk * 32), db, (kb | kk) ? 1u : 0u);
      }
      umma_commit(&empty[st]);   // the stage may be refilled once these MMAs have read it
    }
    umma_commit(done);
  }
  __syncwarp();
  if (!mbar_wait(done, 0)) *u.err = BILD_ERR_TIMEOUT;
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  // ---- accumulators: thread t holds weight row n_base + t for the 16 token rows ----
  float acc0[16], acc1[16];
  {
    float lo16[16];
    const uint32_t t0 = tmem + ((uint32_t)(warp * 32) << 16);
    tmem_ld16(t0, acc0);
    tmem_ld16(t0 + 16, lo16);
#pragma unroll
    for (int i = 0; i < 16; ++i) acc0[i] += lo16[i];
    if (GATED) {
      tmem_ld16(t0 + 32, acc1);
      tmem_ld16(t0 + 48, lo16);
#pragma unroll
      for (int i = 0; i < 16; ++i) acc1[i] += lo16[i];
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");

  if (cs > 1) {
    if (rank != 0) {
      // layout [rank-1][matrix][token i][row tid]: consecutive threads, consecutive words
      float* dst = sRed + (size_t)(rank - 1) * NMAT * UM_TILE_M * 16 + tid;
#pragma unroll
      for (int i = 0; i < 16; ++i) st_cluster_f1(smem_u32(dst + i * UM_TILE_M), 0, acc0[i]);
      if (GATED) {
#pragma unroll
        for (int i = 0; i < 16; ++i) st_cluster_f1(smem_u32(dst + (16 + i) * UM_TILE_M), 0, acc1[i]);
      }
    }
    cluster_sync_all();
  }
  if (rank == 0) {
    for (int r = 1; r < cs; ++r) {   // fixed order: rank 1, 2, ...
      const float* src = sRed + (size_t)(r - 1) * NMAT * UM_TILE_M * 16 + tid;
#pragma unroll
      for (int i = 0; i < 16; ++i) acc0[i] += src[i * UM_TILE_M];
      if (GATED) {
#pragma unroll
        for (int i = 0; i < 16; ++i) acc1[i] += src[(16 + i) * UM_TILE_M];
      }
    }
    // 1 / rms per token row: threads 0..15 add the ranks' sums of squares in rank order
    if (tid < MAXB) {
      float ss = 0.f;
      for (int r = 0; r < cs; ++r) ss += sSS[r * 16 + tid];
      sSS[8 * 16 + tid] = a.gain ? rsqrtf(ss / (float)a.K + a.eps) : 1.f;
    }
    __syncthreads();
  }
  if (rank == 0) {
    const int n = n_base + tid;
    const int mrows = min(MAXB, M);
    const float* sInv = sSS + 8 * 16;
    if (n < a.N) {
      if (a.epi == EPI_RESID) {   // the old values were requested right after the dependency wait
#pragma unroll
        for (int m = 0; m < MAXB; ++m)
          if (m < mrows) a.Y[(size_t)m * a.ldy + n] = old[m] + acc0[m] * sInv[m];
      } else if (a.epi == EPI_HEADS) {
        int part = a.first_part, rr = n;
        if (rr >= a.inner) { rr -= a.inner; ++part; }
        if (rr >= a.inner) { rr -= a.inner; ++part; }
        const int h = rr / a.dkv, c = rr % a.dkv;
#pragma unroll
        for (int m = 0; m < MAXB; ++m) {
          if (m < mrows) {
            const float v = acc0[m] * sInv[m];
            if (part == 0) a.q_out[(size_t)m * a.ldq + rr] = v;
            else if (pos0 + m < a.cap) (part == 1 ? a.kc : a.vc)[((size_t)h * a.cap + pos0 + m) * a.dkv + c] = v;
          }
        }
      } else {
#pragma unroll 1
        for (int m = 0; m < mrows; ++m) {
          // registers cannot be indexed in a rolled loop: pick the row's values with selects
          float y = 0.f, y1 = 0.f;
#pragma unroll
          for (int q = 0; q < MAXB; ++q) { if (q == m) { y = acc0[q]; if (GATED) y1 = acc1[q]; } }
          y *= sInv[m];
          if (a.epi == EPI_RELU) y = fmaxf(y, 0.f);
          else if (a.epi == EPI_GATED) { if (GATED) y = gelu_tanh(y) * (y1 * sInv[m]); }
          a.Y[(size_t)m * a.ldy + n] = y;
        }
      }
    }
  }
  __syncthreads();
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(TCOLS) : "memory");
}

}  // namespace bild
