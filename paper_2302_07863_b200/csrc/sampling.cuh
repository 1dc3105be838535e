// Sampling variant of the decode loop (supplementary material, "BiLD with Sampling"): both models draw their
// tokens by nucleus (top-p) sampling, the fallback and rollback policies stay as they are.  In this mode the LM-head
// kernels leave the logits of the pass in memory and skip the policy step; the kernel below, launched right after
// the head, draws the one token the pass emits (row 0 of a small step; the first violating row, else the last row,
// of a large pass) and then runs the policy step and the loop graph's conditionals.
//
// Definition followed (one row of V logits z, log-sum-exp known from the head, uniform number u of the output
// position): p_i = exp(z_i - lse); tokens in order of decreasing p (equal p: lower index first); nucleus = shortest
// prefix whose probabilities add up to at least top_p; drawn token = first of the prefix at which the running sum
// exceeds u times the prefix's total.  Both prefixes are found without sorting, by a radix search over the bit
// patterns of the probabilities: four passes over the row, each fixing eight more bits of the threshold value from
// the probability mass per bucket.
#pragma once
#include "kernels.cuh"

namespace bild {

constexpr int NS_THREADS = 1024;

struct NucleusShared {
  float mass[256];
  unsigned cnt[256];
  unsigned key;        // bits of the threshold probability fixed so far
  float above;         // mass of the probabilities above the current bucket range
  unsigned ties;       // tokens with exactly the threshold probability that are taken
  unsigned n_eq;       // tokens with exactly the threshold probability
  int row, token;
  unsigned scan[NS_THREADS / 32];
};

// Finds the probability value at which the running sum over the tokens, taken in decreasing order of probability,
// first reaches (strict = false: >=) or exceeds (strict = true: >) `thresh`.  On return sh->key holds its bit
// pattern, sh->above the mass of all larger probabilities, sh->ties how many tokens of exactly that probability the
// prefix takes (at least 1), sh->n_eq how many there are.  If rounding keeps the total below thresh, the prefix is
// everything.
__device__ inline void nucleus_select(const float* __restrict__ z, float lse, int V, float thresh, bool strict, NucleusShared* sh) {
  const int tid = threadIdx.x;
  if (tid == 0) { sh->key = 0u; sh->above = 0.f; }
  unsigned mask = 0u;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) { sh->mass[tid] = 0.f; sh->cnt[tid] = 0u; }
    __syncthreads();
    const unsigned prefix = sh->key;
#pragma unroll 1
    for (int i = tid; i < V; i += NS_THREADS) {
      const float p = expf(z[i] - lse);
      const unsigned key = __float_as_uint(p);
      if ((key & mask) == prefix) {
        atomicAdd(&sh->mass[(key >> shift) & 255u], p);
        atomicAdd(&sh->cnt[(key >> shift) & 255u], 1u);
      }
    }
    __syncthreads();
    if (tid == 0) {
      float run = sh->above;
      int pick = -1, lowest = 0;
      for (int b = 255; b >= 0; --b) {
        if (sh->cnt[b] == 0u) continue;
        lowest = b;
        const float with = run + sh->mass[b];
        if (strict ? with > thresh : with >= thresh) { pick = b; break; }
        run += sh->mass[b];
      }
      if (pick < 0) { pick = lowest; run -= sh->mass[lowest]; }   // the whole row is the prefix
      sh->above = run;
      sh->key = prefix | ((unsigned)pick << shift);
      if (pass == 3) {
        const float kv = __uint_as_float(sh->key);
        const unsigned n = sh->cnt[pick];
        unsigned t = 1u;
        while (t < n && !(strict ? run + (float)t * kv > thresh : run + (float)t * kv >= thresh)) ++t;
        sh->ties = t;
        sh->n_eq = n;
      }
    }
    mask |= 255u << shift;
    __syncthreads();
  }
}

// Index of the t-th (1-based) token whose probability has exactly the bit pattern `key`, in index order.
__device__ inline void nucleus_locate(const float* __restrict__ z, float lse, int V, unsigned key, unsigned t, NucleusShared* sh) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (V + NS_THREADS - 1) / NS_THREADS, i0 = tid * per, i1 = min(V, i0 + per);
  unsigned mine = 0u;
  for (int i = i0; i < i1; ++i) mine += __float_as_uint(expf(z[i] - lse)) == key ? 1u : 0u;
  unsigned inc = mine;   // inclusive scan over the block, thread order = index order
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) sh->scan[warp] = inc;
  __syncthreads();
  unsigned base = 0u;
  for (int w = 0; w < warp; ++w) base += sh->scan[w];
  const unsigned before = base + inc - mine;
  if (mine > 0u && before < t && t <= before + mine) {
    unsigned seen = before;
    for (int i = i0; i < i1; ++i)
      if (__float_as_uint(expf(z[i] - lse)) == key && ++seen == t) { sh->token = i; break; }
  }
  __syncthreads();
}

// logits: [MAXB][V] of the pass that just ran; u: uniform numbers by output position of this model.
__global__ void __launch_bounds__(NS_THREADS) nucleus_policy_kernel(HeadArgs a, const float* __restrict__ logits, const float* __restrict__ u) {
  __shared__ NucleusShared sh;
  pdl_launch_dependents();
  pdl_wait();
  HeadOut* o = a.out;
  const int V = a.V;
  if (threadIdx.x == 0) {
    policy_tests(o, a.desc, a.loop.st, a.which);
    sh.row = a.which == 0 ? 0 : (o->first_violation >= 0 ? o->first_violation : a.desc->k - 1);
    sh.token = o->argmax[sh.row];
  }
  __syncthreads();
  const int r = sh.row;
  const float* z = logits + (size_t)r * V;
  const float lse = o->lse[r];
  const float un = u[a.desc->pos0 + r + 1];   // the position in y the drawn token is written to
  nucleus_select(z, lse, V, a.loop.st->top_p, false, &sh);
  const unsigned key1 = sh.key, ties1 = sh.ties;
  const float total = sh.above + (float)ties1 * __uint_as_float(key1);
  __syncthreads();
  nucleus_select(z, lse, V, un * total, true, &sh);
  unsigned key2 = sh.key, t2 = sh.ties;
  if (key2 < key1 || (key2 == key1 && t2 > ties1)) { key2 = key1; t2 = ties1; }   // rounding: stay inside the nucleus
  __syncthreads();
  nucleus_locate(z, lse, V, key2, t2, &sh);
  if (threadIdx.x == 0) {
    o->argmax[r] = sh.token;
    if (a.cond_while) a.loop.st->cum_draws++;
    HeadArgs b = a;
    b.defer_policy = 0;
    policy_tail(b, o);
  }
}

}  // namespace bild
