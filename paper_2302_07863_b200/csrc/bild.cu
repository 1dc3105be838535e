// libbild host runtime: workspace planning, launch sequences of the encoder and of the
// two decoder passes, the decode loop driver, and the extern "C" boundary (include/bild.h).
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "decode_kernels.cuh"
#include "slice_linear.cuh"
#include "unit_attention.cuh"
#include "slice_head.cuh"
#include "umma_linear.cuh"
#include "enc_gemm.cuh"
#include "enc_attention.cuh"
#include "sublayer.cuh"
#include "sampling.cuh"

using namespace bild;

// ------------------------------------------------------------------------------------
// relative-position buckets, exact integer arithmetic
// ------------------------------------------------------------------------------------
namespace {

struct Big {  // non-negative big integer, little-endian base 2^32
  std::vector<uint32_t> d{1};
  void mul(uint32_t f) {
    uint64_t carry = 0;
    for (auto& w : d) { uint64_t t = (uint64_t)w * f + carry; w = (uint32_t)t; carry = t >> 32; }
    if (carry) d.push_back((uint32_t)carry);
  }
  void mul_pow(uint32_t base, int e) { for (int i = 0; i < e; ++i) mul(base); }
  bool ge(const Big& o) const {
    size_t na = d.size(), nb = o.d.size();
    while (na > 1 && d[na - 1] == 0) --na;
    while (nb > 1 && o.d[nb - 1] == 0) --nb;
    if (na != nb) return na > nb;
    for (size_t i = na; i-- > 0;) if (d[i] != o.d[i]) return d[i] > o.d[i];
    return true;
  }
};

// for dist >= max_exact: max_exact + floor(n_log * ln(dist/max_exact) / ln(max_dist/max_exact)),
// capped at max_exact + n_log - 1: the largest j with dist^n_log * max_exact^j >= max_dist^j * max_exact^n_log
int log_bucket(int dist, int max_exact, int n_log, int max_dist) {
  if (dist >= max_dist) return max_exact + n_log - 1;
  int j = 0;
  while (j + 1 <= n_log - 1) {
    Big lhs, rhs;
    lhs.mul_pow((uint32_t)dist, n_log); lhs.mul_pow((uint32_t)max_exact, j + 1);
    rhs.mul_pow((uint32_t)max_dist, j + 1); rhs.mul_pow((uint32_t)max_exact, n_log);
    if (!lhs.ge(rhs)) break;
    ++j;
  }
  return max_exact + j;
}

int decoder_bucket(int delta, int n_buckets, int max_dist) {  // delta = query - key >= 0
  const int max_exact = n_buckets / 2;
  if (delta < max_exact) return delta;
  return log_bucket(delta, max_exact, n_buckets - max_exact, max_dist);
}

int encoder_bucket(int rel, int n_buckets, int max_dist) {  // rel = key - query
  const int half = n_buckets / 2;
  const int off = rel > 0 ? half : 0;
  const int dist = rel < 0 ? -rel : rel;
  const int max_exact = half / 2;
  if (dist < max_exact) return off + dist;
  return off + log_bucket(dist, max_exact, half - max_exact, max_dist);
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Bump {  // carves the caller's workspace; with base == nullptr it only measures
  char* base;
  size_t off = 0;
  explicit Bump(void* b) : base((char*)b) {}
  template <typename T> T* take(size_t n) {
    off = align_up(off, 256);
    T* p = base ? (T*)(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
};

constexpr int NSPLIT_MAX = 32;
constexpr int HEAD_GRID_MAX = 148 * 4;

struct Model {
  bild_model_cfg c{};
  bild_weights w{};
  std::vector<bild_enc_layer> enc;
  std::vector<bild_dec_layer> dec;
  int inner = 0;
  float *selfK = nullptr, *selfV = nullptr, *crossK = nullptr, *crossV = nullptr;
  float *x = nullptr, *q = nullptr, *att = nullptr, *u = nullptr;
  float *dec_bias = nullptr, *enc_bias = nullptr;
  float* att_part = nullptr;
  unsigned* att_cnt = nullptr;
  Partial* head_part = nullptr;
  unsigned* head_cnt = nullptr;
  HeadOut* head_out = nullptr;
  CallDesc* desc = nullptr;
  int head_grid = 0;
  // TMA descriptors of the decoder's weight matrices (bf16 only): per layer qkv, o, cq, co, wi0, wi1, fo
  std::vector<CUtensorMap> tmaps;
  bool umma = false;
  // encoder GEMM: descriptors of the bf16 head / remainder matrices of the layer input, by row length (d, inner, d_ff)
  CUtensorMap tmH[2][3][2];   // [buffer pair][row length d / inner / d_ff][head, remainder]
  bool enc_gemm = false;
  int index = 0;   // 0 small, 1 large
  // fused sub-layer kernels (bf16 only): two more residual-stream buffers, W_fo transposed per layer
  float *xb = nullptr, *xc = nullptr;
  float* logits = nullptr;           // [MAXB][V] logits of the last pass (sampling variant only)
  bool fused = false;
  int sub_C = 1;                     // blocks per head (cluster size) of the attention sub-layers
  uint4* wfo_one = nullptr;          // [layers][F / 8][d] W_fo in the load order of the fused feed-forward kernels
  uint4* wfo_blk = nullptr;          // [layers][F / 8][pack_wfo_dpad(d)]
  CallDesc* desc_lo = nullptr;       // the two chunks of a block of 9 to 16 rows (split_desc_kernel)
  CallDesc* desc_hi = nullptr;
  AttnSubPlan sub_self[2]{}, sub_cross[2]{};   // chunk sizes of the attention sub-layers: [0] single-row kernel, [1] block kernel
  int sub_parts = 1;                 // launches the feed-forward sub-layer is split into
};

}  // namespace

struct bild_ctx {
  bild_config cfg{};
  Model m[2];
  cudaStream_t stream = nullptr;
  DevState* st = nullptr;
  int* y = nullptr;
  bild_trace_rec* trace = nullptr;
  int trace_cap = 0;
  int* enc_ids = nullptr;
  int* enc_len_dev = nullptr;
  int* bucket_tmp = nullptr;
  float* u_draw[2] = {nullptr, nullptr};   // uniform numbers by output position, small / large model (sampling variant)
  float top_p = 0.f;                       // > 0 while a sampled generation is set up or running
  bool draw = false;                       // decoder passes are followed by the token-drawing kernel
  // encoder temporaries, one set per model (the two encoders run side by side on two streams)
  struct EncBuf {
    float *ex = nullptr, *eq = nullptr, *ek = nullptr, *ev = nullptr, *eatt = nullptr, *eu = nullptr;
    __nv_bfloat16 *exh[2] = {nullptr, nullptr}, *exl[2] = {nullptr, nullptr};   // two pairs (bf16 head, remainder) of layer inputs
  } eb[2];
  cudaStream_t enc_stream = nullptr;   // the small model's encoder runs here, the large model's on the caller's stream
  cudaEvent_t enc_fork = nullptr, enc_join = nullptr;
  bool enc_parallel = true;
  int enc_len = 0;
  bool encoded = false;
  int64_t launches = 0;
  std::string err;
  DevState* pin_state = nullptr;  // pinned host mirror for the loop driver
  HeadOut* pin_head = nullptr;
  size_t ws_bytes = 0;
  // device-side loop: WHILE { small pass; IF (fallback) { large block pass } } and WHILE { large pass }
  // [0], [1]: greedy; [2], [3]: the same two loops with the token-drawing kernel after every LM head
  cudaGraph_t graph[4] = {nullptr, nullptr, nullptr, nullptr};
  cudaGraphExec_t exec[4] = {nullptr, nullptr, nullptr, nullptr};
  int64_t sampled_counted = 0;
  int64_t per_pass[2] = {0, 0};      // kernel launches in one small / one large pass of the graphs
  int64_t per_pass_large1 = 0, per_pass_large8 = 0;
  int64_t* cnt = &launches;         // where launches are counted (redirected while capturing)
  bool fused_embed = true;            // the first fused sub-layer kernel of a pass gathers the embedding rows (no embedding kernel)
  bool enc_kv_streams = true;         // cross K/V projections of the decoder layers dealt to three streams
  cudaStream_t kv_stream[2] = {nullptr, nullptr};
  cudaEvent_t kv_fork = nullptr, kv_join[2] = {nullptr, nullptr};
  cudaStream_t side2 = nullptr;       // second chunk of a block of 9 to 16 rows (fused sub-layer kernels)
  std::vector<cudaEvent_t> chunk_ev;  // per layer: first chunk's self-attention done; then fork and join
  cudaStream_t cap_stream = nullptr;  // capture only (the legacy default stream cannot capture); nothing runs on it
  bool block_simt = false;           // block pass on the SIMT block GEMV instead of the tensor-core kernel
  bool use_pdl = true;               // launch pass kernels with programmatic stream serialization
  bool host_loop = false;            // debug: drive the loop from the host, one read-back per step
  int slice_mode = 2;                // row-slice linear kernel: 0 off, 1 block passes, 2 block and single-row passes
  int sms = 0;
  size_t slice_smem_set = 0;
  int head_stream = 2;               // single-row bf16 heads on the streaming kernel: 0 off, 1 heads of slice_head_min_mb and more, 2 all
  bool enc_split_k = true;           // encoder GEMMs that add to the residual stream split K over grid.z (reductions at the L2)
  bool graph_switch = true;          // the large pass of a loop iteration hangs off one SWITCH node (else: one IF node per kind of pass)
  unsigned long long sw_handle = 0;  // while the small pass of such a loop is captured: the SWITCH node's handle and body count
  int sw_bodies = 0;
  int attn_all_keys = 128;           // fused attention: caches up to this many keys are attended by every rank of a head
  bool unit_attn = true;             // decoder attention on the 256-thread chunked kernel
  bool uattn_smem_set = false;
  bool enc_attn_mma = true;          // encoder self-attention on the mma.sync kernel (d_kv = 64)
  int enc_attn_groups = EA_MAX_GROUPS;   // key groups per block of that kernel (1..3)
  int slice_head = 2;                // tensor-core LM head: 0 off, 1 block passes, 2 also single-row passes (large heads)
  bool slice_head_smem_set = false;
  size_t slice_head_min_bytes = (size_t)32 << 20;
  int slice_mma_min = 3;
  size_t slice_min_bytes = 3000 * 1024;   // single-row passes: smaller matrices stay on the GEMV (measured)
  int fused_on = 3;                  // fused sub-layer kernels where the shapes allow: 0 off, 1 single-row passes, 2 also passes of 2 to 8 rows, 3 also 9 to 16 rows (two chunks)
  int sub_parts_want = 0;            // 0: fewest launches of the feed-forward sub-layer that fit
  bool use_umma = true, use_enc_gemm = true;
  unsigned spin_limit = SPIN_LIMIT;
  bool debug_skip_copies = false;
  bool capturing = false;            // launches are being recorded into a graph, not run
  int64_t graph_counted = 0;         // launches of the loop graphs already added to `launches`
};

namespace {

int fail(bild_ctx* c, int code, const std::string& msg) {
  if (c) c->err = msg;
  return code;
}
#define CUDA_TRY(ctx, expr)                                                               \
  do {                                                                                    \
    cudaError_t e_ = (expr);                                                              \
    if (e_ != cudaSuccess)                                                                \
      return fail(ctx, BILD_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e_)); \
  } while (0)

int check_model(const bild_model_cfg& c, std::string& why) {
  auto bad = [&](const char* s) { why = s; return BILD_ERR_ARG; };
  if (c.n_layers < 1 || c.d_model < 8 || c.n_heads < 1 || c.d_ff < 8 || c.vocab < 2) return bad("model sizes must be positive");
  if (c.d_model % 8 || c.d_ff % 8 || (c.n_heads * c.d_kv) % 8) return bad("d_model, d_ff and n_heads*d_kv must be multiples of 8");
  if (c.d_kv != 16 && c.d_kv != 32 && c.d_kv != 64 && c.d_kv != 128) return bad("d_kv must be 16, 32, 64 or 128");
  if (c.d_model > 2048 || c.d_ff > 16384) return bad("d_model <= 2048 and d_ff <= 16384");
  if (c.ffn_kind != BILD_FFN_RELU && c.ffn_kind != BILD_FFN_GATED_GELU) return bad("ffn_kind");
  if (c.rel_buckets < 4 || c.rel_buckets % 4 || c.rel_max_dist < c.rel_buckets) return bad("rel_buckets / rel_max_dist");
  if (!(c.ln_eps >= 0.f) || !(c.logit_scale > 0.f)) return bad("ln_eps >= 0 and logit_scale > 0");
  return BILD_OK;
}

int check_config(const bild_config* cfg, std::string& why) {
  if (!cfg) { why = "null config"; return BILD_ERR_ARG; }
  int rc = check_model(cfg->small_cfg, why);
  if (rc) return rc;
  rc = check_model(cfg->large_cfg, why);
  if (rc) return rc;
  if (cfg->small_cfg.vocab != cfg->large_cfg.vocab) { why = "the two models must share a vocabulary"; return BILD_ERR_ARG; }
  if (cfg->dtype != BILD_FP32 && cfg->dtype != BILD_BF16) { why = "dtype"; return BILD_ERR_ARG; }
  if (cfg->max_enc_len < 1 || cfg->max_enc_len > 2048) { why = "1 <= max_enc_len <= 2048"; return BILD_ERR_ARG; }
  if (cfg->max_dec_len < 2 || cfg->max_dec_len > 2048) { why = "2 <= max_dec_len <= 2048"; return BILD_ERR_ARG; }
  if (cfg->max_draft < 1 || cfg->max_draft > MAXB - 1) { why = "1 <= max_draft <= 15"; return BILD_ERR_ARG; }
  if (cfg->start_id < 0 || cfg->start_id >= cfg->small_cfg.vocab) { why = "start_id"; return BILD_ERR_ARG; }
  if (cfg->early_exit_layers < 0) { why = "early_exit_layers"; return BILD_ERR_ARG; }
  if (cfg->early_exit_layers > 0) {
    const bild_model_cfg &a = cfg->small_cfg, &b = cfg->large_cfg;
    if (a.n_layers != cfg->early_exit_layers || a.n_layers > b.n_layers || a.d_model != b.d_model || a.n_heads != b.n_heads ||
        a.d_kv != b.d_kv || a.d_ff != b.d_ff || a.ffn_kind != b.ffn_kind || a.rel_buckets != b.rel_buckets ||
        a.rel_max_dist != b.rel_max_dist || a.ln_eps != b.ln_eps) {
      why = "early exit: small_cfg must be large_cfg with n_layers = early_exit_layers";
      return BILD_ERR_ARG;
    }
  }
  return BILD_OK;
}

int head_grid_for(int V) { return std::max(1, std::min(HEAD_GRID_MAX, (V + 63) / 64)); }
// partial records either head kernel may write (block head: grid x MAXB; single-row head: up to V / 8 blocks)
size_t head_partial_count(int V) {
  // block head: grid x MAXB; single-row head: up to V / 8 blocks; one-block-per-SM head: SMs x MAXB
  return std::max(std::max((size_t)head_grid_for(V) * MAXB, (size_t)(V + 7) / 8 + 8), (size_t)MAX_GRID_SM * MAXB);
}

// Lays out everything the context keeps on the device.
void plan(bild_ctx* c, Bump& b) {
  const bild_config& cfg = c->cfg;
  const int cap = cfg.max_dec_len, ecap = cfg.max_enc_len;
  c->st = b.take<DevState>(1);
  c->y = b.take<int>(cap + 1);
  c->trace_cap = cap * (cfg.max_draft + 3);
  c->trace = b.take<bild_trace_rec>(c->trace_cap);
  c->enc_ids = b.take<int>(ecap);
  c->enc_len_dev = b.take<int>(1);
  c->bucket_tmp = b.take<int>(std::max(cap, 2 * ecap));
  c->u_draw[0] = b.take<float>(cap + 1);
  c->u_draw[1] = b.take<float>(cap + 1);
  for (int i = 0; i < 2; ++i) {
    Model& m = c->m[i];
    const bild_model_cfg& mc = i == 0 ? cfg.small_cfg : cfg.large_cfg;
    m.c = mc;
    m.index = i;
    m.inner = mc.n_heads * mc.d_kv;
    const size_t kv = (size_t)mc.n_layers * mc.n_heads * mc.d_kv;
    m.selfK = b.take<float>(kv * cap);
    m.selfV = b.take<float>(kv * cap);
    m.crossK = b.take<float>(kv * ecap);
    m.crossV = b.take<float>(kv * ecap);
    m.x = b.take<float>((size_t)MAXB * mc.d_model);
    m.q = b.take<float>((size_t)MAXB * m.inner);
    m.att = b.take<float>((size_t)MAXB * m.inner);
    m.u = b.take<float>((size_t)MAXB * mc.d_ff);
    m.dec_bias = b.take<float>((size_t)mc.n_heads * cap);
    m.enc_bias = b.take<float>((size_t)mc.n_heads * (2 * ecap - 1));
    m.att_part = b.take<float>((size_t)MAXB * mc.n_heads * NSPLIT_MAX * (mc.d_kv + 2));
    m.att_cnt = b.take<unsigned>((size_t)MAXB * mc.n_heads);
    m.head_grid = head_grid_for(mc.vocab);
    m.head_part = b.take<Partial>(head_partial_count(mc.vocab));
    m.head_cnt = b.take<unsigned>(1);
    m.head_out = b.take<HeadOut>(1);
    m.desc = b.take<CallDesc>(1);
    m.desc_lo = b.take<CallDesc>(1);
    m.desc_hi = b.take<CallDesc>(1);
    m.logits = b.take<float>((size_t)MAXB * mc.vocab);
    m.xb = b.take<float>((size_t)MAXB * mc.d_model);
    m.xc = b.take<float>((size_t)MAXB * mc.d_model);
    {   // W_fo of every decoder layer in the load order of the fused feed-forward kernels (two orders: one row, blocks)
      const size_t units = cfg.dtype == BILD_BF16 && mc.d_ff % 8 == 0 ? (size_t)mc.n_layers * (mc.d_ff / 8) : 0;
      m.wfo_one = b.take<uint4>(units * mc.d_model);
      m.wfo_blk = b.take<uint4>(units * pack_wfo_dpad(mc.d_model));
    }
  }
  const size_t ecap16 = (size_t)(ecap + MAXB - 1) / MAXB * MAXB;   // whole blocks of MAXB rows
  const size_t ecap128 = (size_t)(ecap + EG_TOK - 1) / EG_TOK * EG_TOK;   // whole tiles of 128 tokens
  for (int i = 0; i < 2; ++i) {
    const bild_model_cfg& mc = i == 0 ? cfg.small_cfg : cfg.large_cfg;
    const size_t d = mc.d_model, I = (size_t)mc.n_heads * mc.d_kv, F = mc.d_ff;
    bild_ctx::EncBuf& e = c->eb[i];
    e.ex = b.take<float>(ecap16 * d);
    e.eq = b.take<float>(ecap16 * I);
    e.ek = b.take<float>((size_t)ecap * I);
    e.ev = b.take<float>((size_t)ecap * I);
    e.eatt = b.take<float>(ecap16 * I);
    e.eu = b.take<float>(ecap16 * F);
    for (int pr = 0; pr < 2; ++pr) {
      e.exh[pr] = b.take<__nv_bfloat16>(ecap128 * std::max(std::max(d, I), F));
      e.exl[pr] = b.take<__nv_bfloat16>(ecap128 * std::max(std::max(d, I), F));
    }
  }
  b.off = align_up(b.off, 256);
}

// ---- launches ------------------------------------------------------------------------
// Every kernel of a pass is launched so that it may start while its predecessor drains
// (programmatic dependent launch); each of them waits before touching dependent data.
template <typename... KArgs, typename... Args>
cudaError_t launch_k(bild_ctx* c, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = c->use_pdl ? 1 : 0;
  (*c->cnt)++;
  return cudaLaunchKernelEx(&cfg, kern, args...);
}

int ilog2(int v) { int s = 0; while ((1 << s) < v) ++s; return s; }

// Warps per row group: one 256-column chunk per warp where K allows it (K <= 4096).
int gemv_ksplit(int K) {
  for (int w = std::max(1, (K + 255) / 256); w <= 16; ++w)
    if (K % (8 * w) == 0) return w;
  for (int w = 16; w >= 1; --w)
    if (K % (8 * w) == 0) return w;
  return 1;
}

template <typename WT>
cudaError_t launch_gemv_t(bild_ctx* c, const LinArgs& a0) {
  LinArgs a = a0;
  a.ksplit = gemv_ksplit(a.K);
  a.dkv_shift = ilog2(std::max(1, a.dkv));
  const int groups = std::max(1, 4 / a.ksplit);
  a.groups = groups; a.kl = a.K / a.ksplit; a.inv_k = 1.f / (float)a.K;
  dim3 grid((a.N + 2 * groups - 1) / (2 * groups)), block(32 * a.ksplit * groups);
  if (a.epi == EPI_GATED) return launch_k(c, gemv_kernel<WT, true>, grid, block, 0, a);
  return launch_k(c, gemv_kernel<WT, false>, grid, block, 0, a);
}

template <int MB, bool STAGE>
cudaError_t launch_battn_t(bild_ctx* c, BAttnArgs a, int row_blocks, int keys_cap) {
  a.smem_keys = ((keys_cap + a.nsplit - 1) / a.nsplit + 3) / 4 * 4;
  size_t smem = (size_t)MB * a.smem_keys * sizeof(float);
  if (STAGE) smem += (size_t)a.smem_keys * (2 * a.dkv + 4) * sizeof(float);
  if (smem > 16 * 1024) {  // the kernel's static shared memory takes about 17 KB of the default 48 KB
    cudaError_t e = cudaFuncSetAttribute(battn_kernel<MB, STAGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  return launch_k(c, battn_kernel<MB, STAGE>, dim3(a.H, a.nsplit, row_blocks), dim3(BATT_THREADS), smem, a);
}
// Decoder attention stages its keys / values in shared memory (at most 128 keys per split);
// the encoder's self-attention (mode 2, all keys in one block) reads them from global memory.
cudaError_t launch_battn(bild_ctx* c, int MB, const BAttnArgs& a0, int row_blocks, int keys_cap, __nv_bfloat16* oh = nullptr,
                         __nv_bfloat16* ol = nullptr) {
  if (c->unit_attn && a0.mode != 2 && a0.dkv <= 64 && a0.dkv >= 16) {   // 256-thread kernel with bulk-copied key / value chunks
    DAttnArgs d;
    d.b = a0; d.MB = MB; d.dkv_shift = ilog2(a0.dkv);
    const int bias_len = a0.mode != 0 ? (((keys_cap + a0.nsplit - 1) / a0.nsplit + MAXB + 15) / 16 * 16) : 0;
    const size_t smem = uattn_smem_floats(MB, a0.dkv, a0.nsplit, bias_len) * sizeof(float);
    if (smem <= 200 * 1024) {
      if (smem > 48 * 1024 && !c->uattn_smem_set) {
        cudaError_t e = cudaFuncSetAttribute(uattn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(uattn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        c->uattn_smem_set = true;
      }
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(a0.H, a0.nsplit, row_blocks); cfg.blockDim = dim3(MB == 1 ? UA_THREADS : UA_THREADS_MAX); cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
      cudaLaunchAttribute at[2];
      int na = 0;
      if (c->use_pdl) {
        at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
      }
      if (a0.nsplit > 1) {   // the splits of one head are one cluster
        at[na].id = cudaLaunchAttributeClusterDimension;
        at[na].val.clusterDim.x = 1; at[na].val.clusterDim.y = a0.nsplit; at[na].val.clusterDim.z = 1;
        ++na;
      }
      cfg.attrs = at; cfg.numAttrs = na;
      (*c->cnt)++;
      return MB == 1 ? cudaLaunchKernelEx(&cfg, uattn_kernel<true>, d, bias_len) : cudaLaunchKernelEx(&cfg, uattn_kernel<false>, d, bias_len);
    }
  }
  if (a0.mode == 2 && a0.dkv == EA_D && c->enc_attn_mma) {   // encoder: 64-row tiles on mma.sync
    const int groups = std::min(enc_attn_groups(keys_cap), std::max(1, c->enc_attn_groups));
    const size_t smem = enc_attn_smem_bytes(keys_cap, groups);
    auto kern = groups == 1 ? enc_attn_kernel<1> : groups == 2 ? enc_attn_kernel<2> : enc_attn_kernel<3>;
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    return launch_k(c, kern, dim3(a0.H, (a0.M + EA_ROWS - 1) / EA_ROWS), dim3(EA_THREADS * groups), smem, a0, oh, ol);
  }
  if (a0.mode == 2) return launch_battn_t<MAXB, false>(c, a0, row_blocks, keys_cap);
  BAttnArgs a = a0;
  a.smem_keys = ((keys_cap + a.nsplit - 1) / a.nsplit + 3) / 4 * 4;
  const size_t smem = sizeof(float) * ((size_t)MB * a.dkv + (size_t)MB * a.smem_keys + (size_t)a.smem_keys * (2 * a.dkv + 4) +
                                       (size_t)a.nsplit * (MB == 1 ? 4 : 1) * MB * (a.dkv + 2));
  const int threads = MB == 1 ? 32 : 256;
  if (smem > 40 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(dattn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
  }
  DAttnArgs d;
  d.b = a; d.MB = MB; d.dkv_shift = ilog2(a.dkv);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.H, a.nsplit); cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (c->use_pdl) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (a.nsplit > 1) {   // the splits of one head are one cluster
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = 1; at[na].val.clusterDim.y = a.nsplit; at[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = at; cfg.numAttrs = na;
  (*c->cnt)++;
  return cudaLaunchKernelEx(&cfg, dattn_kernel, d);
}

template <typename WT, int MB, int RW>
cudaError_t launch_linear_t(bild_ctx* c, const LinArgs& a, int rows_y) {
  const int nwarps = LIN_THREADS / 32;
  dim3 grid((a.N + nwarps * RW - 1) / (nwarps * RW), rows_y);
  const int kc = (MB == 1) ? a.K : std::min(a.K, LIN_KC);
  const size_t smem = (size_t)MB * kc * sizeof(float);
  const bool gated = a.epi == EPI_GATED;
  auto kern = gated ? linear_kernel<WT, MB, RW, true> : linear_kernel<WT, MB, RW, false>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  if (gated) return launch_k(c, linear_kernel<WT, MB, RW, true>, grid, dim3(LIN_THREADS), smem, a);
  return launch_k(c, linear_kernel<WT, MB, RW, false>, grid, dim3(LIN_THREADS), smem, a);
}

// Block GEMV (SIMT) for up to MAXB token rows: one block per RW weight rows, warps split K.
template <typename WT, int PC>
cudaError_t launch_gemvk_pc(bild_ctx* c, const LinArgs& a0, int ks) {
  LinArgs a = a0;
  a.dkv_shift = ilog2(std::max(1, a.dkv));
  dim3 grid((a.N + 1) / 2), block(32 * ks);
  if (a.epi == EPI_GATED) return launch_k(c, gemvk_kernel<WT, 2, PC, true>, grid, block, 0, a);
  return launch_k(c, gemvk_kernel<WT, 2, PC, false>, grid, block, 0, a);
}
// false if K cannot be split into at most 16 warps of at most 4 chunks with 8-column alignment
template <typename WT>
bool launch_gemvk_t(bild_ctx* c, const LinArgs& a, cudaError_t* err) {
  int ks = 0;
  for (int w = std::max(1, (a.K + 255) / 256); w <= 16; ++w)
    if (a.K % (8 * w) == 0) { ks = w; break; }
  if (!ks)
    for (int w = 16; w >= 1; --w)
      if (a.K % (8 * w) == 0) { ks = w; break; }
  const int pc = (a.K / ks + 255) / 256;
  if (pc > 4) return false;
  *err = pc == 1 ? launch_gemvk_pc<WT, 1>(c, a, ks) : pc == 2 ? launch_gemvk_pc<WT, 2>(c, a, ks) : launch_gemvk_pc<WT, 4>(c, a, ks);
  return true;
}

// MB == 1: the GEMV of the small-model step (and of the large model at k = 1);
// otherwise the small-M GEMM over up to MAXB rows per row block.
cudaError_t launch_linear(bild_ctx* c, int dtype, int MB, const LinArgs& a, int rows_y = 1) {
  if (dtype == BILD_BF16)
    return MB == 1 ? launch_gemv_t<__nv_bfloat16>(c, a) : launch_linear_t<__nv_bfloat16, MAXB, 2>(c, a, rows_y);
  return MB == 1 ? launch_gemv_t<float>(c, a) : launch_linear_t<float, MAXB, 2>(c, a, rows_y);
}

template <typename WT, int MB, int RW>
cudaError_t launch_head_t(bild_ctx* c, const HeadArgs& a, int grid, int64_t* launches) {
  const size_t smem = (size_t)MB * a.K * sizeof(float);
  auto kern = lm_head_kernel<WT, MB, RW>;
  if (smem > 48 * 1024) {
    cudaFuncAttributes fa;
    int dev = 0, optin = 0;
    cudaError_t e = cudaFuncGetAttributes(&fa, kern);
    if (e == cudaSuccess) e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return e;
    if (smem + fa.sharedSizeBytes > (size_t)optin) return cudaErrorInvalidConfiguration;   // the staged rows do not fit a block
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  if (launches) (*launches)++;
  return launch_k(c, kern, dim3(grid), dim3(HEAD_THREADS), smem, a);
}

template <typename WT, int NCH, int RPW>
cudaError_t launch_head1_t(bild_ctx* c, const HeadArgs& a, int64_t* launches) {
  const int rows = (HEAD1_THREADS / 32) * RPW;
  if (launches) (*launches)++;
  return launch_k(c, head1_kernel<WT, NCH, RPW>, dim3((a.V + rows - 1) / rows), dim3(HEAD1_THREADS), 0, a);
}
// blocks of the single-row head for a vocabulary of V rows and K columns (0: shape not covered)
int head1_grid(int V, int K) {
  const int nch = (K + 255) / 256;
  const int rpw = nch <= 2 ? 4 : nch <= 4 ? 2 : nch <= 8 ? 1 : 0;
  return rpw ? (V + 8 * rpw - 1) / (8 * rpw) : 0;
}
template <typename WT>
cudaError_t launch_head1(bild_ctx* c, const HeadArgs& a, int64_t* launches) {
  const int nch = (a.K + 255) / 256;
  if (nch <= 1) return launch_head1_t<WT, 1, 4>(c, a, launches);
  if (nch <= 2) return launch_head1_t<WT, 2, 4>(c, a, launches);
  if (nch <= 4) return launch_head1_t<WT, 4, 2>(c, a, launches);
  return launch_head1_t<WT, 8, 1>(c, a, launches);
}

// Single row, bf16 weights, rows of at most 1024 columns: the streaming head (two blocks per SM walk the vocabulary).
bool head_stream_fits(int dtype, int MB, const HeadArgs& a) {
  return MB == 1 && dtype == BILD_BF16 && a.K % 8 == 0 && a.K <= 1024 && ((uintptr_t)a.W & 15) == 0;
}
cudaError_t launch_head_stream(bild_ctx* c, const HeadArgs& a, int sms) {
  const int r = a.K <= 512 ? 8 : 4;
  const dim3 grid(std::max(1, std::min(2 * sms, (a.V + 8 * r - 1) / (8 * r)))), block(HEAD1_THREADS);
  if (a.K <= 256) return launch_k(c, head_stream_kernel<1, 8>, grid, block, 0, a);
  if (a.K <= 512) return launch_k(c, head_stream_kernel<2, 8>, grid, block, 0, a);
  return launch_k(c, head_stream_kernel<4, 4>, grid, block, 0, a);
}

cudaError_t launch_head(cudaStream_t s, bool pdl, int dtype, int MB, const HeadArgs& a, int grid, int64_t* launches) {
  bild_ctx tmp;
  tmp.stream = s;
  tmp.use_pdl = pdl;
  if (MB == 1 && head1_grid(a.V, a.K) > 0)
    return dtype == BILD_BF16 ? launch_head1<__nv_bfloat16>(&tmp, a, launches) : launch_head1<float>(&tmp, a, launches);
  if (dtype == BILD_BF16)
    return MB == 1 ? launch_head_t<__nv_bfloat16, 1, 4>(&tmp, a, grid, launches) : launch_head_t<__nv_bfloat16, MAXB, 2>(&tmp, a, grid, launches);
  return MB == 1 ? launch_head_t<float, 1, 4>(&tmp, a, grid, launches) : launch_head_t<float, MAXB, 2>(&tmp, a, grid, launches);
}

// Key splits per head for decoder attention: the splits of a head form one cluster (<= 8 blocks),
// each staging at most 256 keys; more splits until about one block per SM.
int pick_nsplit(int heads, int keys_cap) {
  int ns = 1;
  while (ns < 8 && (heads * ns < 148 / 2 || (keys_cap + ns - 1) / ns > 256) && keys_cap / (ns * 2) >= 16) ns *= 2;
  return ns;
}

cudaError_t launch_embed(bild_ctx* c, const void* E, const int* tokens, const int* cnt_dev, int cnt_host, int rows,
                         int d, int vocab, float* x, float* x_zero = nullptr) {
  if (c->cfg.dtype == BILD_BF16)
    return launch_k(c, embed_kernel<__nv_bfloat16>, dim3(rows), dim3(128), 0, (const __nv_bfloat16*)E, tokens, cnt_dev,
                    cnt_host, d, vocab, x, x_zero);
  return launch_k(c, embed_kernel<float>, dim3(rows), dim3(128), 0, (const float*)E, tokens, cnt_dev, cnt_host, d,
                  vocab, x, x_zero);
}

// ---- tensor-core path of the block pass ---------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Descriptor of a row-major bf16 matrix [N][K] for boxes of 128 rows x 64 columns, 128-byte swizzle.
bool make_tmap(EncodeTiledFn enc, const void* W, int N, int K, CUtensorMap* out) {
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {UM_KB, UM_TILE_M};
  cuuint32_t es[2] = {1, 1};
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(W), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

enum { TM_QKV = 0, TM_O, TM_CQ, TM_CO, TM_WI0, TM_WI1, TM_FO, TM_CKV, TM_EQKV, TM_EO, TM_EWI0, TM_EWI1, TM_EFO, TM_PER_LAYER };

// Builds the descriptors of one model; leaves m.umma false when the shapes do not fit the kernel.
void setup_umma(bild_ctx* c, Model& m) {
  m.umma = false;
  if (!c->use_umma) return;
  if (c->cfg.dtype != BILD_BF16) return;
  const bild_model_cfg& mc = m.c;
  if (mc.d_model % UM_KB || m.inner % UM_KB || mc.d_ff % UM_KB) return;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) {
    cudaGetLastError();
    return;
  }
  EncodeTiledFn enc = (EncodeTiledFn)fn;
  const bool gated = mc.ffn_kind == BILD_FFN_GATED_GELU;
  m.tmaps.resize((size_t)mc.n_layers * TM_PER_LAYER);
  for (int l = 0; l < mc.n_layers; ++l) {
    const bild_dec_layer& w = m.dec[l];
    CUtensorMap* t = &m.tmaps[(size_t)l * TM_PER_LAYER];
    bool ok = make_tmap(enc, w.wqkv, 3 * m.inner, mc.d_model, &t[TM_QKV]) &&
              make_tmap(enc, w.wo, mc.d_model, m.inner, &t[TM_O]) &&
              make_tmap(enc, w.wcq, m.inner, mc.d_model, &t[TM_CQ]) &&
              make_tmap(enc, w.wco, mc.d_model, m.inner, &t[TM_CO]) &&
              make_tmap(enc, w.wi0, mc.d_ff, mc.d_model, &t[TM_WI0]) &&
              make_tmap(enc, gated ? w.wi1 : w.wi0, mc.d_ff, mc.d_model, &t[TM_WI1]) &&
              make_tmap(enc, w.wfo, mc.d_model, mc.d_ff, &t[TM_FO]) &&
              make_tmap(enc, w.wckv, 2 * m.inner, mc.d_model, &t[TM_CKV]);
    const bild_enc_layer& e = m.enc[l];
    ok = ok && make_tmap(enc, e.wqkv, 3 * m.inner, mc.d_model, &t[TM_EQKV]) &&
         make_tmap(enc, e.wo, mc.d_model, m.inner, &t[TM_EO]) &&
         make_tmap(enc, e.wi0, mc.d_ff, mc.d_model, &t[TM_EWI0]) &&
         make_tmap(enc, gated ? e.wi1 : e.wi0, mc.d_ff, mc.d_model, &t[TM_EWI1]) &&
         make_tmap(enc, e.wfo, mc.d_model, mc.d_ff, &t[TM_EFO]);
    if (!ok) { m.tmaps.clear(); return; }
  }
  const int maxsm = 227 * 1024;
  if (cudaFuncSetAttribute(umma_linear_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, maxsm) != cudaSuccess ||
      cudaFuncSetAttribute(umma_linear_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, maxsm) != cudaSuccess) {
    cudaGetLastError();
    m.tmaps.clear();
    return;
  }
  m.umma = true;
  // encoder GEMM over 128-token tiles
  m.enc_gemm = false;
  if (!c->use_enc_gemm) return;
  const int ecap128 = (c->cfg.max_enc_len + EG_TOK - 1) / EG_TOK * EG_TOK;
  const int Ks[3] = {mc.d_model, m.inner, mc.d_ff};
  for (int pr = 0; pr < 2; ++pr)
    for (int i = 0; i < 3; ++i)
      if (!make_tmap(enc, c->eb[m.index].exh[pr], ecap128, Ks[i], &m.tmH[pr][i][0]) ||
          !make_tmap(enc, c->eb[m.index].exl[pr], ecap128, Ks[i], &m.tmH[pr][i][1])) return;
  if (cudaFuncSetAttribute(enc_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)eg_smem_bytes<false>()) != cudaSuccess ||
      cudaFuncSetAttribute(enc_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)eg_smem_bytes<true>()) != cudaSuccess) {
    cudaGetLastError();
    return;
  }
  m.enc_gemm = true;
}

// ---- fused sub-layer kernels ------------------------------------------------------------------
// Decides whether the decoder passes of model `m` run on the fused sub-layer kernels, transposes the
// FFN output matrices into the workspace and fixes the launch shapes.
int setup_fused(bild_ctx* c, Model& m) {
  m.fused = false;
  if (!c->fused_on || c->cfg.dtype != BILD_BF16 || c->sms < 1) return BILD_OK;
  const bild_model_cfg& mc = m.c;
  const int d = mc.d_model, I = m.inner, F = mc.d_ff, H = mc.n_heads, dkv = mc.d_kv;
  const int cap = c->cfg.max_dec_len, ecap = c->cfg.max_enc_len;
  const bool gated = mc.ffn_kind == BILD_FFN_GATED_GELU;
  int C = 8;
  while (C > 1 && (H * C > c->sms || d % (4 * C))) C >>= 1;
  if (d % (4 * C) || d % 16 || F % 8 || d > 1024 || dkv > 64 || dkv < 16 || d / C > SUB_THREADS / 2) return BILD_OK;
  if ((3 * dkv + C - 1) / C > SUB_MAX_ROWS) return BILD_OK;
  auto aligned = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
  for (int l = 0; l < mc.n_layers; ++l) {
    const bild_dec_layer& w = m.dec[l];
    if (!aligned(w.wqkv) || !aligned(w.wo) || !aligned(w.wcq) || !aligned(w.wco) || !aligned(w.wi0) || !aligned(w.wfo) ||
        (gated && !aligned(w.wi1)) || !aligned(w.ln1) || !aligned(w.ln2) || !aligned(w.ln3)) return BILD_OK;
  }
  if (!aligned(m.w.emb)) return BILD_OK;   // (the first sub-layer kernel gathers the embedding rows, 8 bytes per load)
  int smem_max = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
    cudaGetLastError();
    return BILD_OK;
  }
  const int all_keys = c->attn_all_keys;
  AttnSubPlan ps[2], pc[2];
  for (int v = 0; v < 2; ++v) {
    ps[v] = attn_sub_plan(d, dkv, 3, C, cap, all_keys, SUB_HALF_SM, smem_max, v ? SUB_MB : 1);
    pc[v] = attn_sub_plan(d, dkv, 1, C, ecap, all_keys, SUB_HALF_SM, smem_max, v ? SUB_MB : 1);
    if (!ps[v].ok || !pc[v].ok) return BILD_OK;
  }
  int parts = std::max(1, c->sub_parts_want);
  const int nmat = gated ? 2 : 1;
  while (parts <= 8 && (ffn_sub_rows(F, c->sms * parts) * nmat > SUB_MAX_ROWS || ffn_sub_rows(F, c->sms * parts) > SUB_FO_REGS ||
                        ffn_sub_layout(d, F, gated, c->sms * parts, c->sms, SUB_MB).total > smem_max)) ++parts;
  if (parts > 8) return BILD_OK;
  if (cudaFuncSetAttribute(attn_sub_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess ||
      cudaFuncSetAttribute(attn_sub_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess ||
      cudaFuncSetAttribute(ffn_sub_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess ||
      cudaFuncSetAttribute(ffn_sub_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess) {
    cudaGetLastError();
    return BILD_OK;
  }
  for (int l = 0; l < mc.n_layers; ++l) {
    pack_wfo_kernel<<<F / 8, 256, 0, c->stream>>>((const __nv_bfloat16*)m.dec[l].wfo, m.wfo_one + (size_t)l * (F / 8) * d,
                                                  m.wfo_blk + (size_t)l * (F / 8) * pack_wfo_dpad(d), d, F);
    (*c->cnt)++;
  }
  CUDA_TRY(c, cudaGetLastError());
  m.sub_C = C; m.sub_parts = parts;
  for (int v = 0; v < 2; ++v) { m.sub_self[v] = ps[v]; m.sub_cross[v] = pc[v]; }
  m.fused = true;
  return BILD_OK;
}

template <typename Arg>
cudaError_t launch_sub(bild_ctx* c, void (*kern)(Arg), int grid, int cluster, size_t smem, const Arg& a, bool pdl_ok = true) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(SUB_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (c->use_pdl && pdl_ok) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (cluster > 1) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = cluster; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = at; cfg.numAttrs = na;
  (*c->cnt)++;
  return cudaLaunchKernelEx(&cfg, kern, a);
}

// One layer of a decoder pass on the fused sub-layer kernels: the residual stream goes x -> xb -> xc -> x (self-attention,
// cross-attention, feed-forward), each kernel clearing the buffer after its output.  desc / row0: the rows the kernels
// work on (a whole pass, or one chunk of a block of 9 to 16 rows); first_plain: the layer's first kernel follows a
// dependency on another stream and is launched without the programmatic-launch attribute; after_self: called once the
// self-attention kernel is in the stream (its keys and values are what the next chunk's same layer waits for).
template <typename F>
int fused_layer(bild_ctx* c, Model& m, int MB, int l, const CallDesc* desc, int row0, bool first_plain, F after_self) {
  const bild_model_cfg& mc = m.c;
  const int d = mc.d_model, I = m.inner, Fd = mc.d_ff, H = mc.n_heads, dkv = mc.d_kv;
  const int cap = c->cfg.max_dec_len, ecap = c->cfg.max_enc_len;
  const bool gated = mc.ffn_kind == BILD_FFN_GATED_GELU;
  const int C = m.sub_C;
  float* x = m.x + (size_t)row0 * d;
  float* xb = m.xb + (size_t)row0 * d;
  float* xc = m.xc + (size_t)row0 * d;
  const bild_dec_layer& w = m.dec[l];
  const size_t kvoff = (size_t)l * H * dkv;
  AttnSubArgs a{};
  a.desc = desc; a.eps = mc.ln_eps; a.d = d; a.I = I; a.H = H; a.dkv = dkv; a.dkv_shift = ilog2(dkv); a.C = C; a.c_shift = ilog2(C);
  a.mb = MB; a.err = &c->st->err;
  a.spin = c->spin_limit; a.skip_copies = c->debug_skip_copies ? 1 : 0;
  a.n_keys_dev = c->enc_len_dev;
  // S1-S3 / L1-L3 (layer 0: with S0 / L0, the rows come from the embedding table)
  if (l == 0 && c->fused_embed) {
    a.emb = (const __nv_bfloat16*)m.w.emb; a.tokens = m.desc->tokens + row0; a.vocab = mc.vocab;
  }
  a.x_in = x; a.x_out = xb; a.x_zero = xc; a.gain = (const float*)w.ln1;
  a.Wp = (const __nv_bfloat16*)w.wqkv; a.Wo = (const __nv_bfloat16*)w.wo;
  a.kc = m.selfK + kvoff * cap; a.vc = m.selfV + kvoff * cap; a.cap = cap; a.bias = m.dec_bias; a.bias_ld = cap; a.self = 1;
  const AttnSubPlan& pls = m.sub_self[MB == 1 ? 0 : 1];
  a.kc_keys = pls.kc; a.bias_len = pls.bias_len; a.red_keys = pls.red_keys;
  a.L = attn_sub_layout(d, dkv, 3, C, MB, a.kc_keys, a.bias_len);
  CUDA_TRY(c, launch_sub(c, MB == 1 ? attn_sub_kernel<true> : attn_sub_kernel<false>, H * C, C, (size_t)a.L.total, a, !first_plain));
  int rc = after_self();
  if (rc) return rc;
  // S4-S6 / L4-L6
  a.emb = nullptr;
  a.x_in = xb; a.x_out = xc; a.x_zero = x; a.gain = (const float*)w.ln2;
  a.Wp = (const __nv_bfloat16*)w.wcq; a.Wo = (const __nv_bfloat16*)w.wco;
  a.kc = m.crossK + kvoff * ecap; a.vc = m.crossV + kvoff * ecap; a.cap = ecap; a.bias = nullptr; a.bias_ld = 0; a.self = 0;
  const AttnSubPlan& plc = m.sub_cross[MB == 1 ? 0 : 1];
  a.kc_keys = plc.kc; a.bias_len = plc.bias_len; a.red_keys = plc.red_keys;
  a.L = attn_sub_layout(d, dkv, 1, C, MB, a.kc_keys, a.bias_len);
  CUDA_TRY(c, launch_sub(c, MB == 1 ? attn_sub_kernel<true> : attn_sub_kernel<false>, H * C, C, (size_t)a.L.total, a));
  // S7-S8 / L7-L8
  FfnSubArgs f{};
  f.desc = desc; f.eps = mc.ln_eps; f.d = d; f.F = Fd; f.gated = gated ? 1 : 0; f.mb = MB; f.spin = c->spin_limit;
  f.err = &c->st->err; f.x_in = xc; f.x_out = x; f.gain = (const float*)w.ln3;
  f.Wi0 = (const __nv_bfloat16*)w.wi0; f.Wi1 = (const __nv_bfloat16*)w.wi1;
  f.Wfo1 = m.wfo_one + (size_t)l * (Fd / 8) * d; f.Wfo8 = m.wfo_blk + (size_t)l * (Fd / 8) * pack_wfo_dpad(d);
  f.nparts = m.sub_parts;
  f.L = ffn_sub_layout(d, Fd, gated, c->sms * m.sub_parts, c->sms, MB);
  for (int p = 0; p < m.sub_parts; ++p) {
    f.part = p; f.seed = p == 0 ? 1 : 0; f.x_zero = p == 0 ? xb : nullptr;
    CUDA_TRY(c, launch_sub(c, MB == 1 ? ffn_sub_kernel<true> : ffn_sub_kernel<false>, c->sms, 1, (size_t)f.L.total, f));
  }
  return BILD_OK;
}

int fused_layers(bild_ctx* c, Model& m, int MB) {
  for (int l = 0; l < m.c.n_layers; ++l) {
    int rc = fused_layer(c, m, MB, l, m.desc, 0, false, [] { return (int)BILD_OK; });
    if (rc) return rc;
  }
  return BILD_OK;
}

// A block of 9 to 16 rows on the fused sub-layer kernels: two chunks (rows 0..7, then the rest) on two streams, layer l of
// the second chunk waiting only for the self-attention kernel of layer l of the first (whose keys and values it attends
// over), so that the two chunks run side by side, one layer apart.  On return the context's stream has both behind it.
int fused_layers_two_chunks(bild_ctx* c, Model& m) {
  const int L = m.c.n_layers;
  if (!c->side2) CUDA_TRY(c, cudaStreamCreateWithFlags(&c->side2, cudaStreamNonBlocking));
  while ((int)c->chunk_ev.size() < L + 2) {
    cudaEvent_t e;
    CUDA_TRY(c, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    c->chunk_ev.push_back(e);
  }
  cudaStream_t s0 = c->stream, s1 = c->side2;
  split_desc_kernel<<<1, 1, 0, s0>>>(m.desc, m.desc_lo, m.desc_hi);
  (*c->cnt)++;
  CUDA_TRY(c, cudaGetLastError());
  CUDA_TRY(c, cudaEventRecord(c->chunk_ev[L], s0));
  CUDA_TRY(c, cudaStreamWaitEvent(s1, c->chunk_ev[L], 0));
  int rc = BILD_OK;
  for (int l = 0; l < L && rc == BILD_OK; ++l) {
    rc = fused_layer(c, m, SUB_MB, l, m.desc_lo, 0, l == 0, [&] {
      CUDA_TRY(c, cudaEventRecord(c->chunk_ev[l], s0));
      return (int)BILD_OK;
    });
    if (rc) break;
    CUDA_TRY(c, cudaStreamWaitEvent(s1, c->chunk_ev[l], 0));
    c->stream = s1;
    rc = fused_layer(c, m, SUB_MB, l, m.desc_hi, SUB_CHUNK, true, [] { return (int)BILD_OK; });
    c->stream = s0;
  }
  if (rc) return rc;
  CUDA_TRY(c, cudaEventRecord(c->chunk_ev[L + 1], s1));
  CUDA_TRY(c, cudaStreamWaitEvent(s0, c->chunk_ev[L + 1], 0));
  return BILD_OK;
}

// Split of K over a cluster: enough blocks to pull the matrix at full bandwidth, at most 16 k blocks each.
bool umma_plan(int N, int K, bool gated, int* cs_out, int* nkb_out, bool many_row_blocks = false) {
  const int tiles = (N + UM_TILE_M - 1) / UM_TILE_M;
  int best = 0;
  if (many_row_blocks) {   // encoder: row blocks already give enough CTAs; the smallest split of K that fits
    for (int cs = 1; cs <= (gated ? 4 : 8); cs *= 2) {
      if (K % (UM_KB * cs)) break;
      const int nkb = K / UM_KB / cs;
      if (nkb <= 16 && umma_smem_bytes(gated, nkb, cs) <= 227 * 1024) { *cs_out = cs; *nkb_out = nkb; return true; }
    }
    return false;
  }
  for (int cs = 1; cs <= (gated ? 4 : 8); cs *= 2) {
    if (K % (UM_KB * cs)) break;
    const int nkb = K / UM_KB / cs;
    if (nkb > 16 || umma_smem_bytes(gated, nkb, cs) > 227 * 1024) continue;
    best = cs;
    if (tiles * cs >= 96) break;
  }
  if (!best) return false;
  *cs_out = best;
  *nkb_out = K / UM_KB / best;
  return true;
}

cudaError_t launch_umma(bild_ctx* c, const LinArgs& a, const CUtensorMap& t0, const CUtensorMap& t1, int cs, int nkb,
                        int row_blocks = 1) {
  const bool gated = a.epi == EPI_GATED;
  UmmaArgs u;
  u.lin = a; u.cs = cs; u.nkb = nkb; u.err = &c->st->err;
  const int tiles = (a.N + UM_TILE_M - 1) / UM_TILE_M;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles * cs, row_blocks); cfg.blockDim = dim3(UM_THREADS);
  cfg.dynamicSmemBytes = umma_smem_bytes(gated, nkb, cs); cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (c->use_pdl) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (cs > 1) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = cs; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = at; cfg.numAttrs = na;
  (*c->cnt)++;
  if (gated) return cudaLaunchKernelEx(&cfg, umma_linear_kernel<true>, u, t0, t1);
  return cudaLaunchKernelEx(&cfg, umma_linear_kernel<false>, u, t0, t1);
}

// Row-slice kernel (one block per SM, weights fetched ahead of the dependency wait); false if the shape does not fit.
bool launch_slice(bild_ctx* c, int MB, const LinArgs& a0, cudaError_t* err) {
  if (c->cfg.dtype != BILD_BF16 || c->sms < 1 || !a0.desc) return false;
  const LinArgs& a = a0;
  const int nmat = a.epi == EPI_GATED ? 2 : 1;
  const int rows = (a.N + c->sms - 1) / c->sms;
  if (a.K % 8 || a.ldx != a.K || rows * nmat > 4 * SL_QUADS || (a.gain && a.K > 2048)) return false;
  if (((uintptr_t)a.W0 & 15) || (nmat == 2 && ((uintptr_t)a.W1 & 15)) || ((uintptr_t)a.X & 15) || (a.gain && ((uintptr_t)a.gain & 15))) return false;
  SliceArgs s;
  s.lin = a;
  s.lin.dkv_shift = ilog2(std::max(1, a.dkv));
  s.err = &c->st->err;
  s.w_bytes = (int)slice_w_bytes(rows * nmat, a.K);
  int xr = MB == 1 ? 1 : MAXB;   // token rows staged at once: at most 81 KB (5 rows of 4096 columns)
  while (xr > 1 && (size_t)xr * (a.K + SL_XPAD) * 4 > 81 * 1024) --xr;
  s.x_rows = xr;
  s.mma_min = c->slice_mma_min;
  const size_t smem = slice_smem_bytes(s.w_bytes, xr, a.K);
  if (smem > 200 * 1024) return false;
  if (smem > 48 * 1024 && smem > c->slice_smem_set) {
    if (cudaFuncSetAttribute(slice_linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    c->slice_smem_set = 200 * 1024;
  }
  *err = launch_k(c, slice_linear_kernel, dim3(c->sms), dim3(SL_THREADS), smem, s);
  return true;
}

// Linear layer of a decoder pass: tensor cores for the bf16 block pass, SIMT otherwise.
cudaError_t launch_dec_linear(bild_ctx* c, Model& m, int MB, const LinArgs& a, int layer, int which_map) {
  int cs, nkb;
  // single-row passes: only matrices large enough that a block's slice is worth a bulk copy
  const bool big = (size_t)a.N * a.K * 2 >= c->slice_min_bytes;
  if (c->slice_mode >= (MB == 1 ? 2 : 1) && (MB != 1 || big) && !c->block_simt) {
    cudaError_t e = cudaSuccess;
    if (launch_slice(c, MB, a, &e)) return e;
  }
  if (MB != 1 && c->block_simt) {
    const int ks = gemv_ksplit(a.K);
    if (a.K / ks <= 256) {   // compact block GEMV: one chunk per warp
      LinArgs b = a;
      b.ksplit = ks; b.kl = a.K / ks; b.inv_k = 1.f / (float)a.K; b.groups = 1; b.dkv_shift = ilog2(std::max(1, a.dkv));
      dim3 grid((a.N + 1) / 2), block(32 * ks);
      const bool gated = a.epi == EPI_GATED;
      if (c->cfg.dtype == BILD_BF16)
        return gated ? launch_k(c, gemvb_kernel<__nv_bfloat16, true>, grid, block, 0, b) : launch_k(c, gemvb_kernel<__nv_bfloat16, false>, grid, block, 0, b);
      return gated ? launch_k(c, gemvb_kernel<float, true>, grid, block, 0, b) : launch_k(c, gemvb_kernel<float, false>, grid, block, 0, b);
    }
    cudaError_t e = cudaSuccess;
    if (c->cfg.dtype == BILD_BF16 ? launch_gemvk_t<__nv_bfloat16>(c, a, &e) : launch_gemvk_t<float>(c, a, &e)) return e;
  }
  if (MB != 1 && m.umma && umma_plan(a.N, a.K, a.epi == EPI_GATED, &cs, &nkb)) {
    const CUtensorMap* t = &m.tmaps[(size_t)layer * TM_PER_LAYER];
    return launch_umma(c, a, t[which_map], t[which_map == TM_WI0 ? TM_WI1 : which_map], cs, nkb);
  }
  return launch_linear(c, c->cfg.dtype, MB, a);
}

// Encoder linear layer on 128-token tiles: split the (normalised) input into bf16 head + remainder, then the GEMM.
// The input pair is buffer `pair`; `split` false: it already holds the input (written by the kernel in front or by
// an earlier call); `out_pair` >= 0: a ReLU / gated epilogue writes its output as the pair `out_pair` instead of fp32.
cudaError_t launch_enc_gemm(bild_ctx* c, Model& m, const LinArgs& a, int layer, int which_map, bool split, int pair, int out_pair) {
  const int E = a.M, tiles_tok = (E + EG_TOK - 1) / EG_TOK;
  const int ki = a.K == m.c.d_model ? 0 : a.K == m.inner ? 1 : 2;
  if (split) {
    cudaError_t e = launch_k(c, norm_split_kernel, dim3(tiles_tok * EG_TOK / 4), dim3(128), 0, a.X, a.ldx, a.gain, a.eps, E, a.K,
                             c->eb[m.index].exh[pair], c->eb[m.index].exl[pair]);
    if (e != cudaSuccess) return e;
  }
  const CUtensorMap* t = &m.tmaps[(size_t)layer * TM_PER_LAYER];
  const bool gated = a.epi == EPI_GATED;
  __nv_bfloat16* oh = out_pair >= 0 ? c->eb[m.index].exh[out_pair] : nullptr;
  __nv_bfloat16* ol = out_pair >= 0 ? c->eb[m.index].exl[out_pair] : nullptr;
  dim3 grid((a.N + UM_TILE_M - 1) / UM_TILE_M, tiles_tok);
  if (a.epi == EPI_RESID && c->enc_split_k) {   // few tiles, long K: split K until the grid covers the SMs (at least 4 K blocks each)
    const int tiles = (int)(grid.x * grid.y), nkb = a.K / UM_KB;
    int z = 1;
    while (z < 8 && tiles * (z * 2) <= c->sms && nkb / (z * 2) >= 4) z *= 2;
    grid.z = z;
  }
  if (gated)
    return launch_k(c, enc_gemm_kernel<true>, grid, dim3(EG_THREADS), eg_smem_bytes<true>(), a, &c->st->err, oh, ol, t[which_map],
                    t[which_map == TM_EWI0 ? TM_EWI1 : which_map], m.tmH[pair][ki][0], m.tmH[pair][ki][1]);
  return launch_k(c, enc_gemm_kernel<false>, grid, dim3(EG_THREADS), eg_smem_bytes<false>(), a, &c->st->err, oh, ol, t[which_map],
                  t[which_map], m.tmH[pair][ki][0], m.tmH[pair][ki][1]);
}

// Linear layer of the encoder over rb blocks of MAXB rows.
cudaError_t launch_enc_linear(bild_ctx* c, Model& m, const LinArgs& a, int rb, int layer, int which_map, bool split = true,
                              int pair = 0, int out_pair = -1) {
  int cs, nkb;
  if (m.enc_gemm && (a.K == m.c.d_model || a.K == m.inner || a.K == m.c.d_ff))
    return launch_enc_gemm(c, m, a, layer, which_map, split, pair, out_pair);
  if (m.umma && umma_plan(a.N, a.K, a.epi == EPI_GATED, &cs, &nkb, rb >= 4)) {
    const CUtensorMap* t = &m.tmaps[(size_t)layer * TM_PER_LAYER];
    return launch_umma(c, a, t[which_map], t[which_map == TM_EWI0 ? TM_EWI1 : which_map], cs, nkb, rb);
  }
  return launch_linear(c, c->cfg.dtype, MAXB, a, rb);
}

LoopPtrs loop_ptrs(bild_ctx* c) {
  LoopPtrs L;
  L.st = c->st; L.y = c->y; L.trace = c->trace; L.descS = c->m[0].desc; L.descL = c->m[1].desc;
  return L;
}

// One decoder pass of model `which` over the rows described by its CallDesc
// (steps S0..S10 / L0..L10: embed, per layer [norm+QKV+append, self-attention, O+residual,
// norm+cross-Q, cross-attention, cross-O+residual, norm+FFN-up, FFN-down+residual],
// final norm + LM head + policy).  MB = 1 or MAXB selects the kernel variants.
// MBv: rows the pass is built for: 1, SUB_MB (2 to 8 rows) or MAXB.
int decoder_pass(bild_ctx* c, int which, int MBv, float* logits_dbg, unsigned long long cond_while = 0,
                 unsigned long long cond_if = 0, unsigned long long cond_if1 = 0, unsigned long long cond_if8 = 0) {
  const int MB = MBv == 1 ? 1 : MAXB;   // variant of the kernels outside the fused sub-layers
  Model& m = c->m[which];
  const bild_model_cfg& mc = m.c;
  const int d = mc.d_model, I = m.inner, F = mc.d_ff, H = mc.n_heads, dkv = mc.d_kv;
  const int cap = c->cfg.max_dec_len, ecap = c->cfg.max_enc_len, dt = c->cfg.dtype;
  // blocks of 9 to 16 rows: two chunks of the 8-row kernels side by side (the caller guarantees more than 8 rows)
  const bool chunked = m.fused && which == 1 && MBv == MAXB && c->fused_on >= 3;
  const bool fused = chunked || (m.fused && (MBv == 1 || (MBv == SUB_MB && c->fused_on >= 2)));
  // (fused sub-layer kernels: the first one gathers the embedding rows itself; the buffer it adds into is clear, every
  // pass leaves it so and a generation starts with it cleared)
  if (!(fused && c->fused_embed))
    CUDA_TRY(c, launch_embed(c, m.w.emb, m.desc->tokens, &m.desc->k, 0, MB, d, mc.vocab, m.x, fused ? m.xb : nullptr));
  if (fused) {
    int rc = chunked ? fused_layers_two_chunks(c, m) : fused_layers(c, m, MBv);
    if (rc) return rc;
  }
  const bool pdl_was = c->use_pdl;
  if (chunked) c->use_pdl = false;   // the head follows the join of two streams: a plain launch
  struct PdlRestore { bild_ctx* c; bool v; ~PdlRestore() { c->use_pdl = v; } } pdl_restore{c, pdl_was};
  // self-attention: one block per head up to 128 cached rows (no merge step); cross-attention:
  // enough splits of the encoder keys to occupy the SMs
  int ns_self = 1;
  while (ns_self < 8 && (cap + ns_self - 1) / ns_self > 256) ns_self *= 2;
  const int ns_cross = pick_nsplit(H, ecap);
  for (int l = 0; l < (fused ? 0 : mc.n_layers); ++l) {
    const bild_dec_layer& w = m.dec[l];
    const size_t kvoff = (size_t)l * H * dkv;
    LinArgs a{};
    a.desc = m.desc; a.eps = mc.ln_eps;
    // S1 / L1: norm + QKV, K/V appended to the cache
    a.W0 = w.wqkv; a.X = m.x; a.ldx = d; a.gain = (const float*)w.ln1; a.N = 3 * I; a.K = d;
    a.epi = EPI_HEADS; a.inner = I; a.dkv = dkv; a.first_part = 0; a.q_out = m.q; a.ldq = I;
    a.kc = m.selfK + kvoff * cap; a.vc = m.selfV + kvoff * cap; a.cap = cap;
    CUDA_TRY(c, launch_dec_linear(c, m, MB, a, l, TM_QKV));
    // S2 / L2: self-attention over the cache (causal inside the block)
    BAttnArgs t{};
    t.q = m.q; t.ldq = I; t.kc = a.kc; t.vc = a.vc; t.cap = cap; t.out = m.att; t.ldo = I;
    t.bias = m.dec_bias; t.bias_ld = cap; t.bias_off = 0; t.mode = 1; t.dkv = dkv; t.H = H;
    t.n_keys_dev = c->enc_len_dev; t.desc = m.desc; t.part = m.att_part; t.counters = m.att_cnt;
    t.nsplit = ns_self; t.err = &c->st->err;
    CUDA_TRY(c, launch_battn(c, MB, t, 1, cap));
    // S3 / L3: output projection + residual
    LinArgs o{};
    o.desc = m.desc; o.W0 = w.wo; o.X = m.att; o.ldx = I; o.N = d; o.K = I; o.epi = EPI_RESID; o.Y = m.x; o.ldy = d;
    CUDA_TRY(c, launch_dec_linear(c, m, MB, o, l, TM_O));
    // S4 / L4: norm + cross-attention query
    LinArgs cq{};
    cq.desc = m.desc; cq.eps = mc.ln_eps; cq.W0 = w.wcq; cq.X = m.x; cq.ldx = d; cq.gain = (const float*)w.ln2;
    cq.N = I; cq.K = d; cq.epi = EPI_STORE; cq.Y = m.q; cq.ldy = I;
    CUDA_TRY(c, launch_dec_linear(c, m, MB, cq, l, TM_CQ));
    // S5 / L5: cross-attention over the encoder K/V
    BAttnArgs x{};
    x.q = m.q; x.ldq = I; x.kc = m.crossK + kvoff * ecap; x.vc = m.crossV + kvoff * ecap; x.cap = ecap;
    x.out = m.att; x.ldo = I; x.mode = 0; x.dkv = dkv; x.H = H; x.n_keys_dev = c->enc_len_dev; x.desc = m.desc;
    x.part = m.att_part; x.counters = m.att_cnt; x.nsplit = ns_cross; x.err = &c->st->err;
    CUDA_TRY(c, launch_battn(c, MB, x, 1, ecap));
    // S6 / L6: cross output projection + residual
    o.W0 = w.wco;
    CUDA_TRY(c, launch_dec_linear(c, m, MB, o, l, TM_CO));
    // S7 / L7: norm + FFN up (ReLU, or GELU gate)
    LinArgs up{};
    up.desc = m.desc; up.eps = mc.ln_eps; up.W0 = w.wi0; up.W1 = w.wi1; up.X = m.x; up.ldx = d;
    up.gain = (const float*)w.ln3; up.N = F; up.K = d; up.Y = m.u; up.ldy = F;
    up.epi = mc.ffn_kind == BILD_FFN_GATED_GELU ? EPI_GATED : EPI_RELU;
    CUDA_TRY(c, launch_dec_linear(c, m, MB, up, l, TM_WI0));
    // S8 / L8: FFN down + residual
    LinArgs dn{};
    dn.desc = m.desc; dn.W0 = w.wfo; dn.X = m.u; dn.ldx = F; dn.N = d; dn.K = F; dn.epi = EPI_RESID; dn.Y = m.x; dn.ldy = d;
    CUDA_TRY(c, launch_dec_linear(c, m, MB, dn, l, TM_FO));
  }
  // S9+S10 / L9+L10: final norm + LM head + policy
  HeadArgs h{};
  h.W = m.w.lm_head; h.X = m.x; h.ldx = d; h.gain = (const float*)m.w.dec_final_ln; h.eps = mc.ln_eps;
  h.scale = mc.logit_scale; h.V = mc.vocab; h.K = d; h.desc = m.desc; h.partials = m.head_part;
  h.counter = m.head_cnt; h.out = m.head_out; h.logits_dbg = logits_dbg; h.which = which; h.loop = loop_ptrs(c);
  h.cond_while = cond_while; h.cond_if = cond_if; h.cond_if1 = cond_if1; h.cond_if8 = cond_if8;
  if (which == 0) { h.cond_switch = c->sw_handle; h.sw_bodies = c->sw_bodies; }
  h.pass_kind = which == 0 ? 0 : MBv == 1 ? 2 : MBv == SUB_MB ? 3 : 1;
  if (c->draw) {   // sampling: the head leaves its logits and the policy step to the kernel that draws the token
    if (!h.logits_dbg) h.logits_dbg = m.logits;
    h.defer_policy = 1;
  }
  auto draw_token = [&]() -> int {
    if (!c->draw) return BILD_OK;
    CUDA_TRY(c, launch_k(c, nucleus_policy_kernel, dim3(1), dim3(NS_THREADS), 0, h, (const float*)h.logits_dbg, (const float*)c->u_draw[which]));
    return BILD_OK;
  };
  const int head_tr = (MB == 1 && d <= 512) ? 32 : 16;   // rows per tile of the tensor-core head
  const size_t sh_smem = slice_head_smem_bytes(d, head_tr);
  // single-row passes: only heads of 32 MB and more (smaller ones stay on the GEMV head)
  const bool big_head = (size_t)mc.vocab * d * 2 >= c->slice_head_min_bytes;
  if (c->head_stream >= (big_head ? 1 : 2) && c->sms > 0 && (size_t)2 * c->sms <= head_partial_count(mc.vocab) && head_stream_fits(dt, MB, h)) {
    CUDA_TRY(c, launch_head_stream(c, h, c->sms));   // single row: the vocabulary streamed through registers
    return draw_token();
  }
  if (c->slice_head >= (MB == 1 ? 2 : 1) && (MB != 1 || big_head) && dt == BILD_BF16 && c->sms > 0 && c->sms <= MAX_GRID_SM && sh_smem <= 200 * 1024 &&
      d % 8 == 0 && ((uintptr_t)m.w.lm_head & 15) == 0) {
    // tensor-core head, one block per SM
    if (!c->slice_head_smem_set) {
      CUDA_TRY(c, cudaFuncSetAttribute(slice_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
      c->slice_head_smem_set = true;
    }
    CUDA_TRY(c, launch_k(c, slice_head_kernel, dim3(c->sms), dim3(SH_THREADS), sh_smem, h, &c->st->err, head_tr));
    return draw_token();
  }
  CUDA_TRY(c, launch_head(c->stream, c->use_pdl, dt, MB, h, m.head_grid, c->cnt));
  return draw_token();
}

// Encoder of model `which` over the ids in c->enc_ids, then the cross-attention K/V of
// every decoder layer.
int encoder_pass(bild_ctx* c, int which) {
  Model& m = c->m[which];
  bild_ctx::EncBuf& B = c->eb[which];
  const bild_model_cfg& mc = m.c;
  const int d = mc.d_model, I = m.inner, F = mc.d_ff, H = mc.n_heads, dkv = mc.d_kv;
  const int E = c->enc_len, ecap = c->cfg.max_enc_len, dt = c->cfg.dtype;
  const int rb = (E + MAXB - 1) / MAXB;
  CUDA_TRY(c, launch_embed(c, m.w.emb, c->enc_ids, nullptr, E, E, d, mc.vocab, B.ex));
  for (int l = 0; l < mc.n_layers; ++l) {
    const bild_enc_layer& w = m.enc[l];
    LinArgs a{};
    a.M = E; a.eps = mc.ln_eps; a.W0 = w.wqkv; a.X = B.ex; a.ldx = d; a.gain = (const float*)w.ln1;
    a.N = 3 * I; a.K = d; a.epi = EPI_HEADS; a.inner = I; a.dkv = dkv; a.first_part = 0; a.q_out = B.eq; a.ldq = I;
    a.kc = B.ek; a.vc = B.ev; a.cap = ecap; a.pos0_host = 0;
    // with the GEMM path the layer inputs alternate between two (bf16 head, remainder) buffer pairs:
    // norm(x) -> pair 0 -> QKV; attention -> pair 1 -> O; norm(x) -> pair 0 -> FFN-up -> pair 1 -> FFN-down
    const bool fuse = m.enc_gemm && c->enc_attn_mma && dkv == EA_D;
    CUDA_TRY(c, launch_enc_linear(c, m, a, rb, l, TM_EQKV, true, 0));
    BAttnArgs t{};
    t.q = B.eq; t.ldq = I; t.kc = B.ek; t.vc = B.ev; t.cap = ecap; t.out = B.eatt; t.ldo = I;
    t.bias = m.enc_bias; t.bias_ld = 2 * ecap - 1; t.bias_off = ecap - 1; t.mode = 2; t.dkv = dkv; t.H = H;
    t.n_keys_dev = c->enc_len_dev; t.M = E; t.part = m.att_part; t.counters = m.att_cnt; t.nsplit = 1;
    t.err = &c->st->err;
    CUDA_TRY(c, launch_battn(c, MAXB, t, rb, ecap, fuse ? B.exh[1] : nullptr, fuse ? B.exl[1] : nullptr));
    LinArgs o{};
    o.M = E; o.W0 = w.wo; o.X = B.eatt; o.ldx = I; o.N = d; o.K = I; o.epi = EPI_RESID; o.Y = B.ex; o.ldy = d;
    CUDA_TRY(c, launch_enc_linear(c, m, o, rb, l, TM_EO, !fuse, 1));
    LinArgs up{};
    up.M = E; up.eps = mc.ln_eps; up.W0 = w.wi0; up.W1 = w.wi1; up.X = B.ex; up.ldx = d; up.gain = (const float*)w.ln2;
    up.N = F; up.K = d; up.Y = B.eu; up.ldy = F;
    up.epi = mc.ffn_kind == BILD_FFN_GATED_GELU ? EPI_GATED : EPI_RELU;
    CUDA_TRY(c, launch_enc_linear(c, m, up, rb, l, TM_EWI0, true, 0, m.enc_gemm ? 1 : -1));
    LinArgs dn{};
    dn.M = E; dn.W0 = w.wfo; dn.X = B.eu; dn.ldx = F; dn.N = d; dn.K = F; dn.epi = EPI_RESID; dn.Y = B.ex; dn.ldy = d;
    CUDA_TRY(c, launch_enc_linear(c, m, dn, rb, l, TM_EFO, !m.enc_gemm, 1));
  }
  // encoder memory = final norm of ex (fused into the projections); cross K/V per decoder layer.  The projections of the
  // layers are independent of one another (each covers a fraction of the SMs): after the first, which also writes the
  // normalised encoder output, they are dealt to this stream and two more.
  cudaStream_t base = c->stream;
  bool spread = c->enc_kv_streams && m.enc_gemm && mc.n_layers >= 4;
  if (spread && !c->kv_stream[0]) {
    bool ok = cudaEventCreateWithFlags(&c->kv_fork, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      ok = cudaStreamCreateWithFlags(&c->kv_stream[i], cudaStreamNonBlocking) == cudaSuccess &&
           cudaEventCreateWithFlags(&c->kv_join[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { cudaGetLastError(); spread = c->enc_kv_streams = false; }
  }
  int rc = BILD_OK;
  for (int l = 0; l < mc.n_layers && rc == BILD_OK; ++l) {
    const size_t kvoff = (size_t)l * H * dkv;
    LinArgs a{};
    a.M = E; a.eps = mc.ln_eps; a.W0 = m.dec[l].wckv; a.X = B.ex; a.ldx = d; a.gain = (const float*)m.w.enc_final_ln;
    a.N = 2 * I; a.K = d; a.epi = EPI_HEADS; a.inner = I; a.dkv = dkv; a.first_part = 1;
    a.kc = m.crossK + kvoff * ecap; a.vc = m.crossV + kvoff * ecap; a.cap = ecap; a.pos0_host = 0;
    if (spread && l > 0 && l % 3) c->stream = c->kv_stream[l % 3 - 1];
    const cudaError_t e = launch_enc_linear(c, m, a, rb, l, TM_CKV, l == 0, 0);   // the normalised encoder output is split once
    c->stream = base;
    if (e != cudaSuccess) rc = fail(c, BILD_ERR_CUDA, std::string("cross K/V projection: ") + cudaGetErrorString(e));
    if (spread && l == 0 && rc == BILD_OK) {   // the other streams start once the split rows exist
      if (cudaEventRecord(c->kv_fork, base) != cudaSuccess || cudaStreamWaitEvent(c->kv_stream[0], c->kv_fork, 0) != cudaSuccess ||
          cudaStreamWaitEvent(c->kv_stream[1], c->kv_fork, 0) != cudaSuccess) rc = fail(c, BILD_ERR_CUDA, "cross K/V projection: fork");
    }
  }
  if (spread)   // joined in any case, so that nothing is left running beside the caller's stream
    for (int i = 0; i < 2; ++i)
      if (cudaEventRecord(c->kv_join[i], c->kv_stream[i]) != cudaSuccess || cudaStreamWaitEvent(base, c->kv_join[i], 0) != cudaSuccess)
        rc = rc ? rc : fail(c, BILD_ERR_CUDA, "cross K/V projection: join");
  return rc;
}

int build_bias_tables(bild_ctx* c) {
  const int cap = c->cfg.max_dec_len, ecap = c->cfg.max_enc_len;
  for (int i = 0; i < 2; ++i) {
    Model& m = c->m[i];
    std::vector<int> tab(cap);
    for (int x = 0; x < cap; ++x) tab[x] = decoder_bucket(x, m.c.rel_buckets, m.c.rel_max_dist);
    CUDA_TRY(c, cudaMemcpyAsync(c->bucket_tmp, tab.data(), cap * sizeof(int), cudaMemcpyHostToDevice, c->stream));
    bias_table_kernel<<<(cap + 127) / 128, 128, 0, c->stream>>>((const float*)m.w.dec_rel_bias, c->bucket_tmp, cap,
                                                                m.c.n_heads, m.dec_bias);
    (*c->cnt)++;
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    const int ne = 2 * ecap - 1;
    std::vector<int> etab(ne);
    for (int x = 0; x < ne; ++x) etab[x] = encoder_bucket(x - (ecap - 1), m.c.rel_buckets, m.c.rel_max_dist);
    CUDA_TRY(c, cudaMemcpyAsync(c->bucket_tmp, etab.data(), ne * sizeof(int), cudaMemcpyHostToDevice, c->stream));
    bias_table_kernel<<<(ne + 127) / 128, 128, 0, c->stream>>>((const float*)m.w.enc_rel_bias, c->bucket_tmp, ne,
                                                               m.c.n_heads, m.enc_bias);
    (*c->cnt)++;
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  }
  return BILD_OK;
}

// Adds a conditional node to `g` after `deps` and returns its body graph.
int add_cond(bild_ctx* c, cudaGraph_t g, const cudaGraphNode_t* deps, size_t ndeps, cudaGraphConditionalHandle h,
             cudaGraphConditionalNodeType type, cudaGraph_t* body) {
  cudaGraphNodeParams p = {cudaGraphNodeTypeConditional};
  p.conditional.handle = h;
  p.conditional.type = type;
  p.conditional.size = 1;
  cudaGraphNode_t node;
  CUDA_TRY(c, cudaGraphAddNode(&node, g, deps, ndeps, &p));
  *body = p.conditional.phGraph_out[0];
  return BILD_OK;
}

// Captures one decoder pass into `body`; returns the leaf nodes of the capture.
int capture_pass(bild_ctx* c, cudaGraph_t body, int which, int MB, unsigned long long hw, unsigned long long hi,
                 std::vector<cudaGraphNode_t>* leaves, int64_t* count, unsigned long long hi1 = 0, unsigned long long hi8 = 0) {
  if (!c->cap_stream) CUDA_TRY(c, cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking));
  CUDA_TRY(c, cudaStreamBeginCaptureToGraph(c->cap_stream, body, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed));
  int64_t n = 0;
  cudaStream_t user_stream = c->stream;
  c->stream = c->cap_stream;
  c->cnt = &n;
  c->capturing = true;
  int rc = decoder_pass(c, which, MB, nullptr, hw, hi, hi1, hi8);
  c->capturing = false;
  c->cnt = &c->launches;
  c->stream = user_stream;
  if (rc == BILD_OK && leaves) {
    cudaStreamCaptureStatus st;
    const cudaGraphNode_t* deps = nullptr;
    size_t nd = 0;
    if (cudaStreamGetCaptureInfo(c->cap_stream, &st, nullptr, nullptr, &deps, &nd) != cudaSuccess) rc = BILD_ERR_CUDA;
    else leaves->assign(deps, deps + nd);
  }
  cudaGraph_t got = nullptr;
  cudaError_t e = cudaStreamEndCapture(c->cap_stream, &got);
  if (rc != BILD_OK) return rc;
  if (e != cudaSuccess) return fail(c, BILD_ERR_CUDA, std::string("cudaStreamEndCapture: ") + cudaGetErrorString(e));
  *count = n;
  return BILD_OK;
}

// Builds the two device-side loops (CUDA graphs with conditional nodes).  The head
// kernel's last block sets the WHILE handle to "not done" and the IF handle to "fallback".
int build_graphs_once(bild_ctx* c, int base);

void drop_graphs(bild_ctx* c) {
  for (int i = 0; i < 4; ++i) {
    if (c->exec[i]) cudaGraphExecDestroy(c->exec[i]);
    if (c->graph[i]) cudaGraphDestroy(c->graph[i]);
    c->exec[i] = nullptr;
    c->graph[i] = nullptr;
  }
}

// base 0: the greedy loops; base 2: the loops of the sampling variant (a token-drawing kernel after every LM head)
int build_graphs(bild_ctx* c, int base) {
  if (c->exec[base] && c->exec[base + 1]) return BILD_OK;
  // if a loop body refuses programmatic edges, the graphs are built again with plain launches
  const bool want_pdl = c->use_pdl;
  c->draw = base == 2;
  int rc = build_graphs_once(c, base);
  if (rc != BILD_OK && c->graph_switch) {   // no SWITCH nodes here: one IF node per kind of pass
    drop_graphs(c);
    cudaGetLastError();
    c->graph_switch = false;
    rc = build_graphs_once(c, base);
  }
  if (rc != BILD_OK && want_pdl) {
    drop_graphs(c);
    cudaGetLastError();
    c->use_pdl = false;
    rc = build_graphs_once(c, base);
  }
  c->draw = false;
  if (rc != BILD_OK) { drop_graphs(c); cudaGetLastError(); }
  return rc;
}

int build_graphs_once(bild_ctx* c, int base) {
  // launches per pass are recorded from the greedy graphs; the drawing kernels of the sampled ones are counted on the device
  int64_t dummy[2] = {0, 0}, dummy1 = 0, dummy8 = 0;
  int64_t* per_pass = base == 0 ? c->per_pass : dummy;
  int64_t& per_pass_large1 = base == 0 ? c->per_pass_large1 : dummy1;
  int64_t& per_pass_large8 = base == 0 ? c->per_pass_large8 : dummy8;
  cudaGraph_t* graph = c->graph + base;
  cudaGraphExec_t* exec = c->exec + base;
  {  // BiLD (and small-only): WHILE { small pass ; IF { large block pass } ; IF { large single-row pass } }
    CUDA_TRY(c, cudaGraphCreate(&graph[0], 0));
    cudaGraphConditionalHandle hw, hi, hi1, hi8 = 0;
    CUDA_TRY(c, cudaGraphConditionalHandleCreate(&hw, graph[0], 1, cudaGraphCondAssignDefault));
    CUDA_TRY(c, cudaGraphConditionalHandleCreate(&hi, graph[0], 0, cudaGraphCondAssignDefault));
    CUDA_TRY(c, cudaGraphConditionalHandleCreate(&hi1, graph[0], 0, cudaGraphCondAssignDefault));
    // passes of 2 to 8 rows have a branch of their own where they run on the fused sub-layer kernels
    const bool body8 = c->m[1].fused && c->fused_on >= 2;
    if (body8) CUDA_TRY(c, cudaGraphConditionalHandleCreate(&hi8, graph[0], 0, cudaGraphCondAssignDefault));
    cudaGraph_t body = nullptr, ifbody = nullptr, if1body = nullptr, if8body = nullptr;
    int rc = add_cond(c, graph[0], nullptr, 0, hw, cudaGraphCondTypeWhile, &body);
    if (rc) return rc;
    std::vector<cudaGraphNode_t> leaves;
    if (c->graph_switch) {   // one conditional node per iteration: SWITCH { block pass | single-row pass | pass of 2 to 8 rows }
      const int nb = body8 ? 3 : 2;
      cudaGraphConditionalHandle hs;
      CUDA_TRY(c, cudaGraphConditionalHandleCreate(&hs, graph[0], (unsigned)nb, cudaGraphCondAssignDefault));
      c->sw_handle = hs; c->sw_bodies = nb;
      rc = capture_pass(c, body, 0, 1, hw, 0, &leaves, &per_pass[0]);
      c->sw_handle = 0; c->sw_bodies = 0;
      if (rc) return rc;
      cudaGraphNodeParams p = {cudaGraphNodeTypeConditional};
      p.conditional.handle = hs;
      p.conditional.type = cudaGraphCondTypeSwitch;
      p.conditional.size = (unsigned)nb;
      cudaGraphNode_t node;
      CUDA_TRY(c, cudaGraphAddNode(&node, body, leaves.data(), leaves.size(), &p));
      rc = capture_pass(c, p.conditional.phGraph_out[0], 1, MAXB, hw, 0, nullptr, &per_pass[1]);
      if (rc) return rc;
      int64_t n1 = 0;
      rc = capture_pass(c, p.conditional.phGraph_out[1], 1, 1, hw, 0, nullptr, &n1);
      if (rc) return rc;
      per_pass_large1 = n1;
      if (body8) {
        rc = capture_pass(c, p.conditional.phGraph_out[2], 1, SUB_MB, hw, 0, nullptr, &per_pass_large8);
        if (rc) return rc;
      }
      CUDA_TRY(c, cudaGraphInstantiate(&exec[0], graph[0], 0));
    } else {
    rc = capture_pass(c, body, 0, 1, hw, hi, &leaves, &per_pass[0], hi1, hi8);
    if (rc) return rc;
    rc = add_cond(c, body, leaves.data(), leaves.size(), hi, cudaGraphCondTypeIf, &ifbody);
    if (rc) return rc;
    rc = capture_pass(c, ifbody, 1, MAXB, hw, 0, nullptr, &per_pass[1]);
    if (rc) return rc;
    // a fallback right after a large pass verifies one row: that pass runs on the single-row kernels
    rc = add_cond(c, body, leaves.data(), leaves.size(), hi1, cudaGraphCondTypeIf, &if1body);
    if (rc) return rc;
    int64_t n1 = 0;
    rc = capture_pass(c, if1body, 1, 1, hw, 0, nullptr, &n1);
    if (rc) return rc;
    per_pass_large1 = n1;
    if (body8) {
      rc = add_cond(c, body, leaves.data(), leaves.size(), hi8, cudaGraphCondTypeIf, &if8body);
      if (rc) return rc;
      rc = capture_pass(c, if8body, 1, SUB_MB, hw, 0, nullptr, &per_pass_large8);
      if (rc) return rc;
    }
    CUDA_TRY(c, cudaGraphInstantiate(&exec[0], graph[0], 0));
    }
  }
  {  // large-only greedy: WHILE { large pass with k = 1 }
    CUDA_TRY(c, cudaGraphCreate(&graph[1], 0));
    cudaGraphConditionalHandle hw;
    CUDA_TRY(c, cudaGraphConditionalHandleCreate(&hw, graph[1], 1, cudaGraphCondAssignDefault));
    cudaGraph_t body = nullptr;
    int rc = add_cond(c, graph[1], nullptr, 0, hw, cudaGraphCondTypeWhile, &body);
    if (rc) return rc;
    rc = capture_pass(c, body, 1, 1, hw, 0, nullptr, &per_pass_large1);
    if (rc) return rc;
    CUDA_TRY(c, cudaGraphInstantiate(&exec[1], graph[1], 0));
  }
  return BILD_OK;
}

int read_state(bild_ctx* c) {
  CUDA_TRY(c, cudaMemcpyAsync(c->pin_state, c->st, sizeof(DevState), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  {  // kernels launched by the loop graphs so far (the device counts the passes they ran)
    const long long* cp = c->pin_state->cum_passes;
    const int64_t total = cp[0] * c->per_pass[0] + cp[1] * c->per_pass[1] + cp[2] * c->per_pass_large1 + cp[3] * c->per_pass_large8;
    c->launches += total - c->graph_counted;
    c->graph_counted = total;
    c->launches += c->pin_state->cum_draws - c->sampled_counted;
    c->sampled_counted = c->pin_state->cum_draws;
  }
  if (c->pin_state->err) return fail(c, c->pin_state->err, "device-side error flag set");
  return BILD_OK;
}

int reset_state(bild_ctx* c, int mode, float afb, float arb, int max_len) {
  reset_state_kernel<<<1, 1, 0, c->stream>>>(loop_ptrs(c), mode, afb, arb, max_len, c->cfg.max_draft,
                                             c->cfg.eos_id, c->cfg.start_id, c->trace_cap, c->top_p);
  (*c->cnt)++;
  CUDA_TRY(c, cudaGetLastError());
  // the buffer the first fused sub-layer kernel of a pass adds into: every pass leaves it clear; cleared here as well, so
  // that a pass that ended in an error cannot leak into the next generation
  for (int i = 0; i < 2; ++i)
    if (c->m[i].fused && c->m[i].xb) CUDA_TRY(c, cudaMemsetAsync(c->m[i].xb, 0, (size_t)MAXB * c->m[i].c.d_model * sizeof(float), c->stream));
  return BILD_OK;
}

}  // namespace

// ======================================================================================
// extern "C" boundary
// ======================================================================================
extern "C" {

int bild_query_workspace(const bild_config* cfg, size_t* bytes) {
  std::string why;
  if (!bytes) return BILD_ERR_ARG;
  int rc = check_config(cfg, why);
  if (rc) return rc;
  bild_ctx tmp;
  tmp.cfg = *cfg;
  Bump b(nullptr);
  plan(&tmp, b);
  *bytes = b.off;
  return BILD_OK;
}

void bild_tuning_default(bild_tuning* t) {
  if (!t) return;
  t->host_loop = 0; t->pdl = 1; t->fused = 3; t->ffn_parts = 0; t->block_simt = 0; t->slice_mode = 2;
  t->slice_min_kb = 3000; t->slice_mma_min = 3; t->slice_head = 2; t->slice_head_min_mb = 32; t->unit_attn = 1;
  t->umma = 1; t->enc_gemm = 1; t->enc_attn_mma = 1; t->enc_parallel = 1; t->spin_limit = 0; t->debug_skip_copies = 0;
  t->attn_all_keys = 128; t->graph_switch = 1; t->enc_split_k = 1; t->head_stream = 2; t->enc_attn_groups = EA_MAX_GROUPS;
}

int bild_create(const bild_config* cfg, const bild_weights* small_w, const bild_weights* large_w, void* workspace,
                size_t workspace_bytes, void* cuda_stream, bild_ctx** out) {
  return bild_create_tuned(cfg, small_w, large_w, workspace, workspace_bytes, cuda_stream, nullptr, out);
}

int bild_create_tuned(const bild_config* cfg, const bild_weights* small_w, const bild_weights* large_w, void* workspace,
                      size_t workspace_bytes, void* cuda_stream, const bild_tuning* tuning, bild_ctx** out) {
  if (!out) return BILD_ERR_ARG;
  *out = nullptr;
  std::string why;
  int rc = check_config(cfg, why);
  if (rc) return rc;
  const bool early = cfg->early_exit_layers > 0;
  if ((!small_w && !early) || !large_w || !workspace) return BILD_ERR_ARG;
  if ((uintptr_t)workspace % 256) return BILD_ERR_WORKSPACE;
  bild_ctx* c = new (std::nothrow) bild_ctx;
  if (!c) return BILD_ERR_ARG;
  c->cfg = *cfg;
  c->stream = (cudaStream_t)cuda_stream;
  c->cnt = &c->launches;
  {
    bild_tuning t;
    bild_tuning_default(&t);
    if (tuning) t = *tuning;
    c->host_loop = t.host_loop != 0;
    c->use_pdl = t.pdl != 0;
    c->fused_on = std::min(3, std::max(0, t.fused));
    c->sub_parts_want = std::min(8, std::max(0, t.ffn_parts));
    c->block_simt = t.block_simt != 0;
    c->slice_mode = std::min(2, std::max(0, t.slice_mode));
    c->slice_min_bytes = (size_t)std::max(0, t.slice_min_kb) * 1024;
    c->slice_mma_min = std::min(5, std::max(2, t.slice_mma_min));
    c->slice_head = std::min(2, std::max(0, t.slice_head));
    c->slice_head_min_bytes = (size_t)std::max(0, t.slice_head_min_mb) << 20;
    c->unit_attn = t.unit_attn != 0;
    c->use_umma = t.umma != 0;
    c->use_enc_gemm = t.enc_gemm != 0;
    c->enc_attn_mma = t.enc_attn_mma != 0;
    c->enc_parallel = t.enc_parallel != 0;
    c->enc_kv_streams = t.enc_parallel != 0;   // (one switch: everything of the set-up step on one stream, or not)
    c->spin_limit = t.spin_limit > 0 ? (unsigned)t.spin_limit : SPIN_LIMIT;
    c->debug_skip_copies = t.debug_skip_copies != 0;
    c->attn_all_keys = std::min(128, std::max(0, t.attn_all_keys));
    c->graph_switch = t.graph_switch != 0;
    c->enc_split_k = t.enc_split_k != 0;
    c->head_stream = std::min(2, std::max(0, t.head_stream));
    c->enc_attn_groups = std::min(EA_MAX_GROUPS, std::max(1, t.enc_attn_groups));
  }
  {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError();
      c->sms = 0;
    }
  }
  Bump b(workspace);
  plan(c, b);
  c->ws_bytes = b.off;
  if (workspace_bytes < b.off) { delete c; return BILD_ERR_WORKSPACE; }
  if (early) {   // one cache for the shared layers: [layer][head][row][channel], the small model's layers come first
    c->m[0].selfK = c->m[1].selfK; c->m[0].selfV = c->m[1].selfV;
    c->m[0].crossK = c->m[1].crossK; c->m[0].crossV = c->m[1].crossV;
  }
  const bild_weights* ws[2] = {early ? large_w : small_w, large_w};   // early exit: the small model is a prefix of the large one
  for (int i = 0; i < 2; ++i) {
    Model& m = c->m[i];
    const bild_weights* w = ws[i];
    if (!w->emb || !w->lm_head || !w->enc_rel_bias || !w->dec_rel_bias || !w->enc_final_ln || !w->dec_final_ln ||
        !w->enc_layers || !w->dec_layers) { delete c; return BILD_ERR_ARG; }
    m.w = *w;
    m.enc.assign(w->enc_layers, w->enc_layers + m.c.n_layers);
    m.dec.assign(w->dec_layers, w->dec_layers + m.c.n_layers);
    const bool gated = m.c.ffn_kind == BILD_FFN_GATED_GELU;
    for (int l = 0; l < m.c.n_layers; ++l) {
      const bild_enc_layer& e = m.enc[l];
      const bild_dec_layer& d = m.dec[l];
      if (!e.ln1 || !e.wqkv || !e.wo || !e.ln2 || !e.wi0 || !e.wfo || (gated && !e.wi1) || !d.ln1 || !d.wqkv ||
          !d.wo || !d.ln2 || !d.wcq || !d.wckv || !d.wco || !d.ln3 || !d.wi0 || !d.wfo || (gated && !d.wi1)) {
        delete c;
        return BILD_ERR_ARG;
      }
    }
    m.w.enc_layers = nullptr;
    m.w.dec_layers = nullptr;
    setup_umma(c, m);
  }
  if (cudaMallocHost((void**)&c->pin_state, sizeof(DevState)) != cudaSuccess ||
      cudaMallocHost((void**)&c->pin_head, sizeof(HeadOut)) != cudaSuccess) {
    bild_destroy(c);
    return BILD_ERR_CUDA;
  }
  // zero the ticket counters and the state, build the bias-by-distance tables
  if (cudaMemsetAsync(workspace, 0, c->ws_bytes, c->stream) != cudaSuccess) { bild_destroy(c); return BILD_ERR_CUDA; }
  for (int i = 0; i < 2; ++i) {
    rc = setup_fused(c, c->m[i]);
    if (rc) { bild_destroy(c); return rc; }
  }
  rc = build_bias_tables(c);
  if (rc) { bild_destroy(c); return rc; }
  *out = c;
  return BILD_OK;
}

void bild_destroy(bild_ctx* c) {
  if (!c) return;
  drop_graphs(c);
  if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
  if (c->side2) { cudaStreamSynchronize(c->side2); cudaStreamDestroy(c->side2); }
  for (int i = 0; i < 2; ++i) {
    if (c->kv_stream[i]) { cudaStreamSynchronize(c->kv_stream[i]); cudaStreamDestroy(c->kv_stream[i]); }
    if (c->kv_join[i]) cudaEventDestroy(c->kv_join[i]);
  }
  if (c->kv_fork) cudaEventDestroy(c->kv_fork);
  for (cudaEvent_t e : c->chunk_ev) cudaEventDestroy(e);
  if (c->enc_stream) { cudaStreamSynchronize(c->enc_stream); cudaStreamDestroy(c->enc_stream); }
  if (c->enc_fork) cudaEventDestroy(c->enc_fork);
  if (c->enc_join) cudaEventDestroy(c->enc_join);
  if (c->pin_state) cudaFreeHost(c->pin_state);
  if (c->pin_head) cudaFreeHost(c->pin_head);
  delete c;
}

int bild_uses_tensor_cores(const bild_ctx* c) { return c && c->m[1].umma ? 1 : 0; }

const char* bild_last_error(const bild_ctx* c) { return c ? c->err.c_str() : "null context"; }
int64_t bild_launch_count(const bild_ctx* c) { return c ? c->launches : 0; }

int bild_encode(bild_ctx* c, const int32_t* ids, int n_ids) {
  if (!c || !ids) return fail(c, BILD_ERR_ARG, "null argument");
  if (n_ids < 1 || n_ids > c->cfg.max_enc_len) return fail(c, BILD_ERR_CAPACITY, "n_ids outside 1..max_enc_len");
  c->encoded = false;
  c->enc_len = n_ids;
  CUDA_TRY(c, cudaMemcpyAsync(c->enc_ids, ids, n_ids * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaMemcpyAsync(c->enc_len_dev, &c->enc_len, sizeof(int), cudaMemcpyHostToDevice, c->stream));
  // The two encoders are independent: the small model's runs on a side stream, forked from and joined
  // back into the caller's stream with events, while the large model's runs on the caller's stream.
  const bool early = c->cfg.early_exit_layers > 0;   // one encoder: the small model is a prefix of the large model's decoder
  bool side = c->enc_parallel && !early;
  if (side && !c->enc_stream) {
    if (cudaStreamCreateWithFlags(&c->enc_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->enc_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->enc_join, cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      side = c->enc_parallel = false;
    }
  }
  if (side) {
    CUDA_TRY(c, cudaEventRecord(c->enc_fork, c->stream));
    CUDA_TRY(c, cudaStreamWaitEvent(c->enc_stream, c->enc_fork, 0));
    cudaStream_t user_stream = c->stream;
    c->stream = c->enc_stream;
    int rc0 = encoder_pass(c, 0);
    c->stream = user_stream;
    if (rc0) return rc0;
    CUDA_TRY(c, cudaEventRecord(c->enc_join, c->enc_stream));
    int rc1 = encoder_pass(c, 1);
    if (rc1) return rc1;
    CUDA_TRY(c, cudaStreamWaitEvent(c->stream, c->enc_join, 0));
  } else {
    for (int i = early ? 1 : 0; i < 2; ++i) {
      int rc = encoder_pass(c, i);
      if (rc) return rc;
    }
  }
  int rc = reset_state(c, BILD_MODE_BILD, 0.f, INFINITY, c->cfg.max_dec_len - 1);
  if (rc) return rc;
  c->encoded = true;
  return BILD_OK;
}

int bild_reset(bild_ctx* c) {
  if (!c) return BILD_ERR_ARG;
  if (!c->encoded) return fail(c, BILD_ERR_STATE, "bild_encode has not been called");
  return reset_state(c, BILD_MODE_BILD, 0.f, INFINITY, c->cfg.max_dec_len - 1);
}

int bild_small_step(bild_ctx* c, int32_t token, float alpha_fb, bild_step_out* out, float* logits_dbg) {
  if (!c || !out) return fail(c, BILD_ERR_ARG, "null argument");
  if (!c->encoded) return fail(c, BILD_ERR_STATE, "bild_encode has not been called");
  if (token < 0 || token >= c->m[0].c.vocab) return fail(c, BILD_ERR_ARG, "token outside the vocabulary");
  int rc = read_state(c);
  if (rc) return rc;
  if (c->pin_state->S_len + 1 > c->cfg.max_dec_len) return fail(c, BILD_ERR_CAPACITY, "small-model cache is full");
  TokList t{};
  t.t[0] = token;
  set_alpha_kernel<<<1, 1, 0, c->stream>>>(c->st, alpha_fb, c->pin_state->alpha_rb);
  set_desc_kernel<<<1, 1, 0, c->stream>>>(c->m[0].desc, c->st, 0, 1, t);
  c->launches += 2;
  rc = decoder_pass(c, 0, 1, logits_dbg);
  if (rc) return rc;
  CUDA_TRY(c, cudaMemcpyAsync(c->pin_head, c->m[0].head_out, sizeof(HeadOut), cudaMemcpyDeviceToHost, c->stream));
  rc = read_state(c);
  if (rc) return rc;
  out->argmax = c->pin_head->argmax[0];
  out->max_logit = c->pin_head->zmax[0];
  out->lse = c->pin_head->lse[0];
  out->pmax = c->pin_head->pmax;
  out->fallback = c->pin_head->fallback;
  return BILD_OK;
}

int bild_large_verify(bild_ctx* c, const int32_t* tokens, int k, float alpha_rb, bild_verify_out* out,
                      float* logits_dbg) {
  if (!c || !out || !tokens) return fail(c, BILD_ERR_ARG, "null argument");
  if (!c->encoded) return fail(c, BILD_ERR_STATE, "bild_encode has not been called");
  if (k < 1 || k > MAXB) return fail(c, BILD_ERR_ARG, "k outside 1..16");
  for (int i = 0; i < k; ++i)
    if (tokens[i] < 0 || tokens[i] >= c->m[1].c.vocab) return fail(c, BILD_ERR_ARG, "token outside the vocabulary");
  int rc = read_state(c);
  if (rc) return rc;
  if (c->pin_state->L_len + k > c->cfg.max_dec_len) return fail(c, BILD_ERR_CAPACITY, "large-model cache is full");
  TokList t{};
  for (int i = 0; i < k; ++i) t.t[i] = tokens[i];
  set_alpha_kernel<<<1, 1, 0, c->stream>>>(c->st, c->pin_state->alpha_fb, alpha_rb);
  set_desc_kernel<<<1, 1, 0, c->stream>>>(c->m[1].desc, c->st, 1, k, t);
  c->launches += 2;
  rc = decoder_pass(c, 1, k == 1 ? 1 : k <= SUB_MB ? SUB_MB : MAXB, logits_dbg);
  if (rc) return rc;
  CUDA_TRY(c, cudaMemcpyAsync(c->pin_head, c->m[1].head_out, sizeof(HeadOut), cudaMemcpyDeviceToHost, c->stream));
  rc = read_state(c);
  if (rc) return rc;
  for (int i = 0; i < MAXB; ++i) {
    out->argmax[i] = i < k ? c->pin_head->argmax[i] : -1;
    out->lse[i] = i < k ? c->pin_head->lse[i] : 0.f;
    out->d[i] = i < k - 1 ? c->pin_head->d[i] : 0.f;
  }
  out->first_violation = c->pin_head->first_violation;
  out->next_token = c->pin_head->next_token;
  return BILD_OK;
}

int bild_rewind(bild_ctx* c, int which, int new_len) {
  if (!c || (which != 0 && which != 1)) return fail(c, BILD_ERR_ARG, "which must be 0 or 1");
  if (!c->encoded) return fail(c, BILD_ERR_STATE, "bild_encode has not been called");
  int rc = read_state(c);
  if (rc) return rc;
  const int cur = which == 0 ? c->pin_state->S_len : c->pin_state->L_len;
  if (new_len < 0 || new_len > cur) return fail(c, BILD_ERR_ARG, "new_len outside 0..current length");
  rewind_kernel<<<1, 1, 0, c->stream>>>(c->st, which, new_len);
  (*c->cnt)++;
  CUDA_TRY(c, cudaGetLastError());
  return BILD_OK;
}

}  // extern "C"

namespace {
// top_p > 0: the sampling variant, with the uniform numbers of both models by output position (HOST, max_len + 1 each)
int generate_async(bild_ctx* c, int mode, float alpha_fb, float alpha_rb, int max_len, float top_p, const float* u_small,
                   const float* u_large) {
  if (!c) return BILD_ERR_ARG;
  if (!c->encoded) return fail(c, BILD_ERR_STATE, "bild_encode has not been called");
  if (mode < 0 || mode > 2) return fail(c, BILD_ERR_ARG, "mode");
  if (max_len < 0) return fail(c, BILD_ERR_ARG, "max_len < 0");
  if (max_len + 1 > c->cfg.max_dec_len) return fail(c, BILD_ERR_CAPACITY, "max_len + 1 > max_dec_len");
  const bool sampled = top_p > 0.f;
  c->top_p = sampled ? top_p : 0.f;
  if (sampled) {
    if (!(top_p <= 1.f) || !u_small || !u_large) return fail(c, BILD_ERR_ARG, "sampling needs 0 < top_p <= 1 and both arrays of uniform numbers");
    for (int i = 0; i <= max_len; ++i)
      if (!(u_small[i] >= 0.f && u_small[i] < 1.f) || !(u_large[i] >= 0.f && u_large[i] < 1.f))
        return fail(c, BILD_ERR_ARG, "uniform numbers must lie in [0, 1)");
    CUDA_TRY(c, cudaMemcpyAsync(c->u_draw[0], u_small, (max_len + 1) * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(c->u_draw[1], u_large, (max_len + 1) * sizeof(float), cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));   // the caller's arrays may be pageable and go away
  }
  if (!c->host_loop) {
    // device-side loop: no host involvement between the first and the last token
    const int base = sampled ? 2 : 0;
    int rc = build_graphs(c, base);
    if (rc) return rc;
    rc = reset_state(c, mode, alpha_fb, alpha_rb, max_len);
    if (rc) return rc;
    if (max_len == 0 || c->cfg.start_id == c->cfg.eos_id) return BILD_OK;
    // passes the loop may run: bounded by the guard of the device-side policy
    CUDA_TRY(c, cudaGraphLaunch(c->exec[base + (mode == BILD_MODE_LARGE_ONLY ? 1 : 0)], c->stream));
    return BILD_OK;
  }
  int rc = reset_state(c, mode, alpha_fb, alpha_rb, max_len);
  if (rc) return rc;
  struct DrawGuard { bild_ctx* c; ~DrawGuard() { c->draw = false; } } guard_draw{c};
  c->draw = sampled;
  // Debug loop driver: the policy still runs on the device; the host reads two flags per step.
  const int guard = (max_len + 1) * (c->cfg.max_draft + 3);
  rc = read_state(c);
  if (rc) return rc;
  for (int it = 0; it < guard && !c->pin_state->done; ++it) {
    if (mode != BILD_MODE_LARGE_ONLY) {
      rc = decoder_pass(c, 0, 1, nullptr);
      if (rc) return rc;
      rc = read_state(c);
      if (rc) return rc;
      if (!c->pin_state->fallback) continue;
    }
    const int kk = c->pin_state->n - c->pin_state->L_len + 1;   // rows the large model has not seen
    rc = decoder_pass(c, 1, (mode == BILD_MODE_LARGE_ONLY || kk == 1) ? 1 : kk <= SUB_MB ? SUB_MB : MAXB, nullptr);
    if (rc) return rc;
    rc = read_state(c);
    if (rc) return rc;
  }
  return BILD_OK;
}
}  // namespace

extern "C" {

int bild_generate_async(bild_ctx* c, int mode, float alpha_fb, float alpha_rb, int max_len) {
  return generate_async(c, mode, alpha_fb, alpha_rb, max_len, 0.f, nullptr, nullptr);
}

int bild_generate_sampled(bild_ctx* c, int mode, float alpha_fb, float alpha_rb, int max_len, float top_p, const float* u_small,
                          const float* u_large, int32_t* tokens_out, int* n_tokens, bild_trace_rec* trace_out, int trace_cap,
                          int* n_trace, bild_stats* stats) {
  if (!c || !tokens_out || !n_tokens) return fail(c, BILD_ERR_ARG, "null argument");
  if (!(top_p > 0.f)) return fail(c, BILD_ERR_ARG, "top_p must be positive");
  int rc = generate_async(c, mode, alpha_fb, alpha_rb, max_len, top_p, u_small, u_large);
  if (rc) return rc;
  return bild_fetch_result(c, tokens_out, n_tokens, trace_out, trace_cap, n_trace, stats);
}

int bild_fetch_result(bild_ctx* c, int32_t* tokens_out, int* n_tokens, bild_trace_rec* trace_out, int trace_cap,
                      int* n_trace, bild_stats* stats) {
  if (!c || !tokens_out || !n_tokens) return fail(c, BILD_ERR_ARG, "null argument");
  int rc = read_state(c);
  if (rc) return rc;
  const DevState& s = *c->pin_state;
  *n_tokens = s.n;
  if (s.n > 0) CUDA_TRY(c, cudaMemcpyAsync(tokens_out, c->y + 1, s.n * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  if (n_trace) *n_trace = s.n_trace;
  const int nt = std::min(std::min(s.n_trace, trace_cap), c->trace_cap);
  if (trace_out && nt > 0)
    CUDA_TRY(c, cudaMemcpyAsync(trace_out, c->trace, nt * sizeof(bild_trace_rec), cudaMemcpyDeviceToHost, c->stream));
  if (stats) *stats = s.stats;
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return BILD_OK;
}

int bild_generate(bild_ctx* c, int mode, float alpha_fb, float alpha_rb, int max_len, int32_t* tokens_out,
                  int* n_tokens, bild_trace_rec* trace_out, int trace_cap, int* n_trace, bild_stats* stats) {
  if (!c || !tokens_out || !n_tokens) return fail(c, BILD_ERR_ARG, "null argument");
  int rc = bild_generate_async(c, mode, alpha_fb, alpha_rb, max_len);
  if (rc) return rc;
  return bild_fetch_result(c, tokens_out, n_tokens, trace_out, trace_cap, n_trace, stats);
}

int bild_op_linear(const void* W, int w_dtype, const float* X, const float* gain, float eps, float* Y, int M, int N,
                   int K, void* cuda_stream) {
  if (!W || !X || !Y || M < 1 || M > MAXB || N < 1 || K < 8 || K % 8) return BILD_ERR_ARG;
  if (w_dtype != BILD_FP32 && w_dtype != BILD_BF16) return BILD_ERR_ARG;
  bild_ctx tmp;
  tmp.stream = (cudaStream_t)cuda_stream;
  LinArgs a{};
  a.W0 = W; a.X = X; a.ldx = K; a.gain = gain; a.eps = eps; a.Y = Y; a.ldy = N; a.N = N; a.K = K; a.M = M;
  a.epi = EPI_STORE;
  cudaError_t e = launch_linear(&tmp, w_dtype, M == 1 ? 1 : MAXB, a);
  return e == cudaSuccess ? BILD_OK : BILD_ERR_CUDA;
}

size_t bild_op_lm_head_scratch_bytes(int V) {
  if (V < 1) return 0;
  return align_up(head_partial_count(V) * sizeof(Partial), 256) + 256 + align_up(sizeof(HeadOut), 256);
}

int bild_op_lm_head(const void* W, int w_dtype, const float* X, const float* gain, float eps, float scale,
                    const int32_t* target, int M, int V, int K, int32_t* argmax_out, float* max_out, float* lse_out,
                    float* gather_out, float* logits_dbg, void* scratch, void* cuda_stream) {
  if (!W || !X || !scratch || !argmax_out || !max_out || !lse_out) return BILD_ERR_ARG;
  if (M < 1 || M > MAXB || V < 1 || K < 8 || K % 8 || K > 4096) return BILD_ERR_ARG;
  if (w_dtype != BILD_FP32 && w_dtype != BILD_BF16) return BILD_ERR_ARG;
  if ((uintptr_t)scratch % 256) return BILD_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int grid = head_grid_for(V);
  char* p = (char*)scratch;
  HeadArgs h{};
  h.partials = (Partial*)p;
  p += align_up(head_partial_count(V) * sizeof(Partial), 256);
  h.counter = (unsigned*)p;
  p += 256;
  h.out = (HeadOut*)p;
  if (cudaMemsetAsync(h.counter, 0, sizeof(unsigned), s) != cudaSuccess) return BILD_ERR_CUDA;
  h.W = W; h.X = X; h.ldx = K; h.gain = gain; h.eps = eps; h.scale = scale; h.V = V; h.K = K; h.M = M;
  h.target = target; h.logits_dbg = logits_dbg; h.which = 1;
  {
    const cudaError_t le = launch_head(s, false, w_dtype, M == 1 ? 1 : MAXB, h, grid, nullptr);
    if (le == cudaErrorInvalidConfiguration) return BILD_ERR_CAPACITY;   // M >= 2: 16 rows of K floats exceed a block's shared memory
    if (le != cudaSuccess) return BILD_ERR_CUDA;
  }
  const HeadOut* o = h.out;
  cudaError_t e = cudaMemcpyAsync(argmax_out, o->argmax, M * sizeof(int), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(max_out, o->zmax, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(lse_out, o->lse, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess && gather_out && target)
    e = cudaMemcpyAsync(gather_out, o->gather, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  return e == cudaSuccess ? BILD_OK : BILD_ERR_CUDA;
}

// ---- single operations on the hot kernels of the decoder passes ---------------------------------
namespace {
struct OpScratch {          // carved from the caller's scratch, 256-byte aligned pieces
  CallDesc* desc; int* err; int* nkeys; float* zero; char* rest;
};
OpScratch op_scratch(void* scratch, int d) {
  char* p = (char*)scratch;
  OpScratch o;
  o.desc = (CallDesc*)p; p += align_up(sizeof(CallDesc), 256);
  o.err = (int*)p; o.nkeys = (int*)(p + 4); p += 256;
  o.zero = (float*)p; p += align_up((size_t)MAXB * d * sizeof(float), 256);
  o.rest = p;
  return o;
}
int op_sms() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}
int op_finish(cudaStream_t s, const OpScratch& o) {   // the kernels' own error flag (bounded waits) after the call
  int err = 0;
  if (cudaMemcpyAsync(&err, o.err, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess)
    return BILD_ERR_CUDA;
  return err;
}
}  // namespace

size_t bild_op_sublayer_scratch_bytes(int d, int F) {
  return align_up(sizeof(CallDesc), 256) + 256 + align_up((size_t)MAXB * std::max(d, 8) * sizeof(float), 256) +
         align_up((size_t)(std::max(F, 0) / 8) * d * 16, 256) + align_up((size_t)(std::max(F, 0) / 8) * pack_wfo_dpad(d) * 16, 256) + 256;
}

int bild_op_ffn_sublayer(const void* Wi0, const void* Wi1, const void* Wfo, const float* gain, float eps, const float* x_in,
                         float* x_out, int M, int d, int F, int parts, void* scratch, void* cuda_stream) {
  if (!Wi0 || !Wfo || !gain || !x_in || !x_out || !scratch) return BILD_ERR_ARG;
  if (M < 1 || M > SUB_MB || d < 16 || d % 16 || d > 1024 || F < 8 || F % 8 || parts < 0 || parts > 8) return BILD_ERR_ARG;
  if ((uintptr_t)scratch % 256) return BILD_ERR_WORKSPACE;
  const int sms = op_sms();
  if (sms < 1) return BILD_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const bool gated = Wi1 != nullptr;
  const int MB = M == 1 ? 1 : SUB_MB, nmat = gated ? 2 : 1;
  int smem_max = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return BILD_ERR_CUDA;
  int np = std::max(1, parts);
  while (np <= 8 && (ffn_sub_rows(F, sms * np) * nmat > SUB_MAX_ROWS || ffn_sub_rows(F, sms * np) > SUB_FO_REGS ||
                     ffn_sub_layout(d, F, gated, sms * np, sms, MB).total > smem_max)) ++np;
  if (np > 8) return BILD_ERR_CAPACITY;
  OpScratch o = op_scratch(scratch, d);
  uint4* wfo_one = (uint4*)o.rest;
  uint4* wfo_blk = (uint4*)(o.rest + align_up((size_t)(F / 8) * d * 16, 256));
  pack_wfo_kernel<<<F / 8, 256, 0, s>>>((const __nv_bfloat16*)Wfo, wfo_one, wfo_blk, d, F);
  bild_ctx tmp;
  tmp.stream = s;
  tmp.use_pdl = false;
  TokList t{};
  set_desc_at_kernel<<<1, 1, 0, s>>>(o.desc, M, 0, t);
  if (cudaMemsetAsync(o.err, 0, 8, s) != cudaSuccess) return BILD_ERR_CUDA;
  if (cudaMemsetAsync(x_out, 0, (size_t)M * d * sizeof(float), s) != cudaSuccess) return BILD_ERR_CUDA;   // the kernel accumulates into it
  auto kern = MB == 1 ? ffn_sub_kernel<true> : ffn_sub_kernel<false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess) return BILD_ERR_CUDA;
  FfnSubArgs f{};
  f.desc = o.desc; f.eps = eps; f.d = d; f.F = F; f.gated = gated ? 1 : 0; f.mb = MB; f.spin = SPIN_LIMIT; f.err = o.err;
  f.x_in = x_in; f.x_out = x_out; f.gain = gain; f.Wi0 = (const __nv_bfloat16*)Wi0; f.Wi1 = (const __nv_bfloat16*)Wi1; f.Wfo1 = wfo_one; f.Wfo8 = wfo_blk;
  f.nparts = np; f.L = ffn_sub_layout(d, F, gated, sms * np, sms, MB);
  for (int p = 0; p < np; ++p) {
    f.part = p; f.seed = p == 0 ? 1 : 0; f.x_zero = p == 0 ? o.zero : nullptr;
    if (launch_sub(&tmp, kern, sms, 1, (size_t)f.L.total, f) != cudaSuccess) return BILD_ERR_CUDA;
  }
  return op_finish(s, o);
}

int bild_op_attn_sublayer(int self, const void* Wp, const void* Wo, const float* gain, float eps, const float* x_in, float* x_out,
                          float* kc, float* vc, int cap, int n_before, const float* bias_by_dist, int M, int d, int H, int dkv,
                          void* scratch, void* cuda_stream) {
  if (!Wp || !Wo || !gain || !x_in || !x_out || !kc || !vc || !scratch || (self && !bias_by_dist)) return BILD_ERR_ARG;
  if (M < 1 || M > SUB_MB || H < 1 || cap < 1 || n_before < 0) return BILD_ERR_ARG;
  if (self ? n_before + M > cap : (n_before < 1 || n_before > cap)) return BILD_ERR_CAPACITY;
  if ((uintptr_t)scratch % 256) return BILD_ERR_WORKSPACE;
  const int sms = op_sms();
  if (sms < 1) return BILD_ERR_CUDA;
  int C = 8;
  while (C > 1 && (H * C > sms || d % (4 * C))) C >>= 1;
  if (d % (4 * C) || d > 1024 || d % 8 || dkv > 64 || dkv < 16 || (dkv & (dkv - 1)) || d / C > SUB_THREADS / 2 ||
      (3 * dkv + C - 1) / C > SUB_MAX_ROWS) return BILD_ERR_ARG;   // shapes the fused kernel does not take
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int MB = M == 1 ? 1 : SUB_MB, I = H * dkv, P = self ? 3 : 1;
  int smem_max = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return BILD_ERR_CUDA;
  const AttnSubPlan pl = attn_sub_plan(d, dkv, P, C, cap, 128, SUB_HALF_SM, smem_max, MB);
  if (!pl.ok) return BILD_ERR_CAPACITY;
  const int kc_keys = pl.kc, bias_len = pl.bias_len;
  OpScratch o = op_scratch(scratch, d);
  bild_ctx tmp;
  tmp.stream = s;
  tmp.use_pdl = false;
  TokList t{};
  set_desc_at_kernel<<<1, 1, 0, s>>>(o.desc, M, self ? n_before : 0, t);
  if (cudaMemsetAsync(o.err, 0, 4, s) != cudaSuccess) return BILD_ERR_CUDA;
  if (cudaMemcpyAsync(o.nkeys, &n_before, sizeof(int), cudaMemcpyHostToDevice, s) != cudaSuccess) return BILD_ERR_CUDA;
  if (cudaMemsetAsync(x_out, 0, (size_t)M * d * sizeof(float), s) != cudaSuccess) return BILD_ERR_CUDA;   // the kernel accumulates into it
  auto kern = MB == 1 ? attn_sub_kernel<true> : attn_sub_kernel<false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess) return BILD_ERR_CUDA;
  AttnSubArgs a{};
  a.desc = o.desc; a.eps = eps; a.d = d; a.I = I; a.H = H; a.dkv = dkv; a.dkv_shift = ilog2(dkv); a.C = C; a.c_shift = ilog2(C);
  a.kc_keys = kc_keys; a.bias_len = bias_len; a.red_keys = pl.red_keys; a.mb = MB; a.err = o.err; a.spin = SPIN_LIMIT; a.skip_copies = 0;
  a.n_keys_dev = o.nkeys; a.x_in = x_in; a.x_out = x_out; a.x_zero = o.zero; a.gain = gain;
  a.Wp = (const __nv_bfloat16*)Wp; a.Wo = (const __nv_bfloat16*)Wo; a.kc = kc; a.vc = vc; a.cap = cap;
  a.bias = bias_by_dist; a.bias_ld = cap; a.self = self ? 1 : 0;
  a.L = attn_sub_layout(d, dkv, P, C, MB, kc_keys, bias_len);
  if (launch_sub(&tmp, kern, H * C, C, (size_t)a.L.total, a) != cudaSuccess) return BILD_ERR_CUDA;
  return op_finish(s, o);
}

int bild_op_lm_head_sliced(const void* W, const float* X, const float* gain, float eps, float scale, const int32_t* target, int M,
                           int V, int K, int32_t* argmax_out, float* max_out, float* lse_out, float* gather_out, float* logits_dbg,
                           void* scratch, void* cuda_stream) {
  if (!W || !X || !scratch || !argmax_out || !max_out || !lse_out) return BILD_ERR_ARG;
  if (M < 1 || M > MAXB || V < 1 || K < 8 || K % 8 || ((uintptr_t)W & 15)) return BILD_ERR_ARG;
  if ((uintptr_t)scratch % 256) return BILD_ERR_WORKSPACE;
  const int sms = op_sms();
  if (sms < 1 || sms > MAX_GRID_SM) return BILD_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int tr = (M == 1 && K <= 512) ? 32 : 16;
  const size_t smem = slice_head_smem_bytes(K, tr);
  if (smem > 200 * 1024) return BILD_ERR_CAPACITY;
  char* p = (char*)scratch;
  HeadArgs h{};
  h.partials = (Partial*)p;
  p += align_up(head_partial_count(V) * sizeof(Partial), 256);
  h.counter = (unsigned*)p;
  int* err = (int*)(p + 8);
  p += 256;
  h.out = (HeadOut*)p;
  if (cudaMemsetAsync(h.counter, 0, 16, s) != cudaSuccess) return BILD_ERR_CUDA;
  h.W = W; h.X = X; h.ldx = K; h.gain = gain; h.eps = eps; h.scale = scale; h.V = V; h.K = K; h.M = M;
  h.target = target; h.logits_dbg = logits_dbg; h.which = 1;
  if (cudaFuncSetAttribute(slice_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) return BILD_ERR_CUDA;
  slice_head_kernel<<<sms, SH_THREADS, smem, s>>>(h, err, tr);
  if (cudaGetLastError() != cudaSuccess) return BILD_ERR_CUDA;
  const HeadOut* o = h.out;
  cudaError_t e = cudaMemcpyAsync(argmax_out, o->argmax, M * sizeof(int), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(max_out, o->zmax, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(lse_out, o->lse, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess && gather_out && target) e = cudaMemcpyAsync(gather_out, o->gather, M * sizeof(float), cudaMemcpyDeviceToDevice, s);
  return e == cudaSuccess ? BILD_OK : BILD_ERR_CUDA;
}

int bild_op_lm_head_stream(const void* W, const float* X, const float* gain, float eps, float scale, const int32_t* target, int V,
                           int K, int32_t* argmax_out, float* max_out, float* lse_out, float* gather_out, float* logits_dbg,
                           void* scratch, void* cuda_stream) {
  if (!W || !X || !scratch || !argmax_out || !max_out || !lse_out) return BILD_ERR_ARG;
  if (V < 1 || K < 8 || K % 8 || ((uintptr_t)W & 15)) return BILD_ERR_ARG;
  if (K > 1024) return BILD_ERR_CAPACITY;
  if ((uintptr_t)scratch % 256) return BILD_ERR_WORKSPACE;
  const int sms = op_sms();
  if (sms < 1) return BILD_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  char* p = (char*)scratch;
  HeadArgs h{};
  h.partials = (Partial*)p;
  p += align_up(head_partial_count(V) * sizeof(Partial), 256);
  h.counter = (unsigned*)p;
  p += 256;
  h.out = (HeadOut*)p;
  if (cudaMemsetAsync(h.counter, 0, 16, s) != cudaSuccess) return BILD_ERR_CUDA;
  h.W = W; h.X = X; h.ldx = K; h.gain = gain; h.eps = eps; h.scale = scale; h.V = V; h.K = K; h.M = 1;
  h.target = target; h.logits_dbg = logits_dbg; h.which = 1;
  bild_ctx tmp;
  tmp.stream = s;
  tmp.use_pdl = false;
  if (launch_head_stream(&tmp, h, sms) != cudaSuccess) return BILD_ERR_CUDA;
  const HeadOut* o = h.out;
  cudaError_t e = cudaMemcpyAsync(argmax_out, o->argmax, sizeof(int), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(max_out, o->zmax, sizeof(float), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(lse_out, o->lse, sizeof(float), cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess && gather_out && target) e = cudaMemcpyAsync(gather_out, o->gather, sizeof(float), cudaMemcpyDeviceToDevice, s);
  return e == cudaSuccess ? BILD_OK : BILD_ERR_CUDA;
}

int bild_time_pass(bild_ctx* c, int which, int k, int cache_len, int iters, float* ms_per_pass) {
  if (!c || !ms_per_pass || (which != 0 && which != 1)) return fail(c, BILD_ERR_ARG, "null argument / which");
  if (!c->encoded) return fail(c, BILD_ERR_STATE, "bild_encode has not been called");
  const bool cold = iters < 0;   // no untimed first pass: the caches hold whatever ran before
  if (cold) iters = -iters;
  if (k < 1 || k > (which == 0 ? 1 : MAXB) || iters < 1) return fail(c, BILD_ERR_ARG, "k or iters out of range");
  if (cache_len < 0 || cache_len + k > c->cfg.max_dec_len) return fail(c, BILD_ERR_CAPACITY, "cache_len + k > max_dec_len");
  TokList t{};
  for (int i = 0; i < k; ++i) t.t[i] = (7 * i + 3) % c->m[which].c.vocab;
  cudaEvent_t e0, e1;
  CUDA_TRY(c, cudaEventCreate(&e0));
  CUDA_TRY(c, cudaEventCreate(&e1));
  int rc = BILD_OK;
  set_desc_at_kernel<<<1, 1, 0, c->stream>>>(c->m[which].desc, k, cache_len, t);
  (*c->cnt)++;
  // the pass as a CUDA graph (as the decode loop runs it), replayed `iters` times
  cudaGraph_t g = nullptr;
  cudaGraphExec_t ex = nullptr;
  if (cudaGraphCreate(&g, 0) != cudaSuccess) rc = BILD_ERR_CUDA;
  int64_t n_launch = 0;
  if (rc == BILD_OK) rc = capture_pass(c, g, which, k == 1 ? 1 : k <= SUB_MB ? SUB_MB : MAXB, 0, 0, nullptr, &n_launch);
  if (rc == BILD_OK && cudaGraphInstantiate(&ex, g, 0) != cudaSuccess) rc = BILD_ERR_CUDA;
  if (rc == BILD_OK && cudaGraphUpload(ex, c->stream) != cudaSuccess) rc = BILD_ERR_CUDA;
  if (rc == BILD_OK && !cold && cudaGraphLaunch(ex, c->stream) != cudaSuccess) rc = BILD_ERR_CUDA;  // untimed first pass
  if (rc == BILD_OK && cudaEventRecord(e0, c->stream) != cudaSuccess) rc = BILD_ERR_CUDA;
  for (int it = 0; it < iters && rc == BILD_OK; ++it)
    if (cudaGraphLaunch(ex, c->stream) != cudaSuccess) rc = BILD_ERR_CUDA;
  if (rc == BILD_OK && cudaEventRecord(e1, c->stream) != cudaSuccess) rc = BILD_ERR_CUDA;
  if (rc == BILD_OK && cudaEventSynchronize(e1) != cudaSuccess) rc = BILD_ERR_CUDA;
  if (rc == BILD_OK) c->launches += n_launch * (iters + (cold ? 0 : 1));
  if (ex) cudaGraphExecDestroy(ex);
  if (g) cudaGraphDestroy(g);
  float ms = 0.f;
  if (rc == BILD_OK && cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) rc = BILD_ERR_CUDA;
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (rc != BILD_OK) return fail(c, rc, "bild_time_pass failed");
  *ms_per_pass = ms / (float)iters;
  return BILD_OK;
}

#ifdef BILD_STAMPS
// Cycle stamps of the fused sub-layer kernels (debug builds only): 4 x 16 counters, optionally cleared.
int bild_debug_stamps(unsigned long long* out, int reset) {
  if (out && cudaMemcpyFromSymbol(out, g_sub_stamps, sizeof(g_sub_stamps)) != cudaSuccess) return BILD_ERR_CUDA;
  if (reset) {
    static unsigned long long zero[3][4][24];
    if (cudaMemcpyToSymbol(g_sub_stamps, zero, sizeof(zero)) != cudaSuccess) return BILD_ERR_CUDA;
  }
  return BILD_OK;
}
// Cycle stamps of the encoder GEMM (debug builds only): 3 x 16 counters, optionally cleared.
int bild_debug_gemm_stamps(unsigned long long* out, int reset) {
  if (out && cudaMemcpyFromSymbol(out, g_eg_stamps, sizeof(g_eg_stamps)) != cudaSuccess) return BILD_ERR_CUDA;
  if (reset) {
    static unsigned long long zero[3][16];
    if (cudaMemcpyToSymbol(g_eg_stamps, zero, sizeof(zero)) != cudaSuccess) return BILD_ERR_CUDA;
  }
  return BILD_OK;
}
#endif

// Test helper: copies one layer's cached keys or values to the host (synchronises the stream).
// what: 0 cross keys, 1 cross values, 2 self keys, 3 self values; layout [n_heads][capacity][d_kv] fp32,
// capacity = max_enc_len (cross) or max_dec_len (self); dst holds n_heads * capacity * d_kv floats.
int bild_debug_read_cache(bild_ctx* c, int which, int what, int layer, float* dst_host, size_t count) {
  if (!c || !dst_host || (which != 0 && which != 1) || what < 0 || what > 3) return fail(c, BILD_ERR_ARG, "null argument / which / what");
  Model& m = c->m[which];
  if (layer < 0 || layer >= m.c.n_layers) return fail(c, BILD_ERR_ARG, "layer out of range");
  const size_t cap = what < 2 ? c->cfg.max_enc_len : c->cfg.max_dec_len;
  const size_t n = (size_t)m.c.n_heads * cap * m.c.d_kv;
  if (count != n) return fail(c, BILD_ERR_ARG, "count must be n_heads * capacity * d_kv");
  const float* base = what == 0 ? m.crossK : what == 1 ? m.crossV : what == 2 ? m.selfK : m.selfV;
  CUDA_TRY(c, cudaMemcpyAsync(dst_host, base + (size_t)layer * n, n * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return BILD_OK;
}

// Host-only helper for tests of the bucket tables: which = 0 decoder (delta = query - key >= 0),
// 1 encoder (rel = key - query).
int bild_debug_bucket(int which, int rel, int n_buckets, int max_dist) {
  if (n_buckets < 4 || n_buckets % 4 || max_dist < n_buckets) return -1;
  if (which == 0) return rel < 0 ? -1 : decoder_bucket(rel, n_buckets, max_dist);
  return encoder_bucket(rel, n_buckets, max_dist);
}

}  // extern "C"
