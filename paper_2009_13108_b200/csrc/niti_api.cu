// C-ABI entry points of the NITI library: argument checks, engine selection, and the
// accumulate -> bit-width -> shift-and-round sequence of Algorithm 1 for each layer op.
#include "niti_common.cuh"

int niti_launch_im2col32(niti_ctx *ctx, cudaStream_t st, const int8_t *x, int8_t *xcol, int B, int H, int W,
                         int Ci, int R, int S, int pad, int stride, int Ho, int Wo);
int niti_launch_pad_pitch(niti_ctx *ctx, cudaStream_t st, const int8_t *src, int8_t *dst, int rows, int n, int pitch);
int niti_launch_pad_rows32(niti_ctx *ctx, cudaStream_t st, const int8_t *w, int8_t *wcol, int rows, int k);
int niti_launch_round_compact32(niti_ctx *ctx, cudaStream_t st, const int32_t *acc, const WsHeader *hdr, int8_t *out,
                                int rows, int k, int mbits, int round_mode, int32_t *b_out);

// Few-channel convolutions (R*S*Cin <= 32 and Cin not a multiple of 16, i.e. no TMA view of the
// NHWC tensor): gathered into K = 32 rows and run as a plain matrix multiply.
static inline bool few_channel_conv(int Ci, int R, int S) { return R * S * Ci <= 32 && (Ci % 16) != 0; }
static inline size_t round_up(size_t v, size_t a);

extern "C" int niti_create(niti_ctx **out, int device) {
  if (!out) return NITI_ERR_ARG;
  *out = nullptr;
  niti_ctx *ctx = new niti_ctx();
  memset(ctx, 0, sizeof(*ctx));
  ctx->device = device;
  cudaDeviceProp prop;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, device);
  if (e != cudaSuccess) {
    delete ctx;
    return NITI_ERR_CUDA;
  }
  if (prop.major != 10) {   // the kernels are built for sm_100a only
    delete ctx;
    return NITI_ERR_SHAPE;
  }
  ctx->sm_count = prop.multiProcessorCount;
  ctx->smem_optin = prop.sharedMemPerBlockOptin;
  // one allocation: the status words, then the table of speculative-estimate errors
  const size_t dev_bytes = 256 + sizeof(int32_t) * 2 * NITI_SPEC_SLOTS;
  e = cudaMalloc(&ctx->d_status, dev_bytes);
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, dev_bytes);
  if (e != cudaSuccess) {
    delete ctx;
    return NITI_ERR_CUDA;
  }
  ctx->d_spec_tab = (int32_t *)((char *)ctx->d_status + 256);
  cudaDriverEntryPointQueryResult qres;
  void *fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess)
    ctx->encode_tiled = fn;
  *out = ctx;
  return NITI_OK;
}

extern "C" int niti_destroy(niti_ctx *ctx) {
  if (!ctx) return NITI_ERR_ARG;
  if (ctx->prof_ev) {
    for (int i = 0; i < 2 * NITI_PROF_MAX; ++i) cudaEventDestroy(ctx->prof_ev[i]);
    delete[] ctx->prof_ev;
    delete[] ctx->prof_ops;
  }
  cudaFree(ctx->d_status);
  delete ctx;
  return NITI_OK;
}

extern "C" const char *niti_last_error(niti_ctx *ctx) { return ctx ? ctx->err : "null context"; }

extern "C" int niti_set_engine(niti_ctx *ctx, int engine) {
  if (!ctx) return -1;
  int old = ctx->engine;
  ctx->engine = engine;
  return old;
}

extern "C" int niti_set_reduce_hook(niti_ctx *ctx, niti_reduce_fn fn, void *user) {
  if (!ctx) return NITI_ERR_ARG;
  ctx->reduce_fn = fn;
  ctx->reduce_user = fn ? user : nullptr;
  return NITI_OK;
}

extern "C" int niti_begin_step(niti_ctx *ctx, void *stream, void *ws, size_t ws_bytes) {
  if (!ctx) return NITI_ERR_ARG;
  if (!ws) {                                     // forget the prepared workspace: calls clear their header again
    ctx->step_ws = nullptr;
    ctx->step_slot = 0;
    return NITI_OK;
  }
  if (((uintptr_t)ws & 255) || ws_bytes < NITI_WS_HEADER)
    return niti_fail(ctx, NITI_ERR_WORKSPACE, "niti_begin_step: workspace misaligned or too small");
  NITI_CUDA_TRY(ctx, cudaMemsetAsync(ws, 0, NITI_WS_HEADER, (cudaStream_t)stream));
  ctx->launches++;
  ctx->step_ws = ws;
  ctx->step_slot = 0;
  return NITI_OK;
}

extern "C" int niti_set_tap_cache(niti_ctx *ctx, void *buf, size_t bytes) {
  if (!ctx || (buf && (((uintptr_t)buf & 255) || bytes == 0))) return NITI_ERR_ARG;
  ctx->tap_buf = (int8_t *)buf;
  ctx->tap_bytes = buf ? bytes : 0;
  ctx->tap_x = nullptr;
  ctx->tap_dims[8] = 0;
  return NITI_OK;
}

// Does the tap cache hold the gathered rows of exactly this input tensor and geometry?
static bool tap_cache_hit(const niti_ctx *ctx, const void *x, int B, int H, int W, int Ci, int R, int S, int pad,
                          int stride) {
  const int want[8] = {B, H, W, Ci, R, S, pad, stride};
  if (!ctx->tap_buf || !ctx->tap_dims[8] || ctx->tap_x != x) return false;
  for (int i = 0; i < 8; ++i)
    if (ctx->tap_dims[i] != want[i]) return false;
  return true;
}

extern "C" int niti_set_dp_shard(niti_ctx *ctx, int rank, int world) {
  if (!ctx || world < 1 || rank < 0 || rank >= world) return NITI_ERR_ARG;
  ctx->dp_rank = rank;
  ctx->dp_world = world;
  return NITI_OK;
}

extern "C" uint64_t niti_launch_count(niti_ctx *ctx) { return ctx ? ctx->launches : 0; }
extern "C" uint64_t niti_tc_launch_count(niti_ctx *ctx) { return ctx ? ctx->tc_launches : 0; }
extern "C" uint64_t niti_tc_pair_launch_count(niti_ctx *ctx) { return ctx ? ctx->tc2_launches : 0; }

extern "C" int64_t niti_redo_count(niti_ctx *ctx, void *stream) {
  if (!ctx) return -1;
  uint32_t h = 0;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return -1;
  if (cudaMemcpy(&h, ctx->d_status + 1, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  return (int64_t)h;
}

int niti_tc_timeout_probe(niti_ctx *ctx, cudaStream_t st);
extern "C" int niti_selftest_timeout(niti_ctx *ctx, void *stream) {
  if (!ctx) return NITI_ERR_ARG;
  return niti_tc_timeout_probe(ctx, (cudaStream_t)stream);
}

extern "C" int niti_profile_enable(niti_ctx *ctx, int on) {
  if (!ctx) return NITI_ERR_ARG;
  if (on && !ctx->prof_ev) {
    ctx->prof_ev = new cudaEvent_t[2 * NITI_PROF_MAX];
    ctx->prof_ops = new double[NITI_PROF_MAX];
    for (int i = 0; i < 2 * NITI_PROF_MAX; ++i) NITI_CUDA_TRY(ctx, cudaEventCreate(&ctx->prof_ev[i]));
  }
  ctx->profile_on = on ? 1 : 0;
  ctx->prof_used = 0;
  return NITI_OK;
}

extern "C" int niti_profile_read_launches(niti_ctx *ctx, double *ms, double *ops, int max_n) {
  if (!ctx || !ms || !ops || max_n < 0) return -1;
  int n = ctx->prof_used < max_n ? ctx->prof_used : max_n;
  for (int i = 0; i < n; ++i) {
    float t = 0;
    if (cudaEventSynchronize(ctx->prof_ev[2 * i + 1]) != cudaSuccess) return -1;
    if (cudaEventElapsedTime(&t, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]) != cudaSuccess) return -1;
    ms[i] = t;
    ops[i] = ctx->prof_ops[i];
  }
  return n;
}

extern "C" int niti_profile_read(niti_ctx *ctx, double *tc_ms, uint64_t *tc_launches, double *tc_ops) {
  if (!ctx || !tc_ms || !tc_launches || !tc_ops) return NITI_ERR_ARG;
  double ms = 0, ops = 0;
  for (int i = 0; i < ctx->prof_used; ++i) {
    float t = 0;
    NITI_CUDA_TRY(ctx, cudaEventSynchronize(ctx->prof_ev[2 * i + 1]));
    NITI_CUDA_TRY(ctx, cudaEventElapsedTime(&t, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]));
    ms += t;
    ops += ctx->prof_ops[i];
  }
  *tc_ms = ms;
  *tc_launches = (uint64_t)ctx->prof_used;
  *tc_ops = ops;
  ctx->prof_used = 0;
  return NITI_OK;
}

extern "C" int niti_check(niti_ctx *ctx, void *stream, uint32_t *status) {
  if (!ctx) return NITI_ERR_ARG;
  uint32_t h = 0;
  NITI_CUDA_TRY(ctx, cudaStreamSynchronize((cudaStream_t)stream));
  NITI_CUDA_TRY(ctx, cudaMemcpy(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost));
  if (h) NITI_CUDA_TRY(ctx, cudaMemset(ctx->d_status, 0, sizeof(h)));
  if (status) *status = h;
  if (h) {
    snprintf(ctx->err, sizeof(ctx->err), "device status word 0x%x", h);
    return NITI_ERR_DEVICE;
  }
  return NITI_OK;
}

static inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }


static bool fill_conv(GemmProblem &p, int kind, int B, int H, int W, int Ci, int Co, int R, int S,
                      int pad, int stride = 1) {
  p.kind = kind;
  p.B = B; p.H = H; p.W = W; p.Ci = Ci; p.Co = Co; p.R = R; p.S = S; p.pad = pad; p.stride = stride;
  if (stride < 1 || H + 2 * pad < R || W + 2 * pad < S) return false;
  p.Ho = (H + 2 * pad - R) / stride + 1;
  p.Wo = (W + 2 * pad - S) / stride + 1;
  if (p.Ho <= 0 || p.Wo <= 0) return false;
  if (kind == GK_CONV_FWD) { p.gm = (long long)B * p.Ho * p.Wo; p.gn = Co; p.gk = (long long)R * S * Ci; }
  else if (kind == GK_CONV_DGRAD) { p.gm = (long long)B * H * W; p.gn = Ci; p.gk = (long long)R * S * Co; }
  else { p.gm = Co; p.gn = (long long)R * S * Ci; p.gk = (long long)B * p.Ho * p.Wo; }
  return true;
}

// int32 elements of the accumulator scratch of a fully connected backward call: the larger of the weight
// gradient [N][K] and the error [M][K] (times its partial slices when the batch is small)
static size_t linear_bwd_acc_elems(long long M, long long N, long long K) {
  const size_t a = (size_t)(M * K) * (size_t)niti_partial_slices(GK_FC_DGRAD, M), b = (size_t)(N * K);
  return a > b ? a : b;
}

static void fill_fc(GemmProblem &p, int kind, int M, int N, int K) {
  memset(&p, 0, sizeof(p));
  p.kind = kind; p.M = M; p.N = N; p.K = K;
  if (kind == GK_FC_FWD) { p.gm = M; p.gn = N; p.gk = K; }
  else if (kind == GK_FC_DGRAD) { p.gm = M; p.gn = K; p.gk = N; }
  else { p.gm = N; p.gn = K; p.gk = M; }
}

extern "C" size_t niti_workspace_bytes(int op, const int64_t *d, int nd) {
  if (!d) return 0;
  GemmProblem p, p2;
  memset(&p, 0, sizeof(p));
  memset(&p2, 0, sizeof(p2));
  size_t outs = 0, extra = 0;
  switch (op) {
    case NITI_OP_LINEAR_FWD:
      if (nd != 3 || d[0] <= 0 || d[1] <= 0 || d[2] <= 0) return 0;
      fill_fc(p, GK_FC_FWD, (int)d[0], (int)d[1], (int)d[2]);
      outs = (size_t)(d[0] * d[1]) * (size_t)niti_partial_slices(GK_FC_FWD, d[0]);
      extra = niti_tc_scratch_bytes(p);
      break;
    case NITI_OP_LINEAR_BWD_UPDATE:
    case NITI_OP_LINEAR_BWD: {
      if (nd != 3 || d[0] <= 0 || d[1] <= 0 || d[2] <= 0) return 0;
      size_t b = (size_t)(d[1] * d[2]);
      outs = linear_bwd_acc_elems(d[0], d[1], d[2]);
      fill_fc(p, GK_FC_DGRAD, (int)d[0], (int)d[1], (int)d[2]);
      fill_fc(p2, GK_FC_WGRAD, (int)d[0], (int)d[1], (int)d[2]);
      size_t e1 = niti_tc_scratch_bytes(p), e2 = niti_tc_scratch_bytes(p2);
      extra = e1 > e2 ? e1 : e2;
      if (d[1] % 16) extra += round_up((size_t)d[0] * (size_t)((d[1] + 15) / 16 * 16), 256);   // e with padded rows
      if (op == NITI_OP_LINEAR_BWD_UPDATE) extra = round_up(extra, 256) + round_up(b, 256);    // scratch gradient
      break;
    }
    case NITI_OP_CONV_FWD:
    case NITI_OP_CONV_DGRAD:
    case NITI_OP_CONV_WGRAD_UPDATE:
    case NITI_OP_CONV_WGRAD: {
      if (nd != 8 && nd != 9) return 0;                  // a ninth entry is the stride (default 1)
      for (int i = 0; i < 7; ++i)
        if (d[i] <= 0) return 0;
      const int stride = nd == 9 ? (int)d[8] : 1;
      const bool upd = op == NITI_OP_CONV_WGRAD_UPDATE;
      if (upd) op = NITI_OP_CONV_WGRAD;
      int kind = op == NITI_OP_CONV_FWD ? GK_CONV_FWD : (op == NITI_OP_CONV_DGRAD ? GK_CONV_DGRAD : GK_CONV_WGRAD);
      if (!fill_conv(p, kind, (int)d[0], (int)d[1], (int)d[2], (int)d[3], (int)d[4], (int)d[5], (int)d[6], (int)d[7],
                     stride))
        return 0;
      outs = (size_t)(p.gm * p.gn);
      extra = niti_tc_scratch_bytes(p);
      if (few_channel_conv((int)d[3], (int)d[5], (int)d[6]) && op != NITI_OP_CONV_DGRAD) {
        const size_t M = (size_t)d[0] * p.Ho * p.Wo;
        extra += round_up(M * 32, 256) + round_up((size_t)d[4] * 32, 256) + round_up((size_t)d[4] * 32 * 4, 256);
        if (op == NITI_OP_CONV_FWD && outs < M * (size_t)d[4]) outs = M * (size_t)d[4];
      }
      if (upd) extra = round_up(extra, 256) + round_up((size_t)(p.gm * p.gn), 256);             // scratch gradient
      break;
    }
    case NITI_OP_INT_XENT:
      if (nd != 2 || d[0] <= 0 || d[1] <= 0) return 0;
      // two 64-bit scalars per sample + the tables of many-row calls (256 x 256 x (2 + 1) + 256 bytes)
      return NITI_WS_HEADER + round_up((size_t)d[0] * 16, 256) + 196864;
    default:
      return 0;
  }
  return NITI_WS_HEADER + round_up(outs * 4, 256) + round_up(extra, 256);
}

static inline bool misaligned16(const void *p) { return ((uintptr_t)p & 15) != 0; }

int niti_launch_sgd_update(niti_ctx *ctx, cudaStream_t st, int8_t *w, const int8_t *g, long long n);

// Data parallelism (niti_set_reduce_hook), after a multiply has left its int32 accumulators in acc and
// their max magnitude in the header: a weight gradient is summed over the ranks and its max taken
// again from the sums; any other tensor only shares the max.
int niti_reduce_after_gemm(niti_ctx *ctx, cudaStream_t st, int kind, int32_t *acc, long long n, WsHeader *hdr,
                           bool shard_ok) {
  if (!ctx->reduce_fn) return NITI_OK;
  if (!niti_is_wgrad(kind)) return niti_reduce(ctx, st, &hdr->maxabs32, 1, NITI_REDUCE_MAX_U32);
  if (shard_ok && niti_dp_sharded(ctx, kind)) {
    // Sharded (Section 3.3's update distributed over the ranks): every rank receives the sums of its own
    // shard only (reduce-scatter, 4 bytes per weight on the wire), the few elements that do not divide
    // evenly are all-reduced, each rank takes the max over what it holds and the maxima are combined.
    // The caller then rounds its shard and all-gathers the int8 result (1 byte per weight).
    const NitiDpShard sh = niti_dp_shard(ctx, n);
    int rc = NITI_OK;
    if (sh.main > 0) rc = niti_reduce(ctx, st, acc, sh.main, NITI_REDUCE_SCATTER_SUM_I32);
    if (rc == NITI_OK && n > sh.main) rc = niti_reduce(ctx, st, acc + sh.main, n - sh.main, NITI_REDUCE_SUM_I32);
    if (rc != NITI_OK) return rc;
    NITI_CUDA_TRY(ctx, cudaMemsetAsync(&hdr->maxabs32, 0, sizeof(unsigned int), st));
    ctx->launches++;
    if (sh.shard > 0) rc = niti_launch_maxabs(ctx, st, acc + sh.off, sh.shard, hdr);
    if (rc == NITI_OK && n > sh.main) rc = niti_launch_maxabs(ctx, st, acc + sh.main, n - sh.main, hdr);
    if (rc != NITI_OK) return rc;
    return niti_reduce(ctx, st, &hdr->maxabs32, 1, NITI_REDUCE_MAX_U32);
  }
  int rc = niti_reduce(ctx, st, acc, n, NITI_REDUCE_SUM_I32);
  if (rc != NITI_OK) return rc;
  NITI_CUDA_TRY(ctx, cudaMemsetAsync(&hdr->maxabs32, 0, sizeof(unsigned int), st));
  ctx->launches++;
  return niti_launch_maxabs(ctx, st, acc, n, hdr);
}

// One matrix multiply of Algorithm 1 followed by EffectiveBitwidth + ShiftAndRound.
// update_w != null (weight gradients): the rounded gradient is not returned but subtracted from the
// weights in place.  When the int32 accumulators exist (split contractions) the rounding pass does
// that itself and the int8 gradient is never stored; when the multiply rounds in its own epilogue,
// `out` is a scratch tensor and the plain update kernel follows.
int niti_launch_maxpool2_fwd(niti_ctx *ctx, cudaStream_t st, const int8_t *x, int8_t *y, int B, int H, int W, int C);

static int run_gemm_round(niti_ctx *ctx, cudaStream_t st, const GemmProblem &p, void *ws, size_t ws_bytes,
                          size_t need, int8_t *out, int mbits, int round_mode, int relu,
                          const int8_t *mask, const int32_t *s_a, const int32_t *s_w, int32_t *s_out,
                          int32_t *b_out, int8_t *update_w = nullptr, int8_t *pool_out = nullptr) {
  if (!ws || ((uintptr_t)ws & 255) || ws_bytes < need)
    return niti_fail(ctx, NITI_ERR_WORKSPACE, "workspace missing, misaligned or too small");
  WsHeader *hdr = nullptr;
  int32_t *acc = (int32_t *)((char *)ws + NITI_WS_HEADER);
  int rc = niti_take_header(ctx, st, ws, &hdr);                            // zeroed reduction scalars and split maxima
  if (rc != NITI_OK) return rc;
  rc = NITI_ERR_SHAPE;
  bool fused = false;
  bool pooled = false;
  bool updated = false;
  RoundSpec rs = {out, mask, mbits, round_mode, relu, s_a, s_w, s_out, b_out, pool_out, update_w};
  if (ctx->engine != 1) rc = niti_tc_gemm(ctx, st, p, rs, acc, hdr, &fused, &pooled, true, &updated);
  if (rc == NITI_ERR_SHAPE) {
    rc = niti_simt_gemm(ctx, st, p, acc, hdr);
    if (rc == NITI_OK) rc = niti_reduce_after_gemm(ctx, st, p.kind, acc, p.gm * p.gn, hdr, true);
  }
  if (rc != NITI_OK) return rc;
  if (fused) {
    if (update_w && !updated) return niti_launch_sgd_update(ctx, st, update_w, out, p.gm * p.gn);
  } else if (niti_dp_sharded(ctx, p.kind)) {
    // sharded weight gradient: acc holds the sums over the ranks for this rank's shard (and the
    // remainder): round those (into the gradient, or straight into the weights), then every rank
    // collects the other shards' int8 results
    const long long n = p.gm * p.gn;
    const NitiDpShard sh = niti_dp_shard(ctx, n);
    int8_t *dst = update_w ? update_w : out;
    if (sh.shard > 0)
      rc = niti_launch_round(ctx, st, acc + sh.off, hdr, out + sh.off, sh.shard, mbits, round_mode, relu, nullptr,
                             s_a, s_w, s_out, b_out, update_w ? update_w + sh.off : nullptr);
    if (rc == NITI_OK && n > sh.main)
      rc = niti_launch_round(ctx, st, acc + sh.main, hdr, out + sh.main, n - sh.main, mbits, round_mode, relu, nullptr,
                             s_a, s_w, s_out, b_out, update_w ? update_w + sh.main : nullptr);
    if (rc == NITI_OK && sh.main > 0) rc = niti_reduce(ctx, st, dst, sh.main, NITI_ALLGATHER_I8);
    if (rc != NITI_OK) return rc;
  } else {
    rc = niti_launch_round(ctx, st, acc, hdr, out, p.gm * p.gn, mbits, round_mode, relu, mask, s_a, s_w,
                           s_out, b_out, update_w);
    if (rc != NITI_OK) return rc;
  }
  // the pooled copy of a forward convolution, where the multiply's own epilogue did not write it
  if (pool_out && !pooled) return niti_launch_maxpool2_fwd(ctx, st, out, pool_out, p.B, p.Ho, p.Wo, p.Co);
  return NITI_OK;
}

extern "C" int niti_linear_fwd(niti_ctx *ctx, void *stream, const int8_t *a, const int32_t *s_a,
                               const int8_t *w, const int32_t *s_w, int8_t *out, int32_t *s_out,
                               int32_t *b_out, int M, int N, int K, int relu, int round_mode, void *ws,
                               size_t ws_bytes) {
  if (!ctx) return NITI_ERR_ARG;
  if (!a || !w || !out || !s_a || !s_w || M <= 0 || N <= 0 || K <= 0 || (round_mode != 0 && round_mode != 1) ||
      misaligned16(a) || misaligned16(w) || misaligned16(out))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_linear_fwd: bad argument (pointers must be 16-byte aligned)");
  GemmProblem p;
  fill_fc(p, GK_FC_FWD, M, N, K);
  p.p0 = a; p.p1 = w;
  int64_t dims[3] = {M, N, K};
  return run_gemm_round(ctx, (cudaStream_t)stream, p, ws, ws_bytes,
                        niti_workspace_bytes(NITI_OP_LINEAR_FWD, dims, 3), out, 7, round_mode, relu,
                        nullptr, s_a, s_w, s_out, b_out);
}

// Backward pass of a fully connected layer; `g` receives the rounded weight gradient, or, with
// update_w, the gradient is subtracted from update_w (= w) in place after the error of the layer
// below has been computed from the old weights.
static int linear_bwd_impl(niti_ctx *ctx, void *stream, const int8_t *a, const int8_t *e, const int8_t *w,
                           int8_t *e_prev, const int8_t *relu_mask_src, int8_t *g, int8_t *update_w,
                           int32_t *b_e, int32_t *b_g, int M, int N, int K, int m_u, int round_mode, void *ws,
                           size_t ws_bytes, const char *who) {
  if (!ctx) return NITI_ERR_ARG;
  if (!a || !e || !w || (!g && !update_w) || M <= 0 || N <= 0 || K <= 0 || m_u < 1 || m_u > 7 ||
      (round_mode != 0 && round_mode != 1) || misaligned16(a) || misaligned16(e) || misaligned16(w) ||
      misaligned16(g) || misaligned16(e_prev) || misaligned16(relu_mask_src)) {
    snprintf(ctx->err, sizeof(ctx->err), "%s: bad argument (pointers must be 16-byte aligned)", who);
    return NITI_ERR_ARG;
  }
  int64_t dims[3] = {M, N, K};
  const size_t need_base = niti_workspace_bytes(NITI_OP_LINEAR_BWD, dims, 3);
  const size_t need = update_w ? niti_workspace_bytes(NITI_OP_LINEAR_BWD_UPDATE, dims, 3) : need_base;
  if (!ws || ((uintptr_t)ws & 255) || ws_bytes < need)
    return niti_fail(ctx, NITI_ERR_WORKSPACE, "workspace missing, misaligned or too small");
  if (update_w) g = (int8_t *)((char *)ws + need_base);       // scratch, used only if the multiply rounds by itself
  // TMA needs 16-byte row pitches: an error tensor with N % 16 != 0 (10 or 1000 classes) is copied
  // once into rows padded to the next multiple of 16 for the tensor-core engine
  const int8_t *e_tc = e;
  long long e_ld = 0;
  if ((N % 16) != 0 && N >= 32 && ctx->engine != 1) {
    const int pitch = (N + 15) / 16 * 16;
    int8_t *epad = (int8_t *)((char *)ws + NITI_WS_HEADER + round_up(linear_bwd_acc_elems(M, N, K) * 4, 256));
    int rcp = niti_launch_pad_pitch(ctx, (cudaStream_t)stream, e, epad, M, N, pitch);
    if (rcp != NITI_OK) return rcp;
    e_tc = epad;
    e_ld = pitch;
  }
  GemmProblem p;
  int rc;
  if (e_prev && update_w) {                // the error below needs the weights as they were
    fill_fc(p, GK_FC_DGRAD, M, N, K);
    p.p0 = e_tc; p.p1 = w; p.ld0 = e_ld;
    rc = run_gemm_round(ctx, (cudaStream_t)stream, p, ws, ws_bytes, need, e_prev, 7, round_mode, 0,
                        relu_mask_src, nullptr, nullptr, nullptr, b_e);
    if (rc != NITI_OK) return rc;
  }
  fill_fc(p, GK_FC_WGRAD, M, N, K);
  p.p0 = e_tc; p.p1 = a; p.ld0 = e_ld;
  rc = run_gemm_round(ctx, (cudaStream_t)stream, p, ws, ws_bytes, need, g, m_u, round_mode, 0, nullptr,
                      nullptr, nullptr, nullptr, b_g, update_w);
  if (rc != NITI_OK || !e_prev || update_w) return rc;
  fill_fc(p, GK_FC_DGRAD, M, N, K);
  p.p0 = e_tc; p.p1 = w; p.ld0 = e_ld;
  return run_gemm_round(ctx, (cudaStream_t)stream, p, ws, ws_bytes, need, e_prev, 7, round_mode, 0,
                        relu_mask_src, nullptr, nullptr, nullptr, b_e);
}

extern "C" int niti_linear_bwd(niti_ctx *ctx, void *stream, const int8_t *a, const int8_t *e,
                               const int8_t *w, int8_t *e_prev, const int8_t *relu_mask_src, int8_t *g,
                               int32_t *b_e, int32_t *b_g, int M, int N, int K, int m_u, int round_mode,
                               void *ws, size_t ws_bytes) {
  if (ctx && !g) return niti_fail(ctx, NITI_ERR_ARG, "niti_linear_bwd: bad argument (g is null)");
  return linear_bwd_impl(ctx, stream, a, e, w, e_prev, relu_mask_src, g, nullptr, b_e, b_g, M, N, K, m_u,
                         round_mode, ws, ws_bytes, "niti_linear_bwd");
}

extern "C" int niti_linear_bwd_update(niti_ctx *ctx, void *stream, const int8_t *a, const int8_t *e, int8_t *w,
                                      int8_t *e_prev, const int8_t *relu_mask_src, int32_t *b_e, int32_t *b_g,
                                      int M, int N, int K, int m_u, int round_mode, void *ws, size_t ws_bytes) {
  return linear_bwd_impl(ctx, stream, a, e, w, e_prev, relu_mask_src, nullptr, w, b_e, b_g, M, N, K, m_u,
                         round_mode, ws, ws_bytes, "niti_linear_bwd_update");
}

static int conv_args_ok(int B, int H, int W, int Ci, int Co, int R, int S, int pad, int round_mode) {
  return B > 0 && H > 0 && W > 0 && Ci > 0 && Co > 0 && R > 0 && S > 0 && pad >= 0 &&
         (round_mode == 0 || round_mode == 1);
}

static int conv_fwd_impl(niti_ctx *ctx, void *stream, const int8_t *x, const int32_t *s_x, const int8_t *w,
                         const int32_t *s_w, int8_t *y, int8_t *y_pool, int32_t *s_y, int32_t *b_y, int B, int H,
                         int W, int Cin, int Cout, int R, int S, int pad, int stride, int relu, int round_mode,
                         void *ws, size_t ws_bytes) {
  if (!ctx) return NITI_ERR_ARG;
  GemmProblem p;
  memset(&p, 0, sizeof(p));
  if (!x || !w || !y || !s_x || !s_w || !conv_args_ok(B, H, W, Cin, Cout, R, S, pad, round_mode) ||
      misaligned16(x) || misaligned16(w) || misaligned16(y) ||
      !fill_conv(p, GK_CONV_FWD, B, H, W, Cin, Cout, R, S, pad, stride))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_conv_fwd: bad argument (pointers must be 16-byte aligned)");
  p.p0 = x; p.p1 = w;
  int64_t dims[9] = {B, H, W, Cin, Cout, R, S, pad, stride};
  const size_t need = niti_workspace_bytes(NITI_OP_CONV_FWD, dims, 9);
  if (few_channel_conv(Cin, R, S) && ctx->engine != 1) {
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < need)
      return niti_fail(ctx, NITI_ERR_WORKSPACE, "workspace missing, misaligned or too small");
    // gather the taps into [M][32] rows, pad the weights to [Cout][32], then a K = 32 multiply
    cudaStream_t st = (cudaStream_t)stream;
    const size_t M = (size_t)p.gm;
    char *base = (char *)ws + NITI_WS_HEADER + round_up(M * (size_t)Cout * 4, 256);
    int8_t *xcol = (int8_t *)base;
    int8_t *wcol = (int8_t *)(base + round_up(M * 32, 256));
    if (ctx->tap_buf && M * 32 <= ctx->tap_bytes) {
      // gathered into the caller's tap cache: the weight-gradient call of this layer finds the rows there
      xcol = ctx->tap_buf;
      ctx->tap_x = x;
      const int dims[9] = {B, H, W, Cin, R, S, pad, stride, 1};
      memcpy(ctx->tap_dims, dims, sizeof(dims));
    }
    int rc = niti_launch_im2col32(ctx, st, x, xcol, B, H, W, Cin, R, S, pad, stride, p.Ho, p.Wo);
    if (rc == NITI_OK) rc = niti_launch_pad_rows32(ctx, st, w, wcol, Cout, R * S * Cin);
    if (rc != NITI_OK) return rc;
    GemmProblem q;
    fill_fc(q, GK_FC_FWD, (int)M, Cout, 32);
    q.p0 = xcol; q.p1 = wcol;
    rc = run_gemm_round(ctx, st, q, ws, ws_bytes, need, y, 7, round_mode, relu, nullptr, s_x, s_w, s_y, b_y);
    if (rc != NITI_OK || !y_pool) return rc;
    return niti_launch_maxpool2_fwd(ctx, st, y, y_pool, B, p.Ho, p.Wo, Cout);
  }
  return run_gemm_round(ctx, (cudaStream_t)stream, p, ws, ws_bytes, need, y, 7, round_mode, relu, nullptr,
                        s_x, s_w, s_y, b_y, nullptr, y_pool);
}

extern "C" int niti_conv_fwd_strided(niti_ctx *ctx, void *stream, const int8_t *x, const int32_t *s_x,
                                     const int8_t *w, const int32_t *s_w, int8_t *y, int32_t *s_y, int32_t *b_y,
                                     int B, int H, int W, int Cin, int Cout, int R, int S, int pad, int stride,
                                     int relu, int round_mode, void *ws, size_t ws_bytes) {
  return conv_fwd_impl(ctx, stream, x, s_x, w, s_w, y, nullptr, s_y, b_y, B, H, W, Cin, Cout, R, S, pad, stride, relu,
                       round_mode, ws, ws_bytes);
}

extern "C" int niti_conv_fwd_pool(niti_ctx *ctx, void *stream, const int8_t *x, const int32_t *s_x, const int8_t *w,
                                  const int32_t *s_w, int8_t *y, int8_t *y_pool, int32_t *s_y, int32_t *b_y, int B,
                                  int H, int W, int Cin, int Cout, int R, int S, int pad, int relu, int round_mode,
                                  void *ws, size_t ws_bytes) {
  if (!ctx) return NITI_ERR_ARG;
  const int Ho = H + 2 * pad - R + 1, Wo = W + 2 * pad - S + 1;
  if (!y_pool || Ho <= 0 || Wo <= 0 || (Ho & 1) || (Wo & 1) || misaligned16(y_pool))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_conv_fwd_pool: bad argument (output height and width must be even)");
  return conv_fwd_impl(ctx, stream, x, s_x, w, s_w, y, y_pool, s_y, b_y, B, H, W, Cin, Cout, R, S, pad, 1, relu,
                       round_mode, ws, ws_bytes);
}

extern "C" int niti_conv_fwd(niti_ctx *ctx, void *stream, const int8_t *x, const int32_t *s_x,
                             const int8_t *w, const int32_t *s_w, int8_t *y, int32_t *s_y, int32_t *b_y,
                             int B, int H, int W, int Cin, int Cout, int R, int S, int pad, int relu,
                             int round_mode, void *ws, size_t ws_bytes) {
  return niti_conv_fwd_strided(ctx, stream, x, s_x, w, s_w, y, s_y, b_y, B, H, W, Cin, Cout, R, S, pad, 1, relu,
                               round_mode, ws, ws_bytes);
}

extern "C" int niti_conv_dgrad_strided(niti_ctx *ctx, void *stream, const int8_t *e, const int8_t *w,
                                       int8_t *e_prev, const int8_t *relu_mask_src, int32_t *b_e, int B, int H,
                                       int W, int Cin, int Cout, int R, int S, int pad, int stride, int round_mode,
                                       void *ws, size_t ws_bytes) {
  if (!ctx) return NITI_ERR_ARG;
  GemmProblem p;
  memset(&p, 0, sizeof(p));
  if (!e || !w || !e_prev || !conv_args_ok(B, H, W, Cin, Cout, R, S, pad, round_mode) || misaligned16(e) ||
      misaligned16(w) || misaligned16(e_prev) || misaligned16(relu_mask_src) ||
      !fill_conv(p, GK_CONV_DGRAD, B, H, W, Cin, Cout, R, S, pad, stride))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_conv_dgrad: bad argument (pointers must be 16-byte aligned)");
  p.p0 = e; p.p1 = w;
  int64_t dims[9] = {B, H, W, Cin, Cout, R, S, pad, stride};
  return run_gemm_round(ctx, (cudaStream_t)stream, p, ws, ws_bytes,
                        niti_workspace_bytes(NITI_OP_CONV_DGRAD, dims, 9), e_prev, 7, round_mode, 0,
                        relu_mask_src, nullptr, nullptr, nullptr, b_e);
}

extern "C" int niti_conv_dgrad(niti_ctx *ctx, void *stream, const int8_t *e, const int8_t *w,
                               int8_t *e_prev, const int8_t *relu_mask_src, int32_t *b_e, int B, int H,
                               int W, int Cin, int Cout, int R, int S, int pad, int round_mode, void *ws,
                               size_t ws_bytes) {
  return niti_conv_dgrad_strided(ctx, stream, e, w, e_prev, relu_mask_src, b_e, B, H, W, Cin, Cout, R, S, pad, 1,
                                 round_mode, ws, ws_bytes);
}

// Weight gradient of a convolution; with update_w the rounded gradient is subtracted from the
// weights in place instead of being returned.
static int conv_wgrad_impl(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e, int8_t *g,
                           int8_t *update_w, int32_t *b_g, int B, int H, int W, int Cin, int Cout, int R, int S,
                           int pad, int stride, int m_u, int round_mode, void *ws, size_t ws_bytes, const char *who) {
  if (!ctx) return NITI_ERR_ARG;
  GemmProblem p;
  memset(&p, 0, sizeof(p));
  if (!x || !e || (!g && !update_w) || m_u < 1 || m_u > 7 || !conv_args_ok(B, H, W, Cin, Cout, R, S, pad, round_mode) ||
      misaligned16(x) || misaligned16(e) || misaligned16(g) || misaligned16(update_w) ||
      !fill_conv(p, GK_CONV_WGRAD, B, H, W, Cin, Cout, R, S, pad, stride)) {
    snprintf(ctx->err, sizeof(ctx->err), "%s: bad argument (pointers must be 16-byte aligned)", who);
    return NITI_ERR_ARG;
  }
  p.p0 = e; p.p1 = x;
  int64_t dims[9] = {B, H, W, Cin, Cout, R, S, pad, stride};
  const size_t need_base = niti_workspace_bytes(NITI_OP_CONV_WGRAD, dims, 9);
  const size_t need = update_w ? niti_workspace_bytes(NITI_OP_CONV_WGRAD_UPDATE, dims, 9) : need_base;
  if (!ws || ((uintptr_t)ws & 255) || ws_bytes < need)
    return niti_fail(ctx, NITI_ERR_WORKSPACE, "workspace missing, misaligned or too small");
  if (update_w) g = (int8_t *)((char *)ws + need_base);       // scratch, used only where the rounding stores int8
  if (few_channel_conv(Cin, R, S) && ctx->engine != 1 && (Cout % 16) == 0) {
    // g32[co][k] = sum_pix e[pix][co] * xcol[pix][k] over the gathered rows (k < 32), then the first
    // R*S*Cin columns are rounded into g
    cudaStream_t st = (cudaStream_t)stream;
    const size_t M = (size_t)B * p.Ho * p.Wo;
    WsHeader *hdr = nullptr;
    char *base = (char *)ws + NITI_WS_HEADER + round_up((size_t)(p.gm * p.gn) * 4, 256);
    int8_t *xcol = (int8_t *)base;
    int32_t *acc32 = (int32_t *)(base + round_up(M * 32, 256) + round_up((size_t)Cout * 32, 256));
    int rc = niti_take_header(ctx, st, ws, &hdr);
    if (rc != NITI_OK) return rc;
    if (tap_cache_hit(ctx, x, B, H, W, Cin, R, S, pad, stride)) {
      xcol = ctx->tap_buf;                 // gathered by the forward call
      ctx->tap_dims[8] = 0;                // (used once: the next forward call fills the cache again)
    } else rc = niti_launch_im2col32(ctx, st, x, xcol, B, H, W, Cin, R, S, pad, stride, p.Ho, p.Wo);
    if (rc != NITI_OK) return rc;
    GemmProblem q;
    fill_fc(q, GK_FC_WGRAD, (int)M, Cout, 32);     // rows M are the contraction
    q.p0 = e; q.p1 = xcol;
    bool fused = false;
    RoundSpec none = {nullptr, nullptr, m_u, round_mode, 0, nullptr, nullptr, nullptr, nullptr, nullptr};
    const int saved = ctx->engine;
    if (saved == 0) ctx->engine = 4;               // int32 accumulators are needed here, not a fused store
    rc = niti_tc_gemm(ctx, st, q, none, acc32, hdr, &fused);
    ctx->engine = saved;
    if (rc == NITI_ERR_SHAPE) {
      rc = niti_simt_gemm(ctx, st, q, acc32, hdr);
      if (rc == NITI_OK) rc = niti_reduce_after_gemm(ctx, st, q.kind, acc32, (long long)Cout * 32, hdr);
    }
    if (rc != NITI_OK) return rc;
    rc = niti_launch_round_compact32(ctx, st, acc32, hdr, g, Cout, R * S * Cin, m_u, round_mode, b_g);
    if (rc != NITI_OK || !update_w) return rc;
    return niti_launch_sgd_update(ctx, st, update_w, g, (long long)Cout * R * S * Cin);
  }
  return run_gemm_round(ctx, (cudaStream_t)stream, p, ws, ws_bytes, need, g, m_u, round_mode, 0, nullptr,
                        nullptr, nullptr, nullptr, b_g, update_w);
}

extern "C" int niti_conv_wgrad_strided(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e, int8_t *g,
                                       int32_t *b_g, int B, int H, int W, int Cin, int Cout, int R, int S, int pad,
                                       int stride, int m_u, int round_mode, void *ws, size_t ws_bytes) {
  if (ctx && !g) return niti_fail(ctx, NITI_ERR_ARG, "niti_conv_wgrad: bad argument (g is null)");
  return conv_wgrad_impl(ctx, stream, x, e, g, nullptr, b_g, B, H, W, Cin, Cout, R, S, pad, stride, m_u, round_mode,
                         ws, ws_bytes, "niti_conv_wgrad");
}

extern "C" int niti_conv_wgrad(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e, int8_t *g,
                               int32_t *b_g, int B, int H, int W, int Cin, int Cout, int R, int S, int pad,
                               int m_u, int round_mode, void *ws, size_t ws_bytes) {
  return niti_conv_wgrad_strided(ctx, stream, x, e, g, b_g, B, H, W, Cin, Cout, R, S, pad, 1, m_u, round_mode, ws,
                                 ws_bytes);
}

extern "C" int niti_conv_wgrad_update(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e, int8_t *w,
                                      int32_t *b_g, int B, int H, int W, int Cin, int Cout, int R, int S, int pad,
                                      int m_u, int round_mode, void *ws, size_t ws_bytes) {
  if (ctx && !w) return niti_fail(ctx, NITI_ERR_ARG, "niti_conv_wgrad_update: bad argument (w is null)");
  return conv_wgrad_impl(ctx, stream, x, e, nullptr, w, b_g, B, H, W, Cin, Cout, R, S, pad, 1, m_u, round_mode, ws,
                         ws_bytes, "niti_conv_wgrad_update");
}
