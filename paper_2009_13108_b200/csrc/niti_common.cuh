// Shared declarations of the NITI sm_100a library (internal; the public boundary is include/niti.h).
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "../../include/niti.h"

struct niti_ctx {
  int device;
  int sm_count;
  int engine;               // niti_set_engine: 0 auto, 1 CUDA-core kernels only, 2 single-CTA tensor-core kernel,
                            // 3 paired-CTA only, 4 two-pass (int32 spill) epilogue, 5 no resident-weights mode
  uint32_t *d_status;       // device status word (+ counter of recomputations)
  int32_t *d_spec_tab;      // NITI_SPEC_SLOTS x {tag, error}: per call site, by how many bits the sample-based
                            // estimate of the speculative epilogue missed the true bit-width last time
  uint64_t launches;
  uint64_t tc_launches;     // launches of the tensor-core matrix-multiply kernel
  uint64_t tc2_launches;    // of those, launches of the paired-CTA (cta_group::2) variant
  char err[256];
  // optional timing of the tensor-core kernel: event pairs recorded around each launch
  int profile_on;
  int prof_used;
  cudaEvent_t *prof_ev;     // 2 * NITI_PROF_MAX events
  double *prof_ops;         // algorithmic int8 operations (2*M*N*K) of each recorded launch
  // cuTensorMapEncodeTiled, fetched through the runtime so that libcuda is not a link dependency
  void *encode_tiled;
  // data-parallel training (niti_set_reduce_hook): called where a tensor-wide quantity has to be
  // combined over the ranks before the rounding may use it
  niti_reduce_fn reduce_fn;
  void *reduce_user;
  // niti_set_tap_cache: caller-owned buffer that keeps the gathered taps of a few-channel convolution
  // between its forward call and its weight-gradient call, and what it currently holds
  int8_t *tap_buf;
  size_t tap_bytes;
  const void *tap_x;
  int tap_dims[9];          // B, H, W, Cin, R, S, pad, stride, valid
  // niti_begin_step: workspace whose headers were cleared in one go, and how many of them are used up
  void *step_ws;
  int step_slot;
  int dp_rank, dp_world;    // niti_set_dp_shard: > 1 ranks = weight gradients are reduce-scattered, rounded per
                            // shard and all-gathered as int8 (5 bytes per weight on the wire instead of 8)
  // per-device facts of the tensor-core kernel, indexed by CTAs per tile (1 or 2): co-resident CTAs /
  // CTA pairs (0 = not asked yet) and the dynamic shared-memory limit already set on the kernel
  int tc_units[3];
  size_t tc_attr_smem[3];
  // the device's opt-in limit of dynamic shared memory per CTA.  The limit set on a kernel belongs to the
  // device, not to a context: every context therefore sets this same value (a context that set only what it
  // needed would lower the limit under another context of the process)
  size_t smem_optin;
};



#define NITI_PROF_MAX 8192
#define NITI_SPEC_SLOTS 4096
// Every workspace starts with NITI_HDR_SLOTS headers of NITI_HDR_SLOT_BYTES each (reduction scalars, the
// words of the speculative agreement, split maxima).  A call needs a zeroed header.  Without further
// notice it clears and uses the first one.  After niti_begin_step() has cleared all of them with one
// memset, the following calls on that workspace take one header each, in order, without clearing (a
// cleared-per-call header costs a memset node of about 2 us in front of every multiply of a step).
#define NITI_HDR_SLOTS 64
#define NITI_HDR_SLOT_BYTES 4096
#define NITI_WS_HEADER (NITI_HDR_SLOTS * NITI_HDR_SLOT_BYTES)   // bytes in front of the accumulator scratch
// A contraction that is split over CTAs adds int32 partial sums; split s records the largest magnitude
// among its partial sums in split_max[s] (unsigned words from byte NITI_SPLIT_MAX_OFF of the header).
// The sum of those maxima bounds every accumulator of the tensor: when it reaches 2^31 the int32
// contract of Section 3.2 can no longer be vouched for and NITI_DEV_ACC_RANGE is raised.  Every split
// covers at most NITI_SPLIT_MAX_K contraction elements, so a partial sum itself cannot wrap.
#define NITI_SPLIT_MAX_OFF 256
#define NITI_MAX_SPLITS 960
#define NITI_SPLIT_MAX_K 131072

// Scalars at the start of a workspace.
struct WsHeader {
  unsigned int maxabs32;            // a value with the bit length of max |acc| (a max, or an OR of magnitudes)
  unsigned int done_ctas;           // CTAs that have finished (single-wave launches publish b themselves)
  unsigned long long maxabs64;      // same for the 64-bit loss accumulators
  // the three words of the speculative agreement share one 16-byte line so that one load polls them all
  unsigned int est_max;             // max |acc| over the first tile of the CTAs that have reported
  unsigned int tile_counter;        // CTAs that have reported
  unsigned int spec_b;              // 0, or 1 + the bit-width the speculative epilogue rounds with
  unsigned int hits;               // integer cross-entropy: rows whose first arg-max is the label
};
static_assert(sizeof(WsHeader) == 32, "workspace header layout");
static_assert(NITI_SPLIT_MAX_OFF + 4 * NITI_MAX_SPLITS <= NITI_HDR_SLOT_BYTES, "split maxima fit the header");
__host__ __device__ __forceinline__ unsigned int *niti_split_max(WsHeader *hdr) {
  return reinterpret_cast<unsigned int *>(reinterpret_cast<char *>(hdr) + NITI_SPLIT_MAX_OFF);
}

#define NITI_CUDA_TRY(ctx, expr)                                                        \
  do {                                                                                  \
    cudaError_t e__ = (expr);                                                           \
    if (e__ != cudaSuccess) {                                                           \
      snprintf((ctx)->err, sizeof((ctx)->err), "%s failed: %s (%s:%d)", #expr,          \
               cudaGetErrorString(e__), __FILE__, __LINE__);                            \
      return NITI_ERR_CUDA;                                                             \
    }                                                                                   \
  } while (0)

// A zeroed header for the call that is being enqueued: the next unused one of a workspace prepared by
// niti_begin_step(), else the first one, cleared here.
static inline int niti_take_header(niti_ctx *ctx, cudaStream_t st, void *ws, WsHeader **hdr) {
  if (ws == ctx->step_ws && ctx->step_slot < NITI_HDR_SLOTS) {
    *hdr = reinterpret_cast<WsHeader *>(reinterpret_cast<char *>(ws) + (size_t)NITI_HDR_SLOT_BYTES * ctx->step_slot++);
    return NITI_OK;
  }
  *hdr = reinterpret_cast<WsHeader *>(ws);
  ctx->launches++;
  if (cudaMemsetAsync(ws, 0, NITI_HDR_SLOT_BYTES, st) != cudaSuccess) {
    snprintf(ctx->err, sizeof(ctx->err), "clearing the workspace header failed");
    return NITI_ERR_CUDA;
  }
  return NITI_OK;
}

static inline int niti_fail(niti_ctx *ctx, int code, const char *msg) {
  if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s", msg);
  return code;
}

// Runs the caller's reduction over the ranks on a device buffer, ordered on the stream.
static inline int niti_reduce(niti_ctx *ctx, cudaStream_t st, void *dev_ptr, long long count, int kind) {
  if (!ctx->reduce_fn) return NITI_OK;
  if (ctx->reduce_fn(ctx->reduce_user, (void *)st, dev_ptr, (int64_t)count, kind) != 0)
    return niti_fail(ctx, NITI_ERR_ARG, "the reduction hook reported a failure");
  return NITI_OK;
}
// (weight gradients contract over the batch: under data parallelism their int32 sums are added
// over the ranks; every other multiply only shares its max magnitude)
static inline bool niti_is_wgrad(int kind) { return kind == 2 || kind == 5; }   // GK_FC_WGRAD, GK_CONV_WGRAD

// ---- rounding arithmetic (Algorithm 3 and round-to-nearest), on the magnitude ----------------
template <typename U>
__device__ __forceinline__ U niti_round_mag(U m, int bp, U qmax, int round_mode) {
  U q = m >> bp;
  U f = m & ((U(1) << bp) - 1);
  if (round_mode == NITI_ROUND_PSR) {
    f >>= (bp & 1);               // odd binary point: the lowest discarded bit is dropped
    int h = bp >> 1;              // width of each half
    U top = f >> h;
    U bot = f & ((U(1) << h) - 1);
    q += (top > bot) ? 1 : 0;
  } else {
    q += (bp > 0 && (f >> (bp - 1))) ? 1 : 0;
  }
  return q > qmax ? qmax : q;
}

__device__ __forceinline__ int niti_round_i32(int x, int bp, unsigned qmax, int round_mode) {
  unsigned m = x < 0 ? 0u - (unsigned)x : (unsigned)x;
  int q = (int)niti_round_mag<unsigned>(m, bp, qmax, round_mode);
  return x < 0 ? -q : q;
}

__device__ __forceinline__ int niti_bitlen32(unsigned v) { return 32 - __clz(v); }

// ---- internal launchers (defined across the .cu files) ----------------------------------------
// Shape of one matrix multiply D[m][n] = sum_k A(m,k) * B(n,k) with implicit operand addressing.
enum NitiGemmKind {
  GK_FC_FWD = 0,   // A = a[M][K],        B = w[N][K]
  GK_FC_DGRAD,     // A = e[M][N],        B(k', n) = w[n][k']
  GK_FC_WGRAD,     // A(n, m) = e[m][n],  B(k', m) = a[m][k']
  GK_CONV_FWD,     // A(pix, (r,s,ci)) = x shifted, B = w[co][(r,s,ci)]
  GK_CONV_DGRAD,   // A(pix, (r,s,co)) = e shifted, B(ci, (r,s,co)) = w[co][r][s][ci]
  GK_CONV_WGRAD    // A(co, pix) = e[pix][co],      B((r,s,ci), pix) = x shifted
};
static_assert(GK_FC_WGRAD == 2 && GK_CONV_WGRAD == 5, "niti_is_wgrad");

struct GemmProblem {
  int kind;
  const int8_t *p0;  // first operand  (a / e / x)
  const int8_t *p1;  // second operand (w / a / e)
  // fully connected: M, N, K of the layer.  convolution: B,H,W (input), Ho,Wo (output), Ci, Co, R, S, pad, stride
  int M, N, K;
  int B, H, W, Ho, Wo, Ci, Co, R, S, pad, stride;
  // the matrix multiply actually run
  long long gm, gn, gk;
  // row pitch in bytes of p0 when its rows are padded (fully connected kinds; 0 = dense)
  long long ld0;
};

// Fully connected forward / error multiplies with at most 128 output rows (weight streaming: the
// contraction is split over the SMs) keep up to this many int32 partial tensors in the scratch, one
// per split; 1 for every other multiply.  The workspace query reserves room accordingly.
#define NITI_PARTIAL_SLICES 16
static inline int niti_partial_slices(int kind, long long gm) {
  return ((kind == 0 || kind == 1) && gm <= 128) ? NITI_PARTIAL_SLICES : 1;   // GK_FC_FWD, GK_FC_DGRAD
}
// acc holds `splits` partial tensors of n int32 each: adds them into the first, takes max |sum| into
// hdr->maxabs32 and raises NITI_DEV_ACC_RANGE when the magnitudes of an element's partial sums add up to 2^31
int niti_launch_sum_partials(niti_ctx *ctx, cudaStream_t st, int32_t *acc, int splits, long long n, WsHeader *hdr);
// shard_ok: the caller rounds only this rank's shard afterwards (niti_dp_shard) and all-gathers the result
int niti_reduce_after_gemm(niti_ctx *ctx, cudaStream_t st, int kind, int32_t *acc, long long n, WsHeader *hdr,
                           bool shard_ok = false);
// Sharding of a weight-gradient tensor of n elements over the data-parallel ranks: `main` elements are
// split evenly (every shard a multiple of 16 elements, so that vector accesses stay aligned), the
// remaining `n - main` are combined with an all-reduce and handled by every rank.
struct NitiDpShard { long long main, shard, off; };
static inline NitiDpShard niti_dp_shard(const niti_ctx *ctx, long long n) {
  NitiDpShard s;
  const long long unit = 16LL * ctx->dp_world;
  s.main = n / unit * unit;
  s.shard = s.main / ctx->dp_world;
  s.off = s.shard * ctx->dp_rank;
  return s;
}
static inline bool niti_dp_sharded(const niti_ctx *ctx, int kind) {
  return ctx->reduce_fn && ctx->dp_world > 1 && (kind == 2 || kind == 5);   // weight gradients only
}
// max |acc| into hdr->maxabs32; splits > 1: also adds up the split maxima of the header and raises
// NITI_DEV_ACC_RANGE when an accumulator may have left the int32 range
int niti_launch_maxabs(niti_ctx *ctx, cudaStream_t st, const int32_t *acc, long long n, WsHeader *hdr, int splits = 0);
// Plain CUDA-core engine: writes int32 accumulators to acc[gm][gn] and max|acc| to hdr->maxabs32.
int niti_simt_gemm(niti_ctx *ctx, cudaStream_t st, const GemmProblem &p, int32_t *acc, WsHeader *hdr);
// What follows the multiply: rounding target and the scalars of Algorithm 2.
struct RoundSpec {
  int8_t *out;
  const int8_t *mask;      // optional ReLU mask source (zero the output where mask <= 0)
  int mbits, round_mode, relu;
  const int32_t *s_a, *s_w;
  int32_t *s_out, *b_out;
  int8_t *pool_out;        // optional (may be null): 2 x 2 max-pool of `out`, forward convolutions with ReLU
  int8_t *update_w;        // optional (may be null): weight gradients; the caller will subtract `out` from these weights
};
// Tensor-core engine (tcgen05); returns NITI_ERR_SHAPE if the shape is not eligible.  *fused is set
// when the kernel also did the bit-width / shift / round / store (nothing is left to do); otherwise
// acc holds the int32 accumulators and hdr->maxabs32 their max magnitude.
// *pooled (may be null) is set when the kernel's epilogue also wrote r.pool_out.
// *updated (may be null) is set when the epilogue subtracted the rounded gradient from r.update_w itself
// (`out` is then not written).
int niti_tc_gemm(niti_ctx *ctx, cudaStream_t st, const GemmProblem &p, const RoundSpec &r, int32_t *acc,
                 WsHeader *hdr, bool *fused, bool *pooled = nullptr, bool shard_ok = false, bool *updated = nullptr);
size_t niti_tc_scratch_bytes(const GemmProblem &p);

// Epilogue pass: b from hdr->maxabs32, bp = max(0, b - mbits), out = Round(acc) with optional ReLU
// and optional mask; s_out = s_a + s_w + bp if s_out != NULL; b_out = b if != NULL.
int niti_launch_round(niti_ctx *ctx, cudaStream_t st, const int32_t *acc, const WsHeader *hdr,
                      int8_t *out, long long n, int mbits, int round_mode, int relu,
                      const int8_t *mask, const int32_t *s_a, const int32_t *s_w, int32_t *s_out,
                      int32_t *b_out, int8_t *upd_w = nullptr);
