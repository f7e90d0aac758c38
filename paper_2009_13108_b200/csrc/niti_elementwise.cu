// HBM-bound kernels of the NITI library: the shift-and-round pass (Algorithm 2/3), the integer
// cross-entropy gradient (Section 3.5), the weight update (Algorithm 1) and the int8 support ops.
#include "niti_common.cuh"
#include <mutex>

// ---------------------------------------------------------------------------------------------
// Shift-and-round pass over an int32 accumulator tensor (Algorithm 2, with Algorithm 3 rounding).
// Every thread handles 16 consecutive elements: four 16-byte loads, one 16-byte store.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned sat_sub_clamp127(unsigned w, unsigned g) {
  // per byte: clamp(w - g, -127, 127): saturating subtract gives [-128, 127]; lift -128 to -127
  return __vmaxs4(__vsubss4(w, g), 0x81818181u);
}

__global__ void __launch_bounds__(256)
round_i32_kernel(const int32_t *__restrict__ acc, const WsHeader *__restrict__ hdr,
                 int8_t *__restrict__ out, long long n, int mbits, int round_mode, int relu,
                 const int8_t *__restrict__ mask, const int32_t *__restrict__ s_a,
                 const int32_t *__restrict__ s_w, int32_t *__restrict__ s_out,
                 int32_t *__restrict__ b_out, uint32_t *__restrict__ status, int8_t *__restrict__ upd_w) {
  const int b = niti_bitlen32(hdr->maxabs32);
  const int bp = b > mbits ? b - mbits : 0;
  const unsigned qmax = (1u << mbits) - 1u;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (b_out) *b_out = b;
    if (s_out) {
      int s = bp + (s_a ? *s_a : 0) + (s_w ? *s_w : 0);
      *s_out = s;
      if (s < -128 || s > 127) atomicOr(status, NITI_DEV_EXP_RANGE);
    }
  }
  const long long nvec = n >> 4;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride) {
    const int4 *src = reinterpret_cast<const int4 *>(acc) + v * 4;
    int4 x0 = __ldcs(src), x1 = __ldcs(src + 1), x2 = __ldcs(src + 2), x3 = __ldcs(src + 3);
    int xs[16] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w,
                  x2.x, x2.y, x2.z, x2.w, x3.x, x3.y, x3.z, x3.w};
    int4 mk = make_int4(-1, -1, -1, -1);
    if (mask) {
      int4 mv = *(reinterpret_cast<const int4 *>(mask) + v);
      mk.x = __vcmpgts4(mv.x, 0); mk.y = __vcmpgts4(mv.y, 0);
      mk.z = __vcmpgts4(mv.z, 0); mk.w = __vcmpgts4(mv.w, 0);
    }
    unsigned o[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      unsigned word = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int q = niti_round_i32(xs[w * 4 + j], bp, qmax, round_mode);
        if (relu && q < 0) q = 0;
        word |= (unsigned)(q & 0xff) << (8 * j);
      }
      o[w] = word;
    }
    int4 ov = make_int4(o[0] & mk.x, o[1] & mk.y, o[2] & mk.z, o[3] & mk.w);
    if (upd_w) {
      // weight update fused with the rounding of the weight gradient (Section 3.3: the rounded
      // gradient is never stored): w <- clamp(w - q, -127, 127)
      int4 wv = *(reinterpret_cast<int4 *>(upd_w) + v);
      wv.x = sat_sub_clamp127(wv.x, ov.x); wv.y = sat_sub_clamp127(wv.y, ov.y);
      wv.z = sat_sub_clamp127(wv.z, ov.z); wv.w = sat_sub_clamp127(wv.w, ov.w);
      *(reinterpret_cast<int4 *>(upd_w) + v) = wv;
    } else {
      *(reinterpret_cast<int4 *>(out) + v) = ov;
    }
  }
  // ragged tail (fewer than 16 elements)
  long long t = (nvec << 4) + (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) {
    int q = niti_round_i32(acc[t], bp, qmax, round_mode);
    if (relu && q < 0) q = 0;
    if (mask && mask[t] <= 0) q = 0;
    if (upd_w) {
      int d = (int)upd_w[t] - q;
      upd_w[t] = (int8_t)(d > 127 ? 127 : (d < -127 ? -127 : d));
    } else {
      out[t] = (int8_t)q;
    }
  }
}

int niti_launch_round(niti_ctx *ctx, cudaStream_t st, const int32_t *acc, const WsHeader *hdr,
                      int8_t *out, long long n, int mbits, int round_mode, int relu,
                      const int8_t *mask, const int32_t *s_a, const int32_t *s_w, int32_t *s_out,
                      int32_t *b_out, int8_t *upd_w) {
  long long nvec = n >> 4;
  long long blocks = (nvec + 255) / 256;
  long long cap = (long long)ctx->sm_count * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  round_i32_kernel<<<(unsigned)blocks, 256, 0, st>>>(acc, hdr, out, n, mbits, round_mode, relu, mask,
                                                     s_a, s_w, s_out, b_out, ctx->d_status, upd_w);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

// ---------------------------------------------------------------------------------------------
// Few-channel convolutions (first layer: 1 or 3 input channels, R*S*Cin <= 32): the taps of every
// output pixel are gathered into one 32-byte row so that the layer becomes a plain K = 32 matrix
// multiply for the tensor-core engine.  Column k = (r * S + s) * Cin + ci, zero beyond R*S*Cin.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
im2col32_kernel(const int8_t *__restrict__ x, int8_t *__restrict__ xcol, int B, int H, int W, int Ci, int R,
                int S, int pad, int stride, int Ho, int Wo) {
  const long long M = (long long)B * Ho * Wo;
  for (long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x; m < M;
       m += (long long)gridDim.x * blockDim.x) {
    const int j = (int)(m % Wo);
    const long long t = m / Wo;
    const int i = (int)(t % Ho);
    const long long b = t / Ho;
    unsigned w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int k = 0;
    for (int r = 0; r < R; ++r) {
      const int ii = i * stride + r - pad;
      for (int q = 0; q < S; ++q) {
        const int jj = j * stride + q - pad;
        const bool in = ii >= 0 && ii < H && jj >= 0 && jj < W;
        const int8_t *src = x + ((b * H + ii) * W + jj) * Ci;
        for (int c = 0; c < Ci; ++c, ++k) {
          const unsigned v = in ? (unsigned)(uint8_t)src[c] : 0u;
          w[k >> 2] |= v << (8 * (k & 3));
        }
      }
    }
    int4 *dst = reinterpret_cast<int4 *>(xcol + m * 32);
    dst[0] = make_int4(w[0], w[1], w[2], w[3]);
    dst[1] = make_int4(w[4], w[5], w[6], w[7]);
  }
}

// Fast path for the RGB first layer (Cin = 3, 3x3 taps, pad 1, W % 4 == 0): one block per output image
// row stages the three input rows in shared memory (one pixel of zero halo on each side) and every
// thread assembles the 27-byte tap vectors of four consecutive pixels from five aligned words per
// row, with byte offsets known at compile time.  The generic kernel above issues 27 byte loads per
// pixel and ran at a fifth of the memory rate.
__device__ __forceinline__ unsigned win_byte(const unsigned (&w)[5], int idx) {
  return (w[idx >> 2] >> (8 * (idx & 3))) & 0xffu;
}
__global__ void __launch_bounds__(128)
im2col32_rgb3x3_kernel(const int8_t *__restrict__ x, int8_t *__restrict__ xcol, int B, int H, int W) {
  extern __shared__ unsigned rgb_rows[];          // 3 rows x pitch words
  const int row_words = W * 3 / 4;                // data words per image row
  const int pitch = row_words + 2;                // one halo word on each side (3 of its 4 bytes are used)
  const int i = blockIdx.x % H;
  const long long b = blockIdx.x / H;
  for (int idx = threadIdx.x; idx < 3 * pitch; idx += blockDim.x) {
    const int r = idx / pitch, c = idx % pitch - 1;
    const int ii = i + r - 1;
    unsigned v = 0;
    if (c >= 0 && c < row_words && ii >= 0 && ii < H)
      v = reinterpret_cast<const unsigned *>(x + (b * H + ii) * (long long)W * 3)[c];
    rgb_rows[idx] = v;
  }
  __syncthreads();
  // pixel j of a staged row starts at byte 4 + 3 j; the window of pixels 4t-1 .. 4t+4 starts at
  // byte 12 t + 1, i.e. at byte 1 of word 3 t
  for (int t = threadIdx.x; t < W / 4; t += blockDim.x) {
    unsigned win[3][5];
#pragma unroll
    for (int r = 0; r < 3; ++r)
#pragma unroll
      for (int k = 0; k < 5; ++k) win[r][k] = rgb_rows[r * pitch + 3 * t + k];
    int4 *dst = reinterpret_cast<int4 *>(xcol + ((b * H + i) * (long long)W + 4 * t) * 32);
#pragma unroll
    for (int px = 0; px < 4; ++px) {
      unsigned o[8];
#pragma unroll
      for (int wd = 0; wd < 8; ++wd) {
        unsigned v = 0;
#pragma unroll
        for (int by = 0; by < 4; ++by) {
          const int k = 4 * wd + by;              // column of the gathered row: (tap row, tap col, channel)
          if (k < 27) v |= win_byte(win[k / 9], 1 + 3 * px + k % 9) << (8 * by);
        }
        o[wd] = v;
      }
      // one gathered row = one 32-byte sector: a single 256-bit store per pixel
      asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                   ::"l"(dst + 2 * px), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                   : "memory");
    }
  }
}

// weights [Cout][R*S*Cin] -> [Cout][32], zero padded
__global__ void pad_rows32_kernel(const int8_t *__restrict__ w, int8_t *__restrict__ wcol, int rows, int k) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < rows * 32) {
    const int r = idx >> 5, c = idx & 31;
    wcol[idx] = c < k ? w[r * k + c] : (int8_t)0;
  }
}

// rows of n bytes -> rows of pitch bytes (pitch >= n), zero padded
__global__ void pad_pitch_kernel(const int8_t *__restrict__ src, int8_t *__restrict__ dst, int rows, int n, int pitch) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < (long long)rows * pitch) {
    const int r = (int)(idx / pitch), c = (int)(idx % pitch);
    dst[idx] = c < n ? src[(long long)r * n + c] : (int8_t)0;
  }
}

int niti_launch_pad_pitch(niti_ctx *ctx, cudaStream_t st, const int8_t *src, int8_t *dst, int rows, int n, int pitch) {
  long long total = (long long)rows * pitch;
  pad_pitch_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(src, dst, rows, n, pitch);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

// Rounds acc[rows][32] (int32) and keeps the first k columns: out[rows][k].
__global__ void round_compact32_kernel(const int32_t *__restrict__ acc, const WsHeader *__restrict__ hdr,
                                       int8_t *__restrict__ out, int rows, int k, int mbits, int round_mode,
                                       int32_t *__restrict__ b_out) {
  const int b = niti_bitlen32(hdr->maxabs32);
  const int bp = b > mbits ? b - mbits : 0;
  const unsigned qmax = (1u << mbits) - 1u;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx == 0 && b_out) *b_out = b;
  if (idx < rows * k) {
    const int r = idx / k, c = idx % k;
    out[idx] = (int8_t)niti_round_i32(acc[r * 32 + c], bp, qmax, round_mode);
  }
}

int niti_launch_im2col32(niti_ctx *ctx, cudaStream_t st, const int8_t *x, int8_t *xcol, int B, int H, int W,
                         int Ci, int R, int S, int pad, int stride, int Ho, int Wo) {
  if (Ci == 3 && R == 3 && S == 3 && pad == 1 && stride == 1 && (W % 4) == 0 && (long long)B * H < (1LL << 31) &&
      ((uintptr_t)xcol & 31) == 0) {
    const int threads = W / 4 >= 128 ? 128 : (W / 4 > 32 ? 64 : 32);
    const size_t smem = (size_t)3 * (W * 3 / 4 + 2) * sizeof(unsigned);
    if (smem <= 48 * 1024) {
      im2col32_rgb3x3_kernel<<<(unsigned)(B * H), threads, smem, st>>>(x, xcol, B, H, W);
      ctx->launches++;
      NITI_CUDA_TRY(ctx, cudaGetLastError());
      return NITI_OK;
    }
  }
  long long M = (long long)B * Ho * Wo;
  long long blocks = (M + 255) / 256;
  if (blocks > (long long)ctx->sm_count * 16) blocks = (long long)ctx->sm_count * 16;
  im2col32_kernel<<<(unsigned)blocks, 256, 0, st>>>(x, xcol, B, H, W, Ci, R, S, pad, stride, Ho, Wo);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

int niti_launch_pad_rows32(niti_ctx *ctx, cudaStream_t st, const int8_t *w, int8_t *wcol, int rows, int k) {
  pad_rows32_kernel<<<(rows * 32 + 255) / 256, 256, 0, st>>>(w, wcol, rows, k);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

int niti_launch_round_compact32(niti_ctx *ctx, cudaStream_t st, const int32_t *acc, const WsHeader *hdr, int8_t *out,
                                int rows, int k, int mbits, int round_mode, int32_t *b_out) {
  round_compact32_kernel<<<(rows * k + 255) / 256, 256, 0, st>>>(acc, hdr, out, rows, k, mbits, round_mode, b_out);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

// ---------------------------------------------------------------------------------------------
// Integer cross-entropy gradient, Section 3.5.  Pass 1: one warp per sample computes the integer
// T_i (Eq. 2 or Eq. 3-4), their sum, the largest magnitude of e32 = T_i - [i == label] * sum
// (64-bit) and the arg-max hit.  Pass 2: shared binary point, e32 recomputed and rounded to int8.
// ---------------------------------------------------------------------------------------------
// One warp per sample.  Pass 1 keeps two 64-bit scalars per sample (the offset p of Eq. 4 and the
// sum of the T_i) instead of the T_i themselves; pass 2 recomputes T_i from the logit, which is a few
// integer operations, so that the only per-element traffic is the logit read twice and the int8
// result written once.
__device__ __forceinline__ long long warp_reduce_ll(long long v, int op /*0 sum,1 max,2 min*/) {
  for (int o = 16; o > 0; o >>= 1) {
    long long u = __shfl_xor_sync(0xffffffffu, v, o);
    v = op == 0 ? v + u : (op == 1 ? (u > v ? u : v) : (u < v ? u : v));
  }
  return v;
}
// x-hat of Eq. 3: (47274 * a) >> (15 - s), a left shift when s > 15
__device__ __forceinline__ long long xent_xhat(int a, long long sh_amt) {
  const long long P = 47274LL * (long long)a;
  return sh_amt >= 0 ? (P >> sh_amt) : P * (1LL << (-sh_amt));
}
// T_i of Eq. 2 (s <= -7) or Eq. 4
__device__ __forceinline__ long long xent_T(int a, int s, long long sh_amt, long long p) {
  if (s <= -7) {
    const long long ai = a;
    return (1LL << (1 - 2 * s)) + ai * (1LL << (1 - s)) + ai * ai;
  }
  const long long xt = xent_xhat(a, sh_amt) - p;
  return 1LL << (xt > 0 ? xt : 0);
}
constexpr int XENT_WARPS = 8;

__global__ void __launch_bounds__(32 * XENT_WARPS)
xent_row_kernel(const int8_t *__restrict__ a, const int32_t *__restrict__ s_a_ptr,
                const int32_t *__restrict__ labels, long long *__restrict__ rowinfo, WsHeader *hdr,
                int B, int N, uint32_t *__restrict__ status) {
  __shared__ unsigned long long sh_max[XENT_WARPS];
  __shared__ int sh_hit[XENT_WARPS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * XENT_WARPS + warp;
  const int s = *s_a_ptr;
  unsigned long long row_max = 0;
  int hit = 0;
  if (r < B) {
    const int label = labels[r];
    const int8_t *row = a + (long long)r * N;
    if (s < -22 || s > 24 || label < 0 || label >= N) {
      if (lane == 0) {
        atomicOr(status, (s < -22 || s > 24) ? NITI_DEV_XENT_RANGE : NITI_DEV_BAD_LABEL);
        rowinfo[2 * (long long)r] = 0;
        rowinfo[2 * (long long)r + 1] = 0;
      }
    } else {
      const long long LLMIN = -0x7fffffffffffffffLL - 1, LLMAX = 0x7fffffffffffffffLL;
      const long long sh_amt = 15 - (long long)s;
      long long p = 0;
      if (s > -7) {
        long long mx = LLMIN;
        for (int i = lane; i < N; i += 32) {
          const long long xh = xent_xhat(row[i], sh_amt);
          mx = xh > mx ? xh : mx;
        }
        mx = warp_reduce_ll(mx, 1);
        p = LLMAX;
        for (int i = lane; i < N; i += 32) {
          const long long xh = xent_xhat(row[i], sh_amt);
          if (xh > mx - 10 && xh < p) p = xh;
        }
        p = warp_reduce_ll(p, 2);
      }
      // sum of T_i, the largest T_i off the label, and the first arg-max of the row for the hit count
      long long csum = 0, t_other = 0;
      int best_v = -1000, best_i = 0x7fffffff;
      for (int i = lane; i < N; i += 32) {
        const int ai = row[i];
        const long long T = xent_T(ai, s, sh_amt, p);
        csum += T;
        if (i != label && T > t_other) t_other = T;
        if (ai > best_v) { best_v = ai; best_i = i; }
      }
      csum = warp_reduce_ll(csum, 0);
      t_other = warp_reduce_ll(t_other, 1);
      long long key = ((long long)(best_v + 1000) << 32) | (unsigned)(0x7fffffff - best_i);
      key = warp_reduce_ll(key, 1);
      // e32 = T_i off the label (positive) and T_label - sum (not positive) on it
      const long long t_label = xent_T(row[label], s, sh_amt, p);
      const long long on_label = csum - t_label;
      row_max = (unsigned long long)(t_other > on_label ? t_other : on_label);
      hit = (0x7fffffff - (int)(key & 0xffffffffLL)) == label ? 1 : 0;
      if (lane == 0) {
        rowinfo[2 * (long long)r] = p;
        rowinfo[2 * (long long)r + 1] = csum;
      }
    }
  }
  if (lane == 0) { sh_max[warp] = row_max; sh_hit[warp] = hit; }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long m = 0;
    int h = 0;
    for (int w = 0; w < XENT_WARPS; ++w) { m = sh_max[w] > m ? sh_max[w] : m; h += sh_hit[w]; }
    if (m > *(volatile unsigned long long *)&hdr->maxabs64) atomicMax(&hdr->maxabs64, m);
    if (h) atomicAdd(&hdr->hits, (unsigned)h);
  }
}

__global__ void __launch_bounds__(32 * XENT_WARPS)
xent_round_kernel(const int8_t *__restrict__ a, const int32_t *__restrict__ s_a_ptr,
                  const int32_t *__restrict__ labels, const long long *__restrict__ rowinfo,
                  const WsHeader *__restrict__ hdr, int8_t *__restrict__ out, int B, int N, int round_mode,
                  int32_t *__restrict__ b_out, int32_t *__restrict__ n_correct) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * XENT_WARPS + warp;
  const unsigned long long mxv = hdr->maxabs64;
  const int b = 64 - __clzll((long long)mxv);
  const int bp = b > 7 ? b - 7 : 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (b_out) *b_out = b;
    if (n_correct) *n_correct = (int32_t)hdr->hits;
  }
  if (r >= B) return;
  const int s = *s_a_ptr;
  const int label = labels[r];
  const int8_t *row = a + (long long)r * N;
  int8_t *orow = out + (long long)r * N;
  const bool bad = s < -22 || s > 24 || label < 0 || label >= N;
  const long long sh_amt = 15 - (long long)s;
  const long long p = rowinfo[2 * (long long)r], csum = rowinfo[2 * (long long)r + 1];
  auto one = [&](int i, int ai) -> int {
    if (bad) return 0;
    const long long v = xent_T(ai, s, sh_amt, p) - (i == label ? csum : 0);
    const unsigned long long m = v < 0 ? 0ull - (unsigned long long)v : (unsigned long long)v;
    const long long q = (long long)niti_round_mag<unsigned long long>(m, bp, 127ull, round_mode);
    return (int)(v < 0 ? -q : q);
  };
  if ((N & 3) == 0 && (((uintptr_t)a | (uintptr_t)out) & 3) == 0) {
    // four logits per lane per step: 128 contiguous bytes per warp instruction
    for (int i = 4 * lane; i < N; i += 128) {
      const unsigned w = *reinterpret_cast<const unsigned *>(row + i);
      unsigned o = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        o |= ((unsigned)one(i + k, (int)(int8_t)(w >> (8 * k))) & 0xffu) << (8 * k);
      *reinterpret_cast<unsigned *>(orow + i) = o;
    }
  } else {
    for (int i = lane; i < N; i += 32) orow[i] = (int8_t)one(i, row[i]);
  }
}

// ---- fast path (N % 4 == 0, 4-byte aligned rows): packed bytes and per-row tables ---------------
// T_i depends on the logit value alone once the row's offset p is known, and x-hat is monotone in
// the logit, so a row needs: the maxima of the logits before and after the label (packed byte max;
// they also decide the arg-max hit), for Eq. 2 the sums of a and a^2 (dp4a), for Eq. 3-4 the smallest
// logit whose x-hat exceeds max - 10 (a binary search over the 256 logit values gives the threshold,
// a packed min the logit) and the sum of T over a 256-entry table.  Pass 2 builds a 256-entry table
// of rounded results per row and looks every logit up; only the label element is computed apart.
__device__ __forceinline__ int hmax_s8x4(unsigned w) {
  const int b0 = (int)(int8_t)w, b1 = (int)(int8_t)(w >> 8), b2 = (int)(int8_t)(w >> 16), b3 = (int)(int8_t)(w >> 24);
  return max(max(b0, b1), max(b2, b3));
}
__device__ __forceinline__ int hmin_s8x4(unsigned w) {
  const int b0 = (int)(int8_t)w, b1 = (int)(int8_t)(w >> 8), b2 = (int)(int8_t)(w >> 16), b3 = (int)(int8_t)(w >> 24);
  return min(min(b0, b1), min(b2, b3));
}
__device__ __forceinline__ int warp_max_i(int v) {
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_min_i(int v) {
  for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_sum_i(int v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Tables for many rows (B >= XENT_TAB_MIN_ROWS).  The offset p of Eq. 4 is x-hat of one of the 256
// logit values, so there are at most 256 different T tables and, once the shared binary point is
// known, 256 different tables of rounded results: they are computed once per call (two launches of
// 256 x 256 threads) and a row copies the 512- or 256-byte line it needs instead of evaluating
// 2 x 256 64-bit expressions of its own.  ttab[i][v] = T(v - 128) with p = x-hat(i - 128) (16 bits:
// entries a row can use are at most 2^9); thr[t] = 128 + the smallest logit whose x-hat exceeds
// x-hat(t - 128) - 10; qtab[i][v] = T rounded with the shared binary point.  With tables the first
// scalar of a row is p * 256 + (index of its line).
constexpr int XENT_TAB_MIN_ROWS = 1024;
struct XentTables {
  unsigned short *ttab;
  unsigned char *qtab;
  unsigned char *thr;
};

__global__ void __launch_bounds__(256)
xent_ttab_kernel(const int32_t *__restrict__ s_a_ptr, XentTables t) {
  const int s = *s_a_ptr;
  if (s < -22 || s > 24 || s <= -7) return;             // (Eq. 2 needs no table of T)
  const long long sh_amt = 15 - (long long)s;
  const int i = blockIdx.x, v = threadIdx.x;
  const long long p = xent_xhat(i - 128, sh_amt);
  t.ttab[i * 256 + v] = (unsigned short)xent_T(v - 128, s, sh_amt, p);
  if (i == 0) {
    const long long mx = xent_xhat(v - 128, sh_amt);
    int lo = -128, hi = v - 128;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (xent_xhat(mid, sh_amt) > mx - 10) hi = mid; else lo = mid + 1;
    }
    t.thr[v] = (unsigned char)(lo + 128);
  }
}

__global__ void __launch_bounds__(256)
xent_qtab_kernel(const int32_t *__restrict__ s_a_ptr, const WsHeader *__restrict__ hdr, XentTables t, int round_mode) {
  const int s = *s_a_ptr;
  if (s < -22 || s > 24) return;
  const unsigned long long mxv = hdr->maxabs64;
  const int b = 64 - __clzll((long long)mxv);
  const int bp = b > 7 ? b - 7 : 0;
  const long long sh_amt = 15 - (long long)s;
  const int i = blockIdx.x, v = threadIdx.x;
  const long long p = s <= -7 ? 0 : xent_xhat(i - 128, sh_amt);
  const unsigned long long T = (unsigned long long)xent_T(v - 128, s, sh_amt, p);
  t.qtab[i * 256 + v] = (unsigned char)niti_round_mag<unsigned long long>(T, bp, 127ull, round_mode);
}

template <bool TAB>
__global__ void __launch_bounds__(32 * XENT_WARPS)
xent_row_fast_kernel(const int8_t *__restrict__ a, const int32_t *__restrict__ s_a_ptr,
                     const int32_t *__restrict__ labels, long long *__restrict__ rowinfo, WsHeader *hdr,
                     int B, int N, uint32_t *__restrict__ status, XentTables tabs) {
  __shared__ unsigned long long sh_max[XENT_WARPS];
  __shared__ int sh_hit[XENT_WARPS];
  __shared__ __align__(16) unsigned short sh_T[XENT_WARPS][256];     // T(a) of Eq. 4 for a = -128 .. 127 (at most 2^9)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * XENT_WARPS + warp;
  const int s = *s_a_ptr;
  unsigned long long row_max = 0;
  int hit = 0;
  if (r < B) {
    const int label = labels[r];
    if (s < -22 || s > 24 || label < 0 || label >= N) {
      if (lane == 0) {
        atomicOr(status, (s < -22 || s > 24) ? NITI_DEV_XENT_RANGE : NITI_DEV_BAD_LABEL);
        rowinfo[2 * (long long)r] = 0;
        rowinfo[2 * (long long)r + 1] = 0;
      }
    } else {
      const unsigned *row = reinterpret_cast<const unsigned *>(a + (long long)r * N);
      const int words = N >> 2, lw = label >> 2, lb = label & 3;
      const long long sh_amt = 15 - (long long)s;
      const int a_label = (int)a[(long long)r * N + label];
      // sweep 1: packed maxima before / after the label, sums of a and a^2
      unsigned mb = 0x80808080u, ma = 0x80808080u;
      int sum_a = 0, sum_q = 0;
      for (int wi = lane; wi < words; wi += 32) {
        const unsigned w = row[wi];
        sum_a = __dp4a((int)w, 0x01010101, sum_a);
        sum_q = __dp4a((int)w, (int)w, sum_q);
        if (wi < lw) mb = __vmaxs4(mb, w);
        else if (wi > lw) ma = __vmaxs4(ma, w);
        else {
          const unsigned low = lb == 0 ? 0u : (0xffffffffu >> (32 - 8 * lb));          // bytes before the label
          const unsigned high = lb == 3 ? 0u : (0xffffffffu << (8 * (lb + 1)));        // bytes after it
          mb = __vmaxs4(mb, (w & low) | (0x80808080u & ~low));
          ma = __vmaxs4(ma, (w & high) | (0x80808080u & ~high));
        }
      }
      const int max_before = warp_max_i(hmax_s8x4(mb)), max_after = warp_max_i(hmax_s8x4(ma));
      const int max_other = max(max_before, max_after);       // -128 when the row has one element
      const int row_top = max(max_other, a_label);
      hit = (a_label > max_before && a_label >= max_after) ? 1 : 0;   // the first arg-max is the label
      long long p = 0, csum, t_other, t_label;
      int line = 0;                                     // (TAB) the table line of this row
      if (s <= -7) {
        sum_a = warp_sum_i(sum_a);
        sum_q = warp_sum_i(sum_q);
        csum = (long long)N * (1LL << (1 - 2 * s)) + (long long)sum_a * (1LL << (1 - s)) + (long long)sum_q;
        t_other = N > 1 ? xent_T(max_other, s, sh_amt, 0) : 0;     // T is increasing in the logit
        t_label = xent_T(a_label, s, sh_amt, 0);
      } else {
        // smallest logit value whose x-hat exceeds mx - 10 (x-hat is non-decreasing in the logit)
        int lo = -128;
        if (TAB) {
          lo = (int)tabs.thr[row_top + 128] - 128;
        } else {
          const long long mx = xent_xhat(row_top, sh_amt);
          int hi = row_top;
          while (lo < hi) {
            const int mid = (lo + hi) >> 1;          // floor for negative sums as well
            if (xent_xhat(mid, sh_amt) > mx - 10) hi = mid; else lo = mid + 1;
          }
        }
        const unsigned thr4 = (unsigned)(lo & 0xff) * 0x01010101u;
        // sweep 2: the smallest logit of the row that is at least that value
        unsigned mn = 0x7f7f7f7fu;
        for (int wi = lane; wi < words; wi += 32) {
          const unsigned w = row[wi];
          const unsigned m = __vcmpges4(w, thr4);
          mn = __vmins4(mn, (w & m) | (0x7f7f7f7fu & ~m));
        }
        const int a_star = warp_min_i(hmin_s8x4(mn));
        p = xent_xhat(a_star, sh_amt);
        // table of T over the logit values, then sweep 3: the sum
        if (TAB) {
          reinterpret_cast<uint4 *>(sh_T[warp])[lane] =
              reinterpret_cast<const uint4 *>(tabs.ttab + (a_star + 128) * 256)[lane];
          line = a_star + 128;
        } else {
          for (int v = lane; v < 256; v += 32) sh_T[warp][v] = (unsigned short)xent_T(v - 128, s, sh_amt, p);
        }
        __syncwarp();
        int acc = 0;
        for (int wi = lane; wi < words; wi += 32) {
          const unsigned w = row[wi] ^ 0x80808080u;            // logit + 128 per byte
          acc += (int)sh_T[warp][w & 0xff] + (int)sh_T[warp][(w >> 8) & 0xff] + (int)sh_T[warp][(w >> 16) & 0xff] +
                 (int)sh_T[warp][w >> 24];
        }
        csum = (long long)warp_sum_i(acc);
        t_other = N > 1 ? (long long)sh_T[warp][max_other + 128] : 0;
        t_label = (long long)sh_T[warp][a_label + 128];
      }
      const long long on_label = csum - t_label;
      row_max = (unsigned long long)(t_other > on_label ? t_other : on_label);
      if (lane == 0) {
        rowinfo[2 * (long long)r] = TAB ? p * 256 + line : p;
        rowinfo[2 * (long long)r + 1] = csum;
      }
    }
  }
  if (lane == 0) { sh_max[warp] = row_max; sh_hit[warp] = hit; }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long m = 0;
    int h = 0;
    for (int w = 0; w < XENT_WARPS; ++w) { m = sh_max[w] > m ? sh_max[w] : m; h += sh_hit[w]; }
    if (m > *(volatile unsigned long long *)&hdr->maxabs64) atomicMax(&hdr->maxabs64, m);
    if (h) atomicAdd(&hdr->hits, (unsigned)h);
  }
}

template <bool TAB>
__global__ void __launch_bounds__(32 * XENT_WARPS)
xent_round_fast_kernel(const int8_t *__restrict__ a, const int32_t *__restrict__ s_a_ptr,
                       const int32_t *__restrict__ labels, const long long *__restrict__ rowinfo,
                       const WsHeader *__restrict__ hdr, int8_t *__restrict__ out, int B, int N, int round_mode,
                       int32_t *__restrict__ b_out, int32_t *__restrict__ n_correct, XentTables tabs) {
  __shared__ __align__(8) unsigned char sh_q[XENT_WARPS][256];        // rounded T(a) for a = -128 .. 127
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * XENT_WARPS + warp;
  const unsigned long long mxv = hdr->maxabs64;
  const int b = 64 - __clzll((long long)mxv);
  const int bp = b > 7 ? b - 7 : 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (b_out) *b_out = b;
    if (n_correct) *n_correct = (int32_t)hdr->hits;
  }
  if (r >= B) return;
  const int s = *s_a_ptr;
  const int label = labels[r];
  const unsigned *row = reinterpret_cast<const unsigned *>(a + (long long)r * N);
  unsigned *orow = reinterpret_cast<unsigned *>(out + (long long)r * N);
  const int words = N >> 2;
  if (s < -22 || s > 24 || label < 0 || label >= N) {
    for (int wi = lane; wi < words; wi += 32) orow[wi] = 0u;
    return;
  }
  const long long sh_amt = 15 - (long long)s;
  const long long info = rowinfo[2 * (long long)r], csum = rowinfo[2 * (long long)r + 1];
  const long long p = TAB ? (info >> 8) : info;
  // off the label e32 = T(a) > 0: one rounded value per logit value
  if (TAB) {
    reinterpret_cast<uint2 *>(sh_q[warp])[lane] =
        reinterpret_cast<const uint2 *>(tabs.qtab + (int)(info & 0xff) * 256)[lane];
  } else {
    for (int v = lane; v < 256; v += 32) {
      const unsigned long long T = (unsigned long long)xent_T(v - 128, s, sh_amt, p);
      sh_q[warp][v] = (unsigned char)niti_round_mag<unsigned long long>(T, bp, 127ull, round_mode);
    }
  }
  // on the label e32 = T - sum <= 0
  const int a_label = (int)a[(long long)r * N + label];
  const unsigned long long m_label = (unsigned long long)(csum - xent_T(a_label, s, sh_amt, p));
  const unsigned q_label = (unsigned)(0 - (int)niti_round_mag<unsigned long long>(m_label, bp, 127ull, round_mode)) & 0xffu;
  __syncwarp();
  const int lw = label >> 2, lb = label & 3;
  for (int wi = lane; wi < words; wi += 32) {
    const unsigned w = row[wi] ^ 0x80808080u;
    unsigned o = (unsigned)sh_q[warp][w & 0xff] | ((unsigned)sh_q[warp][(w >> 8) & 0xff] << 8) |
                 ((unsigned)sh_q[warp][(w >> 16) & 0xff] << 16) | ((unsigned)sh_q[warp][w >> 24] << 24);
    if (wi == lw) o = (o & ~(0xffu << (8 * lb))) | (q_label << (8 * lb));
    orow[wi] = o;
  }
}

// both passes; the packed path needs whole words per row
// (ctx may be null: the variant without a context; with one, the max magnitude of the 64-bit
// gradients is combined over the ranks between the two passes when a reduction hook is installed)
// tab_mem: 196864 bytes of scratch for the tables of many-row calls, or null
static int launch_xent(niti_ctx *ctx, cudaStream_t st, const int8_t *a, const int32_t *s_a, const int32_t *labels,
                       long long *rowinfo, WsHeader *hdr, int8_t *e, int32_t *b_e, int32_t *n_correct, int B, int N,
                       int round_mode, uint32_t *status, void *tab_mem) {
  const unsigned blocks = (unsigned)((B + XENT_WARPS - 1) / XENT_WARPS);
  const bool packed = (N & 3) == 0 && N >= 64 && (((uintptr_t)a | (uintptr_t)e) & 3) == 0;
  const bool tab = packed && tab_mem != nullptr && B >= XENT_TAB_MIN_ROWS;
  XentTables t = {nullptr, nullptr, nullptr};
  if (tab) {
    t.ttab = (unsigned short *)tab_mem;
    t.qtab = (unsigned char *)tab_mem + 256 * 256 * 2;
    t.thr = t.qtab + 256 * 256;
    xent_ttab_kernel<<<256, 256, 0, st>>>(s_a, t);
    xent_row_fast_kernel<true><<<blocks, 32 * XENT_WARPS, 0, st>>>(a, s_a, labels, rowinfo, hdr, B, N, status, t);
  } else if (packed) {
    xent_row_fast_kernel<false><<<blocks, 32 * XENT_WARPS, 0, st>>>(a, s_a, labels, rowinfo, hdr, B, N, status, t);
  } else {
    xent_row_kernel<<<blocks, 32 * XENT_WARPS, 0, st>>>(a, s_a, labels, rowinfo, hdr, B, N, status);
  }
  if (ctx) {
    int rc = niti_reduce(ctx, st, &hdr->maxabs64, 1, NITI_REDUCE_MAX_U64);
    if (rc != NITI_OK) return rc;
  }
  if (tab) {
    xent_qtab_kernel<<<256, 256, 0, st>>>(s_a, hdr, t, round_mode);
    xent_round_fast_kernel<true><<<blocks, 32 * XENT_WARPS, 0, st>>>(a, s_a, labels, rowinfo, hdr, e, B, N, round_mode, b_e, n_correct, t);
    if (ctx) ctx->launches += 2;
  } else if (packed) {
    xent_round_fast_kernel<false><<<blocks, 32 * XENT_WARPS, 0, st>>>(a, s_a, labels, rowinfo, hdr, e, B, N, round_mode, b_e, n_correct, t);
  } else {
    xent_round_kernel<<<blocks, 32 * XENT_WARPS, 0, st>>>(a, s_a, labels, rowinfo, hdr, e, B, N, round_mode, b_e, n_correct);
  }
  return NITI_OK;
}

extern "C" int niti_int_xent(niti_ctx *ctx, void *stream, const int8_t *a, const int32_t *s_a,
                             const int32_t *labels, int8_t *e, int32_t *b_e, int32_t *n_correct,
                             int B, int N, int round_mode, void *ws, size_t ws_bytes) {
  if (!ctx) return NITI_ERR_ARG;
  if (!a || !s_a || !labels || !e || B <= 0 || N <= 0 || N > 65536 || (round_mode != 0 && round_mode != 1))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_int_xent: bad argument");
  int64_t dims[2] = {B, N};
  if (!ws || ((uintptr_t)ws & 255) || ws_bytes < niti_workspace_bytes(NITI_OP_INT_XENT, dims, 2))
    return niti_fail(ctx, NITI_ERR_WORKSPACE, "niti_int_xent: workspace missing, misaligned or too small");
  cudaStream_t st = (cudaStream_t)stream;
  WsHeader *hdr = nullptr;
  long long *rowinfo = (long long *)((char *)ws + NITI_WS_HEADER);
  const int rch = niti_take_header(ctx, st, ws, &hdr);
  if (rch != NITI_OK) return rch;
  void *tab_mem = (char *)ws + NITI_WS_HEADER + ((size_t)B * 16 + 255) / 256 * 256;
  int rcx = launch_xent(ctx, st, a, s_a, labels, rowinfo, hdr, e, b_e, n_correct, B, N, round_mode, ctx->d_status, tab_mem);
  if (rcx != NITI_OK) return rcx;
  ctx->launches += 2;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

// ---------------------------------------------------------------------------------------------
// niti_int_xent_noalloc: the same two kernels with their scratch (reduction header + two 64-bit
// scalars per sample) in a fixed device array that is part of the library image, for callers that must
// not allocate device memory.  Every GPU that loads the library carries the array until exit.
// ---------------------------------------------------------------------------------------------
#define NITI_NOALLOC_HEADER 256       // reduction scalars of this variant (its last word: status bits)
#define NITI_NOALLOC_BYTES (NITI_NOALLOC_HEADER + 8 * NITI_XENT_NOALLOC_MAX_ELEMS)
static __device__ __align__(256) unsigned char g_xent_scratch[NITI_NOALLOC_BYTES];
// The name above is only a host-side handle in host code; the device address is looked up once per
// device (with that device current) and cached here.
static void *g_xent_scratch_addr[64];
static std::mutex g_xent_scratch_mutex;

extern "C" int niti_int_xent_noalloc(void *stream, const int8_t *a, const int32_t *s_a, const int32_t *labels,
                                     int8_t *e, int32_t *b_e, int32_t *n_correct, int B, int N, int round_mode) {
  if (!a || !s_a || !labels || !e || B <= 0 || N <= 0 || N > 65536 || (round_mode != 0 && round_mode != 1))
    return NITI_ERR_ARG;
  if ((long long)B * N > NITI_XENT_NOALLOC_MAX_ELEMS || B > NITI_XENT_NOALLOC_MAX_ELEMS / 2)
    return NITI_ERR_TOO_LARGE;                   // 16 bytes of scratch per sample must fit the array
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return NITI_ERR_CUDA;
  void *base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_xent_scratch_mutex);
    if (!g_xent_scratch_addr[dev]) {
      void *ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_xent_scratch) != cudaSuccess || !ptr) return NITI_ERR_CUDA;
      g_xent_scratch_addr[dev] = ptr;
    }
    base = g_xent_scratch_addr[dev];
  }
  cudaStream_t st = (cudaStream_t)stream;
  WsHeader *hdr = (WsHeader *)base;
  long long *rowinfo = (long long *)((char *)base + NITI_NOALLOC_HEADER);
  // the array keeps what the previous call left: the reduction scalars must start at zero.  The last
  // word of the header takes the (unreported) status bits of this variant.
  uint32_t *status = (uint32_t *)((char *)base + NITI_NOALLOC_HEADER - sizeof(uint32_t));
  if (cudaMemsetAsync(base, 0, NITI_NOALLOC_HEADER, st) != cudaSuccess) return NITI_ERR_CUDA;
  launch_xent(nullptr, st, a, s_a, labels, rowinfo, hdr, e, b_e, n_correct, B, N, round_mode, status, nullptr);
  if (cudaGetLastError() != cudaSuccess) return NITI_ERR_CUDA;
  return NITI_OK;
}

// ---------------------------------------------------------------------------------------------
// Byte-wise SIMD elementwise ops: 16 int8 per thread per iteration (one 16-byte load per operand).
// ---------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(256)
sgd_update_kernel(int8_t *__restrict__ w, const int8_t *__restrict__ g, long long n) {
  const long long nvec = n >> 4;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (long long v = tid; v < nvec; v += stride) {
    int4 wv = *(reinterpret_cast<int4 *>(w) + v);
    int4 gv = __ldcs(reinterpret_cast<const int4 *>(g) + v);
    wv.x = sat_sub_clamp127(wv.x, gv.x); wv.y = sat_sub_clamp127(wv.y, gv.y);
    wv.z = sat_sub_clamp127(wv.z, gv.z); wv.w = sat_sub_clamp127(wv.w, gv.w);
    *(reinterpret_cast<int4 *>(w) + v) = wv;
  }
  long long t = (nvec << 4) + tid;
  if (t < n) {
    int d = (int)w[t] - (int)g[t];
    d = d > 127 ? 127 : (d < -127 ? -127 : d);
    w[t] = (int8_t)d;
  }
}

__global__ void __launch_bounds__(256)
relu_fwd_kernel(const int8_t *__restrict__ x, int8_t *__restrict__ y, long long n) {
  const long long nvec = n >> 4;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (long long v = tid; v < nvec; v += stride) {
    int4 xv = *(reinterpret_cast<const int4 *>(x) + v);
    xv.x = __vmaxs4(xv.x, 0); xv.y = __vmaxs4(xv.y, 0); xv.z = __vmaxs4(xv.z, 0); xv.w = __vmaxs4(xv.w, 0);
    *(reinterpret_cast<int4 *>(y) + v) = xv;
  }
  long long t = (nvec << 4) + tid;
  if (t < n) y[t] = x[t] > 0 ? x[t] : 0;
}

__global__ void __launch_bounds__(256)
relu_bwd_kernel(const int8_t *__restrict__ y, const int8_t *__restrict__ eo, int8_t *__restrict__ ei,
                long long n) {
  const long long nvec = n >> 4;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (long long v = tid; v < nvec; v += stride) {
    int4 yv = *(reinterpret_cast<const int4 *>(y) + v);
    int4 ev = *(reinterpret_cast<const int4 *>(eo) + v);
    ev.x &= __vcmpgts4(yv.x, 0); ev.y &= __vcmpgts4(yv.y, 0);
    ev.z &= __vcmpgts4(yv.z, 0); ev.w &= __vcmpgts4(yv.w, 0);
    *(reinterpret_cast<int4 *>(ei) + v) = ev;
  }
  long long t = (nvec << 4) + tid;
  if (t < n) ei[t] = y[t] > 0 ? eo[t] : 0;
}

// 2x2 max-pool, NHWC.  VEC = 16: one thread per 16 channels of one output pixel; VEC = 1: scalar.
template <int VEC>
__global__ void __launch_bounds__(256)
maxpool2_fwd_kernel(const int8_t *__restrict__ x, int8_t *__restrict__ y, int B, int H, int W, int C) {
  const int Ho = H >> 1, Wo = W >> 1, Cv = C / VEC;
  const long long total = (long long)B * Ho * Wo * Cv;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    int cv = (int)(t % Cv);
    long long pix = t / Cv;
    int j = (int)(pix % Wo);
    long long bi = pix / Wo;
    int i = (int)(bi % Ho);
    long long b = bi / Ho;
    long long base = (((b * H + 2 * i) * W + 2 * j) * (long long)C) + (long long)cv * VEC;
    long long rs = (long long)W * C;
    if (VEC == 16) {
      int4 v0 = *reinterpret_cast<const int4 *>(x + base);
      int4 v1 = *reinterpret_cast<const int4 *>(x + base + C);
      int4 v2 = *reinterpret_cast<const int4 *>(x + base + rs);
      int4 v3 = *reinterpret_cast<const int4 *>(x + base + rs + C);
      int4 m;
      m.x = __vmaxs4(__vmaxs4(v0.x, v1.x), __vmaxs4(v2.x, v3.x));
      m.y = __vmaxs4(__vmaxs4(v0.y, v1.y), __vmaxs4(v2.y, v3.y));
      m.z = __vmaxs4(__vmaxs4(v0.z, v1.z), __vmaxs4(v2.z, v3.z));
      m.w = __vmaxs4(__vmaxs4(v0.w, v1.w), __vmaxs4(v2.w, v3.w));
      *reinterpret_cast<int4 *>(y + pix * C + (long long)cv * VEC) = m;
    } else {
      int8_t m = x[base];
      int8_t v = x[base + C]; m = v > m ? v : m;
      v = x[base + rs]; m = v > m ? v : m;
      v = x[base + rs + C]; m = v > m ? v : m;
      y[pix * C + cv] = m;
    }
  }
}

__device__ __forceinline__ void pool_bwd_word(unsigned x0, unsigned x1, unsigned x2, unsigned x3,
                                              unsigned e, int relu, unsigned &o0, unsigned &o1,
                                              unsigned &o2, unsigned &o3) {
  unsigned m = __vmaxs4(__vmaxs4(x0, x1), __vmaxs4(x2, x3));
  unsigned s0 = __vcmpeq4(x0, m);
  unsigned s1 = __vcmpeq4(x1, m) & ~s0;
  unsigned s2 = __vcmpeq4(x2, m) & ~(s0 | s1);
  unsigned s3 = ~(s0 | s1 | s2);
  if (relu) {
    unsigned pos = __vcmpgts4(m, 0);   // the routed position holds the maximum
    e &= pos;
  }
  o0 = e & s0; o1 = e & s1; o2 = e & s2; o3 = e & s3;
}

template <int VEC>
__global__ void __launch_bounds__(256)
maxpool2_bwd_kernel(const int8_t *__restrict__ x, const int8_t *__restrict__ eo,
                    int8_t *__restrict__ ei, int B, int H, int W, int C, int relu) {
  const int Ho = H >> 1, Wo = W >> 1, Cv = C / VEC;
  const long long total = (long long)B * Ho * Wo * Cv;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    int cv = (int)(t % Cv);
    long long pix = t / Cv;
    int j = (int)(pix % Wo);
    long long bi = pix / Wo;
    int i = (int)(bi % Ho);
    long long b = bi / Ho;
    long long base = (((b * H + 2 * i) * W + 2 * j) * (long long)C) + (long long)cv * VEC;
    long long rs = (long long)W * C;
    if (VEC == 16) {
      int4 v0 = *reinterpret_cast<const int4 *>(x + base);
      int4 v1 = *reinterpret_cast<const int4 *>(x + base + C);
      int4 v2 = *reinterpret_cast<const int4 *>(x + base + rs);
      int4 v3 = *reinterpret_cast<const int4 *>(x + base + rs + C);
      int4 e = *reinterpret_cast<const int4 *>(eo + pix * C + (long long)cv * VEC);
      int4 o0, o1, o2, o3;
      pool_bwd_word(v0.x, v1.x, v2.x, v3.x, e.x, relu, (unsigned &)o0.x, (unsigned &)o1.x, (unsigned &)o2.x, (unsigned &)o3.x);
      pool_bwd_word(v0.y, v1.y, v2.y, v3.y, e.y, relu, (unsigned &)o0.y, (unsigned &)o1.y, (unsigned &)o2.y, (unsigned &)o3.y);
      pool_bwd_word(v0.z, v1.z, v2.z, v3.z, e.z, relu, (unsigned &)o0.z, (unsigned &)o1.z, (unsigned &)o2.z, (unsigned &)o3.z);
      pool_bwd_word(v0.w, v1.w, v2.w, v3.w, e.w, relu, (unsigned &)o0.w, (unsigned &)o1.w, (unsigned &)o2.w, (unsigned &)o3.w);
      *reinterpret_cast<int4 *>(ei + base) = o0;
      *reinterpret_cast<int4 *>(ei + base + C) = o1;
      *reinterpret_cast<int4 *>(ei + base + rs) = o2;
      *reinterpret_cast<int4 *>(ei + base + rs + C) = o3;
    } else {
      long long idx[4] = {base, base + C, base + rs, base + rs + C};
      int best = 0;
      for (int k = 1; k < 4; ++k)
        if (x[idx[k]] > x[idx[best]]) best = k;
      int8_t e = eo[pix * C + cv];
      if (relu && x[idx[best]] <= 0) e = 0;
      for (int k = 0; k < 4; ++k) ei[idx[k]] = k == best ? e : (int8_t)0;
    }
  }
}

// ---- max-pool that records where the maximum was --------------------------------------------
// The backward pass of a 2x2 max-pool needs, per output element, the position of the first maximum
// of its window and (behind a ReLU) whether that maximum was positive: four bits.  Recording them in
// the forward pass (half a byte per output element) lets the backward pass read the error and the
// codes instead of the whole input tensor: 1.25 + 0.5/4 bytes per input element instead of 2.25.
// Code of one element: bits 0-1 = position (0: (0,0), 1: (0,1), 2: (1,0), 3: (1,1)), bit 2 = max > 0.
// Layout: [B][H/2][W/2][C/2] bytes, channel c in the low (c even) or high (c odd) nibble.
__device__ __forceinline__ unsigned pool_codes_word(unsigned x0, unsigned x1, unsigned x2, unsigned x3, unsigned &m) {
  m = __vmaxs4(__vmaxs4(x0, x1), __vmaxs4(x2, x3));
  const unsigned s0 = __vcmpeq4(x0, m);
  const unsigned s1 = __vcmpeq4(x1, m) & ~s0;
  const unsigned s2 = __vcmpeq4(x2, m) & ~(s0 | s1);
  const unsigned s3 = ~(s0 | s1 | s2);
  const unsigned pos = __vcmpgts4(m, 0);
  return (s1 & 0x01010101u) | (s2 & 0x02020202u) | (s3 & 0x03030303u) | (pos & 0x04040404u);
}
// four byte codes (one per byte) -> 16 bits of nibbles, and back
__device__ __forceinline__ unsigned pool_pack_nibbles(unsigned w) {
  const unsigned t = (w | (w >> 4)) & 0x00ff00ffu;
  return (t | (t >> 8)) & 0xffffu;
}
__device__ __forceinline__ unsigned pool_unpack_nibbles(unsigned p16) {
  const unsigned t = (p16 | (p16 << 8)) & 0x00ff00ffu;
  return (t | (t << 4)) & 0x0f0f0f0fu;
}

__global__ void __launch_bounds__(256)
maxpool2_fwd_idx_kernel(const int8_t *__restrict__ x, int8_t *__restrict__ y, uint8_t *__restrict__ idx, int B, int H,
                        int W, int C) {
  const int Ho = H >> 1, Wo = W >> 1, Cv = C / 16;
  const long long total = (long long)B * Ho * Wo * Cv;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const int cv = (int)(t % Cv);
    const long long pix = t / Cv;
    const int j = (int)(pix % Wo);
    const long long bi = pix / Wo;
    const int i = (int)(bi % Ho);
    const long long b = bi / Ho;
    const long long base = (((b * H + 2 * i) * W + 2 * j) * (long long)C) + (long long)cv * 16;
    const long long rs = (long long)W * C;
    const int4 v0 = *reinterpret_cast<const int4 *>(x + base);
    const int4 v1 = *reinterpret_cast<const int4 *>(x + base + C);
    const int4 v2 = *reinterpret_cast<const int4 *>(x + base + rs);
    const int4 v3 = *reinterpret_cast<const int4 *>(x + base + rs + C);
    int4 m;
    const unsigned c0 = pool_codes_word(v0.x, v1.x, v2.x, v3.x, (unsigned &)m.x);
    const unsigned c1 = pool_codes_word(v0.y, v1.y, v2.y, v3.y, (unsigned &)m.y);
    const unsigned c2 = pool_codes_word(v0.z, v1.z, v2.z, v3.z, (unsigned &)m.z);
    const unsigned c3 = pool_codes_word(v0.w, v1.w, v2.w, v3.w, (unsigned &)m.w);
    *reinterpret_cast<int4 *>(y + pix * C + (long long)cv * 16) = m;
    uint2 packed;
    packed.x = pool_pack_nibbles(c0) | (pool_pack_nibbles(c1) << 16);
    packed.y = pool_pack_nibbles(c2) | (pool_pack_nibbles(c3) << 16);
    *reinterpret_cast<uint2 *>(idx + (pix * C >> 1) + (long long)cv * 8) = packed;
  }
}

__device__ __forceinline__ void pool_route_word(unsigned codes, unsigned e, int relu, unsigned &o0, unsigned &o1,
                                                unsigned &o2, unsigned &o3) {
  const unsigned pos2 = codes & 0x03030303u;
  if (relu) e &= __vcmpne4(codes & 0x04040404u, 0u);
  o0 = e & __vcmpeq4(pos2, 0u);
  o1 = e & __vcmpeq4(pos2, 0x01010101u);
  o2 = e & __vcmpeq4(pos2, 0x02020202u);
  o3 = e & __vcmpeq4(pos2, 0x03030303u);
}

__global__ void __launch_bounds__(256)
maxpool2_bwd_idx_kernel(const int8_t *__restrict__ eo, const uint8_t *__restrict__ idx, int8_t *__restrict__ ei, int B,
                        int H, int W, int C, int relu) {
  const int Ho = H >> 1, Wo = W >> 1, Cv = C / 16;
  const long long total = (long long)B * Ho * Wo * Cv;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const int cv = (int)(t % Cv);
    const long long pix = t / Cv;
    const int j = (int)(pix % Wo);
    const long long bi = pix / Wo;
    const int i = (int)(bi % Ho);
    const long long b = bi / Ho;
    const long long base = (((b * H + 2 * i) * W + 2 * j) * (long long)C) + (long long)cv * 16;
    const long long rs = (long long)W * C;
    const int4 e = __ldcs(reinterpret_cast<const int4 *>(eo + pix * C + (long long)cv * 16));
    const uint2 packed = __ldcs(reinterpret_cast<const uint2 *>(idx + (pix * C >> 1) + (long long)cv * 8));
    int4 o0, o1, o2, o3;
    pool_route_word(pool_unpack_nibbles(packed.x & 0xffffu), e.x, relu, (unsigned &)o0.x, (unsigned &)o1.x, (unsigned &)o2.x, (unsigned &)o3.x);
    pool_route_word(pool_unpack_nibbles(packed.x >> 16), e.y, relu, (unsigned &)o0.y, (unsigned &)o1.y, (unsigned &)o2.y, (unsigned &)o3.y);
    pool_route_word(pool_unpack_nibbles(packed.y & 0xffffu), e.z, relu, (unsigned &)o0.z, (unsigned &)o1.z, (unsigned &)o2.z, (unsigned &)o3.z);
    pool_route_word(pool_unpack_nibbles(packed.y >> 16), e.w, relu, (unsigned &)o0.w, (unsigned &)o1.w, (unsigned &)o2.w, (unsigned &)o3.w);
    *reinterpret_cast<int4 *>(ei + base) = o0;
    *reinterpret_cast<int4 *>(ei + base + C) = o1;
    *reinterpret_cast<int4 *>(ei + base + rs) = o2;
    *reinterpret_cast<int4 *>(ei + base + rs + C) = o3;
  }
}

static inline unsigned ew_blocks(niti_ctx *ctx, long long work_items) {
  long long blocks = (work_items + 255) / 256;
  long long cap = (long long)ctx->sm_count * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (unsigned)blocks;
}

int niti_launch_sgd_update(niti_ctx *ctx, cudaStream_t st, int8_t *w, const int8_t *g, long long n) {
  sgd_update_kernel<<<ew_blocks(ctx, (n >> 4) + 16), 256, 0, st>>>(w, g, n);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

extern "C" int niti_int_sgd_update(niti_ctx *ctx, void *stream, int8_t *w, const int8_t *g, int64_t n) {
  if (!ctx) return NITI_ERR_ARG;
  if (!w || !g || n <= 0) return niti_fail(ctx, NITI_ERR_ARG, "niti_int_sgd_update: bad argument");
  if (((uintptr_t)w | (uintptr_t)g) & 15)
    return niti_fail(ctx, NITI_ERR_ARG, "niti_int_sgd_update: pointers must be 16-byte aligned");
  sgd_update_kernel<<<ew_blocks(ctx, (n >> 4) + 16), 256, 0, (cudaStream_t)stream>>>(w, g, n);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

extern "C" int niti_relu_fwd(niti_ctx *ctx, void *stream, const int8_t *x, int8_t *y, int64_t n) {
  if (!ctx) return NITI_ERR_ARG;
  if (!x || !y || n <= 0 || (((uintptr_t)x | (uintptr_t)y) & 15))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_relu_fwd: bad argument");
  relu_fwd_kernel<<<ew_blocks(ctx, (n >> 4) + 16), 256, 0, (cudaStream_t)stream>>>(x, y, n);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

extern "C" int niti_relu_bwd(niti_ctx *ctx, void *stream, const int8_t *y, const int8_t *e_out,
                             int8_t *e_in, int64_t n) {
  if (!ctx) return NITI_ERR_ARG;
  if (!y || !e_out || !e_in || n <= 0 || (((uintptr_t)y | (uintptr_t)e_out | (uintptr_t)e_in) & 15))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_relu_bwd: bad argument");
  relu_bwd_kernel<<<ew_blocks(ctx, (n >> 4) + 16), 256, 0, (cudaStream_t)stream>>>(y, e_out, e_in, n);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

int niti_launch_maxpool2_fwd(niti_ctx *ctx, cudaStream_t st, const int8_t *x, int8_t *y, int B, int H, int W, int C) {
  bool vec = (C % 16 == 0) && !(((uintptr_t)x | (uintptr_t)y) & 15);
  long long items = (long long)B * (H / 2) * (W / 2) * (vec ? C / 16 : C);
  if (vec)
    maxpool2_fwd_kernel<16><<<ew_blocks(ctx, items), 256, 0, st>>>(x, y, B, H, W, C);
  else
    maxpool2_fwd_kernel<1><<<ew_blocks(ctx, items), 256, 0, st>>>(x, y, B, H, W, C);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

extern "C" int niti_maxpool2_fwd(niti_ctx *ctx, void *stream, const int8_t *x, int8_t *y, int B, int H,
                                 int W, int C) {
  if (!ctx) return NITI_ERR_ARG;
  if (!x || !y || B <= 0 || H <= 0 || W <= 0 || C <= 0 || (H & 1) || (W & 1))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_maxpool2_fwd: bad argument (H and W must be even)");
  return niti_launch_maxpool2_fwd(ctx, (cudaStream_t)stream, x, y, B, H, W, C);
}

extern "C" int niti_maxpool2_fwd_idx(niti_ctx *ctx, void *stream, const int8_t *x, int8_t *y, uint8_t *idx, int B,
                                     int H, int W, int C) {
  if (!ctx) return NITI_ERR_ARG;
  if (!x || !y || !idx || B <= 0 || H <= 0 || W <= 0 || C <= 0 || (H & 1) || (W & 1))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_maxpool2_fwd_idx: bad argument (H and W must be even)");
  if ((C % 16) != 0 || (((uintptr_t)x | (uintptr_t)y) & 15) || ((uintptr_t)idx & 7))
    return niti_fail(ctx, NITI_ERR_SHAPE, "niti_maxpool2_fwd_idx: C must be a multiple of 16 and the tensors aligned");
  const long long items = (long long)B * (H / 2) * (W / 2) * (C / 16);
  maxpool2_fwd_idx_kernel<<<ew_blocks(ctx, items), 256, 0, (cudaStream_t)stream>>>(x, y, idx, B, H, W, C);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

extern "C" int niti_maxpool2_bwd_idx(niti_ctx *ctx, void *stream, const int8_t *e_out, const uint8_t *idx,
                                     int8_t *e_in, int B, int H, int W, int C, int relu) {
  if (!ctx) return NITI_ERR_ARG;
  if (!e_out || !idx || !e_in || B <= 0 || H <= 0 || W <= 0 || C <= 0 || (H & 1) || (W & 1))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_maxpool2_bwd_idx: bad argument (H and W must be even)");
  if ((C % 16) != 0 || (((uintptr_t)e_out | (uintptr_t)e_in) & 15) || ((uintptr_t)idx & 7))
    return niti_fail(ctx, NITI_ERR_SHAPE, "niti_maxpool2_bwd_idx: C must be a multiple of 16 and the tensors aligned");
  const long long items = (long long)B * (H / 2) * (W / 2) * (C / 16);
  maxpool2_bwd_idx_kernel<<<ew_blocks(ctx, items), 256, 0, (cudaStream_t)stream>>>(e_out, idx, e_in, B, H, W, C, relu);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

extern "C" int niti_maxpool2_bwd(niti_ctx *ctx, void *stream, const int8_t *x, const int8_t *e_out,
                                 int8_t *e_in, int B, int H, int W, int C, int relu) {
  if (!ctx) return NITI_ERR_ARG;
  if (!x || !e_out || !e_in || B <= 0 || H <= 0 || W <= 0 || C <= 0 || (H & 1) || (W & 1))
    return niti_fail(ctx, NITI_ERR_ARG, "niti_maxpool2_bwd: bad argument (H and W must be even)");
  bool vec = (C % 16 == 0) && !(((uintptr_t)x | (uintptr_t)e_out | (uintptr_t)e_in) & 15);
  long long items = (long long)B * (H / 2) * (W / 2) * (vec ? C / 16 : C);
  if (vec)
    maxpool2_bwd_kernel<16><<<ew_blocks(ctx, items), 256, 0, (cudaStream_t)stream>>>(x, e_out, e_in, B, H, W, C, relu);
  else
    maxpool2_bwd_kernel<1><<<ew_blocks(ctx, items), 256, 0, (cudaStream_t)stream>>>(x, e_out, e_in, B, H, W, C, relu);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}
