// Plain CUDA-core matrix-multiply engine (dp4a) with implicit operand addressing.
//
// It serves the shapes the tensor-core engine does not take (tiny or oddly strided operands:
// 10-class heads, 1- and 3-channel inputs, general R x S / pad) and lets the tests cross-check the
// two engines against each other.  D[m][n] = sum_k A(m,k) * B(n,k), int8 x int8 -> int32
// (Int8MatrixMultiply of Algorithm 1), for the six operand mappings in NitiGemmKind.
#include "niti_common.cuh"

namespace {

constexpr int TM = 64, TN = 64, TK = 32;   // block tile; 256 threads, 4x4 outputs per thread

struct Addr {
  const int8_t *p0, *p1;
  int kind;
  int M, N, K;                                  // fully connected dims
  int H, W, Ho, Wo, Ci, Co, R, S, pad, stride;  // convolution dims
  long long gm, gn, gk;
  long long pitch0;                             // row pitch of p0 for the fully connected backward kinds
};

// element A(m, k) of the implicit left operand, 0 outside the problem
__device__ __forceinline__ int8_t load_a(const Addr &q, long long m, long long k) {
  if (m >= q.gm || k >= q.gk) return 0;
  switch (q.kind) {
    case GK_FC_FWD: return q.p0[m * q.K + k];
    case GK_FC_DGRAD: return q.p0[m * q.pitch0 + k];          // e[m][n], k == n
    case GK_FC_WGRAD: return q.p0[k * q.pitch0 + m];          // e[mm][n], m == n, k == mm
    case GK_CONV_FWD: {
      int ci = (int)(k % q.Ci);
      int rs = (int)(k / q.Ci);
      int s = rs % q.S, r = rs / q.S;
      int j = (int)(m % q.Wo);
      long long t = m / q.Wo;
      int i = (int)(t % q.Ho);
      long long b = t / q.Ho;
      int ii = i * q.stride + r - q.pad, jj = j * q.stride + s - q.pad;
      if (ii < 0 || ii >= q.H || jj < 0 || jj >= q.W) return 0;
      return q.p0[((b * q.H + ii) * q.W + jj) * q.Ci + ci];
    }
    case GK_CONV_DGRAD: {
      int co = (int)(k % q.Co);
      int rs = (int)(k / q.Co);
      int s = rs % q.S, r = rs / q.S;
      int jj = (int)(m % q.W);
      long long t = m / q.W;
      int ii = (int)(t % q.H);
      long long b = t / q.H;
      // the output pixel (i, j) whose window puts tap (r, s) on this input pixel, if there is one
      int ti = ii - r + q.pad, tj = jj - s + q.pad;
      if (ti < 0 || tj < 0) return 0;
      int i = ti, j = tj;
      if (q.stride > 1) {
        i = ti / q.stride; j = tj / q.stride;
        if (i * q.stride != ti || j * q.stride != tj) return 0;
      }
      if (i >= q.Ho || j >= q.Wo) return 0;
      return q.p0[((b * q.Ho + i) * q.Wo + j) * q.Co + co];
    }
    default: /* GK_CONV_WGRAD */ return q.p0[k * q.Co + m];   // e[pix][co]
  }
}

// element B(n, k) of the implicit right operand
__device__ __forceinline__ int8_t load_b(const Addr &q, long long n, long long k) {
  if (n >= q.gn || k >= q.gk) return 0;
  switch (q.kind) {
    case GK_FC_FWD: return q.p1[n * q.K + k];
    case GK_FC_DGRAD: return q.p1[k * q.K + n];               // w[nn][k'], n == k', k == nn
    case GK_FC_WGRAD: return q.p1[k * q.K + n];               // a[mm][k'], n == k', k == mm
    case GK_CONV_FWD: return q.p1[n * q.gk + k];
    case GK_CONV_DGRAD: {
      int co = (int)(k % q.Co);
      int rs = (int)(k / q.Co);
      return q.p1[((long long)co * q.R * q.S + rs) * q.Ci + n];
    }
    default: { /* GK_CONV_WGRAD: n = (r, s, ci), k = pixel */
      int ci = (int)(n % q.Ci);
      int rs = (int)(n / q.Ci);
      int s = rs % q.S, r = rs / q.S;
      int j = (int)(k % q.Wo);
      long long t = k / q.Wo;
      int i = (int)(t % q.Ho);
      long long b = t / q.Ho;
      int ii = i * q.stride + r - q.pad, jj = j * q.stride + s - q.pad;
      if (ii < 0 || ii >= q.H || jj < 0 || jj >= q.W) return 0;
      return q.p1[((b * q.H + ii) * q.W + jj) * q.Ci + ci];
    }
  }
}

// SPLIT: gridDim.z slices of the contraction, partial sums added with integer atomics (exact and
// order-independent); the max is then taken by a separate pass.
template <bool SPLIT>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(Addr q, int32_t *__restrict__ acc, WsHeader *hdr, long long k_per_split) {
  __shared__ int As[TM][TK / 4 + 1];
  __shared__ int Bs[TN][TK / 4 + 1];
  __shared__ unsigned smax[8];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const long long m0 = (long long)blockIdx.y * TM, n0 = (long long)blockIdx.x * TN;
  const long long k_begin = (long long)blockIdx.z * k_per_split;
  long long k_end = k_begin + k_per_split;
  if (k_end > q.gk) k_end = q.gk;
  int c[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) c[i][j] = 0;

  for (long long k0 = k_begin; k0 < k_end; k0 += TK) {
    // each thread fills two packed words of A and two of B
#pragma unroll
    for (int w = 0; w < 2; ++w) {
      int idx = tid + w * 256;          // 0..511 = 64 rows x 8 words
      int row = idx >> 3, kw = idx & 7;
      unsigned pa = 0, pb = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        long long k = k0 + kw * 4 + j;
        int8_t va = k < k_end ? load_a(q, m0 + row, k) : (int8_t)0;
        int8_t vb = k < k_end ? load_b(q, n0 + row, k) : (int8_t)0;
        pa |= (unsigned)(uint8_t)va << (8 * j);
        pb |= (unsigned)(uint8_t)vb << (8 * j);
      }
      As[row][kw] = (int)pa;
      Bs[row][kw] = (int)pb;
    }
    __syncthreads();
#pragma unroll
    for (int kw = 0; kw < TK / 4; ++kw) {
      int av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[ty * 4 + i][kw];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[tx * 4 + j][kw];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) c[i][j] = __dp4a(av[i], bv[j], c[i][j]);
    }
    __syncthreads();
  }

  unsigned mx = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    long long m = m0 + ty * 4 + i;
    if (m >= q.gm) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      long long n = n0 + tx * 4 + j;
      if (n >= q.gn) continue;
      int v = c[i][j];
      const unsigned a = v < 0 ? 0u - (unsigned)v : (unsigned)v;
      mx = a > mx ? a : mx;
      if (SPLIT) {
        if (v) atomicAdd(&acc[m * q.gn + n], v);
      } else {
        acc[m * q.gn + n] = v;
      }
    }
  }
  // block-wide max magnitude: of the finished accumulators (unsplit), or of this split's partial sums
  // (kept per split in the header; their sum bounds every accumulator of the tensor)
  for (int o = 16; o > 0; o >>= 1) {
    unsigned u = __shfl_xor_sync(0xffffffffu, mx, o);
    mx = u > mx ? u : mx;
  }
  if ((tid & 31) == 0) smax[tid >> 5] = mx;
  __syncthreads();
  if (tid == 0) {
    for (int i = 1; i < 8; ++i) mx = smax[i] > mx ? smax[i] : mx;
    if (mx) atomicMax(SPLIT ? niti_split_max(hdr) + blockIdx.z : &hdr->maxabs32, mx);
  }
}

}  // namespace

// max |v| over an int32 tensor (used after split-K accumulation).  splits > 1: block 0 also adds up the
// largest partial-sum magnitude of every split; that sum bounds every accumulator, and when it reaches
// 2^31 the int32 contract cannot be vouched for.
__global__ void __launch_bounds__(256)
maxabs_i32_kernel(const int32_t *__restrict__ acc, long long n, WsHeader *hdr, int splits, uint32_t *status) {
  if (splits > 1 && blockIdx.x == 0 && threadIdx.x < 32) {
    unsigned long long bound = 0;
    const unsigned *sm = niti_split_max(hdr);
    for (int i = threadIdx.x; i < splits; i += 32) bound += sm[i];
    for (int o = 16; o > 0; o >>= 1) bound += __shfl_xor_sync(0xffffffffu, bound, o);
    if (threadIdx.x == 0 && bound >= 0x80000000ull) atomicOr(status, NITI_DEV_ACC_RANGE);
  }
  unsigned mx = 0;
  const long long nvec = n >> 2;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (long long v = tid; v < nvec; v += stride) {
    int4 x = *(reinterpret_cast<const int4 *>(acc) + v);
    unsigned a0 = abs(x.x), a1 = abs(x.y), a2 = abs(x.z), a3 = abs(x.w);
    a0 = a0 > a1 ? a0 : a1;
    a2 = a2 > a3 ? a2 : a3;
    a0 = a0 > a2 ? a0 : a2;
    mx = a0 > mx ? a0 : mx;
  }
  long long t = (nvec << 2) + tid;
  if (t < n) {
    unsigned a = abs(acc[t]);
    mx = a > mx ? a : mx;
  }
  for (int o = 16; o > 0; o >>= 1) {
    unsigned u = __shfl_xor_sync(0xffffffffu, mx, o);
    mx = u > mx ? u : mx;
  }
  __shared__ unsigned smax[8];
  if ((threadIdx.x & 31) == 0) smax[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < 8; ++i) mx = smax[i] > mx ? smax[i] : mx;
    if (mx) atomicMax(&hdr->maxabs32, mx);
  }
}

int niti_launch_maxabs(niti_ctx *ctx, cudaStream_t st, const int32_t *acc, long long n, WsHeader *hdr, int splits) {
  long long blocks = ((n >> 2) + 255) / 256;
  if (blocks > ctx->sm_count * 8) blocks = ctx->sm_count * 8;
  if (blocks < 1) blocks = 1;
  maxabs_i32_kernel<<<(unsigned)blocks, 256, 0, st>>>(acc, n, hdr, splits, ctx->d_status);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

// Sum of the partial tensors of a split contraction (one slice of n int32 per split) into the first
// slice, the max magnitude of the sums, and the int32 range check: the magnitudes of an element's
// partial sums bound its total, and every partial sum is exact (a split is at most NITI_SPLIT_MAX_K long).
__global__ void __launch_bounds__(256)
sum_partials_kernel(int32_t *__restrict__ acc, int splits, long long n, WsHeader *hdr, uint32_t *status) {
  unsigned mx = 0;
  unsigned long long worst = 0;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    int s = acc[i];
    unsigned long long bound = (unsigned)abs(s);
    for (int k = 1; k < splits; ++k) {
      const int v = acc[(long long)k * n + i];
      s += v;
      bound += (unsigned)abs(v);
    }
    acc[i] = s;
    const unsigned a = (unsigned)abs(s);
    mx = a > mx ? a : mx;
    worst = bound > worst ? bound : worst;
  }
  if (worst >= 0x80000000ull) atomicOr(status, NITI_DEV_ACC_RANGE);
  mx = __reduce_max_sync(0xffffffffu, mx);
  __shared__ unsigned smax[8];
  if ((threadIdx.x & 31) == 0) smax[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < 8; ++i) mx = smax[i] > mx ? smax[i] : mx;
    if (mx) atomicMax(&hdr->maxabs32, mx);
  }
}

int niti_launch_sum_partials(niti_ctx *ctx, cudaStream_t st, int32_t *acc, int splits, long long n, WsHeader *hdr) {
  long long blocks = (n + 255) / 256;
  if (blocks > ctx->sm_count * 8) blocks = ctx->sm_count * 8;
  if (blocks < 1) blocks = 1;
  sum_partials_kernel<<<(unsigned)blocks, 256, 0, st>>>(acc, splits, n, hdr, ctx->d_status);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

int niti_simt_gemm(niti_ctx *ctx, cudaStream_t st, const GemmProblem &p, int32_t *acc, WsHeader *hdr) {
  Addr q;
  q.p0 = p.p0; q.p1 = p.p1; q.kind = p.kind;
  q.M = p.M; q.N = p.N; q.K = p.K;
  q.H = p.H; q.W = p.W; q.Ho = p.Ho; q.Wo = p.Wo; q.Ci = p.Ci; q.Co = p.Co; q.R = p.R; q.S = p.S; q.pad = p.pad;
  q.stride = p.stride > 0 ? p.stride : 1;
  q.gm = p.gm; q.gn = p.gn; q.gk = p.gk;
  q.pitch0 = p.ld0 ? p.ld0 : p.N;
  long long gx = (p.gn + TN - 1) / TN, gy = (p.gm + TM - 1) / TM;
  if (gy > 65535) return niti_fail(ctx, NITI_ERR_SHAPE, "simt gemm: too many row tiles");
  // split the contraction when the output grid alone cannot fill the GPU
  long long tiles = gx * gy;
  long long splits = 1;
  if (tiles < 2LL * ctx->sm_count && p.gk >= 4096) {
    splits = (4LL * ctx->sm_count + tiles - 1) / tiles;
    long long max_splits = p.gk / 1024;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
  }
  // no split longer than NITI_SPLIT_MAX_K (a partial sum then cannot wrap), at most NITI_MAX_SPLITS splits
  const long long min_splits = (p.gk + NITI_SPLIT_MAX_K - 1) / NITI_SPLIT_MAX_K;
  if (splits < min_splits) splits = min_splits;
  if (splits > NITI_MAX_SPLITS) return niti_fail(ctx, NITI_ERR_SHAPE, "simt gemm: contraction too long");
  long long kps = (p.gk + splits - 1) / splits;
  kps = (kps + TK - 1) / TK * TK;
  splits = (p.gk + kps - 1) / kps;
  dim3 grid((unsigned)gx, (unsigned)gy, (unsigned)splits);
  if (splits > 1) {
    NITI_CUDA_TRY(ctx, cudaMemsetAsync(acc, 0, sizeof(int32_t) * (size_t)(p.gm * p.gn), st));
    ctx->launches++;
    simt_gemm_kernel<true><<<grid, 256, 0, st>>>(q, acc, hdr, kps);
    ctx->launches++;
    NITI_CUDA_TRY(ctx, cudaGetLastError());
    return niti_launch_maxabs(ctx, st, acc, p.gm * p.gn, hdr, (int)splits);
  }
  simt_gemm_kernel<false><<<grid, 256, 0, st>>>(q, acc, hdr, kps);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}
