// Tensor-core engine: int8 x int8 -> int32 matrix multiply on the 5th-generation tensor cores
// (tcgen05.mma kind::i8, accumulators in tensor memory, operands staged by TMA), sm_100a only.
//
// One persistent CTA (or CTA pair) per SM, 20 warps: warps 0..2 = TMA producers (each owns every
// third stage of the ring), warp 3 = MMA issuer and TMEM owner, warps 4..19 = epilogue (four per
// 32-lane quarter of TMEM, read with tcgen05.ld).  Up to eight accumulator buffers live in TMEM, so
// the epilogues of finished tiles overlap the main loops of the following ones.
//
// The six operand mappings of the layer ops (Int8MatrixMultiply of Algorithm 1; implicit GEMM for
// convolutions, Section 3.2) differ only in the TMA tensor maps, the per-k-block coordinates the
// producer issues, and the shared-memory matrix descriptors (K-major or MN-major operands).
//
// Every wait in the kernel is bounded: after ~1 s without progress a thread raises
// NITI_DEV_TIMEOUT in the status word, and all roles drain and leave through the common exit
// that frees the tensor memory.
#include "niti_common.cuh"
#include <math.h>
#include <type_traits>

namespace {

constexpr int BM = 128;               // rows of an output tile = TMEM lanes
constexpr int EPI_WARPS = 16;          // four per TMEM lane quarter, interleaved 32-column chunks
constexpr int EPI_PER_Q = EPI_WARPS / 4;
// TMA copies are issued by single threads, and one thread sustains only about one copy per
// 250 ns (measured: four issuing warps give four times the copy rate), so the k-blocks are dealt
// round-robin to PROD_WARPS producer warps.
constexpr int PROD_WARPS = 3;          // each stage of the ring belongs to one producer warp (stage % nprod)
constexpr int MMA_WARP = PROD_WARPS;
constexpr int EPI_WARP0 = PROD_WARPS + 1;
constexpr int NUM_THREADS = 32 * (PROD_WARPS + 1 + EPI_WARPS);
constexpr int MAX_STAGES = 8;
constexpr int MAX_TBUF = 8;
constexpr long long WAIT_LIMIT_CYCLES = 2000000000LL;

struct TcParams {
  int kind;
  int n_tiles_n;                // tiles along the output columns
  int kb_total;                 // k-blocks of the whole contraction
  int kb_per_split;
  int splits;
  long long items;              // tiles * splits
  // set-up arithmetic done on the host (integer divisions at kernel entry delay every launch)
  int blk_per, blk_extra;       // blocked assignment: items per CTA (pair) and how many take one more
  int k_wpq, k_wpq_active, k_epi_active, k_tmem_cols;
  unsigned magic_w, magic_h;    // floor(2^32 / tiles) + 1 for w_tiles, h_tiles: n / d = umulhi(n, magic) while
                                // n * d < 2^32 (0: divide)
  int quorum;                   // CTAs whose first tile must have reported before the speculative bit-width
                                // is fixed (all of them when the sample is the whole tensor)
  int nissue;                   // resident-weights mode: warps that issue MMAs (2: the warp that loaded the
                                // weights takes every other tile)
  int one_commit;               // resident-weights mode with as many patch stages as accumulator buffers:
                                // stage and buffer advance together, one barrier per tile serves both
  int stg_off;                  // > 0: byte offset (from the aligned base) of the epilogue warps' transpose
                                // buffers for coalesced atomic adds, 32 x 33 words per warp
  int mrep;                     // 128-row tiles per item (row-batched mode of short contractions), else 1
  int bn_mma;                   // N of one MMA; bn = mrep * bn_mma accumulator columns per item
  long long gm, gn;             // output extent (rows, columns); row pitch of acc is gn
  int bn;                       // tile width (multiple of 32, <= 256)
  int kdepth;                   // contraction elements per k-block (32, 64 or 128)
  int ksteps;                   // kdepth / 32 MMAs per k-block
  int stages;
  // shared-memory layout of one stage
  int a_bytes, b_bytes;         // bytes of the A and B parts of a stage
  int a_boxes, b_boxes;         // TMA copies per operand per stage
  int a_box_bytes, b_box_bytes;
  int a_box_step, b_box_step;   // coordinate step between consecutive boxes (MN-major operands)
  // MMA descriptors
  unsigned idesc;
  unsigned long long a_desc, b_desc;   // descriptor without the start address
  unsigned a_kstep16, b_kstep16;       // start-address advance per MMA, in 16-byte units
  // convolution geometry (pixels of the tensor that the 4-D map covers)
  int Wt, Ht, Bt;               // pixel box of a tile / k-block: Wt * Ht * Bt == 128
  int w_tiles, h_tiles, b_tiles;
  int PW, PH, PB;               // extent of the pixel grid the output rows (or k-blocks) run over
  int R, S, pad;
  int stride;                   // convolution stride (forward and weight gradient; the shifted operand is then
                                // copied with that element stride, so a box still lands as Wt x Ht pixels)
  int c_chunks;                 // channel chunks per tap along the contraction (fwd / dgrad)
  int Cn;                       // wgrad: input channels Ci (columns per tap)
  int n_chunks;                 // wgrad: column chunks per tap
  int ctas;                     // CTAs per tile: 1, or 2 (cta_group::2, 256-row tiles)
  int m_units;                  // row units: 128-row tiles (ctas = 1) or 256-row pairs (ctas = 2)
  int raster_g;                 // row units per rasterisation group (0: row-major order)
  int blocked;                  // 1: every CTA takes a contiguous range of items (its first tile then
                                //    samples the tensor evenly), 0: items strided over the grid
  int nbuf;                     // accumulator buffers in tensor memory (2..8)
  int egroups;                  // epilogue warp groups (1, 2 or 4); tile `use` belongs to group use % egroups
  int nprod;                    // producer warps in use; divides `stages` (each stage has one owner, so
                                // the waits on a stage's barriers stay in order)
  // halo mode (3x3 convolutions with few channels): the weights of all nine taps stay in shared
  // memory for the whole kernel, every tile loads its 8 x 16 pixel patch once with a one-pixel
  // halo (10 x 18 pixels), and the nine taps are nine row offsets into that patch
  // halo == 2: weight gradient of such a convolution for one (64 output channels, 64 input
  // channels) block.  Per 8 x 16 pixel tile the CTA loads the error tile and the input patch once;
  // the nine taps are row offsets into the patch, two taps share one MMA (M = 2 x 64 input
  // channels through the leading-dimension stride of the MN-major descriptor), N = 64 output
  // channels, and the five accumulators stay in tensor memory over the CTA's whole pixel range.
  int halo;
  int wg_nci;                   // 64-channel blocks of the input channels
  int b_tile_bytes;             // bytes of one tap's weight tile
  int b_res_bytes;              // bytes of the resident weights (all taps), multiple of 1024
  // epilogue
  int epi_mode;                 // EPI_SPILL / EPI_ATOMIC / EPI_SPECULATE / EPI_KNOWN_B
  int mbits, round_mode, relu;
  unsigned spec_mul256;         // the sampled max is scaled by this / 256 before taking its bit length
  int spec_tag;                 // identifies the call site (its b_out scalar) in the table of estimate errors
  int update;                   // 1: out8 holds weights: the epilogue stores clamp(w - rounded gradient, +-127)
  int pool;                     // 1: the epilogue also stores the 2 x 2 max-pool of the (ReLU'd) output tile
  int pool_xh;                  // lane distance of the pixel one image row below (the pixel to the right is lane ^ 1)
  int single_wave;              // every CTA has at most one tile: the sample is the whole tensor, the shift
                                // is exact, and the last CTA to finish publishes b and the exponent
};

// Epilogue modes.  The shift of Algorithm 2 needs the bit-width of the WHOLE accumulator tensor:
//  EPI_SPILL      store int32 accumulators + max; a second kernel rounds (always exact, 8 B / output
//                 of extra traffic)
//  EPI_ATOMIC     split contraction: add partial sums into a zeroed int32 tensor
//  EPI_SPECULATE  every CTA computes its first tile, the grid agrees on the max over those tiles
//                 (one bounded grid-wide wait), and all tiles are rounded and stored as int8 with the
//                 shift that max implies, while the true max is tracked.  If the true bit-width turns
//                 out larger, the EPI_KNOWN_B pass recomputes everything with it (exact in all cases;
//                 the common case costs one multiply and no int32 traffic)
//  EPI_KNOWN_B    bit-width known (hdr->maxabs32): round and store directly.  The kernel returns at
//                 once when the speculative pass was right.
//  EPI_PARTIAL    split contraction of a multiply with few output rows (fully connected layers at batch
//                 <= 128): every split stores its int32 partial tile to its own slice of the scratch
//                 (plain 16-byte stores) and a small kernel adds the slices and takes the max.  An SM
//                 retires only about 1.6 atomic additions per cycle, so the 64 x 256 partial tile of a
//                 weight-streaming multiply took 5 us to add atomically, as long as a 4 MB layer takes
//                 to stream.
enum { EPI_SPILL = 0, EPI_ATOMIC = 1, EPI_SPECULATE = 2, EPI_KNOWN_B = 3, EPI_PARTIAL = 4 };


// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void *p) {
  return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking test of a phase (never suspends the thread).
__device__ __forceinline__ bool mbar_test(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Same, but the thread may sleep in hardware for up to `ns` nanoseconds while the phase is pending
// (it is woken when the phase completes), so a waiting warp does not burn issue slots polling.
__device__ __forceinline__ bool mbar_try_sleep(unsigned bar, unsigned parity, unsigned ns) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}
// A waiting warp that keeps polling takes issue slots next to the working warps of its scheduler (the
// hardware wait above returns after a few tens of cycles: ncu counts a poll loop every ~70 cycles in a
// warp that waits through an epilogue-bound tile).  After two failed polls the warp sleeps between
// polls, 128 ns at first and 256 ns from the eighth poll on.  Run times with and without the sleep
// measured the same within 1 % on five layer shapes; the sleep is kept because it costs nothing and
// leaves the issue slots to the working warps.
__device__ __forceinline__ void wait_backoff(unsigned &polls) {
  ++polls;
  if (polls > 2) __nanosleep(polls > 8 ? 256u : 128u);
}
// Bounded wait.  Returns false (and raises the abort flag) if the barrier did not flip in time or
// another thread already gave up.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int *abort_flag,
                                          uint32_t *status, long long limit_cycles = WAIT_LIMIT_CYCLES) {
  if (mbar_try(bar, parity)) return true;
  long long t0 = clock64();
  unsigned polls = 0;
  while (true) {
    if (mbar_try_sleep(bar, parity, 20000u)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit_cycles) {
      *abort_flag = 1;
      atomicOr(status, NITI_DEV_TIMEOUT);
      return false;
    }
    wait_backoff(polls);
  }
}
// The same bounded wait for a whole converged warp: every lane polls, the votes make the outcome (and
// with it the caller's control flow) warp-uniform, so the compiler can keep the caller's address
// arithmetic in uniform registers.
__device__ __forceinline__ bool mbar_wait_warp(unsigned bar, unsigned parity, volatile int *abort_flag,
                                               uint32_t *status, long long limit_cycles = WAIT_LIMIT_CYCLES) {
  if (__all_sync(0xffffffffu, mbar_try(bar, parity))) return true;
  const long long t0 = clock64();
  unsigned polls = 0;
  while (true) {
    if (__all_sync(0xffffffffu, mbar_try_sleep(bar, parity, 20000u))) return true;
    if (__any_sync(0xffffffffu, *abort_flag != 0)) return false;
    if (__any_sync(0xffffffffu, clock64() - t0 > limit_cycles)) {
      *abort_flag = 1;
      atomicOr(status, NITI_DEV_TIMEOUT);
      return false;
    }
    wait_backoff(polls);
  }
}
// One lane of a converged warp (the same one every time it is asked).
__device__ __forceinline__ bool elect_one() {
  unsigned pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap *map, unsigned bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(unsigned dst, const CUtensorMap *map, unsigned bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(unsigned bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_i8(unsigned tmem_d, unsigned long long da, unsigned long long db,
                                          unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Same with the two 64-bit matrix descriptors given as 32-bit halves: the issuing thread then does
// its address arithmetic in 32 bits (the high halves never change inside a kernel).
__device__ __forceinline__ void tc_mma_i8_lh(unsigned tmem_d, unsigned a_lo, unsigned a_hi, unsigned b_lo,
                                             unsigned b_hi, unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %5, p;\n\t}"
      ::"r"(tmem_d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(unsigned taddr, int (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shift-and-round of four accumulators (Algorithm 2 + 3, or round-to-nearest) packed into four int8.
//
// Pseudo-stochastic rule on a magnitude a with bp discarded bits (h = bp / 2, o = bp & 1): the lowest
// bit is dropped when bp is odd; the next 2h bits are top * 2^h + bot and the integer part is
// incremented iff top > bot.  With mask2 = (2^h - 1) << o the term (~a & mask2) is (2^h - 1 - bot) << o,
// and adding it times 2^h carries into bit bp exactly when top > bot:
//     q = (a + (~a & mask2) * 2^h) >> bp           (the dropped lowest bit cannot carry).
// Round-to-nearest is the same expression with mask2 = 0 and the constant 2^(bp-1) in place of the
// product.  Saturation at 2^mbits - 1 happens only when the integer part is already 2^mbits - 1, so
// clamping the magnitude to cap = (2^mbits - 1) << bp beforehand gives the same result.
//
// The integer pipe of an SM issues one warp instruction every two cycles, and the epilogue of every
// output element runs on it: the instruction count per element here bounds the layers with few
// input channels.  ReLU outputs therefore never form |x|: max(min(x, cap), 0) is one instruction and
// rounds negative inputs to zero by itself; the true extremes are tracked with three-input min/max.
struct RoundConst {
  unsigned mask2;   // (2^h - 1) << o, or 0
  unsigned orc;     // 0, or 1 for round-to-nearest with bp > 0
  unsigned mulp;    // 2^h, or 2^(bp-1)
  int shift;        // bp
  int cap;          // (2^mbits - 1) << bp
  unsigned hi_mul;  // 2^(32 - bp) for bp > 0: the high half of v * hi_mul is v >> bp
  // Byte-aligned form (bp <= 24): with k = (8 - bp % 8) % 8 the sum scaled by 2^k has its integer
  // part exactly in byte B = (bp + k) / 8, so no shift is needed: a byte permute picks the rounded
  // values of two accumulators at once.
  unsigned sc;      // 2^k
  unsigned c2;      // mulp * 2^k
  unsigned sel;     // permute selector: byte B of either operand in bytes 0 and 1, zeros above
  unsigned m16;     // 2^16 (merges two byte pairs with a multiply-add)
  bool aligned;
};
__device__ __forceinline__ RoundConst make_round_const(int bp, int mbits, int round_mode) {
  RoundConst k;
  k.shift = bp;
  k.cap = (int)(((1u << mbits) - 1u) << bp);
  k.hi_mul = bp > 0 ? 1u << (32 - bp) : 0u;
  if (round_mode == NITI_ROUND_PSR) {
    const int h = bp >> 1;
    k.mask2 = ((1u << h) - 1u) << (bp & 1);
    k.orc = 0;
    k.mulp = 1u << h;
  } else {
    k.mask2 = 0;
    k.orc = bp > 0 ? 1u : 0u;
    k.mulp = bp > 0 ? 1u << (bp - 1) : 0u;
  }
  const int kk = (8 - (bp & 7)) & 7, B = (bp + kk) >> 3;
  k.aligned = bp <= 24;
  k.sc = 1u << kk;
  k.c2 = k.mulp << kk;
  // (kept opaque: known to be a power of two, the multiplies would be turned back into shifts on
  // the integer pipe, which is the one that has no slots to spare)
  k.m16 = 0x10000u;
  asm volatile("" : "+r"(k.sc), "+r"(k.c2), "+r"(k.m16));
  // selector nibbles: B (first operand), 4 + B (second operand), then twice "sign of byte B"
  // replicated, which is zero because a rounded magnitude is at most 127
  k.sel = (unsigned)B | ((unsigned)(4 + B) << 4) | ((unsigned)(8 | B) << 8) | ((unsigned)(8 | B) << 12);
  return k;
}
// magnitude already clamped to cap
template <bool SHIFT>
__device__ __forceinline__ unsigned round_mag1(unsigned m, const RoundConst &k) {
  const unsigned v = (((~m) & k.mask2) | k.orc) * k.mulp + m;
  return SHIFT ? __umulhi(v, k.hi_mul) : v;
}
// Extremes of the raw accumulators seen by one thread.
struct Extremes {
  int hi, lo;       // running max (>= 0) and min (<= 0)
  unsigned orv;     // OR of magnitudes (same bit length as their maximum)
  __device__ __forceinline__ unsigned magnitude_bits() const {
    return orv | (unsigned)hi | (0u - (unsigned)lo);
  }
};
template <bool RELU, bool SHIFT>
__device__ __forceinline__ unsigned round_pack4(int x0, int x1, int x2, int x3, const RoundConst &k, Extremes &e) {
  unsigned q0, q1, q2, q3;
  if (RELU) {
    e.hi = __vimax3_s32(e.hi, x0, x1);
    e.hi = __vimax3_s32(e.hi, x2, x3);
    e.lo = __vimin3_s32(e.lo, x0, x1);
    e.lo = __vimin3_s32(e.lo, x2, x3);
    q0 = round_mag1<SHIFT>((unsigned)__vimin_s32_relu(x0, k.cap), k);
    q1 = round_mag1<SHIFT>((unsigned)__vimin_s32_relu(x1, k.cap), k);
    q2 = round_mag1<SHIFT>((unsigned)__vimin_s32_relu(x2, k.cap), k);
    q3 = round_mag1<SHIFT>((unsigned)__vimin_s32_relu(x3, k.cap), k);
    // values below 2^7: bytes assembled with multiply-adds
    return (q1 * 0x100u + q0) + (q3 * 0x1000000u + q2 * 0x10000u);
  }
  const unsigned a0 = (unsigned)abs(x0), a1 = (unsigned)abs(x1), a2 = (unsigned)abs(x2), a3 = (unsigned)abs(x3);
  e.orv |= a0 | a1;
  e.orv |= a2 | a3;
  const unsigned cap = (unsigned)k.cap;
  q0 = round_mag1<SHIFT>(min(a0, cap), k); q1 = round_mag1<SHIFT>(min(a1, cap), k);
  q2 = round_mag1<SHIFT>(min(a2, cap), k); q3 = round_mag1<SHIFT>(min(a3, cap), k);
  // sign as a multiply by +-1: the multiply runs beside the integer pipe
  q0 *= (unsigned)((x0 >> 31) | 1); q1 *= (unsigned)((x1 >> 31) | 1);
  q2 *= (unsigned)((x2 >> 31) | 1); q3 *= (unsigned)((x3 >> 31) | 1);
  return __byte_perm(__byte_perm(q0, q1, 0x4040), __byte_perm(q2, q3, 0x4040), 0x5410);
}
__device__ __forceinline__ unsigned prmt(unsigned a, unsigned b, unsigned sel) {
  unsigned d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
// (clamped magnitude + rounding term) * 2^k: the rounded value sits in byte B
__device__ __forceinline__ unsigned scaled_round(unsigned m, const RoundConst &k) {
  return (((~m) & k.mask2) | k.orc) * k.c2 + m * k.sc;
}
// Byte-aligned form of round_pack4.  Per element the half-rate integer pipe sees the extremes (one
// three-input min or max per element), the clamp, the bit select and half a permute; the two
// multiply-adds and the final merge run on the multiplier pipe.  Measured against the shift form:
// 6.9 instead of 9.0 issue cycles per element with ReLU, 10.9 instead of 15.1 without.
template <bool RELU>
__device__ __forceinline__ unsigned round_pack4_aligned(int x0, int x1, int x2, int x3, const RoundConst &k, Extremes &e) {
  if (RELU) {
    e.hi = __vimax3_s32(e.hi, x0, x1);
    e.hi = __vimax3_s32(e.hi, x2, x3);
    e.lo = __vimin3_s32(e.lo, x0, x1);
    e.lo = __vimin3_s32(e.lo, x2, x3);
    const unsigned v0 = scaled_round((unsigned)__vimin_s32_relu(x0, k.cap), k);
    const unsigned v1 = scaled_round((unsigned)__vimin_s32_relu(x1, k.cap), k);
    const unsigned v2 = scaled_round((unsigned)__vimin_s32_relu(x2, k.cap), k);
    const unsigned v3 = scaled_round((unsigned)__vimin_s32_relu(x3, k.cap), k);
    return prmt(v2, v3, k.sel) * k.m16 + prmt(v0, v1, k.sel);
  }
  const unsigned a0 = (unsigned)abs(x0), a1 = (unsigned)abs(x1), a2 = (unsigned)abs(x2), a3 = (unsigned)abs(x3);
  e.orv |= a0 | a1;
  e.orv |= a2 | a3;
  const unsigned cap = (unsigned)k.cap;
  const unsigned v0 = scaled_round(min(a0, cap), k), v1 = scaled_round(min(a1, cap), k);
  const unsigned v2 = scaled_round(min(a2, cap), k), v3 = scaled_round(min(a3, cap), k);
  const unsigned w = prmt(v2, v3, k.sel) * k.m16 + prmt(v0, v1, k.sel);
  // two's complement of the bytes whose accumulator was negative, four at a time: sm has 0xff in
  // those bytes (sign of the top byte of each accumulator, replicated); on the low seven bits
  // (w ^ sm) + 1 cannot carry into the next byte because w <= 127, and bit 7 is the sign unless the
  // byte is zero, which the last exclusive-or takes care of (0x80 ^ 0x80)
  const unsigned sm = prmt(prmt((unsigned)x0, (unsigned)x1, 0xfbfbu), prmt((unsigned)x2, (unsigned)x3, 0xfbfbu), 0x5410u);
  const unsigned t = ((w ^ sm) & 0x7f7f7f7fu) + (sm & 0x01010101u);
  return t ^ (sm & 0x80808080u);
}
// all variants behind one call: relu and the binary point are the same for every element of a pass
__device__ __forceinline__ void round_chunk32(const int (&v)[32], unsigned (&w8)[8], const RoundConst &k, bool relu,
                                              Extremes &e) {
  if (k.aligned) {
    if (relu) {
#pragma unroll
      for (int j = 0; j < 8; ++j) w8[j] = round_pack4_aligned<true>(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3], k, e);
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) w8[j] = round_pack4_aligned<false>(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3], k, e);
    }
  } else if (relu) {      // (binary point above 24: only with fewer than seven magnitude bits)
#pragma unroll
    for (int j = 0; j < 8; ++j) w8[j] = round_pack4<true, true>(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3], k, e);
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) w8[j] = round_pack4<false, true>(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3], k, e);
  }
}

// per byte: clamp(w - g, -127, 127) (Algorithm 1's update on int8 weights)
__device__ __forceinline__ unsigned bytes_sub_clamp127(unsigned w, unsigned g) {
  return __vmaxs4(__vsubss4(w, g), 0x81818181u);
}
// 0xff in every byte of b that is greater than zero as a signed byte (the ReLU gate of the backward pass).
__device__ __forceinline__ unsigned bytes_gt0(unsigned b) {
  unsigned t = (b & 0x7f7f7f7fu) + 0x7f7f7f7fu;   // bit 7 of a byte: its low seven bits are not all zero
  t = t & ~b & 0x80808080u;                       // ... and its sign bit is clear
  unsigned r;
  asm("prmt.b32 %0, %1, %1, 0xba98;" : "=r"(r) : "r"(t));   // replicate bit 7 over each byte
  return r;
}

// Byte-wise maximum of two words whose bytes are all in [0, 127] (ReLU outputs): bit 7 of
// (a | 0x80..) - b is set per byte exactly where a >= b, and no byte borrows from its neighbour.
__device__ __forceinline__ unsigned bytes_max_u7(unsigned a, unsigned b) {
  const unsigned t = (a | 0x80808080u) - b;
  unsigned m;
  asm("prmt.b32 %0, %1, %1, 0xba98;" : "=r"(m) : "r"(t));   // 0xff where a >= b
  return (a & m) | (b & ~m);
}
// 2 x 2 max-pool of a 32-channel chunk held one pixel per lane: the window's other pixels are the lanes
// lane ^ 1 (next column) and lane ^ xh (next image row); every lane ends up with its window's maximum.
__device__ __forceinline__ void pool_chunk32(unsigned (&w8)[8], int xh) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    unsigned a = w8[j];
    a = bytes_max_u7(a, __shfl_xor_sync(0xffffffffu, a, 1));
    a = bytes_max_u7(a, __shfl_xor_sync(0xffffffffu, a, xh));
    w8[j] = a;
  }
}
__device__ __forceinline__ void store32(int8_t *dst, const unsigned (&w8)[8]) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"l"(dst), "r"(w8[0]), "r"(w8[1]), "r"(w8[2]), "r"(w8[3]), "r"(w8[4]), "r"(w8[5]), "r"(w8[6]), "r"(w8[7])
               : "memory");
}

// Per call site the table keeps the errors (true bit-width minus sample-based estimate, each stored + 2
// in four bits) of the last two calls.  An error that repeats is systematic (the tensor's extremes sit
// outside the sampled tiles, or its distribution has a heavier tail than the scaling assumes) and is
// added to the next estimate; a single miss is the estimator's noise (on drifting training tensors about
// one launch in eight crosses a power of two unnoticed) and following it would only add misses.
__device__ __forceinline__ int spec_correction(int packed) {
  const int e1 = (packed & 15) - 2, e2 = ((packed >> 4) & 15) - 2;
  return e1 == e2 ? e1 : 0;
}

// n / d with the host's reciprocal (exact while n * d < 2^32, which the host checked), else a division
__device__ __forceinline__ int div_tiles(int n, int d, unsigned magic) {
  return magic ? (int)__umulhi((unsigned)n, magic) : n / d;
}
// tile index -> (column tile, row tile, image) with two reciprocal multiplies
__device__ __forceinline__ void tile_coords(const TcParams &p, int idx, int &wt, int &ht, int &bt) {
  const int t = div_tiles(idx, p.w_tiles, p.magic_w);
  wt = idx - t * p.w_tiles;
  bt = div_tiles(t, p.h_tiles, p.magic_h);
  ht = t - bt * p.h_tiles;
}
// Coordinates of an output tile / k-block in the pixel grid of a convolution.
__device__ __forceinline__ void pixel_box(const TcParams &p, int idx, int &w0, int &h0, int &b0) {
  int wt, ht, bt;
  tile_coords(p, idx, wt, ht, bt);
  w0 = wt * p.Wt; h0 = ht * p.Ht; b0 = bt * p.Bt;
}

// ------------------------------------------------------------------------------------------
// Cluster helpers (CTAS == 2: a pair of CTAs on neighbouring SMs works on one 256-row tile with
// tcgen05 cta_group::2; the even CTA of the pair issues the MMAs and owns the barriers).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ unsigned map_to_cta(unsigned local_addr, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(unsigned cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(unsigned dst, const CUtensorMap *map, unsigned bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(unsigned dst, const CUtensorMap *map, unsigned bar, int c0, int c1,
                                                 int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(unsigned bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((unsigned short)3)
      : "memory");
}
__device__ __forceinline__ void tc_mma_i8_pair(unsigned tmem_d, unsigned long long da, unsigned long long db,
                                               unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tc_mma_i8_pair_lh(unsigned tmem_d, unsigned a_lo, unsigned a_hi, unsigned b_lo,
                                                  unsigned b_hi, unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %5, p;\n\t}"
      ::"r"(tmem_d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The issuing thread is a single instruction stream: every scalar instruction between two MMAs is
// on the critical path of the tensor pipe (measured: run-time trip counts, selects and multiplies
// per MMA cost ~35 cycles each time, more than half of an N = 64 MMA).  The issue loops are therefore
// compiled per k-step count, with every offset either a literal or a register filled before the
// tile loop.
//
// One 3x3 tile from the resident patch: nine taps, KS k-steps each, into one accumulator.
template <int KS>
__device__ __forceinline__ void halo_issue_tile(unsigned tmem_d, unsigned a_lo, unsigned a_hi, const unsigned (&a_off)[9],
                                                unsigned b_hi, const unsigned (&b_tap)[9], unsigned b_kstep16,
                                                unsigned idesc) {
#pragma unroll
  for (int tap = 0; tap < 9; ++tap) {
    const unsigned a_t = a_lo + a_off[tap];
#pragma unroll
    for (int k = 0; k < KS; ++k)
      tc_mma_i8_lh(tmem_d, a_t + 2u * k, a_hi, b_tap[tap] + (unsigned)k * b_kstep16, b_hi, idesc,
                   (tap > 0 || k > 0) ? 1u : 0u);
  }
}
// One k-block of the generic loop: KS MMAs whose operands advance by the k-step strides.
template <int CTAS, int KS>
__device__ __forceinline__ void issue_kblock(unsigned tmem_d, unsigned a_lo, unsigned a_hi, unsigned b_lo, unsigned b_hi,
                                             unsigned a_kstep16, unsigned b_kstep16, unsigned idesc, unsigned first_acc) {
#pragma unroll
  for (int k = 0; k < KS; ++k) {
    if (CTAS == 2)
      tc_mma_i8_pair_lh(tmem_d, a_lo + (unsigned)k * a_kstep16, a_hi, b_lo + (unsigned)k * b_kstep16, b_hi, idesc,
                        k > 0 ? 1u : first_acc);
    else
      tc_mma_i8_lh(tmem_d, a_lo + (unsigned)k * a_kstep16, a_hi, b_lo + (unsigned)k * b_kstep16, b_hi, idesc,
                   k > 0 ? 1u : first_acc);
  }
}

template <int CTAS>
__device__ __forceinline__ void load2(unsigned dst, const CUtensorMap *m, unsigned bar, int c0, int c1) {
  if (CTAS == 2) tma_load_2d_pair(dst, m, bar, c0, c1); else tma_load_2d(dst, m, bar, c0, c1);
}
template <int CTAS>
__device__ __forceinline__ void load4(unsigned dst, const CUtensorMap *m, unsigned bar, int c0, int c1, int c2, int c3) {
  if (CTAS == 2) tma_load_4d_pair(dst, m, bar, c0, c1, c2, c3); else tma_load_4d(dst, m, bar, c0, c1, c2, c3);
}

// item -> (row unit, column tile, split).  Row units (one CTA's 128 rows, or a pair's 256) are
// visited in groups of raster_g so that the CTAs running at the same time share operand tiles in L2.
// (32-bit arithmetic throughout: one thread of the producer, issuer and epilogue warps runs this per
// tile, and 64-bit divisions there cost more than a small tile's whole multiply.)
__device__ __forceinline__ void decode_item(const TcParams &p, int item, int &mu, int &nt, int &split) {
  int tile = item;
  split = 0;
  if (p.splits > 1) {
    tile = item / p.splits;
    split = item - tile * p.splits;
  }
  if (p.raster_g <= 0) {
    if (p.n_tiles_n == 1) { mu = tile; nt = 0; return; }
    mu = tile / p.n_tiles_n;
    nt = tile - mu * p.n_tiles_n;
    return;
  }
  const int per_group = p.raster_g * p.n_tiles_n;
  const int g = tile / per_group;
  const int rem = tile - g * per_group;
  int in_group = p.m_units - g * p.raster_g;
  if (in_group > p.raster_g) in_group = p.raster_g;
  mu = g * p.raster_g + rem % in_group;
  nt = rem / in_group;
}

// ------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------
// Issuing loop of the resident-weights mode.  `nissue` warps (1 or 2) run it, warp `issuer` taking
// tiles issuer, issuer + nissue, ... of the CTA's range: with 64 output channels a tile is only 18 MMAs,
// and one warp's per-tile bookkeeping (two barrier tests, fences, two commits) leaves the tensor pipe
// idle for a quarter of the time; two issuers fill each other's gaps.  Tiles go to different
// accumulator buffers, so the order in which the pipe sees the two warps' MMAs does not matter, and
// each warp's commits cover exactly its own MMAs.
__device__ __forceinline__ void halo_mma_loop(const TcParams &p, int issuer, int nissue, int first_item, int item_end,
                                              unsigned smem_base, unsigned tmem_base, unsigned full0, unsigned empty0,
                                              unsigned tfull0, unsigned tempty0, unsigned bres_bar,
                                              volatile int *abort_flag, uint32_t *status) {
  const bool leader = elect_one();
  bool ok = mbar_wait_warp(bres_bar, 0, abort_flag, status);
  // descriptor low words per tap, computed once: the patch row where the tap starts
  // (forward reads x[i + r - 1][j + t - 1], dgrad reads e[i - r + 1][j - t + 1]; the patch
  // starts one pixel up and left of the tile) and the tap's resident weight tile
  const unsigned a_hi = (unsigned)(p.a_desc >> 32), b_hi = (unsigned)(p.b_desc >> 32);
  const unsigned a_lo0 = (unsigned)p.a_desc, b_lo0 = (unsigned)p.b_desc + ((smem_base >> 4) & 0x3fff);
  const unsigned row16 = (unsigned)p.kdepth >> 4, btile16 = (unsigned)p.b_tile_bytes >> 4;
  const bool fwd_taps = p.kind == GK_CONV_FWD;
  const unsigned a_stage16 = (unsigned)p.a_bytes >> 4;
  const unsigned a_stage_lo = a_lo0 + (((smem_base + p.b_res_bytes) >> 4) & 0x3fff);   // stage 0
  const unsigned b_kstep16 = p.b_kstep16, idesc = p.idesc;
  const int ksteps = p.ksteps, stages = p.stages;
  const unsigned nbuf = (unsigned)p.nbuf, bn = (unsigned)p.bn;
  unsigned a_off[9], b_tap[9];
#pragma unroll
  for (int tap = 0; tap < 9; ++tap) {
    const int r = tap / 3, t = tap % 3;
    a_off[tap] = (fwd_taps ? (unsigned)(r * 10 + t) : (unsigned)((2 - r) * 10 + (2 - t))) * row16;
    b_tap[tap] = b_lo0 + (unsigned)tap * btile16;
  }
  const bool one_commit = p.one_commit != 0;
  int stage = 0;
  unsigned phase = 0;
  unsigned hbuf = 0, hpar = 0;          // tile % nbuf, (tile / nbuf) & 1, counted
  if (issuer) {                         // (issuer is 0 or 1)
    if (++stage == stages) { stage = 0; phase ^= 1; }
    if (++hbuf == nbuf) { hbuf = 0; hpar ^= 1u; }
  }
  for (int item = first_item + issuer; ok && item < item_end; item += nissue) {
    // (with one_commit the accumulator buffer is the stage and their parities coincide)
    const unsigned buf = one_commit ? (unsigned)stage : hbuf;
    const unsigned par = one_commit ? phase : hpar;
    if (!mbar_wait_warp(tempty0 + 8 * buf, par ^ 1u, abort_flag, status)) break;
    if (!mbar_wait_warp(full0 + 8 * stage, phase, abort_flag, status)) break;
    tc_fence_after();
    const unsigned tmem_d = tmem_base + buf * bn;
    const unsigned a_lo = a_stage_lo + (unsigned)stage * a_stage16;
    if (leader) {
      if (ksteps == 2) halo_issue_tile<2>(tmem_d, a_lo, a_hi, a_off, b_hi, b_tap, b_kstep16, idesc);
      else if (ksteps == 4) halo_issue_tile<4>(tmem_d, a_lo, a_hi, a_off, b_hi, b_tap, b_kstep16, idesc);
      else halo_issue_tile<1>(tmem_d, a_lo, a_hi, a_off, b_hi, b_tap, b_kstep16, idesc);
      if (!one_commit) tc_commit(empty0 + 8 * stage);
      tc_commit(tfull0 + 8 * buf);
    }
    for (int j = 0; j < nissue; ++j) {
      if (++stage == stages) { stage = 0; phase ^= 1; }
      if (++hbuf == nbuf) { hbuf = 0; hpar ^= 1u; }
    }
  }
}
template <int CTAS>
__global__ void __launch_bounds__(NUM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const TcParams p, int32_t *__restrict__ acc, WsHeader *hdr, uint32_t *status,
               int8_t *__restrict__ out8, const int8_t *__restrict__ mask8, const int32_t *s_a,
               const int32_t *s_w, int32_t *s_out, int32_t *b_out, int32_t *spec_slot, int8_t *__restrict__ pool8) {
  if (p.epi_mode == EPI_SPECULATE && !p.single_wave) {
    // the follow-up launch may be scheduled now (it is launched as a programmatic dependent): its CTAs
    // take the SMs as this grid's CTAs retire and wait there for the whole grid to finish
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  if (p.epi_mode == EPI_KNOWN_B) {
    // follow-up of a speculative pass: publish the scalars, then leave unless the guess was wrong
    asm volatile("griddepcontrol.wait;" ::: "memory");     // the first pass has completed and is visible
    const int b_true = niti_bitlen32(hdr->maxabs32), b_est = (int)hdr->spec_b - 1;   // (stored + 1)
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      if (spec_slot) {
        // remember, for the next calls from this call site, how far the sample-based estimate was off
        // (b_est = raw estimate + the correction this call applied): the last two errors are kept
        const int packed = spec_slot[0] == p.spec_tag ? spec_slot[1] : 0x22;
        int err = b_true - (b_est - spec_correction(packed));
        err = err < -2 ? -2 : (err > 2 ? 2 : err);
        spec_slot[0] = p.spec_tag;
        spec_slot[1] = (err + 2) | ((packed & 15) << 4);
      }
      const int bp = b_true > p.mbits ? b_true - p.mbits : 0;
      if (b_out) *b_out = b_true;
      if (s_out) {
        int s = bp + (s_a ? *s_a : 0) + (s_w ? *s_w : 0);
        *s_out = s;
        if (s < -128 || s > 127) atomicOr(status, NITI_DEV_EXP_RANGE);
      }
    }
    if (b_true == b_est) return;
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(status + 1, 1u);   // count of recomputations
  }
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * MAX_STAGES + 2 * MAX_TBUF + 1];
  __shared__ unsigned tmem_base_slot;
  __shared__ volatile int abort_flag;
  __shared__ volatile int spec_bp_ready;      // 0: not yet; else the speculative binary point + 1
  __shared__ unsigned first_max, first_arrived;   // this CTA's first tile: max magnitude, warps that reported
  __shared__ unsigned cta_max;                    // max magnitude of everything this CTA rounded

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const unsigned rank = CTAS == 2 ? cluster_ctarank() : 0u;
  const unsigned smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int stage_bytes = p.a_bytes + p.b_bytes;
  const unsigned full0 = smem_u32(&bars[0]);
  const unsigned empty0 = smem_u32(&bars[MAX_STAGES]);
  const unsigned tfull0 = smem_u32(&bars[2 * MAX_STAGES]);
  const unsigned tempty0 = smem_u32(&bars[2 * MAX_STAGES + MAX_TBUF]);
  const unsigned bres_bar = smem_u32(&bars[2 * MAX_STAGES + 2 * MAX_TBUF]);   // resident weights landed
  // barriers of the leader CTA as seen from this CTA
  const unsigned lead_full0 = CTAS == 2 ? map_to_cta(full0, 0) : full0;
  const unsigned lead_tempty0 = CTAS == 2 ? map_to_cta(tempty0, 0) : tempty0;
  // items of this CTA (pair): first_item, first_item + item_step, ... below item_end
  int first_item = blockIdx.x / CTAS, item_step = gridDim.x / CTAS, item_end = (int)p.items;
  if (p.blocked) {
    const int u = blockIdx.x / CTAS;
    const int per = p.blk_per, extra = p.blk_extra;
    first_item = u * per + (u < extra ? u : extra);
    item_end = first_item + per + (u < extra ? 1 : 0);
    item_step = 1;
  }

  // epilogue warps with at least one 32-column chunk of the tile (four per chunk phase)
  // The 16 epilogue warps are split into `egroups` groups that drain different tiles at the same
  // time (narrow tiles have too few 32-column chunks to keep every warp busy on one tile).  Inside a
  // group each TMEM lane quarter has wpq warps that interleave the tile's chunks.
  const int egroups = p.halo == 2 ? 1 : p.egroups;
  const int wpq = p.k_wpq;                                   // warps per quarter per tile
  const int wpq_active = p.k_wpq_active;
  const int epi_active = p.k_epi_active;                     // warps that drain one tile
  // TMEM columns: nbuf accumulator buffers of bn columns, rounded up to a power of two >= 32
  const unsigned tmem_cols = (unsigned)p.k_tmem_cols;

  // Set-up is paid by every launch (measured: 1.8 us from entry to the first copy when one thread did
  // all of it): the tensor maps are prefetched at once, every barrier is initialised by its own
  // thread, and tensor memory is allocated by another warp meanwhile.
  if (threadIdx.x == 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
  }
  if (threadIdx.x == 0) {
    abort_flag = 0;
    spec_bp_ready = 0;
    first_max = 0;
    first_arrived = 0;
    cta_max = 0;
  }
  if (threadIdx.x < 2 * MAX_STAGES + 2 * MAX_TBUF + 1) {
    const int bi = (int)threadIdx.x;
    const bool is_tempty = bi >= 2 * MAX_STAGES + MAX_TBUF && bi < 2 * MAX_STAGES + 2 * MAX_TBUF;
    // one arrival per barrier, except "accumulator drained": one per working epilogue warp of every CTA
    mbar_init(smem_u32(&bars[bi]), is_tempty ? epi_active * CTAS : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == MMA_WARP) {
    if (CTAS == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();   // the peer's barriers exist before anyone signals them
  tc_fence_after();
  const unsigned tmem_base = tmem_base_slot;

  if (warp < PROD_WARPS) {
    // ================= TMA producers (every CTA loads its own rows of A and its share of B) ========
    // Each producer warp runs its loop in lock step and one elected lane issues the copies (warp-uniform
    // control flow keeps the coordinate arithmetic in the uniform datapath that feeds the TMA unit).
    {
      const bool leader = elect_one();
      int stage = 0;
      unsigned phase = 0;
      bool ok = true;
      // (an integer division costs a lone warp ~200 cycles: nothing below divides per k-block or per
      // tile; the warp that owns the current stage is counted, stage % nprod)
      int owner = 0;
      const int nprod = p.nprod;
      const int bn_cta = p.bn / CTAS;             // B rows (output columns) staged by this CTA
      if (p.halo == 2) {
        for (int item = first_item; ok && item < item_end; item += item_step) {
          const int split = p.splits > 1 ? item % p.splits : 0;
          const int blk = (int)(item / p.splits);
          const int ci0 = (blk % p.wg_nci) * 64, co0 = (blk / p.wg_nci) * 64;
          const int t0 = split * p.kb_per_split;
          int t1 = t0 + p.kb_per_split;
          if (t1 > p.kb_total) t1 = p.kb_total;
          int wt = t0 % p.w_tiles, ht = (t0 / p.w_tiles) % p.h_tiles, bt = t0 / (p.w_tiles * p.h_tiles);
          for (int t = t0; t < t1; ++t) {
            if (owner == warp) {
              if (!mbar_wait_warp(empty0 + 8 * stage, phase ^ 1, &abort_flag, status)) { ok = false; break; }
              const unsigned full = full0 + 8 * stage;
              const unsigned sa = smem_base + stage * stage_bytes;
              if (leader) {
                mbar_expect_tx(full, (unsigned)(p.a_box_bytes + p.b_box_bytes));
                tma_load_4d(sa, &map_a, full, ci0, wt * 8 - 1, ht * 16 - 1, bt);          // input patch
                tma_load_4d(sa + p.a_bytes, &map_b, full, co0, wt * 8, ht * 16, bt);     // error tile
              }
            }
            if (++owner == nprod) owner = 0;
          if (++stage == p.stages) { stage = 0; phase ^= 1; }
            if (++wt == p.w_tiles) { wt = 0; if (++ht == p.h_tiles) { ht = 0; ++bt; } }
          }
        }
        item_end = first_item;
      } else if (p.halo) {
        // resident weights: one tile per tap, [bn rows][kdepth] K-major (forward) or
        // [kdepth rows][bn] MN-major in b_boxes column chunks (dgrad)
        // (issued by the last producer warp: the first one owns stage 0 and starts with tile 0's patch)
        if (warp == PROD_WARPS - 1 && leader) mbar_expect_tx(bres_bar, (unsigned)(9 * p.b_boxes * p.b_box_bytes));
        for (int tap = 0; warp == PROD_WARPS - 1 && leader && tap < 9; ++tap) {
          const unsigned dst = smem_base + tap * p.b_tile_bytes;
          if (p.kind == GK_CONV_FWD) {
            tma_load_2d(dst, &map_b, bres_bar, tap * p.kdepth, 0);
          } else {
            for (int j = 0; j < p.b_boxes; ++j)
              tma_load_2d(dst + j * p.b_box_bytes, &map_b, bres_bar, tap * p.Cn + j * p.b_box_step, 0);
          }
        }
        if (p.nissue == 2 && warp == PROD_WARPS - 1) {
          // (the other producer warps load the patches; this one issues every other tile's MMAs)
          if (rank == 0)
            halo_mma_loop(p, 1, 2, first_item, item_end, smem_base, tmem_base, full0, empty0, tfull0, tempty0,
                          bres_bar, &abort_flag, status);
          item_end = first_item;
        }
        // consecutive items are consecutive tiles (blocked assignment): step the tile coordinates
        int wt, ht, bt;
        tile_coords(p, first_item, wt, ht, bt);
        const unsigned free0 = p.one_commit ? tfull0 : empty0;   // "tile done" also frees the patch stage
        for (int item = first_item; ok && item < item_end; ++item) {
          if (owner == warp) {
            if (!mbar_wait_warp(free0 + 8 * stage, phase ^ 1, &abort_flag, status)) { ok = false; break; }
            const unsigned full = full0 + 8 * stage;
            if (leader) {
              mbar_expect_tx(full, (unsigned)p.a_box_bytes);
              tma_load_4d(smem_base + p.b_res_bytes + stage * p.a_bytes, &map_a, full, 0, wt * 8 - 1, ht * 16 - 1, bt);
            }
          }
          if (++owner == nprod) owner = 0;
          if (++stage == p.stages) { stage = 0; phase ^= 1; }
          if (++wt == p.w_tiles) { wt = 0; if (++ht == p.h_tiles) { ht = 0; ++bt; } }
        }
        item_end = first_item;                    // nothing left for the generic loop
      }
      // Tile transitions are on the critical path of the whole pipeline (while a producer decodes its
      // next tile no copy is issued and the ring runs dry; measured: ~1500 cycles of integer divisions
      // per tile cost a third of a 256-channel convolution).  Consecutive items of the convolutions
      // are consecutive tiles, so tile and pixel-box coordinates are stepped, not divided.
      const bool stepped = p.blocked && p.splits == 1 && p.raster_g <= 0;
      int c_mu = 0, c_nt = 0, c_wt = 0, c_ht = 0, c_bt = 0;
      for (int item = first_item; ok && item < item_end; item += item_step) {
        int mu, nt, split;
        int w0 = 0, h0 = 0, b0 = 0, tap_n = 0, ci0 = 0;
        if (stepped) {
          if (item == first_item) {
            decode_item(p, item, c_mu, c_nt, split);
            const int mt0 = c_mu * CTAS + (int)rank;
            tile_coords(p, mt0, c_wt, c_ht, c_bt);
          } else if (++c_nt == p.n_tiles_n) {
            c_nt = 0;
            ++c_mu;
            c_wt += CTAS;
            while (c_wt >= p.w_tiles) { c_wt -= p.w_tiles; if (++c_ht == p.h_tiles) { c_ht = 0; ++c_bt; } }
          }
          mu = c_mu; nt = c_nt; split = 0;
          w0 = c_wt * p.Wt; h0 = c_ht * p.Ht; b0 = c_bt * p.Bt;
        } else {
          decode_item(p, item, mu, nt, split);
          if (p.kind == GK_CONV_FWD || p.kind == GK_CONV_DGRAD) pixel_box(p, mu * CTAS + (int)rank, w0, h0, b0);
        }
        if (p.kind == GK_CONV_FWD) { w0 *= p.stride; h0 *= p.stride; }     // output pixel -> window origin in x
        const int mt = mu * CTAS + (int)rank;     // this CTA's 128-row tile
        const int nb = nt * p.bn + (int)rank * bn_cta;
        const int kb0 = split * p.kb_per_split;
        int kb1 = kb0 + p.kb_per_split;
        if (kb1 > p.kb_total) kb1 = p.kb_total;
        if (p.kind == GK_CONV_WGRAD) {
          tap_n = nt / p.n_chunks;
          ci0 = (nt % p.n_chunks) * p.bn + (int)rank * bn_cta;
        }
        // k-block counters, stepped instead of divided inside the loop (one thread issues all copies,
        // so every scalar instruction here is on the critical path):
        //   forward / dgrad: k-block = (tap row r, tap column s, channel chunk cc)
        //   wgrad:           k-block = pixel box (kwt, kht, kbt)
        int cc = 0, ts = 0, tr = 0, kwt = 0, kht = 0, kbt = 0;
        if (kb0 != 0) {
          if (p.kind == GK_CONV_FWD || p.kind == GK_CONV_DGRAD) {
            const int tap = kb0 / p.c_chunks;
            cc = kb0 % p.c_chunks; tr = tap / p.S; ts = tap % p.S;
          } else if (p.kind == GK_CONV_WGRAD) {
            kwt = kb0 % p.w_tiles;
            const int t = kb0 / p.w_tiles;
            kht = t % p.h_tiles; kbt = t / p.h_tiles;
          }
        }
        int wg_r = 0, wg_s = 0;
        if (p.kind == GK_CONV_WGRAD) { wg_r = tap_n / p.S; wg_s = tap_n % p.S; }
        const unsigned tx_bytes = (unsigned)(CTAS * (p.a_boxes * p.a_box_bytes + p.b_boxes * p.b_box_bytes));
        for (int kb = kb0; kb < kb1; ++kb) {
         if (owner == warp) {
          if (!mbar_wait_warp(empty0 + 8 * stage, phase ^ 1, &abort_flag, status)) { ok = false; break; }
          const unsigned full = lead_full0 + 8 * stage;
          const unsigned sa = smem_base + stage * stage_bytes;
          const unsigned sb = sa + p.a_bytes;
          if (leader) {
          if (rank == 0) mbar_expect_tx(full0 + 8 * stage, tx_bytes);
          switch (p.kind) {
            case GK_FC_FWD:       // A [M][K] K-major, B [N][K] K-major
              for (int j = 0; j < p.mrep; ++j)     // rows past the end of A are zero-filled by the copy
                load2<CTAS>(sa + j * p.a_box_bytes, &map_a, full, kb * p.kdepth, (mt * p.mrep + j) * BM);
              load2<CTAS>(sb, &map_b, full, kb * p.kdepth, nb);
              break;
            case GK_FC_DGRAD:     // A = e [M][N] K-major; B(k', n) = w[n][k'] MN-major
              load2<CTAS>(sa, &map_a, full, kb * p.kdepth, mt * BM);
              for (int j = 0; j < p.b_boxes; ++j)
                load2<CTAS>(sb + j * p.b_box_bytes, &map_b, full, nb + j * p.b_box_step, kb * p.kdepth);
              break;
            case GK_FC_WGRAD:     // A(n, m) = e[m][n] MN-major; B(k', m) = a[m][k'] MN-major
              for (int j = 0; j < p.a_boxes; ++j)
                load2<CTAS>(sa + j * p.a_box_bytes, &map_a, full, mt * BM + j * p.a_box_step, kb * p.kdepth);
              for (int j = 0; j < p.b_boxes; ++j)
                load2<CTAS>(sb + j * p.b_box_bytes, &map_b, full, nb + j * p.b_box_step, kb * p.kdepth);
              break;
            case GK_CONV_FWD:     // k-block = (tap, channel chunk)
              load4<CTAS>(sa, &map_a, full, cc * p.kdepth, w0 + ts - p.pad, h0 + tr - p.pad, b0);
              load2<CTAS>(sb, &map_b, full, kb * p.kdepth, nb);
              break;
            case GK_CONV_DGRAD: { // A = e shifted the other way; B(ci, (tap, co)) = w[co][tap][ci]
              load4<CTAS>(sa, &map_a, full, cc * p.kdepth, w0 - ts + p.pad, h0 - tr + p.pad, b0);
              const int col = (tr * p.S + ts) * p.Cn + nb;
              for (int j = 0; j < p.b_boxes; ++j)
                load2<CTAS>(sb + j * p.b_box_bytes, &map_b, full, col + j * p.b_box_step, cc * p.kdepth);
              break;
            }
            default: {            // GK_CONV_WGRAD: k-block = pixel box; A = e, B = x shifted by the tap
              const int kw0 = kwt * p.Wt, kh0 = kht * p.Ht, kbb0 = kbt * p.Bt;
              for (int j = 0; j < p.a_boxes; ++j)
                load4<CTAS>(sa + j * p.a_box_bytes, &map_a, full, mt * BM + j * p.a_box_step, kw0, kh0, kbb0);
              for (int j = 0; j < p.b_boxes; ++j)
                load4<CTAS>(sb + j * p.b_box_bytes, &map_b, full, ci0 + j * p.b_box_step, kw0 * p.stride + wg_s - p.pad,
                            kh0 * p.stride + wg_r - p.pad, kbb0);
              break;
            }
          }
          }
         }
          if (p.kind == GK_CONV_FWD || p.kind == GK_CONV_DGRAD) {
            if (++cc == p.c_chunks) { cc = 0; if (++ts == p.S) { ts = 0; ++tr; } }
          } else if (p.kind == GK_CONV_WGRAD) {
            if (++kwt == p.w_tiles) { kwt = 0; if (++kht == p.h_tiles) { kht = 0; ++kbt; } }
          }
          if (++owner == nprod) owner = 0;
          if (++stage == p.stages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == MMA_WARP) {
    // ================= MMA issuer (leader CTA only) =================
    // The whole warp runs the loops in lock step and one elected lane issues: with warp-uniform
    // control flow the descriptor arithmetic stays in the uniform datapath that feeds tcgen05.mma.
    if (rank == 0) {
      const bool leader = elect_one();
      int stage = 0;
      unsigned phase = 0;
      unsigned use = 0;                 // tiles processed by this CTA (pair)
      bool ok = true;
      if (p.halo == 2) {
        // tap pairs (0,1) (2,3) (4,5) (6,7) (8,-): patch row of the first tap and the row distance to
        // the second one (the leading-dimension stride between the two 64-channel halves of M)
        const unsigned a_hi = (unsigned)(p.a_desc >> 32), b_hi = (unsigned)(p.b_desc >> 32);
        const unsigned b_lo0 = (unsigned)p.b_desc;
        unsigned a_pair[5];
#pragma unroll
        for (int pi = 0; pi < 5; ++pi) {
          const int ta = 2 * pi, tb = 2 * pi + 1 < 9 ? 2 * pi + 1 : 2 * pi - 1;
          const int ra = (ta / 3) * 10 + ta % 3, rb = (tb / 3) * 10 + tb % 3;
          const int lbo_rows = rb > ra ? rb - ra : 1;
          a_pair[pi] = (unsigned)(ra * 4) | ((unsigned)(lbo_rows * 4) << 16);     // 64-byte rows, 16-byte units
        }
        for (int item = first_item; ok && item < item_end; item += item_step, ++use) {
          const int split = p.splits > 1 ? item % p.splits : 0;
          const int t0 = split * p.kb_per_split;
          int t1 = t0 + p.kb_per_split;
          if (t1 > p.kb_total) t1 = p.kb_total;
          if (!mbar_wait_warp(tempty0, (use & 1u) ^ 1u, &abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          for (int t = t0; t < t1; ++t) {
            if (!mbar_wait_warp(full0 + 8 * stage, phase, &abort_flag, status)) { ok = false; break; }
            tc_fence_after();
            const unsigned sa16 = ((smem_base + stage * stage_bytes) >> 4) & 0x3fff;
            const unsigned sb16 = ((smem_base + stage * stage_bytes + p.a_bytes) >> 4) & 0x3fff;
            const unsigned first = t > t0 ? 1u : 0u;
            if (leader) {
#pragma unroll
              for (int pi = 0; pi < 5; ++pi) {
#pragma unroll
                for (int j = 0; j < 4; ++j)      // 32 pixels = four rows of eight per MMA
                  tc_mma_i8_lh(tmem_base + 64u * pi, sa16 + a_pair[pi] + 160u * j, a_hi, b_lo0 + sb16 + 128u * j, b_hi,
                               p.idesc, j > 0 ? 1u : first);
              }
              tc_commit(empty0 + 8 * stage);
            }
            if (++stage == p.stages) { stage = 0; phase ^= 1; }
          }
          if (ok && leader) tc_commit(tfull0);
        }
        item_end = first_item;
      } else if (p.halo) {
        halo_mma_loop(p, 0, p.nissue, first_item, item_end, smem_base, tmem_base, full0, empty0, tfull0, tempty0,
                      bres_bar, &abort_flag, status);
        item_end = first_item;
      }
      // generic loop: everything an MMA needs that does not change is read into registers here
      const unsigned g_a_lo0 = (unsigned)p.a_desc, g_b_lo0 = (unsigned)p.b_desc;
      const unsigned g_a_hi = (unsigned)(p.a_desc >> 32), g_b_hi = (unsigned)(p.b_desc >> 32);
      const unsigned g_ak = p.a_kstep16, g_bk = p.b_kstep16, g_idesc = p.idesc, g_a_bytes = (unsigned)p.a_bytes;
      const int g_ksteps = p.ksteps, g_mrep = p.mrep;
      const unsigned g_bn_mma = (unsigned)p.bn_mma, g_slice16 = (unsigned)p.a_box_bytes >> 4;
      unsigned gbuf = 0, gpar = 0;            // use % nbuf, (use / nbuf) & 1, counted
      for (int item = first_item; ok && item < item_end; item += item_step, ++use) {
        const int split = p.splits > 1 ? item % p.splits : 0;
        const int kb0 = split * p.kb_per_split;
        int kb1 = kb0 + p.kb_per_split;
        if (kb1 > p.kb_total) kb1 = p.kb_total;
        const unsigned buf = gbuf;
        // wait until the epilogue has drained this accumulator buffer (the first nbuf uses pass at once)
        if (!mbar_wait_warp(tempty0 + 8 * buf, gpar ^ 1u, &abort_flag, status)) { ok = false; break; }
        if (++gbuf == (unsigned)p.nbuf) { gbuf = 0; gpar ^= 1u; }
        tc_fence_after();
        const unsigned tmem_d = tmem_base + buf * (unsigned)p.bn;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait_warp(full0 + 8 * stage, phase, &abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const unsigned sa = smem_base + stage * stage_bytes;
          const unsigned a_lo = g_a_lo0 + ((sa >> 4) & 0x3fff), b_lo = g_b_lo0 + (((sa + g_a_bytes) >> 4) & 0x3fff);
          const unsigned first_acc = kb > kb0 ? 1u : 0u;
          if (leader) {
            if (g_mrep > 1) {
              for (int j = 0; j < g_mrep; ++j) {
                const unsigned td = tmem_d + (unsigned)j * g_bn_mma, aj = a_lo + (unsigned)j * g_slice16;
                if (g_ksteps == 1) issue_kblock<CTAS, 1>(td, aj, g_a_hi, b_lo, g_b_hi, g_ak, g_bk, g_idesc, first_acc);
                else if (g_ksteps == 2) issue_kblock<CTAS, 2>(td, aj, g_a_hi, b_lo, g_b_hi, g_ak, g_bk, g_idesc, first_acc);
                else if (g_ksteps == 4) issue_kblock<CTAS, 4>(td, aj, g_a_hi, b_lo, g_b_hi, g_ak, g_bk, g_idesc, first_acc);
                else issue_kblock<CTAS, 3>(td, aj, g_a_hi, b_lo, g_b_hi, g_ak, g_bk, g_idesc, first_acc);
              }
            }
            else if (g_ksteps == 4) issue_kblock<CTAS, 4>(tmem_d, a_lo, g_a_hi, b_lo, g_b_hi, g_ak, g_bk, g_idesc, first_acc);
            else if (g_ksteps == 2) issue_kblock<CTAS, 2>(tmem_d, a_lo, g_a_hi, b_lo, g_b_hi, g_ak, g_bk, g_idesc, first_acc);
            else if (g_ksteps == 1) issue_kblock<CTAS, 1>(tmem_d, a_lo, g_a_hi, b_lo, g_b_hi, g_ak, g_bk, g_idesc, first_acc);
            else issue_kblock<CTAS, 3>(tmem_d, a_lo, g_a_hi, b_lo, g_b_hi, g_ak, g_bk, g_idesc, first_acc);
            // frees the stage (in every CTA of the pair) once these MMAs have read it
            if (CTAS == 2) tc_commit_pair(empty0 + 8 * stage); else tc_commit(empty0 + 8 * stage);
          }
          if (++stage == p.stages) { stage = 0; phase ^= 1; }
        }
        if (ok && leader) {                     // accumulator complete
          if (CTAS == 2) tc_commit_pair(tfull0 + 8 * buf); else tc_commit(tfull0 + 8 * buf);
        }
      }
    }
  } else if (((warp - EPI_WARP0) >> 2) % wpq < wpq_active) {
    // ================= epilogue: TMEM -> int32 accumulators + max magnitude =================
    const int quarter = warp & 3;               // TMEM lanes [32 * quarter, +32)
    const int wq = (warp - EPI_WARP0) >> 2;     // index among the four warps of this quarter
    const int egroup = wq / wpq;                // tiles use % egroups == egroup are this warp's
    const int chunk_phase = wq % wpq;           // it takes 32-column chunks phase, phase + wpq, ...
    const int row_in_tile = quarter * 32 + lane;
    unsigned use = 0;
    unsigned mx = 0;
    unsigned spec_max = 0;
    int bp = 0;
    int h_wt = 0, h_ht = 0, h_bt = 0;
    if (p.epi_mode == EPI_KNOWN_B) {
      const int b = niti_bitlen32(hdr->maxabs32);
      bp = b > p.mbits ? b - p.mbits : 0;
    }
    bool ok = true;
    if (p.halo == 2) {
      // lane = (tap of the pair, input channel), column = output channel; partial sums of this
      // CTA's pixel range are added to g32[co][tap][ci]
      const int which = row_in_tile >> 6, ci = row_in_tile & 63;
      for (int item = first_item; ok && item < item_end; item += item_step, ++use) {
        const int blk = (int)(item / p.splits);
        const int ci0 = (blk % p.wg_nci) * 64, co0 = (blk / p.wg_nci) * 64;
        if (!mbar_wait(tfull0, use & 1u, &abort_flag, status)) { ok = false; break; }
        tc_fence_after();
        unsigned pmx = 0;                       // largest partial-sum magnitude of this item
        for (int job = chunk_phase; job < 10; job += wpq) {
          const int pi = job >> 1, c0 = (job & 1) * 32;
          const int tap = 2 * pi + which;
          int v[32];
          tc_ld32(tmem_base + ((unsigned)(quarter * 32) << 16) + 64u * pi + (unsigned)c0, v);
          if (tap < 9) {
            int32_t *dst = acc + (long long)(co0 + c0) * p.gn + (long long)tap * p.Cn + ci0 + ci;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              pmx = max(pmx, (unsigned)abs(v[j]));
              if (v[j] != 0) atomicAdd(dst + (long long)j * p.gn, v[j]);
            }
          }
        }
        pmx = __reduce_max_sync(0xffffffffu, pmx);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (pmx) atomicMax(niti_split_max(hdr) + (p.splits > 1 ? item % p.splits : 0), pmx);
          mbar_arrive(tempty0);
        }
      }
      item_end = first_item;
    }
    use = (unsigned)egroup;
    unsigned ebuf = (unsigned)egroup, epar = 0;       // use % nbuf, (use / nbuf) & 1 (nbuf is a multiple of egroups)
    // what the fused rounding needs and no tile changes: the rounding constants (replaced once, when the
    // speculative binary point is agreed) and the alignment of the output and mask rows
    RoundConst rk = make_round_const(bp, p.mbits, p.round_mode);
    const bool io_aligned = ((p.gn & 31) == 0) && (((uintptr_t)out8 & 31) == 0) &&
                            (mask8 == nullptr || ((uintptr_t)mask8 & 31) == 0);
    // the lean loop takes over after a warp's first item (which may be the CTA's speculative first
    // tile) when every chunk of every tile is whole and aligned
    const bool lean_ok = (p.epi_mode == EPI_KNOWN_B || p.epi_mode == EPI_SPECULATE) && io_aligned && p.splits == 1 &&
                         (p.bn & 31) == 0 && p.halo != 2 && p.kind != GK_CONV_WGRAD &&
                         (p.mrep == 1 || (p.gn == p.bn_mma && mask8 == nullptr));
    int lean_item = -1;
    Extremes ex_all = {0, 0, 0u};
    // this thread's pixel inside a pixel box (generic convolutions): the box sides are powers of two
    const int wt_d = p.Wt > 0 ? p.Wt : 1, ht_d = p.Ht > 0 ? p.Ht : 1;     // (unset for plain matrix multiplies)
    const int r_ww = row_in_tile % wt_d, r_t = row_in_tile / wt_d;
    const int r_hh = r_t % ht_d, r_bb = r_t / ht_d;
    for (int item = first_item + egroup * item_step; ok && item < item_end;
         item += item_step * egroups, use += (unsigned)egroups) {
      int mu = 0, nt = 0, split = 0;
      if (!p.halo) decode_item(p, item, mu, nt, split);
      const int mt = mu * CTAS + (int)rank;
      const unsigned buf = ebuf;
      const unsigned tpar = epar;
      ebuf += (unsigned)egroups;
      if (ebuf >= (unsigned)p.nbuf) { ebuf -= (unsigned)p.nbuf; epar ^= 1u; }
      // output row / column base of this thread
      long long out_row;
      bool row_ok;
      long long col0;
      int ncols_valid;
      if (p.halo) {
        // 8 x 16 pixel tiles of one image, visited in order: coordinates are stepped, not divided
        if (use == (unsigned)egroup) {
          tile_coords(p, item, h_wt, h_ht, h_bt);
        }
        const int w = h_wt * 8 + (row_in_tile & 7), h = h_ht * 16 + (row_in_tile >> 3);
        row_ok = w < p.PW && h < p.PH;
        out_row = ((long long)h_bt * p.PH + h) * p.PW + w;
        col0 = 0;
        ncols_valid = (int)p.gn;
        for (int st = 0; st < egroups; ++st)
          if (++h_wt == p.w_tiles) { h_wt = 0; if (++h_ht == p.h_tiles) { h_ht = 0; ++h_bt; } }
      } else if (p.kind == GK_CONV_FWD || p.kind == GK_CONV_DGRAD) {
        int w0, h0, b0;
        pixel_box(p, mt, w0, h0, b0);
        const int ww = r_ww, hh = r_hh, bb = r_bb;
        int w = w0 + ww, h = h0 + hh, b = b0 + bb;
        row_ok = w < p.PW && h < p.PH && b < p.PB;
        out_row = ((long long)b * p.PH + h) * p.PW + w;
        col0 = (long long)nt * p.bn;
        long long rem = p.gn - col0;
        ncols_valid = rem < p.bn ? (int)rem : p.bn;
      } else if (p.kind == GK_CONV_WGRAD) {
        out_row = (long long)mt * BM + row_in_tile;
        row_ok = out_row < p.gm;
        int tap = nt / p.n_chunks, ci0 = (nt % p.n_chunks) * p.bn;
        col0 = (long long)tap * p.Cn + ci0;
        int rem = p.Cn - ci0;
        ncols_valid = rem < p.bn ? rem : p.bn;
      } else {
        // (row-batched mode: the row of the first of the item's mrep tiles; column chunk c of the
        // accumulator then belongs to tile c / bn_mma)
        out_row = (long long)mt * (BM * p.mrep) + row_in_tile;
        row_ok = out_row < p.gm;
        col0 = (long long)nt * p.bn;
        long long rem = p.gn - col0;
        ncols_valid = rem < p.bn ? (int)rem : p.bn;
      }
      // fused 2 x 2 max-pool (convolutions only): this lane's pixel and the row of its window in the pooled tensor
      long long pool_row = 0;
      if (p.pool) {
        const long long pw = out_row % p.PW, t2 = out_row / p.PW;
        const long long ph = t2 % p.PH, pb = t2 / p.PH;
        pool_row = (pb * (p.PH >> 1) + (ph >> 1)) * (p.PW >> 1) + (pw >> 1);
      }
      if (!mbar_wait(tfull0 + 8 * buf, tpar, &abort_flag, status)) { ok = false; break; }
      tc_fence_after();
      const unsigned tm_row = tmem_base + ((unsigned)(quarter * 32) << 16) + buf * (unsigned)p.bn;
      if (p.epi_mode == EPI_ATOMIC && p.stg_off > 0) {
        // Partial sums of a split contraction.  A lane holds one row of the chunk, so an atomic add
        // issued straight from the registers touches 32 different lines; the chunk is transposed
        // through shared memory instead and every add instruction covers 32 consecutive columns of
        // one row (one 128-byte line).  Output rows are consecutive here (no pixel-box mapping).
        int *stg = reinterpret_cast<int *>(smem_raw + (smem_base - smem_u32(smem_raw)) + p.stg_off) +
                   (warp - EPI_WARP0) * (32 * 33);
        const long long row0 = out_row - lane;                 // output row of lane 0 of this warp
        unsigned pmx = 0;                                      // largest partial-sum magnitude of this item
        for (int c = 32 * chunk_phase; c < p.bn; c += 32 * wpq) {
          int v[32];
          tc_ld32(tm_row + (unsigned)c, v);
          if (c < ncols_valid) {                               // (uniform across the warp)
#pragma unroll
            for (int j = 0; j < 32; ++j) { stg[lane * 33 + j] = v[j]; pmx = max(pmx, (unsigned)abs(v[j])); }
            __syncwarp();
            const bool col_ok = c + lane < ncols_valid;
            int32_t *dcol = acc + row0 * p.gn + col0 + c + lane;
            long long rows_left = p.gm - row0;
            if (rows_left > 32) rows_left = 32;
            for (int rr = 0; rr < (int)rows_left; ++rr) {
              const int val = stg[rr * 33 + lane];
              if (col_ok && val != 0) atomicAdd(dcol + (long long)rr * p.gn, val);
            }
            __syncwarp();
          }
        }
        pmx = __reduce_max_sync(0xffffffffu, pmx);
        if (lane == 0 && pmx) atomicMax(niti_split_max(hdr) + split, pmx);
      } else if (p.epi_mode <= EPI_ATOMIC || p.epi_mode == EPI_PARTIAL) {
        int32_t *dst = acc + out_row * p.gn + col0;
        if (p.epi_mode == EPI_PARTIAL) dst += (long long)split * p.gm * p.gn;      // this split's slice
        const bool vec_ok = ((p.gn & 3) == 0) && ((col0 & 3) == 0);
        unsigned pmx = 0;                                      // largest partial-sum magnitude of this item
        for (int c = 32 * chunk_phase; c < p.bn; c += 32 * wpq) {
          int v[32];
          tc_ld32(tm_row + (unsigned)c, v);
          if (row_ok && c < ncols_valid) {
            if (p.epi_mode == EPI_ATOMIC) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (c + j < ncols_valid && v[j] != 0) {
                  pmx = max(pmx, (unsigned)abs(v[j]));
                  atomicAdd(dst + c + j, v[j]);
                }
            } else {
              if (vec_ok && c + 32 <= ncols_valid) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                  *reinterpret_cast<int4 *>(dst + c + j) = make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  unsigned a = v[j] < 0 ? 0u - (unsigned)v[j] : (unsigned)v[j];
                  mx = a > mx ? a : mx;
                }
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (c + j < ncols_valid) {
                    dst[c + j] = v[j];
                    unsigned a = v[j] < 0 ? 0u - (unsigned)v[j] : (unsigned)v[j];
                    mx = a > mx ? a : mx;
                  }
              }
            }
          }
        }
        if (p.epi_mode == EPI_ATOMIC) {
          pmx = __reduce_max_sync(0xffffffffu, pmx);
          if (lane == 0 && pmx) atomicMax(niti_split_max(hdr) + split, pmx);
        }
      } else {
        if (p.epi_mode == EPI_SPECULATE && use == (unsigned)egroup && egroup != 0) {
          // the group that drains this CTA's first tile publishes the shift through shared memory
          long long t0 = clock64();
          while (spec_bp_ready == 0) {
            if (abort_flag) break;
            if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
              abort_flag = 1;
              atomicOr(status, NITI_DEV_TIMEOUT);
              break;
            }
          }
          if (abort_flag) { ok = false; break; }
          bp = spec_bp_ready - 1;
          rk = make_round_const(bp, p.mbits, p.round_mode);
        }
        if (p.epi_mode == EPI_SPECULATE && use == 0) {
          // first tile of this CTA: max only, then agree on the estimate with the whole grid
          unsigned m0 = 0;
          for (int c = 32 * chunk_phase; c < p.bn; c += 32 * wpq) {
            int v[32];
            tc_ld32(tm_row + (unsigned)c, v);
            int cc = c;
            bool rok = row_ok;
            if (p.mrep > 1) {
              const int jt = c / p.bn_mma;
              cc = c - jt * p.bn_mma;
              rok = out_row + (long long)jt * BM < p.gm;
            }
            if (rok) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (cc + j < ncols_valid) {
                  unsigned a = v[j] < 0 ? 0u - (unsigned)v[j] : (unsigned)v[j];
                  m0 = a > m0 ? a : m0;
                }
            }
          }
          for (int o = 16; o > 0; o >>= 1) {
            unsigned u = __shfl_xor_sync(0xffffffffu, m0, o);
            m0 = u > m0 ? u : m0;
          }
          // The warps of this CTA combine their maxima in shared memory; the last one to report speaks
          // for the CTA in the grid-wide agreement (one atomic and one poller per CTA: with every warp
          // of every CTA polling the same word the wait itself took microseconds) and publishes the
          // shift to the others through shared memory.
          if (lane == 0) {
            if (m0) atomicMax(&first_max, m0);
            __threadfence_block();
            if (atomicAdd(&first_arrived, 1u) + 1u == (unsigned)epi_active) {
              const unsigned cm = *(volatile unsigned *)&first_max;
              if (cm) atomicMax(&hdr->est_max, cm);
              __threadfence();
              atomicAdd(&hdr->tile_counter, 1u);
              // The bit-width is fixed as soon as a quorum of CTAs has reported, by whichever CTA sees
              // that first (compare-and-swap on the published word); CTAs that start late find it
              // published and never wait.  Waiting for every CTA meant waiting out the launch ramp of
              // the whole grid (~10 k cycles) in every launch.
              const unsigned quorum = (unsigned)p.quorum;
              unsigned pub = 0;
              long long t0 = clock64();
              while (true) {
                // one 16-byte load: {est_max, tile_counter, spec_b, -}
                unsigned v_max, v_cnt, v_pub, v_pad;
                asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(v_max), "=r"(v_cnt), "=r"(v_pub), "=r"(v_pad)
                             : "l"(&hdr->est_max)
                             : "memory");
                if (v_pub) { pub = v_pub; break; }
                if (v_cnt >= quorum) {
                  // (the 16-byte load is not promised to be one atomic snapshot: once the count is seen,
                  // the maximum is read again, after a fence, so that it is at least as new as the count)
                  __threadfence();
                  v_max = *(volatile unsigned *)&hdr->est_max;
                  // the first tiles are a sample: scale their max by the growth expected from the sample
                  // to the whole tensor before taking the bit length (a wrong guess only costs the redo)
                  unsigned long long scaled = ((unsigned long long)v_max * p.spec_mul256) >> 8;
                  if (scaled > 0x7fffffffull) scaled = 0x7fffffffull;
                  // plus what the same estimate missed by at this call site last time (a systematic
                  // error of the sample, e.g. a tensor whose extremes sit outside the first tiles); never
                  // below the bit length of the sample's own maximum, which the tensor's cannot undercut
                  int guess = niti_bitlen32((unsigned)scaled);
                  if (spec_slot && p.spec_mul256 != 256 && *(volatile int *)&spec_slot[0] == p.spec_tag)
                    guess += spec_correction(*(volatile int *)&spec_slot[1]);
                  const int floor_b = niti_bitlen32(v_max);
                  guess = guess < floor_b ? floor_b : (guess > 31 ? 31 : guess);
                  const unsigned mine = (unsigned)guess + 1u;
                  const unsigned old = atomicCAS(&hdr->spec_b, 0u, mine);
                  pub = old ? old : mine;
                  break;
                }
                if (abort_flag) break;
                if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
                  abort_flag = 1;
                  atomicOr(status, NITI_DEV_TIMEOUT);
                  break;
                }
              }
              const int b = (int)pub - 1;
              spec_bp_ready = (b > p.mbits ? b - p.mbits : 0) + 1;
            }
            long long t1 = clock64();
            while (spec_bp_ready == 0) {
              if (abort_flag) break;
              if (clock64() - t1 > WAIT_LIMIT_CYCLES) {
                abort_flag = 1;
                atomicOr(status, NITI_DEV_TIMEOUT);
                break;
              }
            }
          }
          __syncwarp();
          if (abort_flag) { ok = false; break; }
          bp = spec_bp_ready - 1;
          rk = make_round_const(bp, p.mbits, p.round_mode);
        }
        const bool vec_ok = ((p.gn & 15) == 0) && ((col0 & 15) == 0);
        const bool vec32_ok = ((p.gn & 31) == 0) && ((col0 & 31) == 0) && (((uintptr_t)out8 & 31) == 0);
        // Whole 32-column chunks with 32-byte aligned rows (every layer of the networks): the chunk
        // loop below does nothing per chunk but load, round and store; pointers are stepped.  (The
        // epilogue warps share their schedulers' integer pipe, which is the bound of layers with few
        // input channels: every instruction here is paid for 16 times per tile.)
        const bool whole_chunks = io_aligned && ((col0 & 31) == 0) &&
                                  (p.mrep > 1 ? ncols_valid >= p.bn_mma : (ncols_valid & 31) == 0);
        if (whole_chunks) {
          const bool relu = p.relu != 0;
          // (the last column tile of a row may be narrower than the tile: its chunks beyond the
          // matrix are not read at all)
          const int cstep = 32 * wpq, bn = p.mrep > 1 ? p.bn : (ncols_valid < p.bn ? ncols_valid : p.bn);
          const int bn_mma = p.mrep > 1 ? p.bn_mma : p.bn;
          const long long row_off = out_row * p.gn + col0;
          const long long sub_stride = (long long)BM * p.gn;      // next 128-row tile of a row-batched item
          int8_t *drow = out8 + row_off;
          const int8_t *mrow = mask8 ? mask8 + row_off : nullptr;
          long long orow = out_row;
          int cc = 32 * chunk_phase;
          while (cc >= bn_mma) { cc -= bn_mma; orow += BM; drow += sub_stride; if (mrow) mrow += sub_stride; }
          for (int c = 32 * chunk_phase; c < bn; c += cstep) {
            int v[32];
            const bool rok = row_ok && orow < p.gm;
            unsigned m[8];
            unsigned pw8[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};     // pooling input of lanes outside the tensor
            if ((mrow || p.update) && rok)        // the ReLU mask, or the weights this chunk updates
              asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                           : "=r"(m[0]), "=r"(m[1]), "=r"(m[2]), "=r"(m[3]), "=r"(m[4]), "=r"(m[5]), "=r"(m[6]), "=r"(m[7])
                           : "l"((p.update ? (const int8_t *)drow : mrow) + cc));
            tc_ld32(tm_row + (unsigned)c, v);
            if (rok) {
              unsigned w8[8];
              Extremes ex = {0, 0, 0u};
              round_chunk32(v, w8, rk, relu, ex);
              mx |= ex.magnitude_bits();
              if (p.update) {
#pragma unroll
                for (int j = 0; j < 8; ++j) w8[j] = bytes_sub_clamp127(m[j], w8[j]);
              } else if (mrow) {
#pragma unroll
                for (int j = 0; j < 8; ++j) w8[j] &= bytes_gt0(m[j]);
              }
              asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                           ::"l"(drow + cc), "r"(w8[0]), "r"(w8[1]), "r"(w8[2]), "r"(w8[3]), "r"(w8[4]), "r"(w8[5]),
                             "r"(w8[6]), "r"(w8[7])
                           : "memory");
              if (p.pool) {
#pragma unroll
                for (int j = 0; j < 8; ++j) pw8[j] = w8[j];
              }
            }
            if (p.pool) {                          // (warp-uniform: every lane takes part in the exchange)
              pool_chunk32(pw8, p.pool_xh);
              if (rok && (lane & (1 | p.pool_xh)) == 0) store32(pool8 + pool_row * p.gn + col0 + cc, pw8);
            }
            cc += cstep;
            while (cc >= bn_mma) { cc -= bn_mma; orow += BM; drow += sub_stride; if (mrow) mrow += sub_stride; }
          }
        } else
        for (int c = 32 * chunk_phase; c < p.bn; c += 32 * wpq) {
          int v[32];
          // chunk geometry: in row-batched mode chunk c holds columns cc of the item's tile c / bn_mma
          int cc = c;
          long long orow = out_row;
          bool rok = row_ok;
          if (p.mrep > 1) {
            const int jt = c / p.bn_mma;
            cc = c - jt * p.bn_mma;
            orow = out_row + (long long)jt * BM;
            rok = orow < p.gm;
          }
          int8_t *dst8 = out8 + orow * p.gn + col0;
          const int8_t *msk = mask8 ? mask8 + orow * p.gn + col0 : nullptr;
          // the ReLU mask bytes are fetched first so that their latency overlaps the TMEM load and
          // the rounding arithmetic
          int4 m0v = make_int4(0x01010101, 0x01010101, 0x01010101, 0x01010101), m1v = m0v;
          if (msk && vec_ok && rok && cc + 32 <= ncols_valid) {
            if (vec32_ok && (((uintptr_t)mask8 & 31) == 0)) {
              asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                           : "=r"(m0v.x), "=r"(m0v.y), "=r"(m0v.z), "=r"(m0v.w), "=r"(m1v.x), "=r"(m1v.y), "=r"(m1v.z),
                             "=r"(m1v.w)
                           : "l"(msk + cc));
            } else {
              m0v = *reinterpret_cast<const int4 *>(msk + cc);
              m1v = *reinterpret_cast<const int4 *>(msk + cc + 16);
            }
          }
          tc_ld32(tm_row + (unsigned)c, v);
          if (rok && cc < ncols_valid) {
            unsigned w8[8];
            Extremes ex = {0, 0, 0u};
            round_chunk32(v, w8, rk, p.relu != 0, ex);
            if (vec_ok && cc + 32 <= ncols_valid) {
              mx |= ex.magnitude_bits();
              if (msk) {
                w8[0] &= bytes_gt0(m0v.x); w8[1] &= bytes_gt0(m0v.y);
                w8[2] &= bytes_gt0(m0v.z); w8[3] &= bytes_gt0(m0v.w);
                w8[4] &= bytes_gt0(m1v.x); w8[5] &= bytes_gt0(m1v.y);
                w8[6] &= bytes_gt0(m1v.z); w8[7] &= bytes_gt0(m1v.w);
              }
              if (vec32_ok) {
                // one 32-byte sector per lane in a single request (half as many store requests)
                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                             ::"l"(dst8 + cc), "r"(w8[0]), "r"(w8[1]), "r"(w8[2]), "r"(w8[3]), "r"(w8[4]), "r"(w8[5]),
                               "r"(w8[6]), "r"(w8[7])
                             : "memory");
              } else {
                *reinterpret_cast<int4 *>(dst8 + cc) = make_int4(w8[0], w8[1], w8[2], w8[3]);
                *reinterpret_cast<int4 *>(dst8 + cc + 16) = make_int4(w8[4], w8[5], w8[6], w8[7]);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (cc + j < ncols_valid) {
                  mx |= (unsigned)abs(v[j]);
                  int8_t q = (int8_t)((w8[j >> 2] >> (8 * (j & 3))) & 0xff);
                  if (msk && msk[cc + j] <= 0) q = 0;
                  dst8[cc + j] = q;
                }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (CTAS == 2 && rank != 0) mbar_arrive_cluster(lead_tempty0 + 8 * buf);
        else mbar_arrive(tempty0 + 8 * buf);
      }
      if (lean_ok && rk.aligned) {                 // the rest of this warp's items: lean loop below
        lean_item = item + item_step * egroups;
        use += (unsigned)egroups;
        break;
      }
    }
    // ---- lean loop: fused rounding of whole, aligned chunks (every layer of the networks) ----
    // The epilogue warps share their schedulers' integer pipe with everything else, and with few
    // input channels that pipe is the bound of the whole kernel: per tile and per chunk this loop
    // executes only what changes (measured on the first layer: the general loop above spends a third
    // of its integer instructions on tests whose outcome is the same for every tile).
    if (ok && lean_item >= 0) {
      auto lean = [&](auto relu_c, auto mask_c, auto batched_c, auto pool_c, auto upd_c) {
        constexpr bool RELU = decltype(relu_c)::value, MASK = decltype(mask_c)::value, BATCHED = decltype(batched_c)::value;
        constexpr bool POOL = decltype(pool_c)::value;       // fused 2 x 2 max-pool of the ReLU'd tile
        constexpr bool UPD = decltype(upd_c)::value;         // the output rows are weights: subtract the rounded gradient
        const int pool_xh = p.pool_xh;
        const bool pool_lane = (lane & (1 | pool_xh)) == 0;  // the window's top-left pixel stores the maximum
        const int kind = p.halo ? 0 : ((p.kind == GK_CONV_FWD || p.kind == GK_CONV_DGRAD) ? 1 : 2);
        const int istep = item_step * egroups, nbuf = p.nbuf, bn = p.bn, n_tiles_n = p.n_tiles_n;
        const int cstep = 32 * wpq, c_first = 32 * chunk_phase;
        const long long gn = p.gn, gm = p.gm;
        const int bn_mma = BATCHED ? p.bn_mma : p.bn;
        const long long sub_stride = (long long)BM * gn;
        const bool counted = p.blocked && p.raster_g <= 0;     // consecutive items: (mu, nt) are stepped
        int mu = 0, nt = 0, split = 0;
        if (kind != 0) decode_item(p, lean_item, mu, nt, split);
        for (int item = lean_item; item < item_end; item += istep) {
          const unsigned buf = ebuf, tpar = epar;
          ebuf += (unsigned)egroups;
          if (ebuf >= (unsigned)nbuf) { ebuf -= (unsigned)nbuf; epar ^= 1u; }
          long long out_row;
          bool row_ok;
          long long pool_row = 0;
          if (kind == 0) {
            const int w = h_wt * 8 + (row_in_tile & 7), h = h_ht * 16 + (row_in_tile >> 3);
            row_ok = w < p.PW && h < p.PH;
            out_row = ((long long)h_bt * p.PH + h) * p.PW + w;
            if (POOL) pool_row = ((long long)h_bt * (p.PH >> 1) + (h >> 1)) * (p.PW >> 1) + (w >> 1);
            h_wt += egroups;
            while (h_wt >= p.w_tiles) { h_wt -= p.w_tiles; if (++h_ht == p.h_tiles) { h_ht = 0; ++h_bt; } }
          } else if (kind == 1) {
            int w0, h0, b0;
            pixel_box(p, mu * CTAS + (int)rank, w0, h0, b0);
            const int w = w0 + r_ww, h = h0 + r_hh, b = b0 + r_bb;
            row_ok = w < p.PW && h < p.PH && b < p.PB;
            out_row = ((long long)b * p.PH + h) * p.PW + w;
            if (POOL) pool_row = ((long long)b * (p.PH >> 1) + (h >> 1)) * (p.PW >> 1) + (w >> 1);
          } else {
            out_row = (long long)(mu * CTAS + (int)rank) * (BM * p.mrep) + row_in_tile;
            row_ok = out_row < gm;
          }
          const int col0 = nt * bn;
          int cend = BATCHED ? bn : (int)(gn - col0);          // (whole chunks: gn is a multiple of 32)
          if (cend > bn) cend = bn;
          if (kind != 0) {                                      // next item of this warp
            if (counted) { nt += egroups; while (nt >= n_tiles_n) { nt -= n_tiles_n; ++mu; } }
            else if (item + istep < item_end) decode_item(p, item + istep, mu, nt, split);
          }
          if (!mbar_wait(tfull0 + 8 * buf, tpar, &abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const unsigned tm_row = tmem_base + ((unsigned)(quarter * 32) << 16) + buf * (unsigned)bn;
          const long long row_off = out_row * gn + col0;
          int8_t *drow = out8 + row_off;
          const int8_t *mrow = MASK ? mask8 + row_off : nullptr;
          int8_t *prow = POOL ? pool8 + pool_row * gn + col0 : nullptr;
          long long orow = out_row;
          int cc = c_first;
          if (BATCHED) while (cc >= bn_mma) { cc -= bn_mma; orow += BM; drow += sub_stride; if (MASK) mrow += sub_stride; }
          for (int c = c_first; c < cend; c += cstep) {
            int v[32];
            const bool rok = BATCHED ? (row_ok && orow < gm) : row_ok;
            unsigned m[8];
            if ((MASK || UPD) && rok)
              asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                           : "=r"(m[0]), "=r"(m[1]), "=r"(m[2]), "=r"(m[3]), "=r"(m[4]), "=r"(m[5]), "=r"(m[6]), "=r"(m[7])
                           : "l"((UPD ? (const int8_t *)drow : mrow) + cc));
            tc_ld32(tm_row + (unsigned)c, v);
            unsigned w8[8];
            if (POOL) {
#pragma unroll
              for (int j = 0; j < 8; ++j) w8[j] = 0u;          // lanes outside the tensor pool zeros
            }
            if (rok) {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                w8[j] = round_pack4_aligned<RELU>(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3], rk, ex_all);
                if (MASK) w8[j] &= bytes_gt0(m[j]);
                if (UPD) w8[j] = bytes_sub_clamp127(m[j], w8[j]);
              }
              store32(drow + cc, w8);
            }
            if (POOL) {                                        // (warp-uniform: all lanes exchange)
              pool_chunk32(w8, pool_xh);
              if (rok && pool_lane) store32(prow + cc, w8);
            }
            cc += cstep;
            if (BATCHED) while (cc >= bn_mma) { cc -= bn_mma; orow += BM; drow += sub_stride; if (MASK) mrow += sub_stride; }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (CTAS == 2 && rank != 0) mbar_arrive_cluster(lead_tempty0 + 8 * buf);
            else mbar_arrive(tempty0 + 8 * buf);
          }
        }
      };
      using T = std::true_type;
      using F = std::false_type;
      const bool relu = p.relu != 0, masked = mask8 != nullptr, batched = p.mrep > 1;
      if (batched) { if (relu) lean(T{}, F{}, T{}, F{}, F{}); else lean(F{}, F{}, T{}, F{}, F{}); }   // (row-batched: forward only)
      else if (p.update) lean(F{}, F{}, F{}, F{}, T{});                                              // (weight gradients: signed, no mask)
      else if (p.pool) lean(T{}, F{}, F{}, T{}, F{});                                                // (pooling: ReLU, no mask)
      else if (relu) { if (masked) lean(T{}, T{}, F{}, F{}, F{}); else lean(T{}, F{}, F{}, F{}, F{}); }
      else { if (masked) lean(F{}, T{}, F{}, F{}, F{}); else lean(F{}, F{}, F{}, F{}, F{}); }
      mx |= ex_all.magnitude_bits();
    }
    if (p.epi_mode == EPI_SPILL || p.epi_mode == EPI_SPECULATE) {
      for (int o = 16; o > 0; o >>= 1) {
        unsigned u = __shfl_xor_sync(0xffffffffu, mx, o);
        mx = u > mx ? u : mx;
      }
      if (lane == 0 && mx) atomicMax(&cta_max, mx);     // (one global atomic per CTA, below)
    }
  }

  // ================= common exit =================
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && cta_max) atomicMax(&hdr->maxabs32, cta_max);
  if (abort_flag) {
    // give copies and MMAs still in flight time to land before shared and tensor memory go away
    long long t0 = clock64();
    while (clock64() - t0 < 20000000LL) {
    }
    __syncthreads();
  }
  if (p.single_wave && p.epi_mode == EPI_SPECULATE && threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(&hdr->done_ctas, 1u) == gridDim.x - 1) {
      __threadfence();
      const int b_true = niti_bitlen32(*(volatile unsigned *)&hdr->maxabs32);
      const int bpf = b_true > p.mbits ? b_true - p.mbits : 0;
      // the shift every CTA rounded with came from the agreed maximum over ALL tiles, so it must be the
      // true one; anything else means the agreement was broken and the stored int8 values are not exact
      if (b_true != (int)(*(volatile unsigned *)&hdr->spec_b) - 1) atomicOr(status, NITI_DEV_INTERNAL);
      if (b_out) *b_out = b_true;
      if (s_out) {
        int sv = bpf + (s_a ? *s_a : 0) + (s_w ? *s_w : 0);
        *s_out = sv;
        if (sv < -128 || sv > 127) atomicOr(status, NITI_DEV_EXP_RANGE);
      }
    }
  }
  if (CTAS == 2) cluster_sync_all();   // nobody leaves while the peer may still touch this CTA
  if (warp == MMA_WARP) {
    tc_fence_after();
    if (CTAS == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever completes, gives up
// after ~50 ms, raises NITI_DEV_TIMEOUT and returns normally (the context stays usable).
__global__ void timeout_probe_kernel(uint32_t *status) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ volatile int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) (void)mbar_wait(smem_u32(&bar), 0, &abort_flag, status, 100000000LL);
  __syncthreads();
}

// ------------------------------------------------------------------------------------------
// Host side: tensor maps, descriptors, eligibility
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static CUtensorMapSwizzle swizzle_enum(int bytes) {
  return bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}
static unsigned long long layout_bits(int swizzle_bytes) {
  // matrix-descriptor layout type: 2 = 128-byte swizzle, 4 = 64-byte, 6 = 32-byte
  unsigned long long t = swizzle_bytes == 128 ? 2 : (swizzle_bytes == 64 ? 4 : 6);
  return t << 61;
}
// Descriptor (without start address) of a K-major operand whose rows are `sw` bytes wide.
static unsigned long long desc_kmajor(int sw, int group_rows = 8) {
  unsigned long long d = 0;
  d |= (unsigned long long)1 << 16;                          // leading byte offset: unused, 1
  d |= (unsigned long long)((group_rows * sw) >> 4) << 32;   // stride between 8-row groups
  d |= (unsigned long long)1 << 46;                          // descriptor version
  return d | layout_bits(sw);
}
// Descriptor of an MN-major operand stored as sub-tiles [kdepth rows][sw bytes].
static unsigned long long desc_mnmajor(int sw, int kdepth) {
  unsigned long long d = 0;
  d |= (unsigned long long)((kdepth * sw) >> 4) << 16;       // next sw-wide chunk along M/N
  d |= (unsigned long long)((8 * sw) >> 4) << 32;            // next group of 8 k-rows
  d |= (unsigned long long)1 << 46;
  return d | layout_bits(sw);
}
static int pick_swizzle(long long extent) { return extent >= 128 ? 128 : (extent >= 64 ? 64 : (extent >= 32 ? 32 : 0)); }

struct MapSpec {
  int nd;
  cuuint64_t dims[4];
  cuuint64_t strides[3];   // bytes, dims 1..3
  cuuint32_t box[4];       // extent of the box in tensor elements (before the element stride)
  int swizzle;
  const void *base;
  cuuint32_t estr[4];      // element (traversal) stride per dimension; 0 = 1
};

static bool encode(niti_ctx *ctx, CUtensorMap *m, const MapSpec &s) {
  if (!ctx->encode_tiled) return false;
  if (((uintptr_t)s.base & 15) != 0) return false;
  for (int i = 0; i + 1 < s.nd; ++i)
    if (s.strides[i] % 16 != 0) return false;
  for (int i = 0; i < s.nd; ++i)
    if (s.box[i] == 0 || s.box[i] > 256) return false;
  cuuint32_t es[4] = {1, 1, 1, 1};
  for (int i = 0; i < s.nd; ++i)
    if (s.estr[i] > 1) es[i] = s.estr[i];
  CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)s.nd,
                                                  const_cast<void *>(s.base), s.dims, s.strides, s.box, es,
                                                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_enum(s.swizzle),
                                                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Pixel box with Wt * Ht * Bt == 128 (powers of two).
static bool pick_pixel_box(int W, int H, int B, int &Wt, int &Ht, int &Bt) {
  Wt = 1;
  while (Wt < 128 && W % (Wt * 2) == 0) Wt *= 2;
  Ht = 1;
  while (Wt * Ht < 128 && H % (Ht * 2) == 0) Ht *= 2;
  Bt = 128 / (Wt * Ht);
  if (Bt > 256) return false;
  return Wt <= W && Ht <= H && Bt <= B;
}

static int round_up32(long long n) { return (int)((n + 31) / 32 * 32); }

// Builds params and maps; returns false if the shape is not eligible for this engine.
static bool plan(niti_ctx *ctx, const GemmProblem &g, int ctas, bool want_halo, TcParams &p, CUtensorMap &ma,
                 CUtensorMap &mb) {
  memset(&p, 0, sizeof(p));
  p.ctas = ctas;
  p.kind = g.kind;
  p.gm = g.gm;
  p.gn = g.gn;
  p.splits = 1;
  MapSpec sa, sb;
  memset(&sa, 0, sizeof(sa));
  memset(&sb, 0, sizeof(sb));
  int a_mn = 0, b_mn = 0;        // 1 = MN-major operand
  int a_sw = 0, b_sw = 0;
  long long m_tiles = 0;
  if (g.gm * g.gn >= (1LL << 31)) return false;
  switch (g.kind) {
    case GK_FC_FWD: {
      p.kdepth = pick_swizzle(g.gk);
      if (!p.kdepth) return false;
      p.bn = g.gn >= 256 ? 256 : round_up32(g.gn);
      a_sw = b_sw = p.kdepth;
      sa = {2, {(cuuint64_t)g.gk, (cuuint64_t)g.gm}, {(cuuint64_t)g.gk}, {(cuuint32_t)p.kdepth, BM}, a_sw, g.p0};
      sb = {2, {(cuuint64_t)g.gk, (cuuint64_t)g.gn}, {(cuuint64_t)g.gk}, {(cuuint32_t)p.kdepth, (cuuint32_t)(p.bn / ctas)}, b_sw, g.p1};
      p.kb_total = (int)((g.gk + p.kdepth - 1) / p.kdepth);
      m_tiles = (g.gm + BM - 1) / BM;
      p.n_tiles_n = (int)((g.gn + p.bn - 1) / p.bn);
      break;
    }
    case GK_FC_DGRAD: {   // out [M][K'], contraction over N
      p.kdepth = pick_swizzle(g.gk);
      if (!p.kdepth) return false;
      b_mn = 1;
      b_sw = pick_swizzle(g.gn);
      if (!b_sw) return false;
      p.bn = g.gn >= 256 ? 256 : (int)((g.gn + b_sw - 1) / b_sw * b_sw);
      if (p.bn % 32) return false;
      a_sw = p.kdepth;
      sa = {2, {(cuuint64_t)g.gk, (cuuint64_t)g.gm}, {(cuuint64_t)(g.ld0 ? g.ld0 : g.gk)}, {(cuuint32_t)p.kdepth, BM}, a_sw, g.p0};
      sb = {2, {(cuuint64_t)g.gn, (cuuint64_t)g.gk}, {(cuuint64_t)g.gn}, {(cuuint32_t)b_sw, (cuuint32_t)p.kdepth}, b_sw, g.p1};
      p.kb_total = (int)((g.gk + p.kdepth - 1) / p.kdepth);
      m_tiles = (g.gm + BM - 1) / BM;
      p.n_tiles_n = (int)((g.gn + p.bn - 1) / p.bn);
      break;
    }
    case GK_FC_WGRAD: {   // out [N][K'], contraction over M (rows of both operands)
      a_mn = b_mn = 1;
      a_sw = pick_swizzle(g.gm);
      b_sw = pick_swizzle(g.gn);
      if (!a_sw || !b_sw || g.gk < 32) return false;
      p.kdepth = g.gk >= 128 ? 128 : (g.gk >= 64 ? 64 : 32);
      p.bn = g.gn >= 256 ? 256 : (int)((g.gn + b_sw - 1) / b_sw * b_sw);
      if (p.bn % 32) return false;
      sa = {2, {(cuuint64_t)g.gm, (cuuint64_t)g.gk}, {(cuuint64_t)(g.ld0 ? g.ld0 : g.gm)}, {(cuuint32_t)a_sw, (cuuint32_t)p.kdepth}, a_sw, g.p0};
      sb = {2, {(cuuint64_t)g.gn, (cuuint64_t)g.gk}, {(cuuint64_t)g.gn}, {(cuuint32_t)b_sw, (cuuint32_t)p.kdepth}, b_sw, g.p1};
      p.kb_total = (int)((g.gk + p.kdepth - 1) / p.kdepth);
      m_tiles = (g.gm + BM - 1) / BM;
      p.n_tiles_n = (int)((g.gn + p.bn - 1) / p.bn);
      break;
    }
    case GK_CONV_FWD:
    case GK_CONV_DGRAD: {
      // Rows run over the pixels of the OUTPUT tensor of this multiply (forward: the Ho x Wo output;
      // error: the H x W input-shaped tensor); the shifted operand is the other activation tensor and
      // may have another size (padding other than (R-1)/2, strides): its copies start at any
      // coordinate and read zeros outside it.  A forward stride becomes the element stride of those
      // copies.  The error of a strided convolution is left to the CUDA-core engine.
      const bool fwd = g.kind == GK_CONV_FWD;
      const int st = g.stride > 1 ? g.stride : 1;
      if (!fwd && st != 1) return false;
      const int RW = fwd ? g.Wo : g.W, RH = fwd ? g.Ho : g.H;      // pixel grid of the rows
      const int OW = fwd ? g.W : g.Wo, OH = fwd ? g.H : g.Ho;      // pixel grid of the shifted operand
      const bool same = g.Ho == g.H && g.Wo == g.W && st == 1;
      const int Cc = fwd ? g.Ci : g.Co;        // contraction channels
      const int Cn = fwd ? g.Co : g.Ci;        // output channels of this multiply
      p.kdepth = pick_swizzle(Cc);
      if (!p.kdepth || Cc % p.kdepth) return false;
      if (!pick_pixel_box(RW, RH, g.B, p.Wt, p.Ht, p.Bt)) return false;
      if (p.Wt * st > 256 || p.Ht * st > 256) return false;
      p.w_tiles = (RW + p.Wt - 1) / p.Wt;
      p.h_tiles = (RH + p.Ht - 1) / p.Ht;
      p.b_tiles = (g.B + p.Bt - 1) / p.Bt;
      p.PW = RW; p.PH = RH; p.PB = g.B;
      p.R = g.R; p.S = g.S; p.pad = g.pad;
      p.stride = st;
      p.c_chunks = Cc / p.kdepth;
      p.Cn = Cn;
      a_sw = p.kdepth;
      sa = {4, {(cuuint64_t)Cc, (cuuint64_t)OW, (cuuint64_t)OH, (cuuint64_t)g.B},
            {(cuuint64_t)Cc, (cuuint64_t)Cc * OW, (cuuint64_t)Cc * OW * OH},
            {(cuuint32_t)p.kdepth, (cuuint32_t)(p.Wt * st), (cuuint32_t)(p.Ht * st), (cuuint32_t)p.Bt}, a_sw, g.p0,
            {1, (cuuint32_t)st, (cuuint32_t)st, 1}};
      if (fwd) {
        p.bn = Cn >= 256 ? 256 : round_up32(Cn);
        if (ctas == 2 && Cn > 256) {
          // Whole waves: with 256-wide tiles the 14 x 14 layers are 98 tile pairs on 74 pairs of SMs, two
          // waves of which the second is a third full; 192-wide tiles make 147 items, two full waves.
          // (A 192-wide MMA takes as long as a 256-wide one, so an item is not shorter; it moves three
          // quarters of the weights.  Measured 31.0 against 31.5 us; 128-wide tiles, three waves of
          // half the math each, are bound by the shared-memory traffic of their operands: 38.4 us.)
          const long long mu = ((long long)p.w_tiles * p.h_tiles * p.b_tiles + 1) / 2, units = ctx->sm_count / 2;
          const long long w256 = (mu * ((Cn + 255) / 256) + units - 1) / units;
          const long long w192 = (mu * ((Cn + 191) / 192) + units - 1) / units;
          if (w192 * 192 * 10 < w256 * 256 * 9) p.bn = 192;
        }
        b_sw = p.kdepth;
        sb = {2, {(cuuint64_t)g.gk, (cuuint64_t)Cn}, {(cuuint64_t)g.gk}, {(cuuint32_t)p.kdepth, (cuuint32_t)(p.bn / ctas)}, b_sw, g.p1};
      } else {
        b_mn = 1;
        b_sw = pick_swizzle(Cn);
        if (!b_sw || Cn % b_sw) return false;
        p.bn = Cn >= 256 ? 256 : Cn;
        if (p.bn % 32 || Cn % p.bn) return false;
        // w viewed as [Co rows][R*S*Ci]: column = tap * Ci + ci
        sb = {2, {(cuuint64_t)g.R * g.S * g.Ci, (cuuint64_t)g.Co}, {(cuuint64_t)g.R * g.S * g.Ci},
              {(cuuint32_t)b_sw, (cuuint32_t)p.kdepth}, b_sw, g.p1};
      }
      p.kb_total = g.R * g.S * p.c_chunks;
      m_tiles = (long long)p.w_tiles * p.h_tiles * p.b_tiles;
      p.n_tiles_n = (Cn + p.bn - 1) / p.bn;
      // halo mode: one channel chunk, one column tile, weights of all taps fit beside >= 3 patches
      if (want_halo && same && ctas == 1 && g.R == 3 && g.S == 3 && g.pad == 1 && p.c_chunks == 1 && p.n_tiles_n == 1 &&
          g.W >= 10 && g.H >= 18) {
        const int a_stage = (180 * p.kdepth + 1023) / 1024 * 1024;
        const int b_res = (9 * p.bn * p.kdepth + 1023) / 1024 * 1024;
        if (b_res + 3 * a_stage <= 224 * 1024) {
          p.halo = 1;
          p.Wt = 8; p.Ht = 16; p.Bt = 1;
          p.w_tiles = (g.W + 7) / 8;
          p.h_tiles = (g.H + 15) / 16;
          p.b_tiles = g.B;
          m_tiles = (long long)p.w_tiles * p.h_tiles * p.b_tiles;
          sa.box[1] = 10; sa.box[2] = 18; sa.box[3] = 1;
          if (fwd) sb.box[1] = (cuuint32_t)p.bn;
          p.b_tile_bytes = p.bn * p.kdepth;
          p.b_res_bytes = b_res;
        }
      }
      break;
    }
    case GK_CONV_WGRAD: {
      // the contraction runs over the pixels of the OUTPUT grid (Ho x Wo); the input tensor is copied
      // shifted by the tap, with the stride as element stride
      const int st = g.stride > 1 ? g.stride : 1;
      const bool same = g.Ho == g.H && g.Wo == g.W && st == 1;
      p.stride = st;
      // (64 x 64)-channel blocks re-read the activations once per block of the other operand, so this
      // mode is kept for layers with few blocks; wide layers use the per-tap tiles below
      if (want_halo && same && ctas == 1 && g.R == 3 && g.S == 3 && g.pad == 1 && g.Ci % 64 == 0 && g.Co % 64 == 0 &&
          g.W >= 10 && g.H >= 18 && (long long)g.Ci * g.Co <= 32768) {
        p.halo = 2;
        p.kdepth = 128;
        p.bn = 64;
        p.Wt = 8; p.Ht = 16; p.Bt = 1;
        p.w_tiles = (g.W + 7) / 8;
        p.h_tiles = (g.H + 15) / 16;
        p.b_tiles = g.B;
        p.PW = g.W; p.PH = g.H; p.PB = g.B;
        p.Cn = g.Ci;
        p.wg_nci = g.Ci / 64;
        p.kb_total = p.w_tiles * p.h_tiles * p.b_tiles;      // pixel tiles
        // A = input patch (p1 = x), B = error tile (p0 = e); both MN-major, 64-byte rows
        sa = {4, {(cuuint64_t)g.Ci, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.B},
              {(cuuint64_t)g.Ci, (cuuint64_t)g.Ci * g.W, (cuuint64_t)g.Ci * g.W * g.H}, {64, 10, 18, 1}, 64, g.p1};
        sb = {4, {(cuuint64_t)g.Co, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.B},
              {(cuuint64_t)g.Co, (cuuint64_t)g.Co * g.W, (cuuint64_t)g.Co * g.W * g.H}, {64, 8, 16, 1}, 64, g.p0};
        p.a_box_bytes = 180 * 64; p.b_box_bytes = 128 * 64;
        p.a_bytes = 12288; p.b_bytes = 8192;
        p.a_boxes = p.b_boxes = 1;
        p.stages = MAX_STAGES;
        p.nprod = 2;                                          // divides the eight stages
        p.nbuf = 5;                                           // five accumulators of 64 columns
        p.ksteps = 4;
        // MN-major, 64-byte swizzle: 8-row groups one patch row (10 pixels) apart for A, contiguous for B;
        // the leading-dimension field of A is filled per tap pair by the kernel
        p.a_desc = ((unsigned long long)((10 * 64) >> 4) << 32) | ((unsigned long long)1 << 46) | layout_bits(64);
        p.b_desc = ((unsigned long long)1 << 16) | ((unsigned long long)((8 * 64) >> 4) << 32) |
                   ((unsigned long long)1 << 46) | layout_bits(64);
        p.idesc = (2u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((unsigned)(64 >> 3) << 17) |
                  ((unsigned)(BM >> 4) << 24);
        const long long blocks = (long long)(g.Ci / 64) * (g.Co / 64);
        // split the pixel range so that the items fill whole waves of SMs
        int best_s = 1;
        double best_eff = 0;
        const int max_s = p.kb_total / 4 > 0 ? p.kb_total / 4 : 1;
        for (int sp = 1; sp <= max_s && sp <= 4 * ctx->sm_count; ++sp) {
          const long long it = blocks * sp;
          const long long waves = (it + ctx->sm_count - 1) / ctx->sm_count;
          const double eff = (double)it / (double)(waves * ctx->sm_count);
          if (eff > best_eff + 0.02) { best_eff = eff; best_s = sp; }
        }
        p.splits = best_s;
        // (a split covers at most NITI_SPLIT_MAX_K pixels: its partial sums cannot wrap)
        if (p.splits < (p.kb_total + NITI_SPLIT_MAX_K / 128 - 1) / (NITI_SPLIT_MAX_K / 128))
          p.splits = (p.kb_total + NITI_SPLIT_MAX_K / 128 - 1) / (NITI_SPLIT_MAX_K / 128);
        if (p.splits > NITI_MAX_SPLITS) return false;
        p.kb_per_split = (p.kb_total + p.splits - 1) / p.splits;
        p.splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
        p.items = blocks * p.splits;
        p.m_units = 1;
        p.n_tiles_n = 1;
        if (!encode(ctx, &ma, sa) || !encode(ctx, &mb, sb)) return false;
        return true;
      }
      a_mn = b_mn = 1;
      a_sw = pick_swizzle(g.Co);
      b_sw = pick_swizzle(g.Ci);
      if (!a_sw || !b_sw || g.Co % a_sw || g.Ci % b_sw) return false;
      if (!pick_pixel_box(g.Wo, g.Ho, g.B, p.Wt, p.Ht, p.Bt)) return false;
      if (p.Wt * st > 256 || p.Ht * st > 256) return false;
      p.kdepth = 128;
      p.w_tiles = (g.Wo + p.Wt - 1) / p.Wt;
      p.h_tiles = (g.Ho + p.Ht - 1) / p.Ht;
      p.b_tiles = (g.B + p.Bt - 1) / p.Bt;
      p.PW = g.Wo; p.PH = g.Ho; p.PB = g.B;
      p.R = g.R; p.S = g.S; p.pad = g.pad;
      p.Cn = g.Ci;
      p.bn = g.Ci >= 256 ? 256 : g.Ci;
      if (p.bn % 32 || g.Ci % p.bn) return false;
      p.n_chunks = g.Ci / p.bn;
      sa = {4, {(cuuint64_t)g.Co, (cuuint64_t)g.Wo, (cuuint64_t)g.Ho, (cuuint64_t)g.B},
            {(cuuint64_t)g.Co, (cuuint64_t)g.Co * g.Wo, (cuuint64_t)g.Co * g.Wo * g.Ho},
            {(cuuint32_t)a_sw, (cuuint32_t)p.Wt, (cuuint32_t)p.Ht, (cuuint32_t)p.Bt}, a_sw, g.p0};
      sb = {4, {(cuuint64_t)g.Ci, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.B},
            {(cuuint64_t)g.Ci, (cuuint64_t)g.Ci * g.W, (cuuint64_t)g.Ci * g.W * g.H},
            {(cuuint32_t)b_sw, (cuuint32_t)(p.Wt * st), (cuuint32_t)(p.Ht * st), (cuuint32_t)p.Bt}, b_sw, g.p1,
            {1, (cuuint32_t)st, (cuuint32_t)st, 1}};
      p.kb_total = p.w_tiles * p.h_tiles * p.b_tiles;
      m_tiles = (g.Co + BM - 1) / BM;
      p.n_tiles_n = g.R * g.S * p.n_chunks;
      break;
    }
    default:
      return false;
  }
  p.ksteps = p.kdepth / 32;
  // operand staging
  if (a_mn) {
    p.a_boxes = BM / a_sw;
    if ((long long)p.a_boxes * a_sw > (g.gm + a_sw - 1) / a_sw * a_sw) p.a_boxes = (int)((g.gm + a_sw - 1) / a_sw);
    p.a_box_bytes = p.kdepth * a_sw;
    p.a_box_step = a_sw;
    p.a_bytes = (BM / a_sw) * p.a_box_bytes;
    p.a_desc = desc_mnmajor(a_sw, p.kdepth);
    p.a_kstep16 = (unsigned)((32 * a_sw) >> 4);
  } else {
    p.a_boxes = 1;
    p.a_box_bytes = BM * p.kdepth;
    p.a_bytes = p.a_box_bytes;
    p.a_desc = desc_kmajor(a_sw);
    p.a_kstep16 = 2;
  }
  // Row-batched mode: a multiply with one or two k-blocks and a narrow output (the gathered first
  // layer: K = 32, N = 64) is all per-tile bookkeeping.  One item then covers mrep 128-row tiles: one
  // stage holds their A boxes, one MMA per tile writes its own bn_mma columns of the accumulator,
  // and the barriers, commits and tile decoding are paid once per item.
  p.mrep = 1;
  if (g.kind == GK_FC_FWD && ctas == 1 && ctx->engine != 4 && p.n_tiles_n == 1 && p.kb_total <= 2 && p.bn <= 128 &&
      m_tiles >= 8LL * ctx->sm_count) {
    p.mrep = p.bn <= 64 ? 4 : 2;
    p.a_boxes = p.mrep;
    p.a_bytes = p.mrep * p.a_box_bytes;
    m_tiles = (m_tiles + p.mrep - 1) / p.mrep;
  }
  const int bn_cta = p.bn / ctas;               // output columns staged by each CTA
  if (bn_cta % 16) return false;
  if (b_mn) {
    if (bn_cta % b_sw) return false;
    p.b_boxes = bn_cta / b_sw;
    p.b_box_bytes = p.kdepth * b_sw;
    p.b_box_step = b_sw;
    p.b_bytes = p.b_boxes * p.b_box_bytes;
    p.b_desc = desc_mnmajor(b_sw, p.kdepth);
    p.b_kstep16 = (unsigned)((32 * b_sw) >> 4);
  } else {
    p.b_boxes = 1;
    p.b_box_bytes = bn_cta * p.kdepth;
    p.b_bytes = p.b_box_bytes;
    p.b_desc = desc_kmajor(b_sw);
    p.b_kstep16 = 2;
  }
  // stage buffers must start on the swizzle period (1024 bytes)
  p.a_bytes = (p.a_bytes + 1023) / 1024 * 1024;
  p.b_bytes = (p.b_bytes + 1023) / 1024 * 1024;
  int stage_bytes = p.a_bytes + p.b_bytes;
  p.stages = (200 * 1024) / stage_bytes;
  if (p.halo) {
    // a stage is one 10 x 18 pixel patch; consecutive 8-row groups of a tap are one patch row apart
    p.a_box_bytes = 180 * p.kdepth;
    p.a_bytes = (p.a_box_bytes + 1023) / 1024 * 1024;
    p.a_desc = desc_kmajor(a_sw, 10);
    p.b_bytes = 0;
    stage_bytes = p.a_bytes;
    p.stages = (224 * 1024 - p.b_res_bytes) / stage_bytes;
  }
  if (p.stages > MAX_STAGES) p.stages = MAX_STAGES;
  if (p.stages < 2) return false;
  // instruction descriptor: s32 accumulate, signed 8-bit operands, majorness, N, M
  p.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((unsigned)a_mn << 15) | ((unsigned)b_mn << 16) |
            ((unsigned)(p.bn >> 3) << 17) | ((unsigned)((BM * ctas) >> 4) << 24);
  p.bn_mma = p.bn;
  p.bn *= p.mrep;
  p.m_units = (int)((m_tiles + ctas - 1) / ctas);
  long long tiles = (long long)p.m_units * p.n_tiles_n;
  const int units = ctx->sm_count / ctas;       // CTAs (or CTA pairs) that run at the same time
  // visit row units in groups so that concurrently running tiles share operands in L2
  if ((g.kind == GK_FC_FWD || g.kind == GK_FC_DGRAD || g.kind == GK_FC_WGRAD) && p.n_tiles_n > 1 && p.m_units > 1)
    p.raster_g = ctas == 2 ? 8 : 12;
  // split the contraction when the tiles alone cannot fill the SMs
  if (tiles < units && p.kb_total >= 8) {
    // pick the split count with the least modelled time: waves of items, each item running its
    // share of the k-blocks plus a fixed cost (pipeline fill and the atomic epilogue) of about
    // four k-blocks
    double best = 1e30;
    int best_s = 1;
    int max_s = p.kb_total / 4;
    // (multiplies with few output rows keep their splits' partial tiles in separate slices of the scratch)
    const int slices = niti_partial_slices(g.kind, g.gm);
    if (slices > 1 && max_s > slices) max_s = slices;
    for (int sp = 1; sp <= max_s && sp <= 4 * units; ++sp) {
      const long long it = tiles * sp;
      const long long waves = (it + units - 1) / units;
      const double cost = (double)waves * ((double)((p.kb_total + sp - 1) / sp) + 4.0);
      if (cost < best * 0.98) { best = cost; best_s = sp; }
    }
    p.splits = best_s;
  }
  {
    // a contraction longer than NITI_SPLIT_MAX_K is always split, into pieces whose partial sums cannot
    // wrap an int32; the epilogue records the largest partial sum of every piece (overflow detection)
    const int max_kb = NITI_SPLIT_MAX_K / p.kdepth;
    const int min_splits = (p.kb_total + max_kb - 1) / max_kb;
    if (p.splits < min_splits) p.splits = min_splits;
    if (p.splits > NITI_MAX_SPLITS) return false;
  }
  p.kb_per_split = (p.kb_total + p.splits - 1) / p.splits;
  p.splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
  // split contractions add their partial sums atomically: room for the epilogue warps' transpose
  // buffers (consecutive output rows only: every multiply but the pixel-box convolutions)
  p.stg_off = 0;
  if (p.splits > 1 && !p.halo && g.kind != GK_CONV_FWD && g.kind != GK_CONV_DGRAD) {
    const int stg_bytes = EPI_WARPS * 32 * 33 * 4;
    int st = (200 * 1024 - stg_bytes) / stage_bytes;
    if (st > MAX_STAGES) st = MAX_STAGES;
    if (st >= 2) {
      p.stages = st;
      p.stg_off = st * stage_bytes;
    }
  }
  if (p.halo) {
    p.splits = 1;
    p.kb_per_split = p.kb_total;
  }
  // producer warps: the largest count <= PROD_WARPS that divides the number of stages
  if (p.stages == 5 || p.stages == 7) p.stages -= 1;
  p.nissue = p.halo == 1 ? 2 : 1;
  p.nprod = 1;
  for (int d = 2; d <= PROD_WARPS - (p.nissue - 1); ++d)
    if (p.stages % d == 0) p.nprod = d;
  p.nbuf = 512 / p.bn;
  if (p.nbuf > MAX_TBUF) p.nbuf = MAX_TBUF;
  // epilogue groups: as many as leave no warp without a chunk and one spare accumulator buffer
  p.egroups = 1;
  for (int gq = 2; gq <= 4; gq *= 2)
    if (EPI_PER_Q / gq <= p.bn / 32 && p.nbuf >= gq + 1) p.egroups = gq;
  p.nbuf = p.nbuf / p.egroups * p.egroups;     // a buffer always returns to the same group
  p.one_commit = 0;
  if (p.halo == 1 && p.stages >= p.nbuf) {
    p.one_commit = 1;
    p.stages = p.nbuf;
    p.nprod = 1;
    for (int d = 2; d <= PROD_WARPS - (p.nissue - 1); ++d)
      if (p.stages % d == 0) p.nprod = d;
  }
  // convolution outputs are spatially structured (borders, images): contiguous item ranges make the
  // first tile of every CTA an even sample of the tensor for the speculative shift
  p.blocked = (g.kind == GK_CONV_FWD || g.kind == GK_CONV_DGRAD) ? 1 : 0;
  p.items = tiles * p.splits;
  if (p.items >= (1LL << 30)) return false;      // the kernel counts items in 32 bits
  if (!encode(ctx, &ma, sa) || !encode(ctx, &mb, sb)) return false;
  return true;
}

}  // namespace

size_t niti_tc_scratch_bytes(const GemmProblem &) { return 0; }

int niti_tc_timeout_probe(niti_ctx *ctx, cudaStream_t st) {
  timeout_probe_kernel<<<1, 32, 0, st>>>(ctx->d_status);
  ctx->launches++;
  NITI_CUDA_TRY(ctx, cudaGetLastError());
  return NITI_OK;
}

// CTAs (CTAS = 1) or CTA pairs (CTAS = 2) that can be resident at the same time.  SMs pair up inside a
// GPC, so the number of pairs can be below sm_count / 2; a persistent grid larger than that would run
// a second, short wave.
// Dynamic shared-memory limit of the kernel: once per context, and always the most the device allows
// beside the kernel's static shared memory (see niti_ctx::smem_optin for why not "what this launch needs").
template <int CTAS>
static int tc_set_smem_limit(niti_ctx *ctx) {
  cudaFuncAttributes fa;
  NITI_CUDA_TRY(ctx, cudaFuncGetAttributes(&fa, tc_gemm_kernel<CTAS>));
  const size_t limit = ctx->smem_optin > fa.sharedSizeBytes ? ctx->smem_optin - fa.sharedSizeBytes : 0;
  NITI_CUDA_TRY(ctx, cudaFuncSetAttribute(tc_gemm_kernel<CTAS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)limit));
  ctx->tc_attr_smem[CTAS] = limit;
  return NITI_OK;
}

template <int CTAS>
static int tc_units(niti_ctx *ctx) {
  int &cached = ctx->tc_units[CTAS];
  if (cached) return cached;
  cached = ctx->sm_count / CTAS;
  if (CTAS == 2) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(ctx->sm_count / 2 * 2), 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = 200 * 1024;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    (void)tc_set_smem_limit<2>(ctx);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tc_gemm_kernel<2>, &cfg) == cudaSuccess && n > 0 && n < cached) cached = n;
    else (void)cudaGetLastError();
  }
  return cached;
}

template <int CTAS>
static int launch_tc(niti_ctx *ctx, cudaStream_t st, const TcParams &p, const CUtensorMap &ma, const CUtensorMap &mb,
                     int32_t *acc, WsHeader *hdr, const RoundSpec &r) {
  size_t smem = (size_t)p.stages * (p.a_bytes + p.b_bytes) + (size_t)p.b_res_bytes + 1024;
  if (p.stg_off > 0) smem = (size_t)p.stg_off + (size_t)EPI_WARPS * 32 * 33 * 4 + 1024;
  size_t &attr_smem = ctx->tc_attr_smem[CTAS];
  if (!attr_smem) {
    const int rcs = tc_set_smem_limit<CTAS>(ctx);
    if (rcs != NITI_OK) return rcs;
  }
  if (smem > attr_smem) return niti_fail(ctx, NITI_ERR_SHAPE, "tensor-core kernel: stage buffers exceed the shared memory of an SM");
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)(ctx->sm_count / CTAS * CTAS), 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.epi_mode == EPI_KNOWN_B) {
    // programmatic dependent launch: the launch latency of the follow-up overlaps the first pass
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
  const int units = tc_units<CTAS>(ctx);
  long long grid = (p.items < units ? p.items : units) * CTAS;
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  TcParams q = p;
  {
    const int gunits = (int)(grid / CTAS);
    q.blk_per = (int)(p.items / gunits);
    q.blk_extra = (int)(p.items % gunits);
    const int eg = p.halo == 2 ? 1 : p.egroups;
    q.k_wpq = EPI_PER_Q / eg;
    const int chunks_all = p.bn / 32;
    q.k_wpq_active = p.halo == 2 ? EPI_PER_Q : (chunks_all < q.k_wpq ? chunks_all : q.k_wpq);
    q.k_epi_active = 4 * q.k_wpq_active;
    int cols = 32;
    while (cols < p.nbuf * p.bn) cols <<= 1;
    q.k_tmem_cols = cols;
    // reciprocals for tile index -> coordinates; dividends stay below the tile count
    const unsigned long long n_max = (unsigned long long)(p.w_tiles > 0 ? p.w_tiles : 1) * (p.h_tiles > 0 ? p.h_tiles : 1) *
                                     (p.b_tiles > 0 ? p.b_tiles : 1) + 2;
    q.magic_w = (p.w_tiles > 1 && n_max * p.w_tiles < (1ull << 32)) ? (unsigned)((1ull << 32) / p.w_tiles + 1) : 0u;
    q.magic_h = (p.h_tiles > 1 && n_max * p.h_tiles < (1ull << 32)) ? (unsigned)((1ull << 32) / p.h_tiles + 1) : 0u;
  }
  // per call site (keyed by the address of its bit-width scalar): the error of the last speculative estimate
  int32_t *slot = nullptr;
  if (r.b_out && ctx->d_spec_tab) {
    const uintptr_t key = (uintptr_t)r.b_out >> 2;
    slot = ctx->d_spec_tab + 2 * (size_t)((key ^ (key >> 13)) % NITI_SPEC_SLOTS);
    q.spec_tag = (int)(unsigned)(key | 1u);
  }
  NITI_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, tc_gemm_kernel<CTAS>, ma, mb, q, acc, hdr, ctx->d_status, r.out, r.mask,
                                        r.s_a, r.s_w, r.s_out, r.b_out, slot, r.pool_out));
  ctx->launches++;
  ctx->tc_launches++;
  if (CTAS == 2) ctx->tc2_launches++;
  return NITI_OK;
}

// Profiling event of a launch.  On a stream that is being captured the record becomes an event-record
// node of the graph (cudaEventRecordExternal), so that every replay of the graph times its launches
// where they run; a plain record there would only add a dependency.
static void prof_record(cudaEvent_t ev, cudaStream_t st) {
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusActive)
    cudaEventRecordWithFlags(ev, st, cudaEventRecordExternal);
  else
    cudaEventRecord(ev, st);
}

int niti_tc_gemm(niti_ctx *ctx, cudaStream_t st, const GemmProblem &g, const RoundSpec &r_in, int32_t *acc,
                 WsHeader *hdr, bool *fused, bool *pooled, bool shard_ok, bool *updated) {
  TcParams p;
  CUtensorMap ma, mb;
  RoundSpec r = r_in;
  *fused = false;
  if (pooled) *pooled = false;
  if (updated) *updated = false;
  // engine 0: pairs of CTAs (cta_group::2) when there are enough 256-row tiles to fill the GPU.
  // Test switches: 2 / 3 force the single-CTA / paired kernel, 4 keeps the int32 spill epilogue.
  // Test switches: 5 disables the halo mode of small-channel convolutions.
  bool planned = false;
  if ((g.kind == GK_CONV_FWD || g.kind == GK_CONV_DGRAD || g.kind == GK_CONV_WGRAD) && ctx->engine != 3 &&
      ctx->engine != 5)
    planned = plan(ctx, g, 1, true, p, ma, mb) && p.halo;
  if (!planned && g.kind == GK_FC_FWD && ctx->engine != 3)      // row-batched mode of short contractions
    planned = plan(ctx, g, 1, false, p, ma, mb) && p.mrep > 1;
  if (!planned && ctx->engine != 2 && g.gm >= 2 * BM) {
    planned = plan(ctx, g, 2, false, p, ma, mb);
    // (pairs halve the operand traffic per MMA; they are kept unless they would leave more than a
    // third of the GPU idle)
    if (planned && ctx->engine != 3 && p.items * 3 < (long long)(ctx->sm_count / 2) * 2) planned = false;
  }
  if (!planned) {
    if (ctx->engine == 3) return NITI_ERR_SHAPE;
    if (!plan(ctx, g, 1, false, p, ma, mb)) return NITI_ERR_SHAPE;
  }
  {
    // expected ratio between the max of the whole tensor (N values) and the max of the first tile of
    // every CTA (n values) for roughly Gaussian sums: sqrt(ln N / ln n)
    const int units = p.ctas == 2 ? tc_units<2>(ctx) : tc_units<1>(ctx);
    const double n_all = (double)g.gm * (double)g.gn;
    const double frac = p.items > units ? (double)units / (double)p.items : 1.0;
    // (when the tensor has more tiles than the grid, the bit-width is fixed once half of the CTAs have
    // reported; typically a few more have by then)
    const double n_s = n_all * frac * (frac < 1.0 ? 0.6 : 1.0);
    double f = (n_s > 16.0 && frac < 1.0) ? sqrt(log(n_all) / log(n_s)) : 1.0;
    p.spec_mul256 = (unsigned)(f * 256.0 + 0.5);
  }
  // data parallelism (niti_set_reduce_hook): the max magnitude is combined over the ranks between the
  // two launches, so there is always a second launch; weight gradients keep their int32 sums
  const bool dp = ctx->reduce_fn != nullptr, dp_sum = dp && niti_is_wgrad(g.kind);
  p.single_wave = (!dp && p.items <= (p.ctas == 2 ? tc_units<2>(ctx) : tc_units<1>(ctx)) && p.spec_mul256 == 256) ? 1 : 0;
  {
    const long long units = p.ctas == 2 ? tc_units<2>(ctx) : tc_units<1>(ctx);
    const long long grid = (p.items < units ? p.items : units) * p.ctas;
    p.quorum = (int)(p.single_wave ? grid : (grid + 1) / 2);
  }
  p.mbits = r.mbits;
  p.round_mode = r.round_mode;
  p.relu = r.relu;
  p.epi_mode = (p.splits > 1 || p.halo == 2) ? EPI_ATOMIC : ((ctx->engine == 4 || dp_sum) ? EPI_SPILL : EPI_SPECULATE);
  if (p.epi_mode == EPI_ATOMIC && niti_partial_slices(g.kind, g.gm) > 1 && p.splits <= niti_partial_slices(g.kind, g.gm) &&
      !p.halo && p.mrep == 1)
    p.epi_mode = EPI_PARTIAL;
  if (p.epi_mode == EPI_ATOMIC) {
    NITI_CUDA_TRY(ctx, cudaMemsetAsync(acc, 0, sizeof(int32_t) * (size_t)(g.gm * g.gn), st));
    ctx->launches++;
  }
  // Fused 2 x 2 max-pool: the fused epilogue of a forward convolution with ReLU also stores the pooled
  // tile when every pooling window lies inside one warp's 32 pixels (8 x 16 pixel tiles of the
  // resident-weights mode, or pixel boxes at most 16 wide and at least 2 high) and the rows are whole,
  // 32-byte aligned chunks.  Otherwise the caller runs the pooling kernel.
  p.pool = 0;
  if (pooled && r.pool_out && g.kind == GK_CONV_FWD && r.relu && !r.mask && p.epi_mode == EPI_SPECULATE &&
      p.mrep == 1 && (p.PW % 2) == 0 && (p.PH % 2) == 0 && (g.gn % 32) == 0 && ((uintptr_t)r.out & 31) == 0 &&
      ((uintptr_t)r.pool_out & 31) == 0 && r.mbits == 7) {
    if (p.halo == 1) { p.pool = 1; p.pool_xh = 8; }
    else if (!p.halo && p.Wt >= 2 && p.Wt <= 16 && p.Ht >= 2) { p.pool = 1; p.pool_xh = p.Wt; }
    *pooled = p.pool != 0;
  }
  // Weight update inside the epilogue (Section 3.3): a fully connected weight gradient whose epilogue
  // rounds by itself subtracts the rounded values from the weights in place of storing them.  A
  // speculative pass must not touch the weights (a wrong guess could not be taken back), so the update
  // is fused only where the shift is exact when the stores happen: single-wave launches.  (Measured
  // and not kept for the other launches: a first pass for the bit-width alone followed by a rounding
  // pass that updates, 198 us against 185 us for the 4096 x 25088 layer at batch 64.)
  p.update = 0;
  if (updated && r.update_w && g.kind == GK_FC_WGRAD && p.epi_mode == EPI_SPECULATE && p.single_wave && p.mrep == 1 &&
      !p.halo && !r.mask && !r.relu && (g.gn % 32) == 0 && ((uintptr_t)r.update_w & 31) == 0) {
    p.update = 1;
    r.out = r.update_w;
    *updated = true;
  }
  const bool prof = ctx->profile_on && ctx->prof_ev && ctx->prof_used < NITI_PROF_MAX;
  if (prof) prof_record(ctx->prof_ev[2 * ctx->prof_used], st);
  int rc = p.ctas == 2 ? launch_tc<2>(ctx, st, p, ma, mb, acc, hdr, r) : launch_tc<1>(ctx, st, p, ma, mb, acc, hdr, r);
  if (rc != NITI_OK) return rc;
  if (p.epi_mode == EPI_SPECULATE && p.single_wave) {
    *fused = true;                     // exact shift, scalars published by the last CTA: no second launch
  } else if (p.epi_mode == EPI_SPECULATE) {
    // publishes b and the exponent; recomputes with the true bit-width only if the guess was low
    if (dp) {
      rc = niti_reduce(ctx, st, &hdr->maxabs32, 1, NITI_REDUCE_MAX_U32);
      if (rc != NITI_OK) return rc;
    }
    p.epi_mode = EPI_KNOWN_B;
    rc = p.ctas == 2 ? launch_tc<2>(ctx, st, p, ma, mb, acc, hdr, r) : launch_tc<1>(ctx, st, p, ma, mb, acc, hdr, r);
    if (rc != NITI_OK) return rc;
    *fused = true;
  }
  if (prof) {
    prof_record(ctx->prof_ev[2 * ctx->prof_used + 1], st);
    ctx->prof_ops[ctx->prof_used] = 2.0 * (double)g.gm * (double)g.gn * (double)g.gk;
    ctx->prof_used++;
  }
  if (p.epi_mode == EPI_PARTIAL) {     // adds the splits' slices into the first one and takes the max magnitude
    rc = niti_launch_sum_partials(ctx, st, acc, p.splits, g.gm * g.gn, hdr);
    if (rc != NITI_OK || !dp) return rc;
    return niti_reduce(ctx, st, &hdr->maxabs32, 1, NITI_REDUCE_MAX_U32);
  }
  if (p.epi_mode == EPI_ATOMIC) {
    // (weight gradients under data parallelism: the sums over the ranks first, then their max)
    if (dp_sum) return niti_reduce_after_gemm(ctx, st, g.kind, acc, g.gm * g.gn, hdr, shard_ok);
    rc = niti_launch_maxabs(ctx, st, acc, g.gm * g.gn, hdr, p.splits);
    if (rc != NITI_OK || !dp) return rc;
    return niti_reduce(ctx, st, &hdr->maxabs32, 1, NITI_REDUCE_MAX_U32);
  }
  if (p.epi_mode == EPI_SPILL && dp) return niti_reduce_after_gemm(ctx, st, g.kind, acc, g.gm * g.gn, hdr, shard_ok);
  return NITI_OK;
}
