// Channel-gated convolution on tcgen05 tensor cores: one persistent fused kernel per layer.
//
// "Shifted-window" implicit GEMM (stride-1, k = 2*pad+1 convolutions).  A job is a tile of up
// to 128 output pixels that are whole image rows (or whole small images) times NT output
// channels.  The input patch of the tile -- the rows it needs plus the zero padding, which TMA
// out-of-bounds fill provides -- is loaded once per 64-channel chunk into shared memory as
// [pixel][64 channels] rows of 128 bytes (128-byte swizzle).  Rows are laid out with pitch
// W+pad, so that the right padding of one image row is the left padding of the next; then the
// A operand of filter tap (r,s) is the same buffer read from row r*(W+pad)+s onwards: output
// pixel i reads patch pixel i + r*(W+pad) + s.  All k*k taps reuse one patch load.
//
// Per job, following the paper's block (Section 3.1, Eq. 1-3, Section 4):
//   1. base path   P = W_p * x_p : MMAs over the base channels, fp32 accumulator in TMEM;
//   2. gate        d = (P >= t[c]) read from TMEM by the epilogue warps -> mask words, counts;
//   3. conditional R = W_r * x_r into a second TMEM accumulator, only for the 64-channel column
//                  blocks in which a gate fired; its patch chunks and weight tiles are not even
//                  loaded for tiles where none fired;
//   4. combine     y = f(BN1(P)) where d = 0, f(BN2(P+R)) where d = 1, staged in shared memory
//                  and written by one TMA store per 64 channels.
//
// The CTA is persistent (one per SM) and software-pipelined over its jobs:
//   MMA issue order      base(0) | base(1) cond(0) | base(2) cond(1) | ...
//   gate group           gate(0) | gate(1) | gate(2) | ...
//   combine group        combine(0) | combine(1) | ...          (each as soon as its inputs exist)
// so the tensor pipe works on the next tile's base path while the gate of the current tile is
// being evaluated.  TMEM (512 columns) holds a ring of P accumulators and a ring of R
// accumulators: 4 + 4 at NT = 64, 3 + 1 at NT = 128, so the issuer can run ahead of the epilogue.
// Weights stay resident in shared memory when they fit, otherwise they stream through a ring of
// stages of three tiles (the taps of a filter row).
//
// Warp roles: 0 = patch (A) producer, 1 = MMA issuer (owns TMEM), 2 = weight (B) producer,
// 3 = second MMA issuer (conditional path, resident weights), 4-7 = gate group, 8-23 = combine
// group; on single-chunk layers warp 2 becomes a third MMA issuer once it has loaded the
// resident weights.  The producer and issuer warps run convergently and lane 0 issues the
// copies and MMAs.  Every mbarrier wait is bounded; on expiry the CTA records
// CG_ERR_DEVICE_TIMEOUT with the id of the wait and leaves.
#include <cstring>
#include <type_traits>

#include "ptx.cuh"
#include "tc_conv.cuh"
#include "tc2_conv.cuh"

namespace cg {

namespace {

constexpr int kThreads = 768;       // 4 producer/issuer warps + 4 gate warps + 16 combine warps
constexpr int kIssuer3Warp = 2;     // third MMA issuer (single-chunk layers): the weight producer's warp, which has
                                    // nothing to do once resident weights are loaded
constexpr int kEpiWarp0 = 4;        // warps 0-3: patch producer, MMA issuer, weight producer, second MMA issuer
constexpr int kEpiThread0 = kEpiWarp0 * 32;
constexpr int kGateWarps = 4;       // gate group: one warp per TMEM lane quadrant, all columns
constexpr int kCombWarps = 16;      // combine group: quadrant x quarter of the columns
constexpr int kEpiWarps = kGateWarps + kCombWarps;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kCombThreads = kCombWarps * 32;
constexpr int kBM = 128;            // MMA M: patch rows per job
constexpr int kSpinLimit = 1 << 21; // try_wait polls before a wait gives up ...
constexpr long long kWaitCycles = 2000000000ll;   // ... or about one second of SM clocks, whichever is first
constexpr int kMaxWTiles = 192;     // weight tiles per job, both phases
constexpr int kStageTiles = 3;      // weight tiles per ring stage (the taps of a 3x3 filter row)

struct TcParams {
  LayerDims L;
  TcPlan P;
  cg_bn_params bn;
  const float* delta;
  const __nv_bfloat16* residual;   // optional, same layout as y (bf16 layers)
  uint32_t* mask;
  unsigned long long* counters;
  // Channel-wise gate (Eq. 4): thresholds per (image, channel), +inf where the channel is switched
  // off for the image (NULL: the layer's own thresholds); base_only: no conditional path (the
  // counting pass)
  const float* t_img;
  int base_only;
  // CG_COND_COMPACT: per column tile, the pixel rows in which a gate fired, with their partial
  // sums and mask words, for the second (gathered) kernel
  uint32_t* ws_counts;     // [tiles_n] rows listed so far
  uint32_t* ws_list;       // [tiles_n][M] pixel-row indices
  uint32_t* ws_rows;       // [tiles_n][M] records of NT partial sums (fp32) + NT/32 mask words,
                           // NT + 4 words apart
};

// One weight tile: 64 K-elements of NT output channels.
struct WTile {
  int x;        // K coordinate in the weight matrix
  int chunk;    // input-channel chunk (64 channels) it multiplies
};

// Weight tiles in the order the MMA issuer consumes them.  Base path: chunk-major, one tile
// per tap when c_p >= 64; when c_p < 64 a tile covers 64/c_p taps of chunk 0.  Conditional
// path: chunk-major, one tile per tap; when c_p < 64 chunk 0 comes first with the K slices
// behind the base channels.
// (ck = channels per 128-byte patch row: 64 for bf16, 128 for int8.)
__device__ __forceinline__ WTile base_tile(const LayerDims& L, int ck, int bt) {
  const int taps = L.kh * L.kw;
  if (L.c_p >= ck) {
    const int q = bt / taps, t = bt - q * taps;
    return {t * L.c_p + ck * q, q};
  }
  return {bt * ck, 0};
}

__device__ __forceinline__ WTile cond_tile(const LayerDims& L, int ck, int bt, int pad8) {
  const int taps = L.kh * L.kw;
  if (pad8 == 2) return {bt * ck, 0};   // int8, 64 input channels: a tile covers two taps of the only chunk
  if (pad8) {                       // repacked weights: every chunk whole, chunk 0 included
    const int q = bt / taps, t = bt % taps;
    return {t * L.c_r + ck * q, q};
  }
  if (L.c_p >= ck) {
    const int q = L.c_p / ck + bt / taps, t = bt % taps;
    return {t * L.c_r + ck * q - L.c_p, q};
  }
  if (bt < taps) return {bt * L.c_r, 0};
  const int b2 = bt - taps;
  const int q = 1 + b2 / taps, t = b2 % taps;
  return {t * L.c_r + ck * q - L.c_p, q};
}

struct Shared {
  uint64_t a_full[8], a_empty[8];
  uint64_t b_full[8], b_empty[8];
  uint64_t w_ready;
  uint64_t setup_done;       // the epilogue warps have zeroed the patch tails
  uint64_t base_done[4], gate_done[4], p_free[4];   // per P accumulator slot
  uint64_t cond_done[4], r_free[4];                 // per R accumulator slot
  uint32_t tmem_base;
  uint32_t abort_flag;
  uint32_t warp_blk[4][kGateWarps];   // per job slot, per epilogue warp: column blocks with a firing gate
  int row_idx[128];          // compact mode: list slot of each pixel row of the job being combined
};

struct Ctx {
  Shared* sh;
  unsigned long long* counters;
};

#ifdef CG_PROF
// Profiling build only: cycles that each warp of CTA 0 spent inside every bounded wait
// ([warp][site]), and the cycles of its role loops ([warp][31]).
__device__ unsigned long long g_prof[25 * 32];
__device__ unsigned long long g_tl[16 * 16];   // [job][event] clock stamps of CTA 0
#define CG_PROF_EV(j, ev) \
  do { if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && (j) < 16) g_tl[(j) * 16 + (ev)] = (unsigned long long)clock64(); } while (0)
#define CG_PROF_T(var) const long long var = clock64()
#define CG_PROF_ADD(slot, t0, t1) \
  do { if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) atomicAdd(&g_prof[(threadIdx.x >> 5) * 32 + (slot)], (unsigned long long)((t1) - (t0))); } while (0)
#else
#define CG_PROF_EV(j, ev)
#define CG_PROF_T(var)
#define CG_PROF_ADD(slot, t0, t1)
#endif

// Bounded wait.  The first poll is inline; the loop lives in one out-of-line copy so that the
// role loops stay small.  Each poll parks the thread in hardware for a short time; the wait
// gives up after about a second; a CTA that already gave up elsewhere is noticed within a few polls.
__device__ __noinline__ bool wait_bar_slow(Shared* sh, unsigned long long* counters, uint64_t* bar,
                                           uint32_t parity, int site) {
  const long long t0 = clock64();
  for (int i = 0; i < kSpinLimit; ++i) {
    if (ptx::mbar_try_wait(bar, parity)) {
#ifdef CG_PROF
      if (blockIdx.x == 0 && (threadIdx.x & 31) == 0)
        atomicAdd(&g_prof[(threadIdx.x >> 5) * 32 + site], (unsigned long long)(clock64() - t0));
#endif
      return true;
    }
    if ((i & 15) == 15) {
      if (*(volatile uint32_t*)&sh->abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) break;
    }
  }
  if (atomicCAS(&counters[CNT_STATUS], 0ull, (unsigned long long)CG_ERR_DEVICE_TIMEOUT) == 0ull)
    atomicExch(&counters[CNT_SITE], (unsigned long long)site);
  atomicExch(&sh->abort_flag, 1u);
  return false;
}

__device__ __forceinline__ bool wait_bar(const Ctx& cx, uint64_t* bar, uint32_t parity, int site) {
#ifdef CG_PROF
  const long long t0 = clock64();
  const bool fast = ptx::mbar_try_wait(bar, parity, 0u);
  if (blockIdx.x == 0 && (threadIdx.x & 31) == 0)
    atomicAdd(&g_prof[(threadIdx.x >> 5) * 32 + 26 + (fast ? 0 : 1)], (unsigned long long)(clock64() - t0));
  if (fast) return true;
#else
  if (ptx::mbar_try_wait(bar, parity, 0u)) return true;
#endif
  return wait_bar_slow(cx.sh, cx.counters, bar, parity, site);
}

// The same wait taken by every lane of a convergent warp; the outcome is made warp-uniform.
__device__ __forceinline__ bool wait_bar_warp(const Ctx& cx, uint64_t* bar, uint32_t parity, int site) {
  return __all_sync(0xffffffffu, wait_bar(cx, bar, parity, site));
}

__device__ __forceinline__ uint32_t slot_blocks(const Shared* sh, int slot) {
  const volatile uint32_t* w = sh->warp_blk[slot];
  uint32_t b = 0;
#pragma unroll
  for (int i = 0; i < kGateWarps; ++i) b |= w[i];
  return b;
}

// MMA issue for one CTA, run by ONE thread.  Two measured facts shape this code.  (1) The
// whole kernel must fit the instruction cache: with every tap, K step and layer variant unrolled
// at two call sites it was about 260 KB of code, every role ran from instruction-cache misses,
// and one MMA took 130-300 cycles to issue.  (2) A tcgen05.mma slot costs about 50 cycles of
// the issuing thread whether or not its predicate is on, and a rolled loop with run-time
// bounds costs 200-300 cycles per tap; with the three taps of a filter row and their K steps
// unrolled (compile-time K range, descriptors = register + immediate) the same thread issues
// at the rate of the tensor pipe (50-62 cycles per 128x64x16 MMA).  So: 3x3 layers run through
// a few small unrolled variants selected once per phase, everything else through one rolled
// loop, and the phase is inlined at a single call site.  Weight tiles are visited in the order
// base_tile()/cond_tile() enumerate them, which is the order the weight producer loads them.
template <int NT, bool I8>
struct MmaIssuer {
  static constexpr uint32_t kWTile = (uint32_t)(NT * 128) >> 4;   // weight tile, 16-byte units
  Shared* sh;
  Ctx cx;
  uint32_t desc_hi;                      // upper descriptor word (see ptx::smem_desc)
  uint32_t a_base_lo, b_base_lo;         // lower descriptor words of the ring bases
  uint32_t patch_lo;                     // patch buffer size in 16-byte units
  // A-descriptor offset of tap (r, sx) from the first patch buffer of a chunk = f[r] + c[sx]
  // (3x3) or r * row_lo + sx * 8 (other sizes, stride 1).  Stride 1: the patch read from pixel
  // r*(W+pad)+sx on.  Stride 2 (3x3, pad 1): output (h,w) reads input (2h+r-1, 2w+sx-1), i.e.
  // plane (r odd ? 0 : 1, sx odd ? 0 : 1) at (h + (r ? 0 : -1), w + (sx ? 0 : -1)); every plane
  // patch starts one row and one column early, so the offset within the plane's buffer is
  // (r ? 1 : 0) rows + (sx ? 1 : 0) pixels, and plane p is the p-th buffer of the chunk.
  uint32_t f0, f1, f2, c0, c1, c2, row_lo;
  int resident, a0, na /* ring slots [a0, na) */, nb, kp16 /* base K steps per tap */, chunks, base_chunks, base_tiles, kh, kw, planes;
  int pad8;
  int as, bs;                            // ring slots and the parities of their "full" barriers
  uint32_t apar, bpar;
  // per phase
  uint32_t d_tmem, idesc, a_grp, b_lo, acc, blk_off_b;
  int a_first, b_held;
  int st_tile;            // rolled path: tiles used of the current stage
  uint32_t st_base;       // ... and its first tile
  bool ok;
  bool share, release;   // shared patch ring: slot by job index; release: this issuer frees patches
  uint32_t lead;         // 1 in the lane that issues the tcgen05 instructions (the whole warp runs this code)

  // slot0, slots: the part of the patch ring this issuer consumes
  __device__ __forceinline__ void init(Shared* sh_, const Ctx& cx_, const uint8_t* s_a,
                                       const uint8_t* s_b, const TcPlan& P, const LayerDims& L,
                                       int slot0, int slots) {
    sh = sh_; cx = cx_;
    // descriptor words: upper = 8-row groups 1024 bytes apart, 128-byte swizzle, version 1;
    // lower = (address >> 4) | (1 << 16)
    desc_hi = (uint32_t)(ptx::smem_desc(0, 1024, 2) >> 32);
    a_base_lo = (ptx::smem_u32(s_a) >> 4) | 0x10000u;
    b_base_lo = (ptx::smem_u32(s_b) >> 4) | 0x10000u;
    patch_lo = (uint32_t)P.patch_bytes >> 4;
    row_lo = (uint32_t)P.wp * 8u;
    if (P.planes == 4) {
      f0 = 2u * patch_lo; f1 = row_lo; f2 = 2u * patch_lo + row_lo;
      c0 = patch_lo; c1 = 8u; c2 = patch_lo + 8u;
    } else {
      f0 = 0u; f1 = row_lo; f2 = 2u * row_lo;
      c0 = 0u; c1 = 8u; c2 = 16u;
    }
    resident = P.resident; a0 = slot0; na = slot0 + slots; nb = P.nb; kp16 = L.c_p / (P.ck / 4); chunks = P.chunks; pad8 = P.pad8;
    base_chunks = P.base_chunks; base_tiles = P.base_tiles; kh = L.kh; kw = L.kw; planes = P.planes;
    as = slot0; bs = 0; apar = 0; bpar = 0;
    a_first = slot0; b_held = 0; ok = true;
    share = false; release = true;
  }
  __device__ __forceinline__ void mma(uint32_t al, uint32_t bl) {
    const uint64_t da = ((uint64_t)desc_hi << 32) | al;
    const uint64_t db = ((uint64_t)desc_hi << 32) | bl;
    if (I8) ptx::umma_s8_if(lead, d_tmem, da, db, idesc, acc);
    else ptx::umma_bf16_if(lead, d_tmem, da, db, idesc, acc);
    acc = 1u;
  }
  // the patch buffer(s) of the next chunk in the ring: one, or the four planes of a stride-2
  // layer, which sit in consecutive slots (the ring length is then a multiple of four)
  __device__ __forceinline__ void acquire_a() {
    a_first = as;
    a_grp = a_base_lo + (uint32_t)as * patch_lo;
    for (int pl = 0; pl < planes; ++pl) {
      ok = ok && wait_bar_warp(cx, &sh->a_full[as], apar, 7);
      if (++as == na) { as = a0; apar ^= 1; }
    }
  }
  __device__ __forceinline__ void release_a() {
    if (!release) return;
    for (int pl = 0; pl < planes; ++pl) ptx::umma_commit_if(lead, &sh->a_empty[a_first + pl]);
  }
  // Next three weight tiles (a stage).  Resident weights: tiles follow one another from b_lo
  // on (b_lo includes the column-block offset).  Ring: the weight producer fills a ring of
  // stages of up to three consecutive tiles of a phase, one barrier pair per stage, so that the
  // issuer pays one wait and one commit per filter row instead of per tap.
  template <bool RES>
  __device__ __forceinline__ uint32_t acquire_stage() {
    if (RES) { const uint32_t b = b_lo; b_lo += kStageTiles * kWTile; return b; }
    ok = ok && wait_bar_warp(cx, &sh->b_full[bs], bpar, 8);
    b_held = bs;
    const uint32_t b = b_base_lo + (uint32_t)bs * (kStageTiles * kWTile) + blk_off_b;
    if (++bs == nb) { bs = 0; bpar ^= 1; }
    return b;
  }
  template <bool RES>
  __device__ __forceinline__ void release_stage() {
    if (!RES) ptx::umma_commit_if(lead, &sh->b_empty[b_held]);
  }
  // 3x3: K steps [KS0, KS1) of every tap of the next chunk in the ring, one weight tile per tap
  template <bool RES, int KS0, int KS1>
  __device__ __forceinline__ void chunk_taps3() {
    acquire_a();
    if (!ok) return;
    // (the row step is carried in a variable, not selected by r, so that the loop stays rolled)
    uint32_t a_row = a_grp + f0, step = f1 - f0;
#pragma unroll 1
    for (int r = 0; r < 3; ++r) {
      const uint32_t b_row = acquire_stage<RES>();   // the three taps of a filter row = one stage
      if (!RES && !ok) return;
#pragma unroll
      for (int sx = 0; sx < 3; ++sx) {
        const uint32_t b_t = b_row + sx * kWTile;
        const uint32_t a_t = a_row + (sx == 0 ? c0 : sx == 1 ? c1 : c2);
#pragma unroll
        for (int ks = KS0; ks < KS1; ++ks) mma(a_t + ks * 2, b_t + (ks - KS0) * 2);
      }
      release_stage<RES>();
      a_row += step;
      step = f2 - f1;
    }
    release_a();
  }
  // 3x3 base path when c_p < 64: the first KP K steps of chunk 0; a weight tile covers 4/KP taps
  template <bool RES, int KP>
  __device__ __forceinline__ void base_small3() {
    constexpr int TPT = 4 / KP;
    acquire_a();
    if (!ok) return;
    uint32_t b_row = 0;
#pragma unroll
    for (int t = 0; t < 9; ++t) {
      const int tile = t / TPT;                          // (compile-time: the loop is unrolled)
      if (t % TPT == 0 && tile % kStageTiles == 0) b_row = acquire_stage<RES>();
      if (!RES && !ok) return;
      const uint32_t b_t = b_row + (uint32_t)(tile % kStageTiles) * kWTile;
      const uint32_t a_t = a_grp + (t / 3 == 0 ? f0 : t / 3 == 1 ? f1 : f2) + (t % 3 == 0 ? c0 : t % 3 == 1 ? c1 : c2);
#pragma unroll
      for (int ks = 0; ks < KP; ++ks) mma(a_t + ks * 2, b_t + ((t % TPT) * KP + ks) * 2);
      if ((t % TPT == TPT - 1 && tile % kStageTiles == kStageTiles - 1) || t == 8) release_stage<RES>();
    }
    release_a();
  }
  // rolled path: the current tile is done; a stage is released when its last tile is
  __device__ __forceinline__ void next_tile() {
    if (++st_tile == kStageTiles) {
      if (!resident) release_stage<false>();
      st_tile = 0;
    }
  }
  // any kernel size (stride 1): K steps [ks0, ks1) of every tap of the next chunk, a weight
  // tile covering `tpt` taps.  Rolled; slow to issue, small in code.
  __device__ __forceinline__ void chunk_taps_any(int ks0, int ks1, int tpt) {
    acquire_a();
    if (!ok) return;
    int in_tile = 0;          // taps done with the current weight tile
    uint32_t b_t = 0;
    for (int r = 0; r < kh; ++r) {
      const uint32_t a_row = a_grp + (uint32_t)r * row_lo;
      for (int sx = 0; sx < kw; ++sx) {
        if (in_tile == 0) {
          // next tile of the phase: a new stage every kStageTiles tiles
          if (st_tile == 0) {
            st_base = resident ? acquire_stage<true>() : acquire_stage<false>();
            if (!ok) return;
          }
          b_t = st_base + (uint32_t)st_tile * kWTile;
        }
        const uint32_t a_t = a_row + (uint32_t)sx * 8u;
        const uint32_t b_k = b_t + (uint32_t)((in_tile * (ks1 - ks0) - ks0) * 2);
        for (int ks = ks0; ks < ks1; ++ks) mma(a_t + ks * 2, b_k + ks * 2);
        if (++in_tile == tpt) { in_tile = 0; next_tile(); }
      }
    }
    if (in_tile != 0) next_tile();
    release_a();
  }
  // Chunks and K ranges of a phase.
  //   c_p >= one chunk: the base path takes chunks [0, base_chunks), the conditional path the
  //   rest; every tap of a chunk has its own weight tile and four K steps.
  //   c_p < one chunk (kp16 = 1 or 2 K steps): the base path takes K steps [0, kp16) of chunk
  //   0, a weight tile covering 4/kp16 taps; the conditional path takes K steps [kp16, 4) of
  //   chunk 0 and then the remaining chunks.
  template <bool RES>
  __device__ __forceinline__ void phase3(bool cond) {
    int nfull;        // whole chunks (four K steps per tap) after the first, partial one
    int small = 0;    // K steps per tap of a phase that runs on tiles of several taps (one call site each)
    int partial = 0;  // first K step of a conditional path that starts behind the base channels of chunk 0
    if (kp16 >= 4) {
      nfull = cond ? chunks - base_chunks : base_chunks;
    } else if (!cond) {
      small = kp16; nfull = 0;
    } else if (pad8 == 2) {
      small = 2; nfull = 0;         // (int8, 64 input channels: two K steps per tap, two taps per tile)
    } else if (pad8) {
      nfull = chunks;               // (repacked weights: zeros multiply the base channels)
    } else {
      partial = kp16; nfull = chunks - 1;
    }
    if (small == 1) base_small3<RES, 1>(); else if (small == 2) base_small3<RES, 2>();
    if (partial == 1) chunk_taps3<RES, 1, 4>(); else if (partial == 2) chunk_taps3<RES, 2, 4>();
#pragma unroll 1
    for (int q = 0; q < nfull && ok; ++q) chunk_taps3<RES, 0, 4>();
  }
  __device__ __forceinline__ void phase_any(bool cond) {
    if (kp16 >= 4) {
      const int q0 = cond ? base_chunks : 0, q1 = cond ? chunks : base_chunks;
      for (int q = q0; q < q1 && ok; ++q) chunk_taps_any(0, 4, 1);
    } else if (!cond) {
      chunk_taps_any(0, kp16, 4 / kp16);
    } else if (pad8 == 2) {
      chunk_taps_any(0, 2, 2);
    } else {
      chunk_taps_any(pad8 ? 0 : kp16, 4, 1);
      for (int q = 1; q < chunks && ok; ++q) chunk_taps_any(0, 4, 1);
    }
  }
  // base or conditional MMAs of one job into the accumulator at d; `blocks` = column blocks to
  // compute (all of them for the base path)
  __device__ __forceinline__ bool run_phase(uint32_t d, bool cond, uint32_t blocks, int j) {
    constexpr uint32_t kAll = (1u << (NT / 64)) - 1u;
    if (share) { as = j % na; apar = (uint32_t)(j / na) & 1u; }   // (a0 = 0 in this mode)
    // a single block of two: accumulator columns and weight rows 64..127
    d_tmem = d + (blocks == 2u ? 64u : 0u);
    blk_off_b = blocks == 2u ? (64u * 128u / 16u) : 0u;
    const int n = blocks == kAll ? NT : 64;
    idesc = I8 ? ptx::idesc_s8(kBM, n) : ptx::idesc_bf16(kBM, n);
    acc = 0u;   // the first K step overwrites the accumulator
    ok = true;
    b_lo = b_base_lo + blk_off_b + (cond ? (uint32_t)base_tiles * kWTile : 0u);   // resident tiles
    if (kh == 3 && kw == 3) {
      if (resident) phase3<true>(cond); else phase3<false>(cond);
    } else {
      st_tile = 0;
      phase_any(cond);
      // a phase's last stage may hold fewer than kStageTiles tiles
      if (ok && st_tile != 0) {
        if (!resident) release_stage<false>();
        st_tile = 0;
      }
    }
    return ok;
  }
};

template <int NT, bool I8>
__global__ void __launch_bounds__(kThreads, 1)
tc_gated_conv_kernel(const __grid_constant__ CUtensorMap map_x,
                     const __grid_constant__ CUtensorMap map_x1,
                     const __grid_constant__ CUtensorMap map_x2,
                     const __grid_constant__ CUtensorMap map_x3,
                     const __grid_constant__ CUtensorMap map_wb,
                     const __grid_constant__ CUtensorMap map_wc,
                     const __grid_constant__ CUtensorMap map_y,
                     const __grid_constant__ TcParams prm) {
  extern __shared__ uint8_t smem_raw[];
  CG_PROF_T(prof_k0);
  ptx::grid_launch_dependents();   // the next kernel in the stream may start as SMs become free
  // 1024-byte alignment as an offset from the array, so that every pointer below is still known
  // to point into shared memory (shared-memory loads and stores, not generic ones)
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  const LayerDims& L = prm.L;
  const TcPlan& P = prm.P;
  uint8_t* s_a = smem + P.off_a;
  uint8_t* s_b = smem + P.off_b;
  uint8_t* s_y = smem + P.off_y;
  // per-channel constants of this column tile.  Floating point: t, a1, b1, a2, b2.  Integer
  // layers reuse the region: threshold, two multipliers (int32), two offsets (int64).
  float* s_t = (float*)(smem + P.off_consts);
  float4* s_k = (float4*)(s_t + NT);                       // per channel {a1, b1, a2, b2}
  float* s_t2 = s_t + 5 * NT;                              // upper thresholds of the two-sided gate (Section 3.2)
  const bool two_sided = !I8 && prm.bn.delta_high != nullptr;
  int* s_qt = (int*)s_t;
  int* s_qm1 = s_qt + NT;
  int* s_qm2 = s_qm1 + NT;
  long long* s_qo1 = (long long*)(s_qm2 + NT + (NT & 1));
  long long* s_qo2 = s_qo1 + NT;
  uint32_t* s_mask = (uint32_t*)(smem + P.off_mask);       // [4][128][NT/32]
  int* s_wx = (int*)(smem + P.off_tables);                 // [base_tiles + cond_tiles] K coordinates
  Shared* sh = (Shared*)(smem + P.off_bar);
  const Ctx cx{sh, prm.counters};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // jobs of this CTA: a fixed column tile, every `groups`-th row tile
  const int tile_n = blockIdx.x % P.tiles_n;
  const int group = blockIdx.x / P.tiles_n;
  const int groups = gridDim.x / P.tiles_n;
  const int jobs = group < P.tiles_m ? (P.tiles_m - group + groups - 1) / groups : 0;
  const int taps = L.kh * L.kw;
  const bool dense = (P.cond_mode == CG_COND_DENSE);
  const bool compact = (P.cond_mode == CG_COND_COMPACT);   // R is computed by a second kernel
  const bool has_cond = P.cond_tiles > 0 && !compact && !prm.base_only;
  const int cond_first_chunk = L.c_p >= P.ck ? P.base_chunks : 0;
  constexpr int kBlocks = NT / 64;
  // 64-channel column blocks of this tile that hold real output channels (the last tile of a
  // layer whose c_out is not a multiple of NT holds fewer)
  // (bf16 layers: c_out is a multiple of NT, the count is a compile-time constant)
  const int real_blocks = I8 ? min(kBlocks, (L.c_out - (int)(blockIdx.x % P.tiles_n) * NT + 63) / 64) : kBlocks;
  const uint32_t kAllBlocks = (1u << real_blocks) - 1u;
  const int words_here = 2 * real_blocks;                  // mask words of this tile that belong to real channels
  constexpr int kWords = NT / 32;
  constexpr int kNP = NT == 64 ? 4 : 3;      // P accumulators in TMEM
  constexpr int kNR = NT == 64 ? 4 : 1;      // R accumulators in TMEM
  const uint32_t w_tile_bytes = NT * 128;
  const uint32_t patch_tx = (uint32_t)P.box_pixels * 128u;

  auto job_origin = [&](int j, int& n0, int& h0) {
    const int tile_m = group + j * groups;
    if (P.images_mode) { n0 = tile_m * P.ni; h0 = 0; }
    else { n0 = tile_m / P.tiles_per_image; h0 = (tile_m - n0 * P.tiles_per_image) * P.r; }
  };

  // ---------------------------------------------------------------- setup
  if (threadIdx.x == 0) {
    for (int i = 0; i < P.na; ++i) { ptx::mbar_init(&sh->a_full[i], 1); ptx::mbar_init(&sh->a_empty[i], 1); }
    for (int i = 0; i < P.nb; ++i) { ptx::mbar_init(&sh->b_full[i], 1); ptx::mbar_init(&sh->b_empty[i], 1); }
    ptx::mbar_init(&sh->w_ready, 1);
    ptx::mbar_init(&sh->setup_done, kEpiWarps);
    for (int i = 0; i < 4; ++i) {
      ptx::mbar_init(&sh->base_done[i], 1);
      ptx::mbar_init(&sh->gate_done[i], kGateWarps);   // one arrival per warp of the group
      ptx::mbar_init(&sh->p_free[i], kCombWarps);
      ptx::mbar_init(&sh->cond_done[i], 1);
      ptx::mbar_init(&sh->r_free[i], kCombWarps);
    }
    sh->abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_x); ptx::prefetch_tensormap(&map_wb);
    if (P.planes == 4) { ptx::prefetch_tensormap(&map_x1); ptx::prefetch_tensormap(&map_x2); ptx::prefetch_tensormap(&map_x3); }
    ptx::prefetch_tensormap(&map_wc); ptx::prefetch_tensormap(&map_y);
  }
  if (warp == 1) ptx::tmem_alloc(&sh->tmem_base, 512);
  if (warp == 2) {
    // K coordinate of every weight tile, for the weight loads
    for (int bt = lane; bt < P.base_tiles + P.cond_tiles; bt += 32)
      s_wx[bt] = (bt < P.base_tiles ? base_tile(L, P.ck, bt) : cond_tile(L, P.ck, bt - P.base_tiles, P.pad8)).x;
  }
  // Only the barriers, the TMEM address and the tile coordinates are needed before the first
  // copies can be issued: the rest of the set-up (below, epilogue warps) overlaps those copies.
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  // everything above touched only this CTA's own state; from here on global memory is read and
  // written, so the kernel that ran before this one in the stream must be complete
  ptx::grid_dependency_wait();
  if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
    const int et = threadIdx.x - kEpiThread0;
    // zero the rows behind the TMA box of every patch buffer: they stand for the right padding
    // of the last patch row and are never written again; the MMA issuers wait for setup_done
    const int tail0 = P.box_pixels * 128, tail1 = P.patch_rows * 128;
    for (int q = 0; q < P.na; ++q) {
      uint8_t* base = s_a + (size_t)q * P.patch_bytes;
      for (int o = tail0 + et * 16; o < tail1; o += kEpiThreads * 16) *(uint4*)(base + o) = make_uint4(0, 0, 0, 0);
    }
    ptx::fence_proxy_async();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(&sh->setup_done);
    // per-channel constants of this column tile, for the epilogue warps themselves
    for (int c = et; c < NT; c += kEpiThreads) {
      const int cg_ = tile_n * NT + c;
      if (I8) {
        const bool real = cg_ < L.c_out;               // (columns behind c_out: never fire, never stored)
        s_qt[c] = real ? prm.bn.q_gate_thr[cg_] : 0x7fffffff;
        s_qm1[c] = real ? prm.bn.q_mul_base[cg_] : 0; s_qm2[c] = real ? prm.bn.q_mul_full[cg_] : 0;
        s_qo1[c] = real ? prm.bn.q_off_base[cg_] : 0ll; s_qo2[c] = real ? prm.bn.q_off_full[cg_] : 0ll;
      } else {
        const ChannelConsts k = fold_channel(prm.bn, prm.delta, L.eps, cg_);
        s_t[c] = k.t; s_k[c] = make_float4(k.a1, k.b1, k.a2, k.b2); s_t2[c] = k.t2;
      }
    }
    ptx::named_bar_sync(2, kEpiThreads);
  }
  const uint32_t tmem = sh->tmem_base;
#ifdef CG_PROF
  const long long prof_t0 = clock64();
#endif

  if (warp == 0) {
    // ============================================================ patch (A) producer
    // Loads chunks in the order the MMA issuer consumes them: base(0) | base(1) cond(0) | ...
    // With two issuers the ring is either split -- slots [0, split_a) for the base path, the
    // rest for the conditional path, each part with its own cursor -- or, when the layer has a
    // single input chunk, shared: job j's patch is loaded once into slot j % na and serves both
    // paths (the conditional issuer releases it).
    if (jobs > 0) {   // (the whole warp, convergent; lane 0 issues the copies)
      // ring slot and the parity of its "empty" barrier, per ring part
      int as0 = 0, as1 = P.split_a;
      uint32_t apar0 = 1, apar1 = 1;
      const int hi0 = P.split_a ? P.split_a : P.na;
      bool ok = true;
      auto load_chunks = [&](int j, int q0, int q1, int part) {
        int n0, h0;
        job_origin(j, n0, h0);
        const int lead = P.planes == 4 ? 1 : L.pad;   // zero rows/columns in front of the patch
        for (int q = q0; q < q1 && ok; ++q) {
          for (int pl = 0; pl < P.planes && ok; ++pl) {
            const int slot = part ? as1 : as0;
            ok = wait_bar_warp(cx, &sh->a_empty[slot], part ? apar1 : apar0, 1);
            if (!ok) return;
            const CUtensorMap* mx = pl == 0 ? &map_x : (pl == 1 ? &map_x1 : (pl == 2 ? &map_x2 : &map_x3));
            if (lane == 0) {
              ptx::mbar_expect_tx(&sh->a_full[slot], patch_tx);
              ptx::tma_load_4d(s_a + (size_t)slot * P.patch_bytes, mx, &sh->a_full[slot], q * P.ck, -lead,
                               h0 - lead, n0);
            }
            if (part) { if (++as1 == P.na) { as1 = P.split_a; apar1 ^= 1; } }
            else if (++as0 == hi0) { as0 = 0; apar0 ^= 1; }
          }
        }
      };
      const int cond_part = P.split_a ? 1 : 0;
      // Channel grouping (Section 3.3): the column tile lies inside one output group; its base
      // path reads that group's input chunks, its conditional path the others in ascending order.
      // The weight tiles keep their K coordinates: only the chunks of x change.
      const int own0 = L.grouping ? (tile_n * NT) / (L.c_out / L.groups) * P.base_chunks : 0;
      const int cond_lo = L.grouping ? own0 + P.base_chunks : cond_first_chunk;   // first chunk behind the base chunks
      for (int j = 0; j <= jobs && ok; ++j) {
        if (j < jobs) { load_chunks(j, own0, own0 + P.base_chunks, 0); CG_PROF_EV(j, 0); }
        if (j >= 1 && has_cond && ok && !P.share_a) {
          const int jj = j - 1;
          uint32_t blocks = kAllBlocks;
          if (!dense) {
            ok = wait_bar_warp(cx, &sh->gate_done[jj % kNP], (jj / kNP) & 1, 2);
            if (!ok) break;
            blocks = __shfl_sync(0xffffffffu, slot_blocks(sh, jj % kNP), 0);
          }
          if (blocks) {
            // (one call site: the chunks in front of the tile's own group, then those behind it)
#pragma unroll 1
            for (int part2 = L.grouping ? 0 : 1; part2 < 2 && ok; ++part2)
              load_chunks(jj, part2 ? cond_lo : 0, part2 ? P.chunks : own0, cond_part);
          }
        }
      }
    }
  } else if (warp == 2 && P.issuers != 3) {
    // ============================================================ weight (B) producer
    if (jobs > 0) {   // (the whole warp, convergent; lane 0 issues the copies)
      if (P.resident) {
        const uint32_t total = (uint32_t)(P.base_tiles + P.cond_tiles) * w_tile_bytes;
        if (lane == 0) {
          ptx::mbar_expect_tx(&sh->w_ready, total);
          for (int bt = 0; bt < P.base_tiles + P.cond_tiles; ++bt)
            ptx::tma_load_2d(s_b + (size_t)bt * w_tile_bytes, bt < P.base_tiles ? &map_wb : &map_wc,
                             &sh->w_ready, s_wx[bt], tile_n * NT);
        }
      } else {
        int bs = 0;            // ring slot and the parity of its "empty" barrier
        uint32_t bpar = 1;
        bool ok = true;
        // the tiles of a phase, in stages of up to kStageTiles tiles on one barrier
        auto load_tiles = [&](const CUtensorMap* map, int t0, int n) {
          for (int g = 0; g < n && ok; g += kStageTiles) {
            ok = wait_bar_warp(cx, &sh->b_empty[bs], bpar, 3);
            if (!ok) return;
            const int cnt = min(kStageTiles, n - g);
            if (lane == 0) {
              ptx::mbar_expect_tx(&sh->b_full[bs], (uint32_t)cnt * w_tile_bytes);
              for (int k = 0; k < cnt; ++k)
                ptx::tma_load_2d(s_b + (size_t)(bs * kStageTiles + k) * w_tile_bytes, map, &sh->b_full[bs],
                                 s_wx[t0 + g + k], tile_n * NT);
            }
            if (++bs == P.nb) { bs = 0; bpar ^= 1; }
          }
        };
        for (int j = 0; j <= jobs && ok; ++j) {
          if (j < jobs) load_tiles(&map_wb, 0, P.base_tiles);
          if (j >= 1 && has_cond && ok) {
            const int jj = j - 1;
            uint32_t blocks = kAllBlocks;
            if (!dense) {
              ok = wait_bar_warp(cx, &sh->gate_done[jj % kNP], (jj / kNP) & 1, 4);
              if (!ok) break;
              blocks = __shfl_sync(0xffffffffu, slot_blocks(sh, jj % kNP), 0);
            }
            if (blocks) load_tiles(&map_wc, P.base_tiles, P.cond_tiles);
          }
        }
      }
    }
  } else if (warp == 1 || warp == 3 || warp == kIssuer3Warp) {
    // ============================================================ MMA issuer(s)
    // One thread issues the base path of job j+1 and then the conditional path of job j; when
    // the patch ring is split (resident weights), warp 3 takes the conditional path instead, so
    // the per-job bookkeeping of the two paths runs in parallel.
    // Conditional phases: one issuer -> warp 1 does both paths; two issuers (resident weights,
    // several input chunks) -> warp 3; three issuers (resident weights, a single input chunk whose
    // patch serves both paths: 9 base and 27 conditional MMAs per job) -> warps 3 and 2 take
    // alternate jobs, so that two conditional phases are issued at the same time and warp 1 is
    // free to start the base path of the next job as soon as its patch has landed.
    const bool do_base = warp == 1;
    auto cond_is_mine = [&](int jj) {
      if (P.issuers == 1) return warp == 1;
      if (P.issuers == 2) return warp == 3;
      return (jj & 1) ? warp == kIssuer3Warp : warp == 3;
    };
    const bool have_role = warp == 1 || (warp == 3 && P.issuers >= 2) || (warp == kIssuer3Warp && P.issuers == 3);
    if (jobs > 0 && have_role) {   // (the whole warp, convergent; lane 0 issues)
      if (warp == kIssuer3Warp && lane == 0) {
        // (three issuers imply resident weights: this warp loads them once, then issues MMAs)
        ptx::mbar_expect_tx(&sh->w_ready, (uint32_t)(P.base_tiles + P.cond_tiles) * w_tile_bytes);
        for (int bt = 0; bt < P.base_tiles + P.cond_tiles; ++bt)
          ptx::tma_load_2d(s_b + (size_t)bt * w_tile_bytes, bt < P.base_tiles ? &map_wb : &map_wc,
                           &sh->w_ready, s_wx[bt], tile_n * NT);
      }
      __syncwarp();
      MmaIssuer<NT, I8> mi;
      mi.lead = lane == 0 ? 1u : 0u;
      if (P.split_a) mi.init(sh, cx, s_a, s_b, P, L, do_base ? 0 : P.split_a, do_base ? P.split_a : P.na - P.split_a);
      else mi.init(sh, cx, s_a, s_b, P, L, 0, P.na);
      mi.share = P.share_a != 0;
      bool ok = wait_bar_warp(cx, &sh->setup_done, 0, 5);
      if (ok && P.resident) ok = wait_bar_warp(cx, &sh->w_ready, 0, 6);
      // steps 2j (base path of job j) and 2j+1 (conditional path of job j-1), through ONE
      // inlined copy of the issue loop
      for (int s = 0; s < 2 * (jobs + 1) && ok; ++s) {
        const int j = s >> 1;
        const bool cond = (s & 1) != 0;
        uint32_t d, blocks = kAllBlocks;
        int jr;
        uint64_t* done;
        if (!cond) {
          if (!do_base || j >= jobs) continue;
          const int ps = j % kNP;
          ok = wait_bar_warp(cx, &sh->p_free[ps], ((j / kNP) & 1) ^ 1, 9);
          if (!ok) break;
          d = tmem + (uint32_t)(ps * NT); jr = j; done = &sh->base_done[ps];
          CG_PROF_EV(j, 1);
        } else {
          if (j < 1 || !cond_is_mine(j - 1)) continue;
          const int jj = j - 1;
          const int rs = jj % kNR;
          d = tmem + (uint32_t)((kNP + rs) * NT); jr = jj; done = &sh->cond_done[rs];
          bool run = false;
          if (has_cond) {
            if (!dense) {
              ok = wait_bar_warp(cx, &sh->gate_done[jj % kNP], (jj / kNP) & 1, 10);
              if (!ok) break;
              blocks = __shfl_sync(0xffffffffu, slot_blocks(sh, jj % kNP), 0);
            }
            // the R slot's previous user must be done with it even when this job skips the
            // conditional path: otherwise cond_done could run two phases ahead of its waiters
            ok = wait_bar_warp(cx, &sh->r_free[rs], ((jj / kNR) & 1) ^ 1, 14);
            if (!ok) break;
            run = blocks != 0u;
            if (!run && P.share_a && lane == 0) ptx::mbar_arrive(&sh->a_empty[jj % P.na]);   // the job's patch is not needed again
          } else {
            ok = wait_bar_warp(cx, &sh->r_free[rs], ((jj / kNR) & 1) ^ 1, 15);
            if (!ok) break;
          }
          if (!run) {
            ptx::umma_commit_if(mi.lead, done);
            continue;
          }
          CG_PROF_EV(jj, 5);
        }
        ptx::tc_fence_after();
        mi.release = !(P.share_a && !cond);   // a shared patch is released by the conditional phase
        ok = mi.run_phase(d, cond, blocks, jr);
        if (!ok) break;
        ptx::umma_commit_if(mi.lead, done);
        CG_PROF_EV(jr, cond ? 6 : 2);
      }
    }
  } else {
    // ============================================================ epilogue (20 warps)
    // Two groups work on different jobs at the same time: warps 4-7 evaluate the gate of job j
    // (one warp per TMEM lane quadrant, all columns of the tile), warps 8-23 combine and store job
    // j-1 or earlier (quadrant x quarter of the columns).  The combine pass is the long one and
    // is latency-bound -- its shared-memory accesses queue behind the operand fetches of the
    // MMAs -- so it gets four warps per scheduler.
    constexpr int CW = NT / 4;                              // columns per combine warp: 16 or 32
    const bool gate_group = warp < kEpiWarp0 + kGateWarps;
    const int quad = warp & 3;
    const int cgi = gate_group ? 0 : (warp - kEpiWarp0 - kGateWarps) >> 2;   // column quarter
    const int col0 = cgi * CW;
    const bool phantom_cols = I8 && (int)(blockIdx.x % P.tiles_n) * NT + col0 >= L.c_out;   // (uniform over the warp)
    const int row = quad * 32 + lane;                      // TMEM lane = patch row i
    const int ct = threadIdx.x - kEpiThread0 - kGateWarps * 32;   // thread index within the combine group
    const int n_loc = P.images_mode ? row / P.ip : 0;
    const int rem = P.images_mode ? row - n_loc * P.ip : row;
    const int h_loc = rem / P.wp;
    const int w_out = rem - h_loc * P.wp;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    unsigned long long st_active = 0, st_rows_valid = 0, st_rows_active = 0;
    unsigned long long st_blocks_run = 0;                  // ct == 0
    bool ok = true;

    // gate of job j: P -> mask words (global + stash), block activity flags
    // (kExtra: thresholds per image -- the channel-wise gate -- and/or upper thresholds -- the
    // two-sided gate; the plain gate keeps its own, shorter instruction stream: the gate warps are
    // on the critical path of the 64-channel layers)
    auto gate_pass = [&](int j, auto extra_tag) {
      constexpr bool kExtra = decltype(extra_tag)::value;
      const int slot = j % kNP;
      ok = wait_bar(cx, &sh->base_done[slot], (j / kNP) & 1, 11);
      if (!ok) return;
      ptx::tc_fence_after();
      CG_PROF_T(pt0);
      if (warp == kEpiWarp0) CG_PROF_EV(j, 3);
      // the tile's columns go through the registers 32 at a time; the next 32 are loaded while
      // the current ones are compared
      uint32_t r[2][32];
      ptx::tmem_ld_nowait<32>(t_lane + (uint32_t)(slot * NT), r[0]);
      int n0, h0;
      job_origin(j, n0, h0);
      const int rows_here = P.images_mode ? L.ho : min(P.r, L.ho - h0);
      const bool valid = (w_out < L.wo) && (h_loc < rows_here) && (n_loc < P.ni) && (n0 + n_loc < L.n);
      const long long m = ((long long)(n0 + n_loc) * L.ho + (h0 + h_loc)) * L.wo + w_out;
      uint32_t* g_words = prm.mask + m * L.words + tile_n * kWords;
      // (channel-wise gate: the thresholds of this row's image)
      const float* t_row = (kExtra && !I8 && prm.t_img) ? prm.t_img + (size_t)(valid ? n0 + n_loc : 0) * L.c_out + tile_n * NT : nullptr;
      uint32_t* s_words = s_mask + (slot * 128 + row) * kWords;
      uint32_t fired_blocks = 0;
#pragma unroll
      for (int w = 0; w < kWords; ++w) {
        ptx::tmem_ld_wait<32>(r[w & 1]);
        if (w + 1 < kWords) ptx::tmem_ld_nowait<32>(t_lane + (uint32_t)(slot * NT + (w + 1) * 32), r[(w + 1) & 1]);
        // four partial words, so that the bit inserts do not form one dependent chain
        uint32_t pw[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          if (I8) {
            const int4 t4 = *(const int4*)(s_qt + w * 32 + q * 4);
            pw[q & 3] |= ((int)r[w & 1][q * 4 + 0] >= t4.x ? 1u : 0u) << (q * 4 + 0);
            pw[q & 3] |= ((int)r[w & 1][q * 4 + 1] >= t4.y ? 1u : 0u) << (q * 4 + 1);
            pw[q & 3] |= ((int)r[w & 1][q * 4 + 2] >= t4.z ? 1u : 0u) << (q * 4 + 2);
            pw[q & 3] |= ((int)r[w & 1][q * 4 + 3] >= t4.w ? 1u : 0u) << (q * 4 + 3);
          } else {
            float4 t4 = *(const float4*)(s_t + w * 32 + q * 4);
            if constexpr (kExtra) { if (t_row) t4 = __ldg((const float4*)(t_row + w * 32 + q * 4)); }
            pw[q & 3] |= (__uint_as_float(r[w & 1][q * 4 + 0]) >= t4.x ? 1u : 0u) << (q * 4 + 0);
            pw[q & 3] |= (__uint_as_float(r[w & 1][q * 4 + 1]) >= t4.y ? 1u : 0u) << (q * 4 + 1);
            pw[q & 3] |= (__uint_as_float(r[w & 1][q * 4 + 2]) >= t4.z ? 1u : 0u) << (q * 4 + 2);
            pw[q & 3] |= (__uint_as_float(r[w & 1][q * 4 + 3]) >= t4.w ? 1u : 0u) << (q * 4 + 3);
          }
        }
        uint32_t word = (pw[0] | pw[1]) | (pw[2] | pw[3]);
        if (kExtra && two_sided) {
          // Section 3.2: the gate also needs P <= the upper threshold (ties included)
          uint32_t ph[4] = {0u, 0u, 0u, 0u};
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float4 u4 = *(const float4*)(s_t2 + w * 32 + q * 4);
            ph[q & 3] |= (__uint_as_float(r[w & 1][q * 4 + 0]) <= u4.x ? 1u : 0u) << (q * 4 + 0);
            ph[q & 3] |= (__uint_as_float(r[w & 1][q * 4 + 1]) <= u4.y ? 1u : 0u) << (q * 4 + 1);
            ph[q & 3] |= (__uint_as_float(r[w & 1][q * 4 + 2]) <= u4.z ? 1u : 0u) << (q * 4 + 2);
            ph[q & 3] |= (__uint_as_float(r[w & 1][q * 4 + 3]) <= u4.w ? 1u : 0u) << (q * 4 + 3);
          }
          word &= (ph[0] | ph[1]) | (ph[2] | ph[3]);
        }
        if (!valid || w >= words_here) word = 0;
        s_words[w] = word;
        st_active += __popc(word);
        if (valid && prm.mask && w < words_here) g_words[w] = word;
        if (__ballot_sync(0xffffffffu, word != 0u)) fired_blocks |= 1u << (w >> 1);
      }
      // 64-channel column blocks with a firing gate, over the warp
      if (lane == 0) sh->warp_blk[slot][warp - kEpiWarp0] = fired_blocks;
      {
        const uint32_t row_valid = __ballot_sync(0xffffffffu, valid);
        if (lane == 0) st_rows_valid += __popc(row_valid);
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&sh->gate_done[slot]);
      CG_PROF_T(pt1);
      CG_PROF_ADD(16, pt0, pt1);
      if (warp == kEpiWarp0) CG_PROF_EV(j, 4);
    };

    // combine of job j: y = f(BN1(P)) or f(BN2(P+R)) by mask bit, staged and stored
    auto combine_pass = [&](int j) {
      const int slot = j % kNP, rslot = j % kNR;
      CG_PROF_T(pc0);
      // A wait that gives up must not keep its thread from the group barrier below, where the
      // sibling warps (whose waits may still have succeeded) are going to arrive: the decision to
      // leave is taken after that barrier, from the CTA-wide flag, by all of them together.
      ok = wait_bar(cx, &sh->gate_done[slot], (j / kNP) & 1, 12);   // every gate warp's flags and words
      const uint32_t blocks = !has_cond ? 0u : (dense ? kAllBlocks : slot_blocks(sh, slot));
      const uint32_t* s_words = s_mask + (slot * 128 + row) * kWords;
      uint32_t any = 0;                                              // cgi == 0: any gate of the row
      if (cgi == 0) {
#pragma unroll
        for (int cb = 0; cb < kWords; ++cb) any |= s_words[cb];
        const uint32_t row_active = __ballot_sync(0xffffffffu, any != 0);
        if (lane == 0) st_rows_active += __popc(row_active);
      }
      // the mask word that holds this warp's 16 or 32 columns, and their position in it
      const uint32_t wv = s_words[col0 >> 5];
      const int wshift = col0 & 31;
      ok = ok && wait_bar(cx, &sh->cond_done[rslot], (j / kNR) & 1, 13);
      ptx::tc_fence_after();
      if (warp == kEpiWarp0 + kGateWarps) CG_PROF_EV(j, 7);
      // the warp's columns go through the registers 16 at a time; the loads of the next 16 are
      // issued before the current ones are stored.  R is read only where the conditional path
      // ran and a gate of these rows fired.
      const bool block_ran = (blocks >> (col0 >> 6)) & 1u;
      uint32_t p[16], rr[16];
      const uint32_t t_p = t_lane + (uint32_t)(slot * NT + col0), t_r = t_lane + (uint32_t)((kNP + rslot) * NT + col0);
      bool have_r = block_ran && __ballot_sync(0xffffffffu, ((wv >> wshift) & 0xffffu) != 0u) != 0u;
      ptx::tmem_ld_nowait<16>(t_p, p);
      if (have_r) ptx::tmem_ld_nowait<16>(t_r, rr);
      if (ct == 0) {
        ptx::tma_store_wait_read();   // the previous store has finished reading the staging tile
        st_blocks_run += __popc(blocks);
      }
      if (compact && cgi == 0) {
        // rows with a firing gate get a slot in this column tile's list (order is arbitrary)
        const uint32_t act = __ballot_sync(0xffffffffu, any != 0);
        uint32_t base = 0;
        if (lane == 0 && act) base = atomicAdd(&prm.ws_counts[tile_n], (uint32_t)__popc(act));
        base = __shfl_sync(0xffffffffu, base, 0);
        sh->row_idx[row] = any ? (int)(base + __popc(act & ((1u << lane) - 1u))) : -1;
      }
      CG_PROF_T(pc1);
      ptx::named_bar_sync(1, kCombThreads);
      if (*(volatile uint32_t*)&sh->abort_flag) {   // (the same for every thread of the group)
        ptx::tmem_ld_wait_all();
        ok = false;
        return;
      }
      CG_PROF_T(pc2);
      // residual rows (the shortcut of a residual block, added before the activation)
      const __nv_bfloat16* res_row = nullptr;
      if (!I8 && prm.residual) {
        int n0, h0;
        job_origin(j, n0, h0);
        const int rows_here = P.images_mode ? L.ho : min(P.r, L.ho - h0);
        const bool valid = (w_out < L.wo) && (h_loc < rows_here) && (n_loc < P.ni) && (n0 + n_loc < L.n);
        if (valid)
          res_row = prm.residual + (((long long)(n0 + n_loc) * L.ho + (h0 + h_loc)) * L.wo + w_out) * L.c_out + tile_n * NT + col0;
      }
      uint32_t* rec = nullptr;                              // compact mode: this row's record
      if (compact) {
        const int list_idx = sh->row_idx[row];
        if (list_idx >= 0) {
          rec = prm.ws_rows + ((long long)tile_n * L.m + list_idx) * (NT + 4);
          if (cgi == 0) {
            int n0, h0;
            job_origin(j, n0, h0);
            const long long m_row = ((long long)(n0 + n_loc) * L.ho + (h0 + h_loc)) * L.wo + w_out;
            prm.ws_list[(long long)tile_n * L.m + list_idx] = (uint32_t)m_row;
          }
          if (wshift == 0) rec[NT + (col0 >> 5)] = wv;
        }
      }
#pragma unroll
      for (int sc = 0; sc < CW / 16; ++sc) {
      const int colS = col0 + sc * 16;                     // first column of this sub-chunk
      const uint32_t bits = wv >> (wshift + sc * 16);          // its mask bits
      ptx::tmem_ld_wait<16>(p);
      if (have_r) {
        ptx::tmem_ld_wait<16>(rr);
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) rr[i] = 0u;
      }
      if (rec) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *(uint4*)(rec + colS + q * 4) = make_uint4(p[q * 4], p[q * 4 + 1], p[q * 4 + 2], p[q * 4 + 3]);
      }
      if (I8 && phantom_cols) {
        // (columns behind c_out: nothing to compute, the y store clips them)
      } else if (I8) {
        // quantised layer: z = acc*mul + off (64-bit), q = (z + 2^(S-1)) >> S, clamp to int8;
        // 32 channels = 32 bytes = two 16-byte pieces of a 128-channel staging row
        uint8_t* st = s_y + (size_t)(colS >> 7) * P.stage_rows * 128 + (size_t)row * 128;
        const long long half_ulp = 1ll << (L.shift - 1);
        const int lo = L.relu ? 0 : -128;
        {
          constexpr int q = 0;
          uint32_t packed[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            uint32_t w4 = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int jx = q * 16 + e * 4 + k;
              const int c = colS + jx;
              const bool f = (bits >> jx) & 1u;
              const long long acc = f ? (long long)(int)p[jx] + (long long)(int)rr[jx] : (long long)(int)p[jx];
              const long long z = acc * (long long)(f ? s_qm2[c] : s_qm1[c]) + (f ? s_qo2[c] : s_qo1[c]);
              long long qv = (z + half_ulp) >> L.shift;
              qv = qv < lo ? lo : (qv > 127 ? 127 : qv);
              w4 |= ((uint32_t)qv & 0xffu) << (8 * k);
            }
            packed[e] = w4;
          }
          const int c16 = ((colS & 127) >> 4) + q;
          *(uint4*)(st + ((c16 ^ (row & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
      } else {
        uint8_t* st = s_y + (size_t)(colS >> 6) * P.stage_rows * 128 + (size_t)row * 128;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float4 k[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) k[i] = s_k[colS + q * 8 + i];
          uint4 res4 = make_uint4(0u, 0u, 0u, 0u);
          if (res_row) res4 = *(const uint4*)(res_row + sc * 16 + q * 8);
          const uint32_t resw[4] = {res4.x, res4.y, res4.z, res4.w};
          uint32_t packed[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int jx = q * 8 + e * 2;
            const float4 k0 = k[e * 2], k1 = k[e * 2 + 1];
            const bool f0 = (bits >> jx) & 1u, f1 = (bits >> (jx + 1)) & 1u;
            const float p0 = __uint_as_float(p[jx]), p1 = __uint_as_float(p[jx + 1]);
            // Eq. 1: the full sum P+R where the gate fired, the partial sum elsewhere, each
            // under the batch norm of its path (Section 4) as one fused multiply-add
            float v0 = f0 ? fmaf(k0.z, p0 + __uint_as_float(rr[jx]), k0.w) : fmaf(k0.x, p0, k0.y);
            float v1 = f1 ? fmaf(k1.z, p1 + __uint_as_float(rr[jx + 1]), k1.w) : fmaf(k1.x, p1, k1.y);
            if (res_row) {
              v0 += __uint_as_float(resw[e] << 16);
              v1 += __uint_as_float(resw[e] & 0xffff0000u);
            }
            if (L.relu) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); }
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
            packed[e] = *(const uint32_t*)&h2;
          }
          const int c16 = ((colS & 63) >> 3) + q;
          *(uint4*)(st + ((c16 ^ (row & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
      }
      if (sc + 1 < CW / 16) {
        const uint32_t nbits = (wv >> (wshift + (sc + 1) * 16)) & 0xffffu;
        have_r = block_ran && __ballot_sync(0xffffffffu, nbits != 0u) != 0u;
        ptx::tmem_ld_nowait<16>(t_p + (sc + 1) * 16, p);
        if (have_r) ptx::tmem_ld_nowait<16>(t_r + (sc + 1) * 16, rr);
      }
      }
      CG_PROF_T(pcb);
      CG_PROF_ADD(25, pc2, pcb);
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive(&sh->p_free[slot]);
        ptx::mbar_arrive(&sh->r_free[rslot]);
      }
      ptx::fence_proxy_async();
      CG_PROF_T(pc3);
      ptx::named_bar_sync(1, kCombThreads);
      CG_PROF_T(pc4);
      CG_PROF_ADD(17, pc0, pc1);
      CG_PROF_ADD(18, pc1, pc2);
      CG_PROF_ADD(19, pc2, pc3);
      CG_PROF_ADD(20, pc3, pc4);
      if (warp == kEpiWarp0 + kGateWarps) CG_PROF_EV(j, 8);
      if (ct == 0) {
        int n0, h0;
        job_origin(j, n0, h0);
        constexpr int kStoreCh = I8 ? 128 : 64;   // channels per 128-byte staging row
#pragma unroll
        for (int b = 0; b < NT / kStoreCh; ++b)
          ptx::tma_store_4d(&map_y, s_y + (size_t)b * P.stage_rows * 128, tile_n * NT + b * kStoreCh, 0, h0, n0);
        ptx::tma_store_commit();
      }
    };

    if (gate_group) {
      if (prm.t_img || two_sided) {
        for (int j = 0; j < jobs && ok; ++j) gate_pass(j, std::true_type{});
      } else {
        for (int j = 0; j < jobs && ok; ++j) gate_pass(j, std::false_type{});
      }
    } else {
      for (int j = 0; j < jobs && ok; ++j) combine_pass(j);
      if (ct == 0) ptx::tma_store_wait_all();
    }

    // counters of this CTA
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) st_active += __shfl_xor_sync(0xffffffffu, st_active, o);
    if (lane == 0 && ok) {
      atomicAdd(&prm.counters[CNT_ACTIVE], st_active);
      if (cgi == 0) {
        if (gate_group) atomicAdd(&prm.counters[CNT_ROWS_TOTAL], st_rows_valid);
        else atomicAdd(&prm.counters[CNT_ROWS_ACTIVE], st_rows_active);
      }
    }
    if (ct == 0 && ok) {
      const unsigned long long k_p = (unsigned long long)taps * L.c_p, k_r = (unsigned long long)taps * L.c_r;
      if (blockIdx.x == 0) atomicAdd(&prm.counters[CNT_CALLS], 1ull);
      atomicAdd(&prm.counters[CNT_TILES_TOTAL], (unsigned long long)real_blocks * jobs);
      atomicAdd(&prm.counters[CNT_TILES_SKIPPED],
                has_cond ? (unsigned long long)real_blocks * jobs - st_blocks_run : 0ull);
      atomicAdd(&prm.counters[CNT_EXEC_MACS],
                (unsigned long long)kBM * NT * k_p * jobs + (unsigned long long)kBM * 64ull * st_blocks_run * k_r);
    }
  }
#ifdef CG_PROF
  if (blockIdx.x == 0 && lane == 0) atomicAdd(&g_prof[warp * 32 + 31], (unsigned long long)(clock64() - prof_t0));
#endif
  // ---------------------------------------------------------------- teardown
  if (*(volatile uint32_t*)&sh->abort_flag) {
    // a wait gave up somewhere: let copies and MMAs that are still in flight finish (they take
    // microseconds) before the CTA's shared memory and TMEM go back
    const long long t_drain = clock64();
    while (clock64() - t_drain < 4000000ll) {}
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    ptx::tmem_dealloc(tmem, 512);
  }
#ifdef CG_PROF
  if (blockIdx.x == 0 && threadIdx.x == 32) {
    atomicAdd(&g_prof[24 * 32 + 0], (unsigned long long)(prof_t0 - prof_k0));
    atomicAdd(&g_prof[24 * 32 + 1], (unsigned long long)(clock64() - prof_k0));
  }
#endif
}

// ------------------------------------------------------------------------------------------
// Second kernel of CG_COND_COMPACT: the conditional path on compacted rows.
//
// The first kernel left, per column tile, the list of pixel rows in which a gate fired, their
// partial sums P and their mask words.  Here every 128 listed rows form one dense sub-GEMM:
// the A operand is GATHERED -- thread j copies, for each filter tap and 64-channel chunk, the
// 128 bytes of its row's input pixel (or zeros in the padding) into a swizzled tile with
// cp.async -- the weights come by TMA, the MMAs accumulate R in TMEM, and the epilogue
// overwrites y where d = 1 with f(BN2(P + R)) (Eq. 1, second case).  Work is proportional to
// the number of rows with a firing gate, not to the number of pixels.
constexpr int kCpThreads = 320;   // warp 0: weight TMA, warp 1: MMA, warps 2-5: gather, 6-9: epilogue
constexpr int kCpStages = 4;

struct CpShared {
  uint64_t full[kCpStages], empty[kCpStages];   // full: 128 gather arrivals + 1 TMA arrival
  uint64_t acc_done, acc_free;
  uint32_t tmem_base;
  uint32_t abort_flag;
};

struct CpParams {
  LayerDims L;
  TcPlan P;
  cg_bn_params bn;
  const float* delta;
  const __nv_bfloat16* x;
  __nv_bfloat16* y;
  const uint32_t* ws_counts;
  const uint32_t* ws_list;
  const uint32_t* ws_rows;
  unsigned long long* counters;
};

__device__ __forceinline__ bool cp_wait(CpShared* sh, unsigned long long* counters, uint64_t* bar,
                                        uint32_t parity, int site) {
  if (ptx::mbar_try_wait(bar, parity, 0u)) return true;
  const long long t0 = clock64();
  for (int i = 0; i < kSpinLimit; ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 15) == 15) {
      if (*(volatile uint32_t*)&sh->abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) break;
    }
  }
  if (atomicCAS(&counters[CNT_STATUS], 0ull, (unsigned long long)CG_ERR_DEVICE_TIMEOUT) == 0ull)
    atomicExch(&counters[CNT_SITE], (unsigned long long)site);
  atomicExch(&sh->abort_flag, 1u);
  return false;
}

template <int NT>
__global__ void __launch_bounds__(kCpThreads, 1)
tc_compact_cond_kernel(const __grid_constant__ CUtensorMap map_wc, const __grid_constant__ CpParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  const LayerDims& L = prm.L;
  const TcPlan& P = prm.P;
  constexpr int kWords = NT / 32;
  constexpr int kRec = NT + 4;
  constexpr uint32_t kStageBytes = 128 * 128 + NT * 128;
  uint8_t* s_stage = smem;                                        // [kCpStages][A 16 KB | B NT*128]
  float* s_a2 = (float*)(smem + kCpStages * kStageBytes);
  float* s_b2 = s_a2 + P.tiles_n * NT;
  CpShared* sh = (CpShared*)(s_b2 + P.tiles_n * NT);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int taps = L.kh * L.kw;
  const int kp16 = L.c_p >= P.ck ? 4 : L.c_p / (P.ck / 4);        // first conditional K step of chunk 0

  if (threadIdx.x == 0) {
    for (int i = 0; i < kCpStages; ++i) { ptx::mbar_init(&sh->full[i], 129); ptx::mbar_init(&sh->empty[i], 1); }
    ptx::mbar_init(&sh->acc_done, 1);
    ptx::mbar_init(&sh->acc_free, 128);
    sh->abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_wc);
  }
  if (warp == 1) ptx::tmem_alloc(&sh->tmem_base, NT);
  for (int c = threadIdx.x; c < P.tiles_n * NT; c += kCpThreads) {
    const ChannelConsts k = fold_channel(prm.bn, prm.delta, L.eps, c);
    s_a2[c] = k.a2; s_b2[c] = k.b2;
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = sh->tmem_base;

  // work items: (column tile, group of 128 listed rows), strided over the grid
  auto item_of = [&](int it, int& tn, int& g) -> bool {
    for (tn = 0; tn < P.tiles_n; ++tn) {
      const int groups = (int)((prm.ws_counts[tn] + 127u) / 128u);
      if (it < groups) { g = it; return true; }
      it -= groups;
    }
    return false;
  };

  if (warp == 0) {
    // ============================================================ weight (B) producer
    if (lane == 0) {
      int st = 0; uint32_t par = 1; bool ok = true;
      int tn, g;
      for (int it = blockIdx.x; ok && item_of(it, tn, g); it += gridDim.x) {
        for (int bt = 0; bt < P.cond_tiles && ok; ++bt) {
          ok = cp_wait(sh, prm.counters, &sh->empty[st], par, 21);
          if (!ok) break;
          ptx::mbar_expect_tx(&sh->full[st], NT * 128);
          ptx::tma_load_2d(s_stage + (size_t)st * kStageBytes + 128 * 128, &map_wc, &sh->full[st],
                           cond_tile(L, P.ck, bt, 0).x, tn * NT);
          if (++st == kCpStages) { st = 0; par ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ============================================================ MMA issuer (convergent warp)
    const uint32_t issue = lane == 0 ? 1u : 0u;
    const uint32_t desc_hi = (uint32_t)(ptx::smem_desc(0, 1024, 2) >> 32);
    int st = 0; uint32_t par = 0; bool ok = true;
    int tn, g, n_item = 0;
    for (int it = blockIdx.x; ok && item_of(it, tn, g); it += gridDim.x, ++n_item) {
      ok = cp_wait(sh, prm.counters, &sh->acc_free, (n_item & 1) ^ 1, 22);
      if (!ok) break;
      ptx::tc_fence_after();
      uint32_t acc = 0;
      for (int bt = 0; bt < P.cond_tiles && ok; ++bt) {
        ok = cp_wait(sh, prm.counters, &sh->full[st], par, 23);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t a_lo = ((ptx::smem_u32(s_stage + (size_t)st * kStageBytes)) >> 4) | 0x10000u;
        const uint32_t b_lo = a_lo + (128 * 128 >> 4);
        const int ks0 = (L.c_p < P.ck && bt < taps) ? kp16 : 0;     // chunk 0 also holds base channels
        for (int ks = ks0; ks < 4; ++ks) {
          ptx::umma_bf16_if(issue, tmem, ((uint64_t)desc_hi << 32) | (a_lo + ks * 2),
                            ((uint64_t)desc_hi << 32) | (b_lo + (ks - ks0) * 2), ptx::idesc_bf16(kBM, NT), acc);
          acc = 1u;
        }
        ptx::umma_commit_if(issue, &sh->empty[st]);
        if (++st == kCpStages) { st = 0; par ^= 1; }
      }
      if (ok) ptx::umma_commit_if(issue, &sh->acc_done);
    }
    __syncwarp();
  } else if (warp < 6) {
    // ============================================================ gather (A) producers: thread = row
    const int j = threadIdx.x - 64;
    int st = 0; uint32_t par = 1; bool ok = true;
    int tn, g;
    for (int it = blockIdx.x; ok && item_of(it, tn, g); it += gridDim.x) {
      const uint32_t cnt = prm.ws_counts[tn];
      const uint32_t ridx = (uint32_t)g * 128u + (uint32_t)j;
      const bool rvalid = ridx < cnt;
      int n = 0, ho = 0, wo = 0;
      if (rvalid) {
        const uint32_t m = prm.ws_list[(long long)tn * L.m + ridx];
        wo = (int)(m % (uint32_t)L.wo);
        ho = (int)((m / (uint32_t)L.wo) % (uint32_t)L.ho);
        n = (int)(m / ((uint32_t)L.wo * (uint32_t)L.ho));
      }
      int pending = 0;       // stages whose copies are issued but not yet published
      int pub = st;          // next stage to publish
      for (int bt = 0; bt < P.cond_tiles && ok; ++bt) {
        const WTile w = cond_tile(L, P.ck, bt, 0);
        int t;
        if (L.c_p >= P.ck) t = bt % taps; else t = bt < taps ? bt : (bt - taps) % taps;
        const int hi = ho * L.stride + t / L.kw - L.pad, wi = wo * L.stride + t % L.kw - L.pad;
        const bool pv = rvalid && hi >= 0 && hi < L.h && wi >= 0 && wi < L.w;
        const __nv_bfloat16* src = prm.x + ((((long long)n * L.h + (pv ? hi : 0)) * L.w + (pv ? wi : 0)) * L.c_in + w.chunk * 64);
        ok = cp_wait(sh, prm.counters, &sh->empty[st], par, 24);
        if (!ok) break;
        uint8_t* dst = s_stage + (size_t)st * kStageBytes + (size_t)j * 128;
#pragma unroll
        for (int c16 = 0; c16 < 8; ++c16)
          ptx::cp_async_16(dst + ((c16 ^ (j & 7)) << 4), src + c16 * 8, pv);
        ptx::cp_async_commit();
        if (++st == kCpStages) { st = 0; par ^= 1; }
        if (++pending == 3) {     // keep two stages of copies in flight, publish the oldest
          ptx::cp_async_wait<2>();
          ptx::fence_proxy_async();
          ptx::mbar_arrive(&sh->full[pub]);
          if (++pub == kCpStages) pub = 0;
          --pending;
        }
      }
      ptx::cp_async_wait<0>();
      ptx::fence_proxy_async();
      while (pending > 0) {
        ptx::mbar_arrive(&sh->full[pub]);
        if (++pub == kCpStages) pub = 0;
        --pending;
      }
    }
  } else {
    // ============================================================ epilogue: thread = listed row
    const int quad = warp & 3;
    const int j = quad * 32 + lane;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    bool ok = true;
    int tn, g, n_item = 0;
    unsigned long long items_done = 0;
    for (int it = blockIdx.x; ok && item_of(it, tn, g); it += gridDim.x, ++n_item) {
      ok = cp_wait(sh, prm.counters, &sh->acc_done, n_item & 1, 25);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t cnt = prm.ws_counts[tn];
      const uint32_t ridx = (uint32_t)g * 128u + (uint32_t)j;
      const bool rvalid = ridx < cnt;
      const uint32_t* rec = prm.ws_rows + ((long long)tn * L.m + (rvalid ? ridx : 0)) * kRec;
      const long long m = rvalid ? (long long)prm.ws_list[(long long)tn * L.m + ridx] : 0;
      __nv_bfloat16* yrow = prm.y + m * L.c_out + tn * NT;
#pragma unroll
      for (int cb = 0; cb < kWords; ++cb) {
        uint32_t r[32];
        ptx::tmem_ld32(t_lane + (uint32_t)(cb * 32), r);
        if (!rvalid) continue;
        const uint32_t word = rec[NT + cb];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t bits = (word >> (q * 8)) & 0xffu;
          if (bits == 0) continue;
          uint4* slot = (uint4*)(yrow + cb * 32 + q * 8);
          uint4 cur = *slot;
          uint32_t* cw = (uint32_t*)&cur;
          const uint4 p0 = *(const uint4*)(rec + cb * 32 + q * 8), p1 = *(const uint4*)(rec + cb * 32 + q * 8 + 4);
          const uint32_t pp[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int jx = q * 8 + e * 2;
            const int c = tn * NT + cb * 32 + jx;
            float v0 = __fadd_rn(__fmul_rn(s_a2[c], __fadd_rn(__uint_as_float(pp[e * 2]), __uint_as_float(r[jx]))), s_b2[c]);
            float v1 = __fadd_rn(__fmul_rn(s_a2[c + 1], __fadd_rn(__uint_as_float(pp[e * 2 + 1]), __uint_as_float(r[jx + 1]))), s_b2[c + 1]);
            if (L.relu) { v0 = v0 > 0.f ? v0 : 0.f; v1 = v1 > 0.f ? v1 : 0.f; }
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
            const uint32_t nv = *(const uint32_t*)&h2;
            const uint32_t sel = (((bits >> (e * 2)) & 1u) ? 0x0000ffffu : 0u) | (((bits >> (e * 2 + 1)) & 1u) ? 0xffff0000u : 0u);
            cw[e] = (cw[e] & ~sel) | (nv & sel);
          }
          *slot = cur;
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&sh->acc_free);
      ++items_done;
    }
    if (threadIdx.x == 192 && ok && items_done)
      atomicAdd(&prm.counters[CNT_EXEC_MACS], items_done * (unsigned long long)kBM * NT * taps * L.c_r);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, NT);
}

// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault,
                                         &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

bool encode(CUtensorMap* map, int elem_bytes, void* base, int rank, const cuuint64_t* dims,
            const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return fn(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, base, dims, strides_bytes, box,
            es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr int kMaxDevices = 64;

int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

int sm_count(int dev) {
  static int sms[kMaxDevices] = {};
  if (sms[dev] == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    sms[dev] = v;
  }
  return sms[dev];
}

}  // namespace

bool tc_plan(const LayerDims& L_in, int in_dtype, int cond_mode, TcPlan* plan) {
  TcPlan P;
  std::memset(&P, 0, sizeof(P));
  *plan = P;
  // Base slices of 8 channels (bf16) are half a K step: the layer is planned, and later run, as one
  // with 16 base channels and a conditional path over all input channels (weights repacked).
  LayerDims L = L_in;
  if (in_dtype == CG_BF16 && L.c_p == 8 && L.c_r > 0 && !L.grouping) {
    if (cond_mode == CG_COND_COMPACT) return false;
    L.c_p = 16; L.c_r = L.c_in; P.pad8 = 1;
  }
  // int8 layers with 64 input channels: a pixel is half a 128-byte patch row.  The copies of x
  // fill the upper half with zeros (out-of-bounds elements of the tensor map), and the weights
  // are repacked as for 8-channel slices: 32 base channels per tap (zeros behind the real ones), a
  // conditional path over the 64 real channels (zeros in front of the real ones), two taps per
  // weight tile.
  if (in_dtype == CG_I8 && L.c_in == 64 && L.c_p <= 32 && L.c_r > 0 && !L.grouping) {
    if (cond_mode == CG_COND_COMPACT) return false;
    L.c_in = 128; L.c_p = 32; L.c_r = 64; P.pad8 = 2;
  }
  if (in_dtype != CG_BF16 && in_dtype != CG_I8) return false;
  const int eb = in_dtype == CG_BF16 ? 2 : 1;
  const int ck = 128 / eb;          // channels per 128-byte patch row
  const int kst = ck / 4;           // channels per MMA K step (32 bytes)
  // channel grouping: whole 128-byte chunks per group, column tiles inside one output group
  if (L.grouping && (in_dtype != CG_BF16 || L.c_p % ck != 0 || (L.c_out / L.groups) % 64 != 0 || cond_mode == CG_COND_COMPACT)) return false;
  if (L.has_residual && in_dtype != CG_BF16) return false;
  if (L.kh != L.kw || L.kh != 2 * L.pad + 1) return false;
  const bool s2 = L.stride == 2;
  if (L.stride != 1 && !s2) return false;
  // stride 2: 3x3 kernels over even extents; the patch is four sub-images of the input
  if (s2 && (L.kh != 3 || (L.h & 1) || (L.w & 1))) return false;
  if (L.c_in % ck != 0) return false;
  if (!(L.c_p == kst || L.c_p == 2 * kst || L.c_p % ck == 0)) return false;
  if (L.c_out % 64 != 0) return false;   // (int8: the last 128-channel tile may be half empty)
  const int xpad = s2 ? 1 : L.pad;                  // zero columns/rows shared between patch rows
  if (L.wo + xpad > kBM) return false;
  P.elem_bytes = eb;
  P.ck = ck;
  P.planes = s2 ? 4 : 1;
  P.wp = L.wo + xpad;
  P.ip = (L.ho + xpad) * P.wp;
  // rows of one image that fit 128 patch rows; or whole images if at least two fit
  const int last_valid_one_image = (L.ho - 1) * P.wp + L.wo - 1;
  if (last_valid_one_image + P.ip <= kBM - 1) {
    P.images_mode = 1;
    P.ni = 1 + (kBM - 1 - last_valid_one_image) / P.ip;
    P.r = L.ho;
    P.tiles_per_image = 1;
    P.tiles_m = (L.n + P.ni - 1) / P.ni;
    P.box_h = L.ho + xpad;
    P.out_box_h = L.ho + xpad;
  } else {
    P.images_mode = 0;
    P.ni = 1;
    const int rmax = kBM / P.wp;
    const int tiles = (L.ho + rmax - 1) / rmax;
    P.r = (L.ho + tiles - 1) / tiles;
    P.tiles_per_image = tiles;
    P.tiles_m = L.n * tiles;
    P.box_h = s2 ? P.r + 1 : P.r + 2 * L.pad;
    P.out_box_h = P.r;
  }
  if (P.box_h > 256 || P.wp > 256 || P.ni > 256) return false;
  P.box_pixels = P.wp * P.box_h * P.ni;
  P.patch_rows = (int)align_up((size_t)kBM + (size_t)(s2 ? 1 : L.kh - 1) * (P.wp + 1), 8);
  if (P.box_pixels > P.patch_rows) P.patch_rows = (int)align_up(P.box_pixels, 8);
  P.patch_bytes = (int)align_up((size_t)P.patch_rows * 128, 1024);
  P.chunks = L.c_in / ck;
  P.base_chunks = L.c_p >= ck ? L.c_p / ck : 1;
  const int taps = L.kh * L.kw;
  if (L.c_p >= ck) {
    P.base_tiles = (L.c_p / ck) * taps;
    P.cond_tiles = (P.chunks - L.c_p / ck) * taps;
  } else {
    const int tpt = ck / L.c_p;
    P.base_tiles = (taps + tpt - 1) / tpt;
    P.cond_tiles = L.c_r > 0 ? P.chunks * taps : 0;
    if (P.pad8 == 2) P.cond_tiles = (taps + 1) / 2;
  }
  P.stage_rows = (int)align_up((size_t)max(kBM, P.wp * P.out_box_h * P.ni), 8);
  P.cond_mode = cond_mode == CG_COND_AUTO ? CG_COND_SKIP_TILES : cond_mode;
  // row compaction: bf16 layers with a conditional path and no residual input; otherwise block
  // skipping
  if (P.cond_mode == CG_COND_COMPACT && (eb != 2 || L.c_r == 0 || L.has_residual)) P.cond_mode = CG_COND_SKIP_TILES;
  if (P.base_tiles + P.cond_tiles > kMaxWTiles) return false;
  // shared-memory layout: [weights: resident tiles or ring][patch ring][y staging][consts]
  // [mask stash][tile coordinates][barriers].  First choice: a column tile whose weights stay
  // resident next to at least two patch buffers (no weight traffic per job, which otherwise
  // bounds the layer at the per-SM L2 ingest rate); else the widest tile with streamed weights.
  const size_t limit = 227 * 1024 - 1024;
  for (int pass = 0; pass < 2; ++pass)
  for (int nt = 128; nt >= (eb == 1 ? 128 : 64); nt >>= 1) {
    if (L.c_out % nt != 0 && eb != 1) continue;
    if (L.grouping && (L.c_out / L.groups) % nt != 0) continue;
    const size_t fixed = align_up((size_t)(nt * eb / 128) * P.stage_rows * 128, 1024) +
                         align_up((size_t)8 * nt * 4, 128) +
                         align_up((size_t)4 * 128 * (nt / 32) * 4, 128) +
                         align_up((size_t)kMaxWTiles * 4, 128) + align_up(sizeof(Shared), 128);
    const size_t w_tile = (size_t)nt * 128;
    const size_t w_all = (size_t)(P.base_tiles + P.cond_tiles) * w_tile;
    int na = 0, nb = 0, resident = 0;
    const int na_min = 2 * P.planes, na_max = 4 * P.planes > 8 ? 8 : 4 * P.planes;
    if (fixed + w_all + (size_t)na_min * P.patch_bytes <= limit) {
      resident = 1;
      na = (int)((limit - fixed - w_all) / P.patch_bytes);
      if (na > na_max) na = na_max;
    } else if (pass == 0) {
      continue;
    } else {
      // streamed weights are latency-bound (bytes in flight per SM), so the weight ring gets
      // the shared memory that three patch buffers (stride 1) or one set of planes leave
      // (nb counts ring stages of kStageTiles tiles: three stages if they fit, else two)
      bool found = false;
      for (int na_want = P.planes == 1 ? 3 : P.planes; na_want >= (P.planes == 1 ? 2 : P.planes) && !found; --na_want) {
        for (nb = 3; nb >= 2; --nb) {
          const size_t ring = (size_t)nb * kStageTiles * w_tile;
          if (fixed + ring + (size_t)na_want * P.patch_bytes > limit) continue;
          na = (int)((limit - fixed - ring) / P.patch_bytes);
          if (na > na_max) na = na_max;
          found = true;
          break;
        }
      }
      if (!found) continue;
    }
    // the four planes of a stride-2 chunk occupy four consecutive ring slots
    if (P.planes == 4) na = na / 4 * 4;
    if (na < P.planes) continue;
    size_t off = 0;
    P.off_b = (unsigned)off; off += resident ? w_all : (size_t)nb * kStageTiles * w_tile;
    P.off_a = (unsigned)off; off += (size_t)na * P.patch_bytes;
    P.off_y = (unsigned)off; off += align_up((size_t)(nt * eb / 128) * P.stage_rows * 128, 1024);
    P.off_consts = (unsigned)off; off += align_up((size_t)8 * nt * 4, 128);
    P.off_mask = (unsigned)off; off += align_up((size_t)4 * 128 * (nt / 32) * 4, 128);
    P.off_tables = (unsigned)off; off += align_up((size_t)kMaxWTiles * 4, 128);
    P.off_bar = (unsigned)off; off += align_up(sizeof(Shared), 128);
    P.nt = nt; P.na = na; P.nb = nb; P.resident = resident; P.tiles_n = (L.c_out + nt - 1) / nt;
    // resident weights: the base and the conditional path get their own MMA issuer and their own
    // half of the patch ring
    const bool two = resident && P.cond_tiles > 0 && P.cond_mode != CG_COND_COMPACT;
    // (three issuers only at NT = 64: with a single R accumulator two conditional issuers would
    // alternate on one r_free/cond_done barrier pair and could run a whole phase apart)
    P.share_a = (two && P.chunks == 1 && P.planes == 1 && nt == 64) ? 1 : 0;
    P.split_a = (two && !P.share_a && na >= 2 * P.planes && (na / 2) % P.planes == 0) ? na / 2 : 0;
    P.issuers = P.share_a ? 3 : (P.split_a ? 2 : 1);
    P.smem_bytes = (unsigned)(off + 1024);
    P.valid = 1;
    *plan = P;
    return true;
  }
  return false;
}

bool tc_device_ok(int device) {
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return false;
  return prop.major == 10 && encode_tiled_fn() != nullptr;
}

// CG_COND_COMPACT workspace: [row counts, 256 B][row lists: tiles_n x M x u32][row records:
// tiles_n x M x (NT + 4) words]
// int8 weights of a layer with 64 input channels, repacked with whole K steps (see tc_plan):
// W_base [rows][c_p] -> [rows][32], W_cond [rows][64 - c_p] -> [rows][64] with the real channels at
// their input-channel positions [c_p, 64) of 64; everything else zero.  rows = c_out * taps.
__global__ void repack_i8_kernel(const int8_t* __restrict__ wb, const int8_t* __restrict__ wc, int8_t* __restrict__ wb32,
                                 int8_t* __restrict__ wc64, int rows, int c_p) {
  const int total = rows * 96;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int row = i / 96, c = i - row * 96;
    if (c < 32) {
      wb32[(size_t)row * 32 + c] = c < c_p ? wb[(size_t)row * c_p + c] : (int8_t)0;
    } else {
      const int cc = c - 32;
      wc64[(size_t)row * 64 + cc] = cc >= c_p ? wc[(size_t)row * (64 - c_p) + cc - c_p] : (int8_t)0;
    }
  }
}

static size_t repack_i8_bytes(const LayerDims& L) {
  const size_t rows = (size_t)L.c_out * L.kh * L.kw;
  return align_up(rows * 32, 256) + align_up(rows * 64, 256);
}

size_t tc_workspace_bytes(const LayerDims& L, const TcPlan& P) {
  if (P.valid && P.pad8 == 2) return repack_i8_bytes(L);
  if (P.valid && P.pad8) return repack8_bytes(L);
  if (!P.valid || P.cond_mode != CG_COND_COMPACT) return 0;
  const size_t rows = (size_t)P.tiles_n * (size_t)L.m;
  return 256 + align_up(rows * 4, 256) + rows * (size_t)(P.nt + 4) * 4;
}

int launch_tc(const LayerDims& L_in, const TcPlan& P, int in_dtype, TcMaps* maps, const void* x,
              const void* w_base, const void* w_cond, const cg_bn_params& bn, const float* delta,
              const void* residual, void* y, uint32_t* mask, void* workspace,
              unsigned long long* counters, cudaStream_t stream, const float* t_img, int base_only) {
  (void)in_dtype;
  if (!P.valid) return (int)cudaErrorInvalidValue;
  LayerDims L = L_in;
  if (P.pad8 == 2) {
    if (!workspace) return (int)cudaErrorInvalidValue;
    const size_t rows = (size_t)L_in.c_out * L_in.kh * L_in.kw;
    int8_t* b = static_cast<int8_t*>(workspace);
    int8_t* c = b + align_up(rows * 32, 256);
    repack_i8_kernel<<<64, 256, 0, stream>>>(static_cast<const int8_t*>(w_base), static_cast<const int8_t*>(w_cond), b, c,
                                             (int)rows, L_in.c_p);
    if (cudaGetLastError() != cudaSuccess) return (int)cudaErrorLaunchFailure;
    w_base = b; w_cond = c;
    L.c_in = 128; L.c_p = 32; L.c_r = 64;
  } else if (P.pad8) {
    if (!workspace) return (int)cudaErrorInvalidValue;
    const int e = launch_repack8(L_in, w_base, w_cond, workspace, &w_base, &w_cond, stream);
    if (e != 0) return e;
    L.c_p = 16; L.c_r = L.c_in;
  }
  const void* wc_key = w_cond ? w_cond : w_base;
  TcMapSet* ms = nullptr;
  for (int i = 0; i < TcMaps::kEntries; ++i) {
    TcMapSet* c = &maps->set[i];
    if (c->key[0] == x && c->key[1] == w_base && c->key[2] == wc_key && c->key[3] == y) { ms = c; break; }
  }
  if (!ms) {
    ms = &maps->set[maps->next];
    maps->next = (maps->next + 1) % TcMaps::kEntries;
    ms->key[0] = nullptr;
    const int taps = L.kh * L.kw;
    const cuuint64_t eb = (cuuint64_t)P.elem_bytes;
    const cuuint32_t ck = (cuuint32_t)P.ck;
    if (L.stride == 1) {
      const cuuint64_t cx = (cuuint64_t)L_in.c_in;   // (the tensor's own channel count: a box may reach past it)
      cuuint64_t dims[4] = {cx, (cuuint64_t)L.w, (cuuint64_t)L.h, (cuuint64_t)L.n};
      cuuint64_t str[3] = {cx * eb, (cuuint64_t)L.w * cx * eb, (cuuint64_t)L.h * L.w * cx * eb};
      cuuint32_t box[4] = {ck, (cuuint32_t)P.wp, (cuuint32_t)P.box_h, (cuuint32_t)P.ni};
      if (!encode(&ms->x[0], P.elem_bytes, const_cast<void*>(x), 4, dims, str, box)) return (int)cudaErrorInvalidValue;
      ms->x[1] = ms->x[2] = ms->x[3] = ms->x[0];
    } else {
      // plane 2*ph + pw holds the input pixels (2a + ph, 2b + pw)
      for (int pl = 0; pl < 4; ++pl) {
        const int ph = pl >> 1, pw = pl & 1;
        const cuuint64_t cx = (cuuint64_t)L_in.c_in;
        const char* base = static_cast<const char*>(x) + ((size_t)ph * L.w + pw) * cx * eb;
        cuuint64_t dims[4] = {cx, (cuuint64_t)L.w / 2, (cuuint64_t)L.h / 2, (cuuint64_t)L.n};
        cuuint64_t str[3] = {(cuuint64_t)2 * cx * eb, (cuuint64_t)2 * L.w * cx * eb, (cuuint64_t)L.h * L.w * cx * eb};
        cuuint32_t box[4] = {ck, (cuuint32_t)P.wp, (cuuint32_t)P.box_h, (cuuint32_t)P.ni};
        if (!encode(&ms->x[pl], P.elem_bytes, const_cast<char*>(base), 4, dims, str, box)) return (int)cudaErrorInvalidValue;
      }
    }
    {
      cuuint64_t dims[2] = {(cuuint64_t)taps * L.c_p, (cuuint64_t)L.c_out};
      cuuint64_t str[1] = {(cuuint64_t)taps * L.c_p * eb};
      cuuint32_t box[2] = {ck, (cuuint32_t)P.nt};
      if (!encode(&ms->wb, P.elem_bytes, const_cast<void*>(w_base), 2, dims, str, box)) return (int)cudaErrorInvalidValue;
    }
    if (L.c_r > 0) {
      cuuint64_t dims[2] = {(cuuint64_t)taps * L.c_r, (cuuint64_t)L.c_out};
      cuuint64_t str[1] = {(cuuint64_t)taps * L.c_r * eb};
      cuuint32_t box[2] = {ck, (cuuint32_t)P.nt};
      if (!encode(&ms->wc, P.elem_bytes, const_cast<void*>(w_cond), 2, dims, str, box)) return (int)cudaErrorInvalidValue;
    } else {
      ms->wc = ms->wb;
    }
    {
      cuuint64_t dims[4] = {(cuuint64_t)L.c_out, (cuuint64_t)L.wo, (cuuint64_t)L.ho, (cuuint64_t)L.n};
      cuuint64_t str[3] = {(cuuint64_t)L.c_out * eb, (cuuint64_t)L.wo * L.c_out * eb,
                           (cuuint64_t)L.ho * L.wo * L.c_out * eb};
      cuuint32_t box[4] = {ck, (cuuint32_t)P.wp, (cuuint32_t)P.out_box_h, (cuuint32_t)P.ni};
      if (!encode(&ms->y, P.elem_bytes, y, 4, dims, str, box)) return (int)cudaErrorInvalidValue;
    }
    ms->key[0] = x; ms->key[1] = w_base; ms->key[2] = wc_key; ms->key[3] = y;
  }
  TcParams prm;
  prm.L = L; prm.P = P; prm.bn = bn; prm.delta = delta; prm.residual = (const __nv_bfloat16*)residual; prm.mask = mask; prm.counters = counters;
  prm.ws_counts = nullptr; prm.ws_list = nullptr; prm.ws_rows = nullptr;
  prm.t_img = t_img; prm.base_only = base_only;
  const bool compact = P.cond_mode == CG_COND_COMPACT;
  if (compact) {
    if (!workspace) return (int)cudaErrorInvalidValue;
    const size_t rows = (size_t)P.tiles_n * (size_t)L.m;
    char* ws = static_cast<char*>(workspace);
    prm.ws_counts = reinterpret_cast<uint32_t*>(ws);
    prm.ws_list = reinterpret_cast<uint32_t*>(ws + 256);
    prm.ws_rows = reinterpret_cast<uint32_t*>(ws + 256 + align_up(rows * 4, 256));
    const cudaError_t e = cudaMemsetAsync(prm.ws_counts, 0, 256, stream);
    if (e != cudaSuccess) return (int)e;
  }
  // persistent grid: one CTA per SM, a multiple of the number of column tiles
  const int dev = current_device();
  if (dev < 0) return (int)cudaErrorInvalidDevice;
  const int sms = sm_count(dev);
  int grid = sms - sms % P.tiles_n;
  if (grid < P.tiles_n) grid = P.tiles_n;
  if (grid > P.tiles_m * P.tiles_n) grid = P.tiles_m * P.tiles_n;
  // kernel instances: <64, bf16>, <128, bf16>, <128, int8>
  typedef void (*Kernel)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap,
                         CUtensorMap, TcParams);
  const int which = P.elem_bytes == 1 ? 2 : (P.nt == 128 ? 1 : 0);
  const Kernel kernels[3] = {tc_gated_conv_kernel<64, false>, tc_gated_conv_kernel<128, false>,
                             tc_gated_conv_kernel<128, true>};
  static bool attr_set[kMaxDevices][3] = {};   // (the attribute is per device)
  if (!attr_set[dev][which]) {
    const cudaError_t e = cudaFuncSetAttribute(kernels[which], cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               227 * 1024);
    if (e != cudaSuccess) return (int)e;
    attr_set[dev][which] = true;
  }
  // Every layer asks for the same (maximum) amount of dynamic shared memory: consecutive layer
  // kernels then never differ in the SM's shared-memory configuration.  The launch is a
  // programmatic dependent launch: the CTAs of this kernel may start while the last CTAs of the
  // previous kernel in the stream still run; they set up their barriers and TMEM and then wait
  // (griddepcontrol.wait) for that kernel to finish before they touch global memory.
  {
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3((unsigned)kThreads, 1, 1);
    cfg.dynamicSmemBytes = 227 * 1024;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernels[which], ms->x[0], ms->x[1], ms->x[2], ms->x[3], ms->wb,
                                             ms->wc, ms->y, prm);
    if (e != cudaSuccess) return (int)e;
  }
  if (compact) {
    // second kernel: gathered conditional path over the listed rows
    CpParams cp;
    cp.L = L; cp.P = P; cp.bn = bn; cp.delta = delta;
    cp.x = static_cast<const __nv_bfloat16*>(x); cp.y = static_cast<__nv_bfloat16*>(y);
    cp.ws_counts = prm.ws_counts; cp.ws_list = prm.ws_list; cp.ws_rows = prm.ws_rows;
    cp.counters = counters;
    const size_t smem2 = (size_t)kCpStages * (128 * 128 + (size_t)P.nt * 128) + (size_t)2 * L.c_out * 4 +
                         sizeof(CpShared) + 2048;
    long long items = (long long)P.tiles_n * ((L.m + 127) / 128);
    const int grid2 = (int)(items < sms ? items : sms);
    typedef void (*Kernel2)(CUtensorMap, CpParams);
    const Kernel2 k2 = P.nt == 128 ? (Kernel2)tc_compact_cond_kernel<128> : (Kernel2)tc_compact_cond_kernel<64>;
    static bool attr2[kMaxDevices][2] = {};
    if (!attr2[dev][P.nt == 128]) {
      const cudaError_t e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
      if (e != cudaSuccess) return (int)e;
      attr2[dev][P.nt == 128] = true;
    }
    k2<<<grid2, kCpThreads, smem2, stream>>>(ms->wc, cp);
  }
  return (int)cudaGetLastError();
}

#ifdef CG_PROF
// Profiling build only: copies the wait-cycle table to the host and clears it.
extern "C" int cg_prof_read(unsigned long long* host_out) {
  cudaError_t e = cudaMemcpyFromSymbol(host_out, g_prof, sizeof(g_prof));
  if (e != cudaSuccess) return (int)e;
  static unsigned long long zeros[25 * 32];
  return (int)cudaMemcpyToSymbol(g_prof, zeros, sizeof(g_prof));
}
extern "C" int cg_prof_timeline(unsigned long long* host_out) {
  return (int)cudaMemcpyFromSymbol(host_out, g_tl, sizeof(g_tl));
}
#endif

}  // namespace cg
