// Channel-gated convolution on tcgen05 tensor cores, channel-major accumulators.
//
// GEMM view of one job: D[channel, pixel] = sum_k W[channel, k] * X[pixel, k] with the 128
// output channels of the CTA's channel tile on the MMA's M side (TMEM lanes) and up to 256
// output pixels on its N side (TMEM columns): N = 256 instructions run the tensor pipe at its
// full rate while leaving a quarter of the shared-memory bandwidth to the copies that refill
// the operands (an M = 128 x N = 128 instruction takes all of it).
//
// Pixels live in a "stacked" padded space: image rows of all images one after another with
// pitch W+pad, `pad` zero rows after every image.  The right padding of a row is the left
// padding of the next, the bottom padding of an image the top padding of the next, so filter
// tap (r,s) of output position q reads position q + r*(W+pad) + s of the patch: every tap is
// the same shared-memory patch read from another start row (Section 3.1's two convolutions as
// shifted-window implicit GEMMs).  A pixel sub-tile is `r` whole stacked rows; its patch (the
// rows around it, 64 input channels per 128-byte row, 128-byte swizzle) is loaded by one TMA
// box per stacked row; out-of-bounds fill supplies every zero.
//
// Per job (channel tile x two pixel sub-tiles a, b), following the paper's block:
//   1. base path   P = W_p * x_p            K stages [0, nb), fp32 accumulator in TMEM;
//   2. gate        d = (P >= t[c])          epilogue warps read P from TMEM; thread = channel,
//                                           so t, a1, b1, a2, b2 sit in registers; the warp
//                                           ballot of 32 channels is the mask word (Eq. 2, 3);
//                  f(a1*P + b1) is kept in registers as bf16 (Eq. 1, first case);
//   3. conditional R = W_r * x_r            K stages [nb, ns) accumulate ONTO P in the same
//                                           TMEM columns, skipped for a sub-tile in which no gate
//                                           fired;
//   4. combine     y = d ? f(a2*(P+R) + b2) : kept value, stored straight from registers
//                                           (Eq. 1, Section 4's two batch norms).
// Weights stream through a ring of 64-K stages; each stage is used by both sub-tiles, a running
// `lead` stages ahead of b, so that the gate and combine passes of one sub-tile overlap the
// MMAs of the other and the tensor pipe never waits for the epilogue.
//
// Warps: 0 patch producer, 1 MMA issuer (owns TMEM), 2 weight producer, 3 idle, 4-19 epilogue
// (TMEM lane quadrant x quarter of the pixels).  Every mbarrier wait is bounded; a wait that
// expires records CG_ERR_DEVICE_TIMEOUT and the id of the wait, raises a CTA-wide flag that
// makes every role leave its loop, and the CTA idles for a fixed time before it frees TMEM so
// that copies and MMAs in flight have finished.  No barrier other than the final
// __syncthreads is shared between roles, so a role that gives up cannot strand another.
#include <cstring>

#include "ptx.cuh"
#include "tc2_conv.cuh"

namespace cg {

namespace {

constexpr int kThreads2 = 640;
constexpr int kEpiWarp0 = 4;
constexpr int kEpiWarps = 16;
constexpr int kPatchEntries = 3;                  // at most; a plan may use two
constexpr int kMaxRing = 12;
constexpr int kMaxBoxes = 32;
constexpr int kSpinLimit2 = 1 << 21;
constexpr long long kWaitCycles2 = 2000000000ll;
constexpr long long kDrainCycles = 4000000ll;     // ~2 ms: longest copy/MMA in flight is microseconds

struct Tc2Params {
  LayerDims L;
  cg_bn_params bn;
  const float* delta;
  const __nv_bfloat16* residual;
  __nv_bfloat16* y;
  uint32_t* mask;
  unsigned long long* counters;
  Tc2Plan P;
};

struct Shared2 {
  uint64_t w_full[kMaxRing], w_empty[kMaxRing];
  uint64_t p_full[kPatchEntries], p_empty[kPatchEntries];
  uint64_t tmem_free[2], base_done[2], p_read[2], cond_done[2];
  uint64_t a_ahead;               // sub-tile a has issued its first `lead` stages of the job
  uint32_t tmem_base;
  uint32_t abort_flag;
  uint32_t fired[2][kEpiWarps];   // per sub-tile, per epilogue warp: a gate of a valid pixel fired
  float t2[128];                  // upper thresholds of the two-sided gate (Section 3.2) of the channel tile
  // copies that make up the patch being loaded: {shared-memory offset, h, n, tensor map}
  uint32_t box_dst[kMaxBoxes];
  int box_h[kMaxBoxes], box_n[kMaxBoxes], box_map[kMaxBoxes];
};

struct Ctx2 {
  Shared2* sh;
  unsigned long long* counters;
};

// A wait ran out: record the error and where, and make every role of the CTA leave its loop.
__device__ __noinline__ void give_up2(Shared2* sh, unsigned long long* counters, int site) {
  if (atomicCAS(&counters[CNT_STATUS], 0ull, (unsigned long long)CG_ERR_DEVICE_TIMEOUT) == 0ull)
    atomicExch(&counters[CNT_SITE], (unsigned long long)site);
  atomicExch(&sh->abort_flag, 1u);
}

__device__ __noinline__ bool wait2_slow(Shared2* sh, unsigned long long* counters, uint64_t* bar,
                                        uint32_t parity, int site) {
  const long long t0 = clock64();
  for (int i = 0; i < kSpinLimit2; ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 15) == 15) {
      if (*(volatile uint32_t*)&sh->abort_flag) return false;
      if (clock64() - t0 > kWaitCycles2) break;
    }
  }
  give_up2(sh, counters, site);
  return false;
}

__device__ __forceinline__ bool wait2(const Ctx2& cx, uint64_t* bar, uint32_t parity, int site) {
  if (ptx::mbar_try_wait(bar, parity, 0u)) return true;
  return wait2_slow(cx.sh, cx.counters, bar, parity, site);
}

template <int N>
__device__ __forceinline__ void set_max_regs_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void set_max_regs_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// Folded per-channel constants of the four channels an epilogue thread sees in the fragment
// layout: channels ch0 + 8*ci + lane/4, ci = 0..3, of the warp's 32.
struct Consts4 {
  float kt[4], ka1[4], kb1[4], ka2[4], kb2[4];
};

// What an epilogue thread keeps of a sub-tile between its gate pass and its combine pass.  Lane l
// of 32-lane group g stands for pixel l%16 of the warp's piece 2g + l/16.
struct Keep {
  uint32_t off[2];       // [g] output pixel index m of this lane's column, ~0u if padding
  uint32_t fired;        // a gate fired in one of the warp's pieces
};

constexpr int kTilePitch = 80;                    // bytes per pixel row of a warp's staging tile (64 + 16: no bank conflicts)
constexpr int kEpiTileBytes = 16 * kTilePitch;    // 16 pixels x 32 channels of bf16
constexpr uint32_t kOpen = 0xffffu;               // bf16 pattern that marks "gate open" in y between the two passes:
                                                  // a negative NaN, which max(v, lo) never yields

// Output pixel index of this lane's column for both 32-lane groups (~0u: a pad position).
__device__ __forceinline__ void pixel_offsets(const LayerDims& L, const Tc2Plan& P, int gx, int pg, int lane, Keep& kp) {
  const int pieces = P.nmma >> 4;
#pragma unroll
  for (int g = 0; g < 2; ++g) {
    const int pc = pg + 4 * (2 * g + (lane >> 4));
    const int j = pc * 16 + (lane & 15);
    uint32_t off = ~0u;
    if (pc < pieces && j < P.np) {
      // (exact for these small non-negative integers: the quotient of (x + 0.5) / d never sits
      // within 2^-12 of an integer)
      const int dj = (int)(((float)j + 0.5f) * P.inv_wp);
      const int gr = gx + dj, w = j - dj * P.wp;
      const int n = (int)(((float)gr + 0.5f) * P.inv_hp), h = gr - n * P.hp;
      if (w < L.wo && h < L.ho && n < L.n) off = (uint32_t)((n * L.ho + h) * L.wo + w);
    }
    kp.off[g] = off;
  }
}

// The warp's 16 pixels x 32 channels, as packed bf16 pairs pk[ci][octet] in the fragment layout
// of the 16x256b TMEM load, go into the staging tile pixel-major: afterwards lane l finds eight
// consecutive channels of a pixel (16 bytes) at vector_at(l) and vector_at(l + 32).
__device__ __forceinline__ void transpose_piece(const uint32_t (&pk)[4][2], uint8_t* s_tile, int lane) {
  // thread 8*i + j gives the address of pixel row j, channels 8*i..8*i+7
  const uint32_t row_addr = ptx::smem_u32(s_tile + (lane & 7) * kTilePitch + (lane >> 3) * 16);
  ptx::stmatrix_x4_trans(row_addr, pk[0][0], pk[1][0], pk[2][0], pk[3][0]);
  ptx::stmatrix_x4_trans(row_addr + 8 * kTilePitch, pk[0][1], pk[1][1], pk[2][1], pk[3][1]);
  __syncwarp();
}
__device__ __forceinline__ uint4 vector_at(const uint8_t* s_tile, int vidx) {   // pixel vidx/4, channels 8*(vidx%4)..
  return *(const uint4*)(s_tile + (vidx >> 2) * kTilePitch + (vidx & 3) * 16);
}
// per 16-bit half: 0xffff where the half of v is the "gate open" mark, else 0
__device__ __forceinline__ uint32_t open_halves(uint32_t v) { return __vcmpeq2(v, 0xffffffffu); }

// Gate pass of one warp over its pieces of a sub-tile (Eq. 2, 3 and Eq. 1's first case):
// d = (P >= t).  Where d = 0 the output f(a1*P + b1) is final; where d = 1 the "gate open" mark
// is written in its place.  A piece goes through the staging tile to y as 16-byte vectors, and
// the lane that stores a vector reads the eight decisions off it for the pixel's mask word.
// (kTwoSided: the gate of Section 3.2 with upper thresholds t2[4], read from shared memory per
// pass so that the plain gate neither keeps them in registers nor compares against them)
template <bool kHasRes, bool kTwoSided>
__device__ __forceinline__ void gate_pass(const Tc2Params& prm, Keep& kp, const Consts4& kc, const float* s_t2, uint32_t t_acc,
                                          int gx, int pg, int lane, int word_idx, float lo, __nv_bfloat16* y_q,
                                          const __nv_bfloat16* res_q, uint8_t* s_tile, unsigned long long& st_active,
                                          unsigned long long& st_words, unsigned long long& st_words_on) {
  const LayerDims& L = prm.L;
  const Tc2Plan& P = prm.P;
  const int pieces = P.nmma >> 4;
  pixel_offsets(L, P, gx, pg, lane, kp);
  float t2[4] = {0.f, 0.f, 0.f, 0.f};
  if (kTwoSided) {
#pragma unroll
    for (int ci = 0; ci < 4; ++ci) t2[ci] = s_t2[8 * ci + (lane >> 2)];
  }
  bool fired = false;
#pragma unroll 1
  for (int q = 0; q < 4; ++q) {
    const int piece = pg + 4 * q;
    if (piece >= pieces) break;                              // (uniform over the warp)
    const int slot0 = (q & 1) * 16;
    const uint32_t offs = (q >> 1) ? kp.off[1] : kp.off[0];
    uint32_t r0[8], r1[8];                                   // channels 0-15 / 16-31 of the quadrant
    ptx::tmem_ld_frag16(t_acc + (uint32_t)(piece * 16), r0);
    ptx::tmem_ld_frag16(t_acc + (16u << 16) + (uint32_t)(piece * 16), r1);
    ptx::tmem_ld_wait16(r0, r1);
    uint32_t pk[4][2];
#pragma unroll
    for (int ci = 0; ci < 4; ++ci) {
#pragma unroll
      for (int oct = 0; oct < 2; ++oct) {
        float yv[2];
        bool d[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float a = __uint_as_float((ci >> 1) ? r1[4 * oct + 2 * (ci & 1) + e] : r0[4 * oct + 2 * (ci & 1) + e]);
          d[e] = a >= kc.kt[ci];                             // Eq. 2: a tie fires, NaN does not
          if (kTwoSided) d[e] = d[e] && a <= t2[ci];         // Section 3.2: and stays below the upper threshold
          float v = fmaf(kc.ka1[ci], a, kc.kb1[ci]);         // BN1 of the partial sum (Section 4)
          if (kHasRes) {
            const uint32_t oj = __shfl_sync(0xffffffffu, offs, slot0 + 8 * oct + 2 * (lane & 3) + e);
            if (oj != ~0u) v += __bfloat162float(res_q[(size_t)oj * L.c_out + 8 * ci + (lane >> 2)]);
          }
          yv[e] = fmaxf(v, lo);
        }
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(yv[0], yv[1]);
        uint32_t w = *(const uint32_t*)&h2;
        if (d[0]) w |= kOpen;
        if (d[1]) w |= kOpen << 16;
        pk[ci][oct] = w;
      }
    }
    transpose_piece(pk, s_tile, lane);
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int vidx = lane + 32 * k;
      const uint32_t oj = __shfl_sync(0xffffffffu, offs, slot0 + (vidx >> 2));
      const uint4 val = vector_at(s_tile, vidx);
      // decisions of the vector's eight channels, one bit each
      const uint32_t t = (open_halves(val.x) & 0x00020001u) | (open_halves(val.y) & 0x00080004u) |
                         (open_halves(val.z) & 0x00200010u) | (open_halves(val.w) & 0x00800040u);
      uint32_t word = ((t | (t >> 16)) & 0xffu) << (8 * (lane & 3));
      word |= __shfl_xor_sync(0xffffffffu, word, 1);
      word |= __shfl_xor_sync(0xffffffffu, word, 2);
      if (oj != ~0u) {
        *(uint4*)(y_q + (size_t)oj * L.c_out + (vidx & 3) * 8) = val;
        if ((lane & 3) == 0) {
          if (prm.mask) prm.mask[(size_t)oj * L.words + word_idx] = word;
          st_active += __popc(word);
          st_words += 1;
          if (word) { st_words_on += 1; fired = true; }
        }
      }
    }
    __syncwarp();
  }
  kp.fired = __any_sync(0xffffffffu, fired) ? 1u : 0u;
}

// Combine pass (Eq. 1's second case): f(a2*(P+R) + b2) replaces the "gate open" marks the gate
// pass left in y; vectors without a mark are left alone.  The thread that stores a vector here
// stored the same vector in the gate pass, so it reads back its own write.
template <bool kHasRes>
__device__ __forceinline__ void combine_pass(const Tc2Params& prm, const Keep& kp, const Consts4& kc, uint32_t t_acc,
                                             int pg, int lane, float lo, __nv_bfloat16* y_q,
                                             const __nv_bfloat16* res_q, uint8_t* s_tile) {
  const LayerDims& L = prm.L;
  const Tc2Plan& P = prm.P;
  const int pieces = P.nmma >> 4;
  if (!kp.fired) return;                                     // (uniform over the warp: no mark in its pieces)
#pragma unroll 1
  for (int q = 0; q < 4; ++q) {
    const int piece = pg + 4 * q;
    if (piece >= pieces) break;
    const int slot0 = (q & 1) * 16;
    const uint32_t offs = (q >> 1) ? kp.off[1] : kp.off[0];
    // what the gate pass left, requested first: the loads travel while the new values are made
    uint4 old[2];
    uint4* dst[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int vidx = lane + 32 * k;
      const uint32_t oj = __shfl_sync(0xffffffffu, offs, slot0 + (vidx >> 2));
      dst[k] = oj != ~0u ? (uint4*)(y_q + (size_t)oj * L.c_out + (vidx & 3) * 8) : nullptr;
      old[k] = make_uint4(0u, 0u, 0u, 0u);
      if (dst[k]) old[k] = *dst[k];
    }
    uint32_t r0[8], r1[8];
    ptx::tmem_ld_frag16(t_acc + (uint32_t)(piece * 16), r0);
    ptx::tmem_ld_frag16(t_acc + (16u << 16) + (uint32_t)(piece * 16), r1);
    ptx::tmem_ld_wait16(r0, r1);
    uint32_t pk[4][2];
#pragma unroll
    for (int ci = 0; ci < 4; ++ci) {
#pragma unroll
      for (int oct = 0; oct < 2; ++oct) {
        float yv[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float a = __uint_as_float((ci >> 1) ? r1[4 * oct + 2 * (ci & 1) + e] : r0[4 * oct + 2 * (ci & 1) + e]);
          float v = fmaf(kc.ka2[ci], a, kc.kb2[ci]);         // BN2 of the full sum P + R
          if (kHasRes) {
            const uint32_t oj = __shfl_sync(0xffffffffu, offs, slot0 + 8 * oct + 2 * (lane & 3) + e);
            if (oj != ~0u) v += __bfloat162float(res_q[(size_t)oj * L.c_out + 8 * ci + (lane >> 2)]);
          }
          yv[e] = fmaxf(v, lo);
        }
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(yv[0], yv[1]);
        pk[ci][oct] = *(const uint32_t*)&h2;
      }
    }
    transpose_piece(pk, s_tile, lane);
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const uint4 nw = vector_at(s_tile, lane + 32 * k);
      const uint32_t mx = open_halves(old[k].x), my = open_halves(old[k].y), mz = open_halves(old[k].z),
                     mw = open_halves(old[k].w);
      if (dst[k] && ((mx | my) | (mz | mw))) {
        uint4 out;
        out.x = (nw.x & mx) | (old[k].x & ~mx);
        out.y = (nw.y & my) | (old[k].y & ~my);
        out.z = (nw.z & mz) | (old[k].z & ~mz);
        out.w = (nw.w & mw) | (old[k].w & ~mw);
        *dst[k] = out;
      }
    }
    __syncwarp();
  }
}

template <bool kHasRes>
__global__ void __launch_bounds__(kThreads2, 1)
tc2_gated_conv_kernel(const __grid_constant__ CUtensorMap map_r1,
                      const __grid_constant__ CUtensorMap map_r2,
                      const __grid_constant__ CUtensorMap map_r8,
                      const __grid_constant__ CUtensorMap map_i1,
                      const __grid_constant__ CUtensorMap map_i4,
                      const __grid_constant__ CUtensorMap map_wb,
                      const __grid_constant__ CUtensorMap map_wc,
                      const __grid_constant__ Tc2Params prm) {
  extern __shared__ uint8_t smem_raw[];
  ptx::grid_launch_dependents();
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  const LayerDims& L = prm.L;
  const Tc2Plan& P = prm.P;
  uint8_t* s_w = smem + P.off_w;
  uint8_t* s_p = smem + P.off_p;
  Shared2* sh = (Shared2*)(smem + P.off_bar);
  Tc2Stage* s_tab = (Tc2Stage*)(smem + P.off_tab);         // the job's stages, copied from the parameters
  const Ctx2 cx{sh, prm.counters};
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // jobs of this CTA: a fixed channel tile, every `stride_m`-th pixel tile
  const int tile_c = blockIdx.x % P.tiles_c;
  const int first_m = blockIdx.x / P.tiles_c;
  const int stride_m = gridDim.x / P.tiles_c;
  const int jobs = first_m < P.jobs_m ? (P.jobs_m - first_m + stride_m - 1) / stride_m : 0;
  const int ns = P.ns;
  const bool dense = P.cond_mode == CG_COND_DENSE;
  const int rows_per_job = P.r * P.nsub;

  // ---------------------------------------------------------------- set-up
  if (threadIdx.x == 0) {
    for (int i = 0; i < P.ring; ++i) { ptx::mbar_init(&sh->w_full[i], 1); ptx::mbar_init(&sh->w_empty[i], (uint32_t)P.nsub); }
    for (int i = 0; i < kPatchEntries; ++i) { ptx::mbar_init(&sh->p_full[i], 1); ptx::mbar_init(&sh->p_empty[i], 1); }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&sh->tmem_free[i], kEpiWarps);
      ptx::mbar_init(&sh->base_done[i], 1);
      ptx::mbar_init(&sh->p_read[i], kEpiWarps);
      ptx::mbar_init(&sh->cond_done[i], 1);
    }
    ptx::mbar_init(&sh->a_ahead, 1);
    sh->abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_r1); ptx::prefetch_tensormap(&map_r8); ptx::prefetch_tensormap(&map_wb); ptx::prefetch_tensormap(&map_wc);
  }
  if (warp == 1) ptx::tmem_alloc(&sh->tmem_base, 512);
  if (warp == 2) {
    for (int i = lane; i < P.ns; i += 32) s_tab[i] = P.st[i];
  }
  if (warp >= kEpiWarp0) {
    // the first `pad` pixel rows of every patch buffer stand for the padding in front of the first
    // loaded stacked row; no copy ever writes them
    const int et = threadIdx.x - kEpiWarp0 * 32;
    const int n16 = L.pad * 8;                              // 16-byte pieces per buffer
    for (int i = et; i < P.entries * n16; i += kEpiWarps * 32)
      *(uint4*)(s_p + (size_t)(i / n16) * P.patch_bytes + (size_t)(i % n16) * 16) = make_uint4(0, 0, 0, 0);
    ptx::fence_proxy_async();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  ptx::grid_dependency_wait();   // global memory is touched from here on
  const uint32_t tmem = sh->tmem_base;

  if (warp < kEpiWarp0) {
    if (warp == 0) {
      // ============================================================ patch producer
      // Entries are loaded in the order (job, chunk visit, sub-tile); entry e lives in slot e % 3.
      // A patch is a run of stacked rows; it is cut into whole images (one copy per image, or per
      // four images) and runs of rows inside one image (copies of 8, 2 or 1 rows): issuing a copy
      // costs its thread a few hundred cycles, so lane 0 lists the copies and the lanes issue them
      // side by side.
      if (jobs > 0) {
        const int rows_all = L.n * P.hp;
        const uint32_t row_bytes = (uint32_t)P.wp * 128u;
        int slot = 0;
        uint32_t par = 1;
        bool ok = true;
        for (int jb = 0; jb < jobs && ok; ++jb) {
          const int g0 = (first_m + jb * stride_m) * rows_per_job;
          for (int s = 0; s < ns && ok; ++s) {
            if (!(s_tab[s].flags & kStageNewChunk)) continue;
            int chunk = s_tab[s].chunk;
            if (L.grouping) {
              // Channel grouping (Section 3.3): the channel tile lies inside one output group; its
              // base path reads that group's input chunks, its conditional path the others in
              // ascending order.  The weight tiles keep their K coordinates.
              const int bc = L.c_p >> 6, own0 = (tile_c * 128) / (L.c_out / L.groups) * bc;
              if (s_tab[s].flags & kStageCond) { const int i = chunk - bc; chunk = i < own0 ? i : i + bc; }
              else chunk += own0;
            }
            for (int X = 0; X < P.nsub && ok; ++X) {
              int cnt = 0;
              if (lane == 0) {
                ok = wait2(cx, &sh->p_empty[slot], par, 1);
                if (ok) {
                  int g = g0 + X * P.r - L.pad;
                  const int g_hi = g + P.patch_box_rows;
                  uint32_t dst = 0, tx = 0;
                  while (g < g_hi && cnt < kMaxBoxes) {
                    int rows, map, h, n;
                    if (g < 0 || g >= rows_all) {
                      // outside the batch: rows of zeros (h = H is out of bounds)
                      const int len = g < 0 ? min(-g, g_hi - g) : g_hi - g;
                      rows = len >= 8 ? 8 : (len >= 2 ? 2 : 1);
                      map = rows == 8 ? 2 : (rows == 2 ? 1 : 0); h = L.h; n = 0;
                    } else {
                      n = g / P.hp; h = g - n * P.hp;
                      const int whole = (g_hi - g) / P.hp;
                      if (h == 0 && whole >= 1 && P.use_img) {
                        if (whole >= 4 && n + 4 <= L.n) { rows = 4 * P.hp; map = 4; }
                        else { rows = P.hp; map = 3; }
                      } else {
                        const int len = min(P.hp - h, g_hi - g);
                        rows = len >= 8 ? 8 : (len >= 2 ? 2 : 1);
                        map = rows == 8 ? 2 : (rows == 2 ? 1 : 0);
                      }
                    }
                    sh->box_dst[cnt] = dst; sh->box_h[cnt] = h; sh->box_n[cnt] = n; sh->box_map[cnt] = map;
                    ++cnt;
                    g += rows; dst += (uint32_t)rows * row_bytes; tx += (uint32_t)rows * row_bytes;
                  }
                  if (g < g_hi) ok = false;                  // (cannot happen: the plan bounds the number of copies)
                  else ptx::mbar_expect_tx(&sh->p_full[slot], tx);
                }
              }
              ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
              cnt = __shfl_sync(0xffffffffu, cnt, 0);
              if (!ok) break;
              uint8_t* base = s_p + (size_t)slot * P.patch_bytes + (size_t)L.pad * 128;
              for (int i = lane; i < cnt; i += 32) {
                const int map = sh->box_map[i];
                const CUtensorMap* mp = map == 0 ? &map_r1 : (map == 1 ? &map_r2 : (map == 2 ? &map_r8 : (map == 3 ? &map_i1 : &map_i4)));
                ptx::tma_load_4d(base + sh->box_dst[i], mp, &sh->p_full[slot], chunk * 64, 0, sh->box_h[i], sh->box_n[i]);
              }
              __syncwarp();
              if (++slot == P.entries) { slot = 0; par ^= 1u; }
            }
          }
        }
      }
    } else if (warp == 2) {
      // ============================================================ weight producer
      if (lane == 0 && jobs > 0) {
        int slot = 0;
        uint32_t par = 1;
        bool ok = true;
        uint8_t* dst = s_w;
        for (int jb = 0; jb < jobs && ok; ++jb) {
          for (int s = 0; s < ns && ok; ++s) {
            ok = wait2(cx, &sh->w_empty[slot], par, 2);
            if (!ok) break;
            ptx::mbar_expect_tx(&sh->w_full[slot], (uint32_t)P.w_stage_bytes);
            ptx::tma_load_2d(dst, (s_tab[s].flags & kStageCond) ? &map_wc : &map_wb, &sh->w_full[slot],
                             s_tab[s].kx, tile_c * 128);
            dst += P.w_stage_bytes;
            if (++slot == P.ring) { slot = 0; par ^= 1u; dst = s_w; }
          }
        }
      }
    } else {
      // ============================================================ MMA issuers: warp 1 sub-tile a, warp 3 sub-tile b
      // Each sub-tile has its own issuing thread, so that one blocked on its gate pass does not
      // hold up the other.  Both walk the same stage sequence; a weight stage is released when
      // both have committed it.  The per-stage code is kept short: the issuing thread shares its
      // scheduler with four epilogue warps.
      const int X = warp == 1 ? 0 : 1;
      if (lane == 0 && jobs > 0 && X < P.nsub) {
        const uint32_t desc_hi = (uint32_t)(ptx::smem_desc(0, 1024, 2) >> 32);
        const uint32_t w_lo0 = (ptx::smem_u32(s_w) >> 4) | 0x10000u;
        const uint32_t p_lo0 = (ptx::smem_u32(s_p) >> 4) | 0x10000u;
        const uint32_t w_step = (uint32_t)P.w_stage_bytes >> 4, p_step = (uint32_t)P.patch_bytes >> 4;
        const uint32_t idesc = ptx::idesc_bf16(128, (uint32_t)P.nmma);
        const uint32_t d_tmem = tmem + (uint32_t)(X * 256);
        const int rows_all = L.n * P.hp;
        const int lead_stage = (P.lead < ns ? P.lead : ns) - 1;
        int slot = 0;
        uint32_t wpar = 0, a_lo = w_lo0;
        int pnext = X;                                      // next patch entry of this sub-tile
        uint32_t ppar = 0;
        bool ok = true;
        unsigned long long st_sub = 0, st_sub_run = 0;
        uint32_t st_ks = 0;
        for (int jb = 0; jb < jobs && ok; ++jb) {
          const uint32_t par = (uint32_t)jb & 1u;
          int entry = -1;
          bool run = true;
          uint32_t acc = 0u, b_lo = 0u;
          for (int s = 0; s < ns && ok; ++s) {
            // (the stage is unpacked into scalars: indexing a local copy with a run-time K step
            // would put it on the stack, and every access would then travel to L2)
            const uint4 raw = *(const uint4*)&s_tab[s];
            const uint32_t flags = raw.y & 0xffu, ks0 = (raw.y >> 16) & 0xffu, ks1 = raw.y >> 24;
            if (flags & (kStageFirst | kStageFirstCond | kStageNewChunk)) {
              if (flags & kStageFirst) {
                // sub-tile b starts `lead` stages behind a, so that the gate and combine passes of
                // one overlap the MMAs of the other
                if (X == 1) {
                  ok = wait2(cx, &sh->a_ahead, par, 17);
                  if (!ok) break;
                }
                ok = wait2(cx, &sh->tmem_free[X], par ^ 1u, 10 + X);
                if (!ok) break;
                ptx::tc_fence_after();                      // the epilogue's TMEM reads come before the MMAs below
              }
              if (flags & kStageFirstCond) {
                ok = wait2(cx, &sh->p_read[X], par, 12 + X);
                if (!ok) break;
                ptx::tc_fence_after();
                if (!dense) {
                  uint32_t f = 0;
#pragma unroll
                  for (int w = 0; w < kEpiWarps; ++w) f |= *(volatile uint32_t*)&sh->fired[X][w];
                  run = f != 0u;
                }
                // (sub-tiles made of padding rows only do not count as skipped work; a sub-tile
                // taller than an image's padding always holds a real row)
                const int gs = (first_m + jb * stride_m) * rows_per_job + X * P.r;
                bool has_rows = gs < rows_all && P.r > P.hp - L.h;
                if (!has_rows)
                  for (int g = gs, e = gs + P.r; g < e && g < rows_all; ++g) has_rows = has_rows || (g % P.hp) < L.h;
                if (has_rows) { st_sub += 1; if (run) st_sub_run += 1; }
              }
              if (flags & kStageNewChunk) {
                if (entry >= 0) ptx::umma_commit(&sh->p_empty[entry]);
                entry = pnext;
                ok = wait2(cx, &sh->p_full[entry], ppar, 15 + X);
                if (!ok) break;
                pnext += P.nsub;
                if (pnext >= P.entries) { pnext -= P.entries; ppar ^= 1u; }
                b_lo = p_lo0 + (uint32_t)entry * p_step;
              }
            }
            ok = wait2(cx, &sh->w_full[slot], wpar, 14);
            if (!ok) break;
            if (!(flags & kStageCond) || run) {
#pragma unroll
              for (int ks = 0; ks < 4; ++ks) {
                const uint32_t boff = ((ks & 2) ? raw.w : raw.z) >> (16 * (ks & 1)) & 0xffffu;
                if ((uint32_t)ks >= ks0 && (uint32_t)ks < ks1) {
                  ptx::umma_bf16(d_tmem, ((uint64_t)desc_hi << 32) | (a_lo + (uint32_t)ks * 2u),
                                 ((uint64_t)desc_hi << 32) | (b_lo + boff), idesc, acc);
                  acc = 1u;
                }
              }
              st_ks += ks1 - ks0;
            }
            ptx::umma_commit(&sh->w_empty[slot]);
            if (X == 0 && P.nsub == 2 && s == lead_stage) ptx::mbar_arrive(&sh->a_ahead);
            a_lo += w_step;
            if (++slot == P.ring) { slot = 0; wpar ^= 1u; a_lo = w_lo0; }
            if (flags & (kStageLastBase | kStageLast)) {
              if (flags & kStageLastBase) ptx::umma_commit(&sh->base_done[X]);
              if (flags & kStageLast) {
                ptx::umma_commit(&sh->p_empty[entry]);
                ptx::umma_commit(&sh->cond_done[X]);
              }
            }
          }
        }
        if (ok) {
          atomicAdd(&prm.counters[CNT_TILES_TOTAL], st_sub);
          atomicAdd(&prm.counters[CNT_TILES_SKIPPED], st_sub - st_sub_run);
          atomicAdd(&prm.counters[CNT_EXEC_MACS], (unsigned long long)st_ks * 16ull * 128ull * (unsigned long long)P.nmma);
          if (blockIdx.x == 0 && X == 0) atomicAdd(&prm.counters[CNT_CALLS], 1ull);
        }
      }
    }
    __syncwarp();
  } else {
    // ============================================================ epilogue
    // A warp owns one TMEM lane quadrant (32 channels) and every fourth 16-pixel piece of a
    // sub-tile; it reads the accumulators in the 16x256b fragment layout, where a thread holds
    // four channels x four pixels of a piece.
    const int quad = warp & 3;
    const int pg = (warp - kEpiWarp0) >> 2;
    const int ch0 = tile_c * 128 + quad * 32;
    const bool ch_valid = ch0 < L.c_out;                      // (uniform over the warp; c_out is a multiple of 32)
    Consts4 kc;
#pragma unroll
    for (int ci = 0; ci < 4; ++ci) {
      kc.kt[ci] = 0.f; kc.ka1[ci] = 0.f; kc.kb1[ci] = 0.f; kc.ka2[ci] = 0.f; kc.kb2[ci] = 0.f;
      if (ch_valid && jobs > 0) {
        const ChannelConsts k = fold_channel(prm.bn, prm.delta, L.eps, ch0 + 8 * ci + (lane >> 2));
        kc.kt[ci] = k.t; kc.ka1[ci] = k.a1; kc.kb1[ci] = k.b1; kc.ka2[ci] = k.a2; kc.kb2[ci] = k.b2;
        sh->t2[quad * 32 + 8 * ci + (lane >> 2)] = k.t2;   // (the four warps of a quadrant write the same values)
      }
    }
    const float lo = L.relu ? 0.f : -__int_as_float(0x7f800000);   // f = ReLU, or the identity
    const bool two_sided = prm.bn.delta_high != nullptr;
    __syncwarp();                                                  // (sh->t2 is read by the warp's own lanes only)
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const int word_idx = tile_c * 4 + quad;
    __nv_bfloat16* y_q = prm.y + ch0;
    const __nv_bfloat16* res_q = kHasRes ? prm.residual + ch0 : nullptr;
    uint8_t* s_tile = smem + P.off_epi + (warp - kEpiWarp0) * kEpiTileBytes;
    unsigned long long st_active = 0, st_words = 0, st_words_on = 0;
    Keep keep0 = {{~0u, ~0u}, 0u}, keep1 = keep0;
    bool ok = true;
    for (int jb = 0; jb < jobs && ok; ++jb) {
      const uint32_t par = (uint32_t)jb & 1u;
      const int g0 = (first_m + jb * stride_m) * rows_per_job;
      // gate of a, gate of b, combine of a, combine of b: the order in which their inputs complete
#pragma unroll 1
      for (int e = 0; e < 4 && ok; ++e) {
        const int X = e & 1;
        const bool comb = e >= 2;
        if (X == 1 && P.nsub != 2) continue;
        ok = wait2(cx, comb ? &sh->cond_done[X] : &sh->base_done[X], par, 20 + e);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t t_acc = t_lane + (uint32_t)(X * 256);
        Keep kx = X ? keep1 : keep0;
        if (ch_valid) {
          if (!comb)
            if (two_sided)
              gate_pass<kHasRes, true>(prm, kx, kc, sh->t2 + quad * 32, t_acc, g0 + X * P.r, pg, lane, word_idx, lo, y_q, res_q,
                                       s_tile, st_active, st_words, st_words_on);
            else
              gate_pass<kHasRes, false>(prm, kx, kc, nullptr, t_acc, g0 + X * P.r, pg, lane, word_idx, lo, y_q, res_q,
                                        s_tile, st_active, st_words, st_words_on);
          else
            combine_pass<kHasRes>(prm, kx, kc, t_acc, pg, lane, lo, y_q, res_q, s_tile);
        }
        if (!comb) {
          if (X) keep1 = kx; else keep0 = kx;
          if (lane == 0) sh->fired[X][warp - kEpiWarp0] = ch_valid ? kx.fired : 0u;
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(comb ? &sh->tmem_free[X] : &sh->p_read[X]);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      st_active += __shfl_xor_sync(0xffffffffu, st_active, o);
      st_words += __shfl_xor_sync(0xffffffffu, st_words, o);
      st_words_on += __shfl_xor_sync(0xffffffffu, st_words_on, o);
    }
    if (lane == 0 && ok && ch_valid) {
      atomicAdd(&prm.counters[CNT_ACTIVE], st_active);
      atomicAdd(&prm.counters[CNT_ROWS_TOTAL], st_words);
      atomicAdd(&prm.counters[CNT_ROWS_ACTIVE], st_words_on);
    }
  }
  // ---------------------------------------------------------------- teardown
  if (*(volatile uint32_t*)&sh->abort_flag) {
    // a wait gave up somewhere: let copies and MMAs that are still in flight finish before the
    // CTA's shared memory and TMEM go back
    const long long t0 = clock64();
    while (clock64() - t0 < kDrainCycles) {}
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    ptx::tmem_dealloc(tmem, 512);
  }
}

// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn2)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn2 encode_fn2() {
  static EncodeTiledFn2 fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault,
                                         &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn2)p;
  }
  return fn;
}

bool encode2(CUtensorMap* map, void* base, int rank, const cuuint64_t* dims,
             const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  EncodeTiledFn2 fn = encode_fn2();
  if (!fn) return false;
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, base, dims, strides_bytes, box,
            es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t align_up2(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Base slices of 8 channels (G = 8 at 64 input channels) are half of the 16-channel K step of a
// bf16 MMA.  The weights are copied into scratch memory with the K steps made whole: W_base gets 8
// zero channels behind its 8 per tap (the base path then reads input channels [0,16) and multiplies
// the upper 8 by zero), W_cond gets 8 zero channels in front (the conditional path reads every
// channel and multiplies the first 8 by zero).  The sums are unchanged.
__global__ void tc2_repack_kernel(const __nv_bfloat16* __restrict__ wb, const __nv_bfloat16* __restrict__ wc,
                                  __nv_bfloat16* __restrict__ wb16, __nv_bfloat16* __restrict__ wcf, int rows,
                                  int c_in) {
  // rows = c_out * taps
  const int total = rows * (16 + c_in);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int row = i / (16 + c_in), c = i - row * (16 + c_in);
    if (c < 16) {
      wb16[(size_t)row * 16 + c] = c < 8 ? wb[(size_t)row * 8 + c] : __float2bfloat16_rn(0.f);
    } else {
      const int cc = c - 16;
      wcf[(size_t)row * c_in + cc] = cc < 8 ? __float2bfloat16_rn(0.f) : wc[(size_t)row * (c_in - 8) + cc - 8];
    }
  }
}

}  // namespace

size_t repack8_bytes(const LayerDims& L) {
  const size_t rows = (size_t)L.c_out * L.kh * L.kw;
  return align_up2(rows * 16 * 2, 256) + align_up2(rows * (size_t)L.c_in * 2, 256);
}

int launch_repack8(const LayerDims& L, const void* w_base, const void* w_cond, void* workspace, const void** wb16,
                   const void** wcf, cudaStream_t stream) {
  const size_t rows = (size_t)L.c_out * L.kh * L.kw;
  __nv_bfloat16* b = static_cast<__nv_bfloat16*>(workspace);
  __nv_bfloat16* c = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + align_up2(rows * 16 * 2, 256));
  tc2_repack_kernel<<<64, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(w_base), static_cast<const __nv_bfloat16*>(w_cond), b, c,
                                            (int)rows, L.c_in);
  *wb16 = b; *wcf = c;
  return (int)cudaGetLastError();
}

size_t tc2_workspace_bytes(const LayerDims& L, const Tc2Plan& P) {
  if (!P.valid || !P.pad8) return 0;
  return repack8_bytes(L);
}

// K stages of a job in the order the MMA issuer consumes them (and the weight producer loads
// them).  Base path: when c_p >= 64 one stage per (64-channel chunk, filter tap); when c_p is 16
// or 32 a stage covers 64/c_p taps of chunk 0.  Conditional path: one stage per (chunk, tap);
// when c_p < 64 chunk 0 comes first and only its K steps behind the base channels are used.
static int build_stages(const LayerDims& L0, int wp, int pad8, Tc2Stage* st, int* nb_out) {
  // (pad8: the weights are repacked so that the base path reads 16 channels per tap, the upper 8
  // with zero weights, and the conditional path reads every channel, the first 8 with zero weights)
  LayerDims L = L0;
  if (pad8) { L.c_p = 16; L.c_r = L.c_in; }
  const int taps = L.kh * L.kw;
  const int chunks = L.c_in / 64;
  int n = 0;
  auto tap_off = [&](int t) { return (t / L.kw) * wp + (t % L.kw); };
  auto full_stage = [&](int kx, int cond, int chunk, int t, int ks0) {
    if (n >= kTc2MaxStages) { ++n; return; }
    Tc2Stage s;
    std::memset(&s, 0, sizeof(s));
    s.kx = kx; s.flags = (uint8_t)(cond ? kStageCond : 0); s.chunk = (uint8_t)chunk; s.ks0 = (uint8_t)ks0; s.ks1 = 4;
    for (int ks = 0; ks < 4; ++ks) s.boff[ks] = (uint16_t)(tap_off(t) * 8 + ks * 2);
    st[n++] = s;
  };
  if (L.c_p >= 64) {
    for (int q = 0; q < L.c_p / 64; ++q)
      for (int t = 0; t < taps; ++t) full_stage(t * L.c_p + 64 * q, 0, q, t, 0);
  } else {
    const int kp = taps * L.c_p;
    for (int i = 0; i * 64 < kp; ++i) {
      if (n >= kTc2MaxStages) { ++n; continue; }
      Tc2Stage s;
      std::memset(&s, 0, sizeof(s));
      s.kx = 64 * i; s.flags = 0; s.chunk = 0; s.ks0 = 0;
      int ks = 0;
      for (; ks < 4 && 64 * i + 16 * ks < kp; ++ks) {
        const int k = 64 * i + 16 * ks;
        s.boff[ks] = (uint16_t)(tap_off(k / L.c_p) * 8 + (k % L.c_p) / 8);
      }
      s.ks1 = (uint8_t)ks;
      st[n++] = s;
    }
  }
  *nb_out = n;
  if (L.c_r > 0) {
    if (L.c_p >= 64) {
      for (int q = L.c_p / 64; q < chunks; ++q)
        for (int t = 0; t < taps; ++t) full_stage(t * L.c_r + 64 * q - L.c_p, 1, q, t, 0);
    } else if (pad8) {
      for (int q = 0; q < chunks; ++q)
        for (int t = 0; t < taps; ++t) full_stage(t * L.c_r + 64 * q, 1, q, t, 0);
    } else {
      for (int t = 0; t < taps; ++t) full_stage(t * L.c_r - L.c_p, 1, 0, t, L.c_p / 16);
      for (int q = 1; q < chunks; ++q)
        for (int t = 0; t < taps; ++t) full_stage(t * L.c_r + 64 * q - L.c_p, 1, q, t, 0);
    }
  }
  if (n <= kTc2MaxStages) {
    for (int i = 0; i < n; ++i) {
      if (i == 0) st[i].flags |= kStageFirst;
      if (i == *nb_out && *nb_out < n) st[i].flags |= kStageFirstCond;
      if (i == *nb_out - 1) st[i].flags |= kStageLastBase;
      if (i == n - 1) st[i].flags |= kStageLast;
      if (i == 0 || st[i].chunk != st[i - 1].chunk) st[i].flags |= kStageNewChunk;
    }
  }
  return n;
}

bool tc2_plan(const LayerDims& L, int in_dtype, int cond_mode, int sms, Tc2Plan* plan) {
  Tc2Plan& P = *plan;
  std::memset(&P, 0, sizeof(P));
  if (in_dtype != CG_BF16) return false;
  if (L.stride != 1) return false;
  // channel grouping: whole 64-channel chunks per input group, 128-channel tiles inside one output group
  if (L.grouping && (L.c_p % 64 != 0 || (L.c_out / L.groups) % 128 != 0)) return false;
  if (L.kh != L.kw || L.kh != 2 * L.pad + 1) return false;
  if (L.c_in % 64 != 0 || L.c_out % 32 != 0) return false;
  if (!(L.c_p == 8 || L.c_p == 16 || L.c_p == 32 || L.c_p % 64 == 0)) return false;
  P.pad8 = L.c_p == 8 ? 1 : 0;
  if (cond_mode == CG_COND_COMPACT) return false;
  if (L.c_in / 64 > 255) return false;
  P.wp = L.w + L.pad;
  P.hp = L.h + L.pad;
  if (P.wp > 256) return false;                            // a sub-tile is at least one stacked row, at most 256 pixels
  if ((long long)L.n * L.ho * L.wo * L.c_out >= (1ll << 32) - 1) return false;   // y is indexed in 32 bits
  P.chunks = L.c_in / 64;
  P.tiles_c = (L.c_out + 127) / 128;
  P.ns = build_stages(L, P.wp, P.pad8, P.st, &P.nb);
  if (P.ns > kTc2MaxStages) return false;
  // the largest tap offset must fit the 16-bit table entries
  if (((L.kh - 1) * P.wp + L.kw) * 8 + 8 > 65535) return false;
  P.w_rows = L.c_out < 128 ? L.c_out : 128;
  P.w_stage_bytes = P.w_rows * 128;
  P.cond_mode = cond_mode == CG_COND_AUTO ? CG_COND_SKIP_TILES : cond_mode;
  P.inv_wp = 1.0f / (float)P.wp; P.inv_hp = 1.0f / (float)P.hp;
  if ((long long)L.n * P.hp >= (1 << 20)) return false;     // stacked rows are divided in single precision
  P.use_img = P.hp * P.wp <= 256 ? 1 : 0;                  // whole images as single copies
  const long long rows_all = (long long)L.n * P.hp;
  int ksteps = 0;
  for (int i = 0; i < P.ns; ++i) ksteps += P.st[i].ks1 - P.st[i].ks0;
  const size_t limit = 227 * 1024 - 1024;
  const size_t bar_bytes = align_up2(sizeof(Shared2), 128);
  // Search the sub-tile height and the number of sub-tiles: estimated time = rounds of jobs over
  // the SMs x the larger of a job's MMA time and the time to stream its weights from L2.
  double best = 1e300;
  for (int nsub = 2; nsub >= 1; --nsub) {
    for (int r = 1; r * P.wp <= 256 && r <= rows_all; ++r) {
      const int np = r * P.wp;
      const int nmma = (np + 15) / 16 * 16;
      const int patch_rows = nmma + (L.kh - 1) * P.wp + (L.kw - 1) + 1;
      const size_t patch_bytes = align_up2((size_t)patch_rows * 128, 1024);
      {
        // copies per patch, worst case: a run of rows before the first whole image, whole images,
        // a run after the last; a run of len rows takes len/8 + (len%8)/2 + len%2 copies
        const int box_rows = r + 2 * L.pad;
        const int run = P.hp - 1 < box_rows ? P.hp - 1 : box_rows;
        const int per_run = run / 8 + (run % 8) / 2 + run % 2;
        const int images = P.use_img ? box_rows / P.hp + 1 : 0;
        const int runs = P.use_img ? 2 : box_rows / P.hp + 2;
        if (runs * per_run + images + 4 > kMaxBoxes) continue;
      }
      // shared memory: patch entries (three, so that the next input-channel chunk of a sub-tile
      // loads while the current one is read; two where that leaves the weight ring too short),
      // staging tiles, stage table, barriers; the rest is the weight ring
      const int min_ring = nsub == 2 ? 5 : 3;
      int entries = 0, ring = 0;
      for (int en = kPatchEntries; en >= 2 && entries == 0; --en) {
        const size_t fixed = en * patch_bytes + bar_bytes + (P.w_rows < 128 ? 128 * 128 : 0) +
                             kTc2MaxStages * sizeof(Tc2Stage) + (size_t)kEpiWarps * 1280;
        if (fixed + (size_t)min_ring * P.w_stage_bytes > limit) continue;
        entries = en;
        ring = (int)((limit - fixed) / P.w_stage_bytes);
      }
      if (entries == 0) continue;
      if (ring > kMaxRing) ring = kMaxRing;
      int lead = nsub == 2 ? ring - 3 : 0;
      if (lead > 4) lead = 4;
      const long long jobs_m = (rows_all + (long long)r * nsub - 1) / ((long long)r * nsub);
      const long long jobs = jobs_m * P.tiles_c;
      int grid = sms - sms % P.tiles_c;
      if (grid < P.tiles_c) grid = P.tiles_c;
      if (jobs < grid) grid = (int)jobs;
      const long long rounds = (jobs + grid - 1) / grid;
      const double mma = (double)ksteps * (nmma / 2.0) * nsub;
      const double l2 = (double)P.ns * P.w_stage_bytes / 40.0;
      // per job: the gate and combine passes of the last sub-tile are exposed, less what the lead hides
      const double job = (mma > l2 ? mma : l2) + 3000.0 + (nsub == 1 ? 6000.0 : 6000.0 - 1000.0 * lead);
      const double est = rounds * job;
      if (est < best) {
        best = est;
        P.r = r; P.nsub = nsub; P.np = np; P.nmma = nmma; P.jobs_m = (int)jobs_m;
        P.patch_rows = patch_rows; P.patch_bytes = (int)patch_bytes; P.patch_box_rows = r + 2 * L.pad;
        P.ring = ring; P.entries = entries; P.lead = lead; P.grid = grid;
      }
    }
  }
  if (best >= 1e299) return false;
  size_t off = 0;
  P.off_w = (unsigned)off; off += align_up2((size_t)P.ring * P.w_stage_bytes + (P.w_rows < 128 ? 128 * 128 : 0), 1024);
  P.off_p = (unsigned)off; off += (size_t)P.entries * P.patch_bytes;
  P.off_epi = (unsigned)off; off += (size_t)kEpiWarps * kEpiTileBytes;
  P.off_tab = (unsigned)off; off += (size_t)kTc2MaxStages * sizeof(Tc2Stage);
  P.off_bar = (unsigned)off; off += bar_bytes;
  P.smem_bytes = (unsigned)(off + 1024);
  if (P.smem_bytes > 227 * 1024) return false;
  P.valid = 1;
  return true;
}

int launch_tc2(const LayerDims& L, const Tc2Plan& P, Tc2Maps* maps, const void* x,
               const void* w_base_in, const void* w_cond_in, const cg_bn_params& bn, const float* delta,
               const void* residual, void* y, uint32_t* mask, void* workspace, unsigned long long* counters,
               cudaStream_t stream) {
  if (!P.valid) return (int)cudaErrorInvalidValue;
  const void* w_base = w_base_in;
  const void* w_cond = w_cond_in;
  int c_p = L.c_p, c_r = L.c_r;
  if (P.pad8) {
    if (!workspace) return (int)cudaErrorInvalidValue;
    const size_t rows = (size_t)L.c_out * L.kh * L.kw;
    __nv_bfloat16* wb16 = static_cast<__nv_bfloat16*>(workspace);
    __nv_bfloat16* wcf = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + align_up2(rows * 16 * 2, 256));
    tc2_repack_kernel<<<64, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(w_base_in),
                                              static_cast<const __nv_bfloat16*>(w_cond_in), wb16, wcf, (int)rows, L.c_in);
    w_base = wb16; w_cond = wcf; c_p = 16; c_r = L.c_in;
  }
  const void* wc_key = w_cond ? w_cond : w_base;
  Tc2MapSet* ms = nullptr;
  for (int i = 0; i < Tc2Maps::kEntries; ++i) {
    Tc2MapSet* c = &maps->set[i];
    if (c->key[0] == x && c->key[1] == w_base && c->key[2] == wc_key) { ms = c; break; }
  }
  if (!ms) {
    ms = &maps->set[maps->next];
    maps->next = (maps->next + 1) % Tc2Maps::kEntries;
    ms->key[0] = nullptr;
    const int taps = L.kh * L.kw;
    {
      // boxes of whole stacked rows: W real pixels and `pad` out-of-bounds (zero) pixels behind
      // them; 1, 2 or 8 rows of one image, or 1 or 4 whole images with their `pad` zero rows
      cuuint64_t dims[4] = {(cuuint64_t)L.c_in, (cuuint64_t)L.w, (cuuint64_t)L.h, (cuuint64_t)L.n};
      cuuint64_t str[3] = {(cuuint64_t)L.c_in * 2, (cuuint64_t)L.w * L.c_in * 2,
                           (cuuint64_t)L.h * L.w * L.c_in * 2};
      const cuuint32_t hp = (cuuint32_t)(P.use_img ? P.hp : 1);
      const cuuint32_t boxes[5][2] = {{1, 1}, {2, 1}, {8, 1}, {hp, 1}, {hp, 4}};
      for (int i = 0; i < 5; ++i) {
        cuuint32_t box[4] = {64, (cuuint32_t)P.wp, boxes[i][0], boxes[i][1]};
        if (!encode2(&ms->x[i], const_cast<void*>(x), 4, dims, str, box)) return (int)cudaErrorInvalidValue;
      }
    }
    {
      cuuint64_t dims[2] = {(cuuint64_t)taps * c_p, (cuuint64_t)L.c_out};
      cuuint64_t str[1] = {(cuuint64_t)taps * c_p * 2};
      cuuint32_t box[2] = {64, (cuuint32_t)P.w_rows};
      if (!encode2(&ms->wb, const_cast<void*>(w_base), 2, dims, str, box)) return (int)cudaErrorInvalidValue;
    }
    if (c_r > 0) {
      cuuint64_t dims[2] = {(cuuint64_t)taps * c_r, (cuuint64_t)L.c_out};
      cuuint64_t str[1] = {(cuuint64_t)taps * c_r * 2};
      cuuint32_t box[2] = {64, (cuuint32_t)P.w_rows};
      if (!encode2(&ms->wc, const_cast<void*>(w_cond), 2, dims, str, box)) return (int)cudaErrorInvalidValue;
    } else {
      ms->wc = ms->wb;
    }
    ms->key[0] = x; ms->key[1] = w_base; ms->key[2] = wc_key;
  }
  Tc2Params prm;
  prm.L = L; prm.bn = bn; prm.delta = delta;
  prm.residual = (const __nv_bfloat16*)residual;
  prm.y = (__nv_bfloat16*)y; prm.mask = mask; prm.counters = counters;
  prm.P = P;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return (int)cudaErrorInvalidDevice;
  typedef void (*Kernel2)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, Tc2Params);
  const int which = residual ? 1 : 0;
  const Kernel2 kernels[2] = {tc2_gated_conv_kernel<false>, tc2_gated_conv_kernel<true>};
  static bool attr_set[64][2] = {};
  if (!attr_set[dev][which]) {
    const cudaError_t e = cudaFuncSetAttribute(kernels[which], cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               227 * 1024);
    if (e != cudaSuccess) return (int)e;
    attr_set[dev][which] = true;
  }
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)P.grid, 1, 1);
  cfg.blockDim = dim3((unsigned)kThreads2, 1, 1);
  cfg.dynamicSmemBytes = 227 * 1024;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kernels[which], ms->x[0], ms->x[1], ms->x[2], ms->x[3], ms->x[4], ms->wb, ms->wc, prm);
  if (e != cudaSuccess) return (int)e;
  return (int)cudaGetLastError();
}

}  // namespace cg
