// Channel-gated 3x3 convolution for 64 -> 64 channel layers on tcgen05 tensor cores, with the
// three taps of a filter row stacked on the MMA's N side.
//
// A 64-channel layer gives the tensor core only N = 64 columns per MMA (half its rate) and needs 36
// MMAs of K = 16 per 128-pixel tile.  Here the weights of the taps (r,0), (r,1), (r,2) form ONE B
// operand of 192 rows (tap-major, then output channel), so that a single MMA computes, for every
// pixel slot i of the tile and each horizontal tap s,
//     D_s[i, c] = sum_r sum_k X[i + r*W, k] * W[(r,s), k, c]
// from the same A operand: the input patch, stored without any padding between image rows (pitch W),
// read from row r*W on.  The output pixel at slot i is then (Section 3.1: y = W * x)
//     D_0[i-1] + D_1[i] + D_2[i+1],
// where the first term is dropped in image column 0 and the last in column W-1 (the zero padding):
// the epilogue takes the neighbours' values by warp shuffles.  A job needs 12 MMAs of N = 192
// instead of 36 of N = 64, a tile is 128 REAL pixels (no pad columns on the M side), and a TMEM lane
// quadrant holds whole image rows when W divides 32, so no value crosses a warp.
//
// Per job (128 / W output rows of one image), following Section 3.1 and Eq. 1-3:
//   base path    raw P = the three D_s over the base channels (TMEM columns [0,192));
//   gate         8 warps: P = shifted sum of raw P, written back to TMEM as 64 columns (a ring of two)
//                so that raw P is free for the next job at once; d = (P >= t[c]) (and P <= t2[c] for
//                the two-sided gate of Section 3.2) -> mask words;
//   conditional  raw R over the remaining channels (TMEM columns [192,384)), skipped if no gate of the
//                job fired (CG_COND_SKIP_TILES);
//   combine      8 warps: R = shifted sum of raw R; y = f(BN1(P)) or f(BN2(P+R)) by mask bit, staged
//                in shared memory (two tiles) and written by one TMA store.
// Weights are resident in shared memory: every CTA builds the three 192-row tiles itself with plain
// loads (row (s,c) = the 64 input channels of tap (r,s): base channels first, as in x).
//
// Warp roles: 0 = patch producer, 1 = MMA issuer (owns TMEM), 2-3 = help with the weights,
// 4-11 = gate group (TMEM lane quadrant x half of the channels), 12-19 = combine group (same
// split).  Every mbarrier wait is bounded; on expiry the CTA records CG_ERR_DEVICE_TIMEOUT with the
// id of the wait and leaves.
#include <cstring>

#include "ptx.cuh"
#include "tc3_conv.cuh"

namespace cg {

namespace {

constexpr int kT3Threads = 640;
constexpr int kGateWarp0 = 4, kGateWarps = 8;
constexpr int kCombWarp0 = 12, kCombWarps = 8;
constexpr int kEpiThreads = (kGateWarps + kCombWarps) * 32;
constexpr int kCombThreads = kCombWarps * 32;
constexpr int kLoaderWarps = 18;                 // warps 2-19 build the weight tiles
constexpr int kNA = 4;                           // patch buffers
constexpr int kPatchBytes = 192 * 128;           // 128 pixel slots + two image rows of at most 32 pixels
constexpr int kWTileBytes = 192 * 128;           // one filter row: 3 taps x 64 output channels
constexpr int kStageBytes = 128 * 128;           // y staging tile
constexpr uint32_t kColRawP = 0, kColRawR = 192, kColFin = 384;   // TMEM columns
constexpr int kSpinLimit = 1 << 21;
constexpr long long kWaitCycles = 2000000000ll;

// shared-memory map (offsets from a 1024-byte-aligned base)
constexpr unsigned kOffW = 0;
constexpr unsigned kOffA = kOffW + 3 * kWTileBytes;
constexpr unsigned kOffY = kOffA + kNA * kPatchBytes;
constexpr unsigned kOffMask = kOffY + 2 * kStageBytes;        // [2][128][2] mask words
constexpr unsigned kOffConsts = kOffMask + 2 * 128 * 2 * 4;   // t[64], t2[64], {a1,b1,a2,b2}[64]
constexpr unsigned kOffBar = kOffConsts + 64 * 4 * 2 + 64 * 16;
constexpr unsigned kSmemUsed = kOffBar + 256;

struct Tc3Params {
  LayerDims L;
  Tc3Plan P;
  cg_bn_params bn;
  const float* delta;
  const __nv_bfloat16* w_base;
  const __nv_bfloat16* w_cond;
  const __nv_bfloat16* residual;
  uint32_t* mask;
  unsigned long long* counters;
};

struct Shared3 {
  uint64_t a_full[kNA], a_empty[kNA];
  uint64_t w_ready;
  uint64_t rawp_full, rawp_free, rawr_full, rawr_free;
  uint64_t fin_full[2], fin_free[2];
  uint32_t tmem_base;
  uint32_t abort_flag;
  uint32_t fired[2][kGateWarps];   // per P slot, per gate warp: a gate of its rows and channels fired
};
static_assert(sizeof(Shared3) <= 256, "barrier block");

// Bounded wait (the loop lives in one out-of-line copy).  Each poll parks the thread in hardware for
// a short time; the wait gives up after about a second, or within a few polls once another wait of
// the CTA has given up.
__device__ __noinline__ bool wait3_slow(Shared3* sh, unsigned long long* counters, uint64_t* bar, uint32_t parity,
                                        int site) {
  const long long t0 = clock64();
  for (int i = 0; i < kSpinLimit; ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 15) == 15) {
      if (*(volatile uint32_t*)&sh->abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) break;
    }
  }
  if (atomicCAS(&counters[CNT_STATUS], 0ull, (unsigned long long)CG_ERR_DEVICE_TIMEOUT) == 0ull)
    atomicExch(&counters[CNT_SITE], (unsigned long long)(300 + site));
  atomicExch(&sh->abort_flag, 1u);
  return false;
}

// The wait as taken by every lane of a convergent warp; the outcome is warp-uniform.
__device__ __forceinline__ bool wait3(Shared3* sh, unsigned long long* counters, uint64_t* bar, uint32_t parity,
                                      int site) {
  bool ok = ptx::mbar_try_wait(bar, parity, 0u);
  if (!ok) ok = wait3_slow(sh, counters, bar, parity, site);
  return __all_sync(0xffffffffu, ok);
}

// K steps [KS0, KS1) of the three filter rows: 3 * (KS1 - KS0) MMAs of 128 x 192 x 16 into d_tmem.
// a_lo / b_lo: lower descriptor words of the patch and of the first weight tile; row_lo: one image
// row of the patch in 16-byte units.
template <int KS0, int KS1>
__device__ __forceinline__ void issue_rows(uint32_t lead, uint32_t desc_hi, uint32_t a_lo, uint32_t b_lo,
                                           uint32_t row_lo, uint32_t d_tmem) {
  constexpr uint32_t idesc = ptx::idesc_bf16(128, 192);
  uint32_t acc = 0u;
#pragma unroll
  for (int r = 0; r < 3; ++r) {
#pragma unroll
    for (int ks = KS0; ks < KS1; ++ks) {
      const uint64_t da = ((uint64_t)desc_hi << 32) | (a_lo + (uint32_t)r * row_lo + (uint32_t)ks * 2u);
      const uint64_t db = ((uint64_t)desc_hi << 32) | (b_lo + (uint32_t)r * (kWTileBytes >> 4) + (uint32_t)ks * 2u);
      ptx::umma_bf16_if(lead, d_tmem, da, db, idesc, acc);
      acc = 1u;
    }
  }
}

// One output value from the three stacked partial sums of its pixel slot and the neighbours'.
__device__ __forceinline__ float stacked_sum(uint32_t d0, uint32_t d1, uint32_t d2, bool first_col, bool last_col) {
  const float a = __uint_as_float(__shfl_up_sync(0xffffffffu, d0, 1));
  const float b = __uint_as_float(__shfl_down_sync(0xffffffffu, d2, 1));
  return (__uint_as_float(d1) + (first_col ? 0.f : a)) + (last_col ? 0.f : b);
}

__global__ void __launch_bounds__(kT3Threads, 1)
tc3_gated_conv_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                      const __grid_constant__ Tc3Params prm) {
  extern __shared__ uint8_t smem_raw[];
  ptx::grid_launch_dependents();   // the next kernel in the stream may start as SMs become free
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  const LayerDims& L = prm.L;
  const Tc3Plan& P = prm.P;
  uint8_t* s_w = smem + kOffW;
  uint8_t* s_a = smem + kOffA;
  uint8_t* s_y = smem + kOffY;
  uint32_t* s_mask = (uint32_t*)(smem + kOffMask);
  float* s_t = (float*)(smem + kOffConsts);
  float* s_t2 = s_t + 64;
  float4* s_k = (float4*)(s_t2 + 64);
  Shared3* sh = (Shared3*)(smem + kOffBar);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int W = L.w, H = L.h;
  const int jobs = ((int)P.jobs - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // (grid <= jobs)
  const bool dense = P.cond_mode == CG_COND_DENSE;
  const bool has_cond = L.c_r > 0;
  const bool two_sided = prm.bn.delta_high != nullptr;
  const uint32_t patch_tx = (uint32_t)((P.rows + 2) * W) * 128u;

  auto job_origin = [&](int j, int& n0, int& h0) {
    const int t = (int)blockIdx.x + j * (int)gridDim.x;
    n0 = t / P.tiles_per_image;
    h0 = (t - n0 * P.tiles_per_image) * P.rows;
  };
  auto any_fired = [&](int f) {
    const volatile uint32_t* w = sh->fired[f];
    uint32_t b = 0;
#pragma unroll
    for (int i = 0; i < kGateWarps; ++i) b |= w[i];
    return b != 0u;
  };

  // ---------------------------------------------------------------- setup
  if (threadIdx.x == 0) {
    for (int i = 0; i < kNA; ++i) { ptx::mbar_init(&sh->a_full[i], 1); ptx::mbar_init(&sh->a_empty[i], 1); }
    ptx::mbar_init(&sh->w_ready, kLoaderWarps);
    ptx::mbar_init(&sh->rawp_full, 1); ptx::mbar_init(&sh->rawp_free, kGateWarps);
    ptx::mbar_init(&sh->rawr_full, 1); ptx::mbar_init(&sh->rawr_free, kCombWarps);
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&sh->fin_full[i], kGateWarps); ptx::mbar_init(&sh->fin_free[i], kCombWarps); }
    sh->abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_x); ptx::prefetch_tensormap(&map_y);
  }
  if (warp == 1) ptx::tmem_alloc(&sh->tmem_base, 512);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  // everything above touched only this CTA's own state; global memory is used from here on, so the
  // kernel that ran before this one in the stream must be complete
  ptx::grid_dependency_wait();
  const uint32_t tmem = sh->tmem_base;

  if (warp >= 2) {
    // The weight tiles, written in the 128-byte-swizzled K-major layout the MMA reads: 16-byte piece p
    // of row n sits at piece p ^ (n & 7).  4608 pieces, eight per thread, all loads first.
    const int t2 = (int)threadIdx.x - 64;
    uint4 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int idx = t2 + k * (kLoaderWarps * 32);
      const int r = idx / 1536, rem = idx - r * 1536;
      const int n = rem >> 3, p = rem & 7;
      const int tap = 3 * r + (n >> 6), c = n & 63, ch = p * 8;
      const __nv_bfloat16* src = ch < L.c_p ? prm.w_base + ((size_t)c * 9 + tap) * L.c_p + ch
                                            : prm.w_cond + ((size_t)c * 9 + tap) * L.c_r + (ch - L.c_p);
      v[k] = __ldg((const uint4*)src);
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int idx = t2 + k * (kLoaderWarps * 32);
      const int r = idx / 1536, rem = idx - r * 1536;
      const int n = rem >> 3, p = rem & 7;
      *(uint4*)(s_w + (size_t)r * kWTileBytes + (size_t)n * 128 + ((p ^ (n & 7)) << 4)) = v[k];
    }
    ptx::fence_proxy_async();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(&sh->w_ready);
  }
  if (warp >= kGateWarp0) {
    const int et = (int)threadIdx.x - kGateWarp0 * 32;
    if (et < 64) {
      const ChannelConsts k = fold_channel(prm.bn, prm.delta, L.eps, et);
      s_t[et] = k.t; s_t2[et] = k.t2; s_k[et] = make_float4(k.a1, k.b1, k.a2, k.b2);
    }
    ptx::named_bar_sync(2, kEpiThreads);
  }

  if (warp == 0) {
    // ============================================================ patch producer
    bool ok = true;
    for (int j = 0; j < jobs && ok; ++j) {
      const int slot = j % kNA;
      ok = wait3(sh, prm.counters, &sh->a_empty[slot], ((j / kNA) & 1) ^ 1, 1);
      if (!ok) break;
      int n0, h0;
      job_origin(j, n0, h0);
      if (lane == 0) {
        ptx::mbar_expect_tx(&sh->a_full[slot], patch_tx);
        ptx::tma_load_4d(s_a + (size_t)slot * kPatchBytes, &map_x, &sh->a_full[slot], 0, 0, h0 - 1, n0);
      }
    }
  } else if (warp == 1) {
    // ============================================================ MMA issuer
    // (the whole warp, convergent; lane 0 issues)   order: base(0) | base(1) cond(0) | base(2) cond(1) ...
    const uint32_t lead = lane == 0 ? 1u : 0u;
    const uint32_t desc_hi = (uint32_t)(ptx::smem_desc(0, 1024, 2) >> 32);
    const uint32_t a_base_lo = (ptx::smem_u32(s_a) >> 4) | 0x10000u;
    const uint32_t b_lo = (ptx::smem_u32(s_w) >> 4) | 0x10000u;
    const uint32_t row_lo = (uint32_t)W * 8u;
    uint32_t r_use = 0;
    bool ok = jobs > 0 && wait3(sh, prm.counters, &sh->w_ready, 0, 2);
    for (int s = 0; s <= jobs && ok; ++s) {
      if (s < jobs) {
        const int slot = s % kNA;
        ok = wait3(sh, prm.counters, &sh->a_full[slot], (s / kNA) & 1, 3);
        ok = ok && wait3(sh, prm.counters, &sh->rawp_free, (s & 1) ^ 1, 4);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t a_lo = a_base_lo + (uint32_t)slot * (kPatchBytes >> 4);
        switch (P.kp) {
          case 1: issue_rows<0, 1>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawP); break;
          case 2: issue_rows<0, 2>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawP); break;
          case 3: issue_rows<0, 3>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawP); break;
          default: issue_rows<0, 4>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawP); break;
        }
        ptx::umma_commit_if(lead, &sh->rawp_full);
        if (!has_cond) ptx::umma_commit_if(lead, &sh->a_empty[slot]);
      }
      if (s >= 1 && has_cond) {
        const int jj = s - 1, f = jj & 1, slot = jj % kNA;
        bool run = true;
        if (!dense) {
          ok = wait3(sh, prm.counters, &sh->fin_full[f], (jj >> 1) & 1, 5);
          if (!ok) break;
          run = any_fired(f);
        }
        if (run) {
          ok = wait3(sh, prm.counters, &sh->rawr_free, (r_use & 1) ^ 1, 6);
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t a_lo = a_base_lo + (uint32_t)slot * (kPatchBytes >> 4);
          switch (P.kp) {
            case 1: issue_rows<1, 4>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawR); break;
            case 2: issue_rows<2, 4>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawR); break;
            default: issue_rows<3, 4>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawR); break;
          }
          ptx::umma_commit_if(lead, &sh->rawr_full);
          ptx::umma_commit_if(lead, &sh->a_empty[slot]);
          ++r_use;
        } else if (lane == 0) {
          ptx::mbar_arrive(&sh->a_empty[slot]);   // the job's patch is not needed again
        }
      }
    }
  } else if (warp >= kGateWarp0) {
    // ============================================================ epilogue (16 warps)
    const bool gate_group = warp < kCombWarp0;
    const int quad = warp & 3;                                   // TMEM lane quadrant
    const int half = ((warp - kGateWarp0) >> 2) & 1;             // channels [32*half, 32*half + 32) = one mask word
    const int i = quad * 32 + lane;                              // pixel slot = TMEM lane
    const int h_loc = i / W, col = i - h_loc * W;
    const bool first_col = col == 0, last_col = col == W - 1;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const int ct = (int)threadIdx.x - kCombWarp0 * 32;           // thread index within the combine group
    unsigned long long st_active = 0, st_rows = 0;
    uint32_t r_use = 0;
    bool ok = true;

    if (gate_group) {
      for (int j = 0; j < jobs && ok; ++j) {
        const int f = j & 1;
        ok = wait3(sh, prm.counters, &sh->rawp_full, j & 1, 7);
        if (!ok) break;
        ptx::tc_fence_after();
        int n0, h0;
        job_origin(j, n0, h0);
        const bool valid = h0 + h_loc < H;
        const long long m = ((long long)n0 * H + (h0 + h_loc)) * W + col;
        uint32_t word = 0;
#pragma unroll
        for (int piece = 0; piece < 2; ++piece) {
          const int cb = half * 32 + piece * 16;
          uint32_t d0[16], d1[16], d2[16];
          ptx::tmem_ld_nowait<16>(t_lane + kColRawP + (uint32_t)cb, d0);
          ptx::tmem_ld_nowait<16>(t_lane + kColRawP + 64u + (uint32_t)cb, d1);
          ptx::tmem_ld_nowait<16>(t_lane + kColRawP + 128u + (uint32_t)cb, d2);
          ptx::tmem_ld_wait<16>(d0);
          ptx::tmem_ld_wait<16>(d1);
          ptx::tmem_ld_wait<16>(d2);
          if (piece == 1) {
            // raw P has been read: the base path of the next job may overwrite it
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sh->rawp_free);
          }
          uint32_t p[16];
#pragma unroll
          for (int c = 0; c < 16; ++c) p[c] = __float_as_uint(stacked_sum(d0[c], d1[c], d2[c], first_col, last_col));
          if (piece == 0) {
            // the combine group must be done with this P slot's previous job
            ok = wait3(sh, prm.counters, &sh->fin_free[f], ((j >> 1) & 1) ^ 1, 8);
            if (!ok) break;
          }
          ptx::tmem_st16(t_lane + kColFin + (uint32_t)(f * 64 + cb), p);
          // four partial words, so that the bit inserts do not form one dependent chain
          uint32_t pw[4] = {0u, 0u, 0u, 0u};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float4 t4 = *(const float4*)(s_t + cb + q * 4);
            pw[q] |= (__uint_as_float(p[q * 4 + 0]) >= t4.x ? 1u : 0u) << (q * 4 + 0);
            pw[q] |= (__uint_as_float(p[q * 4 + 1]) >= t4.y ? 1u : 0u) << (q * 4 + 1);
            pw[q] |= (__uint_as_float(p[q * 4 + 2]) >= t4.z ? 1u : 0u) << (q * 4 + 2);
            pw[q] |= (__uint_as_float(p[q * 4 + 3]) >= t4.w ? 1u : 0u) << (q * 4 + 3);
          }
          uint32_t bits = (pw[0] | pw[1]) | (pw[2] | pw[3]);
          if (two_sided) {
            // Section 3.2: the gate also needs P <= the upper threshold (ties included)
            uint32_t ph[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float4 u4 = *(const float4*)(s_t2 + cb + q * 4);
              ph[q] |= (__uint_as_float(p[q * 4 + 0]) <= u4.x ? 1u : 0u) << (q * 4 + 0);
              ph[q] |= (__uint_as_float(p[q * 4 + 1]) <= u4.y ? 1u : 0u) << (q * 4 + 1);
              ph[q] |= (__uint_as_float(p[q * 4 + 2]) <= u4.z ? 1u : 0u) << (q * 4 + 2);
              ph[q] |= (__uint_as_float(p[q * 4 + 3]) <= u4.w ? 1u : 0u) << (q * 4 + 3);
            }
            bits &= (ph[0] | ph[1]) | (ph[2] | ph[3]);
          }
          word |= bits << (piece * 16);
        }
        if (!ok) break;
        ptx::tmem_st_wait();
        if (!valid) word = 0;
        s_mask[(f * 128 + i) * 2 + half] = word;
        if (valid && prm.mask) prm.mask[m * 2 + half] = word;
        st_active += __popc(word);
        const uint32_t any = __ballot_sync(0xffffffffu, word != 0u);
        const uint32_t rows_valid = __ballot_sync(0xffffffffu, valid);
        if (lane == 0) {
          sh->fired[f][warp - kGateWarp0] = any;
          if (half == 0) st_rows += __popc(rows_valid);
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh->fin_full[f]);
      }
    } else {
      for (int j = 0; j < jobs; ++j) {
        const int f = j & 1;
        uint8_t* buf = s_y + (size_t)(j & 1) * kStageBytes;
        // A wait that gives up must not keep its warp from the group barrier below, where the sibling
        // warps are going to arrive: the decision to leave is taken after it, from the CTA-wide flag.
        ok = wait3(sh, prm.counters, &sh->fin_full[f], (j >> 1) & 1, 9);
        const bool run = ok && has_cond && (dense || any_fired(f));
        if (run) ok = wait3(sh, prm.counters, &sh->rawr_full, r_use & 1, 10);
        int n0, h0;
        job_origin(j, n0, h0);
        if (ok) {
          ptx::tc_fence_after();
          const uint32_t wv = s_mask[(f * 128 + i) * 2 + half];
          if (half == 0) {
            const uint32_t other = s_mask[(f * 128 + i) * 2 + 1];
            const uint32_t act = __ballot_sync(0xffffffffu, (wv | other) != 0u);
            if (lane == 0) st_rows += __popc(act);
          }
          const bool valid = h0 + h_loc < H;
          const __nv_bfloat16* res_row = nullptr;
          if (prm.residual && valid)
            res_row = prm.residual + (((long long)n0 * H + (h0 + h_loc)) * W + col) * 64 + half * 32;
          uint8_t* st = buf + (size_t)i * 128;
#pragma unroll
          for (int piece = 0; piece < 2; ++piece) {
            const int cb = half * 32 + piece * 16;
            const uint32_t bits = (wv >> (piece * 16)) & 0xffffu;
            // R is read only where the conditional path ran and a gate of these rows and channels fired
            const bool have_r = run && __ballot_sync(0xffffffffu, bits != 0u) != 0u;
            uint32_t p[16], rr[16];
            ptx::tmem_ld_nowait<16>(t_lane + kColFin + (uint32_t)(f * 64 + cb), p);
            if (have_r) {
              uint32_t e0[16], e1[16], e2[16];
              ptx::tmem_ld_nowait<16>(t_lane + kColRawR + (uint32_t)cb, e0);
              ptx::tmem_ld_nowait<16>(t_lane + kColRawR + 64u + (uint32_t)cb, e1);
              ptx::tmem_ld_nowait<16>(t_lane + kColRawR + 128u + (uint32_t)cb, e2);
              ptx::tmem_ld_wait<16>(e0);
              ptx::tmem_ld_wait<16>(e1);
              ptx::tmem_ld_wait<16>(e2);
#pragma unroll
              for (int c = 0; c < 16; ++c) rr[c] = __float_as_uint(stacked_sum(e0[c], e1[c], e2[c], first_col, last_col));
            } else {
#pragma unroll
              for (int c = 0; c < 16; ++c) rr[c] = 0u;
            }
            ptx::tmem_ld_wait<16>(p);
            if (piece == 1) {
              // both accumulators have been read
              ptx::tc_fence_before();
              __syncwarp();
              if (lane == 0) {
                ptx::mbar_arrive(&sh->fin_free[f]);
                if (run) ptx::mbar_arrive(&sh->rawr_free);
              }
            }
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              uint4 res4 = make_uint4(0u, 0u, 0u, 0u);
              if (res_row) res4 = __ldg((const uint4*)(res_row + piece * 16 + q * 8));
              const uint32_t resw[4] = {res4.x, res4.y, res4.z, res4.w};
              uint32_t packed[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int jx = q * 8 + e * 2;
                const float4 k0 = s_k[cb + jx], k1 = s_k[cb + jx + 1];
                const bool f0 = (bits >> jx) & 1u, f1 = (bits >> (jx + 1)) & 1u;
                const float p0 = __uint_as_float(p[jx]), p1 = __uint_as_float(p[jx + 1]);
                // Eq. 1: the full sum P+R where the gate fired, the partial sum elsewhere, each under
                // the batch norm of its path (Section 4) as one fused multiply-add
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
              const int c16 = (cb >> 3) + q;
              *(uint4*)(st + ((c16 ^ (i & 7)) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            }
          }
          if (run) ++r_use;
        }
        ptx::fence_proxy_async();
        // the store of the job before last (the other staging tile was this job's) has long finished
        // reading; after the barrier every warp may overwrite that tile
        if (ct == 0) ptx::tma_store_wait_read();
        ptx::named_bar_sync(1, kCombThreads);
        if (*(volatile uint32_t*)&sh->abort_flag) { ok = false; break; }
        if (ct == 0) {
          ptx::tma_store_4d(&map_y, buf, 0, 0, h0, n0);
          ptx::tma_store_commit();
        }
      }
      if (ct == 0) ptx::tma_store_wait_all();
    }

    // counters of this CTA
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) st_active += __shfl_xor_sync(0xffffffffu, st_active, o);
    if (lane == 0 && ok) {
      if (gate_group) atomicAdd(&prm.counters[CNT_ACTIVE], st_active);
      if (half == 0) atomicAdd(&prm.counters[gate_group ? CNT_ROWS_TOTAL : CNT_ROWS_ACTIVE], st_rows);
    }
    if (!gate_group && ct == 0 && ok) {
      const unsigned long long k_p = 9ull * L.c_p, k_r = 9ull * L.c_r;
      if (blockIdx.x == 0) atomicAdd(&prm.counters[CNT_CALLS], 1ull);
      atomicAdd(&prm.counters[CNT_TILES_TOTAL], (unsigned long long)jobs);
      atomicAdd(&prm.counters[CNT_TILES_SKIPPED], has_cond ? (unsigned long long)jobs - r_use : 0ull);
      atomicAdd(&prm.counters[CNT_EXEC_MACS], 128ull * 64ull * (k_p * jobs + k_r * r_use));
    }
  }
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
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// NHWC bf16 tensor of 64 channels, boxes of `box_h` whole image rows, 128-byte swizzle
bool encode_rows(CUtensorMap* map, const void* base, const LayerDims& L, int box_h) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {64, (cuuint64_t)L.w, (cuuint64_t)L.h, (cuuint64_t)L.n};
  const cuuint64_t str[3] = {128, (cuuint64_t)L.w * 128, (cuuint64_t)L.h * L.w * 128};
  const cuuint32_t box[4] = {64, (cuuint32_t)L.w, (cuuint32_t)box_h, 1};
  const cuuint32_t es[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, str, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tc3_plan(const LayerDims& L, int in_dtype, int cond_mode, int sms, Tc3Plan* plan) {
  Tc3Plan P;
  std::memset(&P, 0, sizeof(P));
  *plan = P;
  if (in_dtype != CG_BF16) return false;
  if (L.kh != 3 || L.kw != 3 || L.stride != 1 || L.pad != 1) return false;
  if (L.c_in != 64 || L.c_out != 64) return false;
  if (L.c_p % 16 != 0) return false;                       // whole K steps per path
  if (L.grouping && L.groups > 1) return false;
  if (L.channel_tau > 0.f) return false;
  if (cond_mode == CG_COND_COMPACT) return false;
  if (L.w != 8 && L.w != 16 && L.w != 32) return false;   // a TMEM lane quadrant holds whole image rows
  P.rows = 128 / L.w;
  P.tiles_per_image = (L.h + P.rows - 1) / P.rows;
  const long long jobs = (long long)L.n * P.tiles_per_image;
  if (jobs > 0x7fffffffll) return false;
  P.jobs = (int)jobs;
  P.kp = L.c_p / 16;
  P.cond_mode = cond_mode == CG_COND_AUTO ? CG_COND_SKIP_TILES : cond_mode;
  P.grid = (int)(jobs < sms ? jobs : sms);
  P.valid = 1;
  *plan = P;
  return true;
}

int launch_tc3(const LayerDims& L, const Tc3Plan& P, Tc3Maps* maps, const void* x, const void* w_base,
               const void* w_cond, const cg_bn_params& bn, const float* delta, const void* residual, void* y,
               uint32_t* mask, unsigned long long* counters, cudaStream_t stream) {
  if (!P.valid) return (int)cudaErrorInvalidValue;
  Tc3MapSet* ms = nullptr;
  for (int i = 0; i < Tc3Maps::kEntries; ++i) {
    Tc3MapSet* c = &maps->set[i];
    if (c->key[0] == x && c->key[1] == y) { ms = c; break; }
  }
  if (!ms) {
    ms = &maps->set[maps->next];
    maps->next = (maps->next + 1) % Tc3Maps::kEntries;
    ms->key[0] = nullptr;
    if (!encode_rows(&ms->x, x, L, P.rows + 2)) return (int)cudaErrorInvalidValue;
    if (!encode_rows(&ms->y, y, L, P.rows)) return (int)cudaErrorInvalidValue;
    ms->key[0] = x; ms->key[1] = y;
  }
  Tc3Params prm;
  prm.L = L; prm.P = P; prm.bn = bn; prm.delta = delta;
  prm.w_base = static_cast<const __nv_bfloat16*>(w_base);
  prm.w_cond = static_cast<const __nv_bfloat16*>(w_cond);
  prm.residual = static_cast<const __nv_bfloat16*>(residual);
  prm.mask = mask; prm.counters = counters;
  static bool attr_set[64] = {};   // (the attribute is per device)
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return (int)cudaErrorInvalidDevice;
  if (!attr_set[dev]) {
    const cudaError_t e = cudaFuncSetAttribute(tc3_gated_conv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               227 * 1024);
    if (e != cudaSuccess) return (int)e;
    attr_set[dev] = true;
  }
  static_assert(kSmemUsed + 1024 <= 227 * 1024, "shared memory");
  // The same (maximum) amount of dynamic shared memory as the other layer kernels, so that
  // consecutive layers never reconfigure the SM; a programmatic dependent launch: the CTAs set up
  // barriers and TMEM while the previous kernel in the stream drains, and wait for it
  // (griddepcontrol.wait) before they touch global memory.
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)P.grid, 1, 1);
  cfg.blockDim = dim3((unsigned)kT3Threads, 1, 1);
  cfg.dynamicSmemBytes = 227 * 1024;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, tc3_gated_conv_kernel, ms->x, ms->y, prm);
  if (e != cudaSuccess) return (int)e;
  return (int)cudaGetLastError();
}

}  // namespace cg
