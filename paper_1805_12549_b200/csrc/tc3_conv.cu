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
// instead of 36 of N = 64 and a tile is up to 128 REAL pixels (no pad columns on the M side).  When W
// divides 32 a TMEM lane quadrant holds whole image rows and no value crosses a warp; otherwise the
// first and last lane of a warp get their neighbour's value from the adjacent quadrant's warp through
// shared memory (one named barrier among the four warps that share a channel group, per path).
//
// Per job (floor(128 / W) output rows of one image), following Section 3.1 and Eq. 1-3:
//   base path    raw P = the three D_s over the base channels (TMEM columns [0,192));
//   conditional  raw R over the remaining channels (TMEM columns [192,384)), issued right behind the
//                base path; with CG_COND_SKIP_TILES only once the gate is known, and not at all if no
//                gate of the job fired;
//   epilogue     16 warps (TMEM lane quadrant x 16 channels), all on the same job: raw P -> registers
//                (raw P is free for the next job at once), P = shifted sum, d = (P >= t[c]) (and
//                P <= t2[c] for the two-sided gate of Section 3.2) -> mask bits; raw R -> registers,
//                R = shifted sum; y = f(BN1(P)) or f(BN2(P+R)) by mask bit, staged in shared memory
//                (a ring of three tiles) and written by one TMA store.  P never leaves the registers.
// Weights are resident in shared memory: every CTA builds the three 192-row tiles itself with plain
// loads (row (s,c) = the 64 input channels of tap (r,s): base channels first, as in x).
//
// Warp roles: 0 = patch producer, 1 = MMA issuer of the base path (owns TMEM), 2 = y and mask stores,
// 3 = MMA issuer of the conditional path, 4-19 = epilogue; warps 2-19 build the weight tiles first.  Every mbarrier wait is bounded; on expiry the CTA records CG_ERR_DEVICE_TIMEOUT with the
// id of the wait and leaves.
#include <cstring>

#include "ptx.cuh"
#include "tc3_conv.cuh"

namespace cg {

namespace {

constexpr int kT3Threads = 640;
constexpr int kStoreWarp = 2;
constexpr int kCondWarp = 3;                     // second MMA issuer (conditional path)
constexpr int kEpiWarp0 = 4, kEpiWarps = 16;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kLoaderWarps = 18;                 // warps 2-19 build the weight tiles
constexpr int kMaxNA = 4;                        // patch buffers, at most
constexpr int kWTileBytes = 192 * 128;           // one filter row: 3 taps x 64 output channels
constexpr int kStageBytes = 128 * 128;           // y staging tile
constexpr int kNY = 3;                           // staging tiles
constexpr uint32_t kColRawP = 0, kColRawR = 192;   // TMEM columns
constexpr int kSpinLimit = 1 << 21;
constexpr long long kWaitCycles = 2000000000ll;

// shared-memory map (offsets from a 1024-byte-aligned base)
constexpr unsigned kOffW = 0;
constexpr unsigned kOffY = kOffW + 3 * kWTileBytes;
constexpr unsigned kOffMask = kOffY + kNY * kStageBytes;       // [kNY][128][4] mask bits, 16 per epilogue warp
constexpr unsigned kOffConsts = kOffMask + kNY * 128 * 4 * 2;   // t[64], t2[64], {a1,b1,a2,b2}[64]
constexpr unsigned kOffBar = kOffConsts + 64 * 4 * 2 + 64 * 16;
constexpr unsigned kOffXch = kOffBar + 512;   // [2 paths][2 directions][4 quadrants][4 channel groups][16] floats
constexpr unsigned kOffA = (kOffXch + 4096 + 1023) / 1024 * 1024;   // patch buffers: the rest
constexpr unsigned kPatchArea = 227 * 1024 - 1024 - kOffA;

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
  uint64_t a_full[kMaxNA], a_empty[kMaxNA];
  uint64_t w_ready;
  uint64_t rawp_full, rawp_free, rawr_full, rawr_free;
  uint64_t y_full[kNY], y_free[kNY];   // staging tiles (with the mask bits) of a job
  uint64_t gate_done[2];           // CG_COND_SKIP_TILES: the job's gate has been evaluated (by job parity)
  uint32_t tmem_base;
  uint32_t abort_flag;
  uint32_t fired[2][kEpiWarps];    // by job parity, per epilogue warp: a gate of its rows and channels fired
};
static_assert(sizeof(Shared3) <= 512, "barrier block");

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
// (no_a / no_b: the slot has no left / right neighbour in its image row, or the neighbour sits in another warp)
__device__ __forceinline__ float stacked_sum(uint32_t d0, uint32_t d1, uint32_t d2, bool no_a, bool no_b) {
  const float a = __uint_as_float(__shfl_up_sync(0xffffffffu, d0, 1));
  const float b = __uint_as_float(__shfl_down_sync(0xffffffffu, d2, 1));
  float v = __uint_as_float(d1);
  if (!no_a) v += a;   // (predicated adds: what wraps around the image edge is dropped, not multiplied by 0)
  if (!no_b) v += b;
  return v;
}


// kXch: the image width does not divide 32 (two instances, so that the common widths carry none of
// the exchange code)
template <bool kXch>
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
  unsigned short* s_bits = (unsigned short*)(smem + kOffMask);
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
  const int na = P.na;
  const uint32_t patch_bytes = (uint32_t)P.patch_bytes;
  float* s_xch = (float*)(smem + kOffXch);

  auto job_origin = [&](int j, int& n0, int& h0) {
    const int t = (int)blockIdx.x + j * (int)gridDim.x;
    n0 = t / P.tiles_per_image;
    h0 = (t - n0 * P.tiles_per_image) * P.rows;
  };
  auto any_fired = [&](int b) {
    const volatile uint32_t* w = sh->fired[b];
    uint32_t v = 0;
#pragma unroll
    for (int i = 0; i < kEpiWarps; ++i) v |= w[i];
    return v != 0u;
  };

  // ---------------------------------------------------------------- setup
  if (threadIdx.x == 0) {
    // (a patch is released by both issuers: each one's commit covers only its own MMAs)
    for (int i = 0; i < kMaxNA; ++i) { ptx::mbar_init(&sh->a_full[i], 1); ptx::mbar_init(&sh->a_empty[i], has_cond ? 2 : 1); }
    ptx::mbar_init(&sh->w_ready, kLoaderWarps);
    ptx::mbar_init(&sh->rawp_full, 1); ptx::mbar_init(&sh->rawp_free, kEpiWarps);
    ptx::mbar_init(&sh->rawr_full, 1); ptx::mbar_init(&sh->rawr_free, kEpiWarps);
    ptx::mbar_init(&sh->gate_done[0], kEpiWarps); ptx::mbar_init(&sh->gate_done[1], kEpiWarps);
    for (int i = 0; i < kNY; ++i) { ptx::mbar_init(&sh->y_full[i], kEpiWarps); ptx::mbar_init(&sh->y_free[i], 1); }
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
  if (warp >= kEpiWarp0) {
    const int et = (int)threadIdx.x - kEpiWarp0 * 32;
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
      const int slot = j % na;
      ok = wait3(sh, prm.counters, &sh->a_empty[slot], ((j / na) & 1) ^ 1, 1);
      if (!ok) break;
      int n0, h0;
      job_origin(j, n0, h0);
      if (lane == 0) {
        ptx::mbar_expect_tx(&sh->a_full[slot], patch_tx);
        ptx::tma_load_4d(s_a + (size_t)slot * patch_bytes, &map_x, &sh->a_full[slot], 0, 0, h0 - 1, n0);
      }
    }
  } else if (warp == 1 || warp == kCondWarp) {
    // ============================================================ MMA issuers
    // Warp 1 issues the base path of every job, warp 3 the conditional path: the two write different
    // accumulators, and a tcgen05.mma keeps the issuing warp's scheduler busy for about as long as the
    // MMA runs, so the two paths sit on different schedulers.  (Each warp whole and convergent; lane 0
    // issues.)  With CG_COND_SKIP_TILES the conditional path of a job waits for its gate.
    const uint32_t lead = lane == 0 ? 1u : 0u;
    const uint32_t desc_hi = (uint32_t)(ptx::smem_desc(0, 1024, 2) >> 32);
    const uint32_t a_base_lo = (ptx::smem_u32(s_a) >> 4) | 0x10000u;
    const uint32_t b_lo = (ptx::smem_u32(s_w) >> 4) | 0x10000u;
    const uint32_t row_lo = (uint32_t)W * 8u;
    bool ok = wait3(sh, prm.counters, &sh->w_ready, 0, 2);
    if (warp == 1) {
      for (int j = 0; j < jobs && ok; ++j) {
        const int slot = j % na;
        ok = wait3(sh, prm.counters, &sh->a_full[slot], (j / na) & 1, 3);
        ok = ok && wait3(sh, prm.counters, &sh->rawp_free, (j & 1) ^ 1, 4);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t a_lo = a_base_lo + (uint32_t)slot * (patch_bytes >> 4);
        switch (P.kp) {
          case 1: issue_rows<0, 1>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawP); break;
          case 2: issue_rows<0, 2>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawP); break;
          case 3: issue_rows<0, 3>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawP); break;
          default: issue_rows<0, 4>(lead, desc_hi, a_lo, b_lo, row_lo, tmem + kColRawP); break;
        }
        ptx::umma_commit_if(lead, &sh->rawp_full);
        ptx::umma_commit_if(lead, &sh->a_empty[slot]);
      }
    } else if (has_cond) {
      uint32_t r_use = 0;
      for (int j = 0; j < jobs && ok; ++j) {
        const int slot = j % na;
        bool run = true;
        if (!dense) {
          ok = wait3(sh, prm.counters, &sh->gate_done[j & 1], (j >> 1) & 1, 5);
          if (!ok) break;
          run = any_fired(j & 1);
        }
        if (run) {
          ok = wait3(sh, prm.counters, &sh->a_full[slot], (j / na) & 1, 12);
          ok = ok && wait3(sh, prm.counters, &sh->rawr_free, (r_use & 1) ^ 1, 6);
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t a_lo = a_base_lo + (uint32_t)slot * (patch_bytes >> 4);
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
  } else if (warp == kStoreWarp) {
    // ============================================================ store warp
    // Writes what the epilogue leaves in shared memory: the y tile (one TMA store) and the mask
    // words of the job's 128 rows (four rows per lane, each from the bits of four epilogue warps).
    // A tile goes back to the epilogue one job late, when the wait for its store to have read it
    // no longer blocks.
    unsigned long long st_rows = 0, st_rows_active = 0;
    bool ok = true;
    int b = 0, u = 0;   // j % kNY, j / kNY
    for (int j = 0; j < jobs && ok; ++j) {
      ok = wait3(sh, prm.counters, &sh->y_full[b], u & 1, 11);
      if (!ok) break;
      int n0, h0;
      job_origin(j, n0, h0);
      if (lane == 0) {
        ptx::tma_store_4d(&map_y, s_y + (size_t)b * kStageBytes, 0, 0, h0, n0);
        ptx::tma_store_commit();
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = k * 32 + lane;
        const int h_loc = i / W, col = i - h_loc * W;
        const bool valid = h_loc < P.rows && h0 + h_loc < H;
        const uint2 w2 = *(const uint2*)&s_bits[(b * 128 + i) * 4];
        if (valid && prm.mask) {
          const long long m = ((long long)n0 * H + (h0 + h_loc)) * W + col;
          prm.mask[m * 2] = w2.x; prm.mask[m * 2 + 1] = w2.y;
        }
        st_rows += valid ? 1 : 0;
        st_rows_active += (w2.x | w2.y) != 0u ? 1 : 0;
      }
      // the tile (and the bits) of the job before: its store has read them
      if (lane == 0) ptx::tma_store_wait_read_but_one();
      __syncwarp();
      if (j >= 1 && lane == 0) ptx::mbar_arrive(&sh->y_free[b == 0 ? kNY - 1 : b - 1]);
      if (++b == kNY) { b = 0; ++u; }
    }
    if (lane == 0) ptx::tma_store_wait_all();
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      st_rows += __shfl_xor_sync(0xffffffffu, st_rows, o);
      st_rows_active += __shfl_xor_sync(0xffffffffu, st_rows_active, o);
    }
    if (lane == 0 && ok) {
      atomicAdd(&prm.counters[CNT_ROWS_TOTAL], st_rows);
      atomicAdd(&prm.counters[CNT_ROWS_ACTIVE], st_rows_active);
    }
  } else if (warp >= kEpiWarp0) {
    // ============================================================ epilogue (16 warps, all on the same job)
    const int quad = warp & 3;                                   // TMEM lane quadrant
    const int cgp = (warp - kEpiWarp0) >> 2;                     // channels [16*cgp, 16*cgp + 16)
    const int cb = cgp * 16;
    const int i = quad * 32 + lane;                              // pixel slot = TMEM lane
    const int h_loc = i / W, col = i - h_loc * W;
    const bool first_col = col == 0, last_col = col == W - 1;
    // W does not divide 32: a warp's first and last lane may have their row neighbour in another warp
    constexpr bool xch = kXch;
    const bool no_a = first_col || (xch && lane == 0), no_b = last_col || (xch && lane == 31);
    const bool fix_a = xch && lane == 0 && !first_col, fix_b = xch && lane == 31 && !last_col && quad < 3;
    // exchange cells, 16 floats each: [path][direction][quadrant][group]; direction 0 = D_0 of the
    // quadrant's last slot (for the next quadrant's first lane), 1 = D_2 of its first slot
    float* x_cell = s_xch + (quad * 4 + cgp) * 16;
    constexpr int kXDir = 256, kXPath = 512, kXQuad = 64;   // strides in floats
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const int et = (int)threadIdx.x - kEpiWarp0 * 32;            // thread index within the group
    unsigned long long st_active = 0;
    uint32_t r_use = 0;
    bool ok = true;
    int b = 0, u = 0;   // j % kNY, j / kNY
    for (int j = 0; j < jobs && ok; ++j, b = (b + 1 == kNY ? 0 : b + 1), u += (b == 0 ? 1 : 0)) {
      uint8_t* buf = s_y + (size_t)b * kStageBytes;
      int n0, h0;
      job_origin(j, n0, h0);
      const bool valid = h_loc < P.rows && h0 + h_loc < H;
      const long long m = ((long long)n0 * H + (h0 + h_loc)) * W + col;
      // residual values (the shortcut of a residual block, added before the activation): fetched early
      uint4 res[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
      const bool has_res = prm.residual != nullptr && valid;
      if (has_res) {
        const uint4* rp = (const uint4*)(prm.residual + m * 64 + cb);
        res[0] = __ldg(rp); res[1] = __ldg(rp + 1);
      }
      ok = wait3(sh, prm.counters, &sh->rawp_full, j & 1, 7);
      if (!ok) break;
      uint32_t p[16];
      uint32_t bits = 0;
      {
        ptx::tc_fence_after();
        uint32_t d0[16], d1[16], d2[16];
        ptx::tmem_ld_nowait<16>(t_lane + kColRawP + (uint32_t)cb, d0);
        ptx::tmem_ld_nowait<16>(t_lane + kColRawP + 64u + (uint32_t)cb, d1);
        ptx::tmem_ld_nowait<16>(t_lane + kColRawP + 128u + (uint32_t)cb, d2);
        // (while the loads are in flight) the store warp must be done with this staging tile and its bits
        ok = wait3(sh, prm.counters, &sh->y_free[b], (u & 1) ^ 1, 10);
        ptx::tmem_ld_wait<16>(d0);
        ptx::tmem_ld_wait<16>(d1);
        ptx::tmem_ld_wait<16>(d2);
        // raw P is in registers: the base path of the next job may overwrite it
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh->rawp_free);
        if (xch) {
          if (lane == 31) {
#pragma unroll
            for (int c = 0; c < 16; ++c) x_cell[c] = __uint_as_float(d0[c]);
          }
          if (lane == 0) {
#pragma unroll
            for (int c = 0; c < 16; ++c) x_cell[kXDir + c] = __uint_as_float(d2[c]);
          }
          ptx::named_bar_sync(3 + cgp, 128);
        }
#pragma unroll
        for (int c = 0; c < 16; ++c) p[c] = __float_as_uint(stacked_sum(d0[c], d1[c], d2[c], no_a, no_b));
        if (fix_a) {
#pragma unroll
          for (int c = 0; c < 16; ++c) p[c] = __float_as_uint(__uint_as_float(p[c]) + x_cell[c - kXQuad]);
        }
        if (fix_b) {
#pragma unroll
          for (int c = 0; c < 16; ++c) p[c] = __float_as_uint(__uint_as_float(p[c]) + x_cell[kXDir + kXQuad + c]);
        }
        // Eq. 2-3 with the batch norm folded into the threshold: d = (P >= t), a compare and a
        // predicated bit insert per channel (a NaN sum does not fire); four partial words, so that the
        // inserts do not form one dependent chain
        uint32_t pw[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 t4 = *(const float4*)(s_t + cb + q * 4);
          if (__uint_as_float(p[q * 4 + 0]) >= t4.x) pw[q] |= 1u << (q * 4 + 0);
          if (__uint_as_float(p[q * 4 + 1]) >= t4.y) pw[q] |= 1u << (q * 4 + 1);
          if (__uint_as_float(p[q * 4 + 2]) >= t4.z) pw[q] |= 1u << (q * 4 + 2);
          if (__uint_as_float(p[q * 4 + 3]) >= t4.w) pw[q] |= 1u << (q * 4 + 3);
        }
        bits = (pw[0] | pw[1]) | (pw[2] | pw[3]);
        if (two_sided) {
          // Section 3.2: the gate also needs P <= the upper threshold (ties included)
          uint32_t ph[4] = {0u, 0u, 0u, 0u};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float4 u4 = *(const float4*)(s_t2 + cb + q * 4);
            if (__uint_as_float(p[q * 4 + 0]) <= u4.x) ph[q] |= 1u << (q * 4 + 0);
            if (__uint_as_float(p[q * 4 + 1]) <= u4.y) ph[q] |= 1u << (q * 4 + 1);
            if (__uint_as_float(p[q * 4 + 2]) <= u4.z) ph[q] |= 1u << (q * 4 + 2);
            if (__uint_as_float(p[q * 4 + 3]) <= u4.w) ph[q] |= 1u << (q * 4 + 3);
          }
          bits &= (ph[0] | ph[1]) | (ph[2] | ph[3]);
        }
        if (!valid) bits = 0;
        if (!ok) break;
        s_bits[(b * 128 + i) * 4 + cgp] = (unsigned short)bits;
        st_active += __popc(bits);
      }
      const uint32_t warp_any = __ballot_sync(0xffffffffu, bits != 0u);
      bool run = has_cond;
      if (!dense && has_cond) {
        // the issuer (and this group) must know whether any gate of the job fired
        if (lane == 0) sh->fired[j & 1][warp - kEpiWarp0] = warp_any;
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&sh->gate_done[j & 1]);
        ok = wait3(sh, prm.counters, &sh->gate_done[j & 1], (j >> 1) & 1, 8);
        if (!ok) break;
        run = any_fired(j & 1);
      }
      // R is read only where the conditional path ran and a gate of these rows and channels fired
      const bool have_r = run && (warp_any != 0u || xch);   // (with the exchange, the neighbours need this warp's R)
      uint32_t rr[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) rr[c] = 0u;
      if (xch && !run) ptx::named_bar_sync(3 + cgp, 128);
      if (run) {
        ok = wait3(sh, prm.counters, &sh->rawr_full, r_use & 1, 9);
        if (!ok) break;
        {
          ptx::tc_fence_after();
          if (have_r) {
            uint32_t e0[16], e1[16], e2[16];
            ptx::tmem_ld_nowait<16>(t_lane + kColRawR + (uint32_t)cb, e0);
            ptx::tmem_ld_nowait<16>(t_lane + kColRawR + 64u + (uint32_t)cb, e1);
            ptx::tmem_ld_nowait<16>(t_lane + kColRawR + 128u + (uint32_t)cb, e2);
            ptx::tmem_ld_wait<16>(e0);
            ptx::tmem_ld_wait<16>(e1);
            ptx::tmem_ld_wait<16>(e2);
            if (xch) {
              // (second half of the exchange cells; the barrier also orders this job's reads of the
              // first half before the next job's writes)
              if (lane == 31) {
#pragma unroll
                for (int c = 0; c < 16; ++c) x_cell[kXPath + c] = __uint_as_float(e0[c]);
              }
              if (lane == 0) {
#pragma unroll
                for (int c = 0; c < 16; ++c) x_cell[kXPath + kXDir + c] = __uint_as_float(e2[c]);
              }
              ptx::named_bar_sync(3 + cgp, 128);
            }
#pragma unroll
            for (int c = 0; c < 16; ++c) rr[c] = __float_as_uint(stacked_sum(e0[c], e1[c], e2[c], no_a, no_b));
            if (fix_a) {
#pragma unroll
              for (int c = 0; c < 16; ++c) rr[c] = __float_as_uint(__uint_as_float(rr[c]) + x_cell[kXPath - kXQuad + c]);
            }
            if (fix_b) {
#pragma unroll
              for (int c = 0; c < 16; ++c) rr[c] = __float_as_uint(__uint_as_float(rr[c]) + x_cell[kXPath + kXDir + kXQuad + c]);
            }
          }
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&sh->rawr_free);
          ++r_use;
        }
      }
      {
        uint8_t* st = buf + (size_t)i * 128;   // (128-byte swizzle: 16-byte piece c16 of row i at c16 ^ (i & 7))
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const uint32_t resw[4] = {res[q].x, res[q].y, res[q].z, res[q].w};
          uint32_t packed[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int jx = q * 8 + e * 2;
            const float4 k0 = s_k[cb + jx], k1 = s_k[cb + jx + 1];
            const bool f0 = (bits >> jx) & 1u, f1 = (bits >> (jx + 1)) & 1u;
            const float p0 = __uint_as_float(p[jx]), p1 = __uint_as_float(p[jx + 1]);
            // Eq. 1: the full sum P+R where the gate fired, the partial sum elsewhere, each under the
            // batch norm of its path (Section 4) as one fused multiply-add
            const float o0 = fmaf(k0.z, p0 + __uint_as_float(rr[jx]), k0.w), c0 = fmaf(k0.x, p0, k0.y);
            const float o1 = fmaf(k1.z, p1 + __uint_as_float(rr[jx + 1]), k1.w), c1 = fmaf(k1.x, p1, k1.y);
            float v0 = f0 ? o0 : c0;
            float v1 = f1 ? o1 : c1;
            if (has_res) {
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
      ptx::fence_proxy_async();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&sh->y_full[b]);
    }

    // counters of this CTA
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) st_active += __shfl_xor_sync(0xffffffffu, st_active, o);
    if (lane == 0 && ok) atomicAdd(&prm.counters[CNT_ACTIVE], st_active);
    if (et == 0 && ok) {
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
  if (L.w > 128) return false;                             // a job is at least one whole image row
  P.rows = 128 / L.w;
  P.xch = (32 % L.w) != 0;                                  // image rows do not line up with the warps
  // a patch: the job's rows plus one above and one below, and what the last filter row's 128-slot
  // window reaches behind them
  P.patch_bytes = (int)(((size_t)(128 + 2 * L.w) * 128 + 1023) / 1024 * 1024);
  P.na = (int)(kPatchArea / (unsigned)P.patch_bytes);
  if (P.na > kMaxNA) P.na = kMaxNA;
  if (P.na < 2) return false;
  P.tiles_per_image = (L.h + P.rows - 1) / P.rows;
  const long long jobs = (long long)L.n * P.tiles_per_image;
  if (jobs > 0x7fffffffll) return false;
  P.jobs = (int)jobs;
  P.kp = L.c_p / 16;
  // CG_COND_AUTO: the conditional path is issued right behind the base path.  A job is 128 pixels x
  // 64 channels: at any useful density some gate of it fires, and waiting for the gate before the
  // conditional MMAs serialises the job (measured: 1.6x the time).
  P.cond_mode = cond_mode == CG_COND_SKIP_TILES ? CG_COND_SKIP_TILES : CG_COND_DENSE;
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
  static bool attr_set[64][2] = {};   // (the attribute is per device and kernel instance)
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return (int)cudaErrorInvalidDevice;
  typedef void (*Kernel)(CUtensorMap, CUtensorMap, Tc3Params);
  const Kernel kernel = P.xch ? (Kernel)tc3_gated_conv_kernel<true> : (Kernel)tc3_gated_conv_kernel<false>;
  if (!attr_set[dev][P.xch ? 1 : 0]) {
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return (int)e;
    attr_set[dev][P.xch ? 1 : 0] = true;
  }
  static_assert(kPatchArea >= 2 * (128 + 2 * 128) * 128, "shared memory");
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
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, ms->x, ms->y, prm);
  if (e != cudaSuccess) return (int)e;
  return (int)cudaGetLastError();
}

}  // namespace cg
