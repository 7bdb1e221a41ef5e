// Channel-gated convolution on tcgen05 tensor cores: one fused kernel per layer.
//
// "Shifted-window" implicit GEMM (stride-1, k = 2*pad+1 convolutions).  A CTA owns a tile of up
// to 128 output pixels that are whole image rows (or whole small images) and NT output
// channels.  The input patch of the tile -- the rows it needs plus the zero padding, which TMA
// out-of-bounds fill provides -- is loaded ONCE per 64-channel chunk into shared memory as
// [pixel][64 channels] rows of 128 bytes (128-byte swizzle).  Rows are laid out with pitch
// W+pad, so that the right padding of one image row is the left padding of the next; then the
// A operand of filter tap (r,s) is simply the same buffer read from row r*(W+pad)+s onwards:
// output pixel i reads patch pixel i + r*(W+pad) + s.  Nine MMAs per K-slice reuse one patch;
// only the weights stream through a TMA ring.
//
// Per tile, following the paper's block (Section 3.1, Eq. 1-3, Section 4):
//   1. base path   P = W_p * x_p : MMAs over the base channels, fp32 accumulator in TMEM;
//   2. gate        d = (P >= t[c]) read from TMEM by the epilogue warps -> mask words, counts,
//                  y_base = f(BN1(P)) staged in shared memory;
//   3. conditional R = W_r * x_r accumulated ONTO P in the same TMEM columns, only for the
//                  64-channel column blocks in which a gate fired (whole tile skipped if none);
//   4. combine     where d = 1 the staged value is replaced by f(BN2(P+R)); one TMA store.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM), warps 2-5 = epilogue.
// Every mbarrier wait is bounded; on expiry the CTA records CG_ERR_DEVICE_TIMEOUT and leaves.
#include <cstring>

#include "ptx.cuh"
#include "tc_conv.cuh"

namespace cg {

namespace {

constexpr int kThreads = 192;
constexpr int kBM = 128;            // MMA M: patch rows per tile
constexpr int kSpinLimit = 1 << 22; // try_wait polls before a wait gives up

struct TcParams {
  LayerDims L;
  TcPlan P;
  cg_bn_params bn;
  const float* delta;
  uint32_t* mask;
  unsigned long long* counters;
};

// One weight tile of the ring: 64 K-elements of NT output channels.
struct WTile {
  int x;        // K coordinate in the weight matrix
  int chunk;    // patch buffer it multiplies
  int t0, ntap; // filter taps covered
  int a_k0;     // first 16-element K step inside the patch row
  int nks;      // K steps per tap
  int b_step;   // K steps between consecutive taps inside the weight tile
};

__device__ __forceinline__ WTile base_tile(const LayerDims& L, int bt) {
  const int taps = L.kh * L.kw;
  WTile w;
  if (L.c_p >= 64) {
    const int q = bt / taps, t = bt - q * taps;
    w = {t * L.c_p + 64 * q, q, t, 1, 0, 4, 0};
  } else {
    const int tpt = 64 / L.c_p;
    const int t0 = bt * tpt;
    w = {bt * 64, 0, t0, min(tpt, taps - t0), 0, L.c_p / 16, L.c_p / 16};
  }
  return w;
}

__device__ __forceinline__ WTile cond_tile(const LayerDims& L, int bt) {
  const int taps = L.kh * L.kw;
  WTile w;
  if (L.c_p >= 64) {
    const int q = L.c_p / 64 + bt / taps, t = bt % taps;
    w = {t * L.c_r + 64 * q - L.c_p, q, t, 1, 0, 4, 0};
  } else if (bt < taps) {
    w = {bt * L.c_r, 0, bt, 1, L.c_p / 16, 4 - L.c_p / 16, 0};
  } else {
    const int b2 = bt - taps;
    const int q = 1 + b2 / taps, t = b2 % taps;
    w = {t * L.c_r + 64 * q - L.c_p, q, t, 1, 0, 4, 0};
  }
  return w;
}

struct Shared {
  uint64_t a_full[8];
  uint64_t b_full[8];
  uint64_t b_empty[8];
  uint64_t base_done, gate_done, cond_done;
  uint32_t tmem_base;
  uint32_t blk_active;      // bit b: a gate fired in column block b (64 channels)
  uint32_t abort_flag;
  uint32_t n_active, n_rows_valid, n_rows_active;
};

__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Shared* sh,
                                         unsigned long long* counters, int site) {
  for (int i = 0; i < kSpinLimit; ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 1023) == 1023 && *(volatile uint32_t*)&sh->abort_flag) return false;
  }
  if (atomicCAS(&counters[CNT_STATUS], 0ull, (unsigned long long)CG_ERR_DEVICE_TIMEOUT) == 0ull)
    atomicExch(&counters[CNT_SITE], (unsigned long long)site);
  atomicExch(&sh->abort_flag, 1u);
  return false;
}

template <int NT>
__global__ void __launch_bounds__(kThreads, 1)
tc_gated_conv_kernel(const __grid_constant__ CUtensorMap map_x,
                     const __grid_constant__ CUtensorMap map_wb,
                     const __grid_constant__ CUtensorMap map_wc,
                     const __grid_constant__ CUtensorMap map_y,
                     const __grid_constant__ TcParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const LayerDims& L = prm.L;
  const TcPlan& P = prm.P;
  uint8_t* s_a = smem + P.off_a;
  uint8_t* s_b = smem + P.off_b;
  uint8_t* s_y = smem + P.off_y;
  float* s_t = (float*)(smem + P.off_consts);
  float* s_a1 = s_t + NT;
  float* s_b1 = s_a1 + NT;
  float* s_a2 = s_b1 + NT;
  float* s_b2 = s_a2 + NT;
  Shared* sh = (Shared*)(smem + P.off_bar);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_n = blockIdx.x % P.tiles_n;
  const int tile_m = blockIdx.x / P.tiles_n;
  int n0, h0;
  if (P.images_mode) { n0 = tile_m * P.ni; h0 = 0; }
  else { n0 = tile_m / P.tiles_per_image; h0 = (tile_m - n0 * P.tiles_per_image) * P.r; }
  const int taps = L.kh * L.kw;
  const bool dense = (P.cond_mode == CG_COND_DENSE);
  constexpr int kBlocks = NT / 64;                       // column blocks of the conditional path
  constexpr uint32_t kAllBlocks = (1u << kBlocks) - 1u;
  const uint32_t b_tile_bytes = NT * 128;

  // ---------------------------------------------------------------- setup
  if (threadIdx.x == 0) {
    for (int i = 0; i < P.chunks; ++i) ptx::mbar_init(&sh->a_full[i], 1);
    for (int i = 0; i < P.stages; ++i) { ptx::mbar_init(&sh->b_full[i], 1); ptx::mbar_init(&sh->b_empty[i], 1); }
    ptx::mbar_init(&sh->base_done, 1);
    ptx::mbar_init(&sh->gate_done, 128);
    ptx::mbar_init(&sh->cond_done, 1);
    sh->blk_active = 0; sh->abort_flag = 0; sh->n_active = 0; sh->n_rows_valid = 0; sh->n_rows_active = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&map_x); ptx::prefetch_tensormap(&map_wb);
    ptx::prefetch_tensormap(&map_wc); ptx::prefetch_tensormap(&map_y);
  }
  if (warp == 1) ptx::tmem_alloc(&sh->tmem_base, NT);
  if (warp >= 2) {
    // zero the patch rows behind the TMA box: they stand for the last row's right padding
    const int tail0 = P.box_pixels * 128, tail1 = P.patch_rows * 128;
    for (int q = 0; q < P.chunks; ++q) {
      uint8_t* base = s_a + (size_t)q * P.patch_bytes;
      for (int o = tail0 + (threadIdx.x - 64) * 16; o < tail1; o += 128 * 16)
        *(uint4*)(base + o) = make_uint4(0, 0, 0, 0);
    }
    for (int c = threadIdx.x - 64; c < NT; c += 128) {
      const int cg_ = tile_n * NT + c;
      if (cg_ < L.c_out) {
        const ChannelConsts k = fold_channel(prm.bn, prm.delta, L.eps, cg_);
        s_t[c] = k.t; s_a1[c] = k.a1; s_b1[c] = k.b1; s_a2[c] = k.a2; s_b2[c] = k.b2;
      } else {
        s_t[c] = __int_as_float(0x7f800000); s_a1[c] = 0.f; s_b1[c] = 0.f; s_a2[c] = 0.f; s_b2[c] = 0.f;
      }
    }
    ptx::fence_proxy_async();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = sh->tmem_base;

  if (warp == 0) {
    // ============================================================ TMA producer
    if (lane == 0) {
      do {
        const uint32_t patch_tx = (uint32_t)P.box_pixels * 128u;
        for (int q = 0; q < P.base_chunks; ++q) {
          ptx::mbar_expect_tx(&sh->a_full[q], patch_tx);
          ptx::tma_load_4d(s_a + (size_t)q * P.patch_bytes, &map_x, &sh->a_full[q], q * 64, -L.pad,
                           h0 - L.pad, n0);
        }
        if (dense) {
          for (int q = P.base_chunks; q < P.chunks; ++q) {
            ptx::mbar_expect_tx(&sh->a_full[q], patch_tx);
            ptx::tma_load_4d(s_a + (size_t)q * P.patch_bytes, &map_x, &sh->a_full[q], q * 64,
                             -L.pad, h0 - L.pad, n0);
          }
        }
        int it = 0;
        bool ok = true;
        for (int bt = 0; bt < P.base_tiles && ok; ++bt, ++it) {
          const int s = it % P.stages;
          ok = wait_bar(&sh->b_empty[s], ((it / P.stages) & 1) ^ 1, sh, prm.counters, 1);
          if (!ok) break;
          const WTile w = base_tile(L, bt);
          ptx::mbar_expect_tx(&sh->b_full[s], b_tile_bytes);
          ptx::tma_load_2d(s_b + (size_t)s * b_tile_bytes, &map_wb, &sh->b_full[s], w.x, tile_n * NT);
        }
        if (!ok || P.cond_tiles == 0) break;
        uint32_t blocks = kAllBlocks;
        if (!dense) {
          if (!wait_bar(&sh->gate_done, 0, sh, prm.counters, 2)) break;
          blocks = *(volatile uint32_t*)&sh->blk_active;
          if (blocks == 0) break;
          for (int q = P.base_chunks; q < P.chunks; ++q) {
            ptx::mbar_expect_tx(&sh->a_full[q], patch_tx);
            ptx::tma_load_4d(s_a + (size_t)q * P.patch_bytes, &map_x, &sh->a_full[q], q * 64,
                             -L.pad, h0 - L.pad, n0);
          }
        }
        for (int bt = 0; bt < P.cond_tiles && ok; ++bt, ++it) {
          const int s = it % P.stages;
          ok = wait_bar(&sh->b_empty[s], ((it / P.stages) & 1) ^ 1, sh, prm.counters, 3);
          if (!ok) break;
          const WTile w = cond_tile(L, bt);
          ptx::mbar_expect_tx(&sh->b_full[s], b_tile_bytes);
          ptx::tma_load_2d(s_b + (size_t)s * b_tile_bytes, &map_wc, &sh->b_full[s], w.x, tile_n * NT);
        }
      } while (0);
    }
    __syncwarp();
  } else if (warp == 1) {
    // ============================================================ MMA issuer
    if (lane == 0) {
      do {
        const uint32_t a_base = ptx::smem_u32(s_a);
        const uint32_t b_base = ptx::smem_u32(s_b);
        int it = 0;
        bool ok = true;
        uint32_t chunk_ready = 0;
        uint32_t first = 1;
        for (int bt = 0; bt < P.base_tiles && ok; ++bt, ++it) {
          const WTile w = base_tile(L, bt);
          if (!((chunk_ready >> w.chunk) & 1u)) {
            ok = wait_bar(&sh->a_full[w.chunk], 0, sh, prm.counters, 4);
            if (!ok) break;
            chunk_ready |= 1u << w.chunk;
          }
          const int s = it % P.stages;
          ok = wait_bar(&sh->b_full[s], (it / P.stages) & 1, sh, prm.counters, 5);
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t a_chunk = a_base + (uint32_t)w.chunk * P.patch_bytes;
          const uint32_t b_stage = b_base + (uint32_t)s * b_tile_bytes;
          for (int j = 0; j < w.ntap; ++j) {
            const int t = w.t0 + j;
            const uint32_t shift = (uint32_t)((t / L.kw) * P.wp + (t % L.kw)) * 128u;
            for (int ks = 0; ks < w.nks; ++ks) {
              const uint64_t da = ptx::smem_desc(a_chunk + shift + (uint32_t)(w.a_k0 + ks) * 32u, 1024, 2);
              const uint64_t db = ptx::smem_desc(b_stage + (uint32_t)(j * w.b_step + ks) * 32u, 1024, 2);
              ptx::umma_bf16(tmem, da, db, ptx::idesc_bf16(kBM, NT), first ? 0u : 1u);
              first = 0;
            }
          }
          ptx::umma_commit(&sh->b_empty[s]);
        }
        if (!ok) break;
        ptx::umma_commit(&sh->base_done);
        if (P.cond_tiles == 0) break;
        // P must have been read by the gate before R is accumulated onto it
        if (!wait_bar(&sh->gate_done, 0, sh, prm.counters, 6)) break;
        ptx::tc_fence_after();
        const uint32_t blocks = dense ? kAllBlocks : *(volatile uint32_t*)&sh->blk_active;
        if (blocks == 0) break;
        for (int bt = 0; bt < P.cond_tiles && ok; ++bt, ++it) {
          const WTile w = cond_tile(L, bt);
          if (!((chunk_ready >> w.chunk) & 1u)) {
            ok = wait_bar(&sh->a_full[w.chunk], 0, sh, prm.counters, 7);
            if (!ok) break;
            chunk_ready |= 1u << w.chunk;
          }
          const int s = it % P.stages;
          ok = wait_bar(&sh->b_full[s], (it / P.stages) & 1, sh, prm.counters, 8);
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t a_chunk = a_base + (uint32_t)w.chunk * P.patch_bytes;
          const uint32_t b_stage = b_base + (uint32_t)s * b_tile_bytes;
          const int t = w.t0;
          const uint32_t shift = (uint32_t)((t / L.kw) * P.wp + (t % L.kw)) * 128u;
          for (int ks = 0; ks < w.nks; ++ks) {
            const uint32_t a_addr = a_chunk + shift + (uint32_t)(w.a_k0 + ks) * 32u;
            const uint32_t b_addr = b_stage + (uint32_t)ks * 32u;
            if (blocks == kAllBlocks) {
              ptx::umma_bf16(tmem, ptx::smem_desc(a_addr, 1024, 2), ptx::smem_desc(b_addr, 1024, 2),
                             ptx::idesc_bf16(kBM, NT), 1u);
            } else {
#pragma unroll
              for (int b = 0; b < kBlocks; ++b) {
                if ((blocks >> b) & 1u)
                  ptx::umma_bf16(tmem + b * 64, ptx::smem_desc(a_addr, 1024, 2),
                                 ptx::smem_desc(b_addr + b * 64 * 128, 1024, 2),
                                 ptx::idesc_bf16(kBM, 64), 1u);
              }
            }
          }
          ptx::umma_commit(&sh->b_empty[s]);
        }
        if (!ok) break;
        ptx::umma_commit(&sh->cond_done);
      } while (0);
    }
    __syncwarp();
  } else {
    // ============================================================ epilogue (128 threads)
    const int quad = warp & 3;
    const int row = quad * 32 + lane;                      // TMEM lane = patch row i
    const int et = threadIdx.x - 64;
    // which output pixel is row i?
    const int n_loc = P.images_mode ? row / P.ip : 0;
    const int rem = P.images_mode ? row - n_loc * P.ip : row;
    const int h_loc = rem / P.wp;
    const int w_out = rem - h_loc * P.wp;
    const int rows_here = P.images_mode ? L.h : min(P.r, L.h - h0);
    const bool valid = (w_out < L.w) && (h_loc < rows_here) && (n_loc < P.ni) && (n0 + n_loc < L.n);
    const long long m = ((long long)(n0 + n_loc) * L.ho + (h0 + h_loc)) * L.wo + w_out;
    const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16);
    uint32_t words[NT / 32];
    bool alive = true;
    do {
      if (!wait_bar(&sh->base_done, 0, sh, prm.counters, 9)) { alive = false; break; }
      ptx::tc_fence_after();
      uint32_t my_active = 0;
      uint32_t my_blocks = 0;
#pragma unroll
      for (int cb = 0; cb < NT / 32; ++cb) {
        uint32_t r[32];
        ptx::tmem_ld32(t_row + cb * 32, r);
        uint32_t word = 0;
        uint32_t packed[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          const int c = cb * 32 + j;
          const float p0 = __uint_as_float(r[j]), p1 = __uint_as_float(r[j + 1]);
          word |= (p0 >= s_t[c] ? 1u : 0u) << j;
          word |= (p1 >= s_t[c + 1] ? 1u : 0u) << (j + 1);
          float v0 = __fadd_rn(__fmul_rn(s_a1[c], p0), s_b1[c]);
          float v1 = __fadd_rn(__fmul_rn(s_a1[c + 1], p1), s_b1[c + 1]);
          if (L.relu) { v0 = v0 > 0.f ? v0 : 0.f; v1 = v1 > 0.f ? v1 : 0.f; }
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
          packed[j >> 1] = *(const uint32_t*)&h2;
        }
        if (!valid) word = 0;
        words[cb] = word;
        my_active += __popc(word);
        if (word) my_blocks |= 1u << (cb >> 1);
        if (valid && prm.mask) prm.mask[m * L.words + tile_n * (NT / 32) + cb] = word;
        uint8_t* st = s_y + (size_t)(cb >> 1) * P.stage_rows * 128 + (size_t)row * 128;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int c16 = (cb & 1) * 4 + q;
          *(uint4*)(st + ((c16 ^ (row & 7)) << 4)) =
              make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
        }
      }
      // tile-level bookkeeping
      const uint32_t row_active = __ballot_sync(0xffffffffu, my_active != 0);
      const uint32_t row_valid = __ballot_sync(0xffffffffu, valid);
      uint32_t wa = my_active, wb_ = my_blocks;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        wa += __shfl_xor_sync(0xffffffffu, wa, o);
        wb_ |= __shfl_xor_sync(0xffffffffu, wb_, o);
      }
      if (lane == 0) {
        if (wa) atomicAdd(&sh->n_active, wa);
        if (wb_) atomicOr(&sh->blk_active, wb_);
        atomicAdd(&sh->n_rows_valid, __popc(row_valid));
        atomicAdd(&sh->n_rows_active, __popc(row_active));
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&sh->gate_done);
      if (P.cond_tiles > 0) {
        // every epilogue thread needs the tile-wide block mask
        if (!wait_bar(&sh->gate_done, 0, sh, prm.counters, 10)) { alive = false; break; }
        const uint32_t blocks = dense ? kAllBlocks : *(volatile uint32_t*)&sh->blk_active;
        if (blocks != 0) {
          if (!wait_bar(&sh->cond_done, 0, sh, prm.counters, 11)) { alive = false; break; }
          ptx::tc_fence_after();
#pragma unroll
          for (int cb = 0; cb < NT / 32; ++cb) {
            const uint32_t word = words[cb];
            if (__ballot_sync(0xffffffffu, word != 0) == 0) continue;   // warp-uniform: tcgen05.ld is .aligned
            uint32_t r[32];
            ptx::tmem_ld32(t_row + cb * 32, r);
            uint8_t* st = s_y + (size_t)(cb >> 1) * P.stage_rows * 128 + (size_t)row * 128;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int c16 = (cb & 1) * 4 + q;
              uint4* slot = (uint4*)(st + ((c16 ^ (row & 7)) << 4));
              uint4 cur = *slot;
              uint32_t* cw = (uint32_t*)&cur;
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int j = q * 8 + e * 2;
                const int c = cb * 32 + j;
                float v0 = __fadd_rn(__fmul_rn(s_a2[c], __uint_as_float(r[j])), s_b2[c]);
                float v1 = __fadd_rn(__fmul_rn(s_a2[c + 1], __uint_as_float(r[j + 1])), s_b2[c + 1]);
                if (L.relu) { v0 = v0 > 0.f ? v0 : 0.f; v1 = v1 > 0.f ? v1 : 0.f; }
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
                const uint32_t nv = *(const uint32_t*)&h2;
                const uint32_t sel = (((word >> j) & 1u) ? 0x0000ffffu : 0u) |
                                     (((word >> (j + 1)) & 1u) ? 0xffff0000u : 0u);
                cw[e] = (cw[e] & ~sel) | (nv & sel);
              }
              *slot = cur;
            }
          }
        }
      }
    } while (0);
    // staged tile -> global: one TMA store per 64-channel block
    ptx::fence_proxy_async();
    ptx::named_bar_sync(1, 128);
    if (et == 0 && alive && !*(volatile uint32_t*)&sh->abort_flag) {
#pragma unroll
      for (int b = 0; b < kBlocks; ++b) {
        if (tile_n * NT + b * 64 < L.c_out)
          ptx::tma_store_4d(&map_y, s_y + (size_t)b * P.stage_rows * 128, tile_n * NT + b * 64, 0,
                            h0, n0);
      }
      ptx::tma_store_commit();
      // counters of this tile
      const uint32_t blocks = dense ? kAllBlocks : sh->blk_active;
      const unsigned long long k_p = (unsigned long long)taps * L.c_p, k_r = (unsigned long long)taps * L.c_r;
      if (blockIdx.x == 0) atomicAdd(&prm.counters[CNT_CALLS], 1ull);
      atomicAdd(&prm.counters[CNT_ACTIVE], (unsigned long long)sh->n_active);
      atomicAdd(&prm.counters[CNT_TILES_TOTAL], (unsigned long long)kBlocks);
      atomicAdd(&prm.counters[CNT_TILES_SKIPPED], (unsigned long long)(kBlocks - __popc(blocks)));
      atomicAdd(&prm.counters[CNT_ROWS_TOTAL], (unsigned long long)sh->n_rows_valid);
      atomicAdd(&prm.counters[CNT_ROWS_ACTIVE], (unsigned long long)sh->n_rows_active);
      atomicAdd(&prm.counters[CNT_EXEC_MACS],
                (unsigned long long)kBM * NT * k_p + (unsigned long long)kBM * 64ull * __popc(blocks) * k_r);
      ptx::tma_store_wait_all();
    }
  }
  // ---------------------------------------------------------------- teardown
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

bool encode(CUtensorMap* map, void* base, int rank, const cuuint64_t* dims,
            const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, base, dims, strides_bytes, box,
            es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

bool tc_plan(const LayerDims& L, int in_dtype, int cond_mode, TcPlan* plan) {
  TcPlan P;
  std::memset(&P, 0, sizeof(P));
  *plan = P;
  if (in_dtype != CG_BF16) return false;
  if (L.has_residual) return false;
  if (L.stride != 1 || L.kh != L.kw || L.kh != 2 * L.pad + 1) return false;
  if (L.c_in % 64 != 0 || L.c_in / 64 > 8) return false;
  if (!(L.c_p == 16 || L.c_p == 32 || L.c_p % 64 == 0)) return false;
  if (L.c_out % 64 != 0) return false;
  if (L.w + L.pad > kBM) return false;
  P.elem_bytes = 2;
  P.ck = 64;
  P.wp = L.w + L.pad;
  P.ip = (L.h + L.pad) * P.wp;
  // rows of one image that fit 128 patch rows; or whole images if at least two fit
  const int last_valid_one_image = (L.h - 1) * P.wp + L.w - 1;
  if (last_valid_one_image + P.ip <= kBM - 1) {
    P.images_mode = 1;
    P.ni = 1 + (kBM - 1 - last_valid_one_image) / P.ip;
    P.r = L.h;
    P.tiles_per_image = 1;
    P.tiles_m = (L.n + P.ni - 1) / P.ni;
    P.box_h = L.h + L.pad;
    P.out_box_h = L.h + L.pad;
  } else {
    P.images_mode = 0;
    P.ni = 1;
    const int rmax = kBM / P.wp;
    const int tiles = (L.h + rmax - 1) / rmax;
    P.r = (L.h + tiles - 1) / tiles;
    P.tiles_per_image = tiles;
    P.tiles_m = L.n * tiles;
    P.box_h = P.r + 2 * L.pad;
    P.out_box_h = P.r;
  }
  if (P.box_h > 256 || P.wp > 256 || P.ni > 256) return false;
  P.box_pixels = P.wp * P.box_h * P.ni;
  P.patch_rows = (int)align_up((size_t)kBM + (size_t)(L.kh - 1) * (P.wp + 1), 8);
  if (P.box_pixels > P.patch_rows) P.patch_rows = (int)align_up(P.box_pixels, 8);
  P.patch_bytes = (int)align_up((size_t)P.patch_rows * 128, 1024);
  P.chunks = L.c_in / 64;
  P.base_chunks = L.c_p >= 64 ? L.c_p / 64 : 1;
  const int taps = L.kh * L.kw;
  if (L.c_p >= 64) {
    P.base_tiles = (L.c_p / 64) * taps;
    P.cond_tiles = (P.chunks - L.c_p / 64) * taps;
  } else {
    const int tpt = 64 / L.c_p;
    P.base_tiles = (taps + tpt - 1) / tpt;
    P.cond_tiles = L.c_r > 0 ? P.chunks * taps : 0;
  }
  P.stage_rows = (int)align_up((size_t)max(kBM, P.wp * P.out_box_h * P.ni), 8);
  P.cond_mode = cond_mode == CG_COND_AUTO ? CG_COND_SKIP_TILES : cond_mode;
  if (P.cond_mode == CG_COND_COMPACT) P.cond_mode = CG_COND_SKIP_TILES;
  // widest column tile (<= 128) whose buffers fit in shared memory
  const size_t limit = 227 * 1024 - 1024;
  for (int nt = 128; nt >= 64; nt >>= 1) {
    if (L.c_out % nt != 0) continue;
    for (int stages = 4; stages >= 2; --stages) {
      size_t off = 0;
      P.off_a = (unsigned)off; off += (size_t)P.chunks * P.patch_bytes;
      P.off_b = (unsigned)off; off += (size_t)stages * nt * 128;
      P.off_y = (unsigned)off; off += align_up((size_t)(nt / 64) * P.stage_rows * 128, 1024);
      P.off_consts = (unsigned)off; off += align_up((size_t)5 * nt * 4, 128);
      P.off_bar = (unsigned)off; off += align_up(sizeof(Shared), 128);
      if (off <= limit) {
        P.nt = nt; P.stages = stages; P.tiles_n = L.c_out / nt;
        P.smem_bytes = (unsigned)(off + 1024);
        P.valid = 1;
        *plan = P;
        return true;
      }
    }
  }
  return false;
}

bool tc_device_ok(int device) {
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return false;
  return prop.major == 10 && encode_tiled_fn() != nullptr;
}

size_t tc_workspace_bytes(const LayerDims&, const TcPlan&) { return 0; }

int launch_tc(const LayerDims& L, const TcPlan& P, int in_dtype, TcMaps* maps, const void* x,
              const void* w_base, const void* w_cond, const cg_bn_params& bn, const float* delta,
              const void* residual, void* y, uint32_t* mask, void* workspace,
              unsigned long long* counters, cudaStream_t stream) {
  (void)in_dtype; (void)residual; (void)workspace;
  if (!P.valid) return (int)cudaErrorInvalidValue;
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
    {
      cuuint64_t dims[4] = {(cuuint64_t)L.c_in, (cuuint64_t)L.w, (cuuint64_t)L.h, (cuuint64_t)L.n};
      cuuint64_t str[3] = {(cuuint64_t)L.c_in * 2, (cuuint64_t)L.w * L.c_in * 2,
                           (cuuint64_t)L.h * L.w * L.c_in * 2};
      cuuint32_t box[4] = {64, (cuuint32_t)P.wp, (cuuint32_t)P.box_h, (cuuint32_t)P.ni};
      if (!encode(&ms->x, const_cast<void*>(x), 4, dims, str, box)) return (int)cudaErrorInvalidValue;
    }
    {
      cuuint64_t dims[2] = {(cuuint64_t)taps * L.c_p, (cuuint64_t)L.c_out};
      cuuint64_t str[1] = {(cuuint64_t)taps * L.c_p * 2};
      cuuint32_t box[2] = {64, (cuuint32_t)P.nt};
      if (!encode(&ms->wb, const_cast<void*>(w_base), 2, dims, str, box)) return (int)cudaErrorInvalidValue;
    }
    if (L.c_r > 0) {
      cuuint64_t dims[2] = {(cuuint64_t)taps * L.c_r, (cuuint64_t)L.c_out};
      cuuint64_t str[1] = {(cuuint64_t)taps * L.c_r * 2};
      cuuint32_t box[2] = {64, (cuuint32_t)P.nt};
      if (!encode(&ms->wc, const_cast<void*>(w_cond), 2, dims, str, box)) return (int)cudaErrorInvalidValue;
    } else {
      ms->wc = ms->wb;
    }
    {
      cuuint64_t dims[4] = {(cuuint64_t)L.c_out, (cuuint64_t)L.wo, (cuuint64_t)L.ho, (cuuint64_t)L.n};
      cuuint64_t str[3] = {(cuuint64_t)L.c_out * 2, (cuuint64_t)L.wo * L.c_out * 2,
                           (cuuint64_t)L.ho * L.wo * L.c_out * 2};
      cuuint32_t box[4] = {64, (cuuint32_t)P.wp, (cuuint32_t)P.out_box_h, (cuuint32_t)P.ni};
      if (!encode(&ms->y, y, 4, dims, str, box)) return (int)cudaErrorInvalidValue;
    }
    ms->key[0] = x; ms->key[1] = w_base; ms->key[2] = wc_key; ms->key[3] = y;
  }
  TcParams prm;
  prm.L = L; prm.P = P; prm.bn = bn; prm.delta = delta; prm.mask = mask; prm.counters = counters;
  const unsigned grid = (unsigned)(P.tiles_m * P.tiles_n);
  cudaError_t e;
  if (P.nt == 128) {
    static bool attr128 = false;
    if (!attr128) {
      e = cudaFuncSetAttribute(tc_gated_conv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
      if (e != cudaSuccess) return (int)e;
      attr128 = true;
    }
    tc_gated_conv_kernel<128><<<grid, kThreads, P.smem_bytes, stream>>>(ms->x, ms->wb, ms->wc, ms->y, prm);
  } else {
    static bool attr64 = false;
    if (!attr64) {
      e = cudaFuncSetAttribute(tc_gated_conv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
      if (e != cudaSuccess) return (int)e;
      attr64 = true;
    }
    tc_gated_conv_kernel<64><<<grid, kThreads, P.smem_bytes, stream>>>(ms->x, ms->wb, ms->wc, ms->y, prm);
  }
  return (int)cudaGetLastError();
}

}  // namespace cg
