// Tensor-core (tcgen05) path of the channel-gated layer: plan, tensor maps, launcher.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace cg {

// Tiling of one layer for the shifted-window implicit GEMM (see tc_conv.cu).
struct TcPlan {
  int valid;
  int elem_bytes;       // 2 (bf16) or 1 (int8)
  int ck;               // channels per 128-byte (bf16) patch row = one K chunk
  int images_mode;      // 0: a tile is `r` output rows of one image; 1: `ni` whole images
  int wp;               // patch row pitch in pixels: w + pad (rows share their zero columns)
  int r;                // output rows per tile (rows mode)
  int ni;               // images per tile (images mode), else 1
  int ip;               // image pitch in patch pixels: (h + pad) * wp
  int tiles_per_image;  // rows mode
  int tiles_m, tiles_n, nt;
  int chunks;           // c_in / ck input-channel chunks
  int base_chunks;      // chunks that hold base-path channels
  int planes;           // patch buffers per chunk: 1 (stride 1) or 4 (stride 2: the input's
                        // even/odd row x even/odd column sub-images)
  int na;               // patch buffers in the ring
  int issuers;          // MMA-issuing threads: 1; 2 (base path / conditional path) when the
                        // weights are resident; 3 (base / conditional of even jobs / of odd jobs)
                        // when in addition one input chunk serves both paths
  int split_a;          // 2 issuers, > 0: slots [0, split_a) serve the base path and the rest the
                        // conditional path
  int share_a;          // 2 issuers, 1: one input chunk serves both paths, so job j's patch stays
                        // in slot j % na from its base MMAs until its conditional MMAs are done
  int nb;               // weight ring depth in stages of three tiles (0 when the weights are resident)
  int resident;         // 1: all weight tiles of a column tile stay in shared memory
  int box_h;            // patch box rows: r + 2*pad (rows mode) or h + pad (images mode)
  int box_pixels;       // wp * box_h * ni
  int patch_rows;       // rows allocated per patch buffer
  int patch_bytes;
  int out_box_h;        // y store box rows
  int stage_rows;       // rows of the y staging tile
  int base_tiles, cond_tiles;   // weight tiles per phase
  int cond_mode;
  int pad8;             // c_in/G = 8 (bf16): computed as 16 base channels + a conditional path over all
                        // input channels, with weights repacked into the workspace (tc2_conv.cuh)
  unsigned off_a, off_b, off_y, off_consts, off_mask, off_tables, off_bar, smem_bytes;
};

struct TcMapSet {
  const void* key[4];   // x, w_base, w_cond, y the maps below were encoded for
  CUtensorMap x[4], wb, wc, y;   // x[1..3] only for stride 2
};

// Small cache of encoded tensor maps, so that callers that rotate a few buffers do not pay
// four cuTensorMapEncodeTiled calls per forward.
struct TcMaps {
  static constexpr int kEntries = 8;
  TcMapSet set[kEntries];
  int next;
};

bool tc_plan(const LayerDims& L, int in_dtype, int cond_mode, TcPlan* plan);
bool tc_device_ok(int device);
size_t tc_workspace_bytes(const LayerDims& L, const TcPlan& plan);
int launch_tc(const LayerDims& L, const TcPlan& plan, int in_dtype, TcMaps* maps, const void* x,
              const void* w_base, const void* w_cond, const cg_bn_params& bn, const float* delta,
              const void* residual, void* y, uint32_t* mask, void* workspace,
              unsigned long long* counters, cudaStream_t stream, const float* t_img = nullptr,
              int base_only = 0);

// Channel-wise gate (Eq. 4) through two passes of the pixel-major kernel (chan_gate.cu).
size_t tc_channel_gate_workspace_bytes(const LayerDims& L, const TcPlan& plan);
int launch_tc_channel_gate(const LayerDims& L, const TcPlan& plan, int in_dtype, TcMaps* maps, const void* x,
                           const void* w_base, const void* w_cond, const cg_bn_params& bn, const float* delta,
                           const void* residual, void* y, uint32_t* mask, void* workspace,
                           unsigned long long* counters, cudaStream_t stream);

}  // namespace cg
