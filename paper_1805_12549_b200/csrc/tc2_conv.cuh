// Channel-major tensor-core path of the channel-gated layer (tc2_conv.cu): plan and launcher.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace cg {

constexpr int kTc2MaxStages = 128;

// One K stage of a job: a weight tile of 64 K-elements (all channels of the CTA's channel
// tile) and the up to four 16-element K steps it holds.  For K step ks the pixel operand is the
// patch of input-channel chunk `chunk` read from `boff[ks]` on (16-byte units: filter-tap row
// offset plus the position of the 16 channels inside the 128-byte patch row).
struct alignas(16) Tc2Stage {   // 16 bytes, read by the kernel as one uint4: {kx, flags|chunk|ks0|ks1, boff[0..3]}
  int32_t kx;            // K coordinate of the tile in the weight matrix (may be negative or reach
                         // past the end: TMA fills those elements with zeros, their K steps are skipped)
  uint8_t flags;         // kStage* bits
  uint8_t chunk;         // 64-channel chunk of x the K steps read
  uint8_t ks0, ks1;      // K steps [ks0, ks1) of the tile are used
  uint16_t boff[4];
};

enum : uint8_t {
  kStageCond = 1,        // the tile comes from W_cond (else W_base)
  kStageFirst = 2,       // first stage of a job
  kStageFirstCond = 4,   // first stage of the conditional path
  kStageLastBase = 8,    // last stage of the base path
  kStageLast = 16,       // last stage of the job
  kStageNewChunk = 32    // reads another input-channel chunk than the stage before
};

struct Tc2Plan {
  int valid;
  int wp, hp;            // pitch of the stacked, padded pixel space: w + pad, h + pad
  float inv_wp, inv_hp;
  int r;                 // stacked rows per pixel sub-tile
  int nsub;              // pixel sub-tiles per job: 1 or 2
  int np;                // pixels (incl. pad positions) per sub-tile: r * wp
  int nmma;              // MMA N: np rounded up to a multiple of 16
  int jobs_m;            // pixel tiles
  int tiles_c;           // channel tiles of 128
  int chunks;            // c_in / 64
  int nb, ns;            // base-path stages, all stages
  int ring;              // weight ring depth in stages
  int entries;           // patch buffers: 2 or 3
  int lead;              // stages by which sub-tile a runs ahead of sub-tile b
  int w_rows;            // channels per weight tile: min(128, c_out)
  int w_stage_bytes;     // w_rows * 128
  int patch_rows;        // 128-byte pixel rows per patch buffer
  int patch_bytes;
  int patch_box_rows;    // stacked rows loaded per patch: r + 2*pad
  int cond_mode;
  int pad8;              // c_p = 8: the weights are repacked into the workspace with whole K steps
  int use_img;           // whole images are loaded by single copies (small images)
  int grid;
  unsigned off_w, off_p, off_epi, off_tab, off_bar, smem_bytes;
  Tc2Stage st[kTc2MaxStages];
};

struct Tc2MapSet {
  const void* key[3];    // x, w_base, w_cond the maps were encoded for
  CUtensorMap x[5], wb, wc;   // x: boxes of 1, 2, 8 rows, 1 image, 4 images
};

struct Tc2Maps {
  static constexpr int kEntries = 8;
  Tc2MapSet set[kEntries];
  int next;
};

// Weights of a layer with c_in/G = 8 repacked into `workspace` (repack8_bytes) with whole K steps:
// W_base gets 8 zero channels behind its 8 per tap, W_cond 8 zero channels in front; the layer is
// then computed as one with 16 base channels and a conditional path over all input channels.
size_t repack8_bytes(const LayerDims& L);
int launch_repack8(const LayerDims& L, const void* w_base, const void* w_cond, void* workspace, const void** wb16,
                   const void** wcf, cudaStream_t stream);

bool tc2_plan(const LayerDims& L, int in_dtype, int cond_mode, int sms, Tc2Plan* plan);
size_t tc2_workspace_bytes(const LayerDims& L, const Tc2Plan& plan);
int launch_tc2(const LayerDims& L, const Tc2Plan& plan, Tc2Maps* maps, const void* x,
               const void* w_base, const void* w_cond, const cg_bn_params& bn, const float* delta,
               const void* residual, void* y, uint32_t* mask, void* workspace,
               unsigned long long* counters, cudaStream_t stream);

}  // namespace cg
