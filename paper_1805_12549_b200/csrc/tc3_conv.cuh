// Tap-stacked tensor-core path of the channel-gated layer (tc3_conv.cu): plan and launcher.
// For 3x3, stride-1 bf16 layers with 64 input and 64 output channels, images up to 128 pixels wide.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace cg {

struct Tc3Plan {
  int valid;
  int rows;              // output rows per job: floor(128 / w)
  int xch;               // 1: w does not divide 32, neighbouring warps exchange their edge values
  int patch_bytes, na;   // input patch buffer and how many of them
  int tiles_per_image;   // ceil(h / rows)
  int jobs;              // n * tiles_per_image
  int kp;                // K steps (16 channels) of the base path: c_p / 16
  int cond_mode;
  int grid;
};

struct Tc3MapSet {
  const void* key[2];    // x, y the maps were encoded for
  CUtensorMap x, y;
};

struct Tc3Maps {
  static constexpr int kEntries = 8;
  Tc3MapSet set[kEntries];
  int next;
};

bool tc3_plan(const LayerDims& L, int in_dtype, int cond_mode, int sms, Tc3Plan* plan);
int launch_tc3(const LayerDims& L, const Tc3Plan& plan, Tc3Maps* maps, const void* x, const void* w_base,
               const void* w_cond, const cg_bn_params& bn, const float* delta, const void* residual, void* y,
               uint32_t* mask, unsigned long long* counters, cudaStream_t stream);

}  // namespace cg
