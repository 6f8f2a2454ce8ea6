// Parameter blocks and launchers of the attention kernels (internal).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace pc {

struct PrefillParams {
  int C, L, w, Hq, Hkv;
  float scale_log2;              // softmax scale * log2(e)
  const double2* rope_tab;       // [L][d/2] (cos, sin)
  float* lse;                    // [C,Hq,L] or null
  float* win_lse;                // [C,Hq,w]
  float* win_score;              // [C,Hkv,L]
  int* status;                   // device status word or null
  int* counter;                  // work-queue counter, zeroed before launch
};

// maps: q (box 64x1x128x1), k_rot, v, o (store), q with a w-row box
cudaError_t launch_prefill_attn(const CUtensorMap* maps, const PrefillParams& prm, int d, int grid, cudaStream_t st);

}  // namespace pc
