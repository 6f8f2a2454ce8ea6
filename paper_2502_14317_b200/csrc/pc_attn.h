// Parameter blocks and launchers of the attention kernels (internal).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace pc {

struct PrefillParams {
  int C, L, w, Hq, Hkv;
  float scale_log2;              // softmax scale * log2(e)
  const int* chunk_len;          // [C] tokens per chunk (window included) or null: all L
  float* lse;                    // [C,Hq,L] or null
  float* win_lse;                // [C,Hq,w]
  float* win_score;              // [C,Hkv,L]
  int* status;                   // device status word or null
  int* counter;                  // work-queue counter, zeroed before launch
  int wait_kcycles;              // limit of every device-side wait, in units of 1024 cycles
  int skip_final_publication;    // test hook of the bounded waits (see pc_debug_bounded_wait_test in pc.h)
};

// maps: rotated q (box 64x1x128x1), k_rot, v, o (store), rotated q with a w-row box
cudaError_t launch_prefill_attn(const CUtensorMap* maps, const PrefillParams& prm, int d, int grid, cudaStream_t st);

// Head size 128: CTA-pair kernel (pc_prefill2.cu).  maps as above plus maps[5] = rotated keys with a 64-token box.
cudaError_t launch_prefill_pair(const CUtensorMap* maps, const PrefillParams& prm, int sm_count, cudaStream_t st);

struct ParallelParams {
  int B, w, Hq, Hkv, Nk;
  int Gs, n_rg;                  // q-heads per row group (Gs * w <= 256), row groups per kv-head
  int n_cache_tiles, n_split, tiles_per_split;
  int alt;                       // 1: the item's rows fit one block; the two blocks take alternate key tiles of the split
  int n_part;                    // partial results per (sequence, q-head): n_split, or 2 * n_split with alt
  float scale_log2;
  float* part_o;                 // [B,Hq,n_part,w,d] fp32 unnormalised partial outputs (n_part > 1)
  float* part_ml;                // [B,Hq,n_part,w,2] (running max in log2 units, sum)
  __nv_bfloat16* out;            // [B,w,Hq,d]
  float* lse_out;                // [B,Hq,w] or null
  int* status;
  int* counter;
  int wait_kcycles;              // limit of every device-side wait, in units of 1024 cycles
};

// maps: rotated q_win (w-row box), k_cache, v_cache (128-key box), k_win, v_win (128-row box over w tokens)
cudaError_t launch_parallel_attn(const CUtensorMap* maps, const ParallelParams& prm, int d, int grid, cudaStream_t st);

// Parallel attention on CTA pairs (head size 128, G * w a multiple of 256, no key split): every pair takes the
// windows of 2 * hpc q-heads of one kv-head (hpc * w = 128 rows per CTA) over the whole cache.
struct ParallelPairParams {
  int B, w, Hq, Hkv, Nk;
  int hpc, n_rg;                 // q-heads per CTA, 256-row groups per kv-head
  float scale_log2;
  float* lse_out;                // [B,Hq,w] or null
  int* status;
  int wait_kcycles;              // limit of every device-side wait, in units of 1024 cycles
};

// maps: rotated q_win (box 64 x 1 head x w tokens), out (same box), k_cache (64 x 64 keys), v_cache (64 x 128 keys),
// k_win (64 x 1 head x 64 tokens), v_win (64 x 1 head x 128 tokens)
cudaError_t launch_parallel_pair(const CUtensorMap* maps, const ParallelPairParams& prm, int sm_count, cudaStream_t st);

}  // namespace pc
