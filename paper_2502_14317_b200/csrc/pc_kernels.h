// Internal launcher declarations shared by the translation units of libpc.
#pragma once
#include <cuda_runtime.h>
#include <cstddef>
#include <cstdint>

namespace pc {

// ---- pc_api.cu
// Every kernel launch of the library is counted here (see pc_launch_count in pc.h).
void note_launch();

// ---- pc_rope.cu
// cos/sin table: tab[p * (d/2) + t] = (cos, sin)(  (pos0 + p) * theta^(-2t/d) ), fp64; tab_hi, tab_lo (may be null): the
// same entries split into an fp32 head and an fp32 tail (value = head + tail to 2^-48), one float4 per two pairs:
// (cos_2i, cos_2i+1, sin_2i, sin_2i+1).
void launch_rope_table(double2* tab, float4* tab_hi, float4* tab_lo, int n_pos, int d, double theta, int pos0, cudaStream_t st);
// y[c,p,h,:] = bf16( RoPE(x[c,p,h,:], position p) ), the fp64 rotation rounded once; x addressed by element strides
// (chunk, token, head), y contiguous [C,L,H,d].
void launch_rope_rows(const void* x, const long long x_stride[3], void* y, const double2* tab, const float4* tab_hi,
                      const float4* tab_lo, int C, int L, int H, int d, cudaStream_t st);

// Per-chunk lengths: zero o[c, p, :, :], lse[c, :, p] and win_score[c, :, p] for p >= clamp(chunk_len[c], w + 1, L).
void launch_zero_chunk_tails(const int* chunk_len, int C, int L, int w, int Hq, int Hkv, int d, void* o,
                             const long long o_stride[3], float* lse, float* win_score, cudaStream_t st);

// ---- pc_select_gather.cu
void launch_chunk_score(const float* win_lse, int C, int n_per_chunk, float* score, cudaStream_t st);
void launch_select_chunks(const float* score, int C, int m, int lower_is_better, int* kept, cudaStream_t st);
// stand-in chunk score (as launch_chunk_score, same bits) followed by the chunk top-m, in one launch for C <= 64
void launch_score_select_chunks(const float* win_lse, int C, int n_per_chunk, int m, int lower_is_better, float* score,
                                int* kept, cudaStream_t st);
// attention calibration (Eq. 8): sizes of the sink and recency regions and the three thresholds; null = off
struct SelCalibArgs {
  int n_s, n_r;
  float lam_s, lam_m, lam_r;
};
cudaError_t launch_select_tokens(const float* win_score, const int* kept, int m, int Hkv, int L, int n_cand, int k,
                                 int* idx, const SelCalibArgs* calib, cudaStream_t st);
// online chunk queue: rank the chunks that move into a slot (slot_src[s] >= 0) and copy their kept rows into the slot
// storage, in one launch; cudaErrorNotSupported when k is too large for that (then rank and gather separately)
cudaError_t launch_select_gather_slots(const float* win_score, const int* slot_src, int m, int Hkv, int L, int n_cand,
                                       int k, const void* k_src, const void* v_src, const long long stride_elems[3],
                                       int d, void* q_k, void* q_v, int* q_pos, cudaStream_t st);
cudaError_t launch_gather_kv(const void* k_src, const void* v_src, const long long stride_elems[3], const int* kept,
                             const int* idx, int m, int Hkv, int k, int d, void* k_out, void* v_out, int* pos_out,
                             int sm_count, bool by_slot, cudaStream_t st);

// caches stored with room to grow: cache[b, hkv, Nk + i, :] = win[b, i, hkv, :] for the w new rows of every sequence
cudaError_t launch_append_kv(const void* k_win, const void* v_win, int B, int w, int Hkv, int d, long long Nk,
                             long long Nk_cap, void* k_cache, void* v_cache, cudaStream_t st);

// ---- pc_queue.cu (online chunk queue)
void launch_queue_init(float* q_score, int* q_chunk, int m, cudaStream_t st);
void launch_queue_update(const float* score, int Cb, int chunk_id0, int lower_is_better, int m, float* q_score,
                         int* q_chunk, int* slot_src, cudaStream_t st);
cudaError_t launch_queue_emit(const int* q_chunk, int m, int Hkv, int k, int d, const void* q_k, const void* q_v,
                              const int* q_pos, int* kept_out, int* slot_order, void* k_out, void* v_out,
                              int* pos_out, int sm_count, cudaStream_t st);

}  // namespace pc
