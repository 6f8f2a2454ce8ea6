// Online chunk queue (Sec. 3.1 "Chunk eviction": a priority queue of fixed size keeps the chunks
// with the lowest self-information while the chunks are prefilled batch by batch).
//
// The queue has m slots.  A slot holds the score and the id of one chunk and, in the caller's
// slot storage, that chunk's compressed keys, values and positions (k tokens per kv-head, the
// result of the token eviction of Eq. 7).  The slots are not kept in any order: a batch only
// overwrites the slots of the chunks it pushes out, so a chunk's compressed cache is written
// once.  pc_queue_emit puts the survivors in ascending chunk order at the end.
//
// Latency-bound bookkeeping (one block) plus an HBM-bound row copy; no tensor cores here.
#include "pc_kernels.h"
#include "pc_rank.cuh"

namespace pc {

constexpr int QUEUE_MAX = 1024;                                // slots + chunks of one batch
constexpr int EMPTY_ID = 0x7FFFFFFF;                           // an empty slot loses every tie

__global__ void queue_init_kernel(float* q_score, int* q_chunk, int m) {
  for (int i = threadIdx.x; i < m; i += blockDim.x) {
    q_score[i] = 0.0f;
    q_chunk[i] = -1;
  }
}

void launch_queue_init(float* q_score, int* q_chunk, int m, cudaStream_t st) {
  note_launch();
  queue_init_kernel<<<1, 256, 0, st>>>(q_score, q_chunk, m);
}

// Candidates 0..m-1 are the slots, m..m+Cb-1 the chunks of the batch.  A candidate survives when fewer
// than m candidates are better (higher key; equal keys: lower chunk id; empty slots last).  The a-th
// surviving batch chunk (ascending id) goes to the a-th slot that lost its chunk (ascending slot).
__global__ void __launch_bounds__(QUEUE_MAX) queue_update_kernel(const float* __restrict__ score, int Cb, int chunk_id0,
                                                                 int lower_is_better, int m, float* __restrict__ q_score,
                                                                 int* __restrict__ q_chunk, int* __restrict__ slot_src) {
  __shared__ uint32_t key[QUEUE_MAX];
  __shared__ int id[QUEUE_MAX];
  __shared__ int keep[QUEUE_MAX];
  const int i = threadIdx.x, n = m + Cb;
  if (i < m) {
    const int c = q_chunk[i];
    id[i] = c < 0 ? EMPTY_ID : c;
    key[i] = c < 0 ? 0u : rank_key(q_score[i], lower_is_better != 0);
  } else if (i < n) {
    id[i] = chunk_id0 + (i - m);
    key[i] = rank_key(score[i - m], lower_is_better != 0);
  }
  __syncthreads();
  int kp = 0;
  if (i < n) {
    const uint32_t mine = key[i];
    const int my_id = id[i];
    int rank = 0;
    for (int j = 0; j < n; ++j) {
      const bool better = key[j] > mine || (key[j] == mine && (id[j] < my_id || (id[j] == my_id && j < i)));
      rank += better ? 1 : 0;
    }
    kp = rank < m ? 1 : 0;
  }
  keep[i] = kp;
  __syncthreads();
  if (i < m) {
    int src = -1;
    if (!kp) {
      int nth = 0;                                             // this is the nth slot (from 0) that lost its chunk
      for (int j = 0; j < i; ++j) nth += keep[j] ? 0 : 1;
      for (int j = m; j < n; ++j) {                            // the nth surviving chunk of the batch moves in
        if (keep[j]) {
          if (nth == 0) { src = j - m; break; }
          --nth;
        }
      }
    }
    slot_src[i] = src;
    if (src >= 0) {
      q_score[i] = score[src];
      q_chunk[i] = chunk_id0 + src;
    }
  }
}

void launch_queue_update(const float* score, int Cb, int chunk_id0, int lower_is_better, int m, float* q_score,
                         int* q_chunk, int* slot_src, cudaStream_t st) {
  note_launch();
  queue_update_kernel<<<1, QUEUE_MAX, 0, st>>>(score, Cb, chunk_id0, lower_is_better, m, q_score, q_chunk, slot_src);
}

// slot_order[i] = the slot holding the i-th smallest chunk id (-1 past the filled slots); kept_out[i] = that id.
__global__ void __launch_bounds__(QUEUE_MAX) queue_order_kernel(const int* __restrict__ q_chunk, int m,
                                                                int* __restrict__ kept_out, int* __restrict__ slot_order) {
  __shared__ int id[QUEUE_MAX];
  const int i = threadIdx.x;
  if (i < m) {
    id[i] = q_chunk[i];
    kept_out[i] = -1;
    slot_order[i] = -1;
  }
  __syncthreads();
  if (i < m && id[i] >= 0) {
    int rank = 0;
    for (int j = 0; j < m; ++j) rank += (id[j] >= 0 && id[j] < id[i]) ? 1 : 0;
    kept_out[rank] = id[i];
    slot_order[rank] = i;
  }
}

// Rows of d bf16 (2d bytes): out[hkv, i*k + t] = slot storage [hkv, slot_order[i]*k + t]; zero rows and
// position -1 for an empty place.  d/8 lanes per row, 16-byte accesses, K and V in the same thread.
template <int D>
__global__ void __launch_bounds__(256) queue_emit_kernel(const uint4* __restrict__ q_k, const uint4* __restrict__ q_v,
                                                         const int* __restrict__ q_pos, const int* __restrict__ slot_order,
                                                         int m, int Hkv, int k, uint4* __restrict__ k_out,
                                                         uint4* __restrict__ v_out, int* __restrict__ pos_out) {
  constexpr int LPR = D / 8;
  const long long n_rows = (long long)Hkv * m * k;
  const long long gthreads = (long long)gridDim.x * blockDim.x;
  const int sub = threadIdx.x % LPR;
  for (long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR; row < n_rows; row += gthreads / LPR) {
    const int hk = (int)(row / ((long long)m * k));
    const int place = (int)(row % ((long long)m * k));
    const int i = place / k, t = place % k;
    const int s = slot_order[i];
    uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
    int p = -1;
    if (s >= 0) {
      const long long src = ((long long)hk * m + s) * k + t;
      kv = __ldg(q_k + src * LPR + sub);
      vv = __ldg(q_v + src * LPR + sub);
      if (sub == 0) p = q_pos[src];
    }
    k_out[row * LPR + sub] = kv;
    v_out[row * LPR + sub] = vv;
    if (pos_out != nullptr && sub == 0) pos_out[row] = p;
  }
}

cudaError_t launch_queue_emit(const int* q_chunk, int m, int Hkv, int k, int d, const void* q_k, const void* q_v,
                              const int* q_pos, int* kept_out, int* slot_order, void* k_out, void* v_out, int* pos_out,
                              int sm_count, cudaStream_t st) {
  note_launch();
  queue_order_kernel<<<1, QUEUE_MAX, 0, st>>>(q_chunk, m, kept_out, slot_order);
  const long long n_rows = (long long)Hkv * m * k;
  const int lpr = d / 8;
  const long long want = (n_rows * lpr + 255) / 256;
  int blocks = (int)(want < (long long)sm_count * 8 ? want : (long long)sm_count * 8);
  if (blocks < 1) blocks = 1;
  note_launch();
  if (d == 128)
    queue_emit_kernel<128><<<blocks, 256, 0, st>>>((const uint4*)q_k, (const uint4*)q_v, q_pos, slot_order, m, Hkv, k,
                                                   (uint4*)k_out, (uint4*)v_out, pos_out);
  else
    queue_emit_kernel<64><<<blocks, 256, 0, st>>>((const uint4*)q_k, (const uint4*)q_v, q_pos, slot_order, m, Hkv, k,
                                                  (uint4*)k_out, (uint4*)v_out, pos_out);
  return cudaGetLastError();
}

}  // namespace pc
