// C ABI of libpc: argument validation on the host, tensor-map construction, launches.
// Nothing here allocates device memory or synchronises.
#include "../../include/pc.h"
#include "pc_attn.h"
#include "pc_kernels.h"
#include "pc_tmap.h"

#include <atomic>
#include <cmath>
#include <cstring>

namespace pc {
static std::atomic<unsigned long long> g_launches{0};
void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
static std::atomic<int> g_wait_kcycles{1 << 21};            // limit of the device-side waits, units of 1024 cycles (~1 s)
static std::atomic<int> g_skip_final_publication{0};        // test hook, see pc_debug_bounded_wait_test
}  // namespace pc

namespace {

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceInfo {
  int ok = 0;          // 1: sm_100, -1: something else
  int sm_count = 0;
};

// Properties of the current device (queried once per device).
const DeviceInfo& device_info() {
  static DeviceInfo info[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { static DeviceInfo bad; bad.ok = -1; return bad; }
  if (info[dev].ok == 0) {
    int major = 0, sms = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    info[dev].sm_count = sms;
    info[dev].ok = (major == 10) ? 1 : -1;
  }
  return info[dev];
}

bool pow2_between(int x, int lo, int hi) { return x >= lo && x <= hi && (x & (x - 1)) == 0; }

void fill_strides(const int64_t in[3], int64_t out[3], int64_t tokens, int64_t heads, int64_t d) {
  if (in[0] == 0 && in[1] == 0 && in[2] == 0) { out[0] = tokens * heads * d; out[1] = heads * d; out[2] = d; }
  else { out[0] = in[0]; out[1] = in[1]; out[2] = in[2]; }
}
bool strides_ok(const int64_t s[3], int64_t d) { return s[0] > 0 && s[1] > 0 && s[2] >= d && s[0] % 8 == 0 && s[1] % 8 == 0 && s[2] % 8 == 0; }

struct PrefillLayout {
  size_t off_counter, off_table, off_table32, off_qrot, off_krot, total;
};
PrefillLayout prefill_layout(const pc_prefill_desc* d, bool krot_in_ws) {
  PrefillLayout l;
  size_t off = 0;
  l.off_counter = off; off += ALIGN;
  l.off_table = off; off += align_up((size_t)d->L * (d->d / 2) * sizeof(double2));
  l.off_table32 = off; off += align_up((size_t)d->L * (d->d / 2) * sizeof(float4));   // fp32 heads, then fp32 tails
  l.off_qrot = off; off += align_up((size_t)d->C * d->L * d->Hq * d->d * 2);         // rotated queries
  l.off_krot = off;
  if (krot_in_ws) off += align_up((size_t)d->C * d->L * d->Hkv * d->d * 2);
  l.total = off;
  return l;
}

int32_t check_prefill_desc(const pc_prefill_desc* d) {
  if (!d) return PC_ERR_INVALID_ARG;
  if (d->C < 1 || d->L < 2 || d->w < 1 || d->w >= d->L || d->Hq < 1 || d->Hkv < 1 || d->Hq % d->Hkv != 0) return PC_ERR_INVALID_ARG;
  if (!(d->rope_theta > 0.0f) || d->softmax_scale < 0.0f) return PC_ERR_INVALID_ARG;
  if (d->d != 64 && d->d != 128) return PC_ERR_UNSUPPORTED;
  if (d->w > 128) return PC_ERR_UNSUPPORTED;
  if ((int64_t)(d->Hq / d->Hkv) * d->w > 1024) return PC_ERR_UNSUPPORTED;
  if ((int64_t)d->C * d->Hkv > (1 << 24) || d->L > (1 << 24)) return PC_ERR_UNSUPPORTED;
  return PC_OK;
}

}  // namespace

extern "C" {

const char* pc_status_string(int32_t status) {
  switch (status) {
    case PC_OK: return "ok";
    case PC_ERR_INVALID_ARG: return "invalid argument";
    case PC_ERR_UNSUPPORTED: return "unsupported shape or device";
    case PC_ERR_WORKSPACE: return "workspace missing or too small";
    case PC_ERR_CUDA: return "CUDA call failed";
    case PC_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case PC_ERR_SCRATCH_LIMIT: return "shape needs more scratch than the built-in PC_STATIC_SCRATCH_BYTES array holds";
    default: return "unknown status";
  }
}

int32_t pc_version(void) { return 1001; }

uint64_t pc_launch_count(void) { return pc::g_launches.load(std::memory_order_relaxed); }

int32_t pc_debug_bounded_wait_test(int64_t wait_limit_cycles, int32_t skip_final_publication) {
  if (wait_limit_cycles < 0 || wait_limit_cycles > (int64_t)2000000000 * 1024) return PC_ERR_INVALID_ARG;
  const int64_t kc = wait_limit_cycles == 0 ? (1 << 21) : (wait_limit_cycles + 1023) / 1024;
  pc::g_wait_kcycles.store((int)(kc < 1 ? 1 : kc));
  pc::g_skip_final_publication.store(skip_final_publication != 0 ? 1 : 0);
  return PC_OK;
}

// ------------------------------------------------------------------------------------ prefill
size_t pc_chunk_prefill_attn_workspace_bytes(const pc_prefill_desc* desc) {
  if (check_prefill_desc(desc) != PC_OK) return 0;
  return prefill_layout(desc, false).total;
}

int32_t pc_chunk_prefill_attn(const pc_prefill_desc* desc, const void* q, const void* k, const void* v,
                              const int32_t* chunk_len, void* o, void* k_rot, float* lse, float* win_score,
                              float* win_lse, int32_t* status_word, void* workspace, size_t workspace_bytes,
                              void* stream) {
  int32_t rc = check_prefill_desc(desc);
  if (rc != PC_OK) return rc;
  if (!q || !k || !v || !o || !win_score || !win_lse) return PC_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(k_rot) || !aligned16(workspace))
    return PC_ERR_INVALID_ARG;
  const int d = desc->d;
  int64_t qs[3], ks[3], vs[3], os[3];
  fill_strides(desc->q_stride, qs, desc->L, desc->Hq, d);
  fill_strides(desc->k_stride, ks, desc->L, desc->Hkv, d);
  fill_strides(desc->v_stride, vs, desc->L, desc->Hkv, d);
  fill_strides(desc->o_stride, os, desc->L, desc->Hq, d);
  if (!strides_ok(qs, d) || !strides_ok(ks, d) || !strides_ok(vs, d) || !strides_ok(os, d)) return PC_ERR_INVALID_ARG;
  const bool krot_in_ws = (k_rot == nullptr);
  const PrefillLayout lay = prefill_layout(desc, krot_in_ws);
  if (!workspace || workspace_bytes < lay.total) return PC_ERR_WORKSPACE;
  const DeviceInfo& dev = device_info();
  if (dev.ok != 1) return PC_ERR_UNSUPPORTED;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int* counter = reinterpret_cast<int*>(ws + lay.off_counter);
  double2* table = reinterpret_cast<double2*>(ws + lay.off_table);
  float4* table_hi = reinterpret_cast<float4*>(ws + lay.off_table32);
  float4* table_lo = table_hi + (size_t)desc->L * (d / 4);
  void* krot = krot_in_ws ? static_cast<void*>(ws + lay.off_krot) : k_rot;
  void* qrot = ws + lay.off_qrot;

  // tensor maps (innermost first: d, head, token, chunk)
  CUtensorMap maps[6];
  const uint64_t q_dims[4] = {(uint64_t)d, (uint64_t)desc->Hq, (uint64_t)desc->L, (uint64_t)desc->C};
  const uint64_t kv_dims[4] = {(uint64_t)d, (uint64_t)desc->Hkv, (uint64_t)desc->L, (uint64_t)desc->C};
  const uint64_t q_str[3] = {(uint64_t)d, (uint64_t)desc->Hq * d, (uint64_t)desc->L * desc->Hq * d};   // rotated queries: contiguous
  const uint64_t v_str[3] = {(uint64_t)vs[2], (uint64_t)vs[1], (uint64_t)vs[0]};
  const uint64_t o_str[3] = {(uint64_t)os[2], (uint64_t)os[1], (uint64_t)os[0]};
  const uint64_t kr_str[3] = {(uint64_t)d, (uint64_t)desc->Hkv * d, (uint64_t)desc->L * desc->Hkv * d};
  const uint32_t box_tile[4] = {64, 1, 128, 1};
  const uint32_t box_win[4] = {64, 1, (uint32_t)((desc->w + 7) & ~7), 1};   // window rows of a head in the score sweep, padded to 8
  const uint32_t box_half[4] = {64, 1, 64, 1};
  if (!pc::make_tmap_bf16_4d(&maps[0], qrot, q_dims, q_str, box_tile) ||
      !pc::make_tmap_bf16_4d(&maps[1], krot, kv_dims, kr_str, box_tile) ||
      !pc::make_tmap_bf16_4d(&maps[2], v, kv_dims, v_str, box_tile) ||
      !pc::make_tmap_bf16_4d(&maps[3], o, q_dims, o_str, box_tile) ||
      !pc::make_tmap_bf16_4d(&maps[4], qrot, q_dims, q_str, box_win) ||
      !pc::make_tmap_bf16_4d(&maps[5], krot, kv_dims, kr_str, box_half))
    return PC_ERR_CUDA;

  if (cudaMemsetAsync(counter, 0, sizeof(int), st) != cudaSuccess) return PC_ERR_CUDA;
  pc::launch_rope_table(table, table_hi, table_lo, desc->L, d, (double)desc->rope_theta, 0, st);
  // queries and keys are rotated once, ahead of the attention kernel (positions 0 .. L-1 in every chunk)
  const long long ks_ll[3] = {ks[0], ks[1], ks[2]}, qs_ll[3] = {qs[0], qs[1], qs[2]}, os_ll[3] = {os[0], os[1], os[2]};
  pc::launch_rope_rows(k, ks_ll, krot, table, table_hi, table_lo, desc->C, desc->L, desc->Hkv, d, st);
  pc::launch_rope_rows(q, qs_ll, qrot, table, table_hi, table_lo, desc->C, desc->L, desc->Hq, d, st);

  if (chunk_len != nullptr)   // rows and scores behind the end of a shorter chunk read as zero: the kernels below skip them
    pc::launch_zero_chunk_tails(chunk_len, desc->C, desc->L, desc->w, desc->Hq, desc->Hkv, d, o, os_ll, lse, win_score, st);

  pc::PrefillParams prm;
  prm.chunk_len = chunk_len;
  prm.C = desc->C; prm.L = desc->L; prm.w = desc->w; prm.Hq = desc->Hq; prm.Hkv = desc->Hkv;
  const double scale = desc->softmax_scale > 0.0f ? (double)desc->softmax_scale : 1.0 / std::sqrt((double)d);
  prm.scale_log2 = (float)(scale * 1.4426950408889634);
  prm.lse = lse; prm.win_lse = win_lse; prm.win_score = win_score;
  prm.status = status_word; prm.counter = counter;
  prm.wait_kcycles = pc::g_wait_kcycles.load();
  prm.skip_final_publication = pc::g_skip_final_publication.load();
  // head size 128 with an even number of q-heads per kv-head runs on CTA pairs (cta_group::2: the two CTAs take
  // the same query tile of two heads that share K/V); head size 64 and odd group sizes (multi-head attention:
  // one q-head per kv-head) run on single CTAs with two query blocks each
  const bool even_group = ((desc->Hq / desc->Hkv) % 2) == 0;
  const cudaError_t le = (d == 128 && even_group && dev.sm_count >= 2)
                             ? pc::launch_prefill_pair(maps, prm, dev.sm_count, st)
                             : pc::launch_prefill_attn(maps, prm, d, dev.sm_count, st);
  if (le != cudaSuccess) return PC_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? PC_OK : PC_ERR_CUDA;
}

// ------------------------------------------------------------------------------------ RoPE with position reuse
size_t pc_rope_position_reuse_workspace_bytes(int32_t L, int32_t d) {
  if (L < 1 || (d != 64 && d != 128)) return 0;
  return align_up((size_t)L * (d / 2) * sizeof(double2)) + align_up((size_t)L * (d / 2) * sizeof(float4));
}

int32_t pc_rope_position_reuse(const void* x, int32_t C, int32_t L, int32_t H, int32_t d, float rope_theta, void* y,
                               void* workspace, size_t workspace_bytes, void* stream) {
  if (!x || !y || C < 1 || L < 1 || H < 1 || !(rope_theta > 0.0f)) return PC_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return PC_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(y) || !aligned16(workspace)) return PC_ERR_INVALID_ARG;
  if ((int64_t)C * H > (1 << 24) || L > (1 << 24)) return PC_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < pc_rope_position_reuse_workspace_bytes(L, d)) return PC_ERR_WORKSPACE;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  double2* table = reinterpret_cast<double2*>(ws);
  float4* table_hi = reinterpret_cast<float4*>(ws + align_up((size_t)L * (d / 2) * sizeof(double2)));
  float4* table_lo = table_hi + (size_t)L * (d / 4);
  pc::launch_rope_table(table, table_hi, table_lo, L, d, (double)rope_theta, 0, st);
  const long long str[3] = {(long long)L * H * d, (long long)H * d, d};
  pc::launch_rope_rows(x, str, y, table, table_hi, table_lo, C, L, H, d, st);
  return cudaGetLastError() == cudaSuccess ? PC_OK : PC_ERR_CUDA;
}

// ------------------------------------------------------------------------------------ chunk score stand-in
int32_t pc_chunk_score_from_lse(const float* win_lse, int32_t C, int32_t Hq, int32_t w, float* chunk_score,
                                void* stream) {
  if (!win_lse || !chunk_score || C < 1 || Hq < 1 || w < 1) return PC_ERR_INVALID_ARG;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  pc::launch_chunk_score(win_lse, C, Hq * w, chunk_score, static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? PC_OK : PC_ERR_CUDA;
}

// ------------------------------------------------------------------------------------ chunk top-m
int32_t pc_select_chunks(const float* chunk_score, int32_t C, int32_t m, int32_t lower_is_better, int32_t* kept,
                         void* stream) {
  if (!chunk_score || !kept || C < 1 || m < 1 || m > C) return PC_ERR_INVALID_ARG;
  if (C > 1024) return PC_ERR_UNSUPPORTED;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  pc::launch_select_chunks(chunk_score, C, m, lower_is_better, kept, static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? PC_OK : PC_ERR_CUDA;
}

// ------------------------------------------------------------------------------------ stand-in score + chunk top-m, one launch
int32_t pc_score_select_chunks(const float* win_lse, int32_t C, int32_t Hq, int32_t w, int32_t m, int32_t lower_is_better,
                               float* chunk_score, int32_t* kept, void* stream) {
  if (!win_lse || !chunk_score || !kept || C < 1 || Hq < 1 || w < 1 || m < 1 || m > C) return PC_ERR_INVALID_ARG;
  if (C > 1024) return PC_ERR_UNSUPPORTED;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  pc::launch_score_select_chunks(win_lse, C, Hq * w, m, lower_is_better, chunk_score, kept, static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? PC_OK : PC_ERR_CUDA;
}

// ------------------------------------------------------------------------------------ token top-k
int32_t pc_select_tokens(const float* win_score, const int32_t* kept, int32_t C, int32_t m, int32_t Hkv, int32_t L,
                         int32_t n_cand, int32_t k, int32_t* idx, void* stream) {
  if (!win_score || !kept || !idx) return PC_ERR_INVALID_ARG;
  if (C < 1 || m < 1 || m > C || Hkv < 1 || L < 1 || n_cand < 1 || n_cand > L || k < 1) return PC_ERR_INVALID_ARG;
  if (n_cand > 32768) return PC_ERR_UNSUPPORTED;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  if (pc::launch_select_tokens(win_score, kept, m, Hkv, L, n_cand, k, idx, nullptr, static_cast<cudaStream_t>(stream)) !=
      cudaSuccess)
    return PC_ERR_CUDA;
  return PC_OK;
}

// ------------------------------------------------------------------------------------ token top-k with attention calibration
int32_t pc_select_tokens_calibrated(const float* win_score, const int32_t* kept, int32_t C, int32_t m, int32_t Hkv,
                                    int32_t L, int32_t n_cand, int32_t k, int32_t n_s, int32_t n_r, float lambda_s,
                                    float lambda_m, float lambda_r, int32_t* idx, void* stream) {
  if (!win_score || !kept || !idx) return PC_ERR_INVALID_ARG;
  if (C < 1 || m < 1 || m > C || Hkv < 1 || L < 1 || n_cand < 1 || n_cand > L || k < 1) return PC_ERR_INVALID_ARG;
  if (n_s < 0 || n_r < 0 || lambda_s != lambda_s || lambda_m != lambda_m || lambda_r != lambda_r) return PC_ERR_INVALID_ARG;
  if (n_cand > 32768) return PC_ERR_UNSUPPORTED;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  const pc::SelCalibArgs calib{n_s, n_r, lambda_s, lambda_m, lambda_r};
  if (pc::launch_select_tokens(win_score, kept, m, Hkv, L, n_cand, k, idx, &calib, static_cast<cudaStream_t>(stream)) !=
      cudaSuccess)
    return PC_ERR_CUDA;
  return PC_OK;
}

// ------------------------------------------------------------------------------------ gather
int32_t pc_gather_kv(const void* k_src, const void* v_src, const int64_t* kv_stride, const int32_t* kept,
                     const int32_t* idx, int32_t m, int32_t Hkv, int32_t k, int32_t d, void* k_out, void* v_out,
                     int32_t* pos_out, void* stream) {
  if (!k_src || !v_src || !kv_stride || !kept || !idx || !k_out || !v_out) return PC_ERR_INVALID_ARG;
  if (m < 1 || Hkv < 1 || k < 1) return PC_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return PC_ERR_UNSUPPORTED;
  if (!aligned16(k_src) || !aligned16(v_src) || !aligned16(k_out) || !aligned16(v_out)) return PC_ERR_INVALID_ARG;
  const long long s[3] = {kv_stride[0], kv_stride[1], kv_stride[2]};
  if (s[0] <= 0 || s[1] <= 0 || s[2] < d || s[0] % 8 || s[1] % 8 || s[2] % 8) return PC_ERR_INVALID_ARG;
  const DeviceInfo& dev = device_info();
  if (dev.ok != 1) return PC_ERR_UNSUPPORTED;
  if (pc::launch_gather_kv(k_src, v_src, s, kept, idx, m, Hkv, k, d, k_out, v_out, pos_out, dev.sm_count, false,
                           static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return PC_ERR_CUDA;
  return PC_OK;
}

// ------------------------------------------------------------------------------------ online chunk queue
int32_t pc_queue_init(int32_t m, float* q_score, int32_t* q_chunk, void* stream) {
  if (!q_score || !q_chunk || m < 1) return PC_ERR_INVALID_ARG;
  if (m > 1023) return PC_ERR_UNSUPPORTED;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  pc::launch_queue_init(q_score, q_chunk, m, static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? PC_OK : PC_ERR_CUDA;
}

int32_t pc_queue_update(const float* chunk_score, int32_t Cb, int32_t chunk_id0, int32_t lower_is_better, int32_t m,
                        float* q_score, int32_t* q_chunk, int32_t* slot_src, void* stream) {
  if (!chunk_score || !q_score || !q_chunk || !slot_src || Cb < 1 || m < 1 || chunk_id0 < 0) return PC_ERR_INVALID_ARG;
  if (chunk_id0 > 0x7FFFFFFF - 1024) return PC_ERR_INVALID_ARG;
  if ((long long)m + Cb > 1024) return PC_ERR_UNSUPPORTED;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  pc::launch_queue_update(chunk_score, Cb, chunk_id0, lower_is_better, m, q_score, q_chunk, slot_src,
                          static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? PC_OK : PC_ERR_CUDA;
}

int32_t pc_queue_gather(const void* k_src, const void* v_src, const int64_t* kv_stride,
                        const int32_t* slot_src, const int32_t* idx, int32_t m, int32_t Hkv, int32_t k, int32_t d,
                        void* q_k, void* q_v, int32_t* q_pos, void* stream) {
  if (!k_src || !v_src || !kv_stride || !slot_src || !idx || !q_k || !q_v || !q_pos) return PC_ERR_INVALID_ARG;
  if (m < 1 || Hkv < 1 || k < 1) return PC_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return PC_ERR_UNSUPPORTED;
  if (!aligned16(k_src) || !aligned16(v_src) || !aligned16(q_k) || !aligned16(q_v)) return PC_ERR_INVALID_ARG;
  const long long s[3] = {kv_stride[0], kv_stride[1], kv_stride[2]};
  if (s[0] <= 0 || s[1] <= 0 || s[2] < d || s[0] % 8 || s[1] % 8 || s[2] % 8) return PC_ERR_INVALID_ARG;
  const DeviceInfo& dev = device_info();
  if (dev.ok != 1) return PC_ERR_UNSUPPORTED;
  if (pc::launch_gather_kv(k_src, v_src, s, slot_src, idx, m, Hkv, k, d, q_k, q_v, q_pos, dev.sm_count, true,
                           static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return PC_ERR_CUDA;
  return PC_OK;
}

int32_t pc_queue_select_gather(const float* win_score, const void* k_src, const void* v_src, const int64_t* kv_stride,
                               const int32_t* slot_src, int32_t m, int32_t Hkv, int32_t L, int32_t n_cand, int32_t k,
                               int32_t d, void* q_k, void* q_v, int32_t* q_pos, void* stream) {
  if (!win_score || !k_src || !v_src || !kv_stride || !slot_src || !q_k || !q_v || !q_pos) return PC_ERR_INVALID_ARG;
  if (m < 1 || Hkv < 1 || L < 1 || n_cand < 1 || n_cand > L || k < 1) return PC_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return PC_ERR_UNSUPPORTED;
  if (n_cand > 32768) return PC_ERR_UNSUPPORTED;
  if (!aligned16(k_src) || !aligned16(v_src) || !aligned16(q_k) || !aligned16(q_v)) return PC_ERR_INVALID_ARG;
  const long long s[3] = {kv_stride[0], kv_stride[1], kv_stride[2]};
  if (s[0] <= 0 || s[1] <= 0 || s[2] < d || s[0] % 8 || s[1] % 8 || s[2] % 8) return PC_ERR_INVALID_ARG;
  if (device_info().ok != 1) return PC_ERR_UNSUPPORTED;
  const cudaError_t e = pc::launch_select_gather_slots(win_score, slot_src, m, Hkv, L, n_cand, k, k_src, v_src, s, d, q_k,
                                                       q_v, q_pos, static_cast<cudaStream_t>(stream));
  if (e == cudaErrorNotSupported) return PC_ERR_UNSUPPORTED;     // k too large to stage: pc_select_tokens + pc_queue_gather
  return e == cudaSuccess ? PC_OK : PC_ERR_CUDA;
}

int32_t pc_queue_emit(const int32_t* q_chunk, int32_t m, int32_t Hkv, int32_t k, int32_t d, const void* q_k,
                      const void* q_v, const int32_t* q_pos, int32_t* kept_out, int32_t* slot_order, void* k_out,
                      void* v_out, int32_t* pos_out, void* stream) {
  if (!q_chunk || !q_k || !q_v || !q_pos || !kept_out || !slot_order || !k_out || !v_out) return PC_ERR_INVALID_ARG;
  if (m < 1 || Hkv < 1 || k < 1) return PC_ERR_INVALID_ARG;
  if (m > 1023) return PC_ERR_UNSUPPORTED;
  if (d != 64 && d != 128) return PC_ERR_UNSUPPORTED;
  if (!aligned16(q_k) || !aligned16(q_v) || !aligned16(k_out) || !aligned16(v_out)) return PC_ERR_INVALID_ARG;
  const DeviceInfo& dev = device_info();
  if (dev.ok != 1) return PC_ERR_UNSUPPORTED;
  if (pc::launch_queue_emit(q_chunk, m, Hkv, k, d, q_k, q_v, q_pos, kept_out, slot_order, k_out, v_out, pos_out,
                            dev.sm_count, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return PC_ERR_CUDA;
  return PC_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------ parallel attention
namespace {

struct ParallelPlan {
  int Gs, n_rg, n_cache_tiles, n_split, tiles_per_split;
  bool alt;                        // single-CTA kernel, rows of an item fit one block: two streams on alternate key tiles
  int n_part;                      // partial results to merge per (sequence, q-head)
  bool pair;                       // CTA-pair kernel: 256-row groups, no key split
  int hpc, n_rg_pair;              // pair kernel: q-heads per CTA, 256-row groups per kv-head
  size_t off_counter, off_table, off_table_hi, off_table_lo, off_qrot, off_ml, off_o, total;
};

// The plan depends only on the sizes and the SM count.
// Head size 128 with whole 256-row groups per (sequence, kv-head) runs on CTA pairs, one group per pair and
// item, without a key split, when the groups fill the pairs' rounds to three quarters or more (the pair kernel is
// about a third faster per tile, a partly filled last round costs it that advantage).
// Otherwise the single-CTA kernel splits the keys.  The number of splits minimises a cost model in units of one
// key tile: rounds of the persistent grid x (fixed cost of an item - query load, pipeline fill, write-out of
// the partial result - of about four tiles + tiles per split).
ParallelPlan parallel_plan(int B, int w, int Hq, int Hkv, int d, int Nk, int sm_count) {
  ParallelPlan p;
  const int G = Hq / Hkv;
  p.Gs = (256 / w) < G ? (256 / w) : G;
  p.n_rg = (G + p.Gs - 1) / p.Gs;
  p.n_cache_tiles = (Nk + 127) / 128;
  const long long base = (long long)B * Hkv * p.n_rg;
  p.pair = false;
  p.hpc = 0; p.n_rg_pair = 0;
  if (d == 128 && w >= 8 && (G * w) % 256 == 0 && sm_count >= 2) {
    const long long pairs = sm_count / 2, groups = (long long)B * Hkv * (G * w / 256);
    const long long rounds = (groups + pairs - 1) / pairs;
    if (4 * groups >= 3 * rounds * pairs) {
      p.pair = true;
      p.hpc = 128 / w;
      p.n_rg_pair = G * w / 256;
    }
  }
  p.tiles_per_split = p.n_cache_tiles;
  if (!p.pair) {
    constexpr long long ITEM_COST_TILES = 4;
    long long best = -1;
    int max_split = p.n_cache_tiles / 2;                       // every split keeps at least two cache tiles
    max_split = max_split < 1 ? 1 : (max_split > 64 ? 64 : max_split);
    for (int s = 1; s <= max_split; ++s) {
      const int tps = (p.n_cache_tiles + s - 1) / s;
      const int ns = (p.n_cache_tiles + tps - 1) / tps;
      const long long rounds = (base * ns + sm_count - 1) / sm_count;
      const long long cost = rounds * (ITEM_COST_TILES + tps + (ns > 1 ? 1 : 0));   // a split run also pays for the merge
      if (best < 0 || cost < best) { best = cost; p.tiles_per_split = tps; }
    }
  }
  if (p.tiles_per_split < 1) p.tiles_per_split = 1;
  p.n_split = p.n_cache_tiles > 0 ? (p.n_cache_tiles + p.tiles_per_split - 1) / p.tiles_per_split : 1;
  size_t off = 0;
  p.off_counter = off; off += ALIGN;
  p.off_table = off; off += align_up((size_t)w * (d / 2) * sizeof(double2));
  p.off_table_hi = off; off += align_up((size_t)w * (d / 4) * sizeof(float4));
  p.off_table_lo = off; off += align_up((size_t)w * (d / 4) * sizeof(float4));
  p.off_qrot = off; off += align_up((size_t)B * w * Hq * d * 2);
  p.alt = !p.pair && p.Gs * w <= 128;
  p.n_part = p.alt ? 2 * p.n_split : p.n_split;
  p.off_ml = off;
  if (p.n_part > 1) off += align_up((size_t)B * Hq * p.n_part * w * 2 * sizeof(float));
  p.off_o = off;
  if (p.n_part > 1) off += align_up((size_t)B * Hq * p.n_part * w * d * sizeof(float));
  p.total = off;
  return p;
}

int32_t check_parallel_args(int B, int w, int Hq, int Hkv, int d, int Nk) {
  if (B < 1 || w < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || Nk < 1) return PC_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return PC_ERR_UNSUPPORTED;
  if (!pow2_between(w, 1, 128)) return PC_ERR_UNSUPPORTED;      // w = 1: one new token decoding over the cache
  if ((long long)B * Hq > (1 << 24) || Nk > (1 << 28)) return PC_ERR_UNSUPPORTED;
  return PC_OK;
}

int plan_sm_count() {
  const DeviceInfo& dev = device_info();
  return dev.ok == 1 && dev.sm_count > 0 ? dev.sm_count : 148;
}

}  // namespace

extern "C" {

size_t pc_parallel_attn_workspace_bytes(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk) {
  if (check_parallel_args(B, w, Hq, Hkv, d, Nk) != PC_OK) return 0;
  return parallel_plan(B, w, Hq, Hkv, d, Nk, plan_sm_count()).total;
}

}  // extern "C"

namespace {

// pc_parallel_attn over caches whose (sequence, kv-head) rows are Nk_cap entries apart (Nk of them valid)
int32_t parallel_attn_impl(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk, int64_t Nk_cap,
                           const void* q_win, int32_t q_pos0, float rope_theta, float softmax_scale, const void* k_cache,
                           const void* v_cache, const void* k_win, const void* v_win, void* out, float* lse_out,
                           int32_t* status_word, void* workspace, size_t workspace_bytes, void* stream) {
  int32_t rc = check_parallel_args(B, w, Hq, Hkv, d, Nk);
  if (rc != PC_OK) return rc;
  if (Nk_cap < Nk || Nk_cap > (1ll << 28)) return PC_ERR_INVALID_ARG;
  if (!q_win || !k_cache || !v_cache || !k_win || !v_win || !out) return PC_ERR_INVALID_ARG;
  if (!aligned16(q_win) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_win) || !aligned16(v_win) ||
      !aligned16(out) || !aligned16(workspace))
    return PC_ERR_INVALID_ARG;
  if (q_pos0 < 0 || !(rope_theta > 0.0f) || softmax_scale < 0.0f) return PC_ERR_INVALID_ARG;
  const DeviceInfo& dev = device_info();
  if (dev.ok != 1) return PC_ERR_UNSUPPORTED;
  const ParallelPlan plan = parallel_plan(B, w, Hq, Hkv, d, Nk, dev.sm_count);
  if (!workspace || workspace_bytes < plan.total) return PC_ERR_WORKSPACE;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int* counter = reinterpret_cast<int*>(ws + plan.off_counter);
  double2* table = reinterpret_cast<double2*>(ws + plan.off_table);

  const uint64_t ud = (uint64_t)d;
  const uint64_t qw_dims[4] = {ud, (uint64_t)Hq, (uint64_t)w, (uint64_t)B};
  const uint64_t qw_str[3] = {ud, (uint64_t)Hq * ud, (uint64_t)w * Hq * ud};
  const uint64_t kc_dims[4] = {ud, (uint64_t)Nk, (uint64_t)Hkv, (uint64_t)B};
  const uint64_t kc_str[3] = {ud, (uint64_t)Nk_cap * ud, (uint64_t)Hkv * (uint64_t)Nk_cap * ud};
  const uint64_t kw_dims[4] = {ud, (uint64_t)Hkv, (uint64_t)w, (uint64_t)B};
  const uint64_t kw_str[3] = {ud, (uint64_t)Hkv * ud, (uint64_t)w * Hkv * ud};
  const uint32_t box_qw[4] = {64, 1, (uint32_t)w, 1};
  const uint32_t box_kc[4] = {64, 128, 1, 1};
  const uint32_t box_kw[4] = {64, 1, 128, 1};

  // rotated queries first (the same pass that serves the chunk-local kernels)
  float4* table_hi = reinterpret_cast<float4*>(ws + plan.off_table_hi);
  float4* table_lo = reinterpret_cast<float4*>(ws + plan.off_table_lo);
  void* q_rot = ws + plan.off_qrot;
  pc::launch_rope_table(table, table_hi, table_lo, w, d, (double)rope_theta, q_pos0, st);
  const long long q_stride[3] = {(long long)w * Hq * d, (long long)Hq * d, (long long)d};
  pc::launch_rope_rows(q_win, q_stride, q_rot, table, table_hi, table_lo, B, w, Hq, d, st);

  if (plan.pair) {
    CUtensorMap pm[6];
    const uint32_t box_kch[4] = {64, 64, 1, 1};
    const uint32_t box_kwh[4] = {64, 1, 64, 1};
    if (!pc::make_tmap_bf16_4d(&pm[0], q_rot, qw_dims, qw_str, box_qw) ||
        !pc::make_tmap_bf16_4d(&pm[1], out, qw_dims, qw_str, box_qw) ||
        !pc::make_tmap_bf16_4d(&pm[2], k_cache, kc_dims, kc_str, box_kch) ||
        !pc::make_tmap_bf16_4d(&pm[3], v_cache, kc_dims, kc_str, box_kc) ||
        !pc::make_tmap_bf16_4d(&pm[4], k_win, kw_dims, kw_str, box_kwh) ||
        !pc::make_tmap_bf16_4d(&pm[5], v_win, kw_dims, kw_str, box_kw))
      return PC_ERR_CUDA;
    pc::ParallelPairParams pp;
    pp.B = B; pp.w = w; pp.Hq = Hq; pp.Hkv = Hkv; pp.Nk = Nk;
    pp.hpc = plan.hpc; pp.n_rg = plan.n_rg_pair;
    const double scale = softmax_scale > 0.0f ? (double)softmax_scale : 1.0 / std::sqrt((double)d);
    pp.scale_log2 = (float)(scale * 1.4426950408889634);
    pp.lse_out = lse_out;
    pp.status = status_word;
    pp.wait_kcycles = pc::g_wait_kcycles.load();
    if (pc::launch_parallel_pair(pm, pp, dev.sm_count, st) != cudaSuccess) return PC_ERR_CUDA;
    return PC_OK;
  }

  CUtensorMap maps[5];
  if (!pc::make_tmap_bf16_4d(&maps[0], q_rot, qw_dims, qw_str, box_qw) ||
      !pc::make_tmap_bf16_4d(&maps[1], k_cache, kc_dims, kc_str, box_kc) ||
      !pc::make_tmap_bf16_4d(&maps[2], v_cache, kc_dims, kc_str, box_kc) ||
      !pc::make_tmap_bf16_4d(&maps[3], k_win, kw_dims, kw_str, box_kw) ||
      !pc::make_tmap_bf16_4d(&maps[4], v_win, kw_dims, kw_str, box_kw))
    return PC_ERR_CUDA;

  if (cudaMemsetAsync(counter, 0, sizeof(int), st) != cudaSuccess) return PC_ERR_CUDA;

  pc::ParallelParams prm;
  prm.B = B; prm.w = w; prm.Hq = Hq; prm.Hkv = Hkv; prm.Nk = Nk;
  prm.Gs = plan.Gs; prm.n_rg = plan.n_rg;
  prm.n_cache_tiles = plan.n_cache_tiles; prm.n_split = plan.n_split; prm.tiles_per_split = plan.tiles_per_split;
  prm.alt = plan.alt ? 1 : 0; prm.n_part = plan.n_part;
  const double scale = softmax_scale > 0.0f ? (double)softmax_scale : 1.0 / std::sqrt((double)d);
  prm.scale_log2 = (float)(scale * 1.4426950408889634);
  prm.part_ml = reinterpret_cast<float*>(ws + plan.off_ml);
  prm.part_o = reinterpret_cast<float*>(ws + plan.off_o);
  prm.out = static_cast<__nv_bfloat16*>(out);
  prm.lse_out = lse_out;
  prm.status = status_word;
  prm.counter = counter;
  prm.wait_kcycles = pc::g_wait_kcycles.load();
  const long long n_items = (long long)B * Hkv * plan.n_rg * plan.n_split;
  const int grid = (int)(n_items < dev.sm_count ? n_items : dev.sm_count);
  if (pc::launch_parallel_attn(maps, prm, d, grid, st) != cudaSuccess) return PC_ERR_CUDA;
  return PC_OK;
}

}  // namespace

extern "C" {

int32_t pc_parallel_attn(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk, const void* q_win,
                         int32_t q_pos0, float rope_theta, float softmax_scale, const void* k_cache,
                         const void* v_cache, const void* k_win, const void* v_win, void* out, float* lse_out,
                         int32_t* status_word, void* workspace, size_t workspace_bytes, void* stream) {
  return parallel_attn_impl(B, w, Hq, Hkv, d, Nk, Nk, q_win, q_pos0, rope_theta, softmax_scale, k_cache, v_cache, k_win,
                            v_win, out, lse_out, status_word, workspace, workspace_bytes, stream);
}

int32_t pc_parallel_attn_append(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk, int32_t Nk_cap,
                                const void* q_win, int32_t q_pos0, float rope_theta, float softmax_scale, void* k_cache,
                                void* v_cache, const void* k_win, const void* v_win, void* out, float* lse_out,
                                int32_t* status_word, void* workspace, size_t workspace_bytes, void* stream) {
  if (Nk_cap < 1 || (int64_t)Nk + w > (int64_t)Nk_cap) return PC_ERR_INVALID_ARG;
  const int32_t rc = parallel_attn_impl(B, w, Hq, Hkv, d, Nk, Nk_cap, q_win, q_pos0, rope_theta, softmax_scale, k_cache,
                                        v_cache, k_win, v_win, out, lse_out, status_word, workspace, workspace_bytes,
                                        stream);
  if (rc != PC_OK) return rc;
  // the attention above reads entries below Nk only (rows behind them read as zeros and are masked): the new rows
  // can follow on the same stream
  if (pc::launch_append_kv(k_win, v_win, B, w, Hkv, d, Nk, Nk_cap, k_cache, v_cache, static_cast<cudaStream_t>(stream)) !=
      cudaSuccess)
    return PC_ERR_CUDA;
  return PC_OK;
}

}  // extern "C"
