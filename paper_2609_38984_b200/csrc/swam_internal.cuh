// Internal declarations shared by the kernels and the C-ABI layer of libswam.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace swam {

// bits of the device status word
enum : int { ST_BAD_MAP = 1, ST_BAD_COUNT = 2, ST_TIMEOUT = 4 };

constexpr int kMaxGroup = 32;  // largest frame-aligned query group the tensor-core scorer handles

struct Dims {
  int B, n_obs, F, N_s, H, N_h, D, Kc, Ks, K, L, Lp, g, dtype;
  int N_kv;   // key/value heads; query head h reads key/value head h / (N_h / N_kv)
  float scale, beta;
};

struct Alpha {
  float w[kMaxGroup];
};

// Layer quality (Eq. 9) of one sample's scores S [F, N_s] (global or shared memory): R = sum S / F, E = mean normalised
// spatial entropy, Q = R (1 - E), written to out3[0..2].  Called by every thread of a group of `n_threads` threads
// (a multiple of 32; `tid` = index inside the group, `sync` = the group's barrier); part_sums: shared memory,
// F * (parts + 1) entries.  With a_f = sum_j s and b_f = sum_j s ln s the entropy of frame f is ln a_f - b_f / a_f.
// Warps take (frame, part) units, one thread per frame then forms the frame's sum and entropy term (the
// double-precision logarithm is the expensive part), and one thread adds the frames up in ascending order: the result
// does not depend on which kernel, or how many threads, compute it.
template <typename SyncFn>
__device__ __forceinline__ void quality_of_scores(const float* s, int F, int N_s, int parts, double2* part_sums,
                                                  float* out3, int tid, int n_threads, SyncFn sync) {
  const int lane = tid & 31, warp = tid >> 5;
  const int per = (N_s + parts - 1) / parts;
  for (int u = warp; u < F * parts; u += n_threads / 32) {
    const int f = u / parts, part = u % parts;
    const int j1 = min(N_s, (part + 1) * per);
    double a = 0.0, bq = 0.0;
    for (int j = part * per + lane; j < j1; j += 32) {
      const float v = s[f * N_s + j];
      a += (double)v;
      if (v > 0.f) bq += (double)(v * logf(v));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      a += __shfl_xor_sync(0xffffffffu, a, o);
      bq += __shfl_xor_sync(0xffffffffu, bq, o);
    }
    if (lane == 0) part_sums[u] = make_double2(a, bq);
  }
  sync();
  double2* frame_terms = part_sums + F * parts;   // (a_f, entropy term of frame f)
  for (int f = tid; f < F; f += n_threads) {
    double a = 0.0, bq = 0.0;
    for (int q = 0; q < parts; ++q) { a += part_sums[f * parts + q].x; bq += part_sums[f * parts + q].y; }
    frame_terms[f] = make_double2(a, (a > 0.0) ? log(a) - bq / a : 0.0);
  }
  sync();
  if (tid == 0) {
    double total = 0.0, ent = 0.0;
    for (int f = 0; f < F; ++f) {
      total += frame_terms[f].x;
      if (frame_terms[f].x > 0.0) ent += frame_terms[f].y;
    }
    const double R = total / (double)F;
    const double E = ent / ((double)F * log((double)N_s));
    out3[0] = (float)R;
    out3[1] = (float)E;
    out3[2] = (float)(R * (1.0 - E));
  }
}
__host__ __device__ inline int quality_parts(int F) { return F >= 32 ? 1 : 32 / F; }

// Bounded wait on an mbarrier phase, shared by every kernel that waits (attention roles, the bulk-copy ring, the
// self-test): polls until the phase with `parity` completes, `limit_cycles` SM clocks have passed, or (when
// abort_flag is given) another role of the CTA has already given up.  Returns false in the last two cases; on expiry
// it raises *abort_flag so that the CTA's other roles stop waiting too.  The caller reports ST_TIMEOUT and returns.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, unsigned long long limit_cycles,
                                                  volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (abort_flag && *abort_flag) return false;
    if ((unsigned long long)(clock64() - t0) > limit_cycles) {
      if (abort_flag) *abort_flag = 1;
      return false;
    }
  }
}

// (max, sum) pairs of a log-sum-exp in the log2 domain: folds (m2, s2) into (m, s); an empty pair is (-inf, 0)
__device__ __forceinline__ void merge_ms(float& m, float& s, float m2, float s2) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { m = mn; s = 0.f; return; }
  s = s * exp2f(m - mn) + s2 * exp2f(m2 - mn);
  m = mn;
}

// SMs of the current device (queried on every call: a process may hold contexts on several devices)
inline int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    sms = 148;
  return sms;
}

// ---- score.cu -------------------------------------------------------------
// S[b,f,j] (Eq. 12) from the action rows of q, the future rows of k and lambda [B,N_h,H].
cudaError_t launch_score(const Dims& d, const Alpha& alpha, const void* q, const void* k, const float* lse,
                         float* scores, cudaStream_t st, int* launches);
// (R, E, Q) of Eq. 9 per sample from stored scores.
cudaError_t launch_quality(const Dims& d, const float* scores, float* quality, cudaStream_t st, int* launches);
// lambda[b,h,i] = log sum over all L keys of exp(scale q_i.k_c); partial: scratch of lse_scratch_bytes().
size_t lse_scratch_bytes(const Dims& d);
// n_keys: the leading keys of the sequence that the action rows see (d.L = all of them)
cudaError_t launch_action_lse(const Dims& d, const void* q, const void* k, float* lse, void* scratch,
                              cudaStream_t st, int* launches, int n_keys);

// ---- score_tc.cu ----------------------------------------------------------
// One pass over the keys for both the normalisers and the scores (bf16, head dim 64 or 128): a tcgen05 kernel streams K
// once, leaves each key range's (max, sum) per action query in `partial` (lse_scratch_bytes()) and the raw products of
// every future key with its frame's queries in `logits` (score_logits_bytes()); the last CTA of a head merges the
// ranges into lambda (`lam2` in the log2 domain and `lse` in natural-log units, both [B,N_h,H]); a second small kernel
// forms S [B,F,N_s].  `counters` (score_counter_bytes()) must be zero before the first launch and is left zero.
bool score_one_pass_supported(const Dims& d);
size_t score_logits_bytes(const Dims& d);
size_t score_counter_bytes(const Dims& d);
cudaError_t launch_score_one_pass(const Dims& d, const Alpha& alpha, const void* q, const void* k, float* lse, float* lam2,
                                  void* partial, unsigned int* counters, float* logits, int* status, float* scores,
                                  cudaStream_t st, int* launches, int n_keys);

// static device scratch of the allocation-free scoring entry point
constexpr size_t kStaticScratchBytes = 8u << 20;
size_t static_scratch_need(const Dims& d);
// device addresses inside the static array for the current device (first call per device looks the symbol up)
cudaError_t static_scratch(const Dims& d, float** lse, void** partial);

// ---- select.cu ------------------------------------------------------------
size_t select_smem_bytes(const Dims& d);
cudaError_t select_prepare(const Dims& d);  // opt in to the dynamic shared memory the kernel needs
// scores: core map (pool, cores); scores_all: anchor map, nullptr => same as scores
// quality: [B, 3] or nullptr; when given (and select_can_fold_quality(d)) the kernel also writes the Eq. 9 diagnostics
// of `scores`, which saves the separate launch of launch_quality
bool select_can_fold_quality(const Dims& d);
cudaError_t launch_select(const Dims& d, const float* scores, const float* scores_all, int32_t* sel_idx,
                          int32_t* pack_map, int32_t* inv_map, int* status, cudaStream_t st, int* launches,
                          float* quality = nullptr);
int max_layers();
// V and V_all from per-layer scores [n_layers, B, F, N_s] and qualities [n_layers, B, 3]
cudaError_t launch_aggregate(const Dims& d, const float* layer_scores, const float* layer_quality, int n_layers, int k_layer,
                             float* v_core, float* v_all, int32_t* core_layers, cudaStream_t st, int* launches);

// ---- pack_scatter.cu ------------------------------------------------------
// dst[b, p] = src[b, map[b,p]] for up to three tensor pairs (row_bytes per row).
// first_row: the first listed row to copy (rows before it are left out of the launch)
cudaError_t launch_pack(const Dims& d, const void* const src[3], void* const dst[3], const int32_t* pack_map,
                        int* status, cudaStream_t st, int* launches, int first_row = 0);
// in place: out[b, map[b,p]] = out_p[b,p];  blend: out[b,t] = inv[b,t] >= 0 ? out_p[b,inv[b,t]] : cached[b,t]
// rows pack_map names, from full tensors in device-mapped host memory to the same rows of full tensors in device memory
// (first_row: the first listed row to bring)
cudaError_t launch_host_rows(const Dims& d, const void* const src[3], void* const dst[3], const int32_t* pack_map,
                             int* status, cudaStream_t st, int* launches, int first_row = 0);
cudaError_t launch_scatter(const Dims& d, const void* out_p, const int32_t* pack_map, const int32_t* inv_map,
                           const void* cached, void* out, int* status, cudaStream_t st, int* launches);

// ---- wait_probe.cu --------------------------------------------------------
// one warp waits, bounded by limit_cycles, on a barrier that nothing completes, and reports ST_TIMEOUT
cudaError_t launch_wait_probe(int* status, unsigned long long limit_cycles, cudaStream_t st, int* launches);
// an empty kernel: the launch-latency floor
cudaError_t launch_noop(cudaStream_t st, int* launches);

// ---- attn_*.cu ------------------------------------------------------------
struct AttnArgs {
  const void* q;
  const void* k;
  const void* v;
  void* out;
  float* lse;        // [B, N_h, lse_rows] or nullptr
  int lse_row0;      // first query row whose normaliser is written
  int lse_rows;      // number of rows written from lse_row0
  int B, n, N_h, D;  // n = sequence length of this call
  float scale;
  int N_kv;          // heads of k and v (q and out have N_h); query head h reads head h / (N_h / N_kv)
  // Gather mode of the tensor-core kernel: the first direct_rows rows (a multiple of 128) of the packed K and V are the
  // same rows of the full tensors k_full and v_full (the observed tokens lead both sequences), so the kernel reads those
  // key tiles from the full tensors and the packed ones need not hold them.  0 = every tile comes from k and v.
  const void* k_full = nullptr;
  const void* v_full = nullptr;
  int direct_rows = 0;
  // Segment-prefix visibility: rows [0, obs_end) see the first lim[0] keys, rows [obs_end, fut_end) the first lim[1],
  // the rest the first lim[2].  Full visibility: every lim = n (then obs_end and fut_end do not matter).
  int obs_end, fut_end, lim[3];
  __host__ __device__ bool full_visibility() const { return lim[0] >= n && lim[1] >= n && lim[2] >= n; }
  __host__ __device__ int row_limit(int row) const { return row < obs_end ? lim[0] : (row < fut_end ? lim[1] : lim[2]); }
  // the largest limit among rows [r0, r1) (r1 > r0)
  __host__ __device__ int max_limit(int r0, int r1) const {
    int m = row_limit(r0);
    if (r1 - 1 >= obs_end && r0 < fut_end) m = m > lim[1] ? m : lim[1];
    if (r1 - 1 >= fut_end) m = m > lim[2] ? m : lim[2];
    return m;
  }
};
cudaError_t launch_attn_f32(const AttnArgs& a, cudaStream_t st, int* launches);
cudaError_t launch_attn_bf16_mma(const AttnArgs& a, cudaStream_t st, int* launches);
// tcgen05 / TMEM / TMA kernel, head_dim 64 or 128; bounded waits report through the status word
// scratch: room for the partial results of the key-split tail items (attn_tc_scratch_bytes), may be nullptr
size_t attn_tc_scratch_bytes(int D);
cudaError_t launch_attn_bf16_tc(const AttnArgs& a, int* status, void* scratch, size_t scratch_bytes, cudaStream_t st,
                                int* launches);
// Packed attention with Eq. 7's scatter and the query third of Sec. 4.2's pack fused in: a.k and a.v are packed
// tensors [B, a.n, N_kv, D]; a.q and a.out are FULL tensors [B, n_full, N_h, D].  The kernel fetches query row
// pack_map[b, i] for attended row i itself and writes the result to row pack_map[b, i] of a.out.  Rows that pack_map
// does not name are not touched.  a.lse is ignored.
// gather_kv: a.k and a.v are FULL tensors [B, n_full, N_kv, D] as well and the kernel fetches the key and value rows
// pack_map names itself (TMA row gathers), so that no packed tensor exists.
cudaError_t launch_attn_bf16_tc_gather(const AttnArgs& a, const int32_t* pack_map, int n_full, bool gather_kv, int* status,
                                       void* scratch, size_t scratch_bytes, cudaStream_t st, int* launches);

}  // namespace swam
