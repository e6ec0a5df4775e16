// Joint softmax attention for fp32 tensors (the small fp32 configuration): fp32 throughout on the FMA pipes.
// One warp per query row, key/value tiles of 32 keys staged in shared memory, online softmax per row.
#include "swam_internal.cuh"

namespace swam {
namespace {

constexpr int kRows = 16;  // query rows (warps) per CTA
constexpr int kKeys = 32;  // keys per tile

template <int D>
__global__ void __launch_bounds__(kRows * 32) attn_f32_kernel(const AttnArgs a) {
  __shared__ float Ks[kKeys][D + 1];
  __shared__ float Vs[kKeys][D];
  __shared__ float Qs[kRows][D];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int h = blockIdx.y, b = blockIdx.z;
  const int row = blockIdx.x * kRows + warp;
  const bool active = row < a.n;
  const int row_keys = a.row_limit(row);   // leading keys of the sequence this row sees
  const int64_t tok = (int64_t)a.N_h * D;
  const float* q = (const float*)a.q + ((int64_t)b * a.n) * tok + (int64_t)h * D;
  const int64_t tok_kv = (int64_t)a.N_kv * D;
  const int h_kv = h / (a.N_h / a.N_kv);
  const float* k = (const float*)a.k + ((int64_t)b * a.n) * tok_kv + (int64_t)h_kv * D;
  const float* v = (const float*)a.v + ((int64_t)b * a.n) * tok_kv + (int64_t)h_kv * D;
  if (active)
    for (int d = lane; d < D; d += 32) Qs[warp][d] = q[(int64_t)row * tok + d];

  constexpr int DV = D / 32;
  float o[DV];
#pragma unroll
  for (int i = 0; i < DV; ++i) o[i] = 0.f;
  float m = -INFINITY, l = 0.f;

  for (int c0 = 0; c0 < a.n; c0 += kKeys) {
    __syncthreads();
    for (int i = threadIdx.x; i < kKeys * D; i += kRows * 32) {
      const int kk = i / D, d = i % D;
      const bool in = c0 + kk < a.n;
      Ks[kk][d] = in ? k[(int64_t)(c0 + kk) * tok_kv + d] : 0.f;
      Vs[kk][d] = in ? v[(int64_t)(c0 + kk) * tok_kv + d] : 0.f;
    }
    __syncthreads();
    if (!active) continue;
    float dot = 0.f;
#pragma unroll 8
    for (int d = 0; d < D; ++d) dot = fmaf(Qs[warp][d], Ks[lane][d], dot);
    const float x = (c0 + lane < row_keys) ? dot * a.scale : -INFINITY;
    float mx = x;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
    const float m_new = fmaxf(m, mx);
    const float corr = expf(m - m_new);
    const float pr = expf(x - m_new);
    float ps = pr;
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, s);
    l = l * corr + ps;
    m = m_new;
#pragma unroll
    for (int i = 0; i < DV; ++i) o[i] *= corr;
    for (int kk = 0; kk < kKeys; ++kk) {
      const float pk = __shfl_sync(0xffffffffu, pr, kk);
#pragma unroll
      for (int i = 0; i < DV; ++i) o[i] = fmaf(pk, Vs[kk][lane + 32 * i], o[i]);
    }
  }
  if (!active) return;
  float* out = (float*)a.out + ((int64_t)b * a.n + row) * tok + (int64_t)h * D;
  const float inv = 1.f / l;
#pragma unroll
  for (int i = 0; i < DV; ++i) out[lane + 32 * i] = o[i] * inv;
  if (a.lse && lane == 0 && row >= a.lse_row0 && row < a.lse_row0 + a.lse_rows)
    a.lse[((int64_t)b * a.N_h + h) * a.lse_rows + (row - a.lse_row0)] = m + logf(l);
}

}  // namespace

cudaError_t launch_attn_f32(const AttnArgs& a, cudaStream_t st, int* launches) {
  dim3 grid((a.n + kRows - 1) / kRows, a.N_h, a.B);
  ++*launches;
  switch (a.D) {
    case 32: attn_f32_kernel<32><<<grid, kRows * 32, 0, st>>>(a); break;
    case 64: attn_f32_kernel<64><<<grid, kRows * 32, 0, st>>>(a); break;
    case 128: attn_f32_kernel<128><<<grid, kRows * 32, 0, st>>>(a); break;
    default: return cudaErrorInvalidConfiguration;
  }
  return cudaGetLastError();
}

}  // namespace swam
