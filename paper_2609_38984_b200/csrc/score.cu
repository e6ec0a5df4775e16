// Action-to-future scoring (Eq. 12) and the action-row normalisers it needs.
//
// The scorer is a stream over the future keys: every key row is read exactly once, multiplied against the
// g = H/F action queries aligned with its frame (Eq. 8), and reduced over heads and queries into one float.
// At g = 8 that is 8 FMAs per loaded bf16 element, more than the FP32 pipes sustain at HBM speed, so the
// bf16 path feeds the (skinny) products to mma.sync m16n8k16 directly from 16-byte global loads: because a
// dot product does not care about the order of its terms, each thread's 16-byte chunk of a key row is used
// as four k-slots of two MMAs and the query fragment is the same 16-byte chunk of the query row.
#include <mutex>

#include "swam_internal.cuh"

namespace swam {
namespace {

// Scratch of the allocation-free scoring entry point: the action-row normalisers followed by the per-chunk
// (max, sum) partials.  It lives in the library image, so every GPU that loads the library holds these bytes until
// the process exits.  In host code the name is only a stand-in for the symbol: kernels must be given the address
// that cudaGetSymbolAddress returns for the current device, never the name itself.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct ScoreParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const float* lse;  // [B, N_h, H]
  float* scores;     // [B, F, N_s]
  int n_obs, F, N_s, H, N_h, L, g;
  float scale_log2, inv_nh;
  Alpha alpha;
};


// smem: query fragments [N_h][D/32][NT][32] uint4, lambda*log2e [N_h][NT*8], partial sums [4][32]
template <int D, int NT, int kHeadGroups, int MT>
__global__ void __launch_bounds__(32 * MT * kHeadGroups, 16 / (MT * kHeadGroups)) score_bf16_kernel(const ScoreParams p) {
  constexpr int KB = D / 32;
  constexpr int kScoreThreads = 32 * MT * kHeadGroups;
  constexpr int kScoreKeys = 16 * MT;  // keys per CTA: MT m-tiles of 16
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* q_frag = reinterpret_cast<uint4*>(smem_raw);
  float* lam2 = reinterpret_cast<float*>(q_frag + (size_t)p.N_h * KB * NT * 32);
  float* red = lam2 + p.N_h * NT * 8;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int f = blockIdx.y, b = blockIdx.z;
  const int key0 = blockIdx.x * kScoreKeys;
  const int64_t act0 = (int64_t)p.n_obs + (int64_t)p.F * p.N_s;
  const int64_t tok = (int64_t)p.N_h * D;

  // stage this frame's query group as MMA B fragments (zero beyond the group): asynchronous 16-byte copies, all in
  // flight at once, overlapped with the first key loads below
  const int n_frag = p.N_h * KB * NT * 32;
  for (int i = tid; i < n_frag; i += kScoreThreads) {
    const int ln = i & 31;
    const int nt = (i >> 5) % NT;
    const int kb = ((i >> 5) / NT) % KB;
    const int h = (i >> 5) / (NT * KB);
    const int n = nt * 8 + (ln >> 2), t = ln & 3;
    const bool in = n < p.g;
    const __nv_bfloat16* src = p.q + ((int64_t)b * p.L + act0 + (int64_t)f * p.g + (in ? n : 0)) * tok + (int64_t)h * D +
                               kb * 32 + t * 8;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(q_frag + i)),
                 "l"(src), "r"(in ? 16 : 0) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  for (int i = tid; i < p.N_h * NT * 8; i += kScoreThreads) {
    const int n = i % (NT * 8), h = i / (NT * 8);
    lam2[i] = (n < p.g) ? p.lse[((int64_t)b * p.N_h + h) * p.H + f * p.g + n] * kLog2e : 0.f;
  }

  const int mt = warp % MT, hg = warp / MT;
  const int gq = lane >> 2, t = lane & 3;
  const int r0 = key0 + mt * 16 + gq, r1 = r0 + 8;
  const bool v0 = r0 < p.N_s, v1 = r1 < p.N_s;
  const __nv_bfloat16* kbase = p.k + ((int64_t)b * p.L + p.n_obs + (int64_t)f * p.N_s) * tok + t * 8;
  const __nv_bfloat16* k0 = kbase + (int64_t)(v0 ? r0 : 0) * tok;
  const __nv_bfloat16* k1 = kbase + (int64_t)(v1 ? r1 : 0) * tok;

  float w[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    w[nt][0] = p.alpha.w[nt * 8 + 2 * t];
    w[nt][1] = p.alpha.w[nt * 8 + 2 * t + 1];
  }

  float sum0 = 0.f, sum1 = 0.f;
  uint4 a0[2][KB], a1[2][KB];
  const uint4 zero = make_uint4(0, 0, 0, 0);
  auto load = [&](int h, int buf) {
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) {
      a0[buf][kb] = v0 ? ldg_stream(k0 + (int64_t)h * D + kb * 32) : zero;
      a1[buf][kb] = v1 ? ldg_stream(k1 + (int64_t)h * D + kb * 32) : zero;
    }
  };
  auto compute = [&](int h, int buf) {
    float c[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const uint4 bq = q_frag[((h * KB + kb) * NT + nt) * 32 + lane];
        mma_bf16_16816(c[nt], a0[buf][kb].x, a1[buf][kb].x, a0[buf][kb].y, a1[buf][kb].y, bq.x, bq.y);
        mma_bf16_16816(c[nt], a0[buf][kb].z, a1[buf][kb].z, a0[buf][kb].w, a1[buf][kb].w, bq.z, bq.w);
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float l0 = lam2[h * NT * 8 + nt * 8 + 2 * t], l1 = lam2[h * NT * 8 + nt * 8 + 2 * t + 1];
      sum0 += w[nt][0] * exp2f(c[nt][0] * p.scale_log2 - l0) + w[nt][1] * exp2f(c[nt][1] * p.scale_log2 - l1);
      sum1 += w[nt][0] * exp2f(c[nt][2] * p.scale_log2 - l0) + w[nt][1] * exp2f(c[nt][3] * p.scale_log2 - l1);
    }
  };

  // heads hg, hg+4, ... with the next head's keys in flight while this head's products run
  int h = hg;
  if (h < p.N_h) load(h, 0);
  if (h + kHeadGroups < p.N_h) load(h + kHeadGroups, 1);
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  for (; h < p.N_h; h += 2 * kHeadGroups) {
    const int h1 = h + kHeadGroups, h2 = h + 2 * kHeadGroups;
    if (h != hg && h1 < p.N_h) load(h1, 1);
    compute(h, 0);
    if (h1 < p.N_h) {
      if (h2 < p.N_h) load(h2, 0);
      compute(h1, 1);
    }
  }

  sum0 += __shfl_xor_sync(0xffffffffu, sum0, 1);
  sum0 += __shfl_xor_sync(0xffffffffu, sum0, 2);
  sum1 += __shfl_xor_sync(0xffffffffu, sum1, 1);
  sum1 += __shfl_xor_sync(0xffffffffu, sum1, 2);
  if (t == 0) {
    red[hg * kScoreKeys + mt * 16 + gq] = sum0;
    red[hg * kScoreKeys + mt * 16 + gq + 8] = sum1;
  }
  __syncthreads();
  if (tid < kScoreKeys && key0 + tid < p.N_s) {
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < kHeadGroups; q += 4)
      s += (red[q * kScoreKeys + tid] + red[(q + 1) * kScoreKeys + tid]) +
           (red[(q + 2) * kScoreKeys + tid] + red[(q + 3) * kScoreKeys + tid]);
    p.scores[((int64_t)b * p.F + f) * p.N_s + key0 + tid] = s * p.inv_nh;
  }
}

// fp32 inputs: one warp per key, lanes across the head dimension
struct ScoreParamsF32 {
  const float* q;
  const float* k;
  const float* lse;
  float* scores;
  int n_obs, F, N_s, H, N_h, D, L, g;
  float scale, inv_nh;
  Alpha alpha;
};

__global__ void __launch_bounds__(256) score_f32_kernel(const ScoreParamsF32 p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int f = blockIdx.y, b = blockIdx.z;
  const int j = blockIdx.x * 8 + warp;
  if (j >= p.N_s) return;
  const int64_t tok = (int64_t)p.N_h * p.D;
  const int64_t act0 = (int64_t)p.n_obs + (int64_t)p.F * p.N_s;
  const float* kt = p.k + ((int64_t)b * p.L + p.n_obs + (int64_t)f * p.N_s + j) * tok;
  float acc = 0.f;
  for (int a = 0; a < p.g; ++a) {
    const int i = f * p.g + a;
    const float* qt = p.q + ((int64_t)b * p.L + act0 + i) * tok;
    for (int h = 0; h < p.N_h; ++h) {
      float dot = 0.f;
      for (int d = lane; d < p.D; d += 32) dot = fmaf(qt[h * p.D + d], kt[h * p.D + d], dot);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      acc += p.alpha.w[a] * expf(p.scale * dot - p.lse[((int64_t)b * p.N_h + h) * p.H + i]);
    }
  }
  if (lane == 0) p.scores[((int64_t)b * p.F + f) * p.N_s + j] = acc * p.inv_nh;
}

// ---- layer quality (Eq. 9): R = sum S / F, E = mean normalised spatial entropy, Q = R (1 - E) ----------
// One CTA per sample, one pass over the scores: with a_f = sum_j s and b_f = sum_j s ln s the entropy of frame f is
// ln a_f - b_f / a_f.  Warps take (frame, part) units; partial sums are combined in a fixed order.
constexpr int kQualThreads = 1024;

__global__ void __launch_bounds__(kQualThreads) quality_kernel(const float* scores, float* quality, int F, int N_s,
                                                               int parts) {
  extern __shared__ double2 part_sums[];  // [F * parts]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, b = blockIdx.x;
  const float* s = scores + (int64_t)b * F * N_s;
  const int per = (N_s + parts - 1) / parts;
  for (int u = warp; u < F * parts; u += kQualThreads / 32) {
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
  __syncthreads();
  if (threadIdx.x == 0) {
    double total = 0.0, ent = 0.0;
    for (int f = 0; f < F; ++f) {
      double a = 0.0, bq = 0.0;
      for (int q = 0; q < parts; ++q) { a += part_sums[f * parts + q].x; bq += part_sums[f * parts + q].y; }
      total += a;
      if (a > 0.0) ent += log(a) - bq / a;
    }
    const double R = total / (double)F;
    const double E = ent / ((double)F * log((double)N_s));
    quality[b * 3 + 0] = (float)R;
    quality[b * 3 + 1] = (float)E;
    quality[b * 3 + 2] = (float)(R * (1.0 - E));
  }
}

// ---- action-row normalisers over all L keys -----------------------------------------------------------
// bf16: each CTA takes 128 keys (8 warps x 16), loops over heads, multiplies against all H action queries
// (NT = H/8 column tiles) and keeps a running (max, sum) per query in the log2 domain; the per-CTA partials
// go to scratch [B, chunks, N_h, H] and a second kernel merges them.
constexpr int kLseKeys = 128;
constexpr int kLseThreads = 256;

struct LseParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  float2* partial;
  int H, N_h, L, n_chunks, NT;
  float scale_log2;
};

__device__ __forceinline__ void merge_ms(float& m, float& s, float m2, float s2) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { m = mn; s = 0.f; return; }
  s = s * exp2f(m - mn) + s2 * exp2f(m2 - mn);
  m = mn;
}

constexpr int kLseHeads = 4;  // heads per CTA

template <int D>
__global__ void __launch_bounds__(kLseThreads) lse_partial_bf16_kernel(const LseParams p) {
  constexpr int KB = D / 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n_frag = KB * p.NT * 32;
  uint4* q_frag = reinterpret_cast<uint4*>(smem_raw);                     // [2][KB][NT][32]
  float2* wpart = reinterpret_cast<float2*>(q_frag + (size_t)2 * n_frag);  // [8 warps][NT*8]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunk = blockIdx.x, h0 = blockIdx.y * kLseHeads, b = blockIdx.z;
  const int64_t tok = (int64_t)p.N_h * D;
  const int gq = lane >> 2, t = lane & 3;
  const int r0 = chunk * kLseKeys + warp * 16 + gq, r1 = r0 + 8;
  const bool v0 = r0 < p.L, v1 = r1 < p.L;
  const __nv_bfloat16* k0 = p.k + ((int64_t)b * p.L + (v0 ? r0 : 0)) * tok + t * 8;
  const __nv_bfloat16* k1 = p.k + ((int64_t)b * p.L + (v1 ? r1 : 0)) * tok + t * 8;
  const int64_t act0 = (int64_t)p.L - p.H;
  const uint4 zero = make_uint4(0, 0, 0, 0);

  auto stage_q = [&](int h, int buf) {  // this head's H queries as B fragments, asynchronously
    for (int i = tid; i < n_frag; i += kLseThreads) {
      const int ln = i & 31;
      const int nt = (i >> 5) % p.NT;
      const int kb = (i >> 5) / p.NT;
      const int n = nt * 8 + (ln >> 2);
      const bool in = n < p.H;
      const __nv_bfloat16* src = p.q + ((int64_t)b * p.L + act0 + (in ? n : 0)) * tok + (int64_t)h * D + kb * 32 + (ln & 3) * 8;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                   ::"r"((uint32_t)__cvta_generic_to_shared(q_frag + (size_t)buf * n_frag + i)), "l"(src), "r"(in ? 16 : 0)
                   : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  uint4 a0[2][KB], a1[2][KB];
  auto load_k = [&](int h, int buf) {
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) {
      a0[buf][kb] = v0 ? ldg_stream(k0 + (int64_t)h * D + kb * 32) : zero;
      a1[buf][kb] = v1 ? ldg_stream(k1 + (int64_t)h * D + kb * 32) : zero;
    }
  };

  stage_q(h0, 0);
  load_k(h0, 0);
#pragma unroll
  for (int hi = 0; hi < kLseHeads; ++hi) {
    const int h = h0 + hi;
    if (h >= p.N_h) break;
    const bool more = (hi + 1 < kLseHeads) && (h + 1 < p.N_h);
    if (more) {
      stage_q(h + 1, (hi + 1) & 1);
      load_k(h + 1, (hi + 1) & 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const uint4* qf = q_frag + (size_t)(hi & 1) * n_frag;
    for (int nt = 0; nt < p.NT; ++nt) {
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kb = 0; kb < KB; ++kb) {
        const uint4 bq = qf[(kb * p.NT + nt) * 32 + lane];
        mma_bf16_16816(c, a0[hi & 1][kb].x, a1[hi & 1][kb].x, a0[hi & 1][kb].y, a1[hi & 1][kb].y, bq.x, bq.y);
        mma_bf16_16816(c, a0[hi & 1][kb].z, a1[hi & 1][kb].z, a0[hi & 1][kb].w, a1[hi & 1][kb].w, bq.z, bq.w);
      }
      // columns 2t, 2t+1; rows gq (c0, c1) and gq+8 (c2, c3): column max over the warp's 16 keys, then the sum
      const float x00 = v0 ? c[0] * p.scale_log2 : -INFINITY, x01 = v0 ? c[1] * p.scale_log2 : -INFINITY;
      const float x10 = v1 ? c[2] * p.scale_log2 : -INFINITY, x11 = v1 ? c[3] * p.scale_log2 : -INFINITY;
      float m0 = fmaxf(x00, x10), m1 = fmaxf(x01, x11);
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
      }
      float s0 = (m0 == -INFINITY) ? 0.f : exp2f(x00 - m0) + exp2f(x10 - m0);
      float s1 = (m1 == -INFINITY) ? 0.f : exp2f(x01 - m1) + exp2f(x11 - m1);
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        s0 += __shfl_xor_sync(0xffffffffu, s0, o);
        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
      }
      if (gq == 0) {
        wpart[warp * p.NT * 8 + nt * 8 + 2 * t] = make_float2(m0, s0);
        wpart[warp * p.NT * 8 + nt * 8 + 2 * t + 1] = make_float2(m1, s1);
      }
    }
    __syncthreads();
    for (int n = tid; n < p.H; n += kLseThreads) {
      float m = -INFINITY, sacc = 0.f;
      for (int w = 0; w < 8; ++w) {
        const float2 ws = wpart[w * p.NT * 8 + n];
        merge_ms(m, sacc, ws.x, ws.y);
      }
      p.partial[(((int64_t)b * p.n_chunks + chunk) * p.N_h + h) * p.H + n] = make_float2(m, sacc);
    }
    // the next head's barrier (after its wait) orders these reads of wpart before its writes
  }
}

// merges the per-chunk partials: lambda = ln2 * (m + log2 s); one warp per (sample, head, query)
__global__ void __launch_bounds__(256) lse_merge_kernel(const float2* partial, float* lse, int n_chunks, int N_h, int H) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int b = blockIdx.y;
  if (i >= N_h * H) return;
  float m = -INFINITY, s = 0.f;
  for (int c = lane; c < n_chunks; c += 32) {
    const float2 ms = partial[((int64_t)b * n_chunks + c) * N_h * H + i];
    merge_ms(m, s, ms.x, ms.y);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o), os = __shfl_xor_sync(0xffffffffu, s, o);
    merge_ms(m, s, om, os);
  }
  if (lane == 0) lse[(int64_t)b * N_h * H + i] = (m + log2f(s)) * 0.6931471805599453f;
}

// fp32: one CTA per (b, h, i); threads stride over keys with a running (max, sum) in natural-log units
__global__ void __launch_bounds__(128) lse_f32_kernel(const float* q, const float* k, float* lse, int L, int H,
                                                      int N_h, int D, float scale) {
  __shared__ float sm[4], ss[4];
  const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int64_t tok = (int64_t)N_h * D;
  const float* qt = q + ((int64_t)b * L + (L - H) + i) * tok + (int64_t)h * D;
  float m = -INFINITY, s = 0.f;
  for (int c = threadIdx.x; c < L; c += blockDim.x) {
    const float* kt = k + ((int64_t)b * L + c) * tok + (int64_t)h * D;
    float dot = 0.f;
    for (int d = 0; d < D; ++d) dot = fmaf(qt[d], kt[d], dot);
    const float x = dot * scale;
    const float mn = fmaxf(m, x);
    s = s * expf(m - mn) + expf(x - mn);
    m = mn;
  }
  auto merge = [](float& m, float& s, float m2, float s2) {
    const float mn = fmaxf(m, m2);
    if (mn == -INFINITY) { s = 0.f; m = mn; return; }
    s = s * expf(m - mn) + s2 * expf(m2 - mn);
    m = mn;
  };
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o), os = __shfl_xor_sync(0xffffffffu, s, o);
    merge(m, s, om, os);
  }
  if ((threadIdx.x & 31) == 0) { sm[threadIdx.x >> 5] = m; ss[threadIdx.x >> 5] = s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) merge(m, s, sm[w], ss[w]);
    lse[((int64_t)b * N_h + h) * H + i] = m + logf(s);
  }
}

template <int D, int NT, int HG, int MT>
cudaError_t launch_score_bf16_hg(const Dims& d, const ScoreParams& p, cudaStream_t st) {
  constexpr int kScoreKeys = 16 * MT;
  const size_t smem = (size_t)d.N_h * (D / 32) * NT * 32 * sizeof(uint4) + (size_t)d.N_h * NT * 8 * sizeof(float) +
                      HG * kScoreKeys * sizeof(float);
  if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
  cudaError_t e = cudaFuncSetAttribute(score_bf16_kernel<D, NT, HG, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((d.N_s + kScoreKeys - 1) / kScoreKeys, d.F, d.B);
  score_bf16_kernel<D, NT, HG, MT><<<grid, 32 * MT * HG, smem, st>>>(p);
  return cudaGetLastError();
}

template <int D, int NT>
cudaError_t launch_score_bf16(const Dims& d, const ScoreParams& p, cudaStream_t st) {
  // 32 keys per CTA, except when that gives between one and two CTAs per SM: then 64-key CTAs (one per SM, half the
  // query-fragment staging) finish sooner
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  }
  const long long n32 = (long long)((d.N_s + 31) / 32) * d.F * d.B;
  if (n32 > sms && n32 <= 2 * sms) return launch_score_bf16_hg<D, NT, 4, 4>(d, p, st);
  return launch_score_bf16_hg<D, NT, 4, 2>(d, p, st);
}

template <int D>
cudaError_t launch_score_bf16_d(const Dims& d, const ScoreParams& p, cudaStream_t st) {
  const int nt = (d.g + 7) / 8;
  switch (nt) {
    case 1: return launch_score_bf16<D, 1>(d, p, st);
    case 2: return launch_score_bf16<D, 2>(d, p, st);
    case 3: case 4: return launch_score_bf16<D, 4>(d, p, st);
    default: return cudaErrorInvalidConfiguration;
  }
}

}  // namespace

cudaError_t launch_score(const Dims& d, const Alpha& alpha, const void* q, const void* k, const float* lse,
                         float* scores, cudaStream_t st, int* launches) {
  ++*launches;
  if (d.dtype == 0) {
    ScoreParamsF32 p{(const float*)q, (const float*)k, lse, scores, d.n_obs, d.F, d.N_s, d.H,
                     d.N_h, d.D, d.L, d.g, d.scale, 1.0f / (float)d.N_h, alpha};
    dim3 grid((d.N_s + 7) / 8, d.F, d.B);
    score_f32_kernel<<<grid, 256, 0, st>>>(p);
    return cudaGetLastError();
  }
  ScoreParams p{(const __nv_bfloat16*)q, (const __nv_bfloat16*)k, lse, scores, d.n_obs, d.F, d.N_s, d.H,
                d.N_h, d.L, d.g, d.scale * kLog2e, 1.0f / (float)d.N_h, alpha};
  switch (d.D) {
    case 32: return launch_score_bf16_d<32>(d, p, st);
    case 64: return launch_score_bf16_d<64>(d, p, st);
    case 128: return launch_score_bf16_d<128>(d, p, st);
    default: return cudaErrorInvalidConfiguration;
  }
}

cudaError_t launch_quality(const Dims& d, const float* scores, float* quality, cudaStream_t st, int* launches) {
  ++*launches;
  int parts = 32 / d.F;
  if (parts < 1) parts = 1;
  quality_kernel<<<d.B, kQualThreads, (size_t)d.F * parts * sizeof(double2), st>>>(scores, quality, d.F, d.N_s, parts);
  return cudaGetLastError();
}

size_t lse_scratch_bytes(const Dims& d) {
  if (d.dtype == 0) return 0;
  const size_t chunks = (d.L + kLseKeys - 1) / kLseKeys;
  return (size_t)d.B * chunks * d.N_h * d.H * sizeof(float2);
}

size_t static_scratch_need(const Dims& d) {
  const size_t lse_bytes = ((size_t)d.B * d.N_h * d.H * sizeof(float) + 255) / 256 * 256;
  return lse_bytes + lse_scratch_bytes(d);
}

cudaError_t static_scratch(const Dims& d, float** lse, void** partial) {
  // one look-up per device, made with that device current; later calls reuse the cached address
  static std::mutex mu;
  static void* base[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!base[dev]) {
      void* ptr = nullptr;
      e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
      if (e != cudaSuccess) return e;
      base[dev] = ptr;
    }
  }
  const size_t lse_bytes = ((size_t)d.B * d.N_h * d.H * sizeof(float) + 255) / 256 * 256;
  *lse = (float*)base[dev];
  *partial = (unsigned char*)base[dev] + lse_bytes;
  return cudaSuccess;
}

cudaError_t launch_action_lse(const Dims& d, const void* q, const void* k, float* lse, void* scratch,
                              cudaStream_t st, int* launches) {
  if (d.dtype == 0) {
    ++*launches;
    dim3 grid(d.H, d.N_h, d.B);
    lse_f32_kernel<<<grid, 128, 0, st>>>((const float*)q, (const float*)k, lse, d.L, d.H, d.N_h, d.D, d.scale);
    return cudaGetLastError();
  }
  const int n_chunks = (d.L + kLseKeys - 1) / kLseKeys;
  const int NT = (d.H + 7) / 8;
  LseParams p{(const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (float2*)scratch, d.H, d.N_h, d.L, n_chunks, NT,
              d.scale * kLog2e};
  const size_t smem = (size_t)2 * (d.D / 32) * NT * 32 * sizeof(uint4) + (size_t)8 * NT * 8 * sizeof(float2);
  if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
  dim3 grid(n_chunks, (d.N_h + kLseHeads - 1) / kLseHeads, d.B);
  cudaError_t e = cudaSuccess;
  *launches += 2;
  switch (d.D) {
    case 32:
      e = cudaFuncSetAttribute(lse_partial_bf16_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e == cudaSuccess) lse_partial_bf16_kernel<32><<<grid, kLseThreads, smem, st>>>(p);
      break;
    case 64:
      e = cudaFuncSetAttribute(lse_partial_bf16_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e == cudaSuccess) lse_partial_bf16_kernel<64><<<grid, kLseThreads, smem, st>>>(p);
      break;
    case 128:
      e = cudaFuncSetAttribute(lse_partial_bf16_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e == cudaSuccess) lse_partial_bf16_kernel<128><<<grid, kLseThreads, smem, st>>>(p);
      break;
    default: return cudaErrorInvalidConfiguration;
  }
  if (e != cudaSuccess) return e;
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 g2((d.N_h * d.H + 7) / 8, d.B);
  lse_merge_kernel<<<g2, 256, 0, st>>>((const float2*)scratch, lse, n_chunks, d.N_h, d.H);
  return cudaGetLastError();
}

}  // namespace swam
