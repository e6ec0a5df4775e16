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
  int N_kv;          // heads of k; query head h reads key head h / (N_h / N_kv)
  int keys_per_cta;  // keys of a frame per CTA (<= 16 * MT; fewer leaves the last 16-key tile partly empty)
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
  const int key0 = blockIdx.x * p.keys_per_cta;
  const int key_end = min(p.N_s, key0 + p.keys_per_cta);
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
  const bool v0 = r0 < key_end, v1 = r1 < key_end;
  const int64_t tok_k = (int64_t)p.N_kv * D;
  const int kv_group = p.N_h / p.N_kv;
  const __nv_bfloat16* kbase = p.k + ((int64_t)b * p.L + p.n_obs + (int64_t)f * p.N_s) * tok_k + t * 8;
  const __nv_bfloat16* k0 = kbase + (int64_t)(v0 ? r0 : 0) * tok_k;
  const __nv_bfloat16* k1 = kbase + (int64_t)(v1 ? r1 : 0) * tok_k;

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
    const int hk = (kv_group == 1) ? h : h / kv_group;   // the division only runs for grouped-query shapes
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) {
      a0[buf][kb] = v0 ? ldg_stream(k0 + hk * D + kb * 32) : zero;
      a1[buf][kb] = v1 ? ldg_stream(k1 + hk * D + kb * 32) : zero;
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
  if (tid < kScoreKeys && key0 + tid < key_end) {
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
  int N_kv;
};

__global__ void __launch_bounds__(256) score_f32_kernel(const ScoreParamsF32 p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int f = blockIdx.y, b = blockIdx.z;
  const int j = blockIdx.x * 8 + warp;
  if (j >= p.N_s) return;
  const int64_t tok = (int64_t)p.N_h * p.D;
  const int64_t act0 = (int64_t)p.n_obs + (int64_t)p.F * p.N_s;
  const int kv_group = p.N_h / p.N_kv;
  const float* kt = p.k + ((int64_t)b * p.L + p.n_obs + (int64_t)f * p.N_s + j) * ((int64_t)p.N_kv * p.D);
  float acc = 0.f;
  for (int a = 0; a < p.g; ++a) {
    const int i = f * p.g + a;
    const float* qt = p.q + ((int64_t)b * p.L + act0 + i) * tok;
    for (int h = 0; h < p.N_h; ++h) {
      float dot = 0.f;
      for (int d = lane; d < p.D; d += 32) dot = fmaf(qt[h * p.D + d], kt[(h / kv_group) * p.D + d], dot);
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
  extern __shared__ double2 part_sums[];  // [F * (parts + 1)]
  const int b = blockIdx.x;
  quality_of_scores(scores + (int64_t)b * F * N_s, F, N_s, parts, part_sums, quality + b * 3, (int)threadIdx.x, kQualThreads,
                    [] { __syncthreads(); });
}

// ---- action-row normalisers over all L keys -----------------------------------------------------------
// bf16: CTAs take (head, range of keys) pairs and leave a running (max, sum) per query in the log2 domain in scratch
// [B, ranges, N_h, H]; a second kernel merges the ranges.  The scratch holds one range per 128 keys at most.
constexpr int kLseKeys = 128;


// ---------------------------------------------------------------------------------------------------------
// lambda over all L keys, flash style (the first half of an attention step: scores and running row statistics,
// no values).  A CTA owns up to 64 action queries of one head and a contiguous range of key tiles: the query tile
// is read once into registers as mma.sync A fragments (ldmatrix), key tiles of 64 rows stream through a two-stage
// cp.async pipeline into XOR-swizzled shared memory, and every thread keeps the running (max, sum) of its two query
// rows over the key columns it owns, so the only cross-lane traffic is one quad reduction at the very end.
// WM warps split the query rows (16 each), the remaining 4 / WM warp groups split each key tile's columns.
// ---------------------------------------------------------------------------------------------------------
constexpr int kFlashBN = 64, kFlashThreads = 128;

struct LseFlashParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  float2* partial;          // [B, n_splits, N_h, H] (max, sum) in the log2 domain
  int H, N_h, L, n_splits, tiles_per_split;
  float scale_log2;
  int N_kv;
  int Lk;                   // leading keys the action rows see (<= L)
};

__device__ __forceinline__ void lse_cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void lse_ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// byte offset of 16-byte chunk c of row r in a tile with CPR chunks per row
template <int CPR>
__device__ __forceinline__ uint32_t lse_swz(int r, int c) {
  const int x = (CPR >= 8) ? (r & 7) : ((r >> 1) & 3);
  return (uint32_t)((r * CPR + (c ^ x)) << 4);
}
// rows [row0, row0 + 64) of one head into a swizzled tile; rows at or beyond row_end are zero-filled
template <int D>
__device__ __forceinline__ void lse_load_tile(uint32_t dst, const __nv_bfloat16* base, int64_t row_stride, int row0,
                                              int row_end, int tid) {
  constexpr int CPR = D / 8;
#pragma unroll
  for (int i = tid; i < 64 * CPR; i += kFlashThreads) {
    const int r = i / CPR, c = i % CPR;
    const int gr = row0 + r;
    const bool in = gr < row_end;
    lse_cp_async16(dst + lse_swz<CPR>(r, c), base + (int64_t)(in ? gr : row0) * row_stride + c * 8, in ? 16 : 0);
  }
}

template <int D, int WM>
__global__ void __launch_bounds__(kFlashThreads) lse_flash_bf16_kernel(const LseFlashParams p) {
  constexpr int CPR = D / 8, KS = D / 16;
  constexpr int WN = 4 / WM;                 // warp groups over the key columns
  constexpr int NPW = kFlashBN / 16 / WN;    // 16-key column pairs per warp and tile
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t sQ = (uint32_t)__cvta_generic_to_shared(smem);
  const uint32_t sK = sQ + 64 * D * 2;
  float2* s_red = reinterpret_cast<float2*>(smem);   // reused after the loop: [WN][64]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gq = lane >> 2, t = lane & 3;
  const int wm = warp % WM, wn = warp / WM;
  const int split = blockIdx.x, h = blockIdx.y;
  const int q_chunks = (p.H + 63) / 64;
  const int b = blockIdx.z / q_chunks, qc = blockIdx.z % q_chunks;
  const int64_t rs = (int64_t)p.N_h * D, rs_k = (int64_t)p.N_kv * D;
  const __nv_bfloat16* kb = p.k + (int64_t)b * p.L * rs_k + (int64_t)(h / (p.N_h / p.N_kv)) * D;
  const __nv_bfloat16* qb = p.q + ((int64_t)b * p.L + (p.L - p.H)) * rs + (int64_t)h * D;   // action rows
  const int n_tiles = (p.Lk + kFlashBN - 1) / kFlashBN;
  const int j0 = split * p.tiles_per_split, j1 = min(n_tiles, j0 + p.tiles_per_split);

  lse_load_tile<D>(sQ, qb, rs, qc * 64, p.H, tid);
  if (j0 < j1) lse_load_tile<D>(sK, kb, rs_k, j0 * kFlashBN, p.Lk, tid);
  asm volatile("cp.async.commit_group;" ::: "memory");
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  uint32_t qf[KS][4];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks)
    lse_ldsm_x4(sQ + lse_swz<CPR>(wm * 16 + (lane & 15), ks * 2 + (lane >> 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);

  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  for (int j = j0; j < j1; ++j) {
    const int buf = (j - j0) & 1;
    if (j + 1 < j1) {
      lse_load_tile<D>(sK + (buf ^ 1) * kFlashBN * D * 2, kb, rs_k, (j + 1) * kFlashBN, p.Lk, tid);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const uint32_t kt = sK + buf * kFlashBN * D * 2;
    float s[2 * NPW][4];
#pragma unroll
    for (int i = 0; i < 2 * NPW; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int np = 0; np < NPW; ++np) {
        const int key16 = (wn * NPW + np) * 16;
        uint32_t b0, b1, b2, b3;
        lse_ldsm_x4(kt + lse_swz<CPR>(key16 + (lane & 7) + ((lane >> 4) << 3), ks * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
        mma_bf16_16816(s[2 * np], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b0, b1);
        mma_bf16_16816(s[2 * np + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], b2, b3);
      }
    }
    // log2 domain; keys beyond the sequence count as -inf
    const int c_base = j * kFlashBN + wn * NPW * 16 + 2 * t;
    const bool tail = (j + 1) * kFlashBN > p.Lk;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 2 * NPW; ++i) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int c = c_base + i * 8 + e;
          float v = s[i][2 * r + e] * p.scale_log2;
          if (tail && c >= p.Lk) v = -INFINITY;
          s[i][2 * r + e] = v;
          mx = fmaxf(mx, v);
        }
      }
      const float m_new = fmaxf(m_run[r], mx);
      if (m_new != -INFINITY) {
        float ps = 0.f;
#pragma unroll
        for (int i = 0; i < 2 * NPW; ++i) ps += exp2f(s[i][2 * r] - m_new) + exp2f(s[i][2 * r + 1] - m_new);
        l_run[r] = l_run[r] * exp2f(m_run[r] - m_new) + ps;
        m_run[r] = m_new;
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
  }
  // rows wm * 16 + gq (+ 8): merge the quad's four column subsets, then the WN warp groups through shared memory
#pragma unroll
  for (int r = 0; r < 2; ++r) {
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, m_run[r], o), os = __shfl_xor_sync(0xffffffffu, l_run[r], o);
      merge_ms(m_run[r], l_run[r], om, os);
    }
  }
  __syncthreads();   // the tiles are no longer read
  if (t == 0) {
    s_red[wn * 64 + wm * 16 + gq] = make_float2(m_run[0], l_run[0]);
    s_red[wn * 64 + wm * 16 + gq + 8] = make_float2(m_run[1], l_run[1]);
  }
  __syncthreads();
  if (tid < WM * 16) {
    const int i = qc * 64 + tid;
    if (i < p.H) {
      float m = -INFINITY, l = 0.f;
#pragma unroll
      for (int g = 0; g < WN; ++g) merge_ms(m, l, s_red[g * 64 + tid].x, s_red[g * 64 + tid].y);
      p.partial[(((int64_t)b * p.n_splits + split) * p.N_h + h) * p.H + i] = make_float2(m, l);
    }
  }
}

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
__global__ void __launch_bounds__(128) lse_f32_kernel(const float* q, const float* k, float* lse, int L, int Lk, int H,
                                                      int N_h, int N_kv, int D, float scale) {
  __shared__ float sm[4], ss[4];
  const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int64_t tok = (int64_t)N_h * D;
  const float* qt = q + ((int64_t)b * L + (L - H) + i) * tok + (int64_t)h * D;
  float m = -INFINITY, s = 0.f;
  for (int c = threadIdx.x; c < Lk; c += blockDim.x) {   // the keys the action rows see
    const float* kt = k + ((int64_t)b * L + c) * ((int64_t)N_kv * D) + (int64_t)(h / (N_h / N_kv)) * D;
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
cudaError_t launch_score_bf16_hg(const Dims& d, ScoreParams p, cudaStream_t st, int keys_per_cta) {
  constexpr int kScoreKeys = 16 * MT;
  const size_t smem = (size_t)d.N_h * (D / 32) * NT * 32 * sizeof(uint4) + (size_t)d.N_h * NT * 8 * sizeof(float) +
                      HG * kScoreKeys * sizeof(float);
  if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
  cudaError_t e = cudaFuncSetAttribute(score_bf16_kernel<D, NT, HG, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  p.keys_per_cta = keys_per_cta;
  dim3 grid((d.N_s + keys_per_cta - 1) / keys_per_cta, d.F, d.B);
  score_bf16_kernel<D, NT, HG, MT><<<grid, 32 * MT * HG, smem, st>>>(p);
  return cudaGetLastError();
}

template <int D, int NT>
cudaError_t launch_score_bf16(const Dims& d, const ScoreParams& p, cudaStream_t st) {
  // 32 keys per CTA, except when that gives between one and two CTAs per SM: then one wave of larger CTAs (half the
  // query-fragment staging) finishes sooner, and the frame is cut into as many equal pieces of at most 64 keys as
  // fill the SMs (a piece of 57 keys leaves its last 16-key tile partly empty, which costs nothing: the kernel is
  // bound by the loads)
  const int sms = sm_count();
  const long long n32 = (long long)((d.N_s + 31) / 32) * d.F * d.B;
  if (n32 > sms && n32 <= 2 * sms) {
    const int pieces = sms / (d.F * d.B);                       // per frame
    int keys = pieces > 0 ? (d.N_s + pieces - 1) / pieces : 64;
    if (keys > 64 || keys < 33) keys = 64;
    return launch_score_bf16_hg<D, NT, 4, 4>(d, p, st, keys);
  }
  return launch_score_bf16_hg<D, NT, 4, 2>(d, p, st, 32);
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
                     d.N_h, d.D, d.L, d.g, d.scale, 1.0f / (float)d.N_h, alpha, d.N_kv};
    dim3 grid((d.N_s + 7) / 8, d.F, d.B);
    score_f32_kernel<<<grid, 256, 0, st>>>(p);
    return cudaGetLastError();
  }
  ScoreParams p{(const __nv_bfloat16*)q, (const __nv_bfloat16*)k, lse, scores, d.n_obs, d.F, d.N_s, d.H,
                d.N_h, d.L, d.g, d.scale * kLog2e, 1.0f / (float)d.N_h, alpha, d.N_kv, 32};
  switch (d.D) {
    case 32: return launch_score_bf16_d<32>(d, p, st);
    case 64: return launch_score_bf16_d<64>(d, p, st);
    case 128: return launch_score_bf16_d<128>(d, p, st);
    default: return cudaErrorInvalidConfiguration;
  }
}

cudaError_t launch_quality(const Dims& d, const float* scores, float* quality, cudaStream_t st, int* launches) {
  ++*launches;
  const int parts = quality_parts(d.F);
  quality_kernel<<<d.B, kQualThreads, (size_t)d.F * (parts + 1) * sizeof(double2), st>>>(scores, quality, d.F, d.N_s, parts);
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
                              cudaStream_t st, int* launches, int n_keys) {
  if (d.dtype == 0) {
    ++*launches;
    dim3 grid(d.H, d.N_h, d.B);
    lse_f32_kernel<<<grid, 128, 0, st>>>((const float*)q, (const float*)k, lse, d.L, n_keys, d.H, d.N_h, d.N_kv, d.D, d.scale);
    return cudaGetLastError();
  }
  // key ranges per CTA: enough CTAs for about four per SM, never more ranges than the scratch has room for
  const int n_tiles = (n_keys + kFlashBN - 1) / kFlashBN;
  const int q_chunks = (d.H + 63) / 64;
  const int max_splits = (d.L + kLseKeys - 1) / kLseKeys;
  const int sms = sm_count();
  int want = (4 * sms + d.N_h * d.B * q_chunks - 1) / (d.N_h * d.B * q_chunks);
  want = want < 1 ? 1 : (want > max_splits ? max_splits : want);
  const int per = (n_tiles + want - 1) / want;
  const int n_chunks = (n_tiles + per - 1) / per;     // = number of key ranges
  LseFlashParams p{(const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (float2*)scratch, d.H, d.N_h, d.L, n_chunks, per,
                   d.scale * kLog2e, d.N_kv, n_keys};
  const int wm = d.H > 32 ? 4 : (d.H > 16 ? 2 : 1);     // warps over the query rows, 16 each: H <= 16, <= 32, more
  dim3 grid(n_chunks, d.N_h, d.B * q_chunks);
  cudaError_t e = cudaSuccess;
  *launches += 2;
#define SWAM_LSE_LAUNCH(D_, WM_)                                                                                        \
  do {                                                                                                                  \
    const size_t smem = (size_t)(64 + 2 * kFlashBN) * D_ * 2;                                                           \
    e = cudaFuncSetAttribute(lse_flash_bf16_kernel<D_, WM_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);   \
    if (e == cudaSuccess) lse_flash_bf16_kernel<D_, WM_><<<grid, kFlashThreads, smem, st>>>(p);                         \
  } while (0)
#define SWAM_LSE_DISPATCH(D_)                                                                                           \
  do {                                                                                                                  \
    if (wm == 4) SWAM_LSE_LAUNCH(D_, 4);                                                                                \
    else if (wm == 2) SWAM_LSE_LAUNCH(D_, 2);                                                                           \
    else SWAM_LSE_LAUNCH(D_, 1);                                                                                        \
  } while (0)
  switch (d.D) {
    case 32: SWAM_LSE_DISPATCH(32); break;
    case 64: SWAM_LSE_DISPATCH(64); break;
    case 128: SWAM_LSE_DISPATCH(128); break;
    default: return cudaErrorInvalidConfiguration;
  }
#undef SWAM_LSE_DISPATCH
#undef SWAM_LSE_LAUNCH
  if (e != cudaSuccess) return e;
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 g2((d.N_h * d.H + 7) / 8, d.B);
  lse_merge_kernel<<<g2, 256, 0, st>>>((const float2*)scratch, lse, n_chunks, d.N_h, d.H);
  return cudaGetLastError();
}

}  // namespace swam
