// Joint softmax attention for bf16 tensors on the warp-level tensor-core path (mma.sync m16n8k16).
// Flash-style: a CTA owns 64 query rows of one (sample, head), 4 warps x 16 rows; key/value tiles of 64 rows
// arrive through a two-stage cp.async pipeline into XOR-swizzled shared memory and are read with ldmatrix;
// scores, running max/sum and the output accumulator stay in fp32 registers (online softmax, exp2 domain).
// This kernel is the validated second opinion for the tcgen05 kernel and serves head dims it does not cover.
#include "swam_internal.cuh"

namespace swam {
namespace {

constexpr int BM = 64, BN = 64, kThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte chunk c of row r in a tile with CPR chunks per row
template <int CPR>
__device__ __forceinline__ uint32_t swz(int r, int c) {
  const int x = (CPR >= 8) ? (r & 7) : ((r >> 1) & 3);
  return (uint32_t)((r * CPR + (c ^ x)) << 4);
}

// rows [row0, row0+64) of one head into a swizzled tile; rows >= n are zero-filled
template <int D>
__device__ __forceinline__ void load_tile(uint32_t dst, const __nv_bfloat16* base, int64_t row_stride, int row0, int n,
                                          int tid) {
  constexpr int CPR = D / 8;
#pragma unroll
  for (int i = tid; i < 64 * CPR; i += kThreads) {
    const int r = i / CPR, c = i % CPR;
    const int gr = row0 + r;
    const bool in = gr < n;
    cp_async16(dst + swz<CPR>(r, c), base + (int64_t)(in ? gr : 0) * row_stride + c * 8, in ? 16 : 0);
  }
}

template <int D>
__global__ void __launch_bounds__(kThreads) attn_bf16_mma_kernel(const AttnArgs a) {
  constexpr int CPR = D / 8, KS = D / 16, DN = D / 8;
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sK = sQ + BM * D * 2;
  const uint32_t sV = sK + 2 * BN * D * 2;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gq = lane >> 2, t = lane & 3;
  const int h = blockIdx.y, b = blockIdx.z;
  const int m0 = blockIdx.x * BM;
  const int64_t rs = (int64_t)a.N_h * D, rs_kv = (int64_t)a.N_kv * D;
  const int h_kv = h / (a.N_h / a.N_kv);
  const __nv_bfloat16* qb = (const __nv_bfloat16*)a.q + (int64_t)b * a.n * rs + (int64_t)h * D;
  const __nv_bfloat16* kb = (const __nv_bfloat16*)a.k + (int64_t)b * a.n * rs_kv + (int64_t)h_kv * D;
  const __nv_bfloat16* vb = (const __nv_bfloat16*)a.v + (int64_t)b * a.n * rs_kv + (int64_t)h_kv * D;
  // key tiles up to what some row of this block sees; each thread's two rows (gq and gq + 8 of the warp's 16) see
  // the first lim_r[0], lim_r[1] keys
  const int block_lim = a.max_limit(m0, min(m0 + BM, a.n) > m0 ? min(m0 + BM, a.n) : m0 + 1);
  const int n_tiles = (block_lim + BN - 1) / BN;
  const int lim_r[2] = {a.row_limit(m0 + warp * 16 + gq), a.row_limit(m0 + warp * 16 + gq + 8)};
  const int lim_min = min(a.lim[0], min(a.lim[1], a.lim[2]));
  const float sl2 = a.scale * kLog2e;

  load_tile<D>(sQ, qb, rs, m0, a.n, tid);
  load_tile<D>(sK, kb, rs_kv, 0, a.n, tid);
  load_tile<D>(sV, vb, rs_kv, 0, a.n, tid);
  cp_async_commit();
  cp_async_wait_all();
  __syncthreads();

  uint32_t qf[KS][4];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks)
    ldsm_x4(sQ + swz<CPR>(warp * 16 + (lane & 15), ks * 2 + (lane >> 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);

  float o[DN][4];
#pragma unroll
  for (int i = 0; i < DN; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

  for (int j = 0; j < n_tiles; ++j) {
    const int buf = j & 1;
    if (j + 1 < n_tiles) {
      load_tile<D>(sK + (buf ^ 1) * BN * D * 2, kb, rs_kv, (j + 1) * BN, a.n, tid);
      load_tile<D>(sV + (buf ^ 1) * BN * D * 2, vb, rs_kv, (j + 1) * BN, a.n, tid);
      cp_async_commit();
    }
    const uint32_t kt = sK + buf * BN * D * 2, vt = sV + buf * BN * D * 2;

    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(kt + swz<CPR>(np * 16 + (lane & 7) + ((lane >> 4) << 3), ks * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
        mma16816(s[2 * np], qf[ks], b0, b1);
        mma16816(s[2 * np + 1], qf[ks], b2, b3);
      }
    }
    // scale into the log2 domain; keys beyond the sequence get -inf
    const int c_base = j * BN + 2 * t;
    const bool tail = (j + 1) * BN > lim_min;     // some row of some block may not see all keys of this tile
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int c = c_base + i * 8 + (e & 1);
        s[i][e] = (tail && c >= lim_r[e >> 1]) ? -INFINITY : s[i][e] * sl2;
      }
    }
    // online softmax: rows gq (elements 0,1) and gq+8 (elements 2,3)
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fmaxf(s[i][2 * r], s[i][2 * r + 1]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run[r], mx);
      const float corr = exp2f(m_run[r] - m_new);
      float ps = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        s[i][2 * r] = exp2f(s[i][2 * r] - m_new);
        s[i][2 * r + 1] = exp2f(s[i][2 * r + 1] - m_new);
        ps += s[i][2 * r] + s[i][2 * r + 1];
      }
      l_run[r] = l_run[r] * corr + ps;
      m_run[r] = m_new;
#pragma unroll
      for (int i = 0; i < DN; ++i) { o[i][2 * r] *= corr; o[i][2 * r + 1] *= corr; }
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t pa[4];
      pa[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
      pa[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
      pa[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      pa[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
      for (int dp = 0; dp < DN / 2; ++dp) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(vt + swz<CPR>(kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), dp * 2 + (lane >> 4)), b0, b1, b2, b3);
        mma16816(o[2 * dp], pa, b0, b1);
        mma16816(o[2 * dp + 1], pa, b2, b3);
      }
    }
    cp_async_wait_all();
    __syncthreads();
  }

  // finish the row sums across the quad, normalise, stage through shared memory, store 16 bytes per thread
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  const float inv0 = 1.f / l_run[0], inv1 = 1.f / l_run[1];
  unsigned char* stage = smem;  // the Q tile is no longer needed; each warp touches only its own 16 rows
  const int lr0 = warp * 16 + gq, lr1 = lr0 + 8;
#pragma unroll
  for (int i = 0; i < DN; ++i) {
    *reinterpret_cast<uint32_t*>(stage + swz<CPR>(lr0, i) + t * 4) = pack_bf16(o[i][0] * inv0, o[i][1] * inv0);
    *reinterpret_cast<uint32_t*>(stage + swz<CPR>(lr1, i) + t * 4) = pack_bf16(o[i][2] * inv1, o[i][3] * inv1);
  }
  __syncwarp();
  __nv_bfloat16* ob = (__nv_bfloat16*)a.out + (int64_t)b * a.n * rs + (int64_t)h * D;
#pragma unroll
  for (int i = lane; i < 16 * CPR; i += 32) {
    const int r = warp * 16 + i / CPR, c = i % CPR;
    if (m0 + r < a.n)
      *reinterpret_cast<uint4*>(ob + (int64_t)(m0 + r) * rs + c * 8) = *reinterpret_cast<const uint4*>(stage + swz<CPR>(r, c));
  }
  if (a.lse && t == 0) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int row = m0 + warp * 16 + gq + 8 * r;
      if (row < a.n && row >= a.lse_row0 && row < a.lse_row0 + a.lse_rows)
        a.lse[((int64_t)b * a.N_h + h) * a.lse_rows + (row - a.lse_row0)] =
            (m_run[r] + log2f(l_run[r])) * 0.6931471805599453f;
    }
  }
}

template <int D>
cudaError_t launch_d(const AttnArgs& a, cudaStream_t st) {
  const size_t smem = (size_t)(BM + 4 * BN) * D * 2;
  cudaError_t e = cudaFuncSetAttribute(attn_bf16_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((a.n + BM - 1) / BM, a.N_h, a.B);
  attn_bf16_mma_kernel<D><<<grid, kThreads, smem, st>>>(a);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_bf16_mma(const AttnArgs& a, cudaStream_t st, int* launches) {
  ++*launches;
  switch (a.D) {
    case 32: return launch_d<32>(a, st);
    case 64: return launch_d<64>(a, st);
    case 128: return launch_d<128>(a, st);
    default: return cudaErrorInvalidConfiguration;
  }
}

}  // namespace swam
