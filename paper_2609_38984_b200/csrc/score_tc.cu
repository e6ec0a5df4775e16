// One-pass scorer (Eq. 12 with the normalisers of Sec. 3.1 computed on the spot) on tcgen05 + TMEM, fed by TMA.
//
// Without a dense pass that supplies the action rows' normalisers lambda, the score S(f, j) needs two things from the
// keys: lambda[h, i] = log sum over ALL visible keys of exp(scale q_i . k_c), and the logit of every future key against
// the g queries aligned with its frame.  The first needs every product q_i . k_c anyway, so ONE stream over K computes
// both: the products of a tile of keys against all action queries of a head are one tensor-core instruction chain,
// their running (max, sum) per query is the normaliser's share of this key range, and the g products per future key
// that Eq. 12 uses are stored raw (fp32) beside it.  A second, small kernel then forms
//   S(f, j) = 1/N_h sum_h sum_i w_i exp2(scale log2e x[h, i, j] - lambda2[h, i])
// from 4 g bytes per (head, key) instead of a second read of the 2 D bytes of the key row.
//
// lse_tc_kernel: CTA = (range of key tiles, head, sample x chunk of <= 128 action queries), two CTAs per SM.
//   warp 8      TMA producer: the query tile once, then key tiles of 16 KB into a ring of four stages (marked as the
//               first lines to leave L2, so that the side output is still there when the second kernel reads it)
//   warp 9      one elected thread issues S = Q K_j^T (M = 128, N = keys per tile) into one of two TMEM buffers
//   warps 0-7   statistics, two groups of four that take alternate tiles (a tile's pass is longer than the tile's
//               share of the stream): thread = TMEM lane = row of S; running maximum and sum in the log2 domain; the
//               products of the keys of the row's own frame go to the row's line of the [head][query][future key] block
// The action queries of a head are few (H = 32 in the paper's set-ups), so the 128 rows of the query tile hold the
// H queries 128 / Hpad times over (Hpad = 32, 64 or 128) and the copies split a tile's key columns among them: every
// warp then has a full set of 32 useful rows and all four exp2 units work.  The last CTA to finish a (sample, head,
// chunk) merges the ranges' partial (max, sum) pairs into lambda (no CTA waits for another one: the order of arrival
// is taken from an atomic ticket).  Every wait on an mbarrier is bounded.
#include "tc_ptx.cuh"

namespace swam {
namespace {

constexpr int kLtThreads = 320;   // warps 0-7 statistics (two groups of four), warp 8 TMA producer, warp 9 MMA issuer
constexpr int kLtStages = 4;
constexpr int kLtStageBytes = 16384;

struct LtParams {
  float2* partial;          // [B, n_splits, N_h, H] (max, sum) in the log2 domain
  float* lam2;              // [B, N_h, H] normalisers in the log2 domain
  float* lse;               // [B, N_h, H] the same in natural-log units
  float* logits;            // [B, N_h, g, F * N_s] raw products q_i . k_j of each future key with its frame's queries
  unsigned int* counters;   // [B * N_h * q_chunks] arrival tickets, zero before and after every launch
  int* status;
  int H, N_h, L, Lk, n_splits, tiles_per_split, kv_group, q_chunks;
  int n_obs, F, N_s, g;
  float scale_log2;
};

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// A key tile is read once: its lines are marked as the first to leave L2, so that the side output, which the second
// kernel reads back, stays there instead
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                                 int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}

// REP: copies of the query chunk in the 128-row tile (1, 2 or 4); a chunk has 128 / REP queries
template <int D, int REP>
__global__ void __launch_bounds__(kLtThreads, 2)
lse_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const LtParams p) {
  constexpr int DB = D / 64;                       // 64-column (128-byte) blocks per row
  constexpr int BN = kLtStageBytes / (D * 2);      // keys per tile: 64 at head dim 128, 128 at head dim 64
  constexpr int HP = kTile / REP;                  // queries per chunk
  constexpr int CW = BN / REP;                     // key columns per thread and tile
  constexpr int CH = CW < 32 ? CW : 32;            // of which this many are in registers at a time
  constexpr int ST = kLtStages;
  constexpr int kQBytes = kTile * D * 2;
  constexpr int kQSub = kTile * 128;               // bytes of one [128 rows x 64 cols] block of the query tile
  constexpr int kKSub = BN * 128;                  // the same of a key tile
  constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
  static_assert(CW % 16 == 0, "a thread reads its columns 16 at a time");

  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_addr(smem_raw) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - smem_addr(smem_raw));
  const uint32_t sQ = base;
  const uint32_t sK = sQ + kQBytes;
  const uint32_t bars = sK + ST * kLtStageBytes;
  unsigned char* tail = base_ptr + kQBytes + ST * kLtStageBytes;
  const uint32_t bar_q = bars;
  auto bar_k_full = [&](int s) { return bars + 8u * (1 + s); };
  auto bar_k_empty = [&](int s) { return bars + 8u * (1 + ST + s); };
  auto bar_s_full = [&](int b) { return bars + 8u * (1 + 2 * ST + b); };
  auto bar_s_free = [&](int b) { return bars + 8u * (3 + 2 * ST + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 132);
  unsigned int* ticket = reinterpret_cast<unsigned int*>(tail + 136);
  float2* s_red = reinterpret_cast<float2*>(tail + 256);     // [2 groups][128]

  const int tid = threadIdx.x, warp = tid >> 5;
  const int split = blockIdx.x, h = blockIdx.y;
  const int b = blockIdx.z / p.q_chunks, qc = blockIdx.z % p.q_chunks;
  const int n_tiles = (p.Lk + BN - 1) / BN;
  const int j0 = split * p.tiles_per_split;
  const int nt = max(0, min(n_tiles, j0 + p.tiles_per_split) - j0);

  if (tid == 0) {
    mbar_init(bar_q, 1);
    for (int s = 0; s < ST; ++s) {
      mbar_init(bar_k_full(s), 1);
      mbar_init(bar_k_empty(s), 1);
    }
    for (int bf = 0; bf < 2; ++bf) {
      mbar_init(bar_s_full(bf), 1);
      mbar_init(bar_s_free(bf), kTile);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)), "n"(2 * BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    const uint32_t el = elect_one();
    const int hk = h / p.kv_group;
    const uint64_t stream_once = policy_evict_first();
    if (el && nt > 0) {
      mbar_expect_tx(bar_q, kQBytes);
      // the chunk's HP action rows (rows beyond the sequence read as zeros), REP times over
#pragma unroll
      for (int rp = 0; rp < REP; ++rp)
#pragma unroll
        for (int db = 0; db < DB; ++db)
          tma_load_4d(sQ + db * kQSub + rp * HP * 128, &map_q, bar_q, db * 64, p.L - p.H + qc * HP, h, b);
    }
    for (int t = 0; t < nt; ++t) {
      const int st = t % ST;
      if (t >= ST) {
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_k_empty(st), (uint32_t)((t / ST - 1) & 1), abort_flag) ? 1 : 0) != 0;
        if (!ok) break;
      }
      if (el) {
        mbar_expect_tx(bar_k_full(st), kLtStageBytes);
#pragma unroll
        for (int db = 0; db < DB; ++db)
          tma_load_4d_hint(sK + st * kLtStageBytes + db * kKSub, &map_k, bar_k_full(st), db * 64, (j0 + t) * BN, hk, b, stream_once);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ MMA issuer
    const uint32_t el = elect_one();
    auto wait_all = [&](uint32_t bar, uint32_t parity) {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag) ? 1 : 0) != 0;
    };
    bool ok = nt == 0 || wait_all(bar_q, 0);
    const uint32_t q_lo = desc_lo(sQ, 16), k_lo0 = desc_lo(sK, 16);
    for (int t = 0; ok && t < nt; ++t) {
      const int st = t % ST, bf = t & 1;
      ok = wait_all(bar_k_full(st), (uint32_t)((t / ST) & 1));
      if (ok && t >= 2) ok = wait_all(bar_s_free(bf), (uint32_t)((t / 2 - 1) & 1));
      if (!ok) break;
      tc_fence_after();
      const uint32_t d = tmem + (uint32_t)(bf * BN);
      const uint32_t k_lo = k_lo0 + ((uint32_t)(st * kLtStageBytes) >> 4);
      mma_ss<false>(d, q_lo, k_lo, kDescHi, kIdesc, el);
#pragma unroll
      for (int ks = 1; ks < D / 16; ++ks) {
        const uint32_t a_off = (uint32_t)((ks >> 2) * (kQSub >> 4) + (ks & 3) * 2);
        const uint32_t b_off = (uint32_t)((ks >> 2) * (kKSub >> 4) + (ks & 3) * 2);
        mma_ss<true>(d, q_lo + a_off, k_lo + b_off, kDescHi, kIdesc, el);
      }
      tc_commit(bar_k_empty(st), el);   // the stage may be refilled once these products have read it
      tc_commit(bar_s_full(bf), el);
    }
  } else {
    // ------------------------------------------------------------------ statistics and side output (2 x 128 threads)
    // group cg takes the tiles t = cg, cg + 2, ... from TMEM buffer cg; thread = TMEM lane ctid
    const int cg = warp >> 2, ctid = tid & (kTile - 1);
    const int row = ctid % HP, share = ctid / HP;
    const int i = qc * HP + row;
    const bool valid = i < p.H;
    // Side output: the keys of this query's frame take their raw product.  A head's block is laid out [query of the
    // group][future key], so a thread's consecutive columns are consecutive floats: a piece that lies inside the
    // frame leaves with 16-byte stores, one that straddles a frame boundary float by float.
    int x_lo = 0, x_hi = 0;
    float* xrow = nullptr;       // this query's row of the head's block, indexed by key
    if (valid) {
      const int fi = i / p.g;
      x_lo = p.n_obs + fi * p.N_s;
      x_hi = x_lo + p.N_s;
      xrow = p.logits + (((int64_t)b * p.N_h + h) * p.g + (i - fi * p.g)) * ((int64_t)p.F * p.N_s) - p.n_obs;
    }
    const bool vec_ok = ((p.n_obs | (p.F * p.N_s)) & 3) == 0;    // 16-byte alignment of every piece's first float
    const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(cg * BN + share * CW);
    float m_run = -INFINITY, l_run = 0.f;
    for (int t = cg; t < nt; t += 2) {
      if (!mbar_wait(bar_s_full(cg), (uint32_t)((t / 2) & 1), abort_flag)) break;
      tc_fence_after();
      // the thread's CW columns in pieces of CH, each folded into the running statistics on its own (a piece's
      // registers are free again before the next one is read)
#pragma unroll
      for (int c0 = 0; c0 < CW; c0 += CH) {
        float x[CH];
#pragma unroll
        for (int cc = 0; cc < CH; cc += 16)
          tmem_ld16(t_lane + (uint32_t)(c0 + cc), *reinterpret_cast<float(*)[16]>(&x[cc]));
        tmem_ld_wait();
        if (c0 + CH == CW) {          // the buffer's last piece is in registers: the next product may overwrite it
          tc_fence_before();
          mbar_arrive(bar_s_free(cg));
        }
        const int key0 = (j0 + t) * BN + share * CW + c0;     // key of column 0 of this piece
        if (key0 + CH > p.Lk) {                                // the sequence ends here: keys beyond it count as -inf
#pragma unroll
          for (int c = 0; c < CH; ++c)
            if (key0 + c >= p.Lk) x[c] = -INFINITY;
        }
        if (key0 < x_hi && key0 + CH > x_lo) {
          float* dst = xrow + key0;
          if (vec_ok && key0 >= x_lo && key0 + CH <= x_hi) {
#pragma unroll
            for (int c = 0; c < CH; c += 4) *reinterpret_cast<float4*>(dst + c) = make_float4(x[c], x[c + 1], x[c + 2], x[c + 3]);
          } else {
#pragma unroll
            for (int c = 0; c < CH; ++c)
              if (key0 + c >= x_lo && key0 + c < x_hi) dst[c] = x[c];
          }
        }
        float mx0 = x[0], mx1 = x[1], mx2 = x[2], mx3 = x[3];     // four chains: the warp has few neighbours to hide latency
#pragma unroll
        for (int c = 4; c < CH; c += 4) {
          mx0 = fmaxf(mx0, x[c]);
          mx1 = fmaxf(mx1, x[c + 1]);
          mx2 = fmaxf(mx2, x[c + 2]);
          mx3 = fmaxf(mx3, x[c + 3]);
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        const float m_new = fmaxf(m_run, mx * p.scale_log2);
        if (m_new != -INFINITY) {
          float ps0 = 0.f, ps1 = 0.f, ps2 = 0.f, ps3 = 0.f;
#pragma unroll
          for (int c = 0; c < CH; c += 4) {
            ps0 += ex2(fmaf(x[c], p.scale_log2, -m_new));
            ps1 += ex2(fmaf(x[c + 1], p.scale_log2, -m_new));
            ps2 += ex2(fmaf(x[c + 2], p.scale_log2, -m_new));
            ps3 += ex2(fmaf(x[c + 3], p.scale_log2, -m_new));
          }
          l_run = l_run * ex2(m_run - m_new) + ((ps0 + ps1) + (ps2 + ps3));
          m_run = m_new;
        }
      }
    }
    s_red[tid] = make_float2(m_run, l_run);
  }

  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag) atomicOr(p.status, ST_TIMEOUT);
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(2 * BN) : "memory");
  }
  // this key range's (max, sum) per query: the REP column shares merged
  const int64_t row_stride = (int64_t)p.N_h * p.H;
  if (tid < HP && qc * HP + tid < p.H) {
    float m = -INFINITY, l = 0.f;
#pragma unroll
    for (int sh = 0; sh < 2 * REP; ++sh) merge_ms(m, l, s_red[sh * HP + tid].x, s_red[sh * HP + tid].y);
    p.partial[((int64_t)b * p.n_splits + split) * row_stride + (int64_t)h * p.H + qc * HP + tid] = make_float2(m, l);
    __threadfence();
  }
  __syncthreads();
  unsigned int* counter = p.counters + ((int64_t)b * p.N_h + h) * p.q_chunks + qc;
  if (tid == 0) *ticket = atomicAdd(counter, 1u);
  __syncthreads();
  if (*ticket != (unsigned int)(p.n_splits - 1)) return;
  // the last CTA of this (sample, head, chunk): every range's partial is visible now
  __threadfence();
  if (tid < HP && qc * HP + tid < p.H) {
    const float2* src = p.partial + (int64_t)b * p.n_splits * row_stride + (int64_t)h * p.H + qc * HP + tid;
    float m = -INFINITY, l = 0.f;
    int c = 0;
    for (; c + 4 <= p.n_splits; c += 4) {
      const float2 a0 = __ldcg(src + (int64_t)c * row_stride), a1 = __ldcg(src + (int64_t)(c + 1) * row_stride);
      const float2 a2 = __ldcg(src + (int64_t)(c + 2) * row_stride), a3 = __ldcg(src + (int64_t)(c + 3) * row_stride);
      merge_ms(m, l, a0.x, a0.y);
      merge_ms(m, l, a1.x, a1.y);
      merge_ms(m, l, a2.x, a2.y);
      merge_ms(m, l, a3.x, a3.y);
    }
    for (; c < p.n_splits; ++c) {
      const float2 a = __ldcg(src + (int64_t)c * row_stride);
      merge_ms(m, l, a.x, a.y);
    }
    const float l2 = m + log2f(l);
    const int64_t o = ((int64_t)b * p.N_h + h) * p.H + qc * HP + tid;
    p.lam2[o] = l2;
    p.lse[o] = l2 * 0.6931471805599453f;
  }
  if (tid == 0) *counter = 0u;
}

// Second half: S(f, j) from the stored products and the finished normalisers.  A CTA owns 32 keys of one frame;
// thread (key, one of 8 head slots) sums the heads of its slot (a warp's loads are 128 consecutive bytes per query)
// and the eight shares meet in shared memory.
constexpr int kFinKeys = 32, kFinSlots = 8, kFinThreads = kFinKeys * kFinSlots;

struct FinishParams {
  const float* logits;     // [B, N_h, g, F * N_s]
  const float* lam2;       // [B, N_h, H]
  float* scores;           // [B, F, N_s]
  int F, N_s, H, N_h, g;
  float scale_log2, inv_nh;
  Alpha alpha;
};

// G = g for the group sizes with an unrolled instance (all of a head's loads in flight at once), 0 = any group size
template <int G>
__global__ void __launch_bounds__(kFinThreads) score_finish_kernel(const FinishParams p) {
  extern __shared__ __align__(16) float fin_smem[];
  float* lam2 = fin_smem;                 // [N_h][g]
  float* red = lam2 + p.N_h * p.g;        // [8][32]
  const int tid = threadIdx.x;
  const int f = blockIdx.y, b = blockIdx.z, key0 = blockIdx.x * kFinKeys;
  for (int idx = tid; idx < p.N_h * p.g; idx += kFinThreads) {
    const int h = idx / p.g, ii = idx - h * p.g;
    lam2[idx] = p.lam2[((int64_t)b * p.N_h + h) * p.H + f * p.g + ii];
  }
  const int jj = tid & (kFinKeys - 1), hs = tid / kFinKeys;
  const int key = key0 + jj;
  const bool in = key < p.N_s;
  const int64_t q_stride = (int64_t)p.F * p.N_s, head_stride = q_stride * p.g;
  const float* x = p.logits + (int64_t)b * p.N_h * head_stride + (int64_t)f * p.N_s + (in ? key : 0);
  float sum = 0.f;
  if (G > 0) {
    constexpr int U = (G >= 16) ? 1 : 2, GV = G > 0 ? G : 1;     // heads in flight
    bool first = true;
    for (int h0 = hs; h0 < p.N_h; h0 += U * kFinSlots) {
      float v[U][GV];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int h = h0 + u * kFinSlots;
#pragma unroll
        for (int ii = 0; ii < GV; ++ii) v[u][ii] = (in && h < p.N_h) ? __ldcs(x + h * head_stride + ii * q_stride) : 0.f;
      }
      if (first) __syncthreads();      // the normalisers are staged (the first loads are already in flight)
      first = false;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int h = h0 + u * kFinSlots;
        if (h < p.N_h) {
          const float* l = lam2 + h * GV;
#pragma unroll
          for (int ii = 0; ii < GV; ++ii) sum += p.alpha.w[ii] * exp2f(fmaf(v[u][ii], p.scale_log2, -l[ii]));
        }
      }
    }
    if (first) __syncthreads();        // slots without a head still take part in the barrier
  } else {
    __syncthreads();
    if (in) {
      for (int h = hs; h < p.N_h; h += kFinSlots) {
        const float* xh = x + h * head_stride;
        const float* l = lam2 + h * p.g;
        for (int ii = 0; ii < p.g; ++ii) sum += p.alpha.w[ii] * exp2f(fmaf(__ldcs(xh + ii * q_stride), p.scale_log2, -l[ii]));
      }
    }
  }
  red[hs * kFinKeys + jj] = in ? sum : 0.f;
  __syncthreads();
  if (tid < kFinKeys && key0 + tid < p.N_s) {
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < kFinSlots; q += 2) s += red[q * kFinKeys + tid] + red[(q + 1) * kFinKeys + tid];
    p.scores[((int64_t)b * p.F + f) * p.N_s + key0 + tid] = s * p.inv_nh;
  }
}

template <int D, int REP>
cudaError_t launch_lse_tc(const Dims& d, const CUtensorMap& mq, const CUtensorMap& mk, const LtParams& p, dim3 grid,
                          cudaStream_t st) {
  constexpr size_t smem = (size_t)kTile * D * 2 + kLtStages * kLtStageBytes + 256 + 2 * kTile * sizeof(float2) + 1024;
  cudaError_t e = cudaFuncSetAttribute(lse_tc_kernel<D, REP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  lse_tc_kernel<D, REP><<<grid, kLtThreads, smem, st>>>(mq, mk, p);
  return cudaGetLastError();
}

}  // namespace

bool score_one_pass_supported(const Dims& d) {
  // bf16 on the tensor-core path; the second kernel keeps N_h * g normalisers in (default-sized) shared memory
  return d.dtype != 0 && (d.D == 64 || d.D == 128) &&
         ((size_t)d.N_h * d.g + kFinSlots * kFinKeys) * sizeof(float) <= 48 * 1024;
}

size_t score_logits_bytes(const Dims& d) {
  return score_one_pass_supported(d) ? (size_t)d.B * d.N_h * d.F * d.N_s * d.g * sizeof(float) : 0;
}
size_t score_counter_bytes(const Dims& d) {
  return score_one_pass_supported(d) ? (size_t)d.B * d.N_h * ((d.H + 31) / 32) * sizeof(unsigned int) : 0;
}

cudaError_t launch_score_one_pass(const Dims& d, const Alpha& alpha, const void* q, const void* k, float* lse, float* lam2,
                                  void* partial, unsigned int* counters, float* logits, int* status, float* scores,
                                  cudaStream_t st, int* launches, int n_keys) {
  if (!score_one_pass_supported(d)) return cudaErrorInvalidConfiguration;
  const int hp = d.H <= 32 ? 32 : (d.H <= 64 ? 64 : 128);
  const int q_chunks = (d.H + hp - 1) / hp;
  const int bn = kLtStageBytes / (d.D * 2);
  const int n_tiles = (n_keys + bn - 1) / bn;
  // Key ranges per (sample, head, chunk): the launch runs in waves of two CTAs per SM; take the count that minimises
  // waves x (tiles per CTA + a CTA's fixed cost of about two tiles), within what the partials' scratch holds.
  const int slots = 2 * sm_count();
  const long long heads = (long long)d.B * d.N_h * q_chunks;
  const int max_splits = (d.L + 127) / 128;
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= max_splits && s <= n_tiles; ++s) {
    const int per = (n_tiles + s - 1) / s;
    if ((n_tiles + per - 1) / per != s) continue;   // this count leaves a range empty
    const double waves = (double)((heads * s + slots - 1) / slots);
    const double cost = waves * (per + 2.0);
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best = s;
    }
  }
  const int per = (n_tiles + best - 1) / best;
  CUtensorMap mq, mk;
  if (!make_map(&mq, q, d.B, d.L, d.N_h, d.D, hp) || !make_map(&mk, k, d.B, d.L, d.N_kv, d.D, bn))
    return cudaErrorInvalidValue;
  LtParams p{(float2*)partial, lam2, lse, logits, counters, status, d.H, d.N_h, d.L, n_keys, best, per,
             d.N_h / d.N_kv, q_chunks, d.n_obs, d.F, d.N_s, d.g, d.scale * kLog2e};
  dim3 grid(best, d.N_h, d.B * q_chunks);
  *launches += 2;
  cudaError_t e;
  if (d.D == 128)
    e = hp == 32 ? launch_lse_tc<128, 4>(d, mq, mk, p, grid, st)
                 : (hp == 64 ? launch_lse_tc<128, 2>(d, mq, mk, p, grid, st) : launch_lse_tc<128, 1>(d, mq, mk, p, grid, st));
  else
    e = hp == 32 ? launch_lse_tc<64, 4>(d, mq, mk, p, grid, st)
                 : (hp == 64 ? launch_lse_tc<64, 2>(d, mq, mk, p, grid, st) : launch_lse_tc<64, 1>(d, mq, mk, p, grid, st));
  if (e != cudaSuccess) return e;
  FinishParams fp{logits, lam2, scores, d.F, d.N_s, d.H, d.N_h, d.g, d.scale * kLog2e, 1.0f / (float)d.N_h, alpha};
  dim3 g2((d.N_s + kFinKeys - 1) / kFinKeys, d.F, d.B);
  const size_t smem = ((size_t)d.N_h * d.g + kFinSlots * kFinKeys) * sizeof(float);
  switch (d.g) {
    case 4: score_finish_kernel<4><<<g2, kFinThreads, smem, st>>>(fp); break;
    case 8: score_finish_kernel<8><<<g2, kFinThreads, smem, st>>>(fp); break;
    case 16: score_finish_kernel<16><<<g2, kFinThreads, smem, st>>>(fp); break;
    default: score_finish_kernel<0><<<g2, kFinThreads, smem, st>>>(fp); break;
  }
  return cudaGetLastError();
}

}  // namespace swam
