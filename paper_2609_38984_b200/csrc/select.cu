// Token selection (Eq. 4-6, 10-11) and packing metadata, one CTA per sample.
//
// Every TopK is a radix select in shared memory: keys are mapped to unsigned integers whose order is the
// order of the floating-point values, 8-bit digits are histogrammed from the top, and the digit holding the
// k-th largest key is located with a warp-shuffle suffix scan.  What remains after the last digit is the
// exact value of the k-th key; keys equal to it are admitted in ascending index order (ballot/popc ranks),
// which is the "ties go to the lower index" rule.  The per-frame core selections run concurrently in thread
// groups synchronised by named barriers; pool and anchor selections use the whole CTA.
//
// The anchor statistic is evaluated in fp64 with individually rounded operations (no fused multiply-add) in
// a fixed order: sum over frames ascending, mean, sum of squared deviations ascending, population standard
// deviation, CV = sd / mu (0 when mu = 0), key = mu / (1 + beta * CV).
#include "swam_internal.cuh"

namespace swam {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kMaxGroups = 8;

__device__ __forceinline__ uint32_t key32(float x) {
  x = x + 0.0f;  // -0 -> +0 so that equal values have equal keys
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ uint64_t key64(double x) {
  x = __dadd_rn(x, 0.0);
  const uint64_t u = (uint64_t)__double_as_longlong(x);
  return (u & 0x8000000000000000ull) ? ~u : (u | 0x8000000000000000ull);
}

// barrier among the `count` threads of one group (count is a multiple of 32); id 0 is the CTA barrier
__device__ __forceinline__ void group_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

struct GroupCtx {
  int bar_id;      // named barrier
  int n_threads;   // threads in the group
  int tid;         // thread index within the group
  int* hist;       // [256] shared
  int* scal;       // [4] shared scalars: digit, remaining
  int* warp_tot;   // [32] shared
};

// Radix select among candidates. key(i) -> KeyT for i in [0,n); cand(i) -> bool.
// Writes flag_out[i] = 1 for the k selected candidates (0 otherwise, for all i in [0,n)).
template <typename KeyT, typename KeyFn, typename CandFn>
__device__ void radix_select(const GroupCtx& g, int n, int k, KeyFn key, CandFn cand, uint8_t* flag_out) {
  constexpr int kBits = sizeof(KeyT) * 8;
  const int lane = g.tid & 31, warp = g.tid >> 5, n_warps = g.n_threads >> 5;
  KeyT prefix = 0, mask = 0;
  int remaining = k;
  if (k > 0) {
    for (int i = g.tid; i < 256; i += g.n_threads) g.hist[i] = 0;
    group_sync(g.bar_id, g.n_threads);
    for (int shift = kBits - 8; shift >= 0; shift -= 8) {
      for (int i0 = 0; i0 < n; i0 += g.n_threads) {
        const int i = i0 + g.tid;
        bool act = false;
        int digit = 0;
        if (i < n && cand(i)) {
          const KeyT kv = key(i);
          act = (kv & mask) == prefix;
          digit = (int)((kv >> shift) & 0xFF);
        }
        // keys often share their leading digits: when the whole warp agrees on the digit, one atomic serves it
        const unsigned live = __ballot_sync(0xffffffffu, act);
        if (live) {
          const int lead = __ffs(live) - 1;
          const int d0 = __shfl_sync(0xffffffffu, digit, lead);
          const bool same = __all_sync(0xffffffffu, !act || digit == d0);
          if (same) {
            if (lane == lead) atomicAdd(&g.hist[d0], __popc(live));
          } else if (act) {
            atomicAdd(&g.hist[digit], 1);
          }
        }
      }
      group_sync(g.bar_id, g.n_threads);
      if (warp == 0) {
        // lane owns bins [8*lane, 8*lane+8); suffix = number of keys in bins above the lane's
        int local[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { local[j] = g.hist[lane * 8 + j]; sum += local[j]; g.hist[lane * 8 + j] = 0; }
        int incl = sum;  // inclusive suffix sum over lanes >= lane
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += v;
        }
        int above = incl - sum;  // keys in bins of higher lanes
        const int total = __shfl_sync(0xffffffffu, incl, 0);
        const int want = remaining < total ? remaining : total;  // fewer candidates than k: take them all
        if (want <= 0) {
          if (lane == 0) { g.scal[0] = 0xFF; g.scal[1] = 0; }
        } else if (above < want && want <= above + sum) {
          // the want-th largest key lies in this lane's bins
          int digit = lane * 8, rem = want;
          bool found = false;
#pragma unroll
          for (int j = 7; j >= 0; --j) {
            if (!found) {
              if (want <= above + local[j]) { digit = lane * 8 + j; rem = want - above; found = true; }
              else above += local[j];
            }
          }
          g.scal[0] = digit;
          g.scal[1] = rem;
        }
      }
      group_sync(g.bar_id, g.n_threads);
      prefix |= (KeyT)g.scal[0] << shift;
      mask |= (KeyT)0xFF << shift;
      remaining = g.scal[1];
      // (warp 0 cleared the bins it read, and the barrier above orders that before the next pass's atomics; scal is
      // rewritten only after the next pass's histogram barrier)
    }
  }
  // prefix is now the k-th largest key; admit keys above it, and the first `remaining` keys equal to it
  int base = 0;
  for (int start = 0; start < n; start += g.n_threads) {
    const int i = start + g.tid;
    bool c = false, eq = false, gt = false;
    if (i < n && k > 0) {
      c = cand(i);
      if (c) { const KeyT kv = key(i); gt = kv > prefix; eq = kv == prefix; }
    }
    const unsigned bal = __ballot_sync(0xffffffffu, eq);
    const int before = __popc(bal & ((1u << lane) - 1u));
    group_sync(g.bar_id, g.n_threads);  // warp_tot free to overwrite
    if (lane == 0) g.warp_tot[warp] = __popc(bal);
    group_sync(g.bar_id, g.n_threads);
    int wbase = 0, total = 0;
    for (int w = 0; w < n_warps; ++w) {
      const int tw = g.warp_tot[w];
      if (w < warp) wbase += tw;
      total += tw;
    }
    if (i < n) flag_out[i] = (gt || (eq && (base + wbase + before) < remaining)) ? 1 : 0;
    base += total;
  }
  group_sync(g.bar_id, g.n_threads);
}

// Ascending compaction of flagged positions: calls emit(i, rank) for each flagged i; returns the count.
template <typename FlagFn, typename EmitFn>
__device__ int ranked_emit(const GroupCtx& g, int n, FlagFn flag, EmitFn emit) {
  const int lane = g.tid & 31, warp = g.tid >> 5, n_warps = g.n_threads >> 5;
  int base = 0;
  for (int start = 0; start < n; start += g.n_threads) {
    const int i = start + g.tid;
    const bool fl = (i < n) && flag(i);
    const unsigned bal = __ballot_sync(0xffffffffu, fl);
    const int before = __popc(bal & ((1u << lane) - 1u));
    group_sync(g.bar_id, g.n_threads);
    if (lane == 0) g.warp_tot[warp] = __popc(bal);
    group_sync(g.bar_id, g.n_threads);
    int wbase = 0, total = 0;
    for (int w = 0; w < n_warps; ++w) {
      const int tw = g.warp_tot[w];
      if (w < warp) wbase += tw;
      total += tw;
    }
    if (i < n) emit(i, fl ? base + wbase + before : -1);
    base += total;
  }
  return base;
}

struct SelectParams {
  const float* scores;
  int32_t* sel_idx;
  int32_t* pack_map;
  int32_t* inv_map;
  int* status;
  int n_obs, F, N_s, H, Kc, Ks, L, Lp, n_groups;
  double beta;
};

__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(const SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int F = p.F, N = p.N_s, K = p.Kc + p.Ks;
  // layout: keyA u64[N] | S f32[F*N] | hist int[(groups+1)*256] | warp_tot int[(groups+1)*32] | scal int[(groups+1)*4]
  //         | pool u8[N] | anchor u8[N] | anycore u8[N] | core u8[F*N]
  uint64_t* keyA = reinterpret_cast<uint64_t*>(smem_raw);
  float* S = reinterpret_cast<float*>(keyA + N);
  int* hist = reinterpret_cast<int*>(S + (size_t)F * N);
  int* warp_tot = hist + (kMaxGroups + 1) * 256;
  int* scal = warp_tot + (kMaxGroups + 1) * 32;
  uint8_t* pool = reinterpret_cast<uint8_t*>(scal + (kMaxGroups + 1) * 4);
  uint8_t* anchor = pool + N;
  uint8_t* anycore = anchor + N;
  uint8_t* core = anycore + N;

  const int tid = threadIdx.x, b = blockIdx.x;
  const float* sg = p.scores + (int64_t)b * F * N;
  for (int i = tid; i < F * N; i += kSelThreads) S[i] = sg[i];
  __syncthreads();

  GroupCtx all{0, kSelThreads, tid, hist, scal, warp_tot};

  // candidate pool: top (N_s - K_s) of max_f S(f, j)                                   (Eq. 4)
  uint32_t* keyM = reinterpret_cast<uint32_t*>(keyA);  // the anchor keys are built later in the same storage
  for (int j = tid; j < N; j += kSelThreads) {
    float m = S[j];
    for (int f = 1; f < F; ++f) m = fmaxf(m, S[f * N + j]);
    keyM[j] = key32(m);
  }
  __syncthreads();
  radix_select<uint32_t>(all, N, N - p.Ks, [&](int j) { return keyM[j]; }, [](int) { return true; }, pool);

  // frame-specific core tokens: top K_c of S(f, .) inside the pool                      (Eq. 5)
  {
    const int gt = kSelThreads / p.n_groups;
    const int grp = tid / gt;
    GroupCtx gc{1 + grp, gt, tid - grp * gt, hist + (1 + grp) * 256, scal + (1 + grp) * 4, warp_tot + (1 + grp) * 32};
    for (int f = grp; f < F; f += p.n_groups) {
      const float* Sf = S + (size_t)f * N;
      radix_select<uint32_t>(gc, N, p.Kc, [&](int j) { return key32(Sf[j]); }, [&](int j) { return pool[j] != 0; },
                             core + (size_t)f * N);
    }
  }
  __syncthreads();

  // positions that are core in no frame (Eq. 10) and the anchor key mu / (1 + beta CV)   (Eq. 11, Eq. 6)
  for (int j = tid; j < N; j += kSelThreads) {
    uint8_t any = 0;
    double sum = 0.0;
    for (int f = 0; f < F; ++f) {
      any |= core[(size_t)f * N + j];
      sum = __dadd_rn(sum, (double)S[f * N + j]);
    }
    const double mu = __ddiv_rn(sum, (double)F);
    double ss = 0.0;
    for (int f = 0; f < F; ++f) {
      const double dv = __dadd_rn((double)S[f * N + j], -mu);
      ss = __dadd_rn(ss, __dmul_rn(dv, dv));
    }
    const double sd = __dsqrt_rn(__ddiv_rn(ss, (double)F));
    const double cv = (mu == 0.0) ? 0.0 : __ddiv_rn(sd, mu);
    const double a = __ddiv_rn(mu, __dadd_rn(1.0, __dmul_rn(p.beta, cv)));
    anycore[j] = any;
    keyA[j] = key64(a);
  }
  __syncthreads();
  radix_select<uint64_t>(all, N, p.Ks, [&](int j) { return keyA[j]; }, [&](int j) { return anycore[j] == 0; }, anchor);

  // retained positions ascending, and the maps
  int32_t* sel = p.sel_idx ? p.sel_idx + (int64_t)b * F * K : nullptr;
  int32_t* pm = p.pack_map ? p.pack_map + (int64_t)b * p.Lp : nullptr;
  int32_t* im = p.inv_map ? p.inv_map + (int64_t)b * p.L : nullptr;
  bool bad = false;
  for (int f = 0; f < F; ++f) {
    const uint8_t* cf = core + (size_t)f * N;
    const int cnt = ranked_emit(
        all, N, [&](int j) { return (cf[j] | anchor[j]) != 0; },
        [&](int j, int r) {
          if (r >= 0 && r < K) {
            if (sel) sel[f * K + r] = j;
            if (pm) pm[p.n_obs + f * K + r] = p.n_obs + f * N + j;
          }
          if (im) im[p.n_obs + f * N + j] = (r >= 0 && r < K) ? p.n_obs + f * K + r : -1;
        });
    bad |= (cnt != K);
  }
  for (int t = tid; t < p.n_obs; t += kSelThreads) {
    if (pm) pm[t] = t;
    if (im) im[t] = t;
  }
  for (int t = tid; t < p.H; t += kSelThreads) {
    if (pm) pm[p.n_obs + F * K + t] = p.n_obs + F * N + t;
    if (im) im[p.n_obs + F * N + t] = p.n_obs + F * K + t;
  }
  if (bad && tid == 0) atomicOr(p.status, ST_BAD_COUNT);
}

}  // namespace

size_t select_smem_bytes(const Dims& d) {
  const size_t N = d.N_s, F = d.F;
  size_t bytes = N * 8 + F * N * 4 + (size_t)(kMaxGroups + 1) * (256 + 32 + 4) * 4 + 3 * N + F * N;
  return (bytes + 15) & ~(size_t)15;
}

cudaError_t select_prepare(const Dims& d) {
  const size_t smem = select_smem_bytes(d);
  if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
  return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

cudaError_t launch_select(const Dims& d, const float* scores, int32_t* sel_idx, int32_t* pack_map,
                          int32_t* inv_map, int* status, cudaStream_t st, int* launches) {
  int groups = 1;
  while (groups * 2 <= d.F && groups * 2 <= kMaxGroups) groups *= 2;
  SelectParams p{scores, sel_idx, pack_map, inv_map, status, d.n_obs, d.F, d.N_s, d.H,
                 d.Kc, d.Ks, d.L, d.Lp, groups, (double)d.beta};
  ++*launches;
  select_kernel<<<d.B, kSelThreads, select_smem_bytes(d), st>>>(p);
  return cudaGetLastError();
}

}  // namespace swam
