// Token selection (Eq. 4-6, 10-11) and packing metadata: one thread-block cluster per sample.
//
// Every TopK is a radix select in shared memory: keys are mapped to unsigned integers whose order is the
// order of the floating-point values, 8-bit digits are histogrammed from the top, and the digit holding the
// k-th largest key is located with a warp-shuffle suffix scan.  The passes stop as soon as the bin that holds
// the k-th key is taken whole; otherwise what remains after the last digit is the exact value of the k-th key and
// keys equal to it are admitted in ascending index order (ballot/popc ranks), which is the "ties go to the lower
// index" rule.
//
// The CTAs of a cluster (up to 8) each hold the sample's scores in shared memory.  The candidate pool and the anchor
// selection are small and are computed by every CTA; the per-frame core selections and the map construction are
// split by frame; core flags and anchor keys are exchanged through distributed shared memory.
//
// The anchor statistic is evaluated in fp64 with individually rounded operations (no fused multiply-add) in
// a fixed order: sum over frames ascending, mean, sum of squared deviations ascending, population standard
// deviation, CV = sd / mu (0 when mu = 0), key = mu / (1 + beta * CV).
#include <cooperative_groups.h>

#include "swam_internal.cuh"

namespace cg = cooperative_groups;

namespace swam {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kMaxCluster = 8;

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

struct Scratch {
  int* hist;      // [256] shared
  int* scal;      // [4] shared: digit, remaining, whole-bin flag
  int* warp_tot;  // [32] shared
};

// exclusive prefix of this warp and the total over all warps of the per-warp counts in s.warp_tot
__device__ __forceinline__ void warp_bases(const Scratch& s, int warp, int lane, int& wbase, int& total) {
  const int v = s.warp_tot[lane];
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  wbase = __shfl_sync(0xffffffffu, incl - v, warp);
  total = __shfl_sync(0xffffffffu, incl, 31);
}

// Radix select among candidates (whole CTA). key(i) -> KeyT for i in [0,n); cand(i) -> bool.
// Writes flag_out[i] = 1 for the k selected candidates (0 otherwise, for all i in [0,n)).
template <typename KeyT, typename KeyFn, typename CandFn>
__device__ void radix_select(const Scratch& s, int n, int k, KeyFn key, CandFn cand, uint8_t* flag_out) {
  constexpr int kBits = sizeof(KeyT) * 8;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  KeyT prefix = 0, mask = 0;
  int remaining = k;
  bool whole_bin = false;  // every key that matches the prefix so far is selected
  if (k > 0) {
    for (int i = tid; i < 256; i += kSelThreads) s.hist[i] = 0;
    __syncthreads();
    for (int shift = kBits - 8; shift >= 0; shift -= 8) {
      for (int i0 = 0; i0 < n; i0 += kSelThreads) {
        const int i = i0 + tid;
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
            if (lane == lead) atomicAdd(&s.hist[d0], __popc(live));
          } else if (act) {
            atomicAdd(&s.hist[digit], 1);
          }
        }
      }
      __syncthreads();
      if (warp == 0) {
        // lane owns bins [8*lane, 8*lane+8); suffix = number of keys in bins above the lane's
        int local[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { local[j] = s.hist[lane * 8 + j]; sum += local[j]; s.hist[lane * 8 + j] = 0; }
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
          if (lane == 0) { s.scal[0] = 0xFF; s.scal[1] = 0; s.scal[2] = 0; }
        } else if (above < want && want <= above + sum) {
          // the want-th largest key lies in this lane's bins
          int digit = lane * 8, rem = want, in_bin = 0;
          bool found = false;
#pragma unroll
          for (int j = 7; j >= 0; --j) {
            if (!found) {
              if (want <= above + local[j]) { digit = lane * 8 + j; rem = want - above; in_bin = local[j]; found = true; }
              else above += local[j];
            }
          }
          s.scal[0] = digit;
          s.scal[1] = rem;
          s.scal[2] = (in_bin == rem) ? 1 : 0;
        }
      }
      __syncthreads();
      prefix |= (KeyT)s.scal[0] << shift;
      mask |= (KeyT)0xFF << shift;
      remaining = s.scal[1];
      whole_bin = s.scal[2] != 0;
      // (warp 0 cleared the bins it read before the barrier above; scal is rewritten only after the next pass's
      // histogram barrier)
      if (whole_bin) break;
    }
  }
  // keys above the prefix are in; of the keys that match it, all (whole bin) or the first `remaining` by index
  int base = 0;
  for (int start = 0; start < n; start += kSelThreads) {
    const int i = start + tid;
    bool eq = false, gt = false;
    if (i < n && k > 0 && cand(i)) {
      const KeyT kv = key(i) & mask;
      gt = kv > prefix;
      eq = kv == prefix;
    }
    if (whole_bin) {
      if (i < n) flag_out[i] = (gt || eq) ? 1 : 0;
      continue;
    }
    const unsigned bal = __ballot_sync(0xffffffffu, eq);
    const int before = __popc(bal & ((1u << lane) - 1u));
    __syncthreads();  // warp_tot free to overwrite
    if (lane == 0) s.warp_tot[warp] = __popc(bal);
    __syncthreads();
    int wbase, total;
    warp_bases(s, warp, lane, wbase, total);
    if (i < n) flag_out[i] = (gt || (eq && (base + wbase + before) < remaining)) ? 1 : 0;
    base += total;
  }
  __syncthreads();
}

// Ascending compaction of flagged positions: calls emit(i, rank) for each i (rank -1 when not flagged); returns the count.
template <typename FlagFn, typename EmitFn>
__device__ int ranked_emit(const Scratch& s, int n, FlagFn flag, EmitFn emit) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int base = 0;
  for (int start = 0; start < n; start += kSelThreads) {
    const int i = start + tid;
    const bool fl = (i < n) && flag(i);
    const unsigned bal = __ballot_sync(0xffffffffu, fl);
    const int before = __popc(bal & ((1u << lane) - 1u));
    __syncthreads();
    if (lane == 0) s.warp_tot[warp] = __popc(bal);
    __syncthreads();
    int wbase, total;
    warp_bases(s, warp, lane, wbase, total);
    if (i < n) emit(i, fl ? base + wbase + before : -1);
    base += total;
  }
  return base;
}

struct SelectParams {
  const float* scores;      // core score map V: pool and cores
  const float* scores_all;  // anchor score map V_all (may equal scores)
  int32_t* sel_idx;
  int32_t* pack_map;
  int32_t* inv_map;
  int* status;
  int n_obs, F, N_s, H, Kc, Ks, L, Lp;
  double beta;
  float* quality;           // [B, 3] (R, E, Q) of Eq. 9 for `scores`, or nullptr
};

// shared-memory layout (bytes), identical in every CTA of the cluster
struct SelLayout {
  size_t keyA, S, Sall, keyM, hist, warp_tot, scal, pool, anchor, anycore, core, total;
};
__host__ __device__ inline SelLayout sel_layout(int F, int N) {
  SelLayout l;
  size_t o = 0;
  l.keyA = o; o += (size_t)N * 8;
  l.S = o; o += (size_t)F * N * 4;
  l.Sall = o; o += (size_t)F * N * 4;
  l.keyM = o; o += (size_t)N * 4;
  l.hist = o; o += 256 * 4;
  l.warp_tot = o; o += 32 * 4;
  l.scal = o; o += 4 * 4;
  l.pool = o; o += (size_t)N;
  l.anchor = o; o += (size_t)N;
  l.anycore = o; o += (size_t)N;
  o = (o + 3) & ~(size_t)3;
  l.core = o; o += ((size_t)N + 3) / 4 * 4 * F;   // each frame's flags start on a 4-byte boundary
  l.total = (o + 15) & ~(size_t)15;
  return l;
}

__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(const SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int F = p.F, N = p.N_s, K = p.Kc + p.Ks;
  const int Npad = (N + 3) / 4 * 4;
  const SelLayout lay = sel_layout(F, N);
  uint64_t* keyA = reinterpret_cast<uint64_t*>(smem_raw + lay.keyA);
  float* S = reinterpret_cast<float*>(smem_raw + lay.S);
  uint32_t* keyM = reinterpret_cast<uint32_t*>(smem_raw + lay.keyM);
  Scratch sc{reinterpret_cast<int*>(smem_raw + lay.hist), reinterpret_cast<int*>(smem_raw + lay.scal),
             reinterpret_cast<int*>(smem_raw + lay.warp_tot)};
  uint8_t* pool = smem_raw + lay.pool;
  uint8_t* anchor = smem_raw + lay.anchor;
  uint8_t* anycore = smem_raw + lay.anycore;
  uint8_t* core = smem_raw + lay.core;  // [F][Npad]

  const int tid = threadIdx.x, b = blockIdx.y;
  const float* sg = p.scores + (int64_t)b * F * N;
  for (int i = tid; i < F * N; i += kSelThreads) S[i] = sg[i];
  const float* Sall = S;  // the anchor statistic reads V_all; with one profiled layer it is the same map
  if (p.scores_all != p.scores) {
    float* sa = reinterpret_cast<float*>(smem_raw + lay.Sall);
    const float* sag = p.scores_all + (int64_t)b * F * N;
    for (int i = tid; i < F * N; i += kSelThreads) sa[i] = sag[i];
    Sall = sa;
  }
  __syncthreads();

  // candidate pool: top (N_s - K_s) of max_f S(f, j)                                   (Eq. 4)
  for (int j = tid; j < N; j += kSelThreads) {
    float m = S[j];
    for (int f = 1; f < F; ++f) m = fmaxf(m, S[f * N + j]);
    keyM[j] = key32(m);
  }
  __syncthreads();
  radix_select<uint32_t>(sc, N, N - p.Ks, [&](int j) { return keyM[j]; }, [](int) { return true; }, pool);

  // frame-specific core tokens of this CTA's frames: top K_c of S(f, .) inside the pool   (Eq. 5)
  for (int f = rank; f < F; f += C) {
    const float* Sf = S + (size_t)f * N;
    radix_select<uint32_t>(sc, N, p.Kc, [&](int j) { return key32(Sf[j]); }, [&](int j) { return pool[j] != 0; },
                           core + (size_t)f * Npad);
  }

  // this CTA's share of the anchor keys mu / (1 + beta CV)                               (Eq. 11, Eq. 6)
  const int share = (N + C - 1) / C;
  const int j_lo = rank * share, j_hi = min(N, j_lo + share);
  for (int j = j_lo + tid; j < j_hi; j += kSelThreads) {
    double sum = 0.0;
    for (int f = 0; f < F; ++f) sum = __dadd_rn(sum, (double)Sall[f * N + j]);
    const double mu = __ddiv_rn(sum, (double)F);
    double ss = 0.0;
    for (int f = 0; f < F; ++f) {
      const double dv = __dadd_rn((double)Sall[f * N + j], -mu);
      ss = __dadd_rn(ss, __dmul_rn(dv, dv));
    }
    const double sd = __dsqrt_rn(__ddiv_rn(ss, (double)F));
    const double cv = (mu == 0.0) ? 0.0 : __ddiv_rn(sd, mu);
    keyA[j] = key64(__ddiv_rn(mu, __dadd_rn(1.0, __dmul_rn(p.beta, cv))));
  }
  __syncthreads();

  // exchange through distributed shared memory: my frames' core flags and my anchor keys go to every other CTA
  if (C > 1) {
    cluster.sync();  // every CTA of the cluster is resident before its shared memory is written remotely
    for (int peer = 1; peer < C; ++peer) {
      const int dst = (rank + peer) % C;
      uint8_t* rbase = cluster.map_shared_rank(smem_raw, dst);
      uint64_t* rkeyA = reinterpret_cast<uint64_t*>(rbase + lay.keyA);
      for (int j = j_lo + tid; j < j_hi; j += kSelThreads) rkeyA[j] = keyA[j];
      for (int f = rank; f < F; f += C) {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(core + (size_t)f * Npad);
        uint32_t* rdst = reinterpret_cast<uint32_t*>(rbase + lay.core + (size_t)f * Npad);
        for (int w = tid; w < Npad / 4; w += kSelThreads) rdst[w] = src[w];
      }
    }
    cluster.sync();
  }

  // positions that are core in no frame (Eq. 10), then the shared anchors
  for (int j = tid; j < N; j += kSelThreads) {
    uint8_t any = 0;
    for (int f = 0; f < F; ++f) any |= core[(size_t)f * Npad + j];
    anycore[j] = any;
  }
  __syncthreads();
  radix_select<uint64_t>(sc, N, p.Ks, [&](int j) { return keyA[j]; }, [&](int j) { return anycore[j] == 0; }, anchor);

  // retained positions ascending, and the maps, for this CTA's frames
  int32_t* sel = p.sel_idx ? p.sel_idx + (int64_t)b * F * K : nullptr;
  int32_t* pm = p.pack_map ? p.pack_map + (int64_t)b * p.Lp : nullptr;
  int32_t* im = p.inv_map ? p.inv_map + (int64_t)b * p.L : nullptr;
  bool bad = false;
  for (int f = rank; f < F; f += C) {
    const uint8_t* cf = core + (size_t)f * Npad;
    const int cnt = ranked_emit(
        sc, N, [&](int j) { return (cf[j] | anchor[j]) != 0; },
        [&](int j, int r) {
          if (r >= 0 && r < K) {
            if (sel) sel[f * K + r] = j;
            if (pm) pm[p.n_obs + f * K + r] = p.n_obs + f * N + j;
          }
          if (im) im[p.n_obs + f * N + j] = (r >= 0 && r < K) ? p.n_obs + f * K + r : -1;
        });
    bad |= (cnt != K);
  }
  for (int t = rank * kSelThreads + tid; t < p.n_obs; t += C * kSelThreads) {
    if (pm) pm[t] = t;
    if (im) im[t] = t;
  }
  for (int t = rank * kSelThreads + tid; t < p.H; t += C * kSelThreads) {
    if (pm) pm[p.n_obs + F * K + t] = p.n_obs + F * N + t;
    if (im) im[p.n_obs + F * N + t] = p.n_obs + F * K + t;
  }
  if (bad && tid == 0) atomicOr(p.status, ST_BAD_COUNT);
  // the layer-quality diagnostics of the scores this CTA already holds: the last CTA of the cluster computes them
  // once its selection work is done (the anchor-key area is free by then and serves as scratch)
  if (p.quality && rank == C - 1) {
    __syncthreads();
    quality_of_scores(S, F, N, quality_parts(F), reinterpret_cast<double2*>(smem_raw + lay.keyA), p.quality + b * 3,
                      kSelThreads);
  }
}

// Multi-layer aggregation (Eq. 3, Eq. 11): V = sum over the k_layer best layers of Q_l S_l / sum Q_l and V_all the
// same over all layers, in fp64 with individually rounded operations, layers in ascending order, stored as fp32.
// Equal qualities go to the lower layer index; weights that sum to zero fall back to the plain mean.
constexpr int kMaxLayers = 256;

__global__ void __launch_bounds__(256) aggregate_kernel(const float* layer_scores, const float* layer_quality, int n_layers,
                                                        int k_layer, int B, int n_elems, float* v_core, float* v_all,
                                                        int32_t* core_layers) {
  __shared__ double q[kMaxLayers];
  __shared__ uint8_t in_core[kMaxLayers];
  __shared__ double wsum[2];
  __shared__ int n_core;
  const int b = blockIdx.y, tid = threadIdx.x;
  for (int l = tid; l < n_layers; l += 256) q[l] = (double)layer_quality[((size_t)l * B + b) * 3 + 2];
  __syncthreads();
  for (int l = tid; l < n_layers; l += 256) {
    int rank = 0;
    for (int m = 0; m < n_layers; ++m) rank += (q[m] > q[l] || (q[m] == q[l] && m < l)) ? 1 : 0;
    in_core[l] = rank < k_layer ? 1 : 0;
  }
  __syncthreads();
  if (tid == 0) {
    double wc = 0.0, wa = 0.0;
    int nc = 0;
    for (int l = 0; l < n_layers; ++l) {
      wa = __dadd_rn(wa, q[l]);
      if (in_core[l]) {
        wc = __dadd_rn(wc, q[l]);
        if (core_layers && blockIdx.x == 0) core_layers[(size_t)b * min(k_layer, n_layers) + nc] = l;
        ++nc;
      }
    }
    wsum[0] = wc; wsum[1] = wa; n_core = nc;
  }
  __syncthreads();
  const double wc = wsum[0], wa = wsum[1];
  const int e = blockIdx.x * 256 + tid;
  if (e >= n_elems) return;
  double sc = 0.0, sa = 0.0;
  for (int l = 0; l < n_layers; ++l) {
    const double s = (double)layer_scores[((size_t)l * B + b) * n_elems + e];
    sa = __dadd_rn(sa, __dmul_rn(wa == 0.0 ? 1.0 : q[l], s));
    if (in_core[l]) sc = __dadd_rn(sc, __dmul_rn(wc == 0.0 ? 1.0 : q[l], s));
  }
  v_all[(size_t)b * n_elems + e] = (float)__ddiv_rn(sa, wa == 0.0 ? (double)n_layers : wa);
  v_core[(size_t)b * n_elems + e] = (float)__ddiv_rn(sc, wc == 0.0 ? (double)n_core : wc);
}

int cluster_size(const Dims& d) {
  int c = 1;
  while (c * 2 <= d.F && c * 2 <= kMaxCluster) c *= 2;
  return c;
}

}  // namespace

size_t select_smem_bytes(const Dims& d) { return sel_layout(d.F, d.N_s).total; }

int max_layers() { return kMaxLayers; }

cudaError_t launch_aggregate(const Dims& d, const float* layer_scores, const float* layer_quality, int n_layers, int k_layer,
                             float* v_core, float* v_all, int32_t* core_layers, cudaStream_t st, int* launches) {
  const int n_elems = d.F * d.N_s;
  dim3 grid((n_elems + 255) / 256, d.B);
  ++*launches;
  aggregate_kernel<<<grid, 256, 0, st>>>(layer_scores, layer_quality, n_layers, k_layer, d.B, n_elems, v_core, v_all,
                                         core_layers);
  return cudaGetLastError();
}

cudaError_t select_prepare(const Dims& d) {
  const size_t smem = select_smem_bytes(d);
  if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
  return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

// the anchor-key area (8 bytes per spatial position) must hold the F * (parts + 1) partial sums (16 bytes each)
bool select_can_fold_quality(const Dims& d) {
  return (size_t)d.N_s * 8 >= (size_t)d.F * (quality_parts(d.F) + 1) * sizeof(double2);
}

cudaError_t launch_select(const Dims& d, const float* scores, const float* scores_all, int32_t* sel_idx,
                          int32_t* pack_map, int32_t* inv_map, int* status, cudaStream_t st, int* launches,
                          float* quality) {
  SelectParams p{scores, scores_all ? scores_all : scores, sel_idx, pack_map, inv_map, status, d.n_obs, d.F, d.N_s, d.H,
                 d.Kc, d.Ks, d.L, d.Lp, (double)d.beta, select_can_fold_quality(d) ? quality : nullptr};
  const int C = cluster_size(d);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(C, d.B, 1);
  cfg.blockDim = dim3(kSelThreads, 1, 1);
  cfg.dynamicSmemBytes = select_smem_bytes(d);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ++*launches;
  return cudaLaunchKernelEx(&cfg, select_kernel, p);
}

}  // namespace swam
