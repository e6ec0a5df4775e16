// Token selection (Eq. 4-6, 10-11) and packing metadata: one thread-block cluster per sample.
//
// The input is small (F * N_s floats, at most a few hundred KB), so the kernel is bound by the latency of its chain
// of dependent steps (scores -> candidate pool -> per-frame cores -> anchors -> maps) and by the instruction
// throughput of the SMs it runs on, not by memory.  The design shortens the chain and spreads the rest:
//   * the CTAs of a cluster (up to 8) each hold the sample's scores in shared memory; the per-frame core selections
//     (Eq. 5) and the map construction are split by frame; which positions are core in some frame is exchanged by
//     OR-ing flag words into every peer's shared memory (distributed shared memory), between the two halves of a
//     split-phase cluster barrier whose first half is posted at kernel start; the small pool and anchor selections
//     are repeated by every CTA rather than exchanged;
//   * inside a CTA one half of the warps selects pool and cores while the other half evaluates the fp64 anchor keys
//     (and, in the last CTA, the Eq. 9 diagnostics), whose long dependent chains would otherwise sit on the path;
//   * every TopK is a radix select over order-preserving integer keys that starts at the highest bit in which the
//     candidates differ (one min/max reduction finds it), takes 8 bits per pass, and stops as soon as the bin that
//     holds the k-th key is taken whole, or holds at most kListMax keys: those few are then ranked directly against
//     each other (key descending, index ascending).  Typical score maps finish in one pass plus the list step;
//     degenerate ones (many equal keys) fall through to further passes and finally to an index-order rank among
//     exactly equal keys, which is the "ties go to the lower index" rule;
//   * the ascending compaction that builds sel_idx / pack_map / inv_map gives every warp a block of consecutive
//     positions (ballot / popc ranks, coalesced stores) and needs one prefix scan over the warps.
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
constexpr int kHalf = kSelThreads / 2;
constexpr int kMaxCluster = 8;
constexpr int kListMax = 32;    // keys ranked directly against each other once the k-th key's bin is this small

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

__device__ __forceinline__ int bit_length(uint32_t x) { return 32 - __clz((int)x); }
__device__ __forceinline__ int bit_length(uint64_t x) { return 64 - __clzll((long long)x); }

// scratch of one group of warps in shared memory
struct GroupScratch {
  int hist[3][256];                  // pass p counts into hist[p % 3]; all three are zero between calls
  unsigned long long red_min[32], red_max[32];
  int red_cnt[32];
  int warp_tot[32];
  int scal[4];                       // digit, remaining, keys in the bin, list fill counter
  unsigned long long list_key[kListMax];
  int list_idx[kListMax];
};

// A group of warps working together: `size` threads (a multiple of 32), thread index t inside the group, named
// barrier `bar` (0 = the whole CTA).
struct Grp {
  int t, size, bar;
  GroupScratch* s;
  __device__ __forceinline__ void sync() const {
    if (bar == 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(size) : "memory");
  }
};

// Ascending ranks of the positions i in [0, n) with pred(i).  Every warp takes a block of consecutive 32-position
// chunks: a first sweep counts (ballot / popc), one scan over the warps' totals gives each warp its base, a second
// sweep calls emit(i, rank) for every position (rank -1 when pred is false) with the lanes on consecutive positions,
// so what emit stores is coalesced.  Returns the number of positions with pred.  Ends with a barrier.
template <typename PredFn, typename EmitFn>
__device__ int ranked(const Grp& g, int n, PredFn pred, EmitFn emit) {
  const int lane = g.t & 31, warp = g.t >> 5, n_warps = g.size >> 5;
  const int chunks = (n + 31) >> 5;
  const int per_warp = (chunks + n_warps - 1) / n_warps;
  const int c0 = min(chunks, warp * per_warp), c1 = min(chunks, c0 + per_warp);
  int cnt = 0;
  for (int c = c0; c < c1; ++c) {          // warp-uniform bounds: every lane takes part in the votes
    const int i = c * 32 + lane;
    cnt += __popc(__ballot_sync(0xffffffffu, i < n && pred(i)));
  }
  if (lane == 0) g.s->warp_tot[warp] = cnt;
  g.sync();
  const int wt = (lane < n_warps) ? g.s->warp_tot[lane] : 0;
  int wincl = wt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, wincl, o);
    if (lane >= o) wincl += v;
  }
  int base = __shfl_sync(0xffffffffu, wincl - wt, warp);
  const int total = __shfl_sync(0xffffffffu, wincl, 31);
  for (int c = c0; c < c1; ++c) {
    const int i = c * 32 + lane;
    const bool f = i < n && pred(i);
    const unsigned bal = __ballot_sync(0xffffffffu, f);
    if (i < n) emit(i, f ? base + __popc(bal & ((1u << lane) - 1u)) : -1);
    base += __popc(bal);
  }
  g.sync();   // warp_tot may be rewritten, and what emit wrote to shared memory is visible to the group
  return total;
}

// What is known about the candidates of a selection before it starts: how many there are (at least; only compared
// with k to recognise "take all"), and bounds of their keys (of a superset of them is fine: the bounds only fix the
// highest bit in which live keys can differ).
template <typename KeyT>
struct KeyRange {
  KeyT mn, mx;
  int cnt;
};

// Group-wide KeyRange of per-thread partial results.  Ends with the group holding the result in registers; the
// scratch slots it used are free again after the group's next barrier.
__device__ __forceinline__ void warp_range(uint64_t& mn, uint64_t& mx, int& cnt) {
  // lexicographic over the two 32-bit halves
  const uint32_t mn_hi = __reduce_min_sync(0xffffffffu, (uint32_t)(mn >> 32));
  const uint32_t mn_lo = __reduce_min_sync(0xffffffffu, (uint32_t)(mn >> 32) == mn_hi ? (uint32_t)mn : 0xffffffffu);
  const uint32_t mx_hi = __reduce_max_sync(0xffffffffu, (uint32_t)(mx >> 32));
  const uint32_t mx_lo = __reduce_max_sync(0xffffffffu, (uint32_t)(mx >> 32) == mx_hi ? (uint32_t)mx : 0u);
  mn = ((uint64_t)mn_hi << 32) | mn_lo;
  mx = ((uint64_t)mx_hi << 32) | mx_lo;
  cnt = __reduce_add_sync(0xffffffffu, cnt);
}
template <typename KeyT>
__device__ KeyRange<KeyT> group_range(const Grp& g, KeyT mn, KeyT mx, int cnt) {
  const int lane = g.t & 31, warp = g.t >> 5, n_warps = g.size >> 5;
  warp_range(mn, mx, cnt);
  if (lane == 0) { g.s->red_min[warp] = mn; g.s->red_max[warp] = mx; g.s->red_cnt[warp] = cnt; }
  g.sync();
  mn = (lane < n_warps) ? (KeyT)g.s->red_min[lane] : ~(KeyT)0;
  mx = (lane < n_warps) ? (KeyT)g.s->red_max[lane] : 0;
  cnt = (lane < n_warps) ? g.s->red_cnt[lane] : 0;
  warp_range(mn, mx, cnt);
  return KeyRange<KeyT>{mn, mx, cnt};
}

// TopK among candidates: flag_out[i] = 1 for the k candidates with the largest keys (ties to the lower index), 0 for
// every other i in [0, n).  key(i) -> KeyT (only called for candidates), cand(i) -> bool; `range` as described above.
// The group must have passed a barrier since `range`, the keys and the candidate flags were written.  Ends with a
// barrier.
template <typename KeyT, typename KeyFn, typename CandFn>
__device__ void topk_flags(const Grp& g, int n, int k, const KeyRange<KeyT>& range, KeyFn key, CandFn cand,
                           uint8_t* flag_out) {
  constexpr int kBits = sizeof(KeyT) * 8;
  GroupScratch* s = g.s;
  const int lane = g.t & 31;

  if (k <= 0 || k >= range.cnt) {       // nothing, or every candidate
    for (int i = g.t; i < n; i += g.size) flag_out[i] = (k > 0 && cand(i)) ? 1 : 0;
    g.sync();
    return;
  }

  // bits at and above `hi` are known: every live key has (key & mask) == prefix
  int hi = bit_length((KeyT)(range.mn ^ range.mx));
  KeyT mask = (hi >= kBits) ? (KeyT)0 : (KeyT)(~(KeyT)0 << hi);
  KeyT prefix = range.mn & mask;
  int remaining = k;
  int pass = 0;
  if (g.t == 0) s->scal[3] = 0;          // list fill counter (read only after later barriers)
  while (hi > 0) {
    const int shift = hi > 8 ? hi - 8 : 0;
    const int width = hi - shift;
    int* hist = s->hist[pass % 3];
    for (int i = g.t; i < n; i += g.size) {
      if (cand(i)) {
        const KeyT kv = key(i);
        if ((kv & mask) == prefix) atomicAdd(&hist[(int)((kv >> shift) & (KeyT)((1 << width) - 1))], 1);
      }
    }
    g.sync();
    // The buffer of the previous pass has been read by every warp (each read it before it arrived here).  It is
    // cleared now and counted into again two passes on, i.e. after the next barrier, which orders the two.
    if (pass > 0 && g.t < 256) s->hist[(pass + 2) % 3][g.t] = 0;
    // every warp locates the bin of the remaining-th largest live key for itself (no broadcast, no second barrier):
    // lane owns bins [8 * lane, 8 * lane + 8); `above` = keys in bins above the lane's
    int digit, rem, in_bin;
    {
      const int4 lo4 = *reinterpret_cast<const int4*>(&hist[lane * 8]), hi4 = *reinterpret_cast<const int4*>(&hist[lane * 8 + 4]);
      const int local[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
      const int sum = (lo4.x + lo4.y) + (lo4.z + lo4.w) + (hi4.x + hi4.y) + (hi4.z + hi4.w);
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += v;
      }
      int above = incl - sum;
      const bool mine = above < remaining && remaining <= above + sum;   // true in exactly one lane
      int d = 0, r = 0, c = 0;
      bool found = false;
#pragma unroll
      for (int j = 7; j >= 0; --j) {
        if (!found) {
          if (remaining <= above + local[j]) { d = lane * 8 + j; r = remaining - above; c = local[j]; found = true; }
          else above += local[j];
        }
      }
      const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
      digit = __shfl_sync(0xffffffffu, d, src);
      rem = __shfl_sync(0xffffffffu, r, src);
      in_bin = __shfl_sync(0xffffffffu, c, src);
    }
    prefix |= (KeyT)digit << shift;
    mask |= (KeyT)((1 << width) - 1) << shift;
    remaining = rem;
    hi = shift;
    if (in_bin == remaining) {
      // the bin is taken whole: everything at or above the prefix is in
      for (int i = g.t; i < n; i += g.size) flag_out[i] = (cand(i) && (key(i) & mask) >= prefix) ? 1 : 0;
      g.sync();
      if (g.t < 256) hist[g.t] = 0;
      g.sync();
      return;
    }
    if (hi > 0 && in_bin <= kListMax) {
      // few keys left in the bin: rank them against each other (key descending, index ascending)
      for (int i = g.t; i < n; i += g.size) {
        uint8_t fl = 0;
        if (cand(i)) {
          const KeyT kv = key(i);
          if ((kv & mask) == prefix) {
            const int slot = atomicAdd(&s->scal[3], 1);
            s->list_key[slot] = (unsigned long long)kv;
            s->list_idx[slot] = i;
            continue;                      // its flag is written by the ranking below
          }
          fl = (kv & mask) > prefix ? 1 : 0;
        }
        flag_out[i] = fl;
      }
      g.sync();
      if (g.t < 256) hist[g.t] = 0;        // every warp has located its bin
      if (g.t < kListMax) {
        const unsigned long long mk = s->list_key[g.t < in_bin ? g.t : 0];
        const int mi = s->list_idx[g.t < in_bin ? g.t : 0];
        int rank = 0;
#pragma unroll 8
        for (int u = 0; u < kListMax; ++u) {
          const unsigned long long uk = s->list_key[u];
          const int ui = s->list_idx[u];
          const int beats = ((uk > mk) | ((uk == mk) & (ui < mi))) & (u < in_bin);
          rank += beats;
        }
        if (g.t < in_bin) flag_out[mi] = rank < remaining ? 1 : 0;
      }
      g.sync();
      return;
    }
    ++pass;
  }
  // every bit is resolved and the bin holds more equal keys than are wanted: the lower indices win
  if (pass > 0) {
    g.sync();
    if (g.t < 256) s->hist[(pass - 1) % 3][g.t] = 0;
  }
  ranked(g, n, [&](int i) { return cand(i) && key(i) == prefix; },
         [&](int i, int r) { flag_out[i] = (r >= 0 ? r < remaining : (cand(i) && key(i) > prefix)) ? 1 : 0; });
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
  size_t keyA, scratch, qual, anycore, S, Sall, keyM, pool, anchor, core, total;
};
__host__ __device__ inline SelLayout sel_layout(int F, int N, bool two_maps) {
  SelLayout l;
  size_t o = 0;
  auto put = [&o](size_t bytes) { const size_t at = o; o = (o + bytes + 15) & ~(size_t)15; return at; };   // 16-byte aligned blocks
  l.keyA = put((size_t)N * 8);
  l.scratch = put(sizeof(GroupScratch));
  l.qual = put((size_t)F * (quality_parts(F) + 1) * sizeof(double2));
  l.anycore = put(((size_t)N + 3) / 4 * 4);          // flag bytes, OR-ed in as 32-bit words
  l.S = put((size_t)F * N * 4);
  l.Sall = put(two_maps ? (size_t)F * N * 4 : 0);
  l.keyM = put((size_t)N * 4);
  l.pool = put((size_t)N);
  l.anchor = put((size_t)N);
  l.core = put(((size_t)N + 3) / 4 * 4 * F);         // each frame's flags start on a 4-byte boundary
  l.total = o;
  return l;
}

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(const SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int F = p.F, N = p.N_s, K = p.Kc + p.Ks;
  const int Npad = (N + 3) / 4 * 4;
  const bool two_maps = p.scores_all != p.scores;
  const SelLayout lay = sel_layout(F, N, two_maps);
  uint64_t* keyA = reinterpret_cast<uint64_t*>(smem_raw + lay.keyA);
  GroupScratch* scratch = reinterpret_cast<GroupScratch*>(smem_raw + lay.scratch);
  float* S = reinterpret_cast<float*>(smem_raw + lay.S);
  uint32_t* keyM = reinterpret_cast<uint32_t*>(smem_raw + lay.keyM);
  uint8_t* pool = smem_raw + lay.pool;
  uint8_t* anchor = smem_raw + lay.anchor;
  uint8_t* anycore = smem_raw + lay.anycore;
  uint8_t* core = smem_raw + lay.core;  // [F][Npad]

  const int tid = threadIdx.x, b = blockIdx.y;
  for (int i = tid; i < 3 * 256; i += kSelThreads) (&scratch->hist[0][0])[i] = 0;
  for (int w = tid; w < Npad / 4; w += kSelThreads) reinterpret_cast<uint32_t*>(anycore)[w] = 0;
  // First half of the cluster barrier: this CTA's shared memory is initialised; its peers may OR core flags into it
  // and store their share of the anchor keys (they wait for every CTA's arrival before they do).
  if (C > 1) cluster_arrive();

  const float* sg = p.scores + (int64_t)b * F * N;
  for (int i = tid; i < F * N; i += kSelThreads) S[i] = sg[i];
  const float* Sall = S;  // the anchor statistic reads V_all; with one profiled layer it is the same map
  if (two_maps) {
    float* sa = reinterpret_cast<float*>(smem_raw + lay.Sall);
    const float* sag = p.scores_all + (int64_t)b * F * N;
    for (int i = tid; i < F * N; i += kSelThreads) sa[i] = sag[i];
    Sall = sa;
  }
  __syncthreads();

  if (tid < kHalf) {
    // ---- warps 0-15: candidate pool, then the core tokens of this CTA's frames
    const Grp half{tid, kHalf, 1, scratch};
    // keys of the pool selection, max_f S(f, j), with their range, and the smallest score key of all frames
    uint32_t mn = 0xffffffffu, mx = 0, mn_all = 0xffffffffu;
    for (int j = tid; j < N; j += kHalf) {
      float m = S[j], lo = S[j];
      for (int f = 1; f < F; ++f) {
        const float v = S[f * N + j];
        m = fmaxf(m, v);
        lo = fminf(lo, v);
      }
      const uint32_t kv = key32(m);
      keyM[j] = kv;
      mn = min(mn, kv);
      mx = max(mx, kv);
      mn_all = min(mn_all, key32(lo));
    }
    {
      const int lane = tid & 31, warp = tid >> 5;
      mn = __reduce_min_sync(0xffffffffu, mn);
      mx = __reduce_max_sync(0xffffffffu, mx);
      mn_all = __reduce_min_sync(0xffffffffu, mn_all);
      if (lane == 0) { scratch->red_min[warp] = mn; scratch->red_max[warp] = mx; scratch->red_cnt[warp] = (int)mn_all; }
      half.sync();                                   // also publishes keyM
      mn = __reduce_min_sync(0xffffffffu, lane < kHalf / 32 ? (uint32_t)scratch->red_min[lane] : 0xffffffffu);
      mx = __reduce_max_sync(0xffffffffu, lane < kHalf / 32 ? (uint32_t)scratch->red_max[lane] : 0u);
      mn_all = __reduce_min_sync(0xffffffffu, lane < kHalf / 32 ? (uint32_t)scratch->red_cnt[lane] : 0xffffffffu);
    }
    // top (N_s - K_s) of max_f S(f, j)                                                       (Eq. 4)
    topk_flags<uint32_t>(half, N, N - p.Ks, KeyRange<uint32_t>{mn, mx, N}, [&](int j) { return keyM[j]; },
                         [](int) { return true; }, pool);
    // top K_c of S(f, .) inside the pool; the pool has exactly N_s - K_s members, and every score key lies between
    // the smallest key of all frames and the largest pool key                                  (Eq. 5)
    for (int f = rank; f < F; f += C) {
      const float* Sf = S + (size_t)f * N;
      topk_flags<uint32_t>(half, N, p.Kc, KeyRange<uint32_t>{mn_all, mx, N - p.Ks}, [&](int j) { return key32(Sf[j]); },
                           [&](int j) { return pool[j] != 0; }, core + (size_t)f * Npad);
    }
  } else {
    // ---- warps 16-31: this CTA's share of the anchor keys mu / (1 + beta CV), sent to every CTA   (Eq. 11, Eq. 6)
    const int t = tid - kHalf;
    const int share = (N + C - 1) / C;
    const int j_lo = rank * share, j_hi = min(N, j_lo + share);
    for (int j = j_lo + t; j < j_hi; j += kHalf) {
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
    if (C > 1) {
      cluster_wait();                      // every CTA of the cluster is resident and initialised
      for (int peer = 1; peer < C; ++peer) {
        uint64_t* rkeyA = cluster.map_shared_rank(keyA, (rank + peer) % C);
        for (int j = j_lo + t; j < j_hi; j += kHalf) rkeyA[j] = keyA[j];
      }
      cluster_arrive();                    // second half of the barrier: this thread's remote stores are done
    }
    // the layer-quality diagnostics of the scores this CTA holds: these warps of the last CTA have the time
    if (p.quality && rank == C - 1)
      quality_of_scores(S, F, N, quality_parts(F), reinterpret_cast<double2*>(smem_raw + lay.qual), p.quality + b * 3, t,
                        kHalf, [] { asm volatile("bar.sync 2, %0;" ::"n"(kHalf) : "memory"); });
  }

  // positions that are core in some frame (Eq. 10): this CTA's frames are OR-ed into every CTA's flag words
  if (tid < kHalf) {
    if (C > 1) cluster_wait();
    for (int f = rank; f < F; f += C) {
      const uint32_t* src = reinterpret_cast<const uint32_t*>(core + (size_t)f * Npad);
      for (int w = tid; w < Npad / 4; w += kHalf) {
        const uint32_t v = src[w];
        if (v) {
          for (int peer = 0; peer < C; ++peer)
            atomicOr(reinterpret_cast<unsigned int*>(cluster.map_shared_rank(anycore, (rank + peer) % C)) + w, v);
        }
      }
    }
    if (C > 1) cluster_arrive();
  }
  if (C > 1) cluster_wait();
  __syncthreads();

  // the shared anchors: top K_s of the anchor key among positions that are core in no frame   (Eq. 6)
  const Grp all{tid, kSelThreads, 0, scratch};
  {
    uint64_t mn = ~0ull, mx = 0;
    int cnt = 0;
    for (int j = tid; j < N; j += kSelThreads) {
      if (anycore[j] == 0) {
        const uint64_t kv = keyA[j];
        mn = kv < mn ? kv : mn;
        mx = kv > mx ? kv : mx;
        ++cnt;
      }
    }
    const KeyRange<uint64_t> rA = group_range<uint64_t>(all, mn, mx, cnt);
    topk_flags<uint64_t>(all, N, p.Ks, rA, [&](int j) { return keyA[j]; }, [&](int j) { return anycore[j] == 0; }, anchor);
  }

  // retained positions ascending, and the maps, for this CTA's frames
  int32_t* sel = p.sel_idx ? p.sel_idx + (int64_t)b * F * K : nullptr;
  int32_t* pm = p.pack_map ? p.pack_map + (int64_t)b * p.Lp : nullptr;
  int32_t* im = p.inv_map ? p.inv_map + (int64_t)b * p.L : nullptr;
  for (int t = rank * kSelThreads + tid; t < p.n_obs; t += C * kSelThreads) {
    if (pm) pm[t] = t;
    if (im) im[t] = t;
  }
  for (int t = rank * kSelThreads + tid; t < p.H; t += C * kSelThreads) {
    if (pm) pm[p.n_obs + F * K + t] = p.n_obs + F * N + t;
    if (im) im[p.n_obs + F * N + t] = p.n_obs + F * K + t;
  }
  bool bad = false;
  for (int f = rank; f < F; f += C) {
    const uint8_t* cf = core + (size_t)f * Npad;
    const int cnt = ranked(
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
  if (bad && tid == 0) atomicOr(p.status, ST_BAD_COUNT);
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

// the largest layout (two score maps) decides whether a shape is supported at all
size_t select_smem_bytes(const Dims& d) { return sel_layout(d.F, d.N_s, true).total; }

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

// the diagnostics always ride along with the selection launch (idle warps of the cluster's last CTA compute them)
bool select_can_fold_quality(const Dims&) { return true; }

cudaError_t launch_select(const Dims& d, const float* scores, const float* scores_all, int32_t* sel_idx,
                          int32_t* pack_map, int32_t* inv_map, int* status, cudaStream_t st, int* launches,
                          float* quality) {
  const bool two_maps = scores_all && scores_all != scores;
  SelectParams p{scores, two_maps ? scores_all : scores, sel_idx, pack_map, inv_map, status, d.n_obs, d.F, d.N_s, d.H,
                 d.Kc, d.Ks, d.L, d.Lp, (double)d.beta, quality};
  const int C = cluster_size(d);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(C, d.B, 1);
  cfg.blockDim = dim3(kSelThreads, 1, 1);
  cfg.dynamicSmemBytes = sel_layout(d.F, d.N_s, two_maps).total;
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
