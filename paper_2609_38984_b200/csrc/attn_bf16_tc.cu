// Joint softmax attention for bf16 tensors on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
// One CTA owns two 128-row query tiles of one (sample, head) and walks over the keys in tiles of 128:
//   warp 9      TMA producer: Q once, then K_j / V_j into a ring of shared-memory stages (128B-swizzled boxes)
//   warp 8      one elected thread issues every tcgen05.mma: S = Q_s K_j^T (both operands K-major in shared
//               memory) into a TMEM score buffer, then O_s += P V_j with P read from TMEM and V_j as an MN-major
//               operand
//   warps 0-3   softmax of query tile 0: one thread per row reads its S row from TMEM, keeps the reference maximum
//   warps 4-7   and the running sum (exp2 domain), writes P as bf16 back over S; same for query tile 1
//   warps 10-11 idle (they complete the third warpgroup, which hands most of its registers to the softmax warps)
// Head dim 64: work is a sequence of items (key tile, query tile); item i uses score buffer i mod 3 and the issuing
// thread keeps Q K^T three items ahead of P V, so one tile's exponentials overlap the other tile's MMAs.
// Head dim 128: TMEM (512 columns) holds only two score buffers beside the two outputs, so P does not go back over
// the scores: each softmax thread stores its bf16 P row into a shared-memory tile laid out like a K-major operand
// (both products then read both operands from shared memory) and releases its score buffer as soon as the scores are
// in its registers.  Q K^T of key tile j+1 therefore never waits for P V of tile j; the tensor pipe runs
// S(0) | S(1), PV(0) | S(2), PV(1) | ... with both query tiles side by side, and K and V tiles share one ring of three
// shared-memory slots that is filled in exactly that order.  O stays in TMEM for the whole key loop; it is rescaled only when a row's maximum has grown by
// more than 2^8 beyond the value its exponentials refer to (the result is exact either way: sums and outputs share
// the same reference maximum).  Work items left over after the last full wave of CTAs are cut over the keys and
// merged by a small combine kernel.  Every wait on an mbarrier is bounded; when a wait runs out the kernel raises
// the timeout bit of the status word, stops issuing work, and every role falls through to the common exit.
#include "tc_ptx.cuh"

namespace swam {
namespace {

constexpr int kThreadsTc = 384;     // 8 softmax warps + MMA warp + TMA warp + 2 idle warps (three full warpgroups)

struct TcParams {
  float* lse;
  int* status;
  float* partial;      // split items: [slot][2 tiles][128 rows][D + 4]: unnormalised O, then reference max and sum
  const int32_t* pack_map;  // gather mode: [B, n] row of the full tensors that each attended row stands for
  int n_full;               // gather modes: rows per sample of the full tensors
  union {
    int kv_rows;            // kGatherKV: rows of the 2-D view of K and V, B * n_full (a row coordinate beyond the tensor)
    int direct_tiles;       // kGather: the first key tiles come from the full K and V (maps in the slots of map_q and map_o)
  };
  const __nv_bfloat16* q_full;  // gather mode: the full [B, n_full, N_h, D] query tensor
  __nv_bfloat16* out_full;      // gather mode: the full [B, n_full, N_h, D] output tensor
  int lse_row0, lse_rows;
  int n, N_h;
  int kv_group;        // query heads per key/value head
  int pairs;           // query tile pairs per (sample, head)
  int total_work;      // n_whole + (items of the last, partly filled wave) * splits: what the CTAs share out
  int n_whole;         // work items that run over all keys and write the output themselves
  int splits;          // pieces per split item (0 when nothing is split)
  int tiles_per_split; // key tiles per piece
  float scale_log2;
  // segment-prefix visibility: rows [0, obs_end) see the first lim0 keys, rows [obs_end, fut_end) the first lim1, the
  // rest the first lim2 (all equal to n: full visibility)
  int obs_end, fut_end, lim0, lim1, lim2;
};

template <int D>
struct TcCfg {
  static constexpr int DB = D / 64;                 // 64-column (128-byte) blocks per row
  static constexpr int kSubTile = kTile * 128;      // bytes of one [128 rows x 64 cols] block
  static constexpr int kTileBytes = DB * kSubTile;  // one 128 x D tile
  // Head dim 128 keeps P in shared memory (see the kernel's header): its key and value tiles then share ONE ring of
  // three slots, filled and consumed in the order K_0, K_1, V_0, K_2, V_1, ... in which the tensor pipe uses them, so
  // that every load has a whole key-tile step to arrive.  Head dim 64 has a ring of kStages slots for K and one for V.
  // (head dim 64 keeps P in TMEM: its three score buffers already let Q K^T run ahead, and with P in shared memory
  // the same launch was 7 % slower)
  static constexpr bool kPSmem = (D == 128);
  static constexpr int kPTileBytes = 2 * kSubTile;   // a 128 x 128 bf16 P tile: two 64-key blocks
  static constexpr int kStages = kPSmem ? 3 : 4;
  static constexpr int kRingTiles = kPSmem ? kStages : 2 * kStages;
  // score buffers in TMEM: two at D = 128 (S0, S1, O0, O1 fill all 512 columns); at D = 64 the outputs need only 128
  // columns, which leaves room for a third score buffer and lets Q K^T run one tile further ahead of the softmax
  static constexpr int kSBufs = (D == 128) ? 2 : 3;
  // of every 8 element pairs of the softmax pass, this many take their exponential on the FMA pipes (measured: one
  // in eight is the optimum at both head dims; every further eighth costs more FMA-pipe time than it frees on the
  // exp2 unit)
  static constexpr int kPolyOf8 = 1;
  // The epilogue stages a query tile's bf16 output in shared memory for the TMA store.  Head dim 64 has room for two
  // staging tiles of their own: the query tiles are then free as soon as the item's last Q K^T has run, and the next
  // item's queries load (and its first Q K^T run) under the current item's tail (3 % on the multi-view launches).
  // Head dim 128 has no room left and stages in the finished query tiles (staging in the P tiles instead, which are
  // also free by then, was 1 % slower: the next item's first P stores then wait for the copy engine).
  static constexpr bool kStageOwn = !kPSmem;
  static constexpr int kStageBytes = kStageOwn ? 2 * kTileBytes : 0;
  static constexpr int kSmemData = (2 + kRingTiles) * kTileBytes + (kPSmem ? 2 * kPTileBytes : 0) + kStageBytes;   // Q tiles, ring(s), P tiles, staging
  static constexpr int kSmemBytes = kSmemData + 1024 /*alignment slack*/ + 512 /*barriers*/;
  static constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTile >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
  static constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(D >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
};

// MODE = kDirect: the tensor maps cover [B, n, N_h, D] tensors in boxes of 128 rows; one output store per query tile.
// MODE = kGather (the sparse step with Eq. 7's scatter and the query third of Sec. 4.2's pack fused in): K and V are
// packed tensors as before, but Q and the output are the FULL [B, n_full, N_h, D] tensors.  Two warps fetch the query
// rows pack_map names with 16-byte asynchronous copies, writing the same swizzled tile layout the tensor map would, so
// the packed Q never exists in memory, and each attended row goes straight to its original position
// pack_map[b, row] (plain 16-byte stores from the staged tile); the rows the packed sequence omits are never touched
// and keep the cached values they hold.  map_q and map_o are not used.  (K and V are shared by every query tile pair
// of a head: packing them once is cheaper than gathering them in every CTA.)
// MODE = kGatherKV: as kGather, and K and V are the FULL tensors as well: the producer warp fetches each key tile's
// rows through pack_map with TMA row gathers (tile::gather4: every lane names four rows of the 2-D view
// [B * n_full, N_kv * D] and gets them as four consecutive rows of the swizzled tile), so that no packed tensor exists
// at all.  Every query tile pair of a head repeats the gather of that head's keys and values, which is why it is an
// option and not the default (see swam_set_option).
enum { kDirect = 0, kGather = 2, kGatherKV = 3 };
constexpr int kGatherThreads = 64;   // warps 10 and 11

// VIS: visibility is restricted (per-row key limits); false = every row sees all n keys and none of that code exists
template <int D, int MODE, bool VIS>
__global__ void __launch_bounds__(kThreadsTc, 1)
attn_bf16_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o, const TcParams p) {
  using C = TcCfg<D>;
  constexpr bool kGath = MODE == kGather || MODE == kGatherKV;   // the queries are gathered by warps 10 and 11
  constexpr int ST = C::kStages;
  // Where the epilogue stages the output: tiles of its own (head dim 64), the P tiles (head dim 128 in the
  // scattering modes, where the staged rows leave by plain loads and stores and are gone when the next item's first
  // P stores come), or the finished query tiles (head dim 128, direct mode).  In the first two cases the query
  // tiles are released by the issuing warp after the item's last Q K^T.
  constexpr bool kStageP = C::kPSmem && MODE != kDirect;
  constexpr bool kQEarly = C::kStageOwn || kStageP;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_addr(smem_raw) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - smem_addr(smem_raw));
  const uint32_t sQ = base;                                 // [2][tile]
  const uint32_t sP = sQ + 2 * C::kTileBytes;               // [2][tile], only with P in shared memory
  const uint32_t sK = sP + (C::kPSmem ? 2 * C::kPTileBytes : 0);   // [ST][tile]; the one ring of both with P in shared memory
  const uint32_t sV = C::kPSmem ? sK : sK + ST * C::kTileBytes;   // [ST][tile]
  const uint32_t sStage = C::kStageOwn ? sV + ST * C::kTileBytes : (kStageP ? sP : sQ);   // [2] output staging tiles
  constexpr uint32_t kStageStride = kStageP ? C::kPTileBytes : C::kTileBytes;
  const uint32_t bars = base + C::kSmemData;
  // barrier slots (8 bytes each)
  const uint32_t bar_q = bars;
  auto bar_k_full = [&](int s) { return bars + 8 * (1 + s); };
  auto bar_k_empty = [&](int s) { return bars + 8 * (1 + ST + s); };
  auto bar_v_full = [&](int s) { return bars + 8 * (1 + 2 * ST + s); };
  auto bar_v_empty = [&](int s) { return bars + 8 * (1 + 3 * ST + s); };
  constexpr int NB = C::kSBufs;
  auto bar_s_full = [&](int buf) { return bars + 8 * (1 + 4 * ST + buf); };
  auto bar_p_full = [&](int buf) { return bars + 8 * (4 + 4 * ST + buf); };
  const uint32_t bar_o_final = bars + 8 * (7 + 4 * ST);
  // P V of a query tile's item has completed: that tile's output accumulator is up to date
  auto bar_pv_tile = [&](int s) { return bars + 8 * (8 + 4 * ST + s); };
  // a CTA works through several items: the output accumulators have been read (the next item's first P V may
  // overwrite them), and the query tiles are free (the next item's queries may be loaded): with staging tiles of
  // their own, when the item's last Q K^T has run; otherwise when the copy engine has read the output staged in them
  const uint32_t bar_o_free = bars + 8 * (10 + 4 * ST);
  const uint32_t bar_q_free = bars + 8 * (11 + 4 * ST);
  // P in shared memory: the softmax threads have read a score buffer into registers (the next Q K^T may overwrite it)
  auto bar_s_free = [&](int s) { return bars + 8 * (12 + 4 * ST + s); };
  // the staged output of query tile s has been read (its threads may write that memory again): by the copy engine
  // in direct mode, by the tile's own threads in the scattering modes
  auto bar_stage_free = [&](int s) { return bars + 8 * (14 + 4 * ST + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + C::kSmemData + 8 * (16 + 4 * ST));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + C::kSmemData + 8 * (16 + 4 * ST) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Work item = (sample, head, query tile pair), pair fastest.  Items below n_whole walk over all keys; the few items
  // of the last, partly filled wave are cut into `splits` pieces over the keys so that they spread over idle SMs,
  // each piece leaving an unnormalised partial result for the combine kernel.  The grid has one CTA per SM (or per
  // work item if there are fewer); CTA c takes work c, c + gridDim.x, ...  Every role walks through the same
  // sequence on its own, and all barrier phases simply keep counting across items (running tile and item counters),
  // so that the next item's key/value tiles stream in while this item's epilogue runs and nothing is set up twice.
  struct Work { int h, b, row0, kv_begin, n_tiles, slot; };
  const int all_tiles = (p.n + kTile - 1) / kTile;
  auto row_limit = [&](int row) { return row < p.obs_end ? p.lim0 : (row < p.fut_end ? p.lim1 : p.lim2); };
  auto decode = [&](int w) {
    Work k;
    int item = w, kv_end = all_tiles;
    k.kv_begin = 0;
    k.slot = -1;
    if (item >= p.n_whole) {
      k.slot = item - p.n_whole;
      item = p.n_whole + k.slot / p.splits;
      k.kv_begin = (k.slot % p.splits) * p.tiles_per_split;
      kv_end = min(all_tiles, k.kv_begin + p.tiles_per_split);
    }
    const int pair = item % p.pairs;
    k.h = (item / p.pairs) % p.N_h;
    k.b = item / (p.pairs * p.N_h);
    k.row0 = pair * 2 * kTile;
    // key tiles beyond what any row of the pair sees are not visited (items are not cut over the keys when visibility
    // is restricted, so kv_begin is 0 then)
    if (VIS) {
      const int r_last = min(k.row0 + 2 * kTile, p.n) - 1;
      int lim = row_limit(k.row0);
      if (r_last >= p.obs_end && k.row0 < p.fut_end) lim = max(lim, p.lim1);
      if (r_last >= p.fut_end) lim = max(lim, p.lim2);
      kv_end = min(kv_end, (lim + kTile - 1) / kTile);
    }
    k.n_tiles = kv_end - k.kv_begin;  // >= 1 by construction
    return k;
  };

  if (threadIdx.x == 0) {
    // direct loads: one arrival (the expect_tx) plus the bytes; gathered loads: one arrival per producer thread
    mbar_init(bar_q, kGath ? kGatherThreads : 1);
    for (int s = 0; s < ST; ++s) {
      mbar_init(bar_k_full(s), 1);
      mbar_init(bar_k_empty(s), 1);
      mbar_init(bar_v_full(s), 1);
      mbar_init(bar_v_empty(s), 1);
    }
    for (int buf = 0; buf < NB; ++buf) {
      mbar_init(bar_s_full(buf), 1);
      mbar_init(bar_p_full(buf), kTile);
    }
    mbar_init(bar_pv_tile(0), 1);
    mbar_init(bar_pv_tile(1), 1);
    mbar_init(bar_s_free(0), kTile);
    mbar_init(bar_s_free(1), kTile);
    mbar_init(bar_o_final, 1);
    mbar_init(bar_o_free, 2 * kTile);
    mbar_init(bar_q_free, kQEarly ? 1 : ((MODE == kDirect) ? 2 : 2 * kTile));
    mbar_init(bar_stage_free(0), (MODE == kDirect) ? 1 : kTile);
    mbar_init(bar_stage_free(1), (MODE == kDirect) ? 1 : kTile);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_addr(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // TMEM columns: NB score buffers of 128 columns, then O0 and O1 (D columns each): 512 in total for both head
  // dims.  Work is a sequence of items i = 2 * tile + query tile; item i uses score buffer i % NB, and its P (bf16)
  // overlays the first 64 columns of that buffer.
  auto tm_S = [&](int buf) { return tmem + (uint32_t)(buf * kTile); };
  auto tm_O = [&](int s) { return tmem + (uint32_t)(NB * kTile + s * D); };

  // register budget: the softmax warpgroups hold a whole S row per thread, the third warpgroup (MMA issuer, TMA
  // producer, two idle warps) needs almost nothing
  // (setmaxnreg is a warpgroup-wide instruction: all four warps of a warpgroup execute the same one.  The kernel
  // starts with 168 registers per thread (384 threads, one CTA per SM); lowering the third warpgroup to 56 releases
  // 112 x 128 = 14336 registers, and raising the two softmax warpgroups to 224 takes exactly those 56 x 256 = 14336.  An
  // increase beyond what was released would wait forever.)
  if (warp >= 8) {
   asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
   if (kGath && warp >= 10) {
    // ------------------------------------------------------------------ gathering producers of Q (64 threads)
    // Tile row rr <- row pack_map[b, prow0 + rr] of the full tensor; 16-byte chunk cc of a row lands where the
    // 128-byte-swizzled box layout puts it: sub-tile cc / 8, row rr, chunk (cc % 8) ^ (rr % 8).  Rows beyond the
    // packed sequence, and rows whose map entry is out of range (flagged), are filled with zeros.
    // Rows are handled in blocks of 32: a warp reads the 32 map entries of a block with one coalesced load and then
    // hands them out by shuffle, so that the copy loop itself contains no loads.
    constexpr int CPR = D / 8;                 // 16-byte chunks per row
    constexpr int RPI = 32 / CPR;              // rows per warp instruction
    const int pw = warp - 10;
    const int cc = lane % CPR, sub = lane / CPR;
    const int64_t row_stride = (int64_t)p.N_h * D;
    const uint32_t dst_cc = (uint32_t)((cc >> 3) * C::kSubTile);
    const int32_t* pm = nullptr;     // map of the current work item's sample
    int64_t base_off = 0;            // first element of (sample, head), this lane's chunk
    // map entries of row block rb of the tile starting at packed row prow0: -1 = fill with zeros
    auto block_rows = [&](int prow0, int rb) {
      const int pr = prow0 + rb * 32 + lane;
      int orow = -1;
      if (pr < p.n) {
        orow = pm[pr];
        if (orow < 0 || orow >= p.n_full) {
          atomicOr(p.status, ST_BAD_MAP);
          orow = -1;
        }
      }
      return orow;
    };
    // per-lane constants of the copy loop: the swizzled chunk position only depends on (row % 8), and a lane's rows
    // advance by RPI per instruction, so the positions repeat every 8 / RPI instructions
    uint32_t dst_lane[8 / RPI];
#pragma unroll
    for (int i = 0; i < 8 / RPI; ++i) {
      const int rl = i * RPI + sub;
      dst_lane[i] = dst_cc + (uint32_t)(rl * 128 + (((cc & 7) ^ (rl & 7)) << 4));
    }
    auto gather_block = [&](uint32_t dst, const __nv_bfloat16* src, int rb, int rows_reg) {
      const __nv_bfloat16* src_lane = src + base_off;
      const uint32_t dst_blk = dst + (uint32_t)(rb * 32 * 128);
#pragma unroll
      for (int i = 0; i < 32 / RPI; ++i) {
        const int orow = __shfl_sync(0xffffffffu, rows_reg, i * RPI + sub);
        cp_async_16(dst_blk + dst_lane[i % (8 / RPI)] + (uint32_t)((i / (8 / RPI)) * 8 * 128),
                    src_lane + (orow < 0 ? 0 : orow) * row_stride, orow < 0 ? 0u : 16u);
      }
    };
    int iter = 0;
    for (int work = blockIdx.x; work < p.total_work; work += gridDim.x, ++iter) {
      const Work wk = decode(work);
      pm = p.pack_map + (int64_t)wk.b * p.n;
      base_off = ((int64_t)wk.b * p.n_full * p.N_h + wk.h) * D + cc * 8;
      if (iter > 0) {
        // the previous item's output has left the query tiles
        int go = 1;
        if (lane == 0) go = mbar_wait(bar_q_free, (iter - 1) & 1, abort_flag) ? 1 : 0;
        if (__shfl_sync(0xffffffffu, go, 0) == 0) break;
      }
      // warp pw copies row blocks pw and pw + 2 of both query tiles
      for (int s = 0; s < 2; ++s) {
        const int prow0 = wk.row0 + s * kTile;
        const int r0 = block_rows(prow0, pw), r1 = block_rows(prow0, pw + 2);
        gather_block(sQ + s * C::kTileBytes, p.q_full, pw, r0);
        gather_block(sQ + s * C::kTileBytes, p.q_full, pw + 2, r1);
      }
      cp_async_arrive(bar_q);
    }
    cp_async_wait_all();   // nothing of this thread is still on its way into shared memory at exit
   } else if (warp == 9) {
    // ------------------------------------------------------------------ TMA producer (one lane; the whole warp when
    // the key and value rows are gathered)
    if (MODE == kGatherKV || lane == 0) {
      // a failed wait ends the loops; when the whole warp runs them it must leave them together
      auto wait = [&](uint32_t bar, uint32_t parity) {
        bool r = mbar_wait(bar, parity, abort_flag);
        if constexpr (MODE == kGatherKV) r = __all_sync(0xffffffffu, r ? 1 : 0) != 0;
        return r;
      };
      bool ok = true;
      int kt = 0;      // key/value tiles loaded so far by this CTA: ring slot kt % ST, pass kt / ST
      int iter = 0;
      for (int work = blockIdx.x; work < p.total_work && ok; work += gridDim.x, ++iter) {
        const Work wk = decode(work);
        const int h_kv = wk.h / p.kv_group;
        // key tile `tile` of K or V into the ring slot at `dst`, completing on `bar`
        auto load_kv = [&](uint32_t dst, bool is_v, int tile, uint32_t bar) {
          if constexpr (MODE == kGatherKV) {
            if (lane == 0) mbar_expect_tx(bar, C::kTileBytes);
            __syncwarp();
            // this lane's four rows of the tile: attended rows 4 * lane .. + 3; rows beyond the packed sequence and
            // map entries out of range (flagged) name a row past the end of the tensor, which reads as zeros
            int y[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int row = tile * kTile + 4 * lane + e;
              y[e] = p.kv_rows;
              if (row < p.n) {
                const int o = p.pack_map[(int64_t)wk.b * p.n + row];
                if (o < 0 || o >= p.n_full) atomicOr(p.status, ST_BAD_MAP);
                else y[e] = wk.b * p.n_full + o;
              }
            }
            for (int db = 0; db < C::DB; ++db)
              tma_gather4(dst + db * C::kSubTile + lane * 4 * 128, is_v ? &map_v : &map_k, bar, h_kv * D + db * 64, y[0], y[1],
                          y[2], y[3]);
          } else {
            mbar_expect_tx(bar, C::kTileBytes);
            // gather mode: the leading tiles (observed tokens, which the packed sequence shares with the full one) come
            // straight from the full tensors, whose maps travel in the slots the direct mode uses for Q and the output
            const CUtensorMap* mp = is_v ? &map_v : &map_k;
            if constexpr (MODE == kGather) {
              if (tile < p.direct_tiles) mp = is_v ? &map_o : &map_q;
            }
            for (int db = 0; db < C::DB; ++db)
              tma_load_4d(dst + db * C::kSubTile, mp, bar, db * 64, tile * kTile, h_kv, wk.b);
          }
        };
        // The first item's queries go first.  A later item's queries have to wait until the previous item's output has
        // left the query tiles, so that item's first key/value tiles (as many as the ring holds) are requested before.
        auto load_q = [&]() {
          if (kGath) return true;
          if (iter > 0 && !wait(bar_q_free, (iter - 1) & 1)) return false;
          mbar_expect_tx(bar_q, 2 * C::kTileBytes);
          for (int s = 0; s < 2; ++s)
            for (int db = 0; db < C::DB; ++db)
              tma_load_4d(sQ + s * C::kTileBytes + db * C::kSubTile, &map_q, bar_q, db * 64, wk.row0 + s * kTile, wk.h, wk.b);
          return true;
        };
        if constexpr (C::kPSmem) {
          // one ring: load m of an item is K_0 (m = 0), K_(m+1)/2 (odd m), V_(m/2-1) (even m), and V of the last tile
          // at the end.  The ring's slots that a new item's first loads wait for are freed by the previous item, so
          // those loads go out before the (possibly long) wait for the query tiles.
          const int n_loads = 2 * wk.n_tiles;
          const int q_after = (iter == 0) ? -1 : min(ST, n_loads) - 1;
          if (q_after < 0) ok = load_q();
          for (int m = 0; m < n_loads && ok; ++m, ++kt) {
            const int st = kt % ST;
            ok = wait(bar_k_empty(st), ((kt / ST) & 1) ^ 1);
            if (!ok) break;
            const bool is_v = (m == n_loads - 1) || (m > 0 && (m & 1) == 0);
            const int j = (m == n_loads - 1) ? wk.n_tiles - 1 : (is_v ? m / 2 - 1 : (m + 1) / 2);
            load_kv(sK + st * C::kTileBytes, is_v, wk.kv_begin + j, bar_k_full(st));
            if (m == q_after) ok = load_q();
          }
          continue;
        }
        const int q_after = (iter == 0) ? -1 : min(ST, wk.n_tiles) - 1;   // tile after which the queries are requested
        if (q_after < 0) ok = load_q();
        for (int j = 0; j < wk.n_tiles && ok; ++j, ++kt) {
          const int st = kt % ST;
          const uint32_t par = ((kt / ST) & 1) ^ 1;  // first pass over the ring: slots start empty
          ok = wait(bar_k_empty(st), par);
          if (!ok) break;
          load_kv(sK + st * C::kTileBytes, false, wk.kv_begin + j, bar_k_full(st));
          ok = wait(bar_v_empty(st), par);
          if (!ok) break;
          load_kv(sV + st * C::kTileBytes, true, wk.kv_begin + j, bar_v_full(st));
          if (j == q_after) ok = load_q();
        }
      }
    }
   } else if (warp == 8) {
    // ------------------------------------------------------------------ MMA issuer (whole warp converged, one lane issues)
    {
      const uint32_t el = elect_one();
      // every lane waits for itself (each then holds the barrier's acquire for what it issues or skips), and the
      // warp agrees on the outcome so that it stays converged
      auto wait_all = [&](uint32_t bar, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag) ? 1 : 0) != 0;
      };
      bool ok = true;
      const uint32_t q_lo0 = desc_lo(sQ, 16), k_lo0 = desc_lo(sK, 16), v_lo0 = desc_lo(sV, C::kSubTile);
      auto issue_qk = [&](int s, int buf, int st) {
        // S = Q_s K^T : K dimension = D, 16 elements (32 bytes) per instruction inside the 128-byte swizzle row
        const uint32_t a_lo = q_lo0 + ((uint32_t)(s * C::kTileBytes) >> 4), b_lo = k_lo0 + ((uint32_t)(st * C::kTileBytes) >> 4);
        const uint32_t d = tm_S(buf);
        mma_ss<false>(d, a_lo, b_lo, kDescHi, C::kIdescQK, el);
#pragma unroll
        for (int ks = 1; ks < D / 16; ++ks) {
          constexpr int kSub16 = C::kSubTile >> 4;
          const uint32_t off = (uint32_t)((ks >> 2) * kSub16 + (ks & 3) * 2);
          mma_ss<true>(d, a_lo + off, b_lo + off, kDescHi, C::kIdescQK, el);
        }
      };
      // the same product with P as a K-major operand in shared memory (laid out like a query tile)
      auto issue_pv_ss = [&](int s, int st, bool accum) {
        const uint32_t a_lo = desc_lo(sP, 16) + ((uint32_t)(s * C::kPTileBytes) >> 4), b_lo = v_lo0 + ((uint32_t)(st * C::kTileBytes) >> 4);
        const uint32_t d = tm_O(s);
        mma_ss_rt(d, a_lo, b_lo, kDescHi, C::kIdescPV, accum ? 1u : 0u, el);
#pragma unroll
        for (int kk = 1; kk < kTile / 16; ++kk) {
          constexpr int kSub16 = C::kSubTile >> 4;
          mma_ss_rt(d, a_lo + (uint32_t)((kk >> 2) * kSub16 + (kk & 3) * 2), b_lo + kk * (2048 >> 4), kDescHi, C::kIdescPV, 1u, el);
        }
      };
      auto issue_pv = [&](int s, int buf, int st, bool accum) {
        // O_s += P V : K dimension = 128 keys, 16 keys (two 8-row groups) per instruction; V is MN-major
        const uint32_t b_lo = v_lo0 + ((uint32_t)(st * C::kTileBytes) >> 4);
        const uint32_t d = tm_O(s), a = tm_S(buf);
        mma_ts(d, a, b_lo, kDescHi, C::kIdescPV, accum ? 1u : 0u, el);
#pragma unroll
        for (int kk = 1; kk < kTile / 16; ++kk) mma_ts(d, a + kk * 8, b_lo + kk * (2048 >> 4), kDescHi, C::kIdescPV, 1u, el);
      };
      // Items are issued in order: Q K^T of the first NB items up front, then for each item its P V followed by the
      // Q K^T of item i + NB into the score buffer that P V has just consumed (the tensor pipe executes one thread's
      // instructions in issue order).  With three buffers the scores of a query tile's next key tile are ready before
      // its softmax warpgroup has finished the current one.
      int kt0 = 0;     // key tiles of the items this CTA has finished (ring position of the current item's tile 0)
      int it0 = 0;     // (key tile, query tile) items finished: score buffer (it0 + i) % NB for the current item's i
      int iter = 0;
      for (int work = blockIdx.x; work < p.total_work && ok; work += gridDim.x, ++iter) {
        const Work wk = decode(work);
        // gathered query tiles were written through the generic proxy and are read by the tensor core through the
        // async proxy: the reader fences after the wait
        ok = wait_all(bar_q, iter & 1);
        if (!ok) break;
        if (kGath) fence_proxy_async();
        if constexpr (C::kPSmem) {
          // Order on the tensor pipe: S(0) | S(1), O += P(0) V(0) | S(2), O += P(1) V(1) | ... with both query tiles
          // side by side in every group.  Score buffer s belongs to query tile s; it is free again as soon as the
          // softmax threads hold its values in registers, long before their P is ready, so S(j+1) never waits for
          // the product of tile j.  kt0 counts the key tiles of finished items, it0 the ring loads consumed.
          auto qk_pair = [&](int j) -> bool {
            const int st = it0 % ST, g = kt0 + j;
            if (!wait_all(bar_k_full(st), (it0 / ST) & 1)) return false;
            for (int sq = 0; sq < 2; ++sq) {
              if (g > 0 && !wait_all(bar_s_free(sq), (g - 1) & 1)) return false;
              tc_fence_after();
              issue_qk(sq, sq, st);
              tc_commit(bar_s_full(sq), el);
            }
            tc_commit(bar_k_empty(st), el);
            if (kQEarly && j == wk.n_tiles - 1) tc_commit(bar_q_free, el);   // the query tiles have been read for the last time
            ++it0;
            return true;
          };
          auto pv_pair = [&](int j) -> bool {
            const int st = it0 % ST, g = kt0 + j;
            if (!wait_all(bar_k_full(st), (it0 / ST) & 1)) return false;
            // the first product of an item overwrites the output accumulators: the previous item's epilogue must
            // have read them
            if (j == 0 && iter > 0 && !wait_all(bar_o_free, (iter - 1) & 1)) return false;
            for (int sq = 0; sq < 2; ++sq) {
              if (!wait_all(bar_p_full(sq), g & 1)) return false;
              tc_fence_after();
              issue_pv_ss(sq, st, j > 0);
              tc_commit(bar_pv_tile(sq), el);
            }
            tc_commit(bar_k_empty(st), el);
            ++it0;
            return true;
          };
          ok = qk_pair(0);
          for (int j = 0; j < wk.n_tiles && ok; ++j) {
            if (j + 1 < wk.n_tiles) ok = qk_pair(j + 1);
            if (ok) ok = pv_pair(j);
          }
          if (ok) tc_commit(bar_o_final, el);
          kt0 += wk.n_tiles;
          continue;
        }
        const int n_items = 2 * wk.n_tiles;
        int k_waited = 0, v_waited = 0;
        auto qk_item = [&](int it) -> bool {
          const int j = it >> 1, sq = it & 1, st = (kt0 + j) % ST, g = it0 + it;
          if (j >= k_waited) {
            if (!wait_all(bar_k_full(st), ((kt0 + j) / ST) & 1)) return false;
            k_waited = j + 1;
            tc_fence_after();
          }
          issue_qk(sq, g % NB, st);
          tc_commit(bar_s_full(g % NB), el);
          if (sq == 1) tc_commit(bar_k_empty(st), el);   // both query tiles have used this key tile
          if (kQEarly && it == n_items - 1) tc_commit(bar_q_free, el);   // the query tiles have been read for the last time
          return true;
        };
        for (int it = 0; it < NB && it < n_items && ok; ++it) ok = qk_item(it);
        for (int it = 0; it < n_items && ok; ++it) {
          const int j = it >> 1, sq = it & 1, st = (kt0 + j) % ST, g = it0 + it, buf = g % NB;
          if (j >= v_waited) {
            ok = wait_all(bar_v_full(st), ((kt0 + j) / ST) & 1);
            if (!ok) break;
            v_waited = j + 1;
          }
          ok = wait_all(bar_p_full(buf), (g / NB) & 1);
          if (!ok) break;
          if (it == 0 && iter > 0) {
            // the first product of an item overwrites the output accumulators: the previous item's epilogue must
            // have read them
            ok = wait_all(bar_o_free, (iter - 1) & 1);
            if (!ok) break;
          }
          tc_fence_after();
          issue_pv(sq, buf, st, j > 0);
          tc_commit(bar_pv_tile(sq), el);
          if (sq == 1) tc_commit(bar_v_empty(st), el);
          if (it + NB < n_items) ok = qk_item(it + NB);
        }
        if (ok) tc_commit(bar_o_final, el);
        kt0 += wk.n_tiles;
        it0 += n_items;
      }
    }
   }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    // ------------------------------------------------------------------ softmax warps: one thread per query row
    const int s = warp >> 2;                 // query tile of this warpgroup
    const int r = (warp & 3) * 32 + lane;    // row inside the tile == TMEM lane
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tO = tm_O(s) + lane_off;
    bool ok = true;
    int kt0 = 0, it0 = 0, iter = 0;   // the same running counters as in the issuing warp
    for (int work = blockIdx.x; work < p.total_work && ok; work += gridDim.x, ++iter) {
    const Work wk = decode(work);
    const int h = wk.h, b = wk.b, row0 = wk.row0, kv_begin = wk.kv_begin, n_tiles = wk.n_tiles, slot = wk.slot;
    float m_used = -INFINITY, l_run = 0.f;
    const int row_keys = VIS ? row_limit(row0 + s * kTile + r) : p.n;   // leading keys of the sequence this row sees
    // 32 packed bf16 pairs of this row's P, part c of four: over the scores in TMEM, or into the row's place in the
    // shared-memory P tile (the swizzled layout of a K-major operand)
    const uint32_t p_row = sP + (uint32_t)(s * C::kPTileBytes + r * 128);
    auto store_p16 = [&](uint32_t tS, int c, const uint32_t* v) {
      if constexpr (C::kPSmem) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int c16 = c * 4 + q;   // 16-byte chunk of the row: 64-key block c16 / 8, chunk c16 % 8
          st_shared_16(p_row + (uint32_t)((c16 >> 3) * C::kSubTile + (((c16 & 7) ^ (r & 7)) << 4)), v[4 * q], v[4 * q + 1],
                       v[4 * q + 2], v[4 * q + 3]);
        }
      } else {
        tmem_st16(tS + c * 16, v);
      }
    };
    for (int j = 0; j < n_tiles; ++j) {
      // P in shared memory: tile s owns score buffer s and phases count key tiles; otherwise items share NB buffers
      const int item = C::kPSmem ? kt0 + j : it0 + 2 * j + s, buf = C::kPSmem ? s : item % NB;
      const uint32_t s_par = C::kPSmem ? (item & 1) : ((item / NB) & 1);
      const uint32_t tS = tm_S(buf) + lane_off;
      ok = mbar_wait(bar_s_full(buf), s_par, abort_flag);
      if (!ok) break;
      tc_fence_after();
      float sv[kTile];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, *reinterpret_cast<float(*)[32]>(&sv[c * 32]));
      tmem_ld_wait();
      if constexpr (C::kPSmem) {
        tc_fence_before();
        mbar_arrive(bar_s_free(s));   // the scores are in registers: the next key tile's may be written
      }
      const int valid = row_keys - (kv_begin + j) * kTile;  // keys of this tile that this row sees (<= 0: none)
      auto mask_tail = [&]() {
        if (valid < kTile) {
#pragma unroll
          for (int c = 0; c < kTile; ++c)
            if (c >= valid) sv[c] = -INFINITY;
        }
      };
      mask_tail();
      if (j == 0) {
        // the first tile fixes the reference maximum of the row (tree of independent partial maxima)
        float m8[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) m8[i] = sv[i];
#pragma unroll
        for (int c = 8; c < kTile; c += 8) {
#pragma unroll
          for (int i = 0; i < 8; ++i) m8[i] = fmaxf(m8[i], sv[c + i]);
        }
        m_used = fmaxf(fmaxf(fmaxf(m8[0], m8[1]), fmaxf(m8[2], m8[3])), fmaxf(fmaxf(m8[4], m8[5]), fmaxf(m8[6], m8[7]))) *
                 p.scale_log2;
      }
      // One pass: exponentials against the current reference maximum, with the row's own maximum tracked on the
      // side.  Only if some row of the warp outgrew its reference by more than the threshold (rare after the first
      // tiles) is the reference raised, O rescaled and the pass repeated; the result is exact either way.
      // packed fp32 pairs halve the FMA-pipe instruction count; growth of the row maximum shows up in the tile's sum
      // (an exponent above the threshold pushes the sum beyond 2^threshold), so no per-element maximum is kept
      const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), negm2 = pack2(-m_used, -m_used);
      uint64_t acc2[4] = {0ull, 0ull, 0ull, 0ull};
      // P over the scores in TMEM: all 64 packed results first, the four stores after (the exp2 unit then sees one
      // uninterrupted stream of 128 instructions per thread instead of four short ones with their fill and drain)
      uint32_t pk[64];
      if constexpr (C::kPSmem) {
        // the P tile is free once the previous product of this query tile has read it (usually long ago), and,
        // where the previous item's output was staged in it, once every thread of the tile has sent its rows
        if (item > 0) {
          ok = mbar_wait(bar_pv_tile(s), (item - 1) & 1, abort_flag);
          if (!ok) break;
        }
        if (kStageP && j == 0 && iter > 0) {
          ok = mbar_wait(bar_stage_free(s), (iter - 1) & 1, abort_flag);
          if (!ok) break;
        }
      }
#pragma unroll
      for (int i = 0; i < 64; ++i) {
        const uint64_t x2 = fma2(pack2(sv[2 * i], sv[2 * i + 1]), scale2, negm2);
        float p0, p1;
        if ((i & 7) < C::kPolyOf8) {
          exp2_poly2(x2, p0, p1);
        } else {
          float t0, t1;
          unpack2(x2, t0, t1);
          p0 = ex2(t0);
          p1 = ex2(t1);
        }
        acc2[i & 3] = add2(acc2[i & 3], pack2(p0, p1));
        pk[i] = pack_bf16x2(p0, p1);
        // shared-memory stores drain while the exponentials go on; the TMEM stores of the other variant wait until
        // all 128 exponentials have been issued
        if constexpr (C::kPSmem) {
          if ((i & 15) == 15) store_p16(tS, i >> 4, &pk[i - 15]);
        }
      }
      float sum;
      {
        float a0, a1;
        unpack2(add2(add2(acc2[0], acc2[1]), add2(acc2[2], acc2[3])), a0, a1);
        sum = a0 + a1;
      }
      const bool grew = !(sum <= 256.f * 128.f);  // some exponent above 2^8 (or 128 of them near it); also catches inf, NaN
      const bool redo = __any_sync(0xffffffffu, grew);
      if constexpr (!C::kPSmem) {
        // P goes over the scores in TMEM only now that the pass is known to stand: the rare redo below reads the
        // scores again from there, so that they need not stay in registers beside the packed results
        if (!redo) {
#pragma unroll
          for (int c = 0; c < 4; ++c) store_p16(tS, c, &pk[c * 16]);
        }
      }
      if (redo) {
        if constexpr (!C::kPSmem) {
#pragma unroll
          for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, *reinterpret_cast<float(*)[32]>(&sv[c * 32]));
          tmem_ld_wait();
          mask_tail();
        }
        // rare: the row's true maximum relative to the reference
        float mraw = sv[0];
#pragma unroll
        for (int c = 1; c < kTile; ++c) mraw = fmaxf(mraw, sv[c]);
        const float t_max = fmaf(mraw, p.scale_log2, -m_used);
        const float delta = fmaxf(t_max, 0.f);
        const float f = ex2(-delta);
        m_used += delta;
        l_run *= f;
        tmem_st_wait();
        // the accumulator must hold every product issued against the old reference before it is rescaled (with three
        // score buffers the previous P V of this tile may still be waiting behind a Q K^T)
        if (j > 0) {
          ok = mbar_wait(bar_pv_tile(s), (kt0 + j - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
        }
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          float ov[32];
          tmem_ld32(tO + c * 32, ov);
          tmem_ld_wait();
          uint32_t ou[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) ou[i] = __float_as_uint(ov[i] * f);
          tmem_st32(tO + c * 32, ou);
        }
        sum = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float p0 = ex2(fmaf(sv[c * 32 + 2 * i], p.scale_log2, -m_used));
            const float p1 = ex2(fmaf(sv[c * 32 + 2 * i + 1], p.scale_log2, -m_used));
            sum += p0 + p1;
            pk[i] = pack_bf16x2(p0, p1);
          }
          store_p16(tS, c, pk);
        }
      }
      l_run += sum;
      tmem_st_wait();
      tc_fence_before();
      if constexpr (C::kPSmem) fence_proxy_async();   // P was written through the generic proxy; the tensor core reads it through the async one
      mbar_arrive(bar_p_full(buf));
    }
    // epilogue
    if (ok) ok = mbar_wait(bar_o_final, iter & 1, abort_flag);
    if (slot >= 0) {
      // a piece of a split item: unnormalised O, reference max and sum go to scratch; the combine kernel finishes
      if (ok) {
        tc_fence_after();
        float* dst = p.partial + (((size_t)slot * 2 + s) * kTile + r) * (D + 4);
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          float ov[32];
          tmem_ld32(tO + c * 32, ov);
          tmem_ld_wait();
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4)
            *reinterpret_cast<float4*>(dst + c * 32 + q4 * 4) = make_float4(ov[q4 * 4], ov[q4 * 4 + 1], ov[q4 * 4 + 2], ov[q4 * 4 + 3]);
        }
        dst[D] = m_used;
        dst[D + 1] = l_run;
        tc_fence_before();
        mbar_arrive(bar_o_free);          // the accumulator row has been read
        // nothing was staged (the barriers' phases still count items)
        if (kStageP) {
          mbar_arrive(bar_stage_free(s));
        } else if (C::kStageOwn) {
          if (MODE == kDirect && (warp & 3) == 0 && lane == 0) mbar_arrive(bar_stage_free(s));
        } else if (MODE != kDirect || ((warp & 3) == 0 && lane == 0)) {
          mbar_arrive(bar_q_free);
        }
      }
    } else {
    // O / l -> bf16 -> swizzled staging tile -> TMA store; rows beyond n are clipped
    if (ok && MODE == kDirect && C::kStageOwn && iter > 0) ok = mbar_wait(bar_stage_free(s), (iter - 1) & 1, abort_flag);
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / l_run;
      unsigned char* stage = base_ptr + (sStage - base) + s * kStageStride;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        float ov[32];
        tmem_ld32(tO + c * 32, ov);
        tmem_ld_wait();
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint4 w;
          w.x = pack_bf16x2(ov[q4 * 8 + 0] * inv, ov[q4 * 8 + 1] * inv);
          w.y = pack_bf16x2(ov[q4 * 8 + 2] * inv, ov[q4 * 8 + 3] * inv);
          w.z = pack_bf16x2(ov[q4 * 8 + 4] * inv, ov[q4 * 8 + 5] * inv);
          w.w = pack_bf16x2(ov[q4 * 8 + 6] * inv, ov[q4 * 8 + 7] * inv);
          const int col = c * 32 + q4 * 8;          // first of 8 output columns
          const int db = col >> 6, chunk = (col & 63) >> 3;
          *reinterpret_cast<uint4*>(stage + db * C::kSubTile + r * 128 + ((chunk ^ (r & 7)) << 4)) = w;
        }
      }
      const int row = row0 + s * kTile + r;
      if (p.lse && row < p.n && row >= p.lse_row0 && row < p.lse_row0 + p.lse_rows)
        p.lse[((int64_t)b * p.N_h + h) * p.lse_rows + (row - p.lse_row0)] = (m_used + log2f(l_run)) * 0.6931471805599453f;
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(bar_o_free);            // the accumulator row has been read
    }
    if (MODE != kDirect) {
      // Eq. 7's scatter: every staged row goes to the place pack_map names in the full tensor.  The warps of the
      // tile write the rows with 16-byte stores, a row (or two) per instruction, so each row leaves as one
      // contiguous segment; thread r looks up row r's destination and the others get it by shuffle.  (One-row TMA
      // stores, 512 per item, took the copy engine longer than these 16 or 32 store instructions per thread.)
      const int prow = row0 + s * kTile + r;
      int my_orow = -1;
      if (ok && prow < p.n) {
        my_orow = p.pack_map[(int64_t)b * p.n + prow];
        if (my_orow < 0 || my_orow >= p.n_full) {
          atomicOr(p.status, ST_BAD_MAP);
          my_orow = -1;
        }
      }
      asm volatile("bar.sync %0, 128;" ::"r"(1 + s) : "memory");  // every row of this query tile has been staged
      {
        constexpr int CPR = D / 8;         // 16-byte chunks per row
        constexpr int RPI = 32 / CPR;      // rows per warp instruction
        const int cc = lane % CPR, sub = lane / CPR;
        const unsigned char* stage = base_ptr + (sStage - base) + s * kStageStride + (cc >> 3) * C::kSubTile;
        __nv_bfloat16* dst = p.out_full + ((int64_t)b * p.n_full * p.N_h + h) * D + cc * 8;
        const int64_t row_stride = (int64_t)p.N_h * D;
#pragma unroll 4
        for (int it = 0; it < 32 / RPI; ++it) {
          const int rl = it * RPI + sub;                    // row among this warp's 32
          const int orow = __shfl_sync(0xffffffffu, my_orow, rl);
          const int rr = (warp & 3) * 32 + rl;
          if (orow >= 0)
            *reinterpret_cast<uint4*>(dst + orow * row_stride) =
                *reinterpret_cast<const uint4*>(stage + rr * 128 + (((cc & 7) ^ (rr & 7)) << 4));
        }
      }
      // this thread has read what it sends from the staged tile
      if (ok) {
        if (kStageP) mbar_arrive(bar_stage_free(s));
        else if (!C::kStageOwn) mbar_arrive(bar_q_free);
      }
    } else {
      asm volatile("bar.sync %0, 128;" ::"r"(1 + s) : "memory");  // the four warps of this query tile
      if (ok && (warp & 3) == 0 && lane == 0) {
        if (row0 + s * kTile < p.n) {
          for (int db = 0; db < C::DB; ++db)
            tma_store_4d(&map_o, sStage + s * kStageStride + db * C::kSubTile, db * 64, row0 + s * kTile, h, b);
          tma_store_commit_wait();
        }
        mbar_arrive(C::kStageOwn ? bar_stage_free(s) : bar_q_free);   // this tile's staging has been read (or was never sent)
      }
    }
    }
    kt0 += n_tiles;
    it0 += 2 * n_tiles;
    }   // work items of this CTA
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, ST_TIMEOUT);
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// Merges the pieces of the split items: out = sum_i 2^(m_i - m) O_i / sum_i 2^(m_i - m) l_i, one warp per query row.
struct CombineParams {
  const float* partial;
  const int32_t* pack_map;  // scatter mode: out is the full tensor and row goes to pack_map[b, row]; nullptr otherwise
  int n_full;
  int* status;
  __nv_bfloat16* out;
  float* lse;
  int lse_row0, lse_rows;
  int n, N_h, D, pairs, n_whole, splits, n_split_items;
};

template <int D>
__global__ void __launch_bounds__(256) attn_combine_kernel(const CombineParams p) {
  constexpr int CPL = D / 32;  // output columns per lane
  const int lane = threadIdx.x & 31;
  const int row_id = blockIdx.x * 8 + (threadIdx.x >> 5);  // (split item, tile, row)
  if (row_id >= p.n_split_items * 2 * kTile) return;
  const int si = row_id / (2 * kTile), tr = row_id % (2 * kTile);
  const int item = p.n_whole + si;
  const int pair = item % p.pairs, h = (item / p.pairs) % p.N_h, b = item / (p.pairs * p.N_h);
  const int row = pair * 2 * kTile + tr;
  if (row >= p.n) return;
  constexpr int stride = D + 4;
  const float* base = p.partial + ((size_t)si * p.splits * 2 * kTile + tr) * stride;  // piece 0 of this row
  const size_t piece = (size_t)2 * kTile * stride;
  // lane i holds piece i's reference maximum and sum (at most 16 pieces)
  const float mi = (lane < p.splits) ? base[lane * piece + D] : -INFINITY;
  const float li = (lane < p.splits) ? base[lane * piece + D + 1] : 0.f;
  float m = mi;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  const float wi = (lane < p.splits) ? exp2f(mi - m) : 0.f;
  float l = wi * li;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  // all pieces' values are loaded before they are used, so the loads overlap
  float v[16][CPL];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
#pragma unroll
    for (int c = 0; c < CPL; ++c) v[i][c] = (i < p.splits) ? base[i * piece + lane * CPL + c] : 0.f;
  }
  float acc[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float w = __shfl_sync(0xffffffffu, wi, i);
#pragma unroll
    for (int c = 0; c < CPL; ++c) acc[c] += w * v[i][c];
  }
  const float inv = 1.f / l;
  int64_t out_row = (int64_t)b * p.n + row;
  if (p.pack_map) {
    const int orow = p.pack_map[(int64_t)b * p.n + row];
    if (orow < 0 || orow >= p.n_full) {
      if (lane == 0) atomicOr(p.status, ST_BAD_MAP);
      return;
    }
    out_row = (int64_t)b * p.n_full + orow;
  }
  __nv_bfloat16* o = p.out + (out_row * p.N_h + h) * D + lane * CPL;
#pragma unroll
  for (int c = 0; c < CPL; c += 2)
    *reinterpret_cast<__nv_bfloat162*>(o + c) = __floats2bfloat162_rn(acc[c] * inv, acc[c + 1] * inv);
  if (p.lse && lane == 0 && row >= p.lse_row0 && row < p.lse_row0 + p.lse_rows)
    p.lse[((int64_t)b * p.N_h + h) * p.lse_rows + (row - p.lse_row0)] = (m + log2f(l)) * 0.6931471805599453f;
}

// ---------------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------------
// [B * n, N_h * D] bf16 viewed as a 2-D tensor (column, row) for row gathers: box = 64 columns x 1 row (a gather
// instruction names four rows), 128-byte swizzle; rows past the end read as zeros
bool make_row_map(CUtensorMap* map, const void* ptr, long long rows, int cols) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64, 1};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// kGather: a.q and a.out are the full [B, n_full, N_h, D] tensors and pack_map [B, a.n] names the row of them that
// each attended row stands for.
template <int D, int MODE, bool VIS>
cudaError_t launch_tc_v(const AttnArgs& a, const int32_t* pack_map, int n_full, int* status, float* partial,
                        size_t partial_bytes, cudaStream_t st, int* launches) {
  CUtensorMap mq, mk, mv, mo;
  if (MODE == kGatherKV) {
    // a.k and a.v are the full tensors too
    const long long rows = (long long)a.B * n_full;
    if (rows >= 0x7fffffffll) return cudaErrorInvalidConfiguration;
    if (!make_row_map(&mk, a.k, rows, a.N_kv * D) || !make_row_map(&mv, a.v, rows, a.N_kv * D)) return cudaErrorInvalidValue;
  } else if (!make_map(&mk, a.k, a.B, a.n, a.N_kv, D) || !make_map(&mv, a.v, a.B, a.n, a.N_kv, D)) {
    return cudaErrorInvalidValue;
  }
  // The gather modes neither load Q nor store the output through tensor maps (gathering warps and plain stores do):
  // in kGather mode the two slots carry the maps of the full K and V for the leading key tiles that are read from there.
  const bool direct_kv = MODE == kGather && a.direct_rows >= kTile && a.k_full && a.v_full;
  if (MODE != kDirect) {
    mq = mk;
    mo = mv;
    if (direct_kv && (!make_map(&mq, a.k_full, a.B, n_full, a.N_kv, D) || !make_map(&mo, a.v_full, a.B, n_full, a.N_kv, D)))
      return cudaErrorInvalidValue;
  } else if (!make_map(&mo, a.out, a.B, a.n, a.N_h, D) || !make_map(&mq, a.q, a.B, a.n, a.N_h, D)) {
    return cudaErrorInvalidValue;
  }
  cudaError_t e = cudaFuncSetAttribute(attn_bf16_tc_kernel<D, MODE, VIS>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<D>::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int pairs = (a.n + 2 * kTile - 1) / (2 * kTile);
  const int items = pairs * a.N_h * a.B;
  const int n_tiles = (a.n + kTile - 1) / kTile;
  const int sms = sm_count();
  // one CTA per SM: the items beyond the last full wave are cut over the keys into pieces that fill the idle SMs
  int rem = items % sms, splits = 0, per = n_tiles;
  if (items > sms && rem > 0 && rem <= sms / 2 && n_tiles >= 4 && a.full_visibility()) {
    int want = sms / rem;
    if (want > 16) want = 16;
    if (want > n_tiles / 2) want = n_tiles / 2;
    per = (n_tiles + want - 1) / want;
    splits = (n_tiles + per - 1) / per;
    const size_t need = (size_t)rem * splits * 2 * kTile * (D + 4) * sizeof(float);
    if (splits < 2 || !partial || need > partial_bytes) { splits = 0; per = n_tiles; }
  }
  const int n_whole = splits ? items - rem : items;
  TcParams p{
      a.lse, status, partial, pack_map, n_full, a.B * n_full, (const __nv_bfloat16*)a.q, (__nv_bfloat16*)a.out, a.lse_row0, a.lse_rows, a.n, a.N_h, a.N_h / a.N_kv, pairs, n_whole + (splits ? rem * splits : 0), n_whole, splits, per,
      a.scale * kLog2e, a.obs_end, a.fut_end, a.lim[0], a.lim[1], a.lim[2]};
  if (MODE == kGather) p.direct_tiles = direct_kv ? a.direct_rows / kTile : 0;
  const int grid = p.total_work < sms ? p.total_work : sms;   // one CTA per SM; each walks through its share of the work
  ++*launches;
  attn_bf16_tc_kernel<D, MODE, VIS><<<grid, kThreadsTc, TcCfg<D>::kSmemBytes, st>>>(mq, mk, mv, mo, p);
  e = cudaGetLastError();
  if (e != cudaSuccess || !splits) return e;
  CombineParams c{partial, MODE != kDirect ? pack_map : nullptr, n_full, status, (__nv_bfloat16*)a.out, a.lse, a.lse_row0, a.lse_rows,
                  a.n, a.N_h, D, pairs, n_whole, splits, rem};
  ++*launches;
  attn_combine_kernel<D><<<(rem * 2 * kTile + 7) / 8, 256, 0, st>>>(c);
  return cudaGetLastError();
}

template <int D, int MODE>
cudaError_t launch_tc_d(const AttnArgs& a, const int32_t* pack_map, int n_full, int* status, float* partial,
                        size_t partial_bytes, cudaStream_t st, int* launches) {
  return a.full_visibility() ? launch_tc_v<D, MODE, false>(a, pack_map, n_full, status, partial, partial_bytes, st, launches)
                             : launch_tc_v<D, MODE, true>(a, pack_map, n_full, status, partial, partial_bytes, st, launches);
}

}  // namespace

size_t attn_tc_scratch_bytes(int D) {
  // room for one piece per SM (the split pieces never outnumber the SMs); 160 covers the SM count of this part
  return (size_t)160 * 2 * kTile * (D + 4) * sizeof(float);
}

cudaError_t launch_attn_bf16_tc(const AttnArgs& a, int* status, void* scratch, size_t scratch_bytes, cudaStream_t st,
                                int* launches) {
  switch (a.D) {
    case 64: return launch_tc_d<64, kDirect>(a, nullptr, a.n, status, (float*)scratch, scratch_bytes, st, launches);
    case 128: return launch_tc_d<128, kDirect>(a, nullptr, a.n, status, (float*)scratch, scratch_bytes, st, launches);
    default: return cudaErrorInvalidConfiguration;
  }
}

cudaError_t launch_attn_bf16_tc_gather(const AttnArgs& a, const int32_t* pack_map, int n_full, bool gather_kv, int* status,
                                       void* scratch, size_t scratch_bytes, cudaStream_t st, int* launches) {
  if (gather_kv) {
    switch (a.D) {
      case 64: return launch_tc_d<64, kGatherKV>(a, pack_map, n_full, status, (float*)scratch, scratch_bytes, st, launches);
      case 128: return launch_tc_d<128, kGatherKV>(a, pack_map, n_full, status, (float*)scratch, scratch_bytes, st, launches);
      default: return cudaErrorInvalidConfiguration;
    }
  }
  switch (a.D) {
    case 64: return launch_tc_d<64, kGather>(a, pack_map, n_full, status, (float*)scratch, scratch_bytes, st, launches);
    case 128: return launch_tc_d<128, kGather>(a, pack_map, n_full, status, (float*)scratch, scratch_bytes, st, launches);
    default: return cudaErrorInvalidConfiguration;
  }
}

}  // namespace swam
