// Packing (Sec. 4.2) and scatter / cached-prediction blend (Eq. 7): row copies by index.
//
// Rows are N_h*D elements (256 B .. 16 KB), contiguous and 16-byte aligned, so pack and the in-place scatter are
// pure HBM streams.  They run on the bulk-copy engine: one thread per warp moves row segments global -> shared ->
// global with cp.async.bulk through a private ring of shared-memory buffers, so no data passes through registers
// and each SM keeps 128 KB of copies in flight.  The 32 lanes of the warp fetch and validate the next 32 map
// entries at once.  Waits on the load barriers are bounded; an out-of-range map entry is skipped and flagged.
// The blend into a separate output buffer (out != cached) reads every row of the full sequence and uses plain
// 16-byte loads and stores.
#include "swam_internal.cuh"

namespace swam {
namespace {

constexpr int kWarps = 8;
constexpr int kStages = 4;
constexpr int kSegMax = 4096;  // bytes per ring buffer
constexpr unsigned long long kWaitCycles = 4000000000ull;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

struct RowCopyParams {
  const unsigned char* src[3];
  unsigned char* dst[3];
  const int32_t* src_idx;  // [B, n_rows] row of src for each listed row, or nullptr (identity)
  const int32_t* dst_idx;  // [B, n_rows] row of dst for each listed row, or nullptr (identity)
  int* status;
  int n_tensors;
  int n_rows;       // listed rows per sample that this launch copies: first_row .. first_row + n_rows - 1
  int first_row;    // first listed row copied
  int idx_rows;     // listed rows per sample in the maps (their stride from sample to sample)
  int src_rows;     // rows per sample in src
  int dst_rows;     // rows per sample in dst
  int row_bytes;
  int seg_bytes;    // row_bytes / segs, <= kSegMax, multiple of 16
  int segs;         // segments per row
  long long units;  // n_tensors * B * n_rows * segs
};

// unit id -> (tensor, sample * n_rows + listed row, segment); units of one row are adjacent
__global__ void __launch_bounds__(kWarps * 32, 1) row_copy_bulk_kernel(const RowCopyParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long bars[kWarps * kStages];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned char* ring = smem + (size_t)warp * kStages * kSegMax;
  const uint32_t ring_a = smem_addr(ring);
  const uint32_t bar0 = smem_addr(&bars[warp * kStages]);
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8 * s) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();

  const long long n_warps = (long long)gridDim.x * kWarps;
  const long long gw = (long long)blockIdx.x * kWarps + warp;
  // this warp's units: gw, gw + n_warps, ...; processed in batches of 32 (one map look-up per lane)
  const long long my_units = (p.units > gw) ? (p.units - gw + n_warps - 1) / n_warps : 0;
  const long long rows_per_tensor = p.units / p.n_tensors / p.segs;

  long long issued = 0, stored = 0;  // lane 0's counters over valid units
  bool ok = true;
  // lane 0 keeps up to kStages - 1 loads in flight; src/dst offsets of issued-but-not-stored units
  long long pend_dst[kStages] = {};
  int pend_z[kStages] = {};

  auto retire_one = [&]() {  // wait for the oldest load, send it out, free one ring slot
    const int st = (int)(stored % kStages);
    if (!mbar_wait_bounded(bar0 + 8 * st, (uint32_t)((stored / kStages) & 1), kWaitCycles, nullptr)) { ok = false; return; }
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(p.dst[pend_z[st]] + pend_dst[st]), "r"(ring_a + st * kSegMax), "r"(p.seg_bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    ++stored;
  };

  for (long long b0 = 0; b0 < my_units && ok; b0 += 32) {
    // every lane resolves one unit of the batch
    const long long u = gw + (b0 + lane) * n_warps;
    long long s_off = -1, d_off = -1;
    int z = 0;
    if (b0 + lane < my_units) {
      const long long row_id = u / p.segs;            // tensor-major: z * rows_per_tensor + (b * n_rows + r)
      const int seg = (int)(u - row_id * p.segs);
      z = (int)(row_id / rows_per_tensor);
      const long long br = row_id - (long long)z * rows_per_tensor;
      const long long b = br / p.n_rows;
      const long long lr = p.first_row + (br - b * p.n_rows);
      long long srow = lr, drow = lr;
      bool valid = true;
      if (p.src_idx) { srow = p.src_idx[b * p.idx_rows + lr]; valid = srow >= 0 && srow < p.src_rows; }
      if (p.dst_idx) { drow = p.dst_idx[b * p.idx_rows + lr]; valid = valid && drow >= 0 && drow < p.dst_rows; }
      if (valid) {
        s_off = (b * p.src_rows + srow) * (long long)p.row_bytes + (long long)seg * p.seg_bytes;
        d_off = (b * p.dst_rows + drow) * (long long)p.row_bytes + (long long)seg * p.seg_bytes;
      } else if (seg == 0) {
        atomicOr(p.status, ST_BAD_MAP);
      }
    }
    const int in_batch = (int)((my_units - b0 < 32) ? (my_units - b0) : 32);
    for (int i = 0; i < in_batch; ++i) {
      const long long src_o = __shfl_sync(0xffffffffu, s_off, i);
      const long long dst_o = __shfl_sync(0xffffffffu, d_off, i);
      const int zz = __shfl_sync(0xffffffffu, z, i);
      if (lane == 0 && ok && src_o >= 0) {
        if (issued - stored == kStages - 1) retire_one();
        if (ok) {
          const int st = (int)(issued % kStages);
          // the store that last read this slot (unit issued - kStages) must have finished reading it
          asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          const uint32_t bar = bar0 + 8 * st;
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(p.seg_bytes) : "memory");
          asm volatile(
              "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
              ::"r"(ring_a + st * kSegMax), "l"(p.src[zz] + src_o), "r"(p.seg_bytes), "r"(bar) : "memory");
          pend_dst[st] = dst_o;
          pend_z[st] = zz;
          ++issued;
        }
      }
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
  }
  if (lane == 0) {
    while (ok && stored < issued) retire_one();
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (!ok) atomicOr(p.status, ST_TIMEOUT);
  }
}

// ---- blend into a separate buffer: out[b,t] = inv[b,t] >= 0 ? out_p[b, inv[b,t]] : cached[b,t] -----------------
constexpr int kBlendThreads = 256;

struct BlendParams {
  const uint4* out_p;
  const uint4* cached;
  uint4* out;
  const int32_t* inv_map;  // [B, L]
  int* status;
  int L, Lp, chunks;
  long long rows;  // B * L
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// one warp per row, lanes stride over the row's 16-byte chunks, four chunks in flight per lane
__global__ void __launch_bounds__(kBlendThreads) blend_kernel(const BlendParams p) {
  const int lane = threadIdx.x & 31;
  const long long warps = (long long)gridDim.x * (kBlendThreads / 32);
  for (long long row = (long long)blockIdx.x * (kBlendThreads / 32) + (threadIdx.x >> 5); row < p.rows; row += warps) {
    const long long b = row / p.L;
    const int pr = p.inv_map[row];
    if (pr >= p.Lp) {
      if (lane == 0) atomicOr(p.status, ST_BAD_MAP);
      continue;
    }
    const uint4* src = (pr >= 0) ? p.out_p + (b * p.Lp + pr) * p.chunks : p.cached + row * p.chunks;
    uint4* dst = p.out + row * p.chunks;
    for (int c0 = lane; c0 < p.chunks; c0 += 128) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c0 + 32 * u < p.chunks) v[u] = ld_stream(src + c0 + 32 * u);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c0 + 32 * u < p.chunks) dst[c0 + 32 * u] = v[u];
    }
  }
}

cudaError_t launch_row_copy(RowCopyParams& p, int batch, cudaStream_t st) {
  int segs = 1;
  while (p.row_bytes / segs > kSegMax || (p.row_bytes % (segs * 16)) != 0) {
    segs *= 2;
    if (segs > 64) return cudaErrorInvalidConfiguration;
  }
  p.segs = segs;
  p.seg_bytes = p.row_bytes / segs;
  p.units = (long long)p.n_tensors * batch * p.n_rows * segs;
  if (p.units == 0) return cudaSuccess;
  const size_t smem = (size_t)kWarps * kStages * kSegMax;
  // the opt-in is per device, and a process may hold contexts on several: set it on every launch
  cudaError_t e = cudaFuncSetAttribute(row_copy_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  long long ctas = (p.units + kWarps * 4 - 1) / (kWarps * 4);  // at least four units per warp
  const int sms = sm_count();
  if (ctas > sms) ctas = sms;
  if (ctas < 1) ctas = 1;
  row_copy_bulk_kernel<<<(int)ctas, kWarps * 32, smem, st>>>(p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_pack(const Dims& d, const void* const src[3], void* const dst[3], const int32_t* pack_map,
                        int* status, cudaStream_t st, int* launches, int first_row) {
  if (d.Lp - first_row <= 0) return cudaSuccess;
  const int eb = d.dtype == 0 ? 4 : 2;
  // tensors with the same row size share a launch: Q has N_h heads per row, K and V have N_kv
  const int rows_of[3] = {d.N_h * d.D * eb, d.N_kv * d.D * eb, d.N_kv * d.D * eb};
  bool done[3] = {false, false, false};
  for (int first = 0; first < 3; ++first) {
    if (done[first] || !src[first] || !dst[first]) continue;
    RowCopyParams p{};
    int n = 0;
    for (int i = first; i < 3; ++i)
      if (!done[i] && src[i] && dst[i] && rows_of[i] == rows_of[first]) {
        p.src[n] = (const unsigned char*)src[i];
        p.dst[n] = (unsigned char*)dst[i];
        ++n;
        done[i] = true;
      }
    p.src_idx = pack_map; p.dst_idx = nullptr; p.status = status;
    p.n_tensors = n; p.n_rows = d.Lp - first_row; p.first_row = first_row; p.idx_rows = d.Lp;
    p.src_rows = d.L; p.dst_rows = d.Lp;
    p.row_bytes = rows_of[first];
    ++*launches;
    cudaError_t e = launch_row_copy(p, d.B, st);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Sparse input transfer of a reuse step (Sec. 4.2: only the retained tokens are processed): the rows pack_map names
// travel from full tensors in pinned, device-mapped HOST memory to the same rows of full tensors in device memory;
// every other row of the destination keeps what it held and is never read by the sparse step.  The loads cross PCIe
// (one warp per row, eight 16-byte loads per lane in flight), so the kernel is the copy: it runs on the copy-in stream.
struct HostRowsParams {
  const uint4* src[3];
  uint4* dst[3];
  const int32_t* idx;   // [B, n_idx] rows to bring
  int* status;
  int n_tensors, n_idx, rows, chunks;   // rows per sample of the full tensors, 16-byte chunks per row
  int first, count;                     // listed rows first .. first + count - 1 of every sample are brought
  long long total;                      // B * count
};

__global__ void __launch_bounds__(256) host_rows_kernel(const HostRowsParams p) {
  const int lane = threadIdx.x & 31;
  const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long it = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; it < p.total; it += n_warps) {
    const long long b = it / p.count;
    const int row = p.idx[b * p.n_idx + p.first + (it - b * p.count)];
    if (row < 0 || row >= p.rows) {
      if (lane == 0) atomicOr(p.status, ST_BAD_MAP);
      continue;
    }
    const long long off = (b * p.rows + row) * p.chunks;
    for (int t = 0; t < p.n_tensors; ++t) {
      const uint4* s = p.src[t] + off;
      uint4* d = p.dst[t] + off;
      for (int c0 = lane; c0 < p.chunks; c0 += 32 * 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (c0 + 32 * u < p.chunks) v[u] = __ldcs(s + c0 + 32 * u);
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (c0 + 32 * u < p.chunks) d[c0 + 32 * u] = v[u];
      }
    }
  }
}

cudaError_t launch_host_rows(const Dims& d, const void* const src[3], void* const dst[3], const int32_t* pack_map,
                             int* status, cudaStream_t st, int* launches, int first_row) {
  if (d.Lp - first_row <= 0) return cudaSuccess;
  const int eb = d.dtype == 0 ? 4 : 2;
  const int rows_of[3] = {d.N_h * d.D * eb, d.N_kv * d.D * eb, d.N_kv * d.D * eb};
  bool done[3] = {false, false, false};
  for (int first = 0; first < 3; ++first) {
    if (done[first]) continue;
    HostRowsParams p{};
    int n = 0;
    for (int i = first; i < 3; ++i)
      if (!done[i] && rows_of[i] == rows_of[first]) {
        p.src[n] = (const uint4*)src[i];
        p.dst[n] = (uint4*)dst[i];
        ++n;
        done[i] = true;
      }
    p.idx = pack_map; p.status = status;
    p.n_tensors = n; p.n_idx = d.Lp; p.rows = d.L; p.chunks = rows_of[first] / 16;
    p.first = first_row; p.count = d.Lp - first_row;
    p.total = (long long)d.B * p.count;
    ++*launches;
    const long long need = (p.total + 7) / 8;
    const long long cap = (long long)sm_count() * 8;
    host_rows_kernel<<<(int)(need < cap ? need : cap), 256, 0, st>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_scatter(const Dims& d, const void* out_p, const int32_t* pack_map, const int32_t* inv_map,
                           const void* cached, void* out, int* status, cudaStream_t st, int* launches) {
  const int row_bytes = d.N_h * d.D * (d.dtype == 0 ? 4 : 2);
  if (d.Lp == 0) return cudaSuccess;
  if (cached == out) {
    RowCopyParams p{};
    p.src[0] = (const unsigned char*)out_p; p.dst[0] = (unsigned char*)out;
    p.src_idx = nullptr; p.dst_idx = pack_map; p.status = status;
    p.n_tensors = 1; p.n_rows = d.Lp; p.first_row = 0; p.idx_rows = d.Lp; p.src_rows = d.Lp; p.dst_rows = d.L;
    p.row_bytes = row_bytes;
    ++*launches;
    return launch_row_copy(p, d.B, st);
  }
  BlendParams p{(const uint4*)out_p, (const uint4*)cached, (uint4*)out, inv_map, status, d.L, d.Lp, row_bytes / 16,
                (long long)d.B * d.L};
  ++*launches;
  const long long need = (p.rows + 7) / 8;
  const long long cap = (long long)sm_count() * 8;
  blend_kernel<<<(int)(need < cap ? need : cap), kBlendThreads, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace swam
