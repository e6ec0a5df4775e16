// Packing (Sec. 4.2) and scatter / cached-prediction blend (Eq. 7): row copies by index.
//
// Rows are N_h*D elements (256 B .. 8 KB), contiguous and 16-byte aligned, so both are pure HBM streams of
// 16-byte chunks.  Each thread moves kUnroll chunks per iteration, all loads issued before the first store,
// and the grid is a multiple of the SM count so that every SM holds the same number of resident CTAs.
#include "swam_internal.cuh"

namespace swam {
namespace {

constexpr int kCopyThreads = 256;
constexpr int kUnroll = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

struct RowCopyParams {
  const uint4* src[3];
  uint4* dst[3];
  const int32_t* src_idx;  // [B, n_rows] row of src for each listed row, or nullptr (identity)
  const int32_t* dst_idx;  // [B, n_rows] row of dst for each listed row, or nullptr (identity)
  int* status;
  int n_tensors;
  int n_rows;       // listed rows per sample
  int src_rows;     // rows per sample in src
  int dst_rows;     // rows per sample in dst
  int chunks;       // 16-byte chunks per row
  long long total;  // n_tensors * B * n_rows * chunks
};

// chunk id -> (tensor, sample, listed row, chunk in row)
__global__ void __launch_bounds__(kCopyThreads) row_copy_kernel(const RowCopyParams p) {
  const long long stride = (long long)gridDim.x * kCopyThreads;
  const long long per_tensor = p.total / p.n_tensors;
  for (long long base = (long long)blockIdx.x * kCopyThreads + threadIdx.x; base < p.total; base += stride * kUnroll) {
    uint4 val[kUnroll];
    uint4* out[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const long long id = base + (long long)u * stride;
      out[u] = nullptr;
      if (id < p.total) {
        const int z = (int)(id / per_tensor);
        const long long r = id - (long long)z * per_tensor;
        const int c = (int)(r % p.chunks);
        const long long row = r / p.chunks;          // b * n_rows + listed row
        const long long b = row / p.n_rows;
        const long long lr = row - b * p.n_rows;
        long long srow = lr, drow = lr;
        bool ok = true;
        if (p.src_idx) { srow = p.src_idx[row]; ok = srow >= 0 && srow < p.src_rows; }
        if (p.dst_idx) { drow = p.dst_idx[row]; ok = ok && drow >= 0 && drow < p.dst_rows; }
        if (ok) {
          val[u] = ld_stream(p.src[z] + (b * p.src_rows + srow) * p.chunks + c);
          out[u] = p.dst[z] + (b * p.dst_rows + drow) * p.chunks + c;
        } else if (c == 0) {
          atomicOr(p.status, ST_BAD_MAP);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (out[u]) *out[u] = val[u];
  }
}

struct BlendParams {
  const uint4* out_p;
  const uint4* cached;
  uint4* out;
  const int32_t* inv_map;  // [B, L]
  int* status;
  int L, Lp, chunks;
  long long total;  // B * L * chunks
};

// out[b,t] = inv[b,t] >= 0 ? out_p[b, inv[b,t]] : cached[b,t]
__global__ void __launch_bounds__(kCopyThreads) blend_kernel(const BlendParams p) {
  const long long stride = (long long)gridDim.x * kCopyThreads;
  for (long long base = (long long)blockIdx.x * kCopyThreads + threadIdx.x; base < p.total; base += stride * kUnroll) {
    uint4 val[kUnroll];
    bool live[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const long long id = base + (long long)u * stride;
      live[u] = id < p.total;
      if (live[u]) {
        const int c = (int)(id % p.chunks);
        const long long row = id / p.chunks;  // b * L + t
        const long long b = row / p.L;
        const int pr = p.inv_map[row];
        if (pr >= p.Lp) {
          if (c == 0) atomicOr(p.status, ST_BAD_MAP);
          live[u] = false;
        } else if (pr >= 0) {
          val[u] = ld_stream(p.out_p + (b * p.Lp + pr) * p.chunks + c);
        } else {
          val[u] = ld_stream(p.cached + id);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (live[u]) p.out[base + (long long)u * stride] = val[u];
  }
}

int copy_grid(long long total) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const long long per_cta = (long long)kCopyThreads * kUnroll;
  long long need = (total + per_cta - 1) / per_cta;
  const long long cap = (long long)sms * 8;  // 8 resident CTAs of 256 threads per SM
  if (need >= cap) return (int)cap;
  return (int)(need < 1 ? 1 : need);
}

}  // namespace

cudaError_t launch_pack(const Dims& d, const void* const src[3], void* const dst[3], const int32_t* pack_map,
                        int* status, cudaStream_t st, int* launches) {
  RowCopyParams p{};
  int n = 0;
  for (int i = 0; i < 3; ++i)
    if (src[i] && dst[i]) { p.src[n] = (const uint4*)src[i]; p.dst[n] = (uint4*)dst[i]; ++n; }
  if (n == 0) return cudaSuccess;
  p.src_idx = pack_map; p.dst_idx = nullptr; p.status = status;
  p.n_tensors = n; p.n_rows = d.Lp; p.src_rows = d.L; p.dst_rows = d.Lp;
  p.chunks = d.N_h * d.D * (d.dtype == 0 ? 4 : 2) / 16;
  p.total = (long long)n * d.B * d.Lp * p.chunks;
  if (p.total == 0) return cudaSuccess;
  ++*launches;
  row_copy_kernel<<<copy_grid(p.total), kCopyThreads, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_scatter(const Dims& d, const void* out_p, const int32_t* pack_map, const int32_t* inv_map,
                           const void* cached, void* out, int* status, cudaStream_t st, int* launches) {
  const int chunks = d.N_h * d.D * (d.dtype == 0 ? 4 : 2) / 16;
  if (cached == out) {
    RowCopyParams p{};
    p.src[0] = (const uint4*)out_p; p.dst[0] = (uint4*)out;
    p.src_idx = nullptr; p.dst_idx = pack_map; p.status = status;
    p.n_tensors = 1; p.n_rows = d.Lp; p.src_rows = d.Lp; p.dst_rows = d.L;
    p.chunks = chunks;
    p.total = (long long)d.B * d.Lp * chunks;
    if (p.total == 0) return cudaSuccess;
    ++*launches;
    row_copy_kernel<<<copy_grid(p.total), kCopyThreads, 0, st>>>(p);
    return cudaGetLastError();
  }
  BlendParams p{(const uint4*)out_p, (const uint4*)cached, (uint4*)out, inv_map, status, d.L, d.Lp, chunks,
                (long long)d.B * d.L * chunks};
  if (p.total == 0) return cudaSuccess;
  ++*launches;
  blend_kernel<<<copy_grid(p.total), kCopyThreads, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace swam
