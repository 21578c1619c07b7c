// scalekv_select_static: per-row top-k of score vectors with all scratch in a fixed device array
// that is part of the library image.  See include/scalekv.h for the contract.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "../../include/scalekv.h"

namespace {

// Scratch of the radix select: one 32-bit sortable key per score.  Every device that loads the
// library carries these 4 MiB until the process exits.
constexpr size_t kStaticEntries = (size_t)SCALEKV_SELECT_STATIC_MAX_ENTRIES;
static __device__ __align__(256) uint32_t g_select_scratch[kStaticEntries];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
uint32_t *g_scratch_ptr[kMaxDevices] = {nullptr};   // device addresses, looked up once per device

// Exclusive prefix sum of v over the block in thread order; *total receives the block sum.
__device__ __forceinline__ int block_scan_excl(int v, int *warp_sums, int *total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  int incl = v;
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();
  if (lane == 31) warp_sums[wid] = incl;
  __syncthreads();
  if (wid == 0) {
    const int ws = (lane < (int)(blockDim.x >> 5)) ? warp_sums[lane] : 0;
    int wi = ws;
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    warp_sums[lane] = wi - ws;
    if (lane == 31) warp_sums[32] = wi;
  }
  __syncthreads();
  *total = warp_sums[32];
  return warp_sums[wid] + incl - v;
}

// Row-wise variant of the select kernel: no page table and no window, scores are dense rows.
// One block of 1024 threads per row.  keys is the row's slice of the static scratch.
__global__ void __launch_bounds__(1024) select_static_kernel(const float *scores, int len, int ld, int k, uint32_t *keys_all,
                                                             int *idx_out) {
  __shared__ int hist[256];
  __shared__ int warp_sums[33];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining;
  const int row = blockIdx.x;
  uint32_t *key = keys_all + (size_t)row * len;
  const float *s = scores + (size_t)row * ld;
  int *out = idx_out + (size_t)row * k;
  for (int i = threadIdx.x; i < len; i += blockDim.x) key[i] = __float_as_uint(s[i]) & 0x7FFFFFFFu;
  __syncthreads();
  uint32_t threshold = 0;
  int n_ties_taken = 0;
  if (k < len) {
    if (threadIdx.x == 0) { sh_prefix = 0; sh_remaining = k; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      const uint32_t mask_hi = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
      if (threadIdx.x < 256) hist[threadIdx.x] = 0;
      __syncthreads();
      const uint32_t prefix = sh_prefix;
      for (int i = threadIdx.x; i < len; i += blockDim.x) {
        const uint32_t kk = key[i];
        if ((kk & mask_hi) == prefix) atomicAdd(&hist[(kk >> shift) & 0xFF], 1);
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        int rem = sh_remaining, dsel = 0;
        for (int dgt = 255; dgt >= 0; --dgt) {
          const int c = hist[dgt];
          if (c >= rem) { dsel = dgt; break; }
          rem -= c;
        }
        sh_remaining = rem;
        sh_prefix = prefix | ((uint32_t)dsel << shift);
      }
      __syncthreads();
    }
    threshold = sh_prefix;
    n_ties_taken = sh_remaining;
  }
  const bool keep_all = k >= len;
  int base_out = 0, base_tie = 0;
  for (int i0 = 0; i0 < len; i0 += blockDim.x) {
    const int i = i0 + threadIdx.x;
    bool gt = false, tie = false;
    if (i < len) {
      const uint32_t kk = key[i];
      if (keep_all) gt = true; else { gt = kk > threshold; tie = kk == threshold; }
    }
    int tie_total, keep_total;
    const int tie_rank = base_tie + block_scan_excl(tie ? 1 : 0, warp_sums, &tie_total);
    const bool keep = gt || (tie && tie_rank < n_ties_taken);
    const int oidx = base_out + block_scan_excl(keep ? 1 : 0, warp_sums, &keep_total);
    if (keep) out[oidx] = i;
    base_tie += tie_total;
    base_out += keep_total;
  }
}

}  // namespace

extern "C" scalekv_status scalekv_select_static(const float *scores, int32_t n_rows, int32_t len, int32_t ld, int32_t k,
                                                int32_t *idx_out, void *stream) {
  if (!scores || !idx_out || n_rows < 1 || len < 1 || ld < len || k < 1 || k > len) {
    fprintf(stderr, "scalekv_select_static: invalid argument (need n_rows >= 1, 1 <= k <= len <= ld)\n");
    return SCALEKV_ERR_INVALID_ARG;
  }
  if ((size_t)n_rows * (size_t)len > kStaticEntries) {
    fprintf(stderr, "scalekv_select_static: n_rows * len = %zu exceeds the static scratch of %zu entries\n",
            (size_t)n_rows * (size_t)len, kStaticEntries);
    return SCALEKV_ERR_CAPACITY;
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SCALEKV_ERR_CUDA;
  uint32_t *scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
      // the symbol's name is only a host-side handle: ask the runtime for its address on this device
      void *p = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&p, g_select_scratch);
      if (e != cudaSuccess || p == nullptr) {
        fprintf(stderr, "scalekv_select_static: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
        return SCALEKV_ERR_CUDA;
      }
      g_scratch_ptr[dev] = static_cast<uint32_t *>(p);
    }
    scratch = g_scratch_ptr[dev];
  }
  select_static_kernel<<<n_rows, 1024, 0, static_cast<cudaStream_t>(stream)>>>(scores, len, ld, k, scratch, idx_out);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    fprintf(stderr, "scalekv_select_static: launch failed: %s\n", cudaGetErrorString(e));
    return SCALEKV_ERR_CUDA;
  }
  return SCALEKV_OK;
}
