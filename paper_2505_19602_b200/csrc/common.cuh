// Shared device-side definitions of the ScaleKV kernels: the view of one layer's paged store
// and small numeric helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace scalekv {

// Sticky device status word values (mirrors scalekv_status).
constexpr int kDevTimeout = 6;
constexpr int kDevCheck = 7;

constexpr int kMaxWindow = 64;

// One layer's slice of the paged per-head store.  Logical slot s of slice `sl` lives in page
// page_table[sl * pages_per_slice + (s >> page_shift)], row (s & page_mask).
struct LayerView {
  char *k_pool;            // [n_pages][page_tokens][row_bytes]
  char *v_pool;            // same geometry
  int *pos_pool;           // [n_pages][page_tokens] original positions
  const int *page_table;   // [n_slices][pages_per_slice]
  int *hist_len;           // [n_slices] entries held before the current map
  int *status;             // sticky device status word
  int pages_per_slice;
  int page_shift, page_mask;
  int row_bytes;           // head_dim * sizeof(element)
  int n_slices;            // batch * n_heads
  int n_heads;
};

__device__ __forceinline__ size_t slot_row(const LayerView &lv, int slice, int slot) {
  int page = __ldg(lv.page_table + (size_t)slice * lv.pages_per_slice + (slot >> lv.page_shift));
  return ((size_t)page << lv.page_shift) + (size_t)(slot & lv.page_mask);
}

// Tensor view with element strides (batch, head, token).
struct TensorView {
  const char *ptr;
  long long sb, sh, st;   // in elements
};

// A current map that has not been copied into the pages: the caller's K and V tensors ([B][H][n_k][d] views,
// strides in elements of esize bytes).  on == 0: the map is in the pages like every other entry.
struct ExternalMap {
  int on;
  const char *k, *v;
  long long sb, sh, st;
  int esize;
};

template <typename T>
__device__ __forceinline__ const T *row_ptr(const TensorView &t, int b, int h, int i) {
  return reinterpret_cast<const T *>(t.ptr) + (long long)b * t.sb + (long long)h * t.sh + (long long)i * t.st;
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_float(float x);
template <> __device__ __forceinline__ float from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Loads 16 bytes of a row and widens to floats (4 for fp32, 8 for bf16).
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float *p, float *out) {
    float4 v = *reinterpret_cast<const float4 *>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float *out) {
    uint4 v = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

}  // namespace scalekv
