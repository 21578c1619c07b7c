// SIMT kernels of the ScaleKV hot path: append, fp32-FMA attention (the f32 x 64 configuration
// and the reference path for bf16), observation-window scoring, segmented radix top-k, in-place
// gather-compaction and the offline layer statistics.
#pragma once
#include "common.cuh"

namespace scalekv {

// Window description handed to the select / score kernels by value.
struct WindowArg {
  int w;                 // number of window rows
  int all;               // 1: the whole current map is the window
  int n_prev;            // N_{k-1}: original position of the current map's first token
  int n_k;               // tokens of the current map
  int pos[kMaxWindow];   // ascending raster indices (unused when all = 1)
};

__device__ __forceinline__ bool is_window_pos(const WindowArg &wa, int p) {
  int r = p - wa.n_prev;
  if (r < 0) return false;
  if (wa.all) return true;
  int lo = 0, hi = wa.w;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (wa.pos[mid] < r) lo = mid + 1; else hi = mid;
  }
  return lo < wa.w && wa.pos[lo] == r;
}

// ------------------------------------------------------------------------------------------
// append: rows of the current map are copied behind the slice's history (Sec. 1; Sec. 3.3).
// grid (ceil(n_k / 64), n_slices), 256 threads, one 16-byte piece per thread per step.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) append_kernel(LayerView lv, TensorView K, TensorView V, int n_k, int n_prev,
                                                      int elem_bytes) {
  const int slice = blockIdx.y;
  const int b = slice / lv.n_heads, h = slice % lv.n_heads;
  const int ppr = lv.row_bytes >> 4;  // 16-byte pieces per row
  const int hist = lv.hist_len[slice];
  if (hist + n_k > (lv.pages_per_slice << lv.page_shift)) {      // would outgrow the page table: report, do not fault
    if (threadIdx.x == 0) atomicExch(lv.status, kDevCheck);
    return;
  }
  const int rows_per_step = 256 / ppr;
  const int r_in = threadIdx.x / ppr, c = threadIdx.x % ppr;
  const int i0 = blockIdx.x * 64;
  if (r_in >= rows_per_step) return;
  for (int r = r_in; r < 64; r += rows_per_step) {
    const int i = i0 + r;
    if (i >= n_k) break;
    const size_t row = slot_row(lv, slice, hist + i);
    const char *ks = K.ptr + ((long long)b * K.sb + (long long)h * K.sh + (long long)i * K.st) * elem_bytes;
    const char *vs = V.ptr + ((long long)b * V.sb + (long long)h * V.sh + (long long)i * V.st) * elem_bytes;
    uint4 kv = __ldg(reinterpret_cast<const uint4 *>(ks) + c);
    uint4 vv = __ldg(reinterpret_cast<const uint4 *>(vs) + c);
    reinterpret_cast<uint4 *>(lv.k_pool + row * lv.row_bytes)[c] = kv;
    reinterpret_cast<uint4 *>(lv.v_pool + row * lv.row_bytes)[c] = vv;
    if (c == 0) lv.pos_pool[row] = n_prev + i;
  }
}

// hist_len += n_k for a current map that no compress has consumed.
__global__ void commit_kernel(LayerView lv, int n_k) {
  int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s < lv.n_slices) lv.hist_len[s] += n_k;
}

// ------------------------------------------------------------------------------------------
// attend (SIMT): O = softmax(scale * Q K^T) V with online softmax, fp32 FMA (Eq. 5).
// grid (ceil(n_k / 64), n_slices), 256 threads.  A block owns 64 query rows and streams the
// slice's cache in tiles of 64 entries; thread (ty, tx) owns rows ty + 16 i, columns tx + 16 j.
// ------------------------------------------------------------------------------------------
template <typename T, int D>
__device__ __forceinline__ void load_tile_rows(float *dst, int ld, const LayerView &lv, const char *pool, int slice,
                                               int j0, int L) {
  constexpr int CH = D * (int)sizeof(T) / 16;
  constexpr int VN = Vec16<T>::N;
  for (int idx = threadIdx.x; idx < 64 * CH; idx += 256) {
    const int r = idx / CH, c = idx % CH;
    float v[VN];
    if (j0 + r < L) {
      const size_t row = slot_row(lv, slice, j0 + r);
      Vec16<T>::load(reinterpret_cast<const T *>(pool + row * lv.row_bytes) + c * VN, v);
    } else {
#pragma unroll
      for (int e = 0; e < VN; ++e) v[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < VN; ++e) dst[r * ld + c * VN + e] = v[e];
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(256) attend_simt_kernel(LayerView lv, TensorView Q, TensorView O, float *lse, int n_k,
                                                          float scale) {
  constexpr int BM = 64, BN = 64, LD = D + 4, LDS = BN + 1;
  constexpr int CH = D * (int)sizeof(T) / 16;
  constexpr int VN = Vec16<T>::N;
  constexpr int NJ = D / 16;
  extern __shared__ float smem[];
  float *Qs = smem;
  float *KVs = Qs + BM * LD;
  float *Ss = KVs + BN * LD;
  float *m_s = Ss + BM * LDS;
  float *l_s = m_s + BM;
  float *a_s = l_s + BM;

  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int slice = blockIdx.y;
  const int b = slice / lv.n_heads, h = slice % lv.n_heads;
  const int q0 = blockIdx.x * BM;
  const int L = lv.hist_len[slice] + n_k;

  for (int idx = tid; idx < BM * CH; idx += 256) {
    const int r = idx / CH, c = idx % CH;
    float v[VN];
    if (q0 + r < n_k) {
      Vec16<T>::load(row_ptr<T>(Q, b, h, q0 + r) + c * VN, v);
    } else {
#pragma unroll
      for (int e = 0; e < VN; ++e) v[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < VN; ++e) Qs[r * LD + c * VN + e] = v[e];
  }
  if (tid < BM) { m_s[tid] = -INFINITY; l_s[tid] = 0.f; }

  float acc[4][NJ];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < NJ; ++j) acc[i][j] = 0.f;

  for (int j0 = 0; j0 < L; j0 += BN) {
    __syncthreads();
    load_tile_rows<T, D>(KVs, LD, lv, lv.k_pool, slice, j0, L);
    __syncthreads();
    float s[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
    for (int c = 0; c < D; c += 4) {
      float4 q[4], k[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) q[i] = *reinterpret_cast<const float4 *>(&Qs[(ty + 16 * i) * LD + c]);
#pragma unroll
      for (int j = 0; j < 4; ++j) k[j] = *reinterpret_cast<const float4 *>(&KVs[(tx + 16 * j) * LD + c]);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          s[i][j] = fmaf(q[i].x, k[j].x, s[i][j]);
          s[i][j] = fmaf(q[i].y, k[j].y, s[i][j]);
          s[i][j] = fmaf(q[i].z, k[j].z, s[i][j]);
          s[i][j] = fmaf(q[i].w, k[j].w, s[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j)
        Ss[(ty + 16 * i) * LDS + tx + 16 * j] = (j0 + tx + 16 * j < L) ? s[i][j] * scale : -INFINITY;
    __syncthreads();
    // K tile is consumed: bring V in while the rows are normalised
    load_tile_rows<T, D>(KVs, LD, lv, lv.v_pool, slice, j0, L);
    {
      const int row = tid >> 2, part = tid & 3;
      float *srow = Ss + row * LDS + part * 16;
      float mx = -INFINITY;
#pragma unroll
      for (int e = 0; e < 16; ++e) mx = fmaxf(mx, srow[e]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_old = m_s[row];
      const float m_new = fmaxf(m_old, mx);
      float sum = 0.f;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        float p = expf(srow[e] - m_new);
        srow[e] = p;
        sum += p;
      }
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      __syncwarp();
      if (part == 0) {
        const float a = expf(m_old - m_new);
        a_s[row] = a;
        m_s[row] = m_new;
        l_s[row] = l_s[row] * a + sum;
      }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = a_s[ty + 16 * i];
#pragma unroll
      for (int j = 0; j < NJ; ++j) acc[i][j] *= a;
    }
    for (int kk = 0; kk < BN; ++kk) {
      float p[4], v[NJ];
#pragma unroll
      for (int i = 0; i < 4; ++i) p[i] = Ss[(ty + 16 * i) * LDS + kk];
#pragma unroll
      for (int j = 0; j < NJ; ++j) v[j] = KVs[kk * LD + tx + 16 * j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < NJ; ++j) acc[i][j] = fmaf(p[i], v[j], acc[i][j]);
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty + 16 * i;
    if (q0 + r >= n_k) continue;
    const float inv = 1.f / l_s[r];
    T *orow = const_cast<T *>(row_ptr<T>(O, b, h, q0 + r));
#pragma unroll
    for (int j = 0; j < NJ; ++j) orow[tx + 16 * j] = from_float<T>(acc[i][j] * inv);
    if (lse != nullptr && tx == 0) lse[(size_t)slice * n_k + q0 + r] = m_s[r] + logf(l_s[r]);
  }
}

// ------------------------------------------------------------------------------------------
// score, step 1 (only when attend did not record them): logits of the window rows against a tile of
// 64 cache entries (Eq. 5), in base-2 units: y = scale * log2(e) * <q, k>.
// grid (ceil(L_max / 64), n_slices), 256 threads.  logits is [n_slices][w][ld_l] fp32.
// ------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(256) score_logits_kernel(LayerView lv, TensorView Qw, WindowArg wa, int full_map,
                                                           float *logits, int ld_l, float scale) {
  constexpr int LD = D + 4;
  constexpr int CH = D * (int)sizeof(T) / 16;
  constexpr int VN = Vec16<T>::N;
  extern __shared__ float smem[];
  float *Qs = smem;             // [64][LD], rows >= w zero
  float *Ks = Qs + 64 * LD;     // [64][LD]
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int slice = blockIdx.y;
  const int b = slice / lv.n_heads, h = slice % lv.n_heads;
  const int L = lv.hist_len[slice] + wa.n_k;
  const int j0 = blockIdx.x * 64;
  if (j0 >= L) return;
  for (int idx = tid; idx < 64 * CH; idx += 256) {
    const int r = idx / CH, c = idx % CH;
    float v[VN];
    if (r < wa.w) {
      const int qi = full_map ? (wa.all ? r : wa.pos[r]) : r;
      Vec16<T>::load(row_ptr<T>(Qw, b, h, qi) + c * VN, v);
    } else {
#pragma unroll
      for (int e = 0; e < VN; ++e) v[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < VN; ++e) Qs[r * LD + c * VN + e] = v[e];
  }
  load_tile_rows<T, D>(Ks, LD, lv, lv.k_pool, slice, j0, L);
  __syncthreads();
  const int ni = (wa.w + 15) >> 4;  // active 16-row groups
  float s[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
  for (int c = 0; c < D; c += 4) {
    float4 k[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) k[j] = *reinterpret_cast<const float4 *>(&Ks[(tx + 16 * j) * LD + c]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (i < ni) {
        const float4 q = *reinterpret_cast<const float4 *>(&Qs[(ty + 16 * i) * LD + c]);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          s[i][j] = fmaf(q.x, k[j].x, s[i][j]);
          s[i][j] = fmaf(q.y, k[j].y, s[i][j]);
          s[i][j] = fmaf(q.z, k[j].z, s[i][j]);
          s[i][j] = fmaf(q.w, k[j].w, s[i][j]);
        }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty + 16 * i;
    if (r >= wa.w) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = j0 + tx + 16 * j;
      if (col < L) logits[((size_t)slice * wa.w + r) * ld_l + col] = s[i][j] * (scale * 1.4426950408889634f);
    }
  }
}

__device__ __forceinline__ float block_reduce_max(float v, float *red) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  const int nw = blockDim.x >> 5;
  float r = red[0];
  for (int i = 1; i < nw; ++i) r = fmaxf(r, red[i]);
  return r;
}
__device__ __forceinline__ float block_reduce_sum(float v, float *red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  const int nw = blockDim.x >> 5;
  float r = 0.f;
  for (int i = 0; i < nw; ++i) r += red[i];   // fixed order: deterministic
  return r;
}

// ------------------------------------------------------------------------------------------
// score, step 2 (Sec. 3.3, Eq. 5): from the base-2 logits y[w][L] of the window rows to the importance
// s_i = (1/w) sum_j 2^(y_ji - lse_j), lse_j the base-2 log-sum-exp of row j (recorded by attend, or
// computed by row_lse_kernel).  Streaming and embarrassingly parallel: grid (ceil(L_max / 256),
// n_slices), one entry per thread, the w loads of a thread independent and coalesced across the warp.
// Besides the score (kept for inspection) it writes the entry's radix key: the bit pattern of the
// non-negative float, or a sentinel for window entries, which never take part in the selection.
// ------------------------------------------------------------------------------------------
constexpr uint32_t kWindowKey = 0xFFFFFFFFu;

__device__ __forceinline__ int block_exclusive_scan(int v, int *warp_sums, int *total) {
  // returns exclusive prefix of v over the block (thread order); *total = block sum
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  int incl = v;
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();
  if (lane == 31) warp_sums[wid] = incl;
  __syncthreads();
  if (wid == 0) {
    int ws = (lane < (int)(blockDim.x >> 5)) ? warp_sums[lane] : 0;
    int wi = ws;
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    warp_sums[lane] = wi - ws;        // exclusive warp offsets
    if (lane == 31) warp_sums[32] = wi;  // block total
  }
  __syncthreads();
  *total = warp_sums[32];
  return warp_sums[wid] + incl - v;
}

// logit_scale: what turns a stored logit into a base-2 logit (1 when the logits kernel wrote them, softmax scale *
// log2(e) when attend recorded raw products).  tile_padded: attend recorded them while the current map was
// not in the store yet, so its entries sit behind the history rounded up to a multiple of 128 columns.
__global__ void __launch_bounds__(256) score_kernel(LayerView lv, WindowArg wa, const float *logits, const float *lse,
                                                    int ld_l, float logit_scale, int tile_padded, float *scores, uint32_t *keys,
                                                    int ld_s) {
  __shared__ float lse_row[kMaxWindow];
  const int slice = blockIdx.y;
  const int hist = lv.hist_len[slice];
  const int L = hist + wa.n_k;
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (blockIdx.x * 256 >= L) return;
  const int w = wa.w;
  if (threadIdx.x < w) lse_row[threadIdx.x] = lse[(size_t)slice * w + threadIdx.x];
  __syncthreads();
  if (i >= L) return;
  const int col = (tile_padded && i >= hist) ? (((hist + 127) >> 7) << 7) + (i - hist) : i;
  const float *y = logits + (size_t)slice * w * ld_l + col;
  float sc = 0.f;
  int j = 0;
  for (; j + 8 <= w; j += 8) {
    float t[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) t[e] = __ldg(y + (size_t)(j + e) * ld_l);
#pragma unroll
    for (int e = 0; e < 8; ++e) sc += exp2f(fmaf(t[e], logit_scale, -lse_row[j + e]));
  }
  for (; j < w; ++j) sc += exp2f(fmaf(__ldg(y + (size_t)j * ld_l), logit_scale, -lse_row[j]));
  sc *= 1.f / (float)w;
  scores[(size_t)slice * ld_s + i] = sc;
  const bool win = is_window_pos(wa, lv.pos_pool[slot_row(lv, slice, i)]);
  keys[(size_t)slice * ld_s + i] = win ? kWindowKey : (__float_as_uint(sc) & 0x7FFFFFFFu);
}

// Head-shared importance (Sec. 3.3, "a unified importance metric" read as shared between the heads of a
// batch element): every entry's importance becomes the mean over the heads, summed in head order, and
// the keys follow.  The heads must hold the same entries: equal lengths and equal original positions,
// else the device status is raised and the selection that follows does not run.
// grid (ceil(L_max / 256), B), 256 threads; scores and keys are [n_slices][ld_s].
__global__ void __launch_bounds__(256) head_mean_kernel(LayerView lv, WindowArg wa, float *scores, uint32_t *keys, int ld_s) {
  const int H = lv.n_heads;
  const int s0 = blockIdx.y * H;
  const int L = lv.hist_len[s0] + wa.n_k;
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (blockIdx.x == 0 && threadIdx.x < H && lv.hist_len[s0 + threadIdx.x] + wa.n_k != L) atomicExch(lv.status, kDevCheck);
  if (i >= L) return;
  const int pos = lv.pos_pool[slot_row(lv, s0, i)];
  float sum = 0.f;
  bool same = true;
  for (int h = 0; h < H; ++h) {
    sum += scores[(size_t)(s0 + h) * ld_s + i];
    same = same && (lv.hist_len[s0 + h] + wa.n_k <= i || lv.pos_pool[slot_row(lv, s0 + h, i)] == pos);
  }
  if (!same) atomicExch(lv.status, kDevCheck);
  const float mean = sum * (1.f / (float)H);
  const uint32_t key = is_window_pos(wa, pos) ? kWindowKey : (__float_as_uint(mean) & 0x7FFFFFFFu);
  for (int h = 0; h < H; ++h) {
    scores[(size_t)(s0 + h) * ld_s + i] = mean;
    keys[(size_t)(s0 + h) * ld_s + i] = key;
  }
}

// Keys of the positional keep rule (the comparison policies of Sec. 4.1: sliding window, sinks + recent
// tokens): entries whose original position is below n_sink carry the sentinel (always kept), every
// other entry competes on its position, most recent first.  grid (ceil(L_max / 256), n_slices).
__global__ void __launch_bounds__(256) recent_keys_kernel(LayerView lv, int n_k, int n_sink, uint32_t *keys, int ld_s) {
  const int slice = blockIdx.y;
  const int L = lv.hist_len[slice] + n_k;
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= L) return;
  const int pos = lv.pos_pool[slot_row(lv, slice, i)];
  keys[(size_t)slice * ld_s + i] = pos < n_sink ? kWindowKey : (uint32_t)pos + 1u;
}

// Base-2 log-sum-exp of every window row of y[w][L] when attend did not record it: one CTA of 1024
// threads per slice, 16 rows per round, a maximum sweep and a sum sweep.  lse is [n_slices][w].
__global__ void __launch_bounds__(1024) row_lse_kernel(LayerView lv, WindowArg wa, const float *logits, int ld_l, float *lse) {
  __shared__ float part[32][16];
  __shared__ float m_row[16];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int slice = blockIdx.x;
  const int L = lv.hist_len[slice] + wa.n_k;
  const int w = wa.w;
  const float *y = logits + (size_t)slice * w * ld_l;
  for (int g0 = 0; g0 < w; g0 += 16) {
    const int nr = w - g0 < 16 ? w - g0 : 16;
    float acc[16];
#pragma unroll
    for (int r = 0; r < 16; ++r) acc[r] = -INFINITY;
    for (int i = tid; i < L; i += 1024) {
#pragma unroll
      for (int r = 0; r < 16; ++r)
        if (r < nr) acc[r] = fmaxf(acc[r], y[(size_t)(g0 + r) * ld_l + i]);
    }
#pragma unroll
    for (int r = 0; r < 16; ++r) {
      float v = acc[r];
      for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
      if (lane == 0) part[wid][r] = v;
    }
    __syncthreads();
    if (tid < 16) {
      float v = part[0][tid];
      for (int k = 1; k < 32; ++k) v = fmaxf(v, part[k][tid]);
      m_row[tid] = v;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 16; ++r) acc[r] = 0.f;
    for (int i = tid; i < L; i += 1024) {
#pragma unroll
      for (int r = 0; r < 16; ++r)
        if (r < nr) acc[r] += exp2f(y[(size_t)(g0 + r) * ld_l + i] - m_row[r]);
    }
#pragma unroll
    for (int r = 0; r < 16; ++r) {
      float v = acc[r];
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) part[wid][r] = v;
    }
    __syncthreads();
    if (tid < 16) {
      float v = 0.f;
      for (int k = 0; k < 32; ++k) v += part[k][tid];     // fixed order: deterministic
      if (tid < nr) lse[(size_t)slice * w + g0 + tid] = m_row[tid] + log2f(v);
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------
// select: per-slice top-k' of the non-window entries by key (Sec. 3.3), one CTA of 1024 threads per
// slice with the slice's keys in shared memory (with pool > 1 a candidate's key is first replaced by
// its importance averaged over the neighbouring entries):
//   radix select of the k'-th largest key, 8 bits per pass, warp-aggregated histogram updates; then
//   the ordered emit of the ascending slot list of survivors (selected U window); ties at the
//   threshold go to the lowest slots = lowest original positions.  Every thread owns a run of
//   consecutive entries, so two block scans order the whole list.  Deterministic.
// Dynamic shared memory: 4 * ld_s bytes of keys.
// ------------------------------------------------------------------------------------------
constexpr int kMaxHeadBudgets = 128;
struct HeadBudgets {     // per-head budgets of one compress call
  int v[kMaxHeadBudgets];
};
// Spreads the per-head budgets of a compress call over the slices (slice = b * n_heads + h), so that the
// select kernel reads its budget with one load instead of indexing a by-value table.
__global__ void head_budget_kernel(HeadBudgets hb, int n_heads, int n_slices, int *slice_budget) {
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s < n_slices) slice_budget[s] = hb.v[s % n_heads];
}
// Shared state of one selection (static shared memory of the calling kernel).
struct SelectShared {
  int hist[256];
  int warp_sums[33];
  uint32_t prefix;
  int remaining;
};

// The selection proper, run by a whole CTA of 1024 threads: key[0 .. L) (shared or global memory) -> out[] = the
// ascending slots of the survivors (the `budget` largest keys, equal keys by lowest slot, plus every sentinel
// entry).  Returns the number of survivors; *kprime_plus_win receives the count the rule demands.
__device__ __forceinline__ int select_and_emit(const uint32_t *key, int L, int budget, int *out, SelectShared &sh,
                                                int *kprime_plus_win) {
  const int tid = threadIdx.x, lane = tid & 31;
  int n_win_local = 0;
  for (int i = tid; i < L; i += 1024) n_win_local += (key[i] == kWindowKey) ? 1 : 0;
  int n_win;
  block_exclusive_scan(n_win_local, sh.warp_sums, &n_win);
  const int cand = L - n_win;
  const int kprime = (budget < 0 || budget > cand) ? cand : budget;
  *kprime_plus_win = kprime + n_win;

  // radix select of the kprime-th largest key
  uint32_t threshold = 0;
  int n_ties_taken = 0;       // how many entries equal to the threshold are kept
  if (kprime > 0 && kprime < cand) {
    if (tid == 0) { sh.prefix = 0; sh.remaining = kprime; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      const uint32_t mask_hi = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
      if (tid < 256) sh.hist[tid] = 0;
      __syncthreads();
      const uint32_t prefix = sh.prefix;
      for (int i0 = 0; i0 < L; i0 += 1024) {
        const int i = i0 + tid;
        const uint32_t k = i < L ? key[i] : kWindowKey;
        const bool in = (k != kWindowKey) && ((k & mask_hi) == prefix);
        const uint32_t digit = in ? ((k >> shift) & 0xFFu) : 256u;
        // one shared-memory atomic per distinct digit in the warp
        const uint32_t peers = __match_any_sync(0xffffffffu, digit);
        if (in && lane == (__ffs(peers) - 1)) atomicAdd(&sh.hist[digit], __popc(peers));
      }
      __syncthreads();
      if (tid < 32) {
        // digits 255 .. 0 in descending order, 8 per lane; find where the running count reaches `rem`
        int c[8], tot = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) { c[e] = sh.hist[255 - (lane * 8 + e)]; tot += c[e]; }
        int incl = tot;
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        const int rem = sh.remaining;
        const int before = incl - tot;
        __syncwarp();
        if (before < rem && incl >= rem) {
          int dsel = 0, r = rem - before;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            if (r > 0) {
              if (c[e] >= r) { dsel = 255 - (lane * 8 + e); sh.remaining = r; r = 0; }
              else r -= c[e];
            }
          }
          sh.prefix = prefix | ((uint32_t)dsel << shift);
        }
      }
      __syncthreads();
    }
    threshold = sh.prefix;
    n_ties_taken = sh.remaining;
  }
  const bool keep_all = (kprime >= cand);
  const bool keep_none = (kprime == 0);

  // ordered emit: thread t owns entries [t * E, (t + 1) * E)
  const int E = (L + 1023) >> 10;
  const int i_lo = tid * E, i_hi = (i_lo + E < L) ? i_lo + E : L;
  int n_tie = 0;
  for (int i = i_lo; i < i_hi; ++i) {
    const uint32_t k = key[i];
    n_tie += (k != kWindowKey && !keep_all && !keep_none && k == threshold) ? 1 : 0;
  }
  int tie_total, keep_total;
  int tie_rank = block_exclusive_scan(n_tie, sh.warp_sums, &tie_total);
  int n_keep = 0;
  {
    int tr = tie_rank;
    for (int i = i_lo; i < i_hi; ++i) {
      const uint32_t k = key[i];
      bool keep = (k == kWindowKey);
      if (!keep) {
        if (keep_all) keep = true;
        else if (!keep_none) {
          if (k > threshold) keep = true;
          else if (k == threshold) { keep = tr < n_ties_taken; ++tr; }
        }
      }
      n_keep += keep ? 1 : 0;
    }
  }
  int oidx = block_exclusive_scan(n_keep, sh.warp_sums, &keep_total);
  for (int i = i_lo; i < i_hi; ++i) {
    const uint32_t k = key[i];
    bool keep = (k == kWindowKey);
    if (!keep) {
      if (keep_all) keep = true;
      else if (!keep_none) {
        if (k > threshold) keep = true;
        else if (k == threshold) { keep = tie_rank < n_ties_taken; ++tie_rank; }
      }
    }
    if (keep) out[oidx++] = i;
  }
  return keep_total;
}

// The importance averaged over `pool` neighbouring entries (zeros beyond both ends), summed in slot order.
__device__ __forceinline__ uint32_t pooled_key(const float *sc, int i, int L, int pool) {
  const int r = pool >> 1;
  float acc = 0.f;
  for (int d = -r; d <= r; ++d)
    if (i + d >= 0 && i + d < L) acc += sc[i + d];
  return __float_as_uint(acc / (float)pool) & 0x7FFFFFFFu;
}

// slice_budget: per-slice budgets (nullptr: every slice takes `budget`).
// in_smem != 0: the slice's keys are staged in dynamic shared memory (4 * ld_s bytes); 0: a slice too long for
// that is selected from the global key array as it stands (with pool > 1 the pooled keys are first written back
// there), every pass streaming the keys through L2.
__global__ void __launch_bounds__(1024) select_kernel(LayerView lv, WindowArg wa, int budget, const int *slice_budget, uint32_t *keys,
                                                      const float *scores, int pool, int ld_s, int in_smem, int *keep_list,
                                                      int *kept_count) {
  extern __shared__ uint32_t key_sm[];         // [L] when in_smem
  __shared__ SelectShared sh;
  const int tid = threadIdx.x;
  const int slice = blockIdx.x;
  const int dev_status = *reinterpret_cast<volatile int *>(lv.status);   // both loads in flight before the test
  const int L = lv.hist_len[slice] + wa.n_k;
  if (dev_status != 0) return;                 // an earlier kernel reported a failed check: leave the store alone
  int *out = keep_list + (size_t)slice * ld_s;
  uint32_t *gkey = keys + (size_t)slice * ld_s;
  const float *sc = scores + (size_t)slice * ld_s;
  for (int i = tid; i < L; i += 1024) {
    uint32_t k = gkey[i];
    if (pool > 1 && k != kWindowKey) k = pooled_key(sc, i, L, pool);
    if (in_smem) key_sm[i] = k;
    else if (pool > 1) gkey[i] = k;
  }
  __syncthreads();
  if (slice_budget != nullptr) budget = slice_budget[slice];
  int want;
  const int keep_total = select_and_emit(in_smem ? key_sm : gkey, L, budget, out, sh, &want);
  if (tid == 0) {
    kept_count[slice] = keep_total;
    // the count rule of the selection: k' candidates and every sentinel entry survive
    if (keep_total != want) atomicExch(lv.status, kDevCheck);
  }
}

// ------------------------------------------------------------------------------------------
// compact: slot j <- old slot keep[j], in place (Sec. 3.3, pruning).  grid (n_slices, 2, 4):
// blockIdx.y = 0 moves K (and, in column block 0, pos), 1 moves V; blockIdx.z picks a quarter of
// the row's 16-byte pieces, so that a slice's move is spread over 8 CTAs that touch disjoint bytes.
// The slice's page table and keep list are staged in shared memory first, so that the row moves
// depend on no further global look-up.  keep is ascending, so keep[j] >= j: within a chunk every
// source is read before any destination is written, and the sources of later chunks lie beyond
// every earlier destination.  256 threads, chunks of 2048 / ppq rows (ppq = pieces per row
// quarter), 8 pieces in flight per thread.  Dynamic shared memory: 4 * (pages_per_slice [+ ld_s]) B.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) compact_kernel(LayerView lv, const int *keep_list, int ld_s, int list_in_smem,
                                                      const int *kept_count) {
  extern __shared__ int csm[];
  int *pt = csm;                   // [pages_per_slice]
  const int slice = blockIdx.x;
  const int which = blockIdx.y;
  const int quarter = blockIdx.z;
  char *pool = which == 0 ? lv.k_pool : lv.v_pool;
  const int dev_status = *reinterpret_cast<volatile int *>(lv.status);   // both loads in flight before the test
  const int kept = kept_count[slice];
  if (dev_status != 0) return;                 // the selection did not run: nothing to move
  // the keep list is staged in shared memory when it fits ([kept] behind the page table), else read where it is
  const int *list = keep_list + (size_t)slice * ld_s;
  if (list_in_smem) {
    int *ls = csm + lv.pages_per_slice;
    for (int i = threadIdx.x; i < kept; i += 256) ls[i] = __ldg(list + i);
    list = ls;
  }
  for (int i = threadIdx.x; i < lv.pages_per_slice; i += 256) pt[i] = __ldg(lv.page_table + (size_t)slice * lv.pages_per_slice + i);
  __syncthreads();
  auto row_of = [&](int slot) { return ((size_t)pt[slot >> lv.page_shift] << lv.page_shift) + (size_t)(slot & lv.page_mask); };
  const int ppr = lv.row_bytes >> 4;       // 16-byte pieces per row
  const int ppq = ppr >> 2;                // pieces of this CTA's quarter (row_bytes is a multiple of 64)
  const int C = 2048 / ppq;                // rows per chunk
  int lo = 0, hi = kept;                   // first j with keep[j] != j (the untouched prefix is skipped)
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (list[mid] == mid) lo = mid + 1; else hi = mid;
  }
  const bool do_pos_cta = which == 0 && quarter == 0;
  const int r_in = threadIdx.x / ppq, c = quarter * ppq + threadIdx.x % ppq;   // piece u of a thread: row r_in + u * 256 / ppq
  const int r_step = 256 / ppq;
  const bool pos_thread = do_pos_cta && (threadIdx.x % ppq == 0);
  for (int c0 = lo; c0 < kept; c0 += C) {
    uint4 buf[8];
    int pv[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = c0 + r_in + u * r_step;
      if (j < kept) {
        const size_t row = row_of(list[j]);
        buf[u] = reinterpret_cast<const uint4 *>(pool + row * lv.row_bytes)[c];
        if (pos_thread) pv[u] = lv.pos_pool[row];
      }
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = c0 + r_in + u * r_step;
      if (j < kept) {
        const size_t row = row_of(j);
        reinterpret_cast<uint4 *>(pool + row * lv.row_bytes)[c] = buf[u];
        if (pos_thread) lv.pos_pool[row] = pv[u];
      }
    }
  }
  // no CTA of this kernel reads the length (the keep list's length is kept_count)
  if (do_pos_cta && threadIdx.x == 0) lv.hist_len[slice] = kept;
}

// ------------------------------------------------------------------------------------------
// compress in one launch (Sec. 3.3, "KV Cache Selection"): importance, selection and pruning of one slice by one
// CTA of 1024 threads, the phases separated by block barriers - what score_kernel, select_kernel and
// compact_kernel do in three launches, for every slice whose keys and keep list fit in shared memory.
//   phase 1  policy 0: s_i = (1/w) sum_j 2^(y_ji * logit_scale - lse_j) from the window rows' logits (see
//            score_kernel) -> scores (global, kept for inspection and for the pooling) and radix keys (shared);
//            policy 1: keys from the original positions (see recent_keys_kernel).
//   phase 2  select_and_emit: radix select in shared memory, ascending keep list in shared memory.
//   phase 3  slot j <- old slot keep[j] for K, V and pos, in chunks: every thread loads its 8 16-byte pieces of
//            the chunk, block barrier, stores them (keep[j] >= j, see compact_kernel); the untouched prefix is skipped.
// ext.on: the current map has not been copied into the pages (a one-call step whose attend left it in the caller's
// tensors): entries hist .. L-1 are rows of those tensors, phase 3 reads the survivors among them there and every kept
// row of the map is written, whatever its index.
// Dynamic shared memory: 4 * (2 * ld_s + pages_per_slice) bytes.  grid = n_slices.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) compress_fused_kernel(LayerView lv, WindowArg wa, int policy, int n_sink,
                                                              const float *logits, const float *lse, int ld_l, float logit_scale,
                                                              int tile_padded, int budget, const int *slice_budget, int pool,
                                                              float *scores, int ld_s, int *kept_count, ExternalMap ext) {
  extern __shared__ uint32_t fsm[];
  uint32_t *key = fsm;                                   // [ld_s]
  int *list = reinterpret_cast<int *>(fsm + ld_s);       // [ld_s]
  int *pt = list + ld_s;                                 // [pages_per_slice]
  __shared__ SelectShared sh;
  __shared__ float lse_row[kMaxWindow];
  const int tid = threadIdx.x;
  const int slice = blockIdx.x;
  const int dev_status = *reinterpret_cast<volatile int *>(lv.status);
  const int hist = lv.hist_len[slice];
  if (dev_status != 0) return;                 // an earlier kernel reported a failed check: leave the store alone
  const int L = hist + wa.n_k;
  const int w = wa.w;
  for (int i = tid; i < lv.pages_per_slice; i += 1024) pt[i] = __ldg(lv.page_table + (size_t)slice * lv.pages_per_slice + i);
  if (policy == 0 && tid < w) lse_row[tid] = lse[(size_t)slice * w + tid];
  __syncthreads();
  auto row_of = [&](int slot) { return ((size_t)pt[slot >> lv.page_shift] << lv.page_shift) + (size_t)(slot & lv.page_mask); };
  // With ext.on the current map (entries hist .. L-1) is not in the pages: entry i is row i - hist of the caller's
  // tensors and its original position follows from its index.
  auto pos_of = [&](int i) { return (ext.on && i >= hist) ? wa.n_prev + (i - hist) : lv.pos_pool[row_of(i)]; };
  const long long ext_base = ext.on ? (long long)(slice / lv.n_heads) * ext.sb + (long long)(slice % lv.n_heads) * ext.sh : 0;

  // ---- phase 1: keys
  float *sc_out = scores + (size_t)slice * ld_s;
  if (policy == 0) {
    const int pad = tile_padded ? ((((hist + 127) >> 7) << 7) - hist) : 0;     // the current map starts at a multiple of 128 columns
    const float inv_w = 1.f / (float)w;
    for (int i = tid; i < L; i += 1024) {
      const float *y = logits + (size_t)slice * w * ld_l + (i >= hist ? i + pad : i);
      float sc = 0.f;
      int j = 0;
      for (; j + 8 <= w; j += 8) {
        float t[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) t[e] = __ldg(y + (size_t)(j + e) * ld_l);
#pragma unroll
        for (int e = 0; e < 8; ++e) sc += exp2f(fmaf(t[e], logit_scale, -lse_row[j + e]));
      }
      for (; j < w; ++j) sc += exp2f(fmaf(__ldg(y + (size_t)j * ld_l), logit_scale, -lse_row[j]));
      sc *= inv_w;
      sc_out[i] = sc;
      const bool win = is_window_pos(wa, pos_of(i));
      key[i] = win ? kWindowKey : (__float_as_uint(sc) & 0x7FFFFFFFu);
    }
    if (pool > 1) {
      __syncthreads();                         // this CTA's scores are visible to all of its threads
      for (int i = tid; i < L; i += 1024)
        if (key[i] != kWindowKey) list[i] = (int)pooled_key(sc_out, i, L, pool);
      __syncthreads();
      for (int i = tid; i < L; i += 1024)
        if (key[i] != kWindowKey) key[i] = (uint32_t)list[i];
    }
  } else {
    for (int i = tid; i < L; i += 1024) {
      const int pos = pos_of(i);
      key[i] = pos < n_sink ? kWindowKey : (uint32_t)pos + 1u;
    }
  }
  __syncthreads();

  // ---- phase 2: selection
  if (slice_budget != nullptr) budget = slice_budget[slice];
  int want;
  const int kept = select_and_emit(key, L, budget, list, sh, &want);
  if (kept != want) {                          // the count rule of the selection (block-uniform)
    if (tid == 0) atomicExch(lv.status, kDevCheck);
    return;
  }
  __syncthreads();

  // ---- phase 3: in-place gather of K, V and pos
  const int ppr = lv.row_bytes >> 4;           // 16-byte pieces per row
  const int per_row = 2 * ppr;                 // K pieces, then V pieces
  const int r_step = 1024 / per_row;           // rows per sweep of the CTA
  const int C = 8 * r_step;                    // rows per chunk
  int lo = 0, hi = kept;                       // first j with keep[j] != j
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (list[mid] == mid) lo = mid + 1; else hi = mid;
  }
  if (ext.on && lo > hist) lo = hist;          // kept rows of the current map are not where they belong yet, whatever their index
  const int r_in = tid / per_row, c = tid % per_row;
  const char *ext_ptr = c < ppr ? ext.k : ext.v;
  char *pool_ptr = c < ppr ? lv.k_pool : lv.v_pool;
  const int piece = c < ppr ? c : c - ppr;
  const bool pos_thread = c == 0;
  if (r_in < r_step) {
    for (int c0 = lo; c0 < kept; c0 += C) {
      uint4 buf[8];
      int pv[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int j = c0 + r_in + u * r_step;
        if (j < kept) {
          const int src = list[j];
          if (ext.on && src >= hist) {
            const long long e = (ext_base + (long long)(src - hist) * ext.st) * ext.esize;
            buf[u] = __ldg(reinterpret_cast<const uint4 *>(ext_ptr + e) + piece);
            if (pos_thread) pv[u] = wa.n_prev + (src - hist);
          } else {
            const size_t row = row_of(src);
            buf[u] = reinterpret_cast<const uint4 *>(pool_ptr + row * lv.row_bytes)[piece];
            if (pos_thread) pv[u] = lv.pos_pool[row];
          }
        }
      }
      __syncthreads();
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int j = c0 + r_in + u * r_step;
        if (j < kept) {
          const size_t row = row_of(j);
          reinterpret_cast<uint4 *>(pool_ptr + row * lv.row_bytes)[piece] = buf[u];
          if (pos_thread) lv.pos_pool[row] = pv[u];
        }
      }
    }
  } else {
    for (int c0 = lo; c0 < kept; c0 += C) __syncthreads();     // keeps the barrier count of the working threads
  }
  if (tid == 0) {
    lv.hist_len[slice] = kept;
    kept_count[slice] = kept;
  }
}

// ------------------------------------------------------------------------------------------
// layer statistics (Eq. 2): for sampled query rows i of the current map, alpha_i = softmax row over all L
// entries, c_i = mass on the current map, t_i = sum of the K' largest alpha_ij over the history.
// A CTA of 256 threads owns 64 sampled rows of one slice and streams a range of the slice's keys in tiles of
// 64, so a key tile is read once for 64 rows.  Per tile: logits by fp32 FMA (thread (ty, tx) owns rows
// ty + 16 i, columns tx + 16 j), staged in shared memory; then four threads per row, 16 columns each, fold the
// tile into the row's running maximum, normaliser and current-map mass (online softmax statistics) and into
// their own descending list of the K' largest history logits seen in their columns (the K' largest weights
// are the K' largest logits).  Nothing of length L is kept.  At the end one thread per row merges the four
// lists (K' steps of a four-way merge).
// The calibration runs few slices (one image), so the keys of a slice are split over gridDim.z CTAs to fill
// the GPU: with one split the block adds its rows' c_i and t_i to the accumulators itself; with several every
// CTA writes, per row, (maximum, normaliser, current mass, K' largest logits) to `partial` and
// layer_stats_merge_kernel combines the splits.
// grid (ceil(n_rows / 64), n_slices, n_split); dynamic shared memory: layer_stats_smem_bytes<D>(K').
// ------------------------------------------------------------------------------------------
template <int D> __host__ __device__ constexpr size_t layer_stats_smem_bytes(int topk) {
  return (size_t)(2 * 64 * (D + 4) + 64 * 65 + 64 + 256 * (topk > 0 ? topk : 1)) * 4;
}
constexpr int kStatsRec = 4 + 64;        // floats per (split, row) record: m, z, cur, unused, then up to 64 logits

__device__ __forceinline__ void stats_block_accumulate(float c_i, float t_i, double *acc, float *red_c, float *red_t) {
  const int tid = threadIdx.x;
  for (int o = 16; o > 0; o >>= 1) {
    c_i += __shfl_xor_sync(0xffffffffu, c_i, o);
    t_i += __shfl_xor_sync(0xffffffffu, t_i, o);
  }
  if ((tid & 31) == 0) { red_c[tid >> 5] = c_i; red_t[tid >> 5] = t_i; }
  __syncthreads();
  if (tid == 0) {
    float cs = 0.f, ts = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { cs += red_c[w]; ts += red_t[w]; }   // fixed order
    atomicAdd(&acc[0], (double)cs);
    atomicAdd(&acc[1], (double)ts);
    // the same sums per slice, behind the two totals
    atomicAdd(&acc[2 + 2 * blockIdx.y], (double)cs);
    atomicAdd(&acc[3 + 2 * blockIdx.y], (double)ts);
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(256) layer_stats_kernel(LayerView lv, TensorView Q, int n_k, int n_prev, int stride, int n_rows,
                                                          int topk_prime, float scale, double *acc, float *partial) {
  constexpr int LD = D + 4, LDS = 65;
  constexpr int CH = D * (int)sizeof(T) / 16;
  constexpr int VN = Vec16<T>::N;
  extern __shared__ float smem[];
  float *Qs = smem;                    // [64][LD]
  float *Ks = Qs + 64 * LD;            // [64][LD]
  float *Ss = Ks + 64 * LD;            // [64][LDS] scaled logits of the tile
  int *is_cur = reinterpret_cast<int *>(Ss + 64 * LDS);   // [64] the tile's entries that belong to the current map
  float *top = reinterpret_cast<float *>(is_cur + 64);    // [256][K'] per-thread descending lists
  __shared__ float red_c[8], red_t[8];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int slice = blockIdx.y;
  const int b = slice / lv.n_heads, h = slice % lv.n_heads;
  const int L = lv.hist_len[slice] + n_k;
  const int r0 = blockIdx.x * 64;
  const int Kp = topk_prime;
  const int n_split = gridDim.z;
  const int tiles = (L + 63) >> 6;
  const int t_lo = (int)((long long)tiles * blockIdx.z / n_split), t_hi = (int)((long long)tiles * (blockIdx.z + 1) / n_split);
  for (int idx = tid; idx < 64 * CH; idx += 256) {
    const int r = idx / CH, c = idx % CH;
    float v[VN];
    if (r0 + r < n_rows) {
      Vec16<T>::load(row_ptr<T>(Q, b, h, (r0 + r) * stride) + c * VN, v);
    } else {
#pragma unroll
      for (int e = 0; e < VN; ++e) v[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < VN; ++e) Qs[r * LD + c * VN + e] = v[e];
  }
  const int Ks_ = Kp > 0 ? Kp : 1;
  float *mine = top + (size_t)tid * Ks_;
  for (int e = 0; e < Kp; ++e) mine[e] = -INFINITY;
  // row statistics of the 4 threads that share a row (row = tid >> 2): kept redundantly in each of them
  const int row = tid >> 2, part = tid & 3;
  float m_run = -INFINITY, z_run = 0.f, cur_run = 0.f;
  float thr = Kp > 0 ? -INFINITY : INFINITY;           // the smallest member of this thread's list (nothing enters when K' = 0)
  // the next key tile (and its positions) travels from global memory into registers while the current one is worked on
  constexpr int PIECES = 64 * CH / 256;                // 16-byte pieces of a tile per thread
  uint4 nxt[PIECES];
  int nxt_pos = 0;
  auto fetch = [&](int t) {
    const int j0 = t << 6;
#pragma unroll
    for (int u = 0; u < PIECES; ++u) {
      const int idx = tid + u * 256, r = idx / CH, c = idx % CH;
      nxt[u] = make_uint4(0u, 0u, 0u, 0u);
      if (j0 + r < L) nxt[u] = reinterpret_cast<const uint4 *>(lv.k_pool + slot_row(lv, slice, j0 + r) * lv.row_bytes)[c];
    }
    if (tid < 64) nxt_pos = (j0 + tid < L) ? lv.pos_pool[slot_row(lv, slice, j0 + tid)] : -1;
  };
  if (t_lo < t_hi) fetch(t_lo);
  for (int t = t_lo; t < t_hi; ++t) {
    const int j0 = t << 6;
    __syncthreads();
#pragma unroll
    for (int u = 0; u < PIECES; ++u) {
      const int idx = tid + u * 256, r = idx / CH, c = idx % CH;
      float v[VN];
      Vec16<T>::load(reinterpret_cast<const T *>(&nxt[u]), v);
#pragma unroll
      for (int e = 0; e < VN; e += 4)                  // 16-byte stores (LD and VN are multiples of 4)
        *reinterpret_cast<float4 *>(&Ks[r * LD + c * VN + e]) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
    }
    if (tid < 64) is_cur[tid] = nxt_pos >= n_prev ? 1 : 0;
    __syncthreads();
    if (t + 1 < t_hi) fetch(t + 1);
    float s[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 4
    for (int c = 0; c < D; c += 4) {
      float4 q[4], k[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) q[i] = *reinterpret_cast<const float4 *>(&Qs[(ty + 16 * i) * LD + c]);
#pragma unroll
      for (int j = 0; j < 4; ++j) k[j] = *reinterpret_cast<const float4 *>(&Ks[(tx + 16 * j) * LD + c]);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          s[i][j] = fmaf(q[i].x, k[j].x, s[i][j]);
          s[i][j] = fmaf(q[i].y, k[j].y, s[i][j]);
          s[i][j] = fmaf(q[i].z, k[j].z, s[i][j]);
          s[i][j] = fmaf(q[i].w, k[j].w, s[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j)
        Ss[(ty + 16 * i) * LDS + tx + 16 * j] = (j0 + tx + 16 * j < L) ? s[i][j] * scale : -INFINITY;
    __syncthreads();
    {
      const float *srow = Ss + row * LDS + part * 16;
      float mx = -INFINITY;
#pragma unroll
      for (int e = 0; e < 16; ++e) mx = fmaxf(mx, srow[e]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run, mx);            // finite: every tile holds at least one entry
      float sum = 0.f, cur = 0.f;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const float v = srow[e];
        const float pe = expf(v - m_new);              // 0 for the padding beyond L
        sum += pe;
        if (is_cur[part * 16 + e]) {
          cur += pe;
        } else if (v > thr) {                          // a history logit that enters this thread's K' largest
          int at = Kp - 1;
          while (at > 0 && mine[at - 1] < v) { mine[at] = mine[at - 1]; --at; }
          mine[at] = v;
          thr = mine[Kp - 1];
        }
      }
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      cur += __shfl_xor_sync(0xffffffffu, cur, 1);
      cur += __shfl_xor_sync(0xffffffffu, cur, 2);
      const float a = expf(m_run - m_new);             // 0 at the first tile
      z_run = z_run * a + sum;
      cur_run = cur_run * a + cur;
      m_run = m_new;
    }
  }
  __syncthreads();
  float c_i = 0.f, t_i = 0.f;
  if (part == 0) {
    // four-way merge of the row's four descending lists: the K' largest history logits of this key range
    const float *l0 = top + (size_t)(tid + 0) * Ks_, *l1 = top + (size_t)(tid + 1) * Ks_;
    const float *l2 = top + (size_t)(tid + 2) * Ks_, *l3 = top + (size_t)(tid + 3) * Ks_;
    float *rec = nullptr;
    if (n_split > 1) {
      rec = partial + ((((size_t)slice * gridDim.x + blockIdx.x) * n_split + blockIdx.z) * 64 + row) * kStatsRec;
      rec[0] = m_run; rec[1] = z_run; rec[2] = cur_run;
    }
    int i0 = 0, i1 = 0, i2 = 0, i3 = 0;
    float tsum = 0.f;
    for (int e = 0; e < Kp; ++e) {
      const float v0 = i0 < Kp ? l0[i0] : -INFINITY, v1 = i1 < Kp ? l1[i1] : -INFINITY;
      const float v2 = i2 < Kp ? l2[i2] : -INFINITY, v3 = i3 < Kp ? l3[i3] : -INFINITY;
      const float best = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
      if (rec) rec[4 + e] = best;                      // (-inf once the range's history is exhausted)
      if (best == -INFINITY) { if (!rec) break; else continue; }
      tsum += expf(best - m_run);
      if (best == v0) ++i0; else if (best == v1) ++i1; else if (best == v2) ++i2; else ++i3;
    }
    if (r0 + row < n_rows) { c_i = cur_run / z_run; t_i = tsum / z_run; }
  }
  if (n_split == 1) stats_block_accumulate(c_i, t_i, acc, red_c, red_t);
}

// Combines the key-range splits of layer_stats_kernel: per row the maxima, normalisers and current masses by
// the usual rescaling, the K' largest history logits by an n_split-way merge of the splits' descending lists.
// grid (ceil(n_rows / 64), n_slices), 64 threads, one row per thread.
__global__ void __launch_bounds__(64) layer_stats_merge_kernel(const float *partial, int n_split, int n_rows, int topk_prime,
                                                               double *acc) {
  __shared__ float red_c[2], red_t[2];
  const int row = threadIdx.x;
  const float *base = partial + (((size_t)blockIdx.y * gridDim.x + blockIdx.x) * n_split * 64 + row) * kStatsRec;
  const size_t step = (size_t)64 * kStatsRec;          // from one split's record of this row to the next
  float m = -INFINITY;
  for (int s = 0; s < n_split; ++s) m = fmaxf(m, base[s * step]);
  float z = 0.f, cur = 0.f;
  for (int s = 0; s < n_split; ++s) {
    const float a = expf(base[s * step] - m);
    z += base[s * step + 1] * a;
    cur += base[s * step + 2] * a;
  }
  int head[16];
  for (int s = 0; s < 16; ++s) head[s] = 0;
  float tsum = 0.f;
  for (int e = 0; e < topk_prime; ++e) {
    float best = -INFINITY;
    int who = -1;
    for (int s = 0; s < n_split; ++s) {
      const float v = head[s] < topk_prime ? base[s * step + 4 + head[s]] : -INFINITY;
      if (v > best) { best = v; who = s; }
    }
    if (who < 0) break;                                // history exhausted
    tsum += expf(best - m);
    ++head[who];
  }
  float c_i = 0.f, t_i = 0.f;
  if (blockIdx.x * 64 + row < n_rows) { c_i = cur / z; t_i = tsum / z; }
  stats_block_accumulate(c_i, t_i, acc, red_c, red_t);
}

}  // namespace scalekv
