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
// score, step 1: scaled logits of the window rows against a tile of 64 cache entries (Eq. 5).
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
      if (col < L) logits[((size_t)slice * wa.w + r) * ld_l + col] = s[i][j] * scale;
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

// score, step 2: row-wise softmax normalisers, then s_i = (1/w) sum_j exp(z_ji - m_j) / Z_j
// (Eq. 5 and the aggregation paragraph).  grid (n_slices), 512 threads.
__global__ void __launch_bounds__(512) score_reduce_kernel(LayerView lv, WindowArg wa, const float *logits, int ld_l,
                                                           float *scores, int ld_s) {
  __shared__ float red[16];
  __shared__ float m_row[kMaxWindow], inv_row[kMaxWindow];
  const int slice = blockIdx.x;
  const int L = lv.hist_len[slice] + wa.n_k;
  const float *z = logits + (size_t)slice * wa.w * ld_l;
  for (int j = 0; j < wa.w; ++j) {
    float mx = -INFINITY;
    for (int i = threadIdx.x; i < L; i += blockDim.x) mx = fmaxf(mx, z[(size_t)j * ld_l + i]);
    mx = block_reduce_max(mx, red);
    float sum = 0.f;
    for (int i = threadIdx.x; i < L; i += blockDim.x) sum += expf(z[(size_t)j * ld_l + i] - mx);
    sum = block_reduce_sum(sum, red);
    if (threadIdx.x == 0) { m_row[j] = mx; inv_row[j] = 1.f / (sum * (float)wa.w); }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < L; i += blockDim.x) {
    float s = 0.f;
    for (int j = 0; j < wa.w; ++j) s += expf(z[(size_t)j * ld_l + i] - m_row[j]) * inv_row[j];
    scores[(size_t)slice * ld_s + i] = s;
  }
}

// ------------------------------------------------------------------------------------------
// select: per-slice top-k' of the non-window entries by score (Sec. 3.3), radix-select on the
// float bit patterns (scores are >= 0, so the patterns order like the values), ties by lowest
// slot = lowest original position.  Emits the ascending slot list of survivors (selected U
// window) and its length.  grid (n_slices), 1024 threads.
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

__global__ void __launch_bounds__(1024) select_kernel(LayerView lv, WindowArg wa, int budget, const float *scores,
                                                      int ld_s, uint32_t *keys, int *keep_list, int *kept_count) {
  __shared__ int hist[256];
  __shared__ int warp_sums[33];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining;
  const int slice = blockIdx.x;
  const int L = lv.hist_len[slice] + wa.n_k;
  uint32_t *key = keys + (size_t)slice * ld_s;
  int *out = keep_list + (size_t)slice * ld_s;

  // pass 0: keys; window entries get a sentinel and never take part in the selection
  int n_win_local = 0;
  for (int i = threadIdx.x; i < L; i += blockDim.x) {
    const int p = lv.pos_pool[slot_row(lv, slice, i)];
    const bool win = is_window_pos(wa, p);
    key[i] = win ? kWindowKey : (__float_as_uint(scores[(size_t)slice * ld_s + i]) & 0x7FFFFFFFu);
    n_win_local += win ? 1 : 0;
  }
  int n_win;
  block_exclusive_scan(n_win_local, warp_sums, &n_win);
  const int cand = L - n_win;
  const int kprime = (budget < 0 || budget > cand) ? cand : budget;

  // radix select of the kprime-th largest key, 8 bits per pass from the top
  uint32_t threshold = 0;
  int n_ties_taken = 0;       // how many entries equal to the threshold are kept
  if (kprime > 0 && kprime < cand) {
    if (threadIdx.x == 0) { sh_prefix = 0; sh_remaining = kprime; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      const uint32_t mask_hi = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
      if (threadIdx.x < 256) hist[threadIdx.x] = 0;
      __syncthreads();
      const uint32_t prefix = sh_prefix;
      for (int i = threadIdx.x; i < L; i += blockDim.x) {
        const uint32_t k = key[i];
        if (k != kWindowKey && (k & mask_hi) == prefix) atomicAdd(&hist[(k >> shift) & 0xFF], 1);
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        int rem = sh_remaining;
        int dsel = 0;
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
  const bool keep_all = (kprime >= cand);
  const bool keep_none = (kprime == 0);

  // ordered emit
  int base_out = 0, base_tie = 0;
  for (int i0 = 0; i0 < L; i0 += blockDim.x) {
    const int i = i0 + threadIdx.x;
    uint32_t k = 0;
    bool win = false, gt = false, tie = false;
    if (i < L) {
      k = key[i];
      win = (k == kWindowKey);
      if (!win) {
        if (keep_all) gt = true;
        else if (!keep_none) { gt = k > threshold; tie = (k == threshold); }
      }
    }
    int tie_total, keep_total;
    const int tie_rank = base_tie + block_exclusive_scan(tie ? 1 : 0, warp_sums, &tie_total);
    const bool keep = win || gt || (tie && tie_rank < n_ties_taken);
    const int oidx = base_out + block_exclusive_scan(keep ? 1 : 0, warp_sums, &keep_total);
    if (keep) out[oidx] = i;
    base_tie += tie_total;
    base_out += keep_total;
  }
  if (threadIdx.x == 0) kept_count[slice] = base_out;
}

// ------------------------------------------------------------------------------------------
// compact: slot j <- old slot keep[j], in place, for K (blockIdx.y = 0, also pos) and V
// (blockIdx.y = 1).  keep is ascending, so keep[j] >= j: within a chunk every source is read
// before any destination is written, and the sources of later chunks lie beyond every earlier
// destination.  grid (n_slices, 2), 256 threads, 16-byte pieces (Sec. 3.3, pruning).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) compact_kernel(LayerView lv, const int *keep_list, int ld_s, const int *kept_count) {
  const int slice = blockIdx.x;
  const int which = blockIdx.y;
  char *pool = which == 0 ? lv.k_pool : lv.v_pool;
  const int *list = keep_list + (size_t)slice * ld_s;
  const int kept = kept_count[slice];
  const int ppr = lv.row_bytes >> 4;
  const int C = 1024 / ppr;        // rows per chunk (4 pieces per thread)
  int lo = 0, hi = kept;           // first j with keep[j] != j (the untouched prefix is skipped)
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (list[mid] == mid) lo = mid + 1; else hi = mid;
  }
  for (int c0 = lo; c0 < kept; c0 += C) {
    uint4 buf[4];
    int pv = 0;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int piece = threadIdx.x + u * 256;
      const int r = piece / ppr, c = piece % ppr;
      const int j = c0 + r;
      if (r < C && j < kept) {
        const size_t row = slot_row(lv, slice, list[j]);
        buf[u] = reinterpret_cast<const uint4 *>(pool + row * lv.row_bytes)[c];
      }
    }
    const bool do_pos = (which == 0) && ((int)threadIdx.x < C) && (c0 + (int)threadIdx.x < kept);
    if (do_pos) pv = lv.pos_pool[slot_row(lv, slice, list[c0 + threadIdx.x])];
    __syncthreads();
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int piece = threadIdx.x + u * 256;
      const int r = piece / ppr, c = piece % ppr;
      const int j = c0 + r;
      if (r < C && j < kept) {
        const size_t row = slot_row(lv, slice, j);
        reinterpret_cast<uint4 *>(pool + row * lv.row_bytes)[c] = buf[u];
      }
    }
    if (do_pos) lv.pos_pool[slot_row(lv, slice, c0 + threadIdx.x)] = pv;
  }
  if (which == 0 && threadIdx.x == 0) lv.hist_len[slice] = kept;
}

// ------------------------------------------------------------------------------------------
// layer statistics (Eq. 2): one block per (sampled query row, slice).  The softmax row is held
// in shared memory; c = mass on the current map, t = sum of the K' largest history weights.
// grid (n_rows, n_slices), 256 threads, dynamic smem = (L + D) floats.
// ------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(256) layer_stats_kernel(LayerView lv, TensorView Q, int n_k, int n_prev, int stride,
                                                          int topk_prime, float scale, double *acc) {
  extern __shared__ float smem[];
  __shared__ float red[8];
  __shared__ float best_v[8];
  __shared__ int best_i[8];
  float *qs = smem;          // [D]
  float *p = smem + D;       // [L]
  constexpr int VN = Vec16<T>::N;
  constexpr int CH = D * (int)sizeof(T) / 16;
  const int slice = blockIdx.y;
  const int b = slice / lv.n_heads, h = slice % lv.n_heads;
  const int qi = blockIdx.x * stride;
  const int L = lv.hist_len[slice] + n_k;
  if (threadIdx.x < CH) {
    float v[VN];
    Vec16<T>::load(row_ptr<T>(Q, b, h, qi) + threadIdx.x * VN, v);
#pragma unroll
    for (int e = 0; e < VN; ++e) qs[threadIdx.x * VN + e] = v[e];
  }
  __syncthreads();
  float mx = -INFINITY;
  for (int i = threadIdx.x; i < L; i += blockDim.x) {
    const size_t row = slot_row(lv, slice, i);
    const T *kr = reinterpret_cast<const T *>(lv.k_pool + row * lv.row_bytes);
    float dot = 0.f;
#pragma unroll 4
    for (int c = 0; c < CH; ++c) {
      float v[VN];
      Vec16<T>::load(kr + c * VN, v);
#pragma unroll
      for (int e = 0; e < VN; ++e) dot = fmaf(qs[c * VN + e], v[e], dot);
    }
    dot *= scale;
    p[i] = dot;
    mx = fmaxf(mx, dot);
  }
  mx = block_reduce_max(mx, red);
  float sum = 0.f;
  for (int i = threadIdx.x; i < L; i += blockDim.x) {
    const float e = expf(p[i] - mx);
    p[i] = e;
    sum += e;
  }
  sum = block_reduce_sum(sum, red);
  const float inv = 1.f / sum;
  float cur = 0.f;
  for (int i = threadIdx.x; i < L; i += blockDim.x) {
    const int ps = lv.pos_pool[slot_row(lv, slice, i)];
    const float a = p[i] * inv;
    if (ps >= n_prev) { cur += a; p[i] = -1.f; } else { p[i] = a; }
  }
  cur = block_reduce_sum(cur, red);
  float top = 0.f;
  for (int round = 0; round < topk_prime; ++round) {
    float bv = -1.f;
    int bi = -1;
    for (int i = threadIdx.x; i < L; i += blockDim.x)
      if (p[i] > bv) { bv = p[i]; bi = i; }
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi >= 0 && (bi < 0 || oi < bi))) { bv = ov; bi = oi; }
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { best_v[threadIdx.x >> 5] = bv; best_i[threadIdx.x >> 5] = bi; }
    __syncthreads();
    bv = best_v[0]; bi = best_i[0];
    for (int w = 1; w < 8; ++w)
      if (best_v[w] > bv || (best_v[w] == bv && best_i[w] >= 0 && (bi < 0 || best_i[w] < bi))) { bv = best_v[w]; bi = best_i[w]; }
    if (bi < 0 || bv < 0.f) break;   // history exhausted (uniform across the block)
    top += bv;
    __syncthreads();
    if (threadIdx.x == 0) p[bi] = -1.f;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    atomicAdd(&acc[0], (double)cur);
    atomicAdd(&acc[1], (double)top);
  }
}

// rows window_pos[j] of a dense [B*H][n_k][d] tensor -> dense [B*H][w][d] (16-byte pieces)
__global__ void gather_rows_kernel(const char *src, char *dst, WindowArg wa, int row_bytes, int n_slices) {
  const int ppr = row_bytes >> 4;
  const long long total = (long long)n_slices * wa.w * ppr;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % ppr);
    const long long rj = idx / ppr;
    const int j = (int)(rj % wa.w);
    const long long sl = rj / wa.w;
    const int qi = wa.all ? j : wa.pos[j];
    reinterpret_cast<uint4 *>(dst + (sl * wa.w + j) * row_bytes)[c] =
        reinterpret_cast<const uint4 *>(src + (sl * wa.n_k + qi) * row_bytes)[c];
  }
}

}  // namespace scalekv
