// CUDA-core pipeline of the verification step: any shape, f32 or bf16 storage, fp32
// arithmetic. It is the variant for shapes the tensor-core kernels do not cover (fp32
// heads, ragged d) and the on-device second opinion the tests compare the fused kernels
// with. Its stages that do not touch W (draft statistics, judge dot products, decision,
// token location) are shared with the batched tensor-core variant.
#include <algorithm>

#include "jd_kernels.h"

namespace jd {

// -----------------------------------------------------------------------------------------
// Stage 1: logits of a [128 vocab] x [16 rows] tile by smem-tiled FMA.
//   kMode 0: per-(row, vocab tile) softmax partials + gather of L[row, x_j]
//   kMode 1: rows are the selected rows (one per sequence); writes the sampling weights and p
//            of that row plus their per-tile masses
//   kMode 2: top-K rule, after the fold: counts the entries of every row that rank above the
//            drafted token and records the lowest token id that attains the row maximum. The
//            logits are recomputed with the same instruction sequence as in mode 0, so they are
//            bit-identical to the gathered logit and to the folded maximum.
// -----------------------------------------------------------------------------------------
constexpr int kSimtRows = 16;
constexpr int kSimtK = 32;

template <typename T, int kMode>
__global__ void __launch_bounds__(kVocabTile) simt_logits_kernel(CallParams cp, Workspace ws, const T* __restrict__ W,
                                                                 const T* __restrict__ H, int R, int np,
                                                                 float* __restrict__ logits_debug,
                                                                 const float* __restrict__ w_scale) {
  __shared__ float sW[kVocabTile][kSimtK + 1];
  __shared__ __align__(16) float sH[kSimtRows][kSimtK];
  __shared__ float s_m[4][kSimtRows], s_s[4][kSimtRows];
  __shared__ double s_d[2][4][kSimtRows];
  __shared__ int s_row[kSimtRows];
  __shared__ float s_scale[kSimtRows];

  constexpr bool kSample = (kMode == 1);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile = blockIdx.x;
  const int v = tile * kVocabTile + tid;
  const int r0 = blockIdx.y * kSimtRows;
  const int d = cp.d, V = cp.V;

  if (tid < kSimtRows) {
    const int r = r0 + tid;
    s_row[tid] = (r < R) ? (kSample ? ws.sel_row[r] : r) : -1;
    s_scale[tid] = (cp.norm == JD_NORM_RMS && s_row[tid] >= 0) ? ws.row_scale[s_row[tid]] : 1.f;
    if (w_scale && s_row[tid] >= 0) s_scale[tid] *= ws.h_scale[s_row[tid]];   // FP8 head: scale of the quantised row
  }
  __syncthreads();

  float acc[kSimtRows];
#pragma unroll
  for (int i = 0; i < kSimtRows; ++i) acc[i] = 0.f;

  for (int k0 = 0; k0 < d; k0 += kSimtK) {
    // W tile: 128 rows x 32 k, coalesced along k
    for (int i = tid; i < kVocabTile * kSimtK; i += kVocabTile) {
      const int rr = i / kSimtK, kk = i % kSimtK;
      const int vv = tile * kVocabTile + rr;
      sW[rr][kk] = (vv < V && k0 + kk < d) ? to_float<T>(W[(size_t)vv * d + k0 + kk]) : 0.f;
    }
    for (int i = tid; i < kSimtRows * kSimtK; i += kVocabTile) {
      const int rr = i / kSimtK, kk = i % kSimtK;
      const int row = s_row[rr];
      sH[rr][kk] = (row >= 0 && k0 + kk < d) ? to_float<T>(H[(size_t)row * d + k0 + kk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kSimtK; kk += 4) {
      const float w0 = sW[tid][kk], w1 = sW[tid][kk + 1], w2 = sW[tid][kk + 2], w3 = sW[tid][kk + 3];
#pragma unroll
      for (int i = 0; i < kSimtRows; ++i) {
        const float4 h = *reinterpret_cast<const float4*>(&sH[i][kk]);
        acc[i] = fmaf(w0, h.x, acc[i]);
        acc[i] = fmaf(w1, h.y, acc[i]);
        acc[i] = fmaf(w2, h.z, acc[i]);
        acc[i] = fmaf(w3, h.w, acc[i]);
      }
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < kSimtRows; ++i) acc[i] *= s_scale[i];   // 1 when no normalisation is asked for
  if (w_scale) {   // FP8 head: scale of this thread's vocabulary row
    const float sv = v < V ? w_scale[v] : 0.f;
#pragma unroll
    for (int i = 0; i < kSimtRows; ++i) acc[i] *= sv;
  }

  const bool valid_v = v < V;
  if (kMode == 2) {
#pragma unroll
    for (int i = 0; i < kSimtRows; ++i) {
      const int row = s_row[i];
      bool above = false;
      if (row >= 0) {
        const int b = row / (cp.M + 1), j = row % (cp.M + 1);
        if (valid_v && acc[i] == ws.row_max[row]) atomicMin(ws.argidx + row, v);
        if (j < cp.M && valid_v) {
          const int x = min(max(cp.draft_tokens[b * cp.M + j], 0), V - 1);
          const float g = ws.gath[row];
          above = acc[i] > g || (acc[i] == g && v < x);
        }
      }
      const unsigned mask = __ballot_sync(0xffffffffu, above);
      if (lane == 0 && mask) atomicAdd(ws.cnt + row, __popc(mask));
    }
  } else if (!kSample) {
#pragma unroll
    for (int i = 0; i < kSimtRows; ++i) {
      const int row = s_row[i];
      float m = (valid_v && row >= 0) ? acc[i] : -INFINITY;
      float s = (valid_v && row >= 0) ? 1.f : 0.f;
      ms_warp_reduce(m, s);
      if (lane == 0) { s_m[warp][i] = m; s_s[warp][i] = s; }
      if (row >= 0 && valid_v) {
        if (logits_debug) logits_debug[(size_t)row * V + v] = acc[i];
        const int b = row / (cp.M + 1), j = row % (cp.M + 1);
        if (j < cp.M) {
          int x = cp.draft_tokens[b * cp.M + j];
          if (x < 0 || x >= V) { set_status(ws.status, JD_ERR_BAD_TOKEN); x = min(max(x, 0), V - 1); }
          if (x == v) ws.gath[row] = acc[i];
        }
      }
    }
    __syncthreads();
    if (tid < kSimtRows && s_row[tid] >= 0) {
      float m = s_m[0][tid], s = s_s[0][tid];
      for (int w = 1; w < 4; ++w) ms_combine(m, s, s_m[w][tid], s_s[w][tid]);
      ws.part_max[(size_t)s_row[tid] * np + tile] = m;
      ws.part_sum[(size_t)s_row[tid] * np + tile] = s;
    }
  } else {
#pragma unroll
    for (int i = 0; i < kSimtRows; ++i) {
      const int row = s_row[i];
      const int b = r0 + i;
      float p = 0.f, r = 0.f;
      if (row >= 0 && valid_v) {
        const int kind = ws.sel_kind[b];
        const int a = row % (cp.M + 1);
        const float dlv = (kind == 0) ? cp.draft_logits[((size_t)b * cp.M + a) * V + v] : 0.f;
        sample_weights(acc[i], ws.sel_lse_p[b], kind, dlv, ws.sel_lse_q[b], p, r);
        ws.w_sel[(size_t)b * V + v] = r;
        ws.p_sel[(size_t)b * V + v] = p;
      }
      const double dr = warp_sum_double((double)r), dp = warp_sum_double((double)p);
      if (lane == 0) { s_d[0][warp][i] = dr; s_d[1][warp][i] = dp; }
    }
    __syncthreads();
    if (tid < kSimtRows && s_row[tid] >= 0) {
      const int b = r0 + tid;
      ws.mass_r[(size_t)b * np + tile] = (s_d[0][0][tid] + s_d[0][1][tid]) + (s_d[0][2][tid] + s_d[0][3][tid]);
      ws.mass_p[(size_t)b * np + tile] = (s_d[1][0][tid] + s_d[1][1][tid]) + (s_d[1][2][tid] + s_d[1][3][tid]);
    }
  }
}

// -----------------------------------------------------------------------------------------
// Draft-row statistics: per (draft row, chunk) online (max, sum exp) and the gather of the
// drafted token's logit. One block per chunk of kQChunk logits.
// -----------------------------------------------------------------------------------------
constexpr int kQChunk = 8192;

__global__ void __launch_bounds__(256) q_stats_kernel(CallParams cp, Workspace ws, int nq) {
  __shared__ float s_m[8], s_s[8];
  const int bm = blockIdx.y, chunk = blockIdx.x;
  const int V = cp.V;
  const float* row = cp.draft_logits + (size_t)bm * V;
  const int lo = chunk * kQChunk, hi = min(V, lo + kQChunk);
  float m = -INFINITY, s = 0.f;
  if (cp.dl_vec4) {
    // rows start on 16-byte boundaries: every thread fetches its eight float4 of the chunk before any
    // arithmetic, then takes the maximum and the sum of exponentials from registers
    float4 x[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int v = lo + (u * 256 + threadIdx.x) * 4;
      x[u] = v < hi ? __ldg(reinterpret_cast<const float4*>(row + v))
                    : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) m = fmaxf(m, fmaxf(fmaxf(x[u].x, x[u].y), fmaxf(x[u].z, x[u].w)));
    if (m > -INFINITY) {
#pragma unroll
      for (int u = 0; u < 8; ++u)
        s += (__expf(x[u].x - m) + __expf(x[u].y - m)) + (__expf(x[u].z - m) + __expf(x[u].w - m));
    }
  } else {
    for (int v = lo + threadIdx.x; v < hi; v += blockDim.x) {
      const float xv = row[v];
      if (xv > m) { s = s * __expf(m - xv) + 1.f; m = xv; }
      else if (xv != -INFINITY) s += __expf(xv - m);
    }
  }
  ms_warp_reduce(m, s);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { s_m[warp] = m; s_s[warp] = s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) ms_combine(m, s, s_m[w], s_s[w]);
    ws.qpart_max[(size_t)bm * nq + chunk] = m;
    ws.qpart_sum[(size_t)bm * nq + chunk] = s;
    if (chunk == 0) {
      int x = cp.draft_tokens[bm];
      if (x < 0 || x >= V) { set_status(ws.status, JD_ERR_BAD_TOKEN); x = min(max(x, 0), V - 1); }
      ws.qgath[bm] = row[x];
    }
  }
}

// FP8 head: quantises every row of H to E4M3 with one scale per row, s = amax / 448 and
// code = e4m3(h * 448 / amax), round to nearest even, saturating. h * 448 is exact in float32 for a
// bf16 h (8 + 3 significant bits) and the division rounds once, to 24 bits; a quotient of two bf16
// values that is not itself a half-way point of the E4M3 grid stays at least 2^-14 (relative) away
// from one, so the second rounding, to E4M3, picks the code the exact quotient would.
__device__ __forceinline__ float e4m3_prescale(float h, float amax, float pre) {
  return __fdiv_rn(__fmul_rn(__fmul_rn(h, pre), 448.f), __fmul_rn(amax, pre));
}
// pre: 2^-64 for rows with a huge amax, so that h * 448 cannot overflow (powers of two: exact)
__device__ __forceinline__ float e4m3_pre(float amax) { return amax > 0x1p100f ? 0x1p-64f : 1.f; }
__global__ void __launch_bounds__(256) quantize_rows_kernel(CallParams cp, Workspace ws,
                                                            const __nv_bfloat16* __restrict__ H) {
  __shared__ float s_p[8];
  __shared__ float s_amax;
  const int row = blockIdx.x;
  const __nv_bfloat16* h = H + (size_t)row * cp.d;
  float amax = 0.f;
  for (int k = threadIdx.x; k < cp.d; k += blockDim.x) amax = fmaxf(amax, fabsf(__bfloat162float(h[k])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) s_p[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < 8; ++i) t = fmaxf(t, s_p[i]);
    s_amax = t;
    ws.h_scale[row] = __fdiv_rn(t, 448.f);
  }
  __syncthreads();
  amax = s_amax;
  const float pre = e4m3_pre(amax);
  const float den = amax > 0.f ? amax : 1.f;   // an all-zero row quantises to zeros
  uint8_t* out = ws.h8 + (size_t)row * cp.d;
  for (int k = 2 * threadIdx.x; k < cp.d; k += 2 * blockDim.x) {
    const float a = e4m3_prescale(__bfloat162float(h[k]), den, pre);
    const float b = k + 1 < cp.d ? e4m3_prescale(__bfloat162float(h[k + 1]), den, pre) : 0.f;
    unsigned short pair;   // upper byte = code of the first operand, lower byte = code of the second
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(b), "f"(a));
    out[k] = (uint8_t)(pair & 0xFF);
    if (k + 1 < cp.d) out[k + 1] = (uint8_t)(pair >> 8);
  }
}

// The same quantisation for d % 8 == 0: the row is read once, eight bf16 per 16-byte load, kept
// in registers across the amax reduction, and written as eight codes per store. kVec = loads
// per thread (blockDim.x * kVec * 8 >= d). Same operations per element as above.
template <int kVec>
__global__ void __launch_bounds__(1024) quantize_rows_vec_kernel(CallParams cp, Workspace ws,
                                                                 const __nv_bfloat16* __restrict__ H) {
  __shared__ float s_p[32];
  __shared__ float s_amax;
  const int row = blockIdx.x, tid = threadIdx.x, nvec = cp.d / 8;
  const uint4* h = reinterpret_cast<const uint4*>(H + (size_t)row * cp.d);
  uint4 v[kVec];
#pragma unroll
  for (int u = 0; u < kVec; ++u) {
    const int idx = tid + u * blockDim.x;
    v[u] = idx < nvec ? __ldg(h + idx) : make_uint4(0u, 0u, 0u, 0u);
  }
  float amax = 0.f;
#pragma unroll
  for (int u = 0; u < kVec; ++u) {
    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {   // a bf16 is the upper half of the float with the same value
      amax = fmaxf(amax, fabsf(__uint_as_float(w[q] << 16)));
      amax = fmaxf(amax, fabsf(__uint_as_float(w[q] & 0xFFFF0000u)));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((tid & 31) == 0) s_p[tid >> 5] = amax;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t = fmaxf(t, s_p[i]);
    s_amax = t;
    ws.h_scale[row] = __fdiv_rn(t, 448.f);
  }
  __syncthreads();
  amax = s_amax;
  const float pre = e4m3_pre(amax);
  const float den = amax > 0.f ? amax : 1.f;   // an all-zero row quantises to zeros
  uint2* out = reinterpret_cast<uint2*>(ws.h8 + (size_t)row * cp.d);
#pragma unroll
  for (int u = 0; u < kVec; ++u) {
    const int idx = tid + u * blockDim.x;
    if (idx >= nvec) continue;
    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
    uint32_t pair[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float a = e4m3_prescale(__uint_as_float(w[q] << 16), den, pre);           // element 2q
      const float b = e4m3_prescale(__uint_as_float(w[q] & 0xFFFF0000u), den, pre);   // element 2q + 1
      unsigned short p;   // upper byte = code of the first operand, lower byte = code of the second
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(p) : "f"(b), "f"(a));
      pair[q] = p;
    }
    out[idx] = make_uint2(pair[0] | (pair[1] << 16), pair[2] | (pair[3] << 16));
  }
}

// Row normalisation factors of JD_NORM_RMS: one block per row, 1 / sqrt(mean_k H[row,k]^2 + eps).
template <typename T>
__global__ void __launch_bounds__(256) row_scale_kernel(CallParams cp, Workspace ws, const T* __restrict__ H) {
  __shared__ float s_p[8];
  const int row = blockIdx.x;
  const T* h = H + (size_t)row * cp.d;
  float acc = 0.f;
  for (int k = threadIdx.x; k < cp.d; k += blockDim.x) { const float x = to_float<T>(h[k]); acc = fmaf(x, x, acc); }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) s_p[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < 8; ++i) t += s_p[i];
    ws.row_scale[row] = rsqrtf(t / (float)cp.d + cp.rms_eps);
  }
}

// Judge dot products: one block per draft slot, w . H[b, j+1].
template <typename T>
__global__ void __launch_bounds__(256) judge_dot_kernel(CallParams cp, Workspace ws, const T* __restrict__ H,
                                                        const T* __restrict__ w) {
  __shared__ float s_p[8];
  const int bm = blockIdx.x;
  const int b = bm / cp.M, j = bm % cp.M;
  const T* h = H + ((size_t)b * (cp.M + 1) + j + 1) * cp.d;
  float acc = 0.f;
  for (int k = threadIdx.x; k < cp.d; k += blockDim.x) acc = fmaf(to_float<T>(w[k]), to_float<T>(h[k]), acc);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) s_p[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < 8; ++i) t += s_p[i];
    ws.judge_logit[bm] = t;
  }
}

// -----------------------------------------------------------------------------------------
// Fold of the partial statistics: one warp per target row and per draft row. Each lane fetches
// its share of the row's partials (eight at a time, all loads first), the warp takes the
// maximum, then the rescaled sum; fixed order, so results repeat bit for bit.
// -----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) fold_stats_kernel(CallParams cp, Workspace ws, int np, int nq, int fold_arg) {
  const int lane = threadIdx.x & 31;
  const int R = cp.B * (cp.M + 1), BM = cp.B * cp.M;
  const int it = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (it >= R + BM) return;
  const bool is_p = it < R;
  const int n = is_p ? np : nq;
  const float* pm = is_p ? ws.part_max + (size_t)it * np : ws.qpart_max + (size_t)(it - R) * nq;
  const float* ps = is_p ? ws.part_sum + (size_t)it * np : ws.qpart_sum + (size_t)(it - R) * nq;
  float m = -INFINITY;
  for (int i0 = 0; i0 < n; i0 += 256) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { const int i = i0 + u * 32 + lane; v[u] = i < n ? pm[i] : -INFINITY; }
#pragma unroll
    for (int u = 0; u < 8; ++u) m = fmaxf(m, v[u]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (fold_arg && is_p) {   // the lowest tile that attains the row maximum holds the lowest such token id
    int first = 0x7FFFFFFF;
    for (int i = lane; i < n; i += 32) if (pm[i] == m) first = min(first, i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, o));
    if (lane == 0 && first < n) ws.argidx[it] = ws.part_idx[(size_t)it * np + first];
  }
  float s = 0.f;
  for (int i0 = 0; i0 < n; i0 += 256) {
    float vm[8], vs[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * 32 + lane;
      vm[u] = i < n ? pm[i] : -INFINITY;
      vs[u] = i < n ? ps[i] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) if (vs[u] > 0.f) s += vs[u] * __expf(vm[u] - m);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) {
    const float lse = m + logf(s);
    if (is_p) {
      ws.row_max[it] = m;
      ws.row_lse[it] = lse;
      if (cp.row_max_out) cp.row_max_out[it] = m;
      if (cp.row_lse_out) cp.row_lse_out[it] = lse;
    } else {
      ws.q_lse[it - R] = lse;
    }
  }
}

// Decision: one warp per sequence runs the tests and the prefix rule on the folded statistics.
__global__ void __launch_bounds__(128) decide_kernel(CallParams cp, Workspace ws) {
  const int b = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (b < cp.B) decide_sequence(cp, ws, b, true);
}

// -----------------------------------------------------------------------------------------
// Token location: inverse CDF in ascending token id over the stored weights of the selected
// row. Tile masses are prefix-summed in double; inside the owning tile the weights are added
// one by one in double.
// -----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32) locate_kernel(CallParams cp, Workspace ws, int np) {
  const int b = blockIdx.x;
  if (threadIdx.x != 0) return;
  const int V = cp.V;
  const int ntiles = (V + kVocabTile - 1) / kVocabTile;
  const double* mass = ws.mass_r + (size_t)b * np;
  const float* wv = ws.w_sel + (size_t)b * V;
  double total = 0.0;
  for (int t = 0; t < ntiles; ++t) total += mass[t];
  if (!(total > 0.0)) {  // identically zero residual: draw from p
    mass = ws.mass_p + (size_t)b * np;
    wv = ws.p_sel + (size_t)b * V;
    total = 0.0;
    for (int t = 0; t < ntiles; ++t) total += mass[t];
  }
  const double T = (double)ws.sel_u[b] * total;
  double prefix = 0.0;
  int token = -1;
  for (int t = 0; t < ntiles && token < 0; ++t) {
    const double incl = prefix + mass[t];
    if (incl > T) {
      double c = prefix;
      const int lo = t * kVocabTile, hi = min(V, lo + kVocabTile);
      int last_pos = -1;
      for (int vv = lo; vv < hi; ++vv) {
        const float x = wv[vv];
        c += (double)x;
        if (x > 0.f) last_pos = vv;
        if (c > T) { token = vv; break; }
      }
      if (token < 0) token = last_pos;  // summation-order rounding inside the tile
    }
    prefix = incl;
  }
  if (token < 0) {  // T >= total after rounding: the last token that carries mass
    for (int vv = V - 1; vv >= 0; --vv)
      if (wv[vv] > 0.f) { token = vv; break; }
  }
  cp.next_token[b] = token < 0 ? 0 : token;
}

__global__ void philox_uniforms_kernel(uint64_t seed, const int32_t* b, const int32_t* slot, const int32_t* stream,
                                       int n, float* out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = philox_uniform(seed, b[i], slot[i], stream[i]);
}

// Measurement aid: reads `n16` 16-byte words once with streaming loads and folds them into one
// word per block, so that nothing of the read can be dropped. The time of this kernel over W is
// the ceiling any kernel that must stream W once can reach on the device at hand.
__global__ void __launch_bounds__(512) stream_read_kernel(const uint4* __restrict__ p, size_t n16, uint32_t* out) {
  uint32_t acc = 0;
  const size_t stride = (size_t)gridDim.x * blockDim.x * 4;
  size_t i = (size_t)blockIdx.x * blockDim.x * 4 + threadIdx.x;
  for (; i + 3 * (size_t)blockDim.x < n16; i += stride) {   // four independent loads in flight per thread
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = __ldcs(p + i + (size_t)u * blockDim.x);
#pragma unroll
    for (int u = 0; u < 4; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  for (; i < n16; i += blockDim.x) {   // ragged end of this block's last group
    const uint4 v = __ldcs(p + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0 && acc != 0) atomicXor(out, acc);
}

// Self-test of the fused variant's fail-stop rule: leaves the status word as a fused launch that gave up
// would (a timeout tagged with the number of the next launch), without any wait having run out.
__global__ void stale_timeout_kernel(Workspace ws) {
  if (threadIdx.x == 0)
    set_status_tagged(ws.status, load_volatile_u32(ws.barrier + kCallCounter) + 1u, JD_ERR_TIMEOUT);
}

// -----------------------------------------------------------------------------------------
// host-side launchers
// -----------------------------------------------------------------------------------------
void launch_stale_timeout(const Workspace& ws, cudaStream_t st) { stale_timeout_kernel<<<1, 32, 0, st>>>(ws); }

int launch_q_stats(const CallParams& cp, const Workspace& ws, cudaStream_t st) {
  const int nq = (cp.V + kQChunk - 1) / kQChunk;
  q_stats_kernel<<<dim3(nq, cp.B * cp.M), 256, 0, st>>>(cp, ws, nq);
  return nq;
}

void launch_judge(const CallParams& cp, const Workspace& ws, const void* H, const void* w, int dtype, cudaStream_t st) {
  if (dtype == JD_DTYPE_BF16)
    judge_dot_kernel<__nv_bfloat16><<<cp.B * cp.M, 256, 0, st>>>(cp, ws, (const __nv_bfloat16*)H, (const __nv_bfloat16*)w);
  else
    judge_dot_kernel<float><<<cp.B * cp.M, 256, 0, st>>>(cp, ws, (const float*)H, (const float*)w);
}

void launch_quantize_rows(const CallParams& cp, const Workspace& ws, const void* H_bf16, cudaStream_t st) {
  const int R = cp.B * (cp.M + 1), nvec = cp.d / 8;
  const __nv_bfloat16* H = (const __nv_bfloat16*)H_bf16;
  if (cp.d % 8 != 0 || nvec > 4096) {
    quantize_rows_kernel<<<R, 256, 0, st>>>(cp, ws, H);
    return;
  }
  const int threads = std::min(1024, (nvec + 31) / 32 * 32);
  const int per = (nvec + threads - 1) / threads;
  if (per == 1) quantize_rows_vec_kernel<1><<<R, threads, 0, st>>>(cp, ws, H);
  else if (per == 2) quantize_rows_vec_kernel<2><<<R, threads, 0, st>>>(cp, ws, H);
  else quantize_rows_vec_kernel<4><<<R, threads, 0, st>>>(cp, ws, H);
}

void launch_row_scale(const CallParams& cp, const Workspace& ws, const void* H, int dtype, cudaStream_t st) {
  const int R = cp.B * (cp.M + 1);
  if (dtype == JD_DTYPE_BF16) row_scale_kernel<__nv_bfloat16><<<R, 256, 0, st>>>(cp, ws, (const __nv_bfloat16*)H);
  else row_scale_kernel<float><<<R, 256, 0, st>>>(cp, ws, (const float*)H);
}

void launch_fold(const CallParams& cp, const Workspace& ws, int np, int nq, cudaStream_t st, bool fold_arg) {
  const int items = cp.B * (2 * cp.M + 1);
  fold_stats_kernel<<<(items + 7) / 8, 256, 0, st>>>(cp, ws, np, nq, fold_arg ? 1 : 0);
}

void launch_decide(const CallParams& cp, const Workspace& ws, cudaStream_t st) {
  decide_kernel<<<(cp.B + 3) / 4, 128, 0, st>>>(cp, ws);
}

void launch_locate(const CallParams& cp, const Workspace& ws, int np, cudaStream_t st) {
  locate_kernel<<<cp.B, 32, 0, st>>>(cp, ws, np);
}

template <typename T>
static void simt_logits(const CallParams& cp, const Workspace& ws, const void* W, const void* H, int mode, int np,
                        float* logits_debug, const float* w_scale, cudaStream_t st) {
  const int R = mode == 1 ? cp.B : cp.B * (cp.M + 1);
  dim3 grid(np, (R + kSimtRows - 1) / kSimtRows);
  if (mode == 1)
    simt_logits_kernel<T, 1><<<grid, kVocabTile, 0, st>>>(cp, ws, (const T*)W, (const T*)H, R, np, nullptr, w_scale);
  else if (mode == 2)
    simt_logits_kernel<T, 2><<<grid, kVocabTile, 0, st>>>(cp, ws, (const T*)W, (const T*)H, R, np, nullptr, w_scale);
  else
    simt_logits_kernel<T, 0><<<grid, kVocabTile, 0, st>>>(cp, ws, (const T*)W, (const T*)H, R, np, logits_debug, w_scale);
}

int run_simt(const CallParams& cp, const Workspace& ws, const void* W, const float* w_scale, const void* w_judge,
             const void* H, int dtype, cudaStream_t st) {
  const int np = (cp.V + kVocabTile - 1) / kVocabTile;
  auto logits = [&](int mode, float* dbg) {
    if (dtype == JD_DTYPE_FP8_E4M3)   // E4M3 weights against the E4M3 rows the caller quantised into ws.h8
      simt_logits<e4m3_t>(cp, ws, W, ws.h8, mode, np, dbg, w_scale, st);
    else if (dtype == JD_DTYPE_BF16) simt_logits<__nv_bfloat16>(cp, ws, W, H, mode, np, dbg, nullptr, st);
    else simt_logits<float>(cp, ws, W, H, mode, np, dbg, nullptr, st);
  };
  const int nq = launch_q_stats(cp, ws, st);
  launch_judge(cp, ws, H, w_judge, dtype == JD_DTYPE_F32 ? JD_DTYPE_F32 : JD_DTYPE_BF16, st);
  logits(0, cp.logits_debug);
  launch_fold(cp, ws, np, nq, st);
  if (cp.rule == JD_RULE_TOPK) {   // ranks and argmax need the folded maxima; the decision writes the token
    logits(2, nullptr);
    launch_decide(cp, ws, st);
    return 6;
  }
  launch_decide(cp, ws, st);
  logits(1, nullptr);
  launch_locate(cp, ws, np, st);
  return 7;
}

void launch_stream_read(const void* p, size_t bytes, uint32_t* out, int num_sms, cudaStream_t st) {
  stream_read_kernel<<<num_sms * 4, 512, 0, st>>>((const uint4*)p, bytes / 16, out);
}

void launch_philox_uniforms(uint64_t seed, const int32_t* b, const int32_t* slot, const int32_t* stream, int n,
                            float* out, cudaStream_t st) {
  philox_uniforms_kernel<<<(n + 255) / 256, 256, 0, st>>>(seed, b, slot, stream, n, out);
}

}  // namespace jd
