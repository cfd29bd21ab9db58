// Shared device-side pieces of the verification library: workspace layout, the
// counter-based generator, online-softmax helpers and the per-sequence decision step.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "jd.h"

namespace jd {

constexpr int kVocabTile = 128;            // vocabulary entries per statistics tile
constexpr int kMaxCtas = 256;              // upper bound on the persistent grid (SM count)
constexpr unsigned kSpinLimit = 1u << 22;  // iteration bound of every device-side wait

// Device workspace owned by a handle. Partial softmax statistics are stored per
// (row, partial index); the number of partials per row depends on the variant
// (vocabulary tiles for the SIMT and batched variants, CTAs for the fused variant).
struct Workspace {
  float* part_max;     // [maxR][np]   running max of the row over one vocabulary slice
  float* part_sum;     // [maxR][np]   sum exp(L - part_max) over that slice
  float* gath;         // [maxR]       L[row, x_j] for rows j < M
  float* qpart_max;    // [maxBM][nq]
  float* qpart_sum;    // [maxBM][nq]
  float* qgath;        // [maxBM]      draft logit at x_j
  float* judge_logit;  // [maxBM]      w . H[b, j+1] (bias not yet added)
  float* row_max;      // [maxR]
  float* row_lse;      // [maxR]
  float* q_lse;        // [maxBM]
  int* sel_row;        // [maxB] global row index b*(M+1)+a of the row the next token is drawn from
  int* sel_kind;       // [maxB] 0: residual max(0,p-q) against draft row a; 1: p alone
  float* sel_lse_p;    // [maxB]
  float* sel_lse_q;    // [maxB]
  float* sel_u;        // [maxB] uniform of the token draw
  double* mass_r;      // [maxB][np] mass of the sampling weights per vocabulary slice
  double* mass_p;      // [maxB][np] mass of p per slice (zero-residual fallback)
  float* w_sel;        // [maxB][V]  sampling weights (SIMT variant); in the batched variant the selected
                       //            draft rows, tile-major [ceil(V/128)][B][128]
  float* p_sel;        // [maxB][V]  p of the selected row (same)
  uint8_t* h8;         // [maxR][d] FP8 head: rows of H quantised to E4M3
  float* h_scale;      // [maxR]    FP8 head: scale of every quantised row
  float* row_scale;    // [maxR] 1 / sqrt(mean square + eps) of every row of H (JD_NORM_RMS)
  int* cnt;            // [maxR] top-K rule: entries of the row that rank above the drafted token
  int* argidx;         // [maxR] top-K rule: lowest token id that attains the row maximum
  int* part_idx;       // [maxR][np] top-K rule: per-CTA argmax candidates (fused variant); lowest token id
                       //            that attains the tile's maximum, per vocabulary tile (batched variant)
  float* cand_ref;     // [maxR] top-K rule, batched variant: L[row, x_j] computed ahead of the GEMM pass
  int* own_i;          // [maxB][2] second pass of the batched variant: CTA that owns each sequence's draw, and whether
                       //           the draw falls back to p (identically zero residual)
  double* own_d;       // [maxB][2] same: mass in front of the owning CTA's slice (< 0: beyond the total), and T
  __nv_bfloat16* h_sel;  // [maxB][d] selected rows of H gathered for the batched variant's second pass
  unsigned* status;    // [1] device status word: jd_status_t of the first device-side problem in bits 0-7; bits 8-31 a
                       //     call tag when the fused kernel wrote it (see kCallCounter), 0 when another kernel did
  unsigned* barrier;   // [8] fused variant: two sets of three grid-barrier counters ([0..2], [3..5]) used by
                       //     alternate launches, [6] = kCallCounter, [7] the self-test's counter
  int np_cap;          // capacity (partials per row) of part_* and mass_*
  int nq_cap;          // capacity of qpart_*
};

__device__ __forceinline__ void set_status(unsigned* status, unsigned code) { atomicCAS(status, 0u, code); }

// The fused kernel keeps its grid-barrier state clean by itself, so that back-to-back calls need no
// memset between them. barrier[kCallCounter] counts the kernel's successful launches since the block
// was last cleared by the host. Launch number c (0-based) uses barrier set c % 2, clears the other
// set (idle since launch c - 1 ended) and, when it has passed its last barrier, CTA 0 publishes c + 1.
// Its status writes carry the tag c + 1, which tells them apart from what earlier launches left in
// the word. A launch in which a wait ran out publishes nothing: the next launch finds that tagged
// JD_ERR_TIMEOUT still in place and gives up at once, and so on until the host has read the status
// and cleared the block (the counters of the failed launch are in an unknown state).
constexpr int kCallCounter = 6;
__device__ __forceinline__ unsigned load_volatile_u32(const unsigned* p) { return *reinterpret_cast<const volatile unsigned*>(p); }
__device__ __forceinline__ void set_status_tagged(unsigned* status, unsigned tag, unsigned code) {
  const unsigned want = (tag << 8) | code;
  unsigned old = load_volatile_u32(status);
  for (int i = 0; i < 64; ++i) {                          // first problem of this launch wins
    if ((old >> 8) == tag && (old & 0xFFu) != 0u) return;
    const unsigned prev = atomicCAS(status, old, want);
    if (prev == old) return;
    old = prev;
  }
}

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): counter (c0..c3), key (k0, k1), ten rounds of
// two 32x32->64 multiplies with the key bumped by the Weyl constants between rounds.
// ---------------------------------------------------------------------------------------
__host__ __device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2,
                                                                 uint32_t c3, uint32_t k0, uint32_t k1) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) {
      k0 += W0;
      k1 += W1;
    }
    const uint64_t p0 = (uint64_t)M0 * c0;
    const uint64_t p1 = (uint64_t)M1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  return c0;
}

// u in [0,1) on the 2^-24 grid for (seed; b, slot, stream): exact in float.
__host__ __device__ __forceinline__ float philox_uniform(uint64_t seed, int b, int slot, int stream) {
  const uint32_t w = philox4x32_10_word0((uint32_t)b, (uint32_t)slot, (uint32_t)stream, 0u,
                                         (uint32_t)seed, (uint32_t)(seed >> 32));
  return (float)(w >> 8) * (1.0f / 16777216.0f);
}

// ---------------------------------------------------------------------------------------
// online softmax pair (m, s): s = sum exp(x - m)
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void ms_combine(float& m, float& s, float m2, float s2) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { m = mn; s = 0.f; return; }
  s = s * __expf(m - mn) + s2 * __expf(m2 - mn);
  m = mn;
}

__device__ __forceinline__ void ms_warp_reduce(float& m, float& s) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
    const float s2 = __shfl_xor_sync(0xffffffffu, s, o);
    ms_combine(m, s, m2, s2);
  }
}

__device__ __forceinline__ double warp_sum_double(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// FP8 E4M3 code (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities).
struct e4m3_t { uint8_t b; };
template <> __device__ __forceinline__ float to_float<e4m3_t>(e4m3_t v) {
  uint32_t h2;   // the hardware conversion widens two codes to two halves; the low one is ours
  asm("{\n\t.reg .b16 t;\n\tcvt.u16.u32 t, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, t;\n\t}" : "=r"(h2) : "r"((uint32_t)v.b));
  return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

// ---------------------------------------------------------------------------------------
// Per-call parameters every kernel family shares.
// ---------------------------------------------------------------------------------------
struct CallParams {
  int B, M, d, V;
  const int32_t* draft_tokens;
  const float* draft_logits;
  float tau, b_judge;
  uint64_t seed;
  int mode, resample;
  int rule, top_k;
  int norm;
  float rms_eps;
  int32_t* accept_len;
  int32_t* next_token;
  float* judge_scores;
  float* p_draft;
  float* q_draft;
  uint8_t* masks;
  float* row_max_out;
  float* row_lse_out;
  float* logits_debug;   // [B, M+1, V] test-only copy of the logits (null in production)
  int dl_vec4;           // 1: every draft-logit row starts on a 16-byte boundary (V % 4 == 0 and an aligned base),
                         //    so the draft statistics may use 16-byte loads; 0: 4-byte loads only
};

// Decision step for one sequence b, executed by one warp (Eq. 4, Sec. 4.1 "Inference"):
// given the rows' log-normalisers, the gathered logits and the judge logits, evaluates both
// tests for every slot, combines them by mode, finds the accepted prefix and records which
// row the next token is drawn from. Every lane returns the accepted length. gath, qgath and
// judge_logit are always global memory (possibly written by other CTAs of the same grid, hence
// the L2 loads); the log-normalisers and the sel_* outputs may live in shared memory.
__device__ __forceinline__ int decide_sequence(const CallParams& cp, const Workspace& ws, int b,
                                               bool write_outputs) {
  const int lane = threadIdx.x & 31;
  const int M = cp.M;
  int first_reject = M;
  for (int j0 = 0; j0 < M; j0 += 32) {
    const int j = j0 + lane;
    bool ok = true;
    if (j < M) {
      const int row = b * (M + 1) + j;
      const int bm = b * M + j;
      const float P = expf(__ldcg(ws.gath + row) - ws.row_lse[row]);
      const float Q = expf(__ldcg(ws.qgath + bm) - ws.q_lse[bm]);
      const float u = philox_uniform(cp.seed, b, j, 0);
      const bool z_std = (cp.rule == JD_RULE_TOPK) ? (__ldcg(ws.cnt + row) < cp.top_k) : (u * Q < P);
      const float s = 1.0f / (1.0f + expf(-(__ldcg(ws.judge_logit + bm) + cp.b_judge)));
      const bool z_judge = (s > cp.tau);
      ok = cp.mode == JD_MODE_STANDARD ? z_std : (cp.mode == JD_MODE_JUDGE ? z_judge : (z_std || z_judge));
      if (write_outputs) {
        cp.judge_scores[bm] = s;
        cp.p_draft[bm] = P;
        if (cp.q_draft) cp.q_draft[bm] = Q;
        if (cp.masks) cp.masks[bm] = (uint8_t)((z_std ? 1 : 0) | (z_judge ? 2 : 0));
      }
    }
    const unsigned rej = __ballot_sync(0xffffffffu, !ok);
    if (rej != 0u && first_reject == M) first_reject = j0 + (__ffs(rej) - 1);
  }
  const int a = first_reject;
  if (lane == 0) {
    const int row = b * (M + 1) + a;
    ws.sel_row[b] = row;
    const bool residual = (a < M) && (cp.resample == JD_RESAMPLE_RESIDUAL);
    ws.sel_kind[b] = (cp.rule == JD_RULE_TOPK) ? 2 : (residual ? 0 : 1);   // 2: greedy token, nothing to draw
    ws.sel_lse_p[b] = ws.row_lse[row];
    ws.sel_lse_q[b] = residual ? ws.q_lse[b * M + a] : 0.f;
    ws.sel_u[b] = philox_uniform(cp.seed, b, a, 1);
    if (write_outputs) {
      cp.accept_len[b] = a;
      // top-K rule: the next token is the row's argmax, known already unless the caller folds it later
      if (cp.rule == JD_RULE_TOPK && ws.argidx) cp.next_token[b] = __ldcg(ws.argidx + row);
    }
  }
  return a;
}

// Sampling weight of one vocabulary entry of the selected row.
__device__ __forceinline__ void sample_weights(float logit, float lse_p, int kind, float dlogit, float lse_q,
                                               float& p, float& r) {
  p = __expf(logit - lse_p);
  r = (kind == 0) ? fmaxf(0.f, p - __expf(dlogit - lse_q)) : p;
}

}  // namespace jd
