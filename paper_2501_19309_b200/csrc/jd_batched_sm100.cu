// Batched variant for many rows (B*(M+1) in the hundreds or thousands): the R x V logits are far
// too many to keep on chip, so the call runs in two tensor-core passes.
//
// Pass 1, gemm_stats_kernel: persistent tcgen05 GEMM, rows of H on the MMA's M axis (128 TMEM
//   lanes = 128 rows), 256 vocabulary entries on N. Each 128 x 256 logits tile lives only in
//   tensor memory: the epilogue warps turn it into one (max, sum exp) pair per row and pick out
//   the drafted token's logit, while the next tile's MMAs fill the other half of tensor memory.
// Then the shared decision kernel folds the per-tile pairs, runs both tests and the prefix rule.
// With the top-K / greedy rule the same pass also counts, per row, the entries that rank above the
//   drafted token (against that token's logit, computed ahead of the pass by a small CUDA-core
//   kernel) and keeps the argmax of every tile: the call is then complete after the fold, and
//   W is streamed once.
// Pass 2: the selected row of every sequence (B rows) is gathered and handed to the fused
//   kernel in its sample-only mode, which recomputes those B rows of logits with W streamed
//   once more and draws the next tokens.
// The logits never reach device memory in either pass.
#include "jd_kernels.h"
#include "jd_sm100_ptx.cuh"

namespace jd {

namespace {

constexpr int kBThreads = 192;
constexpr int kTileM = 128;   // rows per tile
constexpr int kTileN = 256;   // vocabulary entries per tile
constexpr int kTileK = 64;    // bf16 per k-step (one 128-byte swizzle row); E4M3 codes: 128 per k-step
constexpr int kAStage = kTileM * 128;   // 16 KB
constexpr int kBStage = kTileN * 128;   // 32 KB
constexpr int kBStages = 4;
constexpr int kBMisc = 3072;

struct BMisc {
  uint64_t full[kBStages], empty[kBStages];
  uint64_t tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  int go;                 // written by epilogue thread 0 before a sync: 0 once a wait has run out
  float wsc[2][kTileN];   // E4M3 head: weight scales of the tile in each accumulator buffer
};
static_assert(sizeof(BMisc) <= kBMisc, "BMisc outgrew its shared-memory slot");

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// kFp8: W and the quantised rows of H (ws.h8) are E4M3 codes, multiplied by kind::f8f6f4 MMAs (K = 32
//       codes per instruction, 128 per k-step); the epilogue applies the scale of the vocabulary row
//       and of the H row to every accumulator. A template parameter, so that the MMA loop of one
//       instantiation names one instruction kind only.
// kTopK == false: softmax statistics + gather of the drafted token's logit.
// kTopK == true : the same, and for the top-K / greedy rule the epilogue also counts the entries of the
//                 row that rank above the drafted token (its logit is in ws.cand_ref before the kernel
//                 starts; the token's own column is left out of the count, ties rank by token id) and
//                 records the lowest token id that attains the tile's maximum.
template <bool kTopK, bool kFp8>
__global__ void __launch_bounds__(kBThreads, 1)
gemm_stats_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmH, CallParams cp,
                  Workspace ws, int R, int np, const float* __restrict__ w_scale) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  BMisc& ms = *reinterpret_cast<BMisc*>(smem);
  const uint32_t sA = smem_u32(smem + kBMisc);
  const uint32_t sB = sA + kBStages * kAStage;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = gridDim.x;
  volatile int* abort_flag = &ms.abort_flag;
  constexpr int kStepElems = kFp8 ? 2 * kTileK : kTileK;   // elements per 128-byte k-step
  const int num_kb = cp.d / kStepElems;
  const int row_blocks = (R + kTileM - 1) / kTileM;
  const int voc_blocks = (cp.V + kTileN - 1) / kTileN;
  const int num_tiles = row_blocks * voc_blocks;

  if (tid == 0) {
    for (int s = 0; s < kBStages; ++s) { mbar_init(smem_u32(&ms.full[s]), 1); mbar_init(smem_u32(&ms.empty[s]), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&ms.tmem_full[s]), 1); mbar_init(smem_u32(&ms.tmem_empty[s]), 1); }
    ms.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ms.tmem_base)),
                 "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ms.tmem_base;

  // Tile order: consecutive tile ids share the vocabulary block, so the CTAs that run at the
  // same time read the same W slab and all but the first find it in L2.
  if (warp == 4 && lane == 0) {
    const uint64_t pol_w = policy_evict_first(), pol_h = policy_evict_last();
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += G) {
      const int vb = t / row_blocks, rb = t % row_blocks;
      for (int kb = 0; kb < num_kb; ++kb) {
        ok = mbar_wait(smem_u32(&ms.empty[s]), ph ^ 1u, abort_flag);
        if (!ok) break;
        mbar_expect_tx(smem_u32(&ms.full[s]), kAStage + kBStage);
        tma_load_2d(sA + s * kAStage, &tmH, smem_u32(&ms.full[s]), kb * kStepElems, rb * kTileM, pol_h);
        tma_load_2d(sB + s * kBStage, &tmW, smem_u32(&ms.full[s]), kb * kStepElems, vb * kTileN, pol_w);
        if (++s == kBStages) { s = 0; ph ^= 1u; }
      }
    }
    if (!ok) set_status(ws.status, JD_ERR_TIMEOUT);
  } else if (warp == 5 && lane == 0) {
    const uint32_t idesc = kFp8 ? make_idesc_e4m3(kTileN) : make_idesc(kTileN);
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    int it = 0;
    for (int t = blockIdx.x; t < num_tiles && ok; t += G, ++it) {
      const int buf = it & 1;
      ok = mbar_wait(smem_u32(&ms.tmem_empty[buf]), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t dcol = tmem_base + (uint32_t)(buf * kTileN);
      for (int kb = 0; kb < num_kb; ++kb) {
        ok = mbar_wait(smem_u32(&ms.full[s]), ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t ab = sA + s * kAStage, bb = sB + s * kBStage;
#pragma unroll
        for (int k = 0; k < 4; ++k) {   // 32 bytes of K per instruction: 16 bf16 or 32 codes
          const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
          if constexpr (kFp8) umma_e4m3(dcol, make_smem_desc(ab + k * 32), make_smem_desc(bb + k * 32), idesc, acc);
          else umma_bf16(dcol, make_smem_desc(ab + k * 32), make_smem_desc(bb + k * 32), idesc, acc);
        }
        umma_commit(smem_u32(&ms.empty[s]));
        if (++s == kBStages) { s = 0; ph ^= 1u; }
      }
      if (ok) umma_commit(smem_u32(&ms.tmem_full[buf]));
    }
    if (!ok) set_status(ws.status, JD_ERR_TIMEOUT);
  } else if (warp < 4) {
    // Epilogue: thread = row. Online (max, sum exp) over the tile's 256 columns, 32 at a time.
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
    bool ok = true;
    int it = 0;
    for (int t = blockIdx.x; t < num_tiles; t += G, ++it) {
      const int vb = t / row_blocks, rb = t % row_blocks;
      const int buf = it & 1;
      const int row = rb * kTileM + tid;
      const int v0 = vb * kTileN;
      int x = -1;
      if (row < R) {
        const int b = row / (cp.M + 1), j = row % (cp.M + 1);
        if (j < cp.M) {
          x = cp.draft_tokens[b * cp.M + j];
          if (x < 0 || x >= cp.V) { set_status(ws.status, JD_ERR_BAD_TOKEN); x = min(max(x, 0), cp.V - 1); }
        }
      }
      if (kFp8) {   // the previous reader of this buffer's scales finished two tiles (and two syncs) ago
        ms.wsc[buf][tid] = v0 + tid < cp.V ? __ldg(w_scale + v0 + tid) : 0.f;
        ms.wsc[buf][tid + 128] = v0 + tid + 128 < cp.V ? __ldg(w_scale + v0 + tid + 128) : 0.f;
      }
      if (tid == 0) {   // one thread decides for all 128, so that they leave the loop together
        mbar_wait(smem_u32(&ms.tmem_full[buf]), (uint32_t)(it >> 1) & 1u, abort_flag);
        ms.go = (*abort_flag == 0);
      }
      epi_sync();
      ok = ms.go != 0;
      if (!ok) break;
      tc_fence_after();
      float m = -INFINITY, s = 0.f, g = 0.f;
      bool have_g = false;
      int above = 0, arg = 0x7F7F7F7F;
      float g_ref = 0.f;
      float sc = (cp.norm == JD_NORM_RMS && row < R) ? ws.row_scale[row] : 1.f;
      if (kFp8 && row < R) sc *= ws.h_scale[row];
      if (kTopK && x >= 0) g_ref = ws.cand_ref[row];
#pragma unroll 1
      for (int c0 = 0; c0 < kTileN; c0 += 32) {
        float v[32];
        tmem_ld32(lane_base + (uint32_t)(buf * kTileN + c0), v);
        if (kFp8) {
#pragma unroll
          for (int k = 0; k < 32; ++k) v[k] = (v[k] * ms.wsc[buf][c0 + k]) * sc;
        } else {
#pragma unroll
          for (int k = 0; k < 32; ++k) v[k] *= sc;
        }
        const int nvalid = cp.V - (v0 + c0);   // columns of this chunk that exist (>= 32 except at the tail)
        if (cp.logits_debug != nullptr && row < R) {   // test-only copy of the logits
          float* o = cp.logits_debug + (size_t)row * cp.V + v0 + c0;
#pragma unroll
          for (int k = 0; k < 32; ++k) if (k < nvalid) o[k] = v[k];
        }
        if (nvalid < 32) {
#pragma unroll
          for (int k = 0; k < 32; ++k) if (k >= nvalid) v[k] = -INFINITY;
        }
        float cm = v[0];
#pragma unroll
        for (int k = 1; k < 32; ++k) cm = fmaxf(cm, v[k]);
        if (kTopK) {
          if (x >= 0) {
#pragma unroll
            for (int k = 0; k < 32; ++k) {
              const int col = v0 + c0 + k;
              if (col != x && (v[k] > g_ref || (v[k] == g_ref && col < x))) ++above;
            }
          }
          if (cm > m) {   // a new maximum of the tile: its first column in this chunk
#pragma unroll
            for (int k = 31; k >= 0; --k) if (v[k] == cm) arg = v0 + c0 + k;
          }
        }
        const float mn = fmaxf(m, cm);
        if (mn > -INFINITY) {
          const float off = mn * kLog2e;
          float acc = 0.f;
#pragma unroll
          for (int k = 0; k < 32; ++k) acc += fast_exp2(fmaf(v[k], kLog2e, -off));
          s = s * fast_exp2(fmaf(m, kLog2e, -off)) + acc;
          m = mn;
        }
        if ((unsigned)(x - (v0 + c0)) < 32u) {
#pragma unroll
          for (int k = 0; k < 32; ++k) if (x == v0 + c0 + k) g = v[k];
          have_g = true;
        }
      }
      tc_fence_before();
      epi_sync();
      if (tid == 0) mbar_arrive(smem_u32(&ms.tmem_empty[buf]));
      if (row < R) {
        ws.part_max[(size_t)row * np + vb] = m;
        ws.part_sum[(size_t)row * np + vb] = s;
        if (have_g) ws.gath[row] = g;
        if (kTopK) {
          if (above) atomicAdd(ws.cnt + row, above);
          ws.part_idx[(size_t)row * np + vb] = arg;
        }
      }
    }
    if (!ok && tid == 0) set_status(ws.status, JD_ERR_TIMEOUT);
  }

  __syncthreads();
  if (ms.abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
    __syncthreads();
  }
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// Top-K / greedy rule: the logit of every drafted token, L[row, x] = H[row] . W[x] with the scales the
// GEMM's epilogue applies, on CUDA cores ahead of the GEMM pass (one CTA per row, 2 x d elements read).
// The pass ranks the other entries of the row against this value; it differs from the tensor cores'
// own L[row, x] by float32 summation order only, and that column is left out of the count.
template <bool kFp8>
__global__ void __launch_bounds__(128) candidate_logit_kernel(CallParams cp, Workspace ws, const uint8_t* __restrict__ W,
                                                              const uint8_t* __restrict__ H,
                                                              const float* __restrict__ w_scale) {
  __shared__ float part[4];
  const int row = blockIdx.x, tid = threadIdx.x;
  const int b = row / (cp.M + 1), j = row % (cp.M + 1);
  if (j >= cp.M) return;
  const int x = min(max(cp.draft_tokens[b * cp.M + j], 0), cp.V - 1);   // the GEMM pass reports a bad token
  const int row_bytes = kFp8 ? cp.d : cp.d * 2;
  const uint4* wr = reinterpret_cast<const uint4*>(W + (size_t)x * row_bytes);
  const uint4* hr = reinterpret_cast<const uint4*>(H + (size_t)row * row_bytes);
  float acc = 0.f;
  for (int k = tid; k < row_bytes / 16; k += 128) {
    const uint4 a = __ldg(wr + k), h = __ldg(hr + k);
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, hw[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (kFp8) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          acc = fmaf(to_float(e4m3_t{(uint8_t)(aw[q] >> (8 * e))}), to_float(e4m3_t{(uint8_t)(hw[q] >> (8 * e))}), acc);
      } else {
        acc = fmaf(__uint_as_float(aw[q] << 16), __uint_as_float(hw[q] << 16), acc);
        acc = fmaf(__uint_as_float(aw[q] & 0xFFFF0000u), __uint_as_float(hw[q] & 0xFFFF0000u), acc);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((tid & 31) == 0) part[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    float v = (part[0] + part[1]) + (part[2] + part[3]);
    float sc = cp.norm == JD_NORM_RMS ? ws.row_scale[row] : 1.f;
    if (kFp8) { sc *= ws.h_scale[row]; v *= __ldg(w_scale + x); }
    ws.cand_ref[row] = v * sc;
  }
}

// Prepares the second pass: copies the selected row of H of every sequence into a dense [B, d]
// matrix, and the selected draft-logit row (where the residual needs it) into a tile-major
// buffer [vocab tile][sequence][128], so that a CTA of the second pass finds the draft logits of
// its vocabulary slice for all sequences in one contiguous block.
// `H` is the matrix the second pass multiplies: bf16 rows, or (row_bytes = d) the E4M3 codes.
__global__ void __launch_bounds__(256) gather_rows_kernel(CallParams cp, Workspace ws, const uint8_t* __restrict__ H,
                                                          int row_bytes) {
  // b counts within the launch's chunk of sequences (ws.sel_* and cp.B are the chunk's views);
  // the row index is global, and so is the sequence it belongs to
  const int b = blockIdx.x, part = blockIdx.y, parts = gridDim.y;
  const int row = ws.sel_row[b];
  const int b_global = row / (cp.M + 1);
  if (part == 0) {
    const uint4* src = reinterpret_cast<const uint4*>(H + (size_t)row * row_bytes);
    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(ws.h_sel) + (size_t)b * row_bytes);
    for (int k = threadIdx.x; k < row_bytes / 16; k += blockDim.x) dst[k] = src[k];
  }
  if (ws.sel_kind[b] != 0) return;
  const float* dl = cp.draft_logits + ((size_t)b_global * cp.M + (row % (cp.M + 1))) * cp.V;
#pragma unroll 4
  for (int v = part * 256 + threadIdx.x; v < cp.V; v += parts * 256)
    ws.w_sel[((size_t)(v / kVocabTile) * cp.B + b) * kVocabTile + (v % kVocabTile)] = __ldg(dl + v);
}

}  // namespace

static int grid_of(int R, int np, int num_sms) {
  return std::min(num_sms, ((R + kTileM - 1) / kTileM) * np);
}

bool batched_configure() {
  return cudaFuncSetAttribute(gemm_stats_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem) == cudaSuccess &&
         cudaFuncSetAttribute(gemm_stats_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem) == cudaSuccess &&
         cudaFuncSetAttribute(gemm_stats_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem) == cudaSuccess &&
         cudaFuncSetAttribute(gemm_stats_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem) == cudaSuccess;
}

bool batched_supported(int dtype, int B, int d, int V, int num_sms) {
  if (dtype == JD_DTYPE_BF16) { if (d % kTileK != 0 || d < kTileK) return false; }
  else if (dtype == JD_DTYPE_FP8_E4M3) { if (d % (2 * kTileK) != 0 || d < 2 * kTileK) return false; }
  else return false;
  if (num_sms < 1 || num_sms > kMaxCtas) return false;
  // the second pass runs the selected rows through the fused kernel, a chunk of sequences per launch
  FusedPlan plan;
  const int chunk = second_pass_chunk(B);
  if (!fused_supported(dtype, chunk, d, V, num_sms, &plan)) return false;
  return B % chunk == 0 || fused_supported(dtype, B % chunk, d, V, num_sms, &plan);
}

int run_batched(const CallParams& cp, const Workspace& ws, const CUtensorMap& tmW256, const CUtensorMap& tmW128,
                const CUtensorMap& tmH, const CUtensorMap& tmHsel, const CUtensorMap& tmHselTail, const void* H,
                const void* w_judge, int num_sms, cudaStream_t st, const SideStream& side, cudaError_t* err,
                const float* w_scale_fp8, const void* W) {
  const bool fp8 = w_scale_fp8 != nullptr;
  const int dtype = fp8 ? JD_DTYPE_FP8_E4M3 : JD_DTYPE_BF16;
  const int R = cp.B * (cp.M + 1);
  const int np = (cp.V + kTileN - 1) / kTileN;
  const size_t smem = 1024 + kBMisc + (size_t)kBStages * (kAStage + kBStage);
  const bool topk = cp.rule == JD_RULE_TOPK;
  auto gemm = [&]() {
    auto kern = fp8 ? (topk ? gemm_stats_kernel<true, true> : gemm_stats_kernel<false, true>)
                    : (topk ? gemm_stats_kernel<true, false> : gemm_stats_kernel<false, false>);
    kern<<<grid_of(R, np, num_sms), kBThreads, smem, st>>>(tmW256, tmH, cp, ws, R, np, w_scale_fp8);
    return true;
  };
  if (topk) {   // the drafted tokens' logits, which the pass ranks the rows against
    if (fp8) candidate_logit_kernel<true><<<R, 128, 0, st>>>(cp, ws, (const uint8_t*)W, ws.h8, w_scale_fp8);
    else candidate_logit_kernel<false><<<R, 128, 0, st>>>(cp, ws, (const uint8_t*)W, (const uint8_t*)H, nullptr);
  }
  int nq;
  if (side.stream) {
    // The draft statistics (HBM-bound) and the judge dots do not depend on the GEMM (tensor-bound):
    // they run on the handle's side stream next to it and join before the decision.
    if ((*err = cudaEventRecord(side.fork, st)) != cudaSuccess) return -1;
    if (!gemm()) return -1;
    if ((*err = cudaStreamWaitEvent(side.stream, side.fork, 0)) != cudaSuccess) return -1;
    nq = launch_q_stats(cp, ws, side.stream);
    launch_judge(cp, ws, H, w_judge, JD_DTYPE_BF16, side.stream);
    if ((*err = cudaEventRecord(side.join, side.stream)) != cudaSuccess) return -1;
    if ((*err = cudaStreamWaitEvent(st, side.join, 0)) != cudaSuccess) return -1;
  } else {
    nq = launch_q_stats(cp, ws, st);
    launch_judge(cp, ws, H, w_judge, JD_DTYPE_BF16, st);
    if (!gemm()) return -1;
  }
  launch_fold(cp, ws, np, nq, st, /*fold_arg=*/topk);
  if (topk) {   // ranks and argmax came out of the same pass; the decision writes the token, nothing is drawn
    launch_decide(cp, ws, st);
    return 6;
  }
  launch_decide(cp, ws, st);
  int launches = 5;
  const int chunk = second_pass_chunk(cp.B);
  for (int off = 0; off < cp.B; off += chunk) {
    const int nc = std::min(chunk, cp.B - off);
    // this chunk's view of the call: sequences off .. off + nc - 1 become 0 .. nc - 1
    CallParams cc = cp;
    cc.logits_debug = nullptr;   // the second pass recomputes selected rows only
    cc.B = nc;
    cc.next_token = cp.next_token + off;
    Workspace wc = ws;
    wc.sel_row += off; wc.sel_kind += off; wc.sel_lse_p += off; wc.sel_lse_q += off; wc.sel_u += off;
    // second pass operand: the bf16 rows, or their E4M3 codes (one byte per element)
    gather_rows_kernel<<<dim3(nc, 32), 256, 0, st>>>(cc, wc, fp8 ? ws.h8 : (const uint8_t*)H, fp8 ? cp.d : cp.d * 2);
    FusedPlan plan;
    if (!fused_supported(dtype, nc, cp.d, cp.V, num_sms, &plan)) { *err = cudaErrorInvalidValue; return -1; }
    const int n = run_fused(cc, wc, tmW128, nc == chunk ? tmHsel : tmHselTail, ws.h_sel, w_judge, plan, st, err,
                            /*sample_only=*/true, w_scale_fp8);
    if (n < 0) return -1;
    launches += 1 + n;
  }
  return launches;
}

}  // namespace jd
