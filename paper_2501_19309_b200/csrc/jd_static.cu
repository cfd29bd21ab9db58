// jd_verify_static: the fused verification call for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they verify a draft
// block: inference servers that hand the whole device to their own memory pool at start-up
// (a later cudaMalloc fails or fragments the pool), latency-critical decode loops where an
// allocation would add an implicit device synchronisation, and code running under a policy
// that forbids allocation after initialisation. jd_create allocates a workspace, so it is not
// for them. This entry point needs no handle: the scratch memory of the fused kernel (per-CTA
// softmax partials, gathered logits, row normalisers, per-CTA sampling masses, status word, grid-barrier
// counters) lives in a fixed array in the library's device image, which every GPU that loads
// the library holds until the process exits.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "jd_kernels.h"

using namespace jd;

namespace {

constexpr int kStaticMaxRows = 96;                       // B * (M + 1), the fused variant's limit
constexpr int kStaticMaxSeqs = kStaticMaxRows / 2;       // M >= 1, so B <= 48
constexpr size_t kRowPartials = (size_t)kStaticMaxRows * kMaxCtas * sizeof(float);    //  98,304 B
constexpr size_t kSeqMasses = (size_t)kStaticMaxSeqs * kMaxCtas * sizeof(double);     //  98,304 B
constexpr size_t kSmall = 512;                           // 96 floats, rounded to 256-byte units
// part_max, part_sum, qpart_max, qpart_sum | mass_r, mass_p | gath, qgath, judge_logit, row_lse, q_lse |
// status + barrier counters
constexpr size_t kStaticScratchBytes = 4 * kRowPartials + 2 * kSeqMasses + 5 * kSmall + 512;   // 592,896 B

// The scratch itself. In host code this name is only a handle for cudaGetSymbolAddress; it is
// not a device address and must never be passed to a kernel as is.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal
int g_num_sms[kMaxDevices] = {};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool encode_bf16_rows(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t d, uint32_t box_rows) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return false;
    fn = (EncodeTiledFn)p;
  }
  const cuuint64_t dims[2] = {d, rows};
  const cuuint64_t strides[1] = {d * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

std::mutex g_setup_mutex;   // first calls from several host threads set a device up once

}  // namespace

extern "C" jd_status_t jd_verify_static(int32_t d, int32_t V, const void* W, const void* w_judge, float b_judge,
                                        const jd_verify_args_t* a, uint32_t* device_status, void* cuda_stream) {
  if (!a || !W || !w_judge || d < 1 || V < 2) return JD_ERR_INVALID_ARG;
  if (a->B < 1 || a->M < 1) return JD_ERR_INVALID_ARG;
  if (!a->H || !a->draft_tokens || !a->draft_logits) return JD_ERR_INVALID_ARG;
  if (!a->accept_len || !a->next_token || !a->judge_scores || !a->p_draft) return JD_ERR_INVALID_ARG;
  if (a->logits_debug) return JD_ERR_INVALID_ARG;
  if (!(a->tau >= 0.f && a->tau <= 1.f)) return JD_ERR_INVALID_ARG;
  if (a->mode < JD_MODE_STANDARD || a->mode > JD_MODE_JUDGE_OR_STANDARD) return JD_ERR_INVALID_ARG;
  if (a->resample < JD_RESAMPLE_RESIDUAL || a->resample > JD_RESAMPLE_TARGET_P) return JD_ERR_INVALID_ARG;
  if (a->variant != JD_VARIANT_AUTO && a->variant != JD_VARIANT_FUSED) return JD_ERR_INVALID_ARG;
  if (a->rule != JD_RULE_SAMPLING) return JD_ERR_UNSUPPORTED;   // the fixed scratch has no rank counters
  if (a->norm != JD_NORM_NONE) return JD_ERR_UNSUPPORTED;       // nor row normalisation factors
  if (!aligned16(W) || !aligned16(w_judge) || !aligned16(a->H)) return JD_ERR_INVALID_ARG;
  if (!aligned4(a->draft_tokens) || !aligned4(a->draft_logits) || !aligned4(a->accept_len) || !aligned4(a->next_token) ||
      !aligned4(a->judge_scores) || !aligned4(a->p_draft) || !aligned4(a->q_draft) || !aligned4(a->row_max) ||
      !aligned4(a->row_lse) || !aligned4(device_status))
    return JD_ERR_INVALID_ARG;
  // the fixed scratch holds at most 96 rows: larger blocks are refused, never truncated
  if ((int64_t)a->B * (a->M + 1) > kStaticMaxRows) return JD_ERR_UNSUPPORTED;
  const int R = a->B * (a->M + 1);

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return JD_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return JD_ERR_UNSUPPORTED;
  std::unique_lock<std::mutex> setup_lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    // one-time set-up on this device (it is the current one): architecture, SM count, the device
    // address of the scratch array, and the kernels themselves (their shared-memory limit is raised
    // here, which also loads every instantiation, so that no later call has to load code)
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return JD_ERR_CUDA;
    if (major != 10) return JD_ERR_ARCH;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p || !fused_configure()) {
      cudaGetLastError();
      return JD_ERR_CUDA;
    }
    g_num_sms[dev] = sms;
    g_scratch_ptr[dev] = p;
  }
  setup_lock.unlock();

  FusedPlan plan;
  if (!fused_supported(JD_DTYPE_BF16, R, d, V, g_num_sms[dev], &plan)) return JD_ERR_UNSUPPORTED;

  // carve the fixed array; pointers the fused kernel never touches stay null
  char* base = (char*)g_scratch_ptr[dev];
  size_t off = 0;
  auto take = [&](size_t bytes) { char* p = base + off; off += bytes; return p; };
  Workspace ws = {};
  ws.part_max = (float*)take(kRowPartials);
  ws.part_sum = (float*)take(kRowPartials);
  ws.qpart_max = (float*)take(kRowPartials);
  ws.qpart_sum = (float*)take(kRowPartials);
  ws.mass_r = (double*)take(kSeqMasses);
  ws.mass_p = (double*)take(kSeqMasses);
  ws.gath = (float*)take(kSmall);
  ws.qgath = (float*)take(kSmall);
  ws.judge_logit = (float*)take(kSmall);
  ws.row_lse = (float*)take(kSmall);
  ws.q_lse = (float*)take(kSmall);
  unsigned* own_status = (unsigned*)take(256);
  ws.status = device_status ? device_status : own_status;   // the caller's word receives the status if given
  ws.barrier = (unsigned*)take(256);
  ws.np_cap = kMaxCtas;
  ws.nq_cap = kMaxCtas;
  if (off != kStaticScratchBytes) return JD_ERR_CUDA;

  CallParams cp;
  cp.B = a->B; cp.M = a->M; cp.d = d; cp.V = V;
  cp.draft_tokens = a->draft_tokens;
  cp.draft_logits = a->draft_logits;
  cp.tau = a->tau; cp.b_judge = b_judge; cp.seed = a->seed;
  cp.mode = a->mode; cp.resample = a->resample;
  cp.rule = JD_RULE_SAMPLING; cp.top_k = 1;
  cp.norm = JD_NORM_NONE; cp.rms_eps = 0.f;
  cp.accept_len = a->accept_len; cp.next_token = a->next_token;
  cp.judge_scores = a->judge_scores; cp.p_draft = a->p_draft;
  cp.q_draft = a->q_draft; cp.masks = a->masks;
  cp.row_max_out = a->row_max; cp.row_lse_out = a->row_lse;
  cp.logits_debug = nullptr;
  cp.dl_vec4 = (V % 4 == 0 && aligned16(a->draft_logits)) ? 1 : 0;   // else the kernel's 4-byte loads

  CUtensorMap tm_w, tm_h;
  if (!encode_bf16_rows(&tm_w, W, (uint64_t)V, (uint64_t)d, 128) ||
      !encode_bf16_rows(&tm_h, a->H, (uint64_t)R, (uint64_t)d, (uint32_t)plan.n_pad))
    return JD_ERR_CUDA;

  cudaStream_t st = (cudaStream_t)cuda_stream;
  // the array keeps the previous call's contents: the status word and the barrier counters
  // must start at zero, everything else is fully rewritten before it is read
  if (cudaMemsetAsync(own_status, 0, 512, st) != cudaSuccess) return JD_ERR_CUDA;
  if (device_status && cudaMemsetAsync(device_status, 0, sizeof(uint32_t), st) != cudaSuccess) return JD_ERR_CUDA;
  cudaError_t err = cudaSuccess;
  if (run_fused(cp, ws, tm_w, tm_h, a->H, w_judge, plan, st, &err, false, nullptr, nullptr, 0, /*plain_status=*/true) < 0) {
    cudaGetLastError();
    return JD_ERR_CUDA;
  }
  return JD_OK;
}
