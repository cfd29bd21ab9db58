// C-ABI layer: handle, argument validation, variant choice, host-buffer entry point.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>

#include "jd_kernels.h"

using namespace jd;

constexpr int kMaxGuards = 48;
constexpr size_t kGuardBytes = 256;
constexpr unsigned char kGuardByte = 0xC5;

struct jd_handle_s {
  jd_config_t cfg;
  int num_sms;
  void* ws_base;
  size_t ws_bytes;
  Workspace ws;
  const void* W;
  const void* w_judge;
  const float* w_scale;    // FP8 head: one scale per vocabulary row
  float b_judge;
  bool head_set;
  bool tm_w_ok;
  CUtensorMap tm_w;        // W as a [V, d] bf16 tensor, box 64 x 128, 128-byte swizzle
  CUtensorMap tm_w256;     // same tensor, box 64 x 256 (batched variant)
  cudaStream_t last_stream;
  SideStream side;         // batched variant: draft statistics run next to the GEMM
  int last_variant;
  int last_launches;
  bool needs_clear;        // the status / barrier block must be cleared by the host before the next launch
  // device staging of the host-buffer entry point (allocated on first use)
  void* st_H;
  int32_t* st_x;
  float* st_dl;
  void* st_out;            // accept_len | next_token | judge_scores | p_draft | q_draft | row_max | row_lse | masks
  size_t st_out_bytes;
  void* st_out_host;       // pinned mirror of st_out: the results come back in one copy
  // host-buffer calls copy the draft logits on the side stream while the verification starts
  unsigned* dl_flag;       // device word the side stream sets to dl_epoch when the copy has landed
  unsigned dl_epoch;
  cudaEvent_t dl_event;    // recorded on the side stream after that copy
  bool dl_in_flight;       // true only inside jd_verify_host, between enqueueing the copy and jd_verify
  // tensor map of the caller's H, kept from the previous call (decode loops reuse their buffers)
  CUtensorMap tm_h_cached;
  const void* tm_h_base;
  uint64_t tm_h_rows;
  uint32_t tm_h_box;
  bool tm_h_bytes;
  // guard blocks between the regions of the workspace (offsets into ws_base)
  int n_guards;
  size_t guard_off[kMaxGuards];
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// bf16 [rows, d] row-major tensor, box = 64 columns (128 bytes) x box_rows, 128-byte swizzle,
// out-of-range rows read as zero.
bool make_tensor_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t d, uint32_t box_rows,
                     bool bytes = false) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  // bf16: 64 elements per box row; 8-bit codes: 128 elements; 128 bytes either way
  const cuuint64_t dims[2] = {d, rows};
  const cuuint64_t strides[1] = {bytes ? d : d * 2};
  const cuuint32_t box[2] = {bytes ? 128u : 64u, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

typedef CUresult (*WriteValue32Fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);

WriteValue32Fn write_value32_fn() {
  static WriteValue32Fn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (WriteValue32Fn)p;
  }
  return fn;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool config_ok(const jd_config_t* c) {
  if (!c) return false;
  if (c->max_B < 1 || c->max_M < 1 || c->d < 1 || c->V < 2) return false;
  if (c->dtype != JD_DTYPE_F32 && c->dtype != JD_DTYPE_BF16 && c->dtype != JD_DTYPE_FP8_E4M3) return false;
  if ((int64_t)c->max_B * (c->max_M + 1) > (1 << 20)) return false;
  return true;
}

// Carves the workspace; with base == nullptr only measures it. Every region is followed by a guard
// block of kGuardBytes that no kernel may write; guard_off (optional) receives their offsets.
size_t carve(const jd_config_t& c, char* base, Workspace* ws, size_t* guard_off = nullptr, int* n_guards = nullptr,
             unsigned** dl_flag = nullptr) {
  const size_t maxB = c.max_B, maxR = (size_t)c.max_B * (c.max_M + 1), maxBM = (size_t)c.max_B * c.max_M;
  const size_t np = std::max<size_t>((c.V + kVocabTile - 1) / kVocabTile, kMaxCtas);
  const size_t nq = std::max<size_t>((c.V + 8191) / 8192, kMaxCtas);
  size_t off = 0;
  int ng = 0;
  auto take = [&](size_t bytes) {
    char* p = base ? base + off : nullptr;
    off += align_up(bytes, 256);
    if (guard_off && ng < kMaxGuards) guard_off[ng] = off;
    ++ng;
    off += kGuardBytes;
    return p;
  };
  Workspace w;
  w.part_max = (float*)take(maxR * np * 4);
  w.part_sum = (float*)take(maxR * np * 4);
  w.gath = (float*)take(maxR * 4);
  w.qpart_max = (float*)take(maxBM * nq * 4);
  w.qpart_sum = (float*)take(maxBM * nq * 4);
  w.qgath = (float*)take(maxBM * 4);
  w.judge_logit = (float*)take(maxBM * 4);
  w.row_max = (float*)take(maxR * 4);
  w.row_lse = (float*)take(maxR * 4);
  w.q_lse = (float*)take(maxBM * 4);
  w.sel_row = (int*)take(maxB * 4);
  w.sel_kind = (int*)take(maxB * 4);
  w.sel_lse_p = (float*)take(maxB * 4);
  w.sel_lse_q = (float*)take(maxB * 4);
  w.sel_u = (float*)take(maxB * 4);
  w.mass_r = (double*)take(maxB * np * 8);
  w.mass_p = (double*)take(maxB * np * 8);
  w.w_sel = (float*)take(maxB * (((size_t)c.V + kVocabTile - 1) / kVocabTile * kVocabTile) * 4);
  w.p_sel = (float*)take(maxB * (size_t)c.V * 4);
  w.h_sel = (__nv_bfloat16*)take(maxB * (size_t)c.d * 2);
  w.h8 = (uint8_t*)take(c.dtype == JD_DTYPE_FP8_E4M3 ? maxR * (size_t)c.d : 16);
  w.h_scale = (float*)take(maxR * 4);
  w.row_scale = (float*)take(maxR * 4);
  w.cnt = (int*)take(maxR * 4);
  w.argidx = (int*)take(maxR * 4);
  w.part_idx = (int*)take(maxR * np * 4);
  w.cand_ref = (float*)take(maxR * 4);
  w.own_i = (int*)take(maxB * 2 * 4);
  w.own_d = (double*)take(maxB * 2 * 8);
  w.status = (unsigned*)take(512);   // status word and, 256 bytes on, the barrier counters: one memset per call
  w.barrier = w.status ? w.status + 64 : nullptr;
  char* flag = take(256);   // word 0: arrival flag of a host-buffer call's draft logits; outside the per-call memset
  if (dl_flag) *dl_flag = (unsigned*)flag;
  w.np_cap = (int)np;
  w.nq_cap = (int)nq;
  if (ws) *ws = w;
  if (n_guards) *n_guards = ng < kMaxGuards ? ng : kMaxGuards;
  return off;
}

// bytes per element of H and w_judge (an FP8 head keeps bf16 activations)
size_t elem_size(int dtype) { return dtype == JD_DTYPE_F32 ? 4 : 2; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

bool configure_kernels() { return fused_configure() && batched_configure(); }

// The tensor map of the caller's H: re-encoded only when the pointer, the row count or the box changes.
const CUtensorMap* h_tensor_map(jd_handle_t h, const void* base, uint64_t rows, uint32_t box_rows, bool bytes) {
  if (h->tm_h_base != base || h->tm_h_rows != rows || h->tm_h_box != box_rows || h->tm_h_bytes != bytes) {
    h->tm_h_base = nullptr;
    if (!make_tensor_map(&h->tm_h_cached, base, rows, (uint64_t)h->cfg.d, box_rows, bytes)) return nullptr;
    h->tm_h_base = base; h->tm_h_rows = rows; h->tm_h_box = box_rows; h->tm_h_bytes = bytes;
  }
  return &h->tm_h_cached;
}

jd_status_t validate(jd_handle_t h, const jd_verify_args_t* a) {
  if (!h || !a) return JD_ERR_INVALID_ARG;
  if (!h->head_set) return JD_ERR_INVALID_ARG;
  if (a->B < 1 || a->B > h->cfg.max_B || a->M < 1 || a->M > h->cfg.max_M) return JD_ERR_INVALID_ARG;
  if (!a->H || !a->draft_tokens || !a->draft_logits) return JD_ERR_INVALID_ARG;
  if (!a->accept_len || !a->next_token || !a->judge_scores || !a->p_draft) return JD_ERR_INVALID_ARG;
  if (!(a->tau >= 0.f && a->tau <= 1.f)) return JD_ERR_INVALID_ARG;
  if (a->mode < JD_MODE_STANDARD || a->mode > JD_MODE_JUDGE_OR_STANDARD) return JD_ERR_INVALID_ARG;
  if (a->resample < JD_RESAMPLE_RESIDUAL || a->resample > JD_RESAMPLE_TARGET_P) return JD_ERR_INVALID_ARG;
  if (a->variant < JD_VARIANT_AUTO || a->variant > JD_VARIANT_BATCHED) return JD_ERR_INVALID_ARG;
  if (a->rule != JD_RULE_SAMPLING && a->rule != JD_RULE_TOPK) return JD_ERR_INVALID_ARG;
  if (a->rule == JD_RULE_TOPK && a->top_k < 1) return JD_ERR_INVALID_ARG;
  if (a->norm != JD_NORM_NONE && a->norm != JD_NORM_RMS) return JD_ERR_INVALID_ARG;
  if (a->norm == JD_NORM_RMS && !(a->rms_eps >= 0.f)) return JD_ERR_INVALID_ARG;
  // natural alignment of every 4-byte array (device or host); H is checked by the device entry point
  if (!aligned4(a->draft_tokens) || !aligned4(a->draft_logits) || !aligned4(a->accept_len) || !aligned4(a->next_token) ||
      !aligned4(a->judge_scores) || !aligned4(a->p_draft) || !aligned4(a->q_draft) || !aligned4(a->row_max) ||
      !aligned4(a->row_lse) || !aligned4(a->logits_debug))
    return JD_ERR_INVALID_ARG;
  return JD_OK;
}

}  // namespace

extern "C" {

int jd_version(void) { return 100; }

const char* jd_status_string(jd_status_t s) {
  switch (s) {
    case JD_OK: return "ok";
    case JD_ERR_INVALID_ARG: return "invalid argument";
    case JD_ERR_UNSUPPORTED: return "unsupported shape or dtype for the requested variant";
    case JD_ERR_ARCH: return "device is not compute capability 10.x";
    case JD_ERR_ALLOC: return "allocation failed";
    case JD_ERR_CUDA: return "CUDA call failed";
    case JD_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case JD_ERR_BAD_TOKEN: return "a draft token was outside the vocabulary and was clamped";
  }
  return "unknown status";
}

size_t jd_workspace_bytes(const jd_config_t* cfg) {
  if (!config_ok(cfg)) return 0;
  return carve(*cfg, nullptr, nullptr);
}

jd_status_t jd_create(jd_handle_t* out, const jd_config_t* cfg) {
  if (!out || !config_ok(cfg)) return JD_ERR_INVALID_ARG;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev) return JD_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return JD_ERR_CUDA;
  if (prop.major != 10) return JD_ERR_ARCH;
  if (cudaSetDevice(cfg->device) != cudaSuccess) return JD_ERR_CUDA;
  jd_handle_s* h = new (std::nothrow) jd_handle_s();
  if (!h) return JD_ERR_ALLOC;
  std::memset(h, 0, sizeof(*h));
  h->cfg = *cfg;
  h->num_sms = prop.multiProcessorCount;
  h->ws_bytes = carve(*cfg, nullptr, nullptr);
  if (cudaMalloc(&h->ws_base, h->ws_bytes) != cudaSuccess) {
    cudaGetLastError();
    delete h;
    return JD_ERR_ALLOC;
  }
  carve(*cfg, (char*)h->ws_base, &h->ws, h->guard_off, &h->n_guards, &h->dl_flag);
  bool filled = cudaMemset(h->ws_base, 0, h->ws_bytes) == cudaSuccess;
  for (int g = 0; g < h->n_guards && filled; ++g)
    filled = cudaMemset((char*)h->ws_base + h->guard_off[g], kGuardByte, kGuardBytes) == cudaSuccess;
  if (!filled || !configure_kernels()) {
    cudaGetLastError();
    cudaFree(h->ws_base);
    delete h;
    return JD_ERR_CUDA;
  }
  // the side stream is an optimisation: without it the batched variant runs its kernels in series
  if (cudaStreamCreateWithFlags(&h->side.stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->side.fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->side.join, cudaEventDisableTiming) != cudaSuccess) {
    cudaGetLastError();
    if (h->side.stream) cudaStreamDestroy(h->side.stream);
    if (h->side.fork) cudaEventDestroy(h->side.fork);
    if (h->side.join) cudaEventDestroy(h->side.join);
    h->side = SideStream{};
  }
  if (h->side.stream && cudaEventCreateWithFlags(&h->dl_event, cudaEventDisableTiming) != cudaSuccess) {
    cudaGetLastError();
    h->dl_event = nullptr;
  }
  *out = h;
  return JD_OK;
}

jd_status_t jd_destroy(jd_handle_t h) {
  if (!h) return JD_OK;
  cudaSetDevice(h->cfg.device);
  cudaDeviceSynchronize();
  if (h->side.stream) cudaStreamDestroy(h->side.stream);
  if (h->side.fork) cudaEventDestroy(h->side.fork);
  if (h->side.join) cudaEventDestroy(h->side.join);
  if (h->dl_event) cudaEventDestroy(h->dl_event);
  cudaFree(h->ws_base);
  cudaFree(h->st_H);
  cudaFree(h->st_x);
  cudaFree(h->st_dl);
  cudaFree(h->st_out);
  if (h->st_out_host) cudaFreeHost(h->st_out_host);
  delete h;
  return JD_OK;
}

jd_status_t jd_set_head_fp8(jd_handle_t h, const void* W8, const float* w_scale, const void* w_judge, float b_judge) {
  if (!h || !W8 || !w_scale || !w_judge) return JD_ERR_INVALID_ARG;
  if (h->cfg.dtype != JD_DTYPE_FP8_E4M3) return JD_ERR_INVALID_ARG;
  if (!aligned16(W8) || !aligned16(w_judge)) return JD_ERR_INVALID_ARG;
  h->W = W8;
  h->w_scale = w_scale;
  h->w_judge = w_judge;
  h->b_judge = b_judge;
  h->head_set = true;
  h->tm_w_ok = false;
  if (h->cfg.d % 128 == 0)
    h->tm_w_ok = make_tensor_map(&h->tm_w, W8, (uint64_t)h->cfg.V, (uint64_t)h->cfg.d, 128, true) &&
                 make_tensor_map(&h->tm_w256, W8, (uint64_t)h->cfg.V, (uint64_t)h->cfg.d, 256, true);
  return JD_OK;
}

jd_status_t jd_set_head(jd_handle_t h, const void* W, const void* w_judge, float b_judge) {
  if (!h || !W || !w_judge) return JD_ERR_INVALID_ARG;
  if (h->cfg.dtype == JD_DTYPE_FP8_E4M3) return JD_ERR_INVALID_ARG;   // use jd_set_head_fp8
  if (!aligned16(W) || !aligned16(w_judge)) return JD_ERR_INVALID_ARG;
  h->W = W;
  h->w_judge = w_judge;
  h->b_judge = b_judge;
  h->head_set = true;
  h->tm_w_ok = false;
  if (h->cfg.dtype == JD_DTYPE_BF16 && h->cfg.d % 64 == 0)
    h->tm_w_ok = make_tensor_map(&h->tm_w, W, (uint64_t)h->cfg.V, (uint64_t)h->cfg.d, 128) &&
                 make_tensor_map(&h->tm_w256, W, (uint64_t)h->cfg.V, (uint64_t)h->cfg.d, 256);
  return JD_OK;
}

jd_status_t jd_verify(jd_handle_t h, const jd_verify_args_t* a, void* cuda_stream) {
  jd_status_t v = validate(h, a);
  if (v != JD_OK) return v;
  if (!aligned16(a->H)) return JD_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const jd_config_t& c = h->cfg;
  const int R = a->B * (a->M + 1);

  CallParams cp;
  cp.B = a->B; cp.M = a->M; cp.d = c.d; cp.V = c.V;
  cp.draft_tokens = a->draft_tokens;
  cp.draft_logits = a->draft_logits;
  cp.tau = a->tau; cp.b_judge = h->b_judge; cp.seed = a->seed;
  cp.mode = a->mode; cp.resample = a->resample;
  cp.rule = a->rule; cp.top_k = a->top_k;
  cp.norm = a->norm; cp.rms_eps = a->rms_eps;
  cp.accept_len = a->accept_len; cp.next_token = a->next_token;
  cp.judge_scores = a->judge_scores; cp.p_draft = a->p_draft;
  cp.q_draft = a->q_draft; cp.masks = a->masks;
  cp.row_max_out = a->row_max; cp.row_lse_out = a->row_lse;
  cp.logits_debug = a->logits_debug;
  // 16-byte loads of the draft logits need every row on a 16-byte boundary; a 4-byte-aligned view
  // (a slice of a larger buffer) takes the kernels' 4-byte path instead
  cp.dl_vec4 = (c.V % 4 == 0 && aligned16(a->draft_logits)) ? 1 : 0;

  FusedPlan plan;
  const bool fused_ok = h->tm_w_ok && fused_supported(c.dtype, R, c.d, c.V, h->num_sms, &plan);
  const bool fp8 = c.dtype == JD_DTYPE_FP8_E4M3;
  const bool batched_ok = h->tm_w_ok && batched_supported(c.dtype, a->B, c.d, c.V, h->num_sms);
  int variant = a->variant;
  if (variant == JD_VARIANT_AUTO) {
    if (fused_ok) variant = JD_VARIANT_FUSED;
    else if (batched_ok) variant = JD_VARIANT_BATCHED;
    else variant = JD_VARIANT_SIMT;
  }
  if (variant == JD_VARIANT_FUSED && !fused_ok) return JD_ERR_UNSUPPORTED;
  if (variant == JD_VARIANT_BATCHED && !batched_ok) return JD_ERR_UNSUPPORTED;

  if (cudaSetDevice(c.device) != cudaSuccess) return JD_ERR_CUDA;
  // Status word and barrier block. The fused kernel keeps them clean across its own launches, so a fused call
  // that follows a fused call enqueues no memset; anything else (another variant before or now, an uncleared
  // timeout, the handle's first call) starts from zeroes.
  if (variant != JD_VARIANT_FUSED || h->last_variant != JD_VARIANT_FUSED || h->needs_clear) {
    if (cudaMemsetAsync(h->ws.status, 0, 512, st) != cudaSuccess) return JD_ERR_CUDA;
    h->needs_clear = false;
  }
  if (a->rule == JD_RULE_TOPK) {   // rank counters start at zero, argmax candidates at a large id
    if (cudaMemsetAsync(h->ws.cnt, 0, (size_t)R * 4, st) != cudaSuccess ||
        cudaMemsetAsync(h->ws.argidx, 0x7F, (size_t)R * 4, st) != cudaSuccess)
      return JD_ERR_CUDA;
  }
  int launches = 0;
  if (a->norm == JD_NORM_RMS) {   // per-row normalisation factors, read by every variant
    launch_row_scale(cp, h->ws, a->H, c.dtype == JD_DTYPE_F32 ? JD_DTYPE_F32 : JD_DTYPE_BF16, st);
    launches = 1;
  }
  if (fp8) {   // rows of H to E4M3 with one scale per row; the judge keeps reading a->H
    launch_quantize_rows(cp, h->ws, a->H, st);
    launches += 1;
  }
  if (h->dl_in_flight && variant != JD_VARIANT_FUSED) {
    // Draft logits still being copied on the side stream: the batched variant reads them there first
    // (its statistics kernels follow the copy in stream order) and here only after the join; the
    // CUDA-core variant waits for the copy. The fused kernel is told where to look instead.
    if (variant == JD_VARIANT_SIMT && cudaStreamWaitEvent(st, h->dl_event, 0) != cudaSuccess) return JD_ERR_CUDA;
  }
  if (variant == JD_VARIANT_SIMT) {
    launches += run_simt(cp, h->ws, h->W, h->w_scale, h->w_judge, a->H, c.dtype, st);
  } else if (variant == JD_VARIANT_BATCHED) {
    // second pass: the selected rows go through the fused kernel, a chunk of sequences per launch
    const int chunk = second_pass_chunk(a->B), tail = a->B % chunk;
    FusedPlan plan2, plan3;
    if (!fused_supported(c.dtype, chunk, c.d, c.V, h->num_sms, &plan2)) return JD_ERR_UNSUPPORTED;
    if (tail && !fused_supported(c.dtype, tail, c.d, c.V, h->num_sms, &plan3)) return JD_ERR_UNSUPPORTED;
    CUtensorMap tm_hsel, tm_hsel_tail;
    const CUtensorMap* tm_hp = h_tensor_map(h, fp8 ? (const void*)h->ws.h8 : a->H, (uint64_t)R, 128, fp8);
    if (!tm_hp) return JD_ERR_CUDA;
    const CUtensorMap& tm_h = *tm_hp;
    if (!make_tensor_map(&tm_hsel, h->ws.h_sel, (uint64_t)chunk, (uint64_t)c.d, (uint32_t)plan2.n_pad, fp8))
      return JD_ERR_CUDA;
    tm_hsel_tail = tm_hsel;
    if (tail && !make_tensor_map(&tm_hsel_tail, h->ws.h_sel, (uint64_t)tail, (uint64_t)c.d, (uint32_t)plan3.n_pad, fp8))
      return JD_ERR_CUDA;
    cudaError_t err = cudaSuccess;
    const int n = run_batched(cp, h->ws, h->tm_w256, h->tm_w, tm_h, tm_hsel, tm_hsel_tail, a->H, h->w_judge, h->num_sms,
                              st, h->side, &err, fp8 ? h->w_scale : nullptr, h->W);
    if (n < 0) return JD_ERR_CUDA;
    launches += n;
  } else {
    const CUtensorMap* tm_hp = h_tensor_map(h, fp8 ? (const void*)h->ws.h8 : a->H, (uint64_t)R, (uint32_t)plan.n_pad, fp8);
    if (!tm_hp) return JD_ERR_CUDA;
    cudaError_t err = cudaSuccess;
    const int n = run_fused(cp, h->ws, h->tm_w, *tm_hp, a->H, h->w_judge, plan, st, &err, false, fp8 ? h->w_scale : nullptr,
                            h->dl_in_flight ? h->dl_flag : nullptr, h->dl_epoch);
    if (n < 0) return JD_ERR_CUDA;
    launches += n;
  }
  if (cudaGetLastError() != cudaSuccess) return JD_ERR_CUDA;
  h->last_stream = st;
  h->last_variant = variant;
  h->last_launches = launches;
  return JD_OK;
}

jd_status_t jd_verify_host(jd_handle_t h, const jd_verify_args_t* a, void* cuda_stream) {
  jd_status_t v = validate(h, a);
  if (v != JD_OK) return v;
  if (a->logits_debug) return JD_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const jd_config_t& c = h->cfg;
  if (cudaSetDevice(c.device) != cudaSuccess) return JD_ERR_CUDA;
  const size_t maxB = c.max_B, maxR = (size_t)c.max_B * (c.max_M + 1), maxBM = (size_t)c.max_B * c.max_M;
  if (!h->st_H) {
    h->st_out_bytes = align_up(maxB * 4, 256) * 2 + align_up(maxBM * 4, 256) * 3 + align_up(maxR * 4, 256) * 2 +
                      align_up(maxBM, 256);
    if (cudaMalloc(&h->st_H, maxR * c.d * elem_size(c.dtype)) != cudaSuccess ||
        cudaMalloc((void**)&h->st_x, maxBM * 4) != cudaSuccess ||
        cudaMalloc((void**)&h->st_dl, maxBM * (size_t)c.V * 4) != cudaSuccess ||
        cudaMalloc(&h->st_out, h->st_out_bytes) != cudaSuccess ||
        cudaMallocHost(&h->st_out_host, h->st_out_bytes) != cudaSuccess) {
      cudaGetLastError();
      cudaFree(h->st_H); cudaFree(h->st_x); cudaFree(h->st_dl); cudaFree(h->st_out);
      if (h->st_out_host) cudaFreeHost(h->st_out_host);
      h->st_H = nullptr; h->st_x = nullptr; h->st_dl = nullptr; h->st_out = nullptr; h->st_out_host = nullptr;
      return JD_ERR_ALLOC;
    }
  }
  const size_t B = a->B, R = (size_t)a->B * (a->M + 1), BM = (size_t)a->B * a->M;
  char* o = (char*)h->st_out;
  size_t off = 0;
  auto take = [&](size_t bytes) { char* p = o + off; off += align_up(bytes, 256); return p; };
  int32_t* d_acc = (int32_t*)take(maxB * 4);
  int32_t* d_next = (int32_t*)take(maxB * 4);
  float* d_js = (float*)take(maxBM * 4);
  float* d_pd = (float*)take(maxBM * 4);
  float* d_qd = (float*)take(maxBM * 4);
  float* d_rm = (float*)take(maxR * 4);
  float* d_rl = (float*)take(maxR * 4);
  uint8_t* d_mk = (uint8_t*)take(maxBM);

  if (cudaMemcpyAsync(h->st_H, a->H, R * c.d * elem_size(c.dtype), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(h->st_x, a->draft_tokens, BM * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return JD_ERR_CUDA;
  // The draft logits are most of the bytes. They go over on the side stream, so that the verification
  // can start as soon as H and the tokens are in; whoever reads them first waits for them (see jd_verify).
  // Every earlier use of the staging buffer has finished: this function synchronises before it returns.
  WriteValue32Fn write_value = write_value32_fn();
  const bool overlap = h->side.stream && h->dl_event && write_value;
  cudaStream_t dl_stream = overlap ? h->side.stream : st;
  if (cudaMemcpyAsync(h->st_dl, a->draft_logits, BM * (size_t)c.V * 4, cudaMemcpyHostToDevice, dl_stream) != cudaSuccess)
    return JD_ERR_CUDA;
  if (overlap) {
    h->dl_epoch += 1;
    if (write_value((CUstream)dl_stream, (CUdeviceptr)(uintptr_t)h->dl_flag, h->dl_epoch, 0) != CUDA_SUCCESS ||
        cudaEventRecord(h->dl_event, dl_stream) != cudaSuccess) {
      cudaStreamSynchronize(dl_stream);
      return JD_ERR_CUDA;
    }
    h->dl_in_flight = true;
  }

  jd_verify_args_t dev = *a;
  dev.H = h->st_H; dev.draft_tokens = h->st_x; dev.draft_logits = h->st_dl;
  dev.accept_len = d_acc; dev.next_token = d_next; dev.judge_scores = d_js; dev.p_draft = d_pd;
  dev.q_draft = a->q_draft ? d_qd : nullptr;
  dev.masks = a->masks ? d_mk : nullptr;
  dev.row_max = a->row_max ? d_rm : nullptr;
  dev.row_lse = a->row_lse ? d_rl : nullptr;
  jd_status_t s = jd_verify(h, &dev, cuda_stream);
  if (overlap) {
    h->dl_in_flight = false;
    if (s != JD_OK) cudaStreamSynchronize(dl_stream);   // the caller's buffer must not be in use when we return
  }
  if (s != JD_OK) return s;

  // all results in one device-to-host copy (the sections are a few KB), then plain host copies
  if (cudaMemcpyAsync(h->st_out_host, h->st_out, off, cudaMemcpyDeviceToHost, st) != cudaSuccess) return JD_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return JD_ERR_CUDA;
  auto back = [&](void* dst, const void* dev_section, size_t bytes) {
    if (dst) std::memcpy(dst, (const char*)h->st_out_host + ((const char*)dev_section - o), bytes);
  };
  back(a->accept_len, d_acc, B * 4);
  back(a->next_token, d_next, B * 4);
  back(a->judge_scores, d_js, BM * 4);
  back(a->p_draft, d_pd, BM * 4);
  back(a->q_draft, d_qd, BM * 4);
  back(a->masks, d_mk, BM);
  back(a->row_max, d_rm, R * 4);
  back(a->row_lse, d_rl, R * 4);
  return JD_OK;
}

jd_status_t jd_last_device_status(jd_handle_t h, int* out) {
  if (!h || !out) return JD_ERR_INVALID_ARG;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return JD_ERR_CUDA;
  if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) return JD_ERR_CUDA;
  // status word and, 256 bytes on, the barrier block with the fused kernel's launch counter
  unsigned blk[64 + kCallCounter + 1];
  if (cudaMemcpy(blk, h->ws.status, sizeof(blk), cudaMemcpyDeviceToHost) != cudaSuccess) return JD_ERR_CUDA;
  const unsigned word = blk[0], done = blk[64 + kCallCounter];
  const unsigned tag = word >> 8, code = word & 0xFFu;
  // untagged: written since the host last cleared the block; tagged: by the last launch that finished
  // (tag == done) or by one that gave up (tag == done + 1). Older tags belong to earlier calls.
  const bool current = tag == 0u || tag == (done & 0xFFFFFFu) || tag == ((done + 1u) & 0xFFFFFFu);   // tags are 24 bits
  *out = current ? (int)code : (int)JD_OK;
  if (*out == JD_ERR_TIMEOUT) h->needs_clear = true;   // the counters of a launch that gave up are in an unknown state
  return JD_OK;
}

jd_status_t jd_selftest_timeout(jd_handle_t h, uint32_t spin_limit, void* cuda_stream) {
  if (!h || spin_limit < 1 || spin_limit > (1u << 20)) return JD_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return JD_ERR_CUDA;
  if (cudaMemsetAsync(h->ws.status, 0, 512, st) != cudaSuccess) return JD_ERR_CUDA;
  launch_timeout_probe(h->ws, spin_limit, st);
  if (cudaGetLastError() != cudaSuccess) return JD_ERR_CUDA;
  h->needs_clear = true;
  h->last_stream = st;
  return JD_OK;
}

jd_status_t jd_selftest_stale_timeout(jd_handle_t h, void* cuda_stream) {
  if (!h) return JD_ERR_INVALID_ARG;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return JD_ERR_CUDA;
  launch_stale_timeout(h->ws, (cudaStream_t)cuda_stream);
  if (cudaGetLastError() != cudaSuccess) return JD_ERR_CUDA;
  h->last_stream = (cudaStream_t)cuda_stream;
  return JD_OK;   // on purpose not remembered on the host: the device-side rule is what is being tested
}

jd_status_t jd_debug_phase_stamps(uint64_t* out, int32_t capacity) {
  if (!out || capacity < kMaxCtas * kPhaseStampSlots) return JD_ERR_INVALID_ARG;
  static_assert(sizeof(uint64_t) == sizeof(unsigned long long), "stamp type");
  return read_phase_stamps(reinterpret_cast<unsigned long long*>(out)) ? JD_OK : JD_ERR_UNSUPPORTED;
}

jd_status_t jd_stream_read_probe(const void* data, size_t bytes, uint32_t* out, void* cuda_stream) {
  if (!data || !out || bytes < 16 || !aligned16(data)) return JD_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return JD_ERR_CUDA;
  launch_stream_read(data, bytes, out, sms, (cudaStream_t)cuda_stream);
  return cudaGetLastError() == cudaSuccess ? JD_OK : JD_ERR_CUDA;
}

jd_status_t jd_last_launch_info(jd_handle_t h, int* variant, int* kernel_launches) {
  if (!h) return JD_ERR_INVALID_ARG;
  if (variant) *variant = h->last_variant;
  if (kernel_launches) *kernel_launches = h->last_launches;
  return JD_OK;
}

jd_status_t jd_philox_uniforms(uint64_t seed, const int32_t* b, const int32_t* slot, const int32_t* stream,
                               int32_t n, float* out, void* cuda_stream) {
  if (!b || !slot || !stream || !out || n < 0) return JD_ERR_INVALID_ARG;
  if (n == 0) return JD_OK;
  launch_philox_uniforms(seed, b, slot, stream, n, out, (cudaStream_t)cuda_stream);
  return cudaGetLastError() == cudaSuccess ? JD_OK : JD_ERR_CUDA;
}

jd_status_t jd_quantize_rows_e4m3(const void* H, int32_t rows, int32_t d, uint8_t* codes, float* scale,
                                  void* cuda_stream) {
  if (!H || !codes || !scale || rows < 1 || d < 1) return JD_ERR_INVALID_ARG;
  if (!aligned16(H) || !aligned16(codes) || !aligned4(scale)) return JD_ERR_INVALID_ARG;
  CallParams cp = {};
  cp.B = rows; cp.M = 0; cp.d = d;   // rows x 1 "sequences": the launcher quantises B * (M + 1) rows
  Workspace ws = {};
  ws.h8 = codes;
  ws.h_scale = scale;
  launch_quantize_rows(cp, ws, H, (cudaStream_t)cuda_stream);
  return cudaGetLastError() == cudaSuccess ? JD_OK : JD_ERR_CUDA;
}

jd_status_t jd_check_workspace_guards(jd_handle_t h, int32_t* damaged) {
  if (!h || !damaged) return JD_ERR_INVALID_ARG;
  if (cudaSetDevice(h->cfg.device) != cudaSuccess) return JD_ERR_CUDA;
  if (cudaDeviceSynchronize() != cudaSuccess) return JD_ERR_CUDA;
  unsigned char block[kGuardBytes];
  int bad = 0;
  for (int g = 0; g < h->n_guards; ++g) {
    if (cudaMemcpy(block, (const char*)h->ws_base + h->guard_off[g], kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess)
      return JD_ERR_CUDA;
    for (size_t i = 0; i < kGuardBytes; ++i)
      if (block[i] != kGuardByte) { ++bad; break; }
  }
  *damaged = bad;
  return JD_OK;
}

}  // extern "C"
