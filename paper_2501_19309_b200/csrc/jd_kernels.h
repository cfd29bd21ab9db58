// Internal interface between the C-ABI layer and the kernel families.
#pragma once

#include <cuda.h>

#include "jd_common.cuh"

namespace jd {

// CUDA-core pipeline (jd_simt.cu). Each returns after enqueueing on `st`.
int run_simt(const CallParams& cp, const Workspace& ws, const void* W, const float* w_scale, const void* w_judge,
             const void* H, int dtype, cudaStream_t st);
int launch_q_stats(const CallParams& cp, const Workspace& ws, cudaStream_t st);   // returns partials per draft row
void launch_judge(const CallParams& cp, const Workspace& ws, const void* H, const void* w, int dtype, cudaStream_t st);
void launch_quantize_rows(const CallParams& cp, const Workspace& ws, const void* H_bf16, cudaStream_t st);
void launch_row_scale(const CallParams& cp, const Workspace& ws, const void* H, int dtype, cudaStream_t st);
// fold_arg: also folds the per-tile argmax candidates in ws.part_idx into ws.argidx (batched variant, top-K rule)
void launch_fold(const CallParams& cp, const Workspace& ws, int np, int nq, cudaStream_t st, bool fold_arg = false);
void launch_decide(const CallParams& cp, const Workspace& ws, cudaStream_t st);
void launch_locate(const CallParams& cp, const Workspace& ws, int np, cudaStream_t st);
void launch_stream_read(const void* p, size_t bytes, uint32_t* out, int num_sms, cudaStream_t st);
void launch_philox_uniforms(uint64_t seed, const int32_t* b, const int32_t* slot, const int32_t* stream, int n,
                            float* out, cudaStream_t st);

// Persistent tensor-core kernel with the logits parked in tensor memory (jd_fused_sm100.cu).
struct FusedPlan {
  int num_ctas;       // persistent grid = number of SMs
  int n_pad;          // MMA N: rows padded to a multiple of 16
  int max_tiles;      // vocabulary tiles of the busiest CTA
  int tmem_tiles;     // tiles whose accumulators stay in tensor memory
  int tile_stride;    // TMEM columns between consecutive tiles
  size_t smem_bytes;  // dynamic shared memory of the launch
  int stages;         // W ring depth
  int h_stages;       // H ring depth
};
// Raises the dynamic shared-memory limit of every instantiation of a family's kernels on the CURRENT
// device (which also loads them), once per device, ahead of the first launch: the launch paths set no
// function attributes themselves.
constexpr int kMaxDynamicSmem = 227 * 1024;
bool fused_configure();
bool batched_configure();
// Phase stamps of the fused kernel's last launch (builds with -DJD_PHASE_STAMPS only; false otherwise):
// kMaxCtas x kPhaseStampSlots global-timer values in ns, slot = 0 start of the epilogue, 1 draft statistics and
// judge dots done, 12 early sweep complete, 2 stream complete, 3 row statistics done, 4 barrier 1 passed,
// 5 fold done, 6 barrier 2 passed, 7 decisions done, 8 sampling masses done, 9 barrier 3 passed, 10 owner
// found, 11 end of the epilogue, 13 the previous launch's slot 11, 14 statistics (sample-only mode: masses) of the
// early tiles done.
constexpr int kPhaseStampSlots = 16;
bool read_phase_stamps(unsigned long long* host_out);
void launch_timeout_probe(const Workspace& ws, unsigned limit, cudaStream_t st);
void launch_stale_timeout(const Workspace& ws, cudaStream_t st);
bool fused_supported(int dtype, int R, int d, int V, int num_sms, FusedPlan* plan);
// Returns the number of kernels launched, or -1 with *err set. dl_flag (optional): a device word
// that another stream sets to dl_epoch once the draft logits have been copied in; the kernel then
// starts streaming W at once and waits for the word before it first reads the draft logits.
// plain_status: the caller clears ws.status and ws.barrier before every launch and wants untagged status
// codes; otherwise the kernel keeps the barrier block clean across launches by itself (jd_common.cuh).
int run_fused(const CallParams& cp, const Workspace& ws, const CUtensorMap& tmW, const CUtensorMap& tmH,
              const void* H, const void* w_judge, const FusedPlan& plan, cudaStream_t st, cudaError_t* err,
              bool sample_only = false, const float* w_scale_fp8 = nullptr, const unsigned* dl_flag = nullptr,
              unsigned dl_epoch = 0, bool plain_status = false);

// Two-pass tensor-core variant for many rows (jd_batched_sm100.cu). tmW256 / tmW128: W with
// 256- and 128-row boxes; tmH: H with a 128-row box; tmHsel: the handle's [B, d] gather buffer
// with the fused plan's box. With w_scale_fp8 set, W is E4M3 and tmH / tmHsel describe the
// quantised rows (ws.h8) and the gather buffer as bytes. Returns the number of kernels launched, or -1 with *err set.
// Optional second stream of a handle (with the two events that fork to it and join from it).
struct SideStream {
  cudaStream_t stream;
  cudaEvent_t fork, join;
};
// The second pass takes up to 96 sequences in one launch; larger batches go through it 64 at a time
// (64 selected rows x 7 tiles fill tensor memory exactly), each launch streaming W once more.
// second_pass_chunk(B) = sequences per launch; tmHsel / tmHselTail describe the gather buffer for a
// whole chunk and for the ragged last one (ignored when B is a multiple of the chunk).
constexpr int kSecondPassMax = 96;
constexpr int kSecondPassChunk = 64;
inline int second_pass_chunk(int B) { return B <= kSecondPassMax ? B : kSecondPassChunk; }
bool batched_supported(int dtype, int B, int d, int V, int num_sms);
int run_batched(const CallParams& cp, const Workspace& ws, const CUtensorMap& tmW256, const CUtensorMap& tmW128,
                const CUtensorMap& tmH, const CUtensorMap& tmHsel, const CUtensorMap& tmHselTail, const void* H,
                const void* w_judge, int num_sms, cudaStream_t st, const SideStream& side, cudaError_t* err,
                const float* w_scale_fp8 = nullptr, const void* W = nullptr);

}  // namespace jd
