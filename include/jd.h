/*
 * jd.h - C ABI of the judge-decoding verification step for NVIDIA B200 (sm_100a).
 *
 * One call, jd_verify, performs what follows every target-model forward over a block of M
 * draft tokens in judge decoding (arXiv 2501.19309):
 *   1. LM-head projection of the target's last-layer embeddings, L = H W^T      (Sec. 3.1, Eq. 2)
 *   2. softmax over the vocabulary, p_j = softmax(L[j,:]), and q_j = softmax(draft logits)
 *   3. the standard speculative-sampling test u_j q_j[x_j] < p_j[x_j]            (Sec. 3.1, Eq. 4)
 *      and the judge test sigmoid(w . H[b,j+1] + b0) > tau                      (Sec. 4.1 "Inference")
 *   4. mask = standard OR judge (or one of them), accepted prefix length        (Sec. 4.1; App. B.2)
 *   5. the next token: from normalised max(0, p - q) at the first rejection, from the extra
 *      row p_M after a fully accepted block                                     (Sec. 3.1, after Eq. 4)
 * The logits exist only on chip; they are never written to device memory unless the
 * test-only logits_debug pointer is set.
 *
 * Conventions
 *   - Indices are 0-based. Row j of H[b] (j = 0..M) yields p_j, the target distribution of draft
 *     slot j; row 0 belongs to the last context token, row j >= 1 to draft token j-1. The judge
 *     score of draft token j is read from row j+1. Row M also yields the bonus distribution.
 *   - All tensors are dense, row-major (last index fastest).
 *   - Unless a function says "host", every data pointer is a DEVICE pointer owned by the caller.
 *     The library never frees or keeps caller memory, except that W and w_judge given to
 *     jd_set_head are borrowed until the next jd_set_head or jd_destroy.
 *   - jd_verify is asynchronous on the given CUDA stream and never synchronises it.
 *   - No function throws, prints or exits; every failure is a jd_status_t.
 *   - Uniforms: Philox4x32-10, key = (seed low word, seed high word), counter =
 *     (b, slot, stream, 0), first output word, u = (word >> 8) * 2^-24. stream 0 is the
 *     acceptance draw of slot j, stream 1 the token draw at slot accept_len[b].
 */
#ifndef JD_H_
#define JD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  JD_OK = 0,
  JD_ERR_INVALID_ARG = 1, /* null pointer, size out of range, bad enum, misaligned pointer */
  JD_ERR_UNSUPPORTED = 2, /* shape or dtype that no kernel variant covers */
  JD_ERR_ARCH = 3,        /* the current device is not compute capability 10.x */
  JD_ERR_ALLOC = 4,       /* device or host allocation failed */
  JD_ERR_CUDA = 5,        /* a CUDA runtime or driver call failed */
  JD_ERR_TIMEOUT = 6,     /* device status: a bounded wait inside a kernel ran out */
  JD_ERR_BAD_TOKEN = 7    /* device status: a draft token was outside [0, V) and was clamped */
} jd_status_t;

/* Storage type of the head. F32 / BF16: W, H and w_judge all have that type. FP8_E4M3: W holds
 * FP8 E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities) with one
 * float32 scale per vocabulary row, registered with jd_set_head_fp8; H and w_judge are bf16. */
typedef enum { JD_DTYPE_F32 = 0, JD_DTYPE_BF16 = 1, JD_DTYPE_FP8_E4M3 = 2 } jd_dtype_t;

/* Which tests form the accept mask (Sec. 4.1 "Inference"): the standard test alone (Eq. 4),
 * the judge alone, or their logical OR (the paper's judge decoding). */
typedef enum { JD_MODE_STANDARD = 0, JD_MODE_JUDGE = 1, JD_MODE_JUDGE_OR_STANDARD = 2 } jd_mode_t;

/* Distribution of the token drawn at the first rejected slot a < M.
 * RESIDUAL: normalised max(0, p_a - q_a), the form under which the standard test is lossless;
 *           an identically zero residual falls back to p_a.
 * TARGET_P: p_a itself, which is how Sec. 3.1 words the correction when read literally.
 * After a fully accepted block the token always comes from p_M. */
typedef enum { JD_RESAMPLE_RESIDUAL = 0, JD_RESAMPLE_TARGET_P = 1 } jd_resample_t;

/* How the standard (non-judge) test decides, and how the next token is chosen.
 * SAMPLING: the stochastic test of Eq. 4 with the residual / bonus draw described above.
 * TOPK:     deterministic verification: the candidate passes iff it is among the top_k highest-valued
 *           entries of p_j (Sec. 5.1 "Training-free baseline"); top_k = 1 is greedy verification
 *           (acceptance against a greedily decoded target, Sec. 3.2), top_k = V accepts everything. The next
 *           token is the target's greedy token argmax p_a, at a rejection and after a full block.
 *           Equal logits rank by token id (lower id first); the batched variant compares the row against
 *           a float32 dot product for the candidate, so there an entry equal to the candidate's logit to
 *           within float32 summation order may rank on either side of it. No uniform is drawn; the
 *           draft logits only feed the q_draft output. */
typedef enum { JD_RULE_SAMPLING = 0, JD_RULE_TOPK = 1 } jd_rule_t;

/* Normalisation applied to the rows of H in front of the LM head. The paper's judge takes the last
 * embedding ahead of the model's final RMS norm and LM head (Sec. 4.1 "Model design and training"):
 * with JD_NORM_RMS the logits are W . (H[b,j] / sqrt(mean_k H[b,j,k]^2 + rms_eps)) while the judge
 * dot product still uses H[b,j+1] as given. The norm's gain vector is expected folded into W. */
typedef enum { JD_NORM_NONE = 0, JD_NORM_RMS = 1 } jd_norm_t;

/* Kernel family used by jd_verify. AUTO picks the fastest one that supports the shape. */
typedef enum {
  JD_VARIANT_AUTO = 0,
  JD_VARIANT_SIMT = 1,   /* CUDA-core reference pipeline: any shape; f32, bf16 or FP8 head */
  JD_VARIANT_FUSED = 2,  /* one persistent tcgen05/TMA kernel, logits parked in tensor memory;
                            bf16 with d % 64 == 0 or FP8 head with d % 128 == 0, B*(M+1) <= 96, V
                            small enough for every CTA to keep its vocabulary tiles on chip
                            (128256 fits on 148 SMs) */
  JD_VARIANT_BATCHED = 3 /* tcgen05 GEMM with fused statistics + second pass over the selected
                            rows (one launch per 64 sequences beyond 96); same dtypes and d as
                            the fused variant, any number of rows and sequences */
} jd_variant_t;

typedef struct {
  int32_t max_B;    /* largest number of sequences per call, >= 1 */
  int32_t max_M;    /* largest number of draft tokens per sequence, >= 1 */
  int32_t d;        /* embedding width */
  int32_t V;        /* vocabulary size */
  int32_t dtype;    /* jd_dtype_t: storage type of W, H and w_judge */
  int32_t device;   /* CUDA device ordinal the handle lives on */
} jd_config_t;

typedef struct jd_handle_s* jd_handle_t;

typedef struct {
  int32_t B;                   /* sequences in this call, 1..max_B */
  int32_t M;                   /* draft tokens per sequence, 1..max_M */
  const void* H;               /* [B, M+1, d] embeddings, dtype of the handle (bf16 for an FP8 head),
                                  16-byte aligned */
  const int32_t* draft_tokens; /* [B, M] drafted token ids x_j in [0, V) */
  const float* draft_logits;   /* [B, M, V] draft-model logits; q_j = softmax at temperature 1. 4-byte aligned
                                  like every int32 / float array here; a 16-byte aligned base with V % 4 == 0
                                  lets the kernels use 16-byte loads, anything else takes 4-byte loads */
  float tau;                   /* judge threshold in [0, 1]; accept iff score > tau (strict) */
  uint64_t seed;               /* Philox key */
  int32_t mode;                /* jd_mode_t */
  int32_t resample;            /* jd_resample_t */
  int32_t variant;             /* jd_variant_t; JD_VARIANT_AUTO in production */
  int32_t rule;                /* jd_rule_t */
  int32_t top_k;               /* K of JD_RULE_TOPK, >= 1; ignored by JD_RULE_SAMPLING */
  int32_t norm;                /* jd_norm_t */
  float rms_eps;               /* epsilon of JD_NORM_RMS, >= 0 */
  /* outputs, always written */
  int32_t* accept_len;         /* [B] number of accepted draft tokens, 0..M */
  int32_t* next_token;         /* [B] the corrected (accept_len < M) or bonus (== M) token */
  float* judge_scores;         /* [B, M] sigmoid(w . H[b,j+1] + b0) */
  float* p_draft;              /* [B, M] p_j[x_j] */
  /* optional outputs, may be NULL */
  float* q_draft;              /* [B, M] q_j[x_j] */
  uint8_t* masks;              /* [B, M] bit0 = standard test passed, bit1 = judge test passed */
  float* row_max;              /* [B, M+1] max_v L[b,j,v] */
  float* row_lse;              /* [B, M+1] log sum_v exp L[b,j,v] */
  float* logits_debug;         /* [B, M+1, V] the logits as the softmax sees them (normalisation and FP8
                                  scales applied); tests only: every variant honours it, at the price of
                                  writing R x V floats */
} jd_verify_args_t;

/* Library version, major*10000 + minor*100 + patch. */
int jd_version(void);

/* Static text for a status code; never NULL. */
const char* jd_status_string(jd_status_t s);

/* Bytes of device workspace a handle with this configuration allocates (informational;
 * the handle owns its workspace). Returns 0 for an invalid configuration. */
size_t jd_workspace_bytes(const jd_config_t* cfg);

/* Creates a handle on cfg->device: checks the architecture (JD_ERR_ARCH unless compute
 * capability 10.x), allocates the workspace (JD_ERR_ALLOC) and stores the configuration.
 * *out is set only on JD_OK. Not thread-safe per handle; distinct handles are independent. */
jd_status_t jd_create(jd_handle_t* out, const jd_config_t* cfg);

/* Frees the workspace. Synchronises the device first. NULL is accepted. */
jd_status_t jd_destroy(jd_handle_t h);

/* Registers the LM head W [V, d] and the judge head (w_judge [d], bias b_judge); device
 * pointers in the handle's dtype, 16-byte aligned, borrowed until replaced or jd_destroy.
 * The judge head is the paper's linear map R^d -> R (Sec. 4.1 "Model design and training",
 * App. B.1). Builds the TMA descriptors of W. Must precede jd_verify. */
jd_status_t jd_set_head(jd_handle_t h, const void* W, const void* w_judge, float b_judge);

/* 8-bit head (the paper runs its targets with 8-bit weights: Table 1 caption, App. B.3). Handles
 * created with JD_DTYPE_FP8_E4M3 register W8 [V, d] (uint8 E4M3 codes, 16-byte aligned) and w_scale [V]
 * (float32): the logical weight is w_scale[v] * e4m3(W8[v,k]). Every call then quantises the rows
 * of H the same way on the device, s_r = max_k |H[r,k]| / 448 and h8 = e4m3(H[r,k] * 448 / max_k |H[r,k]|)
 * rounded to nearest even, and the tensor cores multiply FP8 by FP8 with fp32 accumulation:
 * L[r,v] = w_scale[v] * s_r * sum_k e4m3(W8[v,k]) * h8[r,k]. The judge still reads the bf16 rows.
 * h8 is the E4M3 value nearest to that quotient, ties to the even mantissa (the device computes
 * H * 448 in float32, exactly, and divides with one rounding, which yields the same codes as the
 * exact quotient for bf16 rows). w_judge [d] is bf16. Pointers are borrowed like those of
 * jd_set_head. The fused and the batched tensor-core variants need d % 128 == 0; the CUDA-core
 * variant takes any d. */
jd_status_t jd_set_head_fp8(jd_handle_t h, const void* W8, const float* w_scale, const void* w_judge,
                            float b_judge);

/* One verification call (steps 1-5 above) enqueued on `cuda_stream` (a cudaStream_t, NULL =
 * default stream). Host-side checks return JD_ERR_INVALID_ARG / JD_ERR_UNSUPPORTED before
 * anything is launched. Device-side conditions (clamped tokens, timed-out waits) are recorded
 * in the handle's device status word, read with jd_last_device_status. Calls on one handle
 * must be ordered on the device (same stream or explicit dependencies): they share the
 * workspace. */
jd_status_t jd_verify(jd_handle_t h, const jd_verify_args_t* args, void* cuda_stream);

/* Same call for callers whose per-step data live in HOST memory: `args` holds HOST pointers
 * for H, draft_tokens, draft_logits and for every output (pinned memory recommended; W stays
 * on the device via jd_set_head). Inputs are copied to handle-owned device staging buffers,
 * the verification runs, the outputs are copied back (one copy through a pinned mirror), and the
 * stream is synchronised before returning. The draft logits, most of the bytes, travel on a second
 * stream of the handle while the verification already runs; each variant waits for them where it
 * first reads them (the fused kernel on a device word that the copy's stream sets, with a bounded
 * wait). Pinned host buffers are needed for that overlap; pageable ones work, serially.
 * logits_debug must be NULL. */
jd_status_t jd_verify_host(jd_handle_t h, const jd_verify_args_t* args, void* cuda_stream);

/* Synchronises the stream of the handle's last jd_verify and reads the device status of that call:
 * *out = JD_OK, JD_ERR_TIMEOUT or JD_ERR_BAD_TOKEN. Consecutive calls of the fused variant enqueue
 * no memset between them (the kernel keeps its grid-barrier counters clean and tags its status
 * writes with a launch number, so a clamped token of an earlier call is not reported for a later
 * one). JD_ERR_TIMEOUT is different: a call in which a wait ran out leaves those counters in an
 * unknown state, so every later fused call on the handle gives up at once and reports
 * JD_ERR_TIMEOUT too, until this function has been called; the next jd_verify then starts from a
 * cleared block. */
jd_status_t jd_last_device_status(jd_handle_t h, int* out);

/* Test helper for the failure path: launches a two-CTA kernel whose barrier wait can never be
 * satisfied and gives up after `spin_limit` polls (1 .. 2^20, about 40 ns each). No memory is
 * touched beyond the handle's status word; afterwards jd_last_device_status reports
 * JD_ERR_TIMEOUT and the handle stays usable. Every wait inside the real kernels is bounded the
 * same way (limit 2^22). */
jd_status_t jd_selftest_timeout(jd_handle_t h, uint32_t spin_limit, void* cuda_stream);

/* Test helper for the fail-stop rule described at jd_last_device_status: marks the handle's device
 * status as a fused call that gave up would have left it (nothing waits, nothing runs out, the host
 * side of the handle is not told). A fused jd_verify enqueued afterwards must return at once with
 * device status JD_ERR_TIMEOUT, and the first call after jd_last_device_status has reported it must
 * run normally again. */
jd_status_t jd_selftest_stale_timeout(jd_handle_t h, void* cuda_stream);

/* Variant the last jd_verify on this handle ran (jd_variant_t), 0 before the first call, and
 * the number of kernels it launched. Either pointer may be NULL. */
jd_status_t jd_last_launch_info(jd_handle_t h, int* variant, int* kernel_launches);

/* Measurement aid (the paper has no counterpart): reads the first bytes/16*16 bytes at `data`
 * (device pointer, 16-byte aligned) exactly once with streaming loads and XORs all 32-bit words
 * read into *out (device pointer, one word, which the caller zeroes beforehand). The call's
 * device time over the LM head is the read-only streaming ceiling a verification call that must
 * fetch W once can approach. Asynchronous on the stream; uses the current device. */
jd_status_t jd_stream_read_probe(const void* data, size_t bytes, uint32_t* out, void* cuda_stream);

/* Measurement aid (the paper has no counterpart). A library built with -DJD_PHASE_STAMPS
 * (python -m paper_2501_19309_b200.build --stamps) makes thread 0 of every CTA of the fused kernel
 * record the GPU's global timer at the phase boundaries of the call; this function copies the
 * stamps of the most recent fused launch on the current device to the HOST array `out`:
 * 256 CTAs x 16 slots of nanosecond values (capacity >= 4096 entries), slot meanings as printed by
 * paper_2501_19309_b200/phase_times.py. Synchronise the stream first. The normal library records
 * nothing and returns JD_ERR_UNSUPPORTED. */
jd_status_t jd_debug_phase_stamps(uint64_t* out, int32_t capacity);

/* Test helper: fills out[i] = Philox uniform for (seed, b[i], slot[i], stream[i]), i < n, with
 * the device generator; device pointers. Used to compare the generator bit for bit with an
 * independent host implementation. */
jd_status_t jd_philox_uniforms(uint64_t seed, const int32_t* b, const int32_t* slot,
                               const int32_t* stream, int32_t n, float* out, void* cuda_stream);

/* Test helper for the FP8 head: quantises `rows` bf16 rows of width d (device pointer, 16-byte
 * aligned) exactly as jd_verify does for a JD_DTYPE_FP8_E4M3 handle and writes the E4M3 codes
 * [rows, d] (device pointer, 16-byte aligned) and the per-row scales [rows] (float32). Asynchronous
 * on the stream; uses the current device. */
jd_status_t jd_quantize_rows_e4m3(const void* H, int32_t rows, int32_t d, uint8_t* codes, float* scale,
                                  void* cuda_stream);

/* Test helper (the paper has no counterpart): the handle's workspace regions are separated by guard
 * blocks of a fixed byte pattern that no kernel may touch. Synchronises the device and sets
 * *damaged to the number of guard blocks whose pattern is no longer intact (0 = no kernel wrote
 * past the end of a region). */
jd_status_t jd_check_workspace_guards(jd_handle_t h, int32_t* damaged);

/* Handle-free form of jd_verify for callers that must not allocate device memory when they
 * verify: servers whose own pool already owns the whole device, decode loops that cannot afford
 * the synchronisation an allocation implies, code barred from allocating after start-up.
 * (The paper has no counterpart; this is a deployment convenience of this library.)
 * It runs the fused tensor-core variant only: bf16, d % 64 == 0, B*(M+1) <= 96, and V small
 * enough for that variant; anything else returns JD_ERR_UNSUPPORTED and launches nothing.
 * The kernel's scratch (592,896 bytes) is a fixed array inside the library's device image: every
 * GPU that loads the library holds it until the process exits. No cudaMalloc, cudaFree or other
 * allocating call is made here.
 *   d, V, W, w_judge, b_judge : the head, as for jd_set_head (device pointers, 16-byte aligned)
 *   args                     : as for jd_verify (device pointers); variant must be AUTO or FUSED,
 *                              rule JD_RULE_SAMPLING, norm JD_NORM_NONE, logits_debug NULL
 *   device_status            : optional device pointer to one uint32 that receives the call's
 *                              device status (JD_OK, JD_ERR_TIMEOUT, JD_ERR_BAD_TOKEN); NULL to skip
 * The call uses the CURRENT device. Its first call on a device looks up the array's device
 * address and the SM count and loads every instantiation of the kernel (so that no later call has
 * to load code); make that first call outside any stream capture. First calls from several host
 * threads are serialised by a lock. All calls on a
 * device share the one array, which keeps the previous call's contents (the words that must
 * start at zero are cleared on the stream each time): calls that overlap on the GPU, from any
 * stream or thread, race with each other, so order them. Asynchronous on `cuda_stream`. */
jd_status_t jd_verify_static(int32_t d, int32_t V, const void* W, const void* w_judge, float b_judge,
                             const jd_verify_args_t* args, uint32_t* device_status, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* JD_H_ */
