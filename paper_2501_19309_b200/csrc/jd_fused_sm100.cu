// Persistent tensor-core kernel for small row counts (B*(M+1) <= 96): one cooperative launch,
// one CTA per SM, the whole verification step in a single kernel.
//
// Orientation ("swap-AB"): the MMA's M axis (128 TMEM lanes) is the vocabulary, its N axis
// (TMEM columns) the rows of H. D[v, r] = sum_k W[v, k] H[r, k]. Each CTA owns a contiguous
// range of 128-entry vocabulary tiles (at most seven for V = 128256 on 148 SMs) and keeps the
// fp32 logits of ALL of them on chip until the call ends: tile i occupies TMEM columns
// [i*S, i*S + rows), S = rows rounded up to 8; tiles that do not fit in the 512 columns are
// computed first and moved to shared memory. The logits never reach device memory.
//
// Warp roles (192 threads): warps 0-3 statistics / decisions / sampling (one TMEM lane
// quadrant each), warp 4 lane 0 TMA producer, warp 5 lane 0 MMA issuer (warp 5 owns the TMEM
// allocation).
//
// Main loop, K-outer: for every 64-wide slice of d the H slice [N_PAD x 64] is loaded once and
// multiplied with the W slice [128 x 64] of every tile of the group, so W streams from HBM
// exactly once and H is re-read (from L2) once per group, not once per tile. A ring slot holds
// two consecutive k-slices (when d / 64 is even), so that the single producer thread and the
// single MMA thread spend one wait and one commit per eight MMAs: with one slice per slot their
// per-tile work (about 0.36 us per 16 KB of W) was as long as HBM needs for those bytes, and longer
// in a sweep over one tile.
// Where it pays (see run_fused), a CTA whose tiles all fit in TMEM sweeps d twice: first over all
// tiles but the last, then over the last one, that one with W and H of a pair of k-slices under a
// single barrier. The epilogue warps take the row statistics of the early tiles (in sample-only
// mode: their sampling masses) while the last tile still streams, so only one tile's worth is left
// for the time after the stream.
//
// After the main loop the grid meets three times:
//   per-CTA (max, sum exp) of every row, logit of the drafted tokens            -> barrier 1
//   the rows' partials are folded, each CTA taking a share of the rows          -> barrier 2
//   every CTA runs the tests and the prefix rule (identical results), then computes its slice
//   of the sampling mass of each sequence's selected row                        -> barrier 3
//   the CTA whose slice contains T = u * total mass locates the token.
// (Sample-only mode skips the first two meetings and uses the first counter once more after the third: the
// searches for the owning CTAs of its up to 96 sequences are dealt out over the grid and exchanged there.)
// The barriers are counters in global memory, legal because the launch is cooperative (all
// CTAs co-resident); every wait in the kernel is bounded and reports JD_ERR_TIMEOUT.
#include <cooperative_groups.h>

#include "jd_kernels.h"
#include "jd_sm100_ptx.cuh"

namespace jd {

// Measurement aid, compiled in only with -DJD_PHASE_STAMPS (a library of its own, see build.py): thread 0
// of every CTA writes the global timer at the phase boundaries of the epilogue, so that a host tool can
// print where a call's time goes. In the normal build JD_STAMP expands to nothing.
#ifdef JD_PHASE_STAMPS
__device__ unsigned long long g_phase_stamps[kMaxCtas * kPhaseStampSlots];
#define JD_STAMP(n)                                                      \
  do {                                                                   \
    if (tid == 0) {                                                      \
      unsigned long long t_;                                             \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));             \
      g_phase_stamps[cta * kPhaseStampSlots + (n)] = t_;                 \
    }                                                                    \
  } while (0)
#else
#define JD_STAMP(n) do { } while (0)
#endif

namespace {

constexpr int kThreads = 192;
constexpr int kBlockK = 64;                      // bf16 elements per k-slice = one 128-byte swizzle row
constexpr int kBlockK8 = 128;                    // FP8 codes per k-slice (same 128 bytes)
constexpr int kWStageBytes = kVocabTile * 128;   // 16 KB
constexpr int kTmemCols = 512;
constexpr int kMiscBytes = 21504;                // barriers + reduction scratch at the head of smem
constexpr int kMaxStages = 12;
constexpr int kMinHStages = 4;
constexpr int kPreferredHStages = 6;
constexpr int kMaxHStages = 8;


struct FusedParams {
  int num_kb;       // d / 64
  int num_tiles;    // ceil(V / 128)
  int stages;       // W ring depth
  int h_stages;     // H ring depth
  int tmem_tiles;   // tiles resident in TMEM
  int tile_stride;  // TMEM columns between consecutive tiles (>= rows, multiple of 8, <= N_PAD)
  int R;            // rows of the H matrix given to the MMA: B * (M + 1), or B in sample-only mode
  int fp8;          // 1: W and H tiles hold FP8 E4M3 codes (128 per 128-byte row), kind::f8f6f4 MMAs
  int late_tiles;   // > 0: a CTA whose tiles all fit in TMEM finishes all but its last `late_tiles` tiles first
                    // (own sweep over d), so that their row statistics are taken while the rest still streams
  // Host-buffer calls: the draft logits may still be on their way to the device when the kernel
  // starts. Non-null: the word that the copy's stream sets to dl_epoch once they have arrived;
  // the epilogue warps wait for it (bounded) before their first read of the draft logits.
  const unsigned* dl_flag;
  unsigned dl_epoch;
  int plain_status; // 1: the caller clears status word and barrier block before every launch and wants plain codes
                    //    in the word (no call tag)
  uint32_t off_h;   // byte offsets inside dynamic smem (from the 1024-aligned base)
  uint32_t off_ovf;
  uint32_t off_w;
};

// ------------------------------------------------------------------------------ shared scratch
template <int N_PAD>
struct Misc {
  uint64_t full_w[kMaxStages], empty_w[kMaxStages];
  uint64_t full_h[kMaxHStages], empty_h[kMaxHStages];
  uint64_t full2[kMaxStages / 2], empty2[kMaxStages / 2];   // one-tile sweep: a pair of k-slices per barrier
  uint64_t acc_full[2];
  uint64_t drained;
  uint32_t tmem_base;
  int abort_flag;
  int glist_n;              // rows whose drafted token lies in this CTA's vocabulary slice
  unsigned launch_index;    // barrier[kCallCounter] at the start of this launch
  int give_up;              // 1: an earlier launch's timeout has not been cleared by the host yet
  float wmax[4][N_PAD];
  float wsum[4][N_PAD];
  float cta_max[N_PAD];
  float lse[N_PAD];         // log-normaliser of every row
  float qlse[N_PAD];
  int x_row[N_PAD];         // drafted token of row r (rows j < M), -1 otherwise
  float scale[N_PAD];       // factor applied to TMEM column r: RMS normalisation and, for an FP8 head, the row's scale
  float swt[8][kVocabTile]; // FP8 head: scale of this thread's vocabulary entry in each of the CTA's tiles (else 1)
  int glist[N_PAD];
  // per sequence (B <= N_PAD / 2 in the full mode, B <= N_PAD in sample-only mode)
  int sel_row[N_PAD];
  int sel_kind[N_PAD];
  float sel_lse_p[N_PAD];
  float sel_lse_q[N_PAD];
  float sel_u[N_PAD];
  double wd_r[N_PAD][4];
  double wd_p[N_PAD][4];
  int own_cta[N_PAD];
  int own_usep[N_PAD];
  double own_prefix[N_PAD];
  double own_T[N_PAD];
  double tsum[4][8];
  double wscan[4];
  int cand[4];
  int lastpos[4];
};

// logits of rows c0..c0+15 for this thread's lane in tiles i0 and i0+1 (zeros past T): from TMEM,
// or from the overflow copy in shared memory
template <int N_PAD>
__device__ __forceinline__ void load_chunk2(int i0, int T, int c0, int n_ovf, int ts, uint32_t tmem_lane_base,
                                            const float* ovf, int tid, const float* sc, const float* swt, float* v0, float* v1) {
  uint32_t a[16], b[16];
#pragma unroll
  for (int k = 0; k < 16; ++k) { a[k] = 0u; b[k] = 0u; }
  if (i0 < n_ovf) {
#pragma unroll
    for (int k = 0; k < 16; ++k) a[k] = __float_as_uint(ovf[((size_t)i0 * N_PAD + c0 + k) * kVocabTile + tid]);
  } else {
    tmem_ld16_issue(tmem_lane_base + (uint32_t)((i0 - n_ovf) * ts + c0), a);
  }
  if (i0 + 1 < T) {
    if (i0 + 1 < n_ovf) {
#pragma unroll
      for (int k = 0; k < 16; ++k) b[k] = __float_as_uint(ovf[((size_t)(i0 + 1) * N_PAD + c0 + k) * kVocabTile + tid]);
    } else {
      tmem_ld16_issue(tmem_lane_base + (uint32_t)((i0 + 1 - n_ovf) * ts + c0), b);
    }
  }
  tmem_wait_ld32(a, b);
  const float w0 = swt[min(i0, 7) * kVocabTile + tid], w1 = swt[min(i0 + 1, 7) * kVocabTile + tid];
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const float f = sc[c0 + k];   // factor of the row (shared memory)
    v0[k] = __uint_as_float(a[k]) * (f * w0);
    v1[k] = __uint_as_float(b[k]) * (f * w1);
  }
}
// logits of row r in tiles i0 .. i0+7 (those below T) for this thread's lane, fetched together
template <int N_PAD>
__device__ __forceinline__ void load_cols8(int i0, int T, int r, int n_ovf, int ts, uint32_t tmem_lane_base,
                                           const float* ovf, int tid, float f, const float* swt, float* out) {
  uint32_t raw[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int i = i0 + u;
    raw[u] = 0u;
    if (i < T) {
      if (i < n_ovf) raw[u] = __float_as_uint(ovf[((size_t)i * N_PAD + r) * kVocabTile + tid]);
      else tmem_ld1_issue(tmem_lane_base + (uint32_t)((i - n_ovf) * ts + r), raw[u]);
    }
  }
  tmem_wait_ld8(raw);
#pragma unroll
  for (int u = 0; u < 8; ++u) out[u] = __uint_as_float(raw[u]) * (f * swt[min(i0 + u, 7) * kVocabTile + tid]);
}

// Test-only: copies the logits of this CTA's vocabulary slice to out[row, v] exactly as the
// statistics passes read them (normalisation factors and FP8 scales applied). Called by the four
// epilogue warps together; kept out of line so that the kernel's register allocation ignores it.
template <int N_PAD>
__device__ __noinline__ void dump_logits(float* __restrict__ out, int T, int t0, int R, int V, int n_ovf, int ts,
                                         uint32_t tmem_lane_base, const float* ovf, int tid, const float* sc,
                                         const float* swt) {
  for (int i0 = 0; i0 < T; i0 += 2) {
    const int vg0 = (t0 + i0) * kVocabTile + tid, vg1 = vg0 + kVocabTile;
    const bool val0 = vg0 < V, val1 = (i0 + 1 < T) && vg1 < V;
    for (int c0 = 0; c0 < N_PAD; c0 += 16) {
      float v0[16], v1[16];
      load_chunk2<N_PAD>(i0, T, c0, n_ovf, ts, tmem_lane_base, ovf, tid, sc, swt, v0, v1);
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const int r = c0 + k;
        if (r < R && val0) out[(size_t)r * V + vg0] = v0[k];
        if (r < R && val1) out[(size_t)r * V + vg1] = v1[k];
      }
    }
  }
}

// kFp8 is a template parameter, not a runtime flag: a kernel whose MMA loop can reach both
// tcgen05.mma kinds ran its bf16 main loop 40 % slower.
// kKind selects what the epilogue contains, so that each instantiation carries only its own code:
//   kFullSampling  the whole verification step with the stochastic test of Eq. 4 and the token draw
//   kFullTopK      the whole step with the deterministic top-K / greedy rule (rank counts, argmax)
//   kSampleOnly    H holds one already selected row per sequence; only the token draw runs
enum : int { kFullSampling = 0, kFullTopK = 1, kSampleOnlyKind = 2 };

template <int N_PAD, bool kFp8, int kKind>
__global__ void __launch_bounds__(kThreads, 1)
fused_verify_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmH, CallParams cp,
                    Workspace ws, const __nv_bfloat16* __restrict__ H, const __nv_bfloat16* __restrict__ wj,
                    const float* __restrict__ w_scale, FusedParams fp) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Misc<N_PAD>& ms = *reinterpret_cast<Misc<N_PAD>*>(smem);
  static_assert(sizeof(Misc<N_PAD>) <= kMiscBytes, "misc block too large");
  const uint32_t sH = smem_u32(smem + fp.off_h);
  const uint32_t sW = smem_u32(smem + fp.off_w);
  const float* ovf = reinterpret_cast<const float*>(smem + fp.off_ovf);
  float* ovf_w = reinterpret_cast<float*>(smem + fp.off_ovf);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, G = gridDim.x;
  volatile int* abort_flag = &ms.abort_flag;
  constexpr bool kSampleOnly = (kKind == kSampleOnlyKind);
  constexpr bool kTopK = (kKind == kFullTopK);

  // vocabulary tiles of this CTA
  const int base = fp.num_tiles / G, rem = fp.num_tiles % G;
  const int T = base + (cta < rem ? 1 : 0);
  const int t0 = cta * base + min(cta, rem);
  const int n_ovf = max(0, T - fp.tmem_tiles);   // first n_ovf tiles go through TMEM into smem
  const int R = fp.R, M = cp.M, V = cp.V;
  const int BM = cp.B * M;
  // device-side problems go to the status word, tagged with this launch's number unless the caller
  // clears the word before every launch (the counter does not move while a launch can still report)
  auto report = [&](unsigned code) {
    if (fp.plain_status) set_status(ws.status, code);
    else set_status_tagged(ws.status, load_volatile_u32(ws.barrier + kCallCounter) + 1u, code);
  };

  // The producer warp sets up the barriers and leaves the prologue without waiting for the other
  // warps (it arrives at the block's hand-over barrier, they wait on it), so that W starts to
  // stream while they still fetch the drafted tokens and allocate tensor memory.
  if (warp == 4 && lane == 0) {
    for (int s = 0; s < fp.stages; ++s) { mbar_init(smem_u32(&ms.full_w[s]), 1); mbar_init(smem_u32(&ms.empty_w[s]), 1); }
    for (int s = 0; s < fp.h_stages; ++s) { mbar_init(smem_u32(&ms.full_h[s]), 1); mbar_init(smem_u32(&ms.empty_h[s]), 1); }
    for (int s = 0; s < kMaxStages / 2; ++s) { mbar_init(smem_u32(&ms.full2[s]), 1); mbar_init(smem_u32(&ms.empty2[s]), 1); }
    mbar_init(smem_u32(&ms.acc_full[0]), 1);
    mbar_init(smem_u32(&ms.acc_full[1]), 1);
    mbar_init(smem_u32(&ms.drained), 1);
    ms.abort_flag = 0;
    ms.glist_n = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid == 0) {
    const unsigned c = fp.plain_status ? 0u : load_volatile_u32(ws.barrier + kCallCounter);
    ms.launch_index = c;
    ms.give_up = (!fp.plain_status && load_volatile_u32(ws.status) == (((c + 1u) << 8) | (unsigned)JD_ERR_TIMEOUT)) ? 1 : 0;
  }
  if (tid < N_PAD) {
    int x = -1;
    if (tid < R && !kSampleOnly) {
      const int b = tid / (M + 1), j = tid % (M + 1);
      if (j < M) {
        x = cp.draft_tokens[b * M + j];
        if (x < 0 || x >= V) { report(JD_ERR_BAD_TOKEN); x = min(max(x, 0), V - 1); }
      }
    }
    ms.x_row[tid] = x;
    float f = 1.f;   // normalisation factor of the row held in TMEM column tid
    if (cp.norm == JD_NORM_RMS && tid < R) f = ws.row_scale[kSampleOnly ? ws.sel_row[tid] : tid];
    if (fp.fp8 && tid < R) f *= ws.h_scale[kSampleOnly ? ws.sel_row[tid] : tid];
    ms.scale[tid] = f;
  }
  if (tid < kVocabTile) {   // per-vocabulary-row scales of an FP8 head, one per tile of this CTA; 1 otherwise
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int vg = (t0 + u) * kVocabTile + tid;
      ms.swt[u][tid] = (fp.fp8 && u < T && vg < V) ? __ldg(w_scale + vg) : 1.f;
    }
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ms.tmem_base)),
                 "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  if (warp == 4) {
    __syncwarp();
    asm volatile("bar.arrive 2, 192;" ::: "memory");
  } else {
    asm volatile("bar.sync 2, 192;" ::: "memory");
  }
  tc_fence_after();
  const uint32_t tmem_base = ms.tmem_base;   // (not meaningful in the producer warp, which does not use it)
#ifdef JD_PHASE_STAMPS
  if (tid == 0) g_phase_stamps[cta * kPhaseStampSlots + 13] = g_phase_stamps[cta * kPhaseStampSlots + 11];   // previous launch's end
#endif
  JD_STAMP(0);
  if (tid < R) {   // rows whose drafted token this CTA's slice holds (usually none or one)
    const int x = ms.x_row[tid];
    if (x >= t0 * kVocabTile && x < (t0 + T) * kVocabTile) ms.glist[atomicAdd(&ms.glist_n, 1)] = tid;
  }

  // Two sweeps over d. With overflow: group 0 = the n_ovf overflow tiles, group 1 = the
  // TMEM-resident tiles, which reuse the columns the overflow tiles have left. Without overflow
  // and with late_tiles set: group 0 = the first T_early tiles, group 1 = the rest, every tile in
  // columns of its own; the statistics of group 0 are taken while group 1 streams.
  const int T_early = (n_ovf == 0 && fp.late_tiles > 0 && T > fp.late_tiles + 1) ? T - fp.late_tiles : 0;
  const int g_split = n_ovf > 0 ? n_ovf : T_early;
  const int g_begin[2] = {0, g_split};
  const int g_end[2] = {g_split, T};
  const uint32_t g_col[2] = {0u, (uint32_t)(T_early * fp.tile_stride)};   // first TMEM column of each group
  // A sweep over a single tile is bound by what the MMA thread does per k-step (two waits, four MMAs, two
  // commits: about 0.5 us for 16 KB of W), not by HBM. The one-tile late sweep therefore moves two k-slices
  // of W and of H per barrier: ring slots 2s and 2s + 1 form a pair with barriers of its own, so that one
  // wait and one commit serve eight MMAs. The pairs take over the slots once the first sweep has finished
  // with all of them.
  const int pairs = min(fp.stages, fp.h_stages) / 2;
  const bool paired_late = T_early > 0 && T - T_early == 1 && (fp.num_kb & 1) == 0 && pairs >= 1;
  // The other sweeps, too, move two k-slices per ring slot whenever d allows it (kk = 2): one wait and one
  // commit then serve eight MMAs of a tile instead of four, which keeps the producer and MMA threads'
  // per-tile work safely below the time HBM needs for the tile's bytes.
  // (not with rings too short for two slots each: 81 to 96 rows at the full vocabulary leave three W slices)
  const int kk = ((fp.num_kb & 1) == 0 && fp.stages >= 4 && fp.h_stages >= 4) ? 2 : 1;
  const int w_slots = fp.stages / kk, h_slots = fp.h_stages / kk;   // ring depths in slots of kk slices

  if (warp == 4 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    const uint64_t pol_w = policy_evict_first(), pol_h = policy_evict_last();
    const int kelems = fp.fp8 ? kBlockK8 : kBlockK;   // elements per 128-byte k-slice
    int ws_i = 0, hs_i = 0;
    uint32_t wph = 0, hph = 0;
    bool ok = true;
    for (int g = 0; g < 2 && ok; ++g) {
      if (g_begin[g] == g_end[g]) continue;
      if (g == 1 && paired_late) {
        // every MMA of the first sweep has completed: all ring slots are free for the pairs
        ok = mbar_wait(smem_u32(&ms.acc_full[0]), 0u, abort_flag);
        int s2 = 0;
        uint32_t ph2 = 0;
        const int row0 = (t0 + g_begin[1]) * kVocabTile;
        for (int kb = 0; kb < fp.num_kb && ok; kb += 2) {
          ok = mbar_wait(smem_u32(&ms.empty2[s2]), ph2 ^ 1u, abort_flag);
          if (!ok) break;
          const uint32_t fb = smem_u32(&ms.full2[s2]);
          mbar_expect_tx(fb, 2 * (kWStageBytes + N_PAD * 128));
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            tma_load_2d(sH + (2 * s2 + j) * (N_PAD * 128), &tmH, fb, (kb + j) * kelems, 0, pol_h);
            tma_load_2d(sW + (2 * s2 + j) * kWStageBytes, &tmW, fb, (kb + j) * kelems, row0, pol_w);
          }
          if (++s2 == pairs) { s2 = 0; ph2 ^= 1u; }
        }
        continue;
      }
      for (int kb = 0; kb < fp.num_kb && ok; kb += kk) {
        ok = mbar_wait(smem_u32(&ms.empty_h[hs_i]), hph ^ 1u, abort_flag);
        if (!ok) break;
        mbar_expect_tx(smem_u32(&ms.full_h[hs_i]), kk * N_PAD * 128);
        for (int j = 0; j < kk; ++j)
          tma_load_2d(sH + (hs_i * kk + j) * (N_PAD * 128), &tmH, smem_u32(&ms.full_h[hs_i]), (kb + j) * kelems, 0, pol_h);
        if (++hs_i == h_slots) { hs_i = 0; hph ^= 1u; }
        for (int i = g_begin[g]; i < g_end[g]; ++i) {
          ok = mbar_wait(smem_u32(&ms.empty_w[ws_i]), wph ^ 1u, abort_flag);
          if (!ok) break;
          mbar_expect_tx(smem_u32(&ms.full_w[ws_i]), kk * kWStageBytes);
          for (int j = 0; j < kk; ++j)
            tma_load_2d(sW + (ws_i * kk + j) * kWStageBytes, &tmW, smem_u32(&ms.full_w[ws_i]), (kb + j) * kelems,
                        (t0 + i) * kVocabTile, pol_w);
          if (++ws_i == w_slots) { ws_i = 0; wph ^= 1u; }
        }
      }
    }
    if (!ok) report(JD_ERR_TIMEOUT);
  } else if (warp == 5 && lane == 0) {
    // ------------------------------------------------------------------ MMA issuer
    const uint32_t idesc = kFp8 ? make_idesc_e4m3(N_PAD) : make_idesc(N_PAD);
    int ws_i = 0, hs_i = 0;
    uint32_t wph = 0, hph = 0;
    bool ok = true;
    for (int g = 0; g < 2 && ok; ++g) {
      if (g_begin[g] == g_end[g]) continue;
      if (g == 1 && n_ovf > 0) {   // the overflow tiles must have left TMEM before it is reused
        ok = mbar_wait(smem_u32(&ms.drained), 0u, abort_flag);
        if (!ok) break;
        tc_fence_after();
      }
      if (g == 1 && paired_late) {
        int s2 = 0;
        uint32_t ph2 = 0;
        const uint32_t dcol = tmem_base + g_col[1];
        for (int kb = 0; kb < fp.num_kb && ok; kb += 2) {
          ok = mbar_wait(smem_u32(&ms.full2[s2]), ph2, abort_flag);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint32_t wb = sW + (2 * s2 + j) * kWStageBytes, hb = sH + (2 * s2 + j) * (N_PAD * 128);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const uint64_t da = make_smem_desc(wb + k * 32), db = make_smem_desc(hb + k * 32);
              const uint32_t acc = (kb > 0 || j > 0 || k > 0) ? 1u : 0u;
              if constexpr (kFp8) umma_e4m3(dcol, da, db, idesc, acc);
              else umma_bf16(dcol, da, db, idesc, acc);
            }
          }
          umma_commit(smem_u32(&ms.empty2[s2]));
          if (++s2 == pairs) { s2 = 0; ph2 ^= 1u; }
        }
        if (ok) umma_commit(smem_u32(&ms.acc_full[1]));
        continue;
      }
      for (int kb = 0; kb < fp.num_kb && ok; kb += kk) {
        ok = mbar_wait(smem_u32(&ms.full_h[hs_i]), hph, abort_flag);
        if (!ok) break;
        for (int i = g_begin[g]; i < g_end[g]; ++i) {
          ok = mbar_wait(smem_u32(&ms.full_w[ws_i]), wph, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t dcol = tmem_base + g_col[g] + (uint32_t)((i - g_begin[g]) * fp.tile_stride);
          for (int j = 0; j < kk; ++j) {
            const uint32_t wb = sW + (ws_i * kk + j) * kWStageBytes, hb = sH + (hs_i * kk + j) * (N_PAD * 128);
#pragma unroll
            for (int k = 0; k < 4; ++k) {   // four MMAs of 32 bytes of K each: 16 bf16 or 32 FP8 codes
              const uint64_t da = make_smem_desc(wb + k * 32), db = make_smem_desc(hb + k * 32);
              const uint32_t acc = (kb > 0 || j > 0 || k > 0) ? 1u : 0u;
              if constexpr (kFp8) umma_e4m3(dcol, da, db, idesc, acc);
              else umma_bf16(dcol, da, db, idesc, acc);
            }
          }
          umma_commit(smem_u32(&ms.empty_w[ws_i]));
          if (++ws_i == w_slots) { ws_i = 0; wph ^= 1u; }
        }
        if (!ok) break;
        umma_commit(smem_u32(&ms.empty_h[hs_i]));
        if (++hs_i == h_slots) { hs_i = 0; hph ^= 1u; }
      }
      if (ok) umma_commit(smem_u32(&ms.acc_full[g]));
    }
    if (!ok) report(JD_ERR_TIMEOUT);
  } else if (warp < 4) {
    // ------------------------------------------------------------------ epilogue warps
    const uint32_t tmem_lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
    const int ts = fp.tile_stride;
    unsigned* const bar = ws.barrier + (ms.launch_index & 1u) * 3u;   // this launch's set of barrier counters
    bool ok = true;
    if (ms.give_up) {   // an uncleared timeout of an earlier launch: every role leaves through the failure path
      ok = false;
      if (tid == 0) *abort_flag = 1;
    }

    // (a) overflow tiles: TMEM -> smem as soon as their accumulation is complete
    if (n_ovf > 0) {
      // one thread polls the barrier; the other 127 sleep in the hardware barrier below
      if (tid == 0) mbar_wait(smem_u32(&ms.acc_full[0]), 0u, abort_flag);
      epi_sync();
      ok = (*abort_flag == 0);
      if (ok) {
        tc_fence_after();
        for (int i = 0; i < n_ovf; ++i) {
#pragma unroll
          for (int c0 = 0; c0 < N_PAD; c0 += 16) {
            float v[16];
            tmem_ld16(tmem_lane_base + (uint32_t)(i * ts + c0), v);
#pragma unroll
            for (int k = 0; k < 16; ++k) ovf_w[((size_t)i * N_PAD + c0 + k) * kVocabTile + tid] = v[k];
          }
        }
        tc_fence_before();
      }
      epi_sync();
      if (tid == 0) mbar_arrive(smem_u32(&ms.drained));
    }

    // (b)-(e) draft statistics and judge dots, then the row statistics in one or two phases. Phase 1
    // covers the tiles of the last sweep and starts when the whole accumulation is complete. A CTA that ran an early sweep (T_early > 0)
    // first takes, in phase 0, the statistics of the early tiles while the last sweep still streams,
    // and merges the two (max, sum exp) pairs per row at the end.
    if constexpr (kSampleOnly) {
      // an earlier kernel made the decisions; fetch what the token draw needs
      if (tid < cp.B) {
        ms.sel_row[tid] = ws.sel_row[tid];
        ms.sel_kind[tid] = ws.sel_kind[tid];
        ms.sel_lse_p[tid] = ws.sel_lse_p[tid];
        ms.sel_lse_q[tid] = ws.sel_lse_q[tid];
        ms.sel_u[tid] = ws.sel_u[tid];
      }
      epi_sync();
    }
    // Order of the steps: (b), then phase 0 (if there is an early sweep), then phase 1. A call whose draft
    // logits are still on their way from the host runs phase 0 first, so that the copy has the early
    // sweep's time to land before anything waits for it.
    const bool defer_b = fp.dl_flag != nullptr && T_early > 0;
    for (int step = 0; step < 3; ++step) {
      const int ph = defer_b ? (step == 0 ? 0 : (step == 1 ? -1 : 1)) : step - 1;
      if (ph < 0) {
      // (b) while W streams: draft-row statistics over this CTA's vocabulary slice, judge dots
      if (fp.dl_flag != nullptr) {   // draft logits still in flight: wait for the copy stream's signal
        if (tid == 0) {
          bool arrived = false;
          for (unsigned it = 0; it < kSpinLimit / 4 && !arrived; ++it) {
            unsigned v;
            asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(fp.dl_flag) : "memory");
            arrived = (v == fp.dl_epoch);
            if (!arrived) {
              if (*abort_flag) break;
              __nanosleep(100);
            }
          }
          if (!arrived) {
            *abort_flag = 1;
            report(JD_ERR_TIMEOUT);
          }
        }
        epi_sync();
      }
      const int v_lo = t0 * kVocabTile, v_hi = min(V, (t0 + T) * kVocabTile);
      const bool vec4 = cp.dl_vec4 != 0;   // rows start on 16-byte boundaries only then
      for (int bm = warp; bm < (kSampleOnly ? 0 : BM); bm += 4) {
        const float* row = cp.draft_logits + (size_t)bm * V;
        float m = -INFINITY, s = 0.f;
        if (vec4) {
          // eight 128-entry tiles per pass: all loads of the pass are issued before any arithmetic
          for (int i0 = 0; i0 < T; i0 += 8) {
            float4 x[8];
  #pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int v = v_lo + (i0 + u) * kVocabTile + lane * 4;
              x[u] = (i0 + u < T && v < V) ? __ldcg(reinterpret_cast<const float4*>(row + v))
                                           : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            }
            float mm = -INFINITY;
  #pragma unroll
            for (int u = 0; u < 8; ++u) mm = fmaxf(mm, fmaxf(fmaxf(x[u].x, x[u].y), fmaxf(x[u].z, x[u].w)));
            const float mn = fmaxf(m, mm);
            if (mn == -INFINITY) continue;
            float acc = 0.f;
            const float off = mn * kLog2e;
  #pragma unroll
            for (int u = 0; u < 8; ++u) {
              acc += exp2f(fmaf(x[u].x, kLog2e, -off)) + exp2f(fmaf(x[u].y, kLog2e, -off));
              acc += exp2f(fmaf(x[u].z, kLog2e, -off)) + exp2f(fmaf(x[u].w, kLog2e, -off));
            }
            s = s * __expf(m - mn) + acc;
            m = mn;
          }
        } else {
          for (int v = v_lo + lane; v < v_hi; v += 32) {
            const float xv = __ldcg(row + v);
            if (xv > m) { s = s * __expf(m - xv) + 1.f; m = xv; }
            else if (xv != -INFINITY) s += __expf(xv - m);
          }
        }
        ms_warp_reduce(m, s);
        if (lane == 0) {
          ws.qpart_max[(size_t)bm * G + cta] = m;
          ws.qpart_sum[(size_t)bm * G + cta] = s;
          const int b = bm / M, j = bm % M;
          const int x = ms.x_row[b * (M + 1) + j];
          if (x >= v_lo && x < v_hi) ws.qgath[bm] = __ldcg(row + x);
        }
      }
      for (int bm = cta * 4 + warp; bm < (kSampleOnly ? 0 : BM); bm += G * 4) {
        const int b = bm / M, j = bm % M;
        const uint4* h4 = reinterpret_cast<const uint4*>(H + ((size_t)b * (M + 1) + j + 1) * cp.d);
        const uint4* w4 = reinterpret_cast<const uint4*>(wj);
        float acc = 0.f;
        for (int k = lane; k < cp.d / 8; k += 32) {
          const uint4 hv = __ldg(h4 + k), wv = __ldg(w4 + k);
          const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hv);
          const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&wv);
  #pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 a = __bfloat1622float2(hp[e]), c = __bfloat1622float2(wp[e]);
            acc = fmaf(a.x, c.x, acc);
            acc = fmaf(a.y, c.y, acc);
          }
        }
  #pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) ws.judge_logit[bm] = acc;
      }

        JD_STAMP(1);
        continue;
      }
      if (ph == 0 && T_early == 0) continue;
      if (tid == 0 && ok && (ph == 0 || T > n_ovf)) mbar_wait(smem_u32(&ms.acc_full[ph]), 0u, abort_flag);
      epi_sync();
      tc_fence_after();
      ok = ok && (*abort_flag == 0);
      if (ph == 1) JD_STAMP(2); else JD_STAMP(12);
      const int i_lo = ph == 0 ? 0 : T_early, i_hi = ph == 0 ? T_early : T;
      if constexpr (kSampleOnly) {
        // (h) mass of the sampling weights of each selected row over the phase's tiles.
        // Sample-only mode: every TMEM column is a selected row, so the tiles are read 16 columns
        // (= 16 sequences) at a time, like the statistics passes.
        if (ok) {
#pragma unroll
          for (int c0 = 0; c0 < N_PAD; c0 += 16) {
            if (c0 >= cp.B) break;
            // A thread adds at most a handful of tiles per sequence, so its own partial sums stay in
            // fp32 (32 double accumulators would not fit in registers); everything summed across
            // lanes, warps and CTAs is double. The loop body is branch-free: with one warp per
            // scheduler, branches around each sequence would serialise sixteen latency chains.
            float sr[16], sp[16], lp2[16], lq2[16];
            int kd[16];   // 0: residual, 1: p alone, 2: column past the last sequence
#pragma unroll
            for (int k = 0; k < 16; ++k) {
              const int b = min(c0 + k, cp.B - 1);
              sr[k] = 0.f; sp[k] = 0.f;
              kd[k] = (c0 + k < cp.B) ? ms.sel_kind[b] : 2;
              lp2[k] = ms.sel_lse_p[b] * kLog2e;
              lq2[k] = ms.sel_lse_q[b] * kLog2e;
            }
            const int last_tile = fp.num_tiles - 1;
            for (int i0 = i_lo; i0 < i_hi; i0 += 2) {
              const int vg0 = (t0 + i0) * kVocabTile + tid, vg1 = vg0 + kVocabTile;
              const bool val0 = vg0 < V, val1 = (i0 + 1 < i_hi) && vg1 < V;
              // ws.w_sel holds the selected draft rows tile-major, [vocab tile][sequence][128]: this
              // CTA's share is one contiguous block. Rows that need no residual were not gathered;
              // what is read for them is discarded by the select below.
              const float* base0 = ws.w_sel + ((size_t)(t0 + i0) * cp.B + min(c0, cp.B - 1)) * kVocabTile + tid;
              const float* base1 = ws.w_sel + ((size_t)min(t0 + i0 + 1, last_tile) * cp.B + min(c0, cp.B - 1)) * kVocabTile + tid;
              float d0[16], d1[16], v0[16], v1[16];
#pragma unroll
              for (int k = 0; k < 16; ++k) {
                const int ks = min(k, cp.B - 1 - min(c0, cp.B - 1));   // stay inside the buffer in a ragged last chunk
                d0[k] = __ldg(base0 + ks * kVocabTile);
                d1[k] = __ldg(base1 + ks * kVocabTile);
              }
              load_chunk2<N_PAD>(i0, i_hi, c0, n_ovf, ts, tmem_lane_base, ovf, tid, ms.scale, &ms.swt[0][0], v0, v1);
#pragma unroll
              for (int k = 0; k < 16; ++k) {
                const float p0 = fast_exp2(fmaf(v0[k], kLog2e, -lp2[k])), q0 = fast_exp2(fmaf(d0[k], kLog2e, -lq2[k]));
                const float p1 = fast_exp2(fmaf(v1[k], kLog2e, -lp2[k])), q1 = fast_exp2(fmaf(d1[k], kLog2e, -lq2[k]));
                const float r0 = kd[k] == 0 ? fmaxf(0.f, p0 - q0) : p0;
                const float r1 = kd[k] == 0 ? fmaxf(0.f, p1 - q1) : p1;
                const bool on0 = val0 && kd[k] < 2, on1 = val1 && kd[k] < 2;
                sr[k] += (on0 ? r0 : 0.f) + (on1 ? r1 : 0.f);
                sp[k] += (on0 ? p0 : 0.f) + (on1 ? p1 : 0.f);
              }
            }
            double dsum[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) dsum[k] = (double)sr[k];
            const double red_r = warp_reduce16<false, double>(dsum, lane);
#pragma unroll
            for (int k = 0; k < 16; ++k) dsum[k] = (double)sp[k];
            const double red_p = warp_reduce16<false, double>(dsum, lane);
            const int bq = c0 + reduce16_index(lane);
            if ((lane & 1) == 0 && bq < cp.B) {
              if (ph == 1 && T_early > 0) { ms.wd_r[bq][warp] += red_r; ms.wd_p[bq][warp] += red_p; }   // same thread wrote phase 0
              else { ms.wd_r[bq][warp] = red_r; ms.wd_p[bq][warp] = red_p; }
            }
          }
        }
        if (ph == 0) JD_STAMP(14);
        continue;
      }

      // (d) gather of the drafted tokens' logits (rows listed in the prologue), per-row max
      if (ok && ph == 1) {
        const int ng = ms.glist_n;
        for (int e = 0; e < ng; ++e) {
          const int r = ms.glist[e], x = ms.x_row[r];
          const int i = x / kVocabTile - t0;
          float one[8];
          load_cols8<N_PAD>(i, i + 1, r, n_ovf, ts, tmem_lane_base, ovf, tid, ms.scale[r], &ms.swt[0][0], one);
          if (tid == (x % kVocabTile)) ws.gath[r] = one[0];
        }
      }
#pragma unroll
      for (int c0 = 0; c0 < N_PAD; c0 += 16) {
        float mx[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) mx[k] = -INFINITY;
        if (ok) {
          for (int i0 = i_lo; i0 < i_hi; i0 += 2) {
            float v0[16], v1[16];
            load_chunk2<N_PAD>(i0, i_hi, c0, n_ovf, ts, tmem_lane_base, ovf, tid, ms.scale, &ms.swt[0][0], v0, v1);
            const bool val0 = (t0 + i0) * kVocabTile + tid < V;
            const bool val1 = (i0 + 1 < i_hi) && ((t0 + i0 + 1) * kVocabTile + tid < V);
            if (val0) {
#pragma unroll
              for (int k = 0; k < 16; ++k) mx[k] = fmaxf(mx[k], v0[k]);
            }
            if (val1) {
#pragma unroll
              for (int k = 0; k < 16; ++k) mx[k] = fmaxf(mx[k], v1[k]);
            }
          }
        }
        const float red = warp_reduce16<true, float>(mx, lane);
        if ((lane & 1) == 0) ms.wmax[warp][c0 + reduce16_index(lane)] = red;
      }
      epi_sync();
      if (tid < N_PAD) ms.cta_max[tid] = fmaxf(fmaxf(ms.wmax[0][tid], ms.wmax[1][tid]), fmaxf(ms.wmax[2][tid], ms.wmax[3][tid]));
      epi_sync();

      // (e) per-row sum exp(L - max of the phase)
#pragma unroll
      for (int c0 = 0; c0 < N_PAD; c0 += 16) {
        float acc[16], cm[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) { acc[k] = 0.f; cm[k] = ms.cta_max[c0 + k] * kLog2e; }
        if (ok) {
          for (int i0 = i_lo; i0 < i_hi; i0 += 2) {
            float v0[16], v1[16];
            load_chunk2<N_PAD>(i0, i_hi, c0, n_ovf, ts, tmem_lane_base, ovf, tid, ms.scale, &ms.swt[0][0], v0, v1);
            const bool val0 = (t0 + i0) * kVocabTile + tid < V;
            const bool val1 = (i0 + 1 < i_hi) && ((t0 + i0 + 1) * kVocabTile + tid < V);
            if (val0) {
#pragma unroll
              for (int k = 0; k < 16; ++k) acc[k] += fast_exp2(fmaf(v0[k], kLog2e, -cm[k]));
            }
            if (val1) {
#pragma unroll
              for (int k = 0; k < 16; ++k) acc[k] += fast_exp2(fmaf(v1[k], kLog2e, -cm[k]));
            }
          }
        }
        const float red = warp_reduce16<false, float>(acc, lane);
        if ((lane & 1) == 0) ms.wsum[warp][c0 + reduce16_index(lane)] = red;
      }
      epi_sync();
      if (tid < N_PAD) {
        float m = ms.cta_max[tid];
        float sum = (ms.wsum[0][tid] + ms.wsum[1][tid]) + (ms.wsum[2][tid] + ms.wsum[3][tid]);
        if (ph == 0) {
          // parked in the slots of the rows' log-normalisers, which are not written before barrier 2
          ms.lse[tid] = m;
          ms.qlse[tid] = sum;
        } else {
          if (T_early > 0) {
            const float m0 = ms.lse[tid], s0 = ms.qlse[tid];
            const float mm = fmaxf(m, m0);
            if (mm > -INFINITY)
              sum = s0 * fast_exp2((m0 - mm) * kLog2e) + sum * fast_exp2((m - mm) * kLog2e);
            m = mm;
            ms.cta_max[tid] = m;   // the top-K rule compares against the maximum of the whole slice
          }
          if (tid < R) {
            ws.part_max[(size_t)tid * G + cta] = m;
            ws.part_sum[(size_t)tid * G + cta] = sum;
          }
        }
      }
      epi_sync();
      if (ph == 0) JD_STAMP(14);
    }
    JD_STAMP(3);
    if constexpr (!kSampleOnly) {
    if (ok && cp.logits_debug != nullptr)
      dump_logits<N_PAD>(cp.logits_debug, T, t0, R, V, n_ovf, ts, tmem_lane_base, ovf, tid, ms.scale, &ms.swt[0][0]);
    __threadfence();
    epi_sync();

    // ------------------------------------------------------------------ grid barrier 1
    if (tid == 0) {
      if (!ok || !grid_arrive_and_wait(bar + 0, (unsigned)G, abort_flag)) {
        *abort_flag = 1;
        report(JD_ERR_TIMEOUT);
      }
    }
    epi_sync();
    ok = (*abort_flag == 0);
    JD_STAMP(4);

    // (f0) top-K rule: over the parked tiles, count the entries of every draft row that rank above
    // the drafted token (its logit is known grid-wide since barrier 1) and note the lowest token id
    // that attains this CTA's row maximum. Counts go to global counters with integer atomics
    // (order-independent), the argmax candidates beside the per-CTA maxima.
    if (kTopK && ok) {
      int* wcnt = reinterpret_cast<int*>(&ms.wmax[0][0]);   // the float statistics have been written out
      int* widx = reinterpret_cast<int*>(&ms.wsum[0][0]);
#pragma unroll
      for (int c0 = 0; c0 < N_PAD; c0 += 16) {
        float gref[16], cmx[16];
        int xr[16], cnt[16], neg[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int r = c0 + k;
          xr[k] = ms.x_row[r];
          gref[k] = (r < R && xr[k] >= 0) ? __ldcg(ws.gath + r) : INFINITY;   // nothing ranks above +inf
          cmx[k] = ms.cta_max[r];
          cnt[k] = 0;
          neg[k] = -0x7F7F7F7F;
        }
        for (int i0 = 0; i0 < T; i0 += 2) {
          float v0[16], v1[16];
          load_chunk2<N_PAD>(i0, T, c0, n_ovf, ts, tmem_lane_base, ovf, tid, ms.scale, &ms.swt[0][0], v0, v1);
          const int vg0 = (t0 + i0) * kVocabTile + tid, vg1 = vg0 + kVocabTile;
          const bool val0 = vg0 < V, val1 = (i0 + 1 < T) && vg1 < V;
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            if (val0) {
              cnt[k] += (v0[k] > gref[k] || (v0[k] == gref[k] && vg0 < xr[k])) ? 1 : 0;
              if (v0[k] == cmx[k]) neg[k] = max(neg[k], -vg0);
            }
            if (val1) {
              cnt[k] += (v1[k] > gref[k] || (v1[k] == gref[k] && vg1 < xr[k])) ? 1 : 0;
              if (v1[k] == cmx[k]) neg[k] = max(neg[k], -vg1);
            }
          }
        }
        const int red_c = warp_reduce16<false, int>(cnt, lane);
        const int red_i = warp_reduce16<true, int>(neg, lane);
        if ((lane & 1) == 0) {
          wcnt[warp * N_PAD + c0 + reduce16_index(lane)] = red_c;
          widx[warp * N_PAD + c0 + reduce16_index(lane)] = red_i;
        }
      }
      epi_sync();
      if (tid < R) {
        const int c = (wcnt[tid] + wcnt[N_PAD + tid]) + (wcnt[2 * N_PAD + tid] + wcnt[3 * N_PAD + tid]);
        const int i = max(max(widx[tid], widx[N_PAD + tid]), max(widx[2 * N_PAD + tid], widx[3 * N_PAD + tid]));
        if (c > 0 && ms.x_row[tid] >= 0) atomicAdd(ws.cnt + tid, c);
        ws.part_idx[(size_t)tid * G + cta] = -i;
      }
    }

    // (f) fold the per-CTA statistics: the R target rows and the B*M draft rows are dealt out
    // over the grid, one per warp, so that no CTA reads more than a few rows' worth of partials
    if (ok) {
      for (int it = cta + G * warp; it < R + BM; it += 4 * G) {
        const bool is_p = it < R;
        const float* pm = is_p ? ws.part_max + (size_t)it * G : ws.qpart_max + (size_t)(it - R) * G;
        const float* ps = is_p ? ws.part_sum + (size_t)it * G : ws.qpart_sum + (size_t)(it - R) * G;
        float vm[8], vs[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int c = lane + 32 * u;
          vm[u] = c < G ? __ldcg(pm + c) : -INFINITY;
          vs[u] = c < G ? __ldcg(ps + c) : 0.f;
        }
        float m = vm[0];
#pragma unroll
        for (int u = 1; u < 8; ++u) m = fmaxf(m, vm[u]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float sacc = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (vs[u] > 0.f) sacc += vs[u] * fast_exp2((vm[u] - m) * kLog2e);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, o);
        if (lane == 0) {
          const float lse = m + logf(sacc);
          if (is_p) {
            ws.row_lse[it] = lse;
            if (cp.row_max_out) cp.row_max_out[it] = m;
            if (cp.row_lse_out) cp.row_lse_out[it] = lse;
          } else {
            ws.q_lse[it - R] = lse;
          }
        }
      }
    }
    JD_STAMP(5);
    __threadfence();
    epi_sync();

    // ------------------------------------------------------------------ grid barrier 2
    if (tid == 0) {
      if (!ok || !grid_arrive_and_wait(bar + 1, (unsigned)G, abort_flag)) {
        *abort_flag = 1;
        report(JD_ERR_TIMEOUT);
      }
    }
    epi_sync();
    ok = (*abort_flag == 0);
    JD_STAMP(6);
    if (ok) {
      if (tid < R) ms.lse[tid] = __ldcg(ws.row_lse + tid);
      if (tid < BM) ms.qlse[tid] = __ldcg(ws.q_lse + tid);
    }
    epi_sync();
    if (ok) {
      // (g) tests, mask, accepted prefix (Eq. 4; Sec. 4.1): one warp per sequence, identical in
      // every CTA; CTA 0 writes the outputs
      Workspace lw = ws;
      lw.row_lse = ms.lse;
      lw.q_lse = ms.qlse;
      lw.sel_row = ms.sel_row;
      lw.sel_kind = ms.sel_kind;
      lw.sel_lse_p = ms.sel_lse_p;
      lw.sel_lse_q = ms.sel_lse_q;
      lw.sel_u = ms.sel_u;
      lw.argidx = nullptr;   // top-K rule: the next token is folded below, not read from global
      for (int b = warp; b < cp.B; b += 4) decide_sequence(cp, lw, b, cta == 0);
    }
    epi_sync();

    }

    JD_STAMP(7);
    // top-K rule: the next token is the argmax of the selected row; CTA 0 folds the per-CTA maxima
    // and their candidates (larger value first, then lower token id). Nothing is drawn.
    constexpr bool draw = !kTopK;
    if (ok && !draw && cta == 0) {
      for (int b = warp; b < cp.B; b += 4) {
        const int row = ms.sel_row[b];
        float bm = -INFINITY;
        int bi = 0x7F7F7F7F;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int c = lane + 32 * u;
          if (c < G) {
            const float m = __ldcg(ws.part_max + (size_t)row * G + c);
            const int i = __ldcg(ws.part_idx + (size_t)row * G + c);
            if (m > bm || (m == bm && i < bi)) { bm = m; bi = i; }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float m = __shfl_xor_sync(0xffffffffu, bm, o);
          const int i = __shfl_xor_sync(0xffffffffu, bi, o);
          if (m > bm || (m == bm && i < bi)) { bm = m; bi = i; }
        }
        if (lane == 0) cp.next_token[b] = bi;
      }
    }

    // (h) mass of the sampling weights of each selected row over this CTA's slice (sample-only mode:
    // done above, phase by phase, as the tiles completed).
    // Full mode: the few selected rows sit in scattered columns; four sequences at a time so
    // that their draft-logit loads are in flight together.
    if (ok && draw && !kSampleOnly) {
      for (int b0 = 0; b0 < cp.B; b0 += 4) {
        double sr[4] = {0.0, 0.0, 0.0, 0.0}, sp[4] = {0.0, 0.0, 0.0, 0.0};
        for (int i0 = 0; i0 < T; i0 += 8) {
          float dv[4][8], lg[4][8];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (b0 + q >= cp.B) continue;   // uniform over the CTA: no work for sequences that do not exist
            const int b = b0 + q;
            const int row = ms.sel_row[b], kind = ms.sel_kind[b];
            const float* dlrow = cp.draft_logits + ((size_t)b * M + (row % (M + 1))) * V;   // read only when kind == 0
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int vg = (t0 + i0 + u) * kVocabTile + tid;
              dv[q][u] = (kind == 0 && b0 + q < cp.B && i0 + u < T && vg < V) ? __ldcg(dlrow + vg) : 0.f;
            }
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (b0 + q >= cp.B) continue;   // uniform over the CTA: no work for sequences that do not exist
            const int b = b0 + q;
            const int col = kSampleOnly ? b : ms.sel_row[b];   // TMEM column of this sequence's selected row
            load_cols8<N_PAD>(i0, T, col, n_ovf, ts, tmem_lane_base, ovf, tid, ms.scale[col], &ms.swt[0][0], lg[q]);
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (b0 + q >= cp.B) continue;   // uniform over the CTA: no work for sequences that do not exist
            const int b = b0 + q;
            const int kind = ms.sel_kind[b];
            const float lse_p = ms.sel_lse_p[b], lse_q = ms.sel_lse_q[b];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int vg = (t0 + i0 + u) * kVocabTile + tid;
              if (i0 + u < T && vg < V) {
                float p, r;
                sample_weights(lg[q][u], lse_p, kind, dv[q][u], lse_q, p, r);
                sr[q] += (double)r;
                sp[q] += (double)p;
              }
            }
          }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const double a_r = warp_sum_double(sr[q]), a_p = warp_sum_double(sp[q]);
          if (lane == 0 && b0 + q < cp.B) { ms.wd_r[b0 + q][warp] = a_r; ms.wd_p[b0 + q][warp] = a_p; }
        }
      }
    }
    epi_sync();
    if (ok && draw && tid < cp.B) {
      ws.mass_r[(size_t)tid * G + cta] = (ms.wd_r[tid][0] + ms.wd_r[tid][1]) + (ms.wd_r[tid][2] + ms.wd_r[tid][3]);
      ws.mass_p[(size_t)tid * G + cta] = (ms.wd_p[tid][0] + ms.wd_p[tid][1]) + (ms.wd_p[tid][2] + ms.wd_p[tid][3]);
    }
    JD_STAMP(8);
    __threadfence();
    epi_sync();

    // ------------------------------------------------------------------ grid barrier 3
    if (tid == 0 && draw) {
      if (!ok || !grid_arrive_and_wait(bar + 2, (unsigned)G, abort_flag)) {
        *abort_flag = 1;
        report(JD_ERR_TIMEOUT);
      }
    }
    epi_sync();
    ok = (*abort_flag == 0);
    JD_STAMP(9);

    // (i) inverse CDF in ascending token id. First, one warp per sequence finds the CTA whose
    // slice contains T = u * total (same arithmetic in every CTA, so every CTA agrees) ...
    if (ok && draw) {
      const int per = (G + 31) / 32;   // lane l owns CTAs [l*per, (l+1)*per), per <= 8
      // Sample-only mode (up to 96 sequences): the searches are dealt out over the grid, one per warp, and
      // their results exchanged through global memory behind one more grid barrier; otherwise every CTA
      // searches for every sequence itself.
      const int b_first = kSampleOnly ? cta + G * warp : warp;
      const int b_step = kSampleOnly ? 4 * G : 4;
      double nx[8];                    // the next sequence's masses, fetched while this one is searched
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int c = lane * per + u;
        nx[u] = (b_first < cp.B && u < per && c < G) ? __ldcg(ws.mass_r + (size_t)b_first * G + c) : 0.0;
      }
      for (int b = b_first; b < cp.B; b += b_step) {
        const double* mass = ws.mass_r + (size_t)b * G;
        double mc[8];
        double chunk = 0.0;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int c = lane * per + u;
          mc[u] = nx[u];
          chunk += mc[u];
          if (b + b_step < cp.B) nx[u] = (u < per && c < G) ? __ldcg(mass + (size_t)b_step * G + c) : 0.0;
        }
        double total = warp_sum_double(chunk);
        int use_p = 0;
        if (!(total > 0.0)) {   // identically zero residual: draw from p
          use_p = 1;
          mass = ws.mass_p + (size_t)b * G;
          chunk = 0.0;
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int c = lane * per + u;
            mc[u] = (u < per && c < G) ? __ldcg(mass + c) : 0.0;
            chunk += mc[u];
          }
        }
        // exclusive prefix of the lane chunks (fixed-order warp scan, the same in every CTA)
        double incl = chunk;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += up;
        }
        const double excl = incl - chunk;
        total = __shfl_sync(0xffffffffu, incl, 31);
        const double Tt = (double)ms.sel_u[b] * total;
        int owner = -1, last_mass = -1;
        double my_prefix = 0.0;
        {
          double c = excl;
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int cc = lane * per + u;
            if (u < per && cc < G) {
              if (mc[u] > 0.0) last_mass = cc;
              if (owner < 0 && c + mc[u] > Tt) { owner = cc; my_prefix = c; }
              c += mc[u];
            }
          }
        }
        const unsigned found = __ballot_sync(0xffffffffu, owner >= 0);
        double owner_prefix;
        if (found) {
          const int src = __ffs(found) - 1;
          owner = __shfl_sync(0xffffffffu, owner, src);
          owner_prefix = __shfl_sync(0xffffffffu, my_prefix, src);
        } else {   // T at or beyond the total after rounding: the last CTA that carries mass
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) last_mass = max(last_mass, __shfl_xor_sync(0xffffffffu, last_mass, o));
          owner = last_mass;
          owner_prefix = -1.0;
        }
        if (lane == 0) {
          if constexpr (kSampleOnly) {
            ws.own_i[2 * b] = owner;
            ws.own_i[2 * b + 1] = use_p;
            ws.own_d[2 * b] = owner_prefix;
            ws.own_d[2 * b + 1] = Tt;
          } else {
            ms.own_cta[b] = owner;
            ms.own_prefix[b] = owner_prefix;
            ms.own_T[b] = Tt;
            ms.own_usep[b] = use_p;
          }
        }
      }
    }
    if constexpr (kSampleOnly) {
      // exchange of the search results: the counter of barrier 1, which this mode does not use otherwise
      __threadfence();
      epi_sync();
      if (tid == 0) {
        if (!ok || !grid_arrive_and_wait(bar + 0, (unsigned)G, abort_flag)) {
          *abort_flag = 1;
          report(JD_ERR_TIMEOUT);
        }
      }
      epi_sync();
      ok = (*abort_flag == 0);
      if (ok) {
        for (int b = tid; b < cp.B; b += 128) {
          ms.own_cta[b] = __ldcg(ws.own_i + 2 * b);
          ms.own_usep[b] = __ldcg(ws.own_i + 2 * b + 1);
          ms.own_prefix[b] = __ldcg(ws.own_d + 2 * b);
          ms.own_T[b] = __ldcg(ws.own_d + 2 * b + 1);
        }
      }
    }
    epi_sync();
    JD_STAMP(10);
    // ... then the owning CTA finds the tile from the tile masses and the token inside that tile
    if (ok && draw) {
      for (int b = 0; b < cp.B; ++b) {
        if (ms.own_cta[b] != cta) continue;
        const int row = ms.sel_row[b];
        const int col = kSampleOnly ? b : row;
        const int kind = ms.own_usep[b] ? 1 : ms.sel_kind[b];
        const float lse_p = ms.sel_lse_p[b], lse_q = ms.sel_lse_q[b];
        const float* dlrow = cp.draft_logits + ((size_t)b * M + (row % (M + 1))) * V;
        const double Tt = ms.own_T[b];
        const bool beyond = ms.own_prefix[b] < 0.0;
        double c_run = beyond ? 0.0 : ms.own_prefix[b];
        int token = -1, last_token = -1;
        for (int i0 = 0; i0 < T && token < 0; i0 += 8) {
          float dv[8], lg[8], rw[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int vg = (t0 + i0 + u) * kVocabTile + tid;
            const float* src = kSampleOnly ? ws.w_sel + ((size_t)(t0 + i0 + u) * cp.B + b) * kVocabTile + tid
                                              : dlrow + vg;
            dv[u] = (kind == 0 && i0 + u < T && vg < V) ? __ldcg(src) : 0.f;
          }
          load_cols8<N_PAD>(i0, T, col, n_ovf, ts, tmem_lane_base, ovf, tid, ms.scale[col], &ms.swt[0][0], lg);
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int vg = (t0 + i0 + u) * kVocabTile + tid;
            float p = 0.f, r = 0.f;
            if (i0 + u < T && vg < V) sample_weights(lg[u], lse_p, kind, dv[u], lse_q, p, r);
            rw[u] = r;
            const double su = warp_sum_double((double)r);
            if (lane == 0) ms.tsum[warp][u] = su;
          }
          epi_sync();
          // the tile that contains T, else the last tile of this pass that carries mass
          int ustar = -1, ulast = -1;
          double c_before = c_run;
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const double tt = (ms.tsum[0][u] + ms.tsum[1][u]) + (ms.tsum[2][u] + ms.tsum[3][u]);
            if (tt > 0.0) ulast = u;
            if (ustar < 0) {
              if (!beyond && c_run + tt > Tt) { ustar = u; c_before = c_run; }
              c_run += tt;
            }
          }
          const int usel = ustar >= 0 ? ustar : ulast;
          if (usel >= 0) {
            float r = 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) if (u == usel) r = rw[u];
            double incl = (double)r;   // ordered inclusive scan over the 128 lanes of the tile
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
              const double up = __shfl_up_sync(0xffffffffu, incl, o);
              if (lane >= o) incl += up;
            }
            if (lane == 31) ms.wscan[warp] = incl;
            const unsigned pos = __ballot_sync(0xffffffffu, r > 0.f);
            if (lane == 0) ms.lastpos[warp] = pos ? (31 - __clz(pos)) : -1;
            epi_sync();
            double off = c_before;
            for (int w = 0; w < warp; ++w) off += ms.wscan[w];
            const unsigned hit = (ustar >= 0) ? __ballot_sync(0xffffffffu, off + incl > Tt) : 0u;
            if (lane == 0) ms.cand[warp] = hit ? (__ffs(hit) - 1) : -1;
            epi_sync();
            const int tile_v0 = (t0 + i0 + usel) * kVocabTile;
            for (int w = 0; w < 4; ++w) {
              if (token < 0 && ms.cand[w] >= 0) token = tile_v0 + w * 32 + ms.cand[w];
              if (ms.lastpos[w] >= 0) last_token = tile_v0 + w * 32 + ms.lastpos[w];
            }
            // summation-order rounding can leave the tile without a hit: its last token with mass
            if (ustar >= 0 && token < 0) token = last_token;
          }
          epi_sync();
        }
        if (token < 0) token = last_token;   // T beyond the total: the last token that carries mass
        if (tid == 0) cp.next_token[b] = token < 0 ? 0 : token;
      }
    }
    JD_STAMP(11);
    // Every barrier of this launch lies behind CTA 0 now and nothing can report any more: clear the set
    // the previous launch used and publish this launch as done (the next one then takes that set).
    if (!fp.plain_status && cta == 0 && tid == 0 && ok) {
      unsigned* other = ws.barrier + ((ms.launch_index & 1u) ^ 1u) * 3u;
      other[0] = 0u; other[1] = 0u; other[2] = 0u;
      __threadfence();
      *reinterpret_cast<volatile unsigned*>(ws.barrier + kCallCounter) = ms.launch_index + 1u;
    }
    tc_fence_before();
  }

  // ------------------------------------------------------------------ teardown
  __syncthreads();
  if (ms.abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
    __syncthreads();
  }
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols)
                 : "memory");
  }
}

template <int N_PAD, bool kFp8, int kKind>
cudaError_t launch_fused(const CUtensorMap& tmW, const CUtensorMap& tmH, const CallParams& cp, const Workspace& ws,
                         const void* H, const void* wj, const float* w_scale, const FusedParams& fp,
                         const FusedPlan& plan, cudaStream_t st) {
  auto kern = fused_verify_kernel<N_PAD, kFp8, kKind>;   // its shared-memory limit was raised by fused_configure()
  const __nv_bfloat16* Hp = (const __nv_bfloat16*)H;
  const __nv_bfloat16* wp = (const __nv_bfloat16*)wj;
  void* args[] = {(void*)&tmW, (void*)&tmH, (void*)&cp, (void*)&ws, (void*)&Hp, (void*)&wp, (void*)&w_scale, (void*)&fp};
  return cudaLaunchCooperativeKernel((const void*)kern, dim3(plan.num_ctas), dim3(kThreads), args, plan.smem_bytes,
                                     st);
}

// Self-test of the bounded wait: two CTAs arrive at a barrier that expects three, so the wait can
// only end by running out of its (short) limit; each records JD_ERR_TIMEOUT and returns.
__global__ void timeout_probe_kernel(Workspace ws, unsigned limit) {
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    if (!grid_arrive_and_wait(ws.barrier + 7, gridDim.x + 1, &abort_flag, limit)) set_status(ws.status, JD_ERR_TIMEOUT);
  }
}

}  // namespace

bool read_phase_stamps(unsigned long long* host_out) {
#ifdef JD_PHASE_STAMPS
  return cudaMemcpyFromSymbol(host_out, g_phase_stamps, sizeof(unsigned long long) * kMaxCtas * kPhaseStampSlots) == cudaSuccess;
#else
  (void)host_out;
  return false;
#endif
}

void launch_timeout_probe(const Workspace& ws, unsigned limit, cudaStream_t st) {
  timeout_probe_kernel<<<2, 32, 0, st>>>(ws, limit);
}

namespace {
template <int N_PAD, bool kFp8>
bool configure_kinds() {
  return cudaFuncSetAttribute(fused_verify_kernel<N_PAD, kFp8, kFullSampling>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem) == cudaSuccess &&
         cudaFuncSetAttribute(fused_verify_kernel<N_PAD, kFp8, kFullTopK>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem) == cudaSuccess &&
         cudaFuncSetAttribute(fused_verify_kernel<N_PAD, kFp8, kSampleOnlyKind>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem) == cudaSuccess;
}
template <int N_PAD>
bool configure_pair() { return configure_kinds<N_PAD, false>() && configure_kinds<N_PAD, true>(); }

template <int N_PAD>
cudaError_t launch_n(bool fp8, int kind, const CUtensorMap& tmW, const CUtensorMap& tmH, const CallParams& cp,
                     const Workspace& ws, const void* H, const void* wj, const float* w_scale, const FusedParams& fp,
                     const FusedPlan& plan, cudaStream_t st) {
#define JD_LAUNCH(FP8, KIND) launch_fused<N_PAD, FP8, KIND>(tmW, tmH, cp, ws, H, wj, w_scale, fp, plan, st)
  if (fp8) return kind == kSampleOnlyKind ? JD_LAUNCH(true, kSampleOnlyKind)
                                          : (kind == kFullTopK ? JD_LAUNCH(true, kFullTopK) : JD_LAUNCH(true, kFullSampling));
  return kind == kSampleOnlyKind ? JD_LAUNCH(false, kSampleOnlyKind)
                                 : (kind == kFullTopK ? JD_LAUNCH(false, kFullTopK) : JD_LAUNCH(false, kFullSampling));
#undef JD_LAUNCH
}
}  // namespace

bool fused_configure() {
  return configure_pair<16>() && configure_pair<32>() && configure_pair<48>() && configure_pair<64>() &&
         configure_pair<80>() && configure_pair<96>();
}

bool fused_supported(int dtype, int R, int d, int V, int num_sms, FusedPlan* plan) {
  const bool fp8 = dtype == JD_DTYPE_FP8_E4M3;
  if (dtype != JD_DTYPE_BF16 && !fp8) return false;
  const int kelems = fp8 ? kBlockK8 : kBlockK;
  if (d % kelems != 0 || d < kelems || R < 1 || R > 96) return false;
  if (num_sms < 1 || num_sms > kMaxCtas) return false;
  const int n_pad = (R + 15) / 16 * 16;
  const int num_tiles = (V + kVocabTile - 1) / kVocabTile;
  const int max_tiles = (num_tiles + num_sms - 1) / num_sms;
  // Tiles sit `stride` TMEM columns apart, stride = rows rounded up to 8. When stride < n_pad the
  // last n_pad - stride columns an MMA writes fall on the next tile's first columns; they belong
  // to zero-padded rows of H, so after that tile's own first (overwriting) MMA, which is issued
  // later in the same k-step, every further write there adds exactly zero.
  const int stride = (R + 7) / 8 * 8;
  const int tmem_tiles = std::min(max_tiles, (kTmemCols - n_pad) / stride + 1);
  const int n_ovf = max_tiles - tmem_tiles;
  if (n_ovf > tmem_tiles) return false;   // the overflow group itself must fit in TMEM
  if (fp8 && max_tiles > 8) return false;  // the per-tile vocabulary scales are kept for eight tiles
  const size_t base_fixed = 1024 /*alignment slack*/ + kMiscBytes + (size_t)n_ovf * kVocabTile * n_pad * 4;
  const size_t h_stage = (size_t)n_pad * 128;
  const size_t budget = kMaxDynamicSmem;
  if (base_fixed + kMinHStages * h_stage + 3 * (size_t)kWStageBytes > budget) return false;   // at least a three-deep W ring
  // Ring slots hold two k-slices, and the one-tile late sweep runs on min(W, H) / 2 pairs of them, so an H ring
  // of four slices means two slots and two pairs in flight: measured 2-3 % slower per call than six or more
  // (cfg1, cfg2, cfg3). Six H slices are set aside first wherever that still leaves a W ring of six.
  int h_min = kPreferredHStages;
  if (base_fixed + h_min * h_stage + 6 * (size_t)kWStageBytes > budget) h_min = kMinHStages;
  int stages = (int)((budget - base_fixed - h_min * h_stage) / kWStageBytes);
  stages = std::min(stages, kMaxStages);
  // the H ring then takes whatever the W ring leaves over
  int h_stages = (int)((budget - base_fixed - (size_t)stages * kWStageBytes) / h_stage);
  h_stages = std::max(h_min, std::min(h_stages, kMaxHStages));
  const size_t fixed = base_fixed + h_stages * h_stage;
  if (plan) {
    plan->num_ctas = num_sms;
    plan->n_pad = n_pad;
    plan->max_tiles = max_tiles;
    plan->tmem_tiles = tmem_tiles;
    plan->tile_stride = stride;
    plan->stages = stages;
    plan->h_stages = h_stages;
    plan->smem_bytes = fixed + (size_t)stages * kWStageBytes;
  }
  return true;
}

int run_fused(const CallParams& cp, const Workspace& ws, const CUtensorMap& tmW, const CUtensorMap& tmH,
              const void* H, const void* w_judge, const FusedPlan& plan, cudaStream_t st, cudaError_t* err,
              bool sample_only, const float* w_scale_fp8, const unsigned* dl_flag, unsigned dl_epoch,
              bool plain_status) {
  FusedParams fp;
  fp.plain_status = plain_status ? 1 : 0;
  fp.dl_flag = sample_only ? nullptr : dl_flag;
  fp.dl_epoch = dl_epoch;
  fp.fp8 = w_scale_fp8 ? 1 : 0;
  fp.num_kb = cp.d / (fp.fp8 ? kBlockK8 : kBlockK);
  fp.num_tiles = (cp.V + kVocabTile - 1) / kVocabTile;
  fp.stages = plan.stages;
  fp.h_stages = plan.h_stages;
  fp.tmem_tiles = plan.tmem_tiles;
  fp.tile_stride = plan.tile_stride;
  fp.R = sample_only ? cp.B : cp.B * (cp.M + 1);
  // Early sweep + one late tile: the statistics of all tiles but the last (in sample-only mode: their sampling
  // masses) are taken while the last tile streams. With the late sweep moving two k-slices per barrier it costs
  // the stream nothing measurable, and per call it gains 3.5 % at 16 padded rows (d = 4096), about as much as
  // before at 80 (cfg2) and is even with a single sweep at 32 rows and d = 16384 (cfg3): on wherever the sweep
  // over d is long enough to hide something (32 k-steps) or the statistics passes are long (48 padded rows).
  fp.late_tiles = (sample_only || plan.n_pad >= 48 || fp.num_kb >= 32) ? 1 : 0;
  // Sample-only mode with an FP8 head and many sequences: one tile of codes streams in half the time the
  // masses of the early tiles take, so two tiles are left for the late sweep.
  if (sample_only && w_scale_fp8 != nullptr && plan.n_pad >= 48) fp.late_tiles = 2;
  fp.off_h = kMiscBytes;
  fp.off_ovf = fp.off_h + plan.h_stages * plan.n_pad * 128;
  const int n_ovf = plan.max_tiles - plan.tmem_tiles;
  fp.off_w = fp.off_ovf + (uint32_t)n_ovf * kVocabTile * plan.n_pad * 4;
  fp.off_w = (fp.off_w + 1023u) & ~1023u;
  const int kind = sample_only ? kSampleOnlyKind : (cp.rule == JD_RULE_TOPK ? kFullTopK : kFullSampling);
  const bool f8 = fp.fp8 != 0;
  cudaError_t e;
  switch (plan.n_pad) {
    case 16: e = launch_n<16>(f8, kind, tmW, tmH, cp, ws, H, w_judge, w_scale_fp8, fp, plan, st); break;
    case 32: e = launch_n<32>(f8, kind, tmW, tmH, cp, ws, H, w_judge, w_scale_fp8, fp, plan, st); break;
    case 48: e = launch_n<48>(f8, kind, tmW, tmH, cp, ws, H, w_judge, w_scale_fp8, fp, plan, st); break;
    case 64: e = launch_n<64>(f8, kind, tmW, tmH, cp, ws, H, w_judge, w_scale_fp8, fp, plan, st); break;
    case 80: e = launch_n<80>(f8, kind, tmW, tmH, cp, ws, H, w_judge, w_scale_fp8, fp, plan, st); break;
    case 96: e = launch_n<96>(f8, kind, tmW, tmH, cp, ws, H, w_judge, w_scale_fp8, fp, plan, st); break;
    default: e = cudaErrorInvalidValue; break;
  }
  *err = e;
  return e == cudaSuccess ? 1 : -1;
}

}  // namespace jd
