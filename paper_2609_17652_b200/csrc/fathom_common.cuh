// Internal definitions shared by the translation units of libfathom (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stdio.h>

#include "fathom.h"

#define FATHOM_D 128            // channels per head (Sec. 1: Qwen3-8B head size)
#define FATHOM_BLOCK 64         // tokens per scale block (Sec. 3.2)
#define FATHOM_NPLANES 4        // bits per code (Sec. 3.2)
#define FATHOM_CTL_BYTES 8192   // device control block of a context (zeroed once at creation)
#define FATHOM_CTL_TICKETS 64   // first ticket counter (word index); counters re-arm themselves
#define FATHOM_CTL_MAX_HEADS ((FATHOM_CTL_BYTES / 4) - FATHOM_CTL_TICKETS)

struct fathom_ctx {
  int device;
  void* scratch;               // device arena, 256-byte aligned
  size_t scratch_bytes;
  uint32_t* dev_status;        // device control block: word 0 = status word, words FATHOM_CTL_TICKETS.. = ticket counters
  cudaError_t last_cuda;
};

static inline int fathom_cuda_fail(fathom_ctx* ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda = e;
  return FATHOM_ERR_CUDA;
}

#define FATHOM_CUDA_TRY(ctx, expr)                              \
  do {                                                          \
    cudaError_t e__ = (expr);                                   \
    if (e__ != cudaSuccess) return fathom_cuda_fail((ctx), e__);\
  } while (0)

// Checks every host-visible property of a layout.  Returns FATHOM_OK or the error.
int fathom_check_layout(const fathom_layout* L);

static inline int64_t fathom_nblocks(int64_t n) { return (n + FATHOM_BLOCK - 1) / FATHOM_BLOCK; }
static inline bool fathom_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t fathom_round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- programmatic dependent launch (sm_90+): a kernel launched with fathom_launch_dependent may become resident while
// the previous kernel of the stream still runs (once every CTA of that kernel has passed FATHOM_PDL_RELEASE or exited) and
// must execute FATHOM_PDL_WAIT before it touches anything the previous kernels wrote; the wait returns when they have
// completed and their writes are visible.  Both are no-ops in a normally launched kernel, and a kernel that never
// releases simply serialises.  Every kernel of the decode step waits at its top, so completion is transitive.
#define FATHOM_PDL_WAIT() asm volatile("griddepcontrol.wait;" ::: "memory")
#define FATHOM_PDL_RELEASE() asm volatile("griddepcontrol.launch_dependents;" ::: "memory")
template <typename... P, typename... A>
static inline cudaError_t fathom_launch_dependent(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

// ---- pieces shared by scan.cu and topk.cu for the fused scan + selection (fathom_scan_topk) -------------------
// A launch that belongs to one of two alternative continuations decides on the device whether it runs.  A first
// attempt collects, per head, the tokens above an ESTIMATED threshold; it goes on only if every head collected at
// least `want` of them.  Otherwise the second attempt, enqueued behind it with a threshold that is a guaranteed
// bound, does the work.  The host enqueues both and never synchronises.
struct fathom_gate {
  const uint32_t* counts;       // [heads] candidates the first attempt collected per head
  uint32_t want;
  int heads;
  int mode;                     // 0: always run; 1: only if every head collected enough; 2: only if some head did not;
                                // 5: always run - the kernel itself looks at its head's count and picks its input
};
// Called by every thread of the CTA at the top of a gated kernel.
__device__ __forceinline__ bool fathom_gate_open(const fathom_gate& g) {
  if (g.mode == 0 || g.mode == 5) return true;
  bool ok = true;
  for (int h = threadIdx.x; h < g.heads; h += blockDim.x) ok = ok && (__ldcg(g.counts + h) >= g.want);
  const bool all_ok = __syncthreads_and(ok) != 0;
  return g.mode == 1 ? all_ok : !all_ok;
}

struct fathom_scan_fuse {       // extra arguments of the sampling / filtering scan variants
  int tile_step;                // sample: scan every tile_step-th tile
  const uint32_t* state;        // filter: [Hq][8] (pointer already offset to the word to read): a threshold bin, or,
  int state_is_score;           //         if state_is_score, the fp32 bits of the score a candidate must reach
  fathom_gate gate;             // filter: whether this launch runs at all
  long long sink_end, local_begin;   // filter: eligible tokens are sink_end <= i < local_begin
  float* cand_score;            // filter: [Hq][capacity] scores of the candidates
  int32_t* cand_idx;            // filter: [Hq][capacity] their tokens
  uint32_t* cand_count;         // filter: [Hq]
  long long capacity;
};
int fathom_scan_tile_tokens();  // tokens per scan tile (the sampling granularity)
int fathom_fused_tile_step(long long n, int k);   // 16, or 1 when the sequence is too short to sample
int fathom_launch_scan_sample(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                              const uint8_t* depth, int heads_per_plan, float* sample, long long sample_stride,
                              int tile_step, cudaStream_t st);
int fathom_launch_scan_filter(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                              const uint8_t* depth, int heads_per_plan, const fathom_scan_fuse& fz, cudaStream_t st);

// ---- scratch arena carving (one place, used by fathom_scratch_bytes and by the calls) --------
#define FATHOM_TOPK_BINS 4096            // 12 leading bits of the ordered score key
#define FATHOM_ATTN_CHUNK 128            // selected rows handled by one CTA of the partial kernel

struct fathom_topk_scratch {
  uint32_t* hist;        // [Hq][FATHOM_TOPK_BINS]
  uint32_t* state;       // [Hq][8]: 0 threshold bin, 1 count above it, 2 needed from it, 3 bound bin (sampled paths),
                         //          4 candidates written, 5 tickets
  uint32_t* cand_count;  // [Hq] candidates collected above an estimated threshold (single-pass top-k, fused path)
  uint32_t* cand_count2; // [Hq] candidates of the second attempt (threshold that is a bound, not an estimate)
  uint32_t* bitmap;      // [Hq][bitmap_words] selection bitmap, token i at bit (i % 32) of word i / 32
  int32_t* cand;         // [Hq][n] token indices of the threshold bin
  uint32_t* tile_count;  // [Hq][ceil(n / 8192)] selected tokens per filter tile, then their exclusive prefix
  float* cand_score;     // [Hq][n] scores of the fused path's candidates
  float* sample;         // [Hq][sample_stride] scores of the sampled scan tiles (fused path)
  long long sample_stride;
  long long bitmap_words;
  size_t bytes;
};
struct fathom_attn_scratch {
  float* partial;        // [Hq][splits][d + 2]: running max, denominator, weighted V sum
  int splits;
  size_t bytes;
};
fathom_topk_scratch fathom_carve_topk(void* base, int Hq, int64_t n, int k);
fathom_attn_scratch fathom_carve_attn(void* base, int Hq, int k);
size_t fathom_union_scratch_bytes(int Hkv, long long n, int capacity);
size_t fathom_rotate_tc_scratch_bytes(int Hkv);                            // split, transposed basis of the tensor-core rotation
int fathom_launch_rotate_tc(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, const float* mean,
                            const float* basis, float* K_rot, void* scratch, cudaStream_t st);
int fathom_launch_rotate_build_tc(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, const float* mean,
                                  const float* basis, uint64_t* planes, uint16_t* scales, void* scratch, cudaStream_t st);
int fathom_cov_tc_ctas_per_head(int Hkv);                                  // CTAs (= partials) per head of the tensor-core covariance
int fathom_launch_cov_tc(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, float* shift, float* partial,
                         float* partial_sum, int ctas_per_head, cudaStream_t st);
size_t fathom_calib_scratch_bytes(int Hkv, long long n);                  // partial means and covariances   // bitmap + word ranks + union list
