// fathom_gather_union: union of the winners of the query heads that share a KV head, fetched once
// (Sec. 1: the heads of a group mostly pick the same tokens, so a KV head's distinct rows - at most G k - cross the link
// once; Sec. 4 "Offload harness": the row fetch of a decode step is that union).
//
// Three kernels on the caller's stream, no host round trip:
//   mark    every selected token sets its bit in a per-KV-head bitmap (atomic OR: idempotent, so order-free);
//   rank    one CTA per KV head: popcount prefix over the bitmap words gives every word its rank base, the
//           ascending list of distinct tokens and their number;
//   fetch   one warp per staged row copies the K and the V row (16-byte loads; rows may live in pinned host
//           memory and are then read over the host link exactly once), and every (head, i) learns the position
//           of its token among the staged rows: rank base of its word + popcount of the lower bits.
#include "fathom_common.cuh"

namespace {

constexpr int GU_THREADS = 256;
constexpr int RANK_THREADS = 1024;

__global__ void __launch_bounds__(GU_THREADS)
union_mark_kernel(const int32_t* __restrict__ idx, int k, long long n, int G, long long total, uint32_t* __restrict__ bitmap,
                  long long words) {
  const long long e = (long long)blockIdx.x * GU_THREADS + threadIdx.x;
  if (e >= total) return;
  const int h = (int)(e / k);
  int32_t t = idx[e];
  t = t < 0 ? 0 : ((long long)t >= n ? (int32_t)(n - 1) : t);   // out-of-range indices are clamped like in attention
  atomicOr(&bitmap[(size_t)(h / G) * words + (t >> 5)], 1u << (t & 31));
}

__global__ void __launch_bounds__(RANK_THREADS)
union_rank_kernel(const uint32_t* __restrict__ bitmap, long long words, uint32_t* __restrict__ word_rank,
                  int32_t* __restrict__ ulist, int capacity, int32_t* __restrict__ union_count) {
  __shared__ uint32_t s_warp[33];
  const int kv = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t* bm = bitmap + (size_t)kv * words;
  uint32_t* wr = word_rank + (size_t)kv * words;
  int32_t* ul = ulist + (size_t)kv * capacity;
  uint32_t base = 0;
  for (long long w0 = 0; w0 < words; w0 += RANK_THREADS) {     // rounds of 1024 consecutive words: coalesced
    const long long w = w0 + tid;
    const uint32_t bits = (w < words) ? bm[w] : 0u;
    const uint32_t c = __popc(bits);
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const uint32_t v = s_warp[lane];
      uint32_t vi = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, vi, o);
        if (lane >= o) vi += y;
      }
      s_warp[lane] = vi - v;
      if (lane == 31) s_warp[32] = vi;
    }
    __syncthreads();
    uint32_t pos = base + s_warp[warp] + incl - c;
    if (w < words) wr[w] = pos;
    uint32_t b = bits;
    while (b) {
      const int l = __ffs(b) - 1;
      b &= b - 1;
      if (pos < (uint32_t)capacity) ul[pos] = (int32_t)(w * 32 + l);
      ++pos;
    }
    base += s_warp[32];
    __syncthreads();                                           // s_warp is reused by the next round
  }
  if (tid == 0) union_count[kv] = (int32_t)base;
}

template <typename T>
__global__ void __launch_bounds__(GU_THREADS)
union_fetch_kernel(const T* __restrict__ Krows, const T* __restrict__ Vrows, long long n, const int32_t* __restrict__ ulist,
                   const int32_t* __restrict__ union_count, int capacity, T* __restrict__ K_stage, T* __restrict__ V_stage,
                   const int32_t* __restrict__ idx, int k, int G, int Hq, const uint32_t* __restrict__ bitmap,
                   const uint32_t* __restrict__ word_rank, long long words, int32_t* __restrict__ idx_local) {
  constexpr int ROW_U4 = FATHOM_D * sizeof(T) / 16;           // 16-byte pieces per row: 16 (bf16) or 32 (fp32)
  constexpr int ROWS_PER_WARP_STEP = 32 / ROW_U4 > 0 ? 32 / ROW_U4 : 1;
  const int kv = blockIdx.y, lane = threadIdx.x & 31;
  const int warp_global = blockIdx.x * (GU_THREADS / 32) + (threadIdx.x >> 5);
  const int nwarps = gridDim.x * (GU_THREADS / 32);
  const int count = min(union_count[kv], capacity);
  const T* Kh = Krows + (size_t)kv * (size_t)n * FATHOM_D;
  const T* Vh = Vrows + (size_t)kv * (size_t)n * FATHOM_D;
  T* Ks = K_stage + (size_t)kv * (size_t)capacity * FATHOM_D;
  T* Vs = V_stage + (size_t)kv * (size_t)capacity * FATHOM_D;
  // ---- rows: a warp moves ROWS_PER_WARP_STEP rows of K and of V per step (two rows in bf16, one in fp32)
  for (int r0 = warp_global * ROWS_PER_WARP_STEP; r0 < count; r0 += nwarps * ROWS_PER_WARP_STEP) {
    const int r = r0 + (ROW_U4 < 32 ? lane / ROW_U4 : 0), piece = lane % ROW_U4;
    if (r < count) {
      const size_t src = (size_t)ulist[(size_t)kv * capacity + r] * FATHOM_D;
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(Kh + src) + piece);
      const uint4 b = __ldg(reinterpret_cast<const uint4*>(Vh + src) + piece);
      reinterpret_cast<uint4*>(Ks + (size_t)r * FATHOM_D)[piece] = a;
      reinterpret_cast<uint4*>(Vs + (size_t)r * FATHOM_D)[piece] = b;
    }
  }
  // ---- positions of the G heads' picks among the staged rows
  const uint32_t* bm = bitmap + (size_t)kv * words;
  const uint32_t* wr = word_rank + (size_t)kv * words;
  const long long picks = (long long)G * k;
  for (long long e = (long long)blockIdx.x * GU_THREADS + threadIdx.x; e < picks; e += (long long)gridDim.x * GU_THREADS) {
    const size_t at = (size_t)kv * G * k + e;                  // heads kv*G .. kv*G+G-1 are contiguous in idx
    int32_t t = idx[at];
    t = t < 0 ? 0 : ((long long)t >= n ? (int32_t)(n - 1) : t);
    idx_local[at] = (int32_t)(wr[t >> 5] + __popc(bm[t >> 5] & ((1u << (t & 31)) - 1u)));
  }
  (void)Hq;
}

}  // namespace

size_t fathom_union_scratch_bytes(int Hkv, long long n, int capacity) {
  const size_t words = (size_t)((n + 31) / 32);
  return fathom_round_up(Hkv * words * 4, 256) * 2 + fathom_round_up((size_t)Hkv * capacity * 4, 256);
}

extern "C" int fathom_gather_union(fathom_ctx* ctx, const fathom_layout* L, const int32_t* idx, int k, const void* Krows,
                                   const void* Vrows, int row_dtype, void* K_stage, void* V_stage, int32_t* idx_local,
                                   int32_t* union_count, void* stream) {
  if (!ctx || !idx || !Krows || !Vrows || !K_stage || !V_stage || !idx_local || !union_count) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k < 1 || k > L->n) return FATHOM_ERR_INVALID_ARG;
  if (row_dtype != FATHOM_BF16 && row_dtype != FATHOM_F32) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(Krows) || !fathom_aligned16(Vrows) || !fathom_aligned16(K_stage) || !fathom_aligned16(V_stage))
    return FATHOM_ERR_ALIGNMENT;
  const int Hkv = L->n_kv_heads, Hq = L->n_q_heads, G = Hq / Hkv;
  const long long cap_ll = (long long)G * k;
  if (cap_ll > 0x7fffffffLL) return FATHOM_ERR_UNSUPPORTED;
  const int capacity = (int)cap_ll;
  const long long words = (L->n + 31) / 32;
  if (fathom_union_scratch_bytes(Hkv, L->n, capacity) > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
  char* base = static_cast<char*>(ctx->scratch);
  const size_t bm_bytes = fathom_round_up((size_t)Hkv * words * 4, 256);
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(base);
  uint32_t* word_rank = reinterpret_cast<uint32_t*>(base + bm_bytes);
  int32_t* ulist = reinterpret_cast<int32_t*>(base + 2 * bm_bytes);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(bitmap, 0, bm_bytes, st));
  const long long total = (long long)Hq * k;
  union_mark_kernel<<<(unsigned)((total + GU_THREADS - 1) / GU_THREADS), GU_THREADS, 0, st>>>(idx, k, L->n, G, total, bitmap, words);
  union_rank_kernel<<<Hkv, RANK_THREADS, 0, st>>>(bitmap, words, word_rank, ulist, capacity, union_count);
  // enough warps to keep a slow link busy: 16 CTAs of 8 warps per KV head, each warp 2 x 256-byte rows in flight per step
  dim3 grid((unsigned)max(1, min(64, (capacity + 63) / 64)), (unsigned)Hkv);
  if (row_dtype == FATHOM_BF16)
    union_fetch_kernel<__nv_bfloat16><<<grid, GU_THREADS, 0, st>>>(
        static_cast<const __nv_bfloat16*>(Krows), static_cast<const __nv_bfloat16*>(Vrows), L->n, ulist, union_count, capacity,
        static_cast<__nv_bfloat16*>(K_stage), static_cast<__nv_bfloat16*>(V_stage), idx, k, G, Hq, bitmap, word_rank, words,
        idx_local);
  else
    union_fetch_kernel<float><<<grid, GU_THREADS, 0, st>>>(static_cast<const float*>(Krows), static_cast<const float*>(Vrows),
                                                           L->n, ulist, union_count, capacity, static_cast<float*>(K_stage),
                                                           static_cast<float*>(V_stage), idx, k, G, Hq, bitmap, word_rank,
                                                           words, idx_local);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
