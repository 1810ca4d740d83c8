// fathom_scan: variable-depth bit-plane key scan (Sec. 3.2 prefix dequantiser, Sec. 3.3).
//
// A t-plane read of channel j dequantises to  a * sum_{p<t} (2 b_p - 1) 2^-(p+1)  with a = 8 s the
// block range, so a score is a signed sum of per-(block, channel, plane) weights
//     w[beta][j][p][h] = q_hj * a_{beta,j} * 2^-(p+1),      score = 2 * sum_{b_p = 1} w  -  sum w.
// A CTA owns one plan (NH query heads sharing the planes that are read) and a tile of TILE_BLOCKS
// 64-token blocks.  The active (channel, plane) rows of the plan are processed in chunks: the
// chunk's plane words for the tile are staged in shared memory with 16-byte loads (every row is one
// contiguous run, Sec. 3.5), the weights 2w and the bias -sum w are computed once per (block, row)
// from the fp16 scales, and then each lane owns tokens l and l + 32 of a block and adds 2w for every
// set bit.  Only planes p < t_j and scales of active channels are touched.
#include "fathom_common.cuh"

namespace {

constexpr int TILE_BLOCKS = 32;          // 2048 tokens per CTA
constexpr int ROW_CHUNK = 32;            // active rows staged per pass
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_WARPS = SCAN_THREADS / 32;
constexpr int BLOCKS_PER_WARP = TILE_BLOCKS / SCAN_WARPS;   // 4

template <int NH>
struct alignas(16) Wvec { float v[NH]; };

template <int NH>
__global__ void __launch_bounds__(SCAN_THREADS)
scan_kernel(const uint64_t* __restrict__ planes, const uint16_t* __restrict__ scales,
            const float* __restrict__ q, const uint8_t* __restrict__ depth, float* __restrict__ scores,
            long long n, long long nb, long long plane_stride, long long scale_stride, long long score_stride,
            int G) {
  __shared__ uint16_t row_ch[FATHOM_D * FATHOM_NPLANES];      // channel of active row r
  __shared__ uint8_t row_pl[FATHOM_D * FATHOM_NPLANES];       // plane of active row r
  __shared__ int s_nrows;
  __shared__ float s_q[NH][FATHOM_D];
  __shared__ alignas(16) uint64_t s_words[ROW_CHUNK][TILE_BLOCKS];
  __shared__ Wvec<NH> s_w[TILE_BLOCKS][ROW_CHUNK];            // 2 w per (block, row), all heads
  __shared__ float s_bias[TILE_BLOCKS][NH];                   // sum of w over all active rows

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int plan = blockIdx.y;
  const int h0 = plan * NH;
  const int kv = h0 / G;
  const long long blk0 = (long long)blockIdx.x * TILE_BLOCKS;
  const int nblk = (int)min((long long)TILE_BLOCKS, nb - blk0);

  // ---- active row list of this plan, ordered by channel then plane (thread 0..127 = channel)
  if (tid < FATHOM_D) {
    const int t = depth[(size_t)plan * FATHOM_D + tid];
    // exclusive prefix of depths over channels via warp scans + a 4-entry carry
    int incl = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    __shared__ int warp_tot[4];
    if (lane == 31) warp_tot[warp] = incl;
    // the four channel warps synchronise through the named barrier below
    asm volatile("bar.sync 1, 128;");
    int base = 0;
    for (int w = 0; w < warp; ++w) base += warp_tot[w];
    const int start = base + incl - t;
    for (int p = 0; p < t; ++p) { row_ch[start + p] = (uint16_t)tid; row_pl[start + p] = (uint8_t)p; }
    if (tid == FATHOM_D - 1) s_nrows = base + incl;
  }
  for (int e = tid; e < NH * FATHOM_D; e += SCAN_THREADS) s_q[e / FATHOM_D][e % FATHOM_D] = q[(size_t)h0 * FATHOM_D + e];
  for (int e = tid; e < TILE_BLOCKS * NH; e += SCAN_THREADS) (&s_bias[0][0])[e] = 0.0f;
  __syncthreads();
  const int nrows = s_nrows;

  float acc[BLOCKS_PER_WARP][2][NH];
#pragma unroll
  for (int b = 0; b < BLOCKS_PER_WARP; ++b)
#pragma unroll
    for (int x = 0; x < 2; ++x)
#pragma unroll
      for (int h = 0; h < NH; ++h) acc[b][x][h] = 0.0f;

  const uint64_t* planes_kv = planes + (size_t)kv * FATHOM_D * FATHOM_NPLANES * (size_t)plane_stride;
  const uint16_t* scales_kv = scales + (size_t)kv * FATHOM_D * (size_t)scale_stride;

  for (int r0 = 0; r0 < nrows; r0 += ROW_CHUNK) {
    const int rc = min(ROW_CHUNK, nrows - r0);
    // ---- stage plane words: 16 threads x 16 B per row
    for (int e = tid; e < rc * (TILE_BLOCKS / 2); e += SCAN_THREADS) {
      const int r = e / (TILE_BLOCKS / 2), c = e % (TILE_BLOCKS / 2);
      uint4 val = make_uint4(0u, 0u, 0u, 0u);
      if (2 * c < nblk) {
        const int j = row_ch[r0 + r], p = row_pl[r0 + r];
        const uint64_t* src = planes_kv + ((size_t)j * FATHOM_NPLANES + p) * (size_t)plane_stride + blk0 + 2 * c;
        val = __ldg(reinterpret_cast<const uint4*>(src));
      }
      *reinterpret_cast<uint4*>(&s_words[r][2 * c]) = val;
    }
    // ---- weights: thread handles block beta = tid / 8 and rows (tid % 8) + 8 i
    {
      const int beta = tid >> 3, sub = tid & 7;
      float part[NH];
#pragma unroll
      for (int h = 0; h < NH; ++h) part[h] = 0.0f;
      if (beta < nblk) {
        for (int r = sub; r < rc; r += 8) {
          const int j = row_ch[r0 + r], p = row_pl[r0 + r];
          const float s = __half2float(__ushort_as_half(__ldg(scales_kv + (size_t)j * scale_stride + blk0 + beta)));
          const float a_p = s * (8.0f / (float)(2 << p));     // a * 2^-(p+1), exact
          Wvec<NH> w2;
#pragma unroll
          for (int h = 0; h < NH; ++h) {
            const float w = s_q[h][j] * a_p;
            part[h] += w;
            w2.v[h] = 2.0f * w;
          }
          s_w[beta][r] = w2;
        }
      }
      // fixed-order reduction of the 8 partial sums of a block (lanes 8k .. 8k+7)
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        float v = part[h];
        v += __shfl_xor_sync(0xffffffffu, v, 1);
        v += __shfl_xor_sync(0xffffffffu, v, 2);
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        if (sub == 0 && beta < nblk) s_bias[beta][h] += v;
      }
    }
    __syncthreads();
    // ---- accumulate: warp w owns blocks w, w + 8, ...; lane owns tokens lane and lane + 32
#pragma unroll
    for (int b = 0; b < BLOCKS_PER_WARP; ++b) {
      const int beta = warp + b * SCAN_WARPS;
      if (beta < nblk) {
        for (int r = 0; r < rc; ++r) {
          const uint64_t word = s_words[r][beta];
          const Wvec<NH> w2 = s_w[beta][r];
          const bool lo = ((uint32_t)word >> lane) & 1u;
          const bool hi = ((uint32_t)(word >> 32) >> lane) & 1u;
#pragma unroll
          for (int h = 0; h < NH; ++h) {
            if (lo) acc[b][0][h] += w2.v[h];
            if (hi) acc[b][1][h] += w2.v[h];
          }
        }
      }
    }
    __syncthreads();
  }

  // ---- epilogue: score = 2 sum_{bit=1} w - sum w
#pragma unroll
  for (int b = 0; b < BLOCKS_PER_WARP; ++b) {
    const int beta = warp + b * SCAN_WARPS;
    if (beta < nblk) {
      const long long tok = (blk0 + beta) * FATHOM_BLOCK + lane;
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        const float bias = s_bias[beta][h];
        float* row = scores + (size_t)(h0 + h) * (size_t)score_stride;
        if (tok < n) row[tok] = acc[b][0][h] - bias;
        if (tok + 32 < n) row[tok + 32] = acc[b][1][h] - bias;
      }
    }
  }
}

template <int NH>
int launch_scan(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                const uint8_t* depth, float* scores, cudaStream_t st) {
  const long long nb = fathom_nblocks(L->n);
  const int plans = L->n_q_heads / NH;
  dim3 grid((unsigned)((nb + TILE_BLOCKS - 1) / TILE_BLOCKS), (unsigned)plans);
  scan_kernel<NH><<<grid, SCAN_THREADS, 0, st>>>(planes, scales, q, depth, scores, L->n, nb, L->plane_stride_words,
                                                 L->scale_stride, L->score_stride, L->n_q_heads / L->n_kv_heads);
  return 0;
}

}  // namespace

extern "C" int fathom_scan(fathom_ctx* ctx, const fathom_layout* L, const uint64_t* planes, const uint16_t* scales,
                           const float* q, const uint8_t* depth, int heads_per_plan, float* scores, void* stream) {
  if (!ctx || !planes || !scales || !q || !depth || !scores) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  const int G = L->n_q_heads / L->n_kv_heads;
  if (heads_per_plan < 1 || G % heads_per_plan != 0) return FATHOM_ERR_INVALID_ARG;
  if (!fathom_aligned16(planes) || !fathom_aligned16(scales) || !fathom_aligned16(scores)) return FATHOM_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  switch (heads_per_plan) {
    case 1: launch_scan<1>(L, planes, scales, q, depth, scores, st); break;
    case 2: launch_scan<2>(L, planes, scales, q, depth, scores, st); break;
    case 4: launch_scan<4>(L, planes, scales, q, depth, scores, st); break;
    case 8: launch_scan<8>(L, planes, scales, q, depth, scores, st); break;
    default: return FATHOM_ERR_UNSUPPORTED;
  }
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
