// fathom_rotate_keys on the 5th-generation tensor cores: K' = (K - mu) V  (Sec. 3.5 "Basis rule").
//
// The rotation is the one dense contraction next to the decode path (n x 128 by 128 x 128 per KV head), so it runs
// as tcgen05.mma with the accumulator in tensor memory.  The rotated keys feed a quantiser, so tf32's 11 significant
// bits are not enough; both operands are split into a tf32 head and a tf32 tail, x = xh + xl, v = vh + vl, and three
// products are accumulated in fp32:  xh vh + xh vl + xl vh  (the dropped xl vl term is below 2^-22 of |x||v|).
//
// One persistent CTA per SM walks a contiguous range of 128-token tiles.  Per tile and per chunk of 32 channels
// (128 bytes of tf32: one row of the 128-byte swizzle) all 256 threads take the chunk from registers (loaded one
// tile ahead), subtract the mean, split, and store head and tail into shared memory in the K-major 128-byte-swizzled
// layout the MMA descriptors describe; one thread then issues the 4 x 3 MMAs of the chunk (M = 128 tokens, N = 128
// rotated channels, K = 8) and commits them to the mbarrier that frees the chunk buffer (two buffers).  The split
// basis (transposed, K-major) stays in shared memory for the whole tile range.  After the fourth chunk the 128 x 128
// fp32 accumulator is read back with tcgen05.ld (warp w: lanes 32 (w mod 4).., columns 64 (w div 4)..), staged per
// warp in shared memory and written to global memory in 128-byte rows.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets FATHOM_DEV_WAIT_EXPIRED in the context status and
// the CTA stops waiting, finishes its loops, frees its tensor memory and returns.
#include "fathom_common.cuh"

namespace {

constexpr int TC_THREADS = 256;
constexpr int TILE_M = 128;                                  // tokens per tile (MMA M)
constexpr int KC = 32;                                       // channels per chunk = 128 bytes of tf32
constexpr int NCHUNK = FATHOM_D / KC;                        // 4
constexpr int SLAB = TILE_M * KC * 4;                        // 16 KB: 128 rows of 128 bytes
constexpr int UMMA_K = 8;                                    // tf32 elements per MMA along K (32 bytes)
constexpr uint32_t TMEM_COLS = 128;                          // fp32 accumulator columns
constexpr uint32_t WAIT_TRIES = 1u << 22;

// shared-memory map (bytes from a 1024-byte aligned base)
constexpr int OFF_VH = 0;                                    // 4 slabs: basis head, [chunk][rotated channel][32 channels]
constexpr int OFF_VL = OFF_VH + NCHUNK * SLAB;               // 4 slabs: basis tail
constexpr int OFF_XH = OFF_VL + NCHUNK * SLAB;               // 2 slabs: key head (double buffer)
constexpr int OFF_XL = OFF_XH + 2 * SLAB;                    // 2 slabs: key tail
constexpr int OFF_STAGE = OFF_XL + 2 * SLAB;                 // 8 warps x 32 x 32 floats
constexpr int OFF_MU = OFF_STAGE + 8 * 32 * 32 * 4;          // 128 floats
constexpr int OFF_BAR = OFF_MU + FATHOM_D * 4;               // 3 mbarriers + tensor-memory base
constexpr int TC_SMEM = OFF_BAR + 64 + 1024;                 // + slack for the manual 1024-byte alignment

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ float tf32_head(float x) { return __uint_as_float(__float_as_uint(x) & 0xffffe000u); }

// byte offset inside a slab of the 16-byte piece `c4` (0..7) of row `row`: rows are 128 bytes, eight rows form a
// 1024-byte group, and inside a group piece c4 of row r sits at position c4 ^ r (the 128-byte swizzle)
__device__ __forceinline__ int slab_offset(int row, int c4) { return (row >> 3) * 1024 + (row & 7) * 128 + ((c4 ^ (row & 7)) << 4); }

// K-major, 128-byte swizzle: start address, leading offset 1 (unused), 1024 bytes between 8-row groups, version 1
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// fp32 accumulator, tf32 A and B, both K-major, N = 128, M = 128
constexpr uint32_t UMMA_IDESC = (1u << 4) | (2u << 7) | (2u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
      :: "r"(tmem_d), "l"(a), "l"(b), "r"(UMMA_IDESC), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
// Bounded wait for the phase with the given parity; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < WAIT_TRIES; ++i) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    if (i > 64) __nanosleep(32);
  }
  return false;
}

// ---- basis prepared for the MMA: transposed (K-major for the B operand) and split into tf32 head and tail
__global__ void __launch_bounds__(FATHOM_D)
split_basis_kernel(const float* __restrict__ basis, float* __restrict__ vh_t, float* __restrict__ vl_t) {
  const int kv = blockIdx.y, j = blockIdx.x, c = threadIdx.x;                 // out[kv][j][c] = basis[kv][c][j]
  const float v = basis[((size_t)kv * FATHOM_D + c) * FATHOM_D + j];
  const float h = tf32_head(v);
  vh_t[((size_t)kv * FATHOM_D + j) * FATHOM_D + c] = h;
  vl_t[((size_t)kv * FATHOM_D + j) * FATHOM_D + c] = tf32_head(v - h);
}

template <typename T> __device__ __forceinline__ float4 load_row4(const T* p);
template <> __device__ __forceinline__ float4 load_row4<float>(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
template <> __device__ __forceinline__ float4 load_row4<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                     __uint_as_float(u.y & 0xffff0000u));
}

template <typename T>
__global__ void __launch_bounds__(TC_THREADS, 1)
rotate_keys_tc_kernel(const T* __restrict__ K, const float* __restrict__ mean, const float* __restrict__ vh_t,
                      const float* __restrict__ vl_t, float* __restrict__ K_rot, long long n, long long tiles_per_head,
                      long long total_tiles, uint32_t* __restrict__ dev_status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-byte aligned in the shared window
  const uint32_t sm_base = smem_u32(sm);
  float* s_mu = reinterpret_cast<float*>(sm + OFF_MU);
  float* s_stage = reinterpret_cast<float*>(sm + OFF_STAGE);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm + OFF_BAR + 32);
  const uint32_t bar_empty0 = sm_base + OFF_BAR, bar_empty1 = sm_base + OFF_BAR + 8, bar_acc = sm_base + OFF_BAR + 16;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // contiguous range of tiles of this CTA over the (KV head, tile) space
  const long long g0 = total_tiles * blockIdx.x / gridDim.x, g1 = total_tiles * (blockIdx.x + 1) / gridDim.x;

  if (tid == 0) {
    mbar_init(bar_empty0, 1);
    mbar_init(bar_empty1, 1);
    mbar_init(bar_acc, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {                                            // one warp owns the tensor-memory allocation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = *s_tmem;

  // the thread's share of a chunk: four 16-byte pieces, rows row0 + 32 i, piece c4 of the row
  const int c4 = tid & 7, row0 = tid >> 3;
  float4 xr[NCHUNK][4];                                       // one tile ahead, in registers
  auto load_tile = [&](long long g, int kc) {
    const long long kv = g / tiles_per_head, r0 = (g % tiles_per_head) * TILE_M;
    const T* Kh = K + ((size_t)kv * (size_t)n) * FATHOM_D + kc * KC + c4 * 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const long long r = r0 + row0 + 32 * i;
      xr[kc][i] = (g < g1 && r < n) ? load_row4<T>(Kh + (size_t)r * FATHOM_D) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  if (g0 < g1) {
#pragma unroll
    for (int kc = 0; kc < NCHUNK; ++kc) load_tile(g0, kc);
  }

  bool alive = true;                                          // false once a bounded wait ran out
  uint32_t q = 0, tcount = 0;                                 // chunks and tiles handled so far (mbarrier phases)
  long long cur_kv = -1;
  for (long long g = g0; g < g1; ++g, ++tcount) {
    const long long kv = g / tiles_per_head, r0 = (g % tiles_per_head) * TILE_M;
    if (kv != cur_kv) {                                       // new head: its split basis and mean into shared memory
      __syncthreads();                                        // the previous tile's epilogue waited for all MMAs: nobody reads the old ones
      const float4* gh = reinterpret_cast<const float4*>(vh_t + (size_t)kv * FATHOM_D * FATHOM_D);
      const float4* gl = reinterpret_cast<const float4*>(vl_t + (size_t)kv * FATHOM_D * FATHOM_D);
      for (int e = tid; e < FATHOM_D * (FATHOM_D / 4); e += TC_THREADS) {
        const int j = e >> 5, f = e & 31, kc = f >> 3, p = f & 7;       // row j, 16-byte piece f of the row
        const int off = kc * SLAB + slab_offset(j, p);
        *reinterpret_cast<float4*>(sm + OFF_VH + off) = __ldg(gh + e);
        *reinterpret_cast<float4*>(sm + OFF_VL + off) = __ldg(gl + e);
      }
      if (tid < FATHOM_D) s_mu[tid] = mean[(size_t)kv * FATHOM_D + tid];
      cur_kv = kv;
      __syncthreads();
    }
#pragma unroll
    for (int kc = 0; kc < NCHUNK; ++kc, ++q) {
      const int buf = q & 1;
      const uint32_t bar_empty = buf ? bar_empty1 : bar_empty0;
      if (q >= 2 && alive && !mbar_wait(bar_empty, ((q >> 1) - 1) & 1)) alive = false;   // the MMAs that read this buffer are done
      const float4 mu = *reinterpret_cast<const float4*>(s_mu + kc * KC + c4 * 4);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float4 x = xr[kc][i];
        const float a0 = x.x - mu.x, a1 = x.y - mu.y, a2 = x.z - mu.z, a3 = x.w - mu.w;
        const float h0 = tf32_head(a0), h1 = tf32_head(a1), h2 = tf32_head(a2), h3 = tf32_head(a3);
        const int row = row0 + 32 * i;
        const bool real = r0 + row < n;                       // rows past the end stay zero (the mean is not subtracted)
        const int off = buf * SLAB + slab_offset(row, c4);
        *reinterpret_cast<float4*>(sm + OFF_XH + off) = real ? make_float4(h0, h1, h2, h3) : make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4*>(sm + OFF_XL + off) =
            real ? make_float4(tf32_head(a0 - h0), tf32_head(a1 - h1), tf32_head(a2 - h2), tf32_head(a3 - h3))
                 : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      load_tile(g + 1, kc);                                   // the registers are free: fetch the next tile's chunk
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> visible to the MMA
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();
      if (tid == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t xh = sm_base + OFF_XH + buf * SLAB, xl = sm_base + OFF_XL + buf * SLAB;
        const uint32_t vh = sm_base + OFF_VH + kc * SLAB, vl = sm_base + OFF_VL + kc * SLAB;
#pragma unroll
        for (int ks = 0; ks < KC / UMMA_K; ++ks) {
          const uint32_t ko = ks * UMMA_K * 4;                // bytes along K inside the swizzled row
          umma_tf32(tmem_d, umma_desc(xl + ko), umma_desc(vh + ko), (kc | ks) ? 1u : 0u);
          umma_tf32(tmem_d, umma_desc(xh + ko), umma_desc(vl + ko), 1u);
          umma_tf32(tmem_d, umma_desc(xh + ko), umma_desc(vh + ko), 1u);
        }
        umma_commit(bar_empty);
        if (kc == NCHUNK - 1) umma_commit(bar_acc);
      }
    }
    // ---- epilogue: accumulator -> registers -> per-warp staging -> 128-byte rows in global memory
    if (alive && !mbar_wait(bar_acc, tcount & 1)) alive = false;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    {
      const int lq = warp & 3, cb = (warp >> 2) * 64;
      float* st = s_stage + warp * 1024;
      float* out = K_rot + ((size_t)kv * (size_t)n + (size_t)r0 + lq * 32) * FATHOM_D + cb;
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        uint32_t r[32];
        const uint32_t taddr = tmem_d + ((uint32_t)(lq * 32) << 16) + (uint32_t)(cb + p * 32);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
              "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
              "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
              "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
            : "r"(taddr) : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int c = 0; c < 32; ++c) st[lane * 32 + (c ^ lane)] = __uint_as_float(r[c]);   // lane = row of the warp's 32
        __syncwarp();
#pragma unroll 8
        for (int rr = 0; rr < 32; ++rr)
          if (r0 + lq * 32 + rr < n) out[(size_t)rr * FATHOM_D + p * 32 + lane] = st[rr * 32 + (lane ^ rr)];
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");   // the next tile's first MMA overwrites the accumulator
  }

  // ---- all MMAs issued by this CTA are complete (their commits were waited for) unless a wait ran out
  if (!alive && dev_status) atomicOr(dev_status, FATHOM_DEV_WAIT_EXPIRED);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace

size_t fathom_rotate_tc_scratch_bytes(int Hkv) { return fathom_round_up((size_t)2 * Hkv * FATHOM_D * FATHOM_D * 4, 256); }

// Enqueues the tensor-core rotation; scratch holds the split, transposed basis (fathom_rotate_tc_scratch_bytes).
int fathom_launch_rotate_tc(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, const float* mean,
                            const float* basis, float* K_rot, void* scratch, cudaStream_t st) {
  const int Hkv = L->n_kv_heads;
  const long long n = L->n;
  float* vh_t = static_cast<float*>(scratch);
  float* vl_t = vh_t + (size_t)Hkv * FATHOM_D * FATHOM_D;
  split_basis_kernel<<<dim3(FATHOM_D, Hkv), FATHOM_D, 0, st>>>(basis, vh_t, vl_t);
  int dev = 0, sms = 0;
  FATHOM_CUDA_TRY(ctx, cudaGetDevice(&dev));
  FATHOM_CUDA_TRY(ctx, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const long long tiles_per_head = (n + TILE_M - 1) / TILE_M, total = tiles_per_head * Hkv;
  const unsigned grid = (unsigned)(total < sms ? total : sms);
  if (k_dtype == FATHOM_F32) {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(rotate_keys_tc_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM));
    rotate_keys_tc_kernel<float><<<grid, TC_THREADS, TC_SMEM, st>>>(static_cast<const float*>(K), mean, vh_t, vl_t, K_rot, n,
                                                                     tiles_per_head, total, ctx->dev_status);
  } else {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(rotate_keys_tc_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM));
    rotate_keys_tc_kernel<__nv_bfloat16><<<grid, TC_THREADS, TC_SMEM, st>>>(static_cast<const __nv_bfloat16*>(K), mean, vh_t, vl_t,
                                                                             K_rot, n, tiles_per_head, total, ctx->dev_status);
  }
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
