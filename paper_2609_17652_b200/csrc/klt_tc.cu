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
// basis (transposed, K-major) stays in shared memory for the whole tile range.  Two 128 x 128 fp32 accumulators
// alternate: while the tensor cores work on tile t, the accumulator of tile t - 1 is read back with tcgen05.ld (warp
// w: lanes 32 (w mod 4).., columns 64 (w div 4)..), staged per warp in shared memory and written to global memory in
// 128-byte rows.
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
constexpr uint32_t TMEM_COLS = 256;                          // two fp32 accumulators of 128 columns
constexpr uint32_t WAIT_TRIES = 1u << 22;

// shared-memory map (bytes from a 1024-byte aligned base)
constexpr int OFF_VH = 0;                                    // 4 slabs: basis head, [chunk][rotated channel][32 channels]
constexpr int OFF_VL = OFF_VH + NCHUNK * SLAB;               // 4 slabs: basis tail
constexpr int OFF_XH = OFF_VL + NCHUNK * SLAB;               // 2 slabs: key head (double buffer)
constexpr int OFF_XL = OFF_XH + 2 * SLAB;                    // 2 slabs: key tail
constexpr int OFF_STAGE = OFF_XL + 2 * SLAB;                 // 8 warps x 32 x 32 floats
constexpr int OFF_MU = OFF_STAGE + 8 * 32 * 32 * 4;          // 128 floats
constexpr int OFF_BAR = OFF_MU + FATHOM_D * 4;               // 4 mbarriers + tensor-memory base
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t tries = WAIT_TRIES) {
  for (uint32_t i = 0; i < tries; ++i) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    if (i > 64) __nanosleep(32);
  }
  return false;
}

// The give-up path of the bounded wait, exercised on its own: one thread waits `tries` times on a barrier that nothing will
// ever arrive on (no copy, no MMA, nothing asynchronous is outstanding), reports FATHOM_DEV_WAIT_EXPIRED and returns.
__global__ void wait_expiry_selftest_kernel(uint32_t* dev_status, uint32_t tries) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait(b, 0, tries)) atomicOr(dev_status, FATHOM_DEV_WAIT_EXPIRED);
  }
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
  const uint32_t bar_empty0 = sm_base + OFF_BAR, bar_empty1 = sm_base + OFF_BAR + 8, bar_acc0 = sm_base + OFF_BAR + 16,
                 bar_acc1 = sm_base + OFF_BAR + 24;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // contiguous range of tiles of this CTA over the (KV head, tile) space
  const long long g0 = total_tiles * blockIdx.x / gridDim.x, g1 = total_tiles * (blockIdx.x + 1) / gridDim.x;

  if (tid == 0) {
    mbar_init(bar_empty0, 1);
    mbar_init(bar_empty1, 1);
    mbar_init(bar_acc0, 1);
    mbar_init(bar_acc1, 1);
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
  const int x_off = slab_offset(row0, c4);
  float4 xr[NCHUNK][4];                                       // one tile ahead, in registers
  // rows r_first + row0 + 32 i of the head whose keys start at Kh (nullptr: no such tile, zeros)
  auto load_tile = [&](const T* Kh, long long r_first, int kc) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const long long r = r_first + row0 + 32 * i;
      xr[kc][i] = (Kh != nullptr && r < n) ? load_row4<T>(Kh + (size_t)r * FATHOM_D + kc * KC + c4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  auto head_keys = [&](long long kv) { return K + (size_t)kv * (size_t)n * FATHOM_D; };
  if (g0 < g1) {
#pragma unroll
    for (int kc = 0; kc < NCHUNK; ++kc) load_tile(head_keys(g0 / tiles_per_head), (g0 % tiles_per_head) * TILE_M, kc);
  }

  bool alive = true;                                          // false once a bounded wait ran out
  uint32_t q = 0, tcount = 0;                                 // chunks and tiles handled so far (mbarrier phases)
  long long cur_kv = -1;

  // accumulator `acc` (tile number t, rows r0.. of head kv) -> registers -> per-warp staging -> 128-byte rows in global
  // memory.  It runs one tile late, while the tensor cores work on the next tile in the other accumulator.
  auto epilogue = [&](long long kv, long long r0, uint32_t t) {
    const uint32_t acc = t & 1u;
    if (alive && !mbar_wait(acc ? bar_acc1 : bar_acc0, (t >> 1) & 1u)) alive = false;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int lq = warp & 3, cb = (warp >> 2) * 64;
    float4* st4 = reinterpret_cast<float4*>(s_stage + warp * 1024);     // 32 rows of 8 16-byte pieces, piece f of row r at f ^ (r & 7)
    float* out = K_rot + ((size_t)kv * (size_t)n + (size_t)r0 + lq * 32) * FATHOM_D + cb;
    const int rows_valid = (int)min((long long)32, n - r0 - lq * 32);  // rows of this warp inside the sequence (may be <= 0)
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      uint32_t r[32];
      const uint32_t taddr = tmem_d + ((uint32_t)(lq * 32) << 16) + acc * 128u + (uint32_t)(cb + p * 32);
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
      for (int f = 0; f < 8; ++f)                                        // lane = row: its 32 columns as eight pieces
        st4[lane * 8 + (f ^ (lane & 7))] = make_float4(__uint_as_float(r[4 * f]), __uint_as_float(r[4 * f + 1]),
                                                        __uint_as_float(r[4 * f + 2]), __uint_as_float(r[4 * f + 3]));
      __syncwarp();
#pragma unroll
      for (int it = 0; it < 8; ++it) {                                   // four rows of 128 bytes per store instruction
        const int rr = it * 4 + (lane >> 3), f = lane & 7;
        if (rr < rows_valid)
          *reinterpret_cast<float4*>(out + (size_t)rr * FATHOM_D + p * 32 + f * 4) = st4[rr * 8 + (f ^ (rr & 7))];
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");   // a later MMA overwrites this accumulator
  };

  long long prev_kv = -1, prev_r0 = 0;                        // tile whose epilogue is still due
  long long kv = g0 / tiles_per_head, tile_in_head = g0 % tiles_per_head;
  for (long long g = g0; g < g1; ++g, ++tcount) {
    const long long r0 = tile_in_head * TILE_M;
    long long kv_next = kv, tile_next = tile_in_head + 1;     // the tile after this one (fetched while this one is handled)
    if (tile_next == tiles_per_head) { tile_next = 0; ++kv_next; }
    const T* K_next = (g + 1 < g1) ? head_keys(kv_next) : nullptr;
    const long long r_next = tile_next * TILE_M;
    if (kv != cur_kv) {                                       // new head: its split basis and mean into shared memory
      if (prev_kv >= 0) { epilogue(prev_kv, prev_r0, tcount - 1); prev_kv = -1; }   // also waits for every MMA issued so far
      __syncthreads();                                        // nobody reads the old basis any more
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
    const uint32_t acc_col = tmem_d + (tcount & 1u) * 128u;
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
        const int off = buf * SLAB + x_off + i * 4096;        // row0 + 32 i: four 8-row groups further, same place in the group
        // (rows past the end of the sequence give rows of the accumulator that are never written out)
        *reinterpret_cast<float4*>(sm + OFF_XH + off) = make_float4(h0, h1, h2, h3);
        *reinterpret_cast<float4*>(sm + OFF_XL + off) = make_float4(tf32_head(a0 - h0), tf32_head(a1 - h1), tf32_head(a2 - h2), tf32_head(a3 - h3));
      }
      load_tile(K_next, r_next, kc);                          // the registers are free: fetch the next tile's chunk
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
          umma_tf32(acc_col, umma_desc(xl + ko), umma_desc(vh + ko), (kc | ks) ? 1u : 0u);
          umma_tf32(acc_col, umma_desc(xh + ko), umma_desc(vl + ko), 1u);
          umma_tf32(acc_col, umma_desc(xh + ko), umma_desc(vh + ko), 1u);
        }
        umma_commit(bar_empty);
        if (kc == NCHUNK - 1) umma_commit((tcount & 1u) ? bar_acc1 : bar_acc0);
      }
    }
    if (prev_kv >= 0) epilogue(prev_kv, prev_r0, tcount - 1);  // the previous tile, while this one's MMAs run
    prev_kv = kv;
    prev_r0 = r0;
    kv = kv_next;
    tile_in_head = tile_next;
  }
  if (prev_kv >= 0) epilogue(prev_kv, prev_r0, tcount - 1);

  // ---- all MMAs issued by this CTA are complete (their commits were waited for) unless a wait ran out
  if (!alive && dev_status) atomicOr(dev_status, FATHOM_DEV_WAIT_EXPIRED);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"(TMEM_COLS) : "memory");
  }
}

// ---- rotation fused with the plane builder: planes and scales of (K - mu) V without ever storing the rotated keys ----
// Same tile pipeline and the same sequence of MMAs as rotate_keys_tc_kernel (so every accumulator value is bit for bit
// the rotated key that kernel would store), but the epilogue quantises instead of storing: a CTA takes 256 tokens at a
// time (two tiles, one per accumulator = four 64-token blocks), and per block and channel forms a = max |k'| (one
// redux per channel over the warp's 32 tokens, the two halves of a block meet in shared memory), the fp16 scale a/8,
// the four plane bits of every code by the plane builder's comparisons with exact multiples of the stored scale, and
// the plane words by warp ballots.  The four blocks' words of a (channel, plane) row are one 32-byte sector, written whole.
constexpr int FB_PITCH = FATHOM_NPLANES * 4 * 2 + 1;         // words per channel in the staging: [plane][block][half], padded
constexpr int FB_OFF_OUT = OFF_XL + 2 * SLAB;                // 128 x FB_PITCH words
constexpr int FB_OFF_SCALE = FB_OFF_OUT + FATHOM_D * FB_PITCH * 4;          // 128 x 4 fp16
constexpr int FB_OFF_AMAX = FB_OFF_SCALE + FATHOM_D * 4 * 2;                // [2 blocks][2 halves][128] floats
constexpr int FB_OFF_MU = FB_OFF_AMAX + 2 * 2 * FATHOM_D * 4;
constexpr int FB_OFF_BAR = FB_OFF_MU + FATHOM_D * 4;
constexpr int FB_SMEM = FB_OFF_BAR + 64 + 1024;

template <typename T>
__global__ void __launch_bounds__(TC_THREADS, 1)
rotate_build_tc_kernel(const T* __restrict__ K, const float* __restrict__ mean, const float* __restrict__ vh_t,
                       const float* __restrict__ vl_t, uint32_t* __restrict__ planes32, uint16_t* __restrict__ scales,
                       long long n, long long plane_stride, long long scale_stride, uint32_t* __restrict__ dev_status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sm_base = smem_u32(sm);
  float* s_mu = reinterpret_cast<float*>(sm + FB_OFF_MU);
  uint32_t* s_out = reinterpret_cast<uint32_t*>(sm + FB_OFF_OUT);
  uint16_t* s_scale = reinterpret_cast<uint16_t*>(sm + FB_OFF_SCALE);
  float* s_amax = reinterpret_cast<float*>(sm + FB_OFF_AMAX);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm + FB_OFF_BAR + 32);
  const uint32_t bar_empty0 = sm_base + FB_OFF_BAR, bar_empty1 = sm_base + FB_OFF_BAR + 8, bar_acc0 = sm_base + FB_OFF_BAR + 16,
                 bar_acc1 = sm_base + FB_OFF_BAR + 24;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, kv = blockIdx.y;
  const long long nb = (n + FATHOM_BLOCK - 1) / FATHOM_BLOCK;
  const long long supers = (n + 255) / 256;                   // 256-token units of this head
  const long long u0 = supers * blockIdx.x / gridDim.x, u1 = supers * (blockIdx.x + 1) / gridDim.x;
  const T* Kh = K + (size_t)kv * (size_t)n * FATHOM_D;

  if (tid == 0) {
    mbar_init(bar_empty0, 1);
    mbar_init(bar_empty1, 1);
    mbar_init(bar_acc0, 1);
    mbar_init(bar_acc1, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  {                                                           // the head's split basis and mean
    const float4* gh = reinterpret_cast<const float4*>(vh_t + (size_t)kv * FATHOM_D * FATHOM_D);
    const float4* gl = reinterpret_cast<const float4*>(vl_t + (size_t)kv * FATHOM_D * FATHOM_D);
    for (int e = tid; e < FATHOM_D * (FATHOM_D / 4); e += TC_THREADS) {
      const int j = e >> 5, f = e & 31, kc = f >> 3, p = f & 7;
      const int off = kc * SLAB + slab_offset(j, p);
      *reinterpret_cast<float4*>(sm + OFF_VH + off) = __ldg(gh + e);
      *reinterpret_cast<float4*>(sm + OFF_VL + off) = __ldg(gl + e);
    }
    if (tid < FATHOM_D) s_mu[tid] = mean[(size_t)kv * FATHOM_D + tid];
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = *s_tmem;

  const int c4 = tid & 7, row0 = tid >> 3;
  const int x_off = slab_offset(row0, c4);
  float4 xr[NCHUNK][4];                                       // one 128-token tile ahead, in registers
  const long long tile_end = u1 * 2;                          // tiles of this CTA: [2 u0, 2 u1)
  auto load_tile = [&](long long tile, int kc) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const long long r = tile * TILE_M + row0 + 32 * i;
      xr[kc][i] = (tile < tile_end && r < n) ? load_row4<T>(Kh + (size_t)r * FATHOM_D + kc * KC + c4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  if (u0 < u1) {
#pragma unroll
    for (int kc = 0; kc < NCHUNK; ++kc) load_tile(2 * u0, kc);
  }

  bool alive = true;
  uint32_t q = 0, ucount = 0;
  for (long long u = u0; u < u1; ++u, ++ucount) {
    // ---- both tiles of the unit: chunks -> shared memory -> MMAs into accumulator 0 / 1
#pragma unroll
    for (int sub = 0; sub < 2; ++sub) {
      const long long tile = 2 * u + sub;
      const uint32_t acc_col = tmem_d + (uint32_t)sub * 128u;
#pragma unroll
      for (int kc = 0; kc < NCHUNK; ++kc, ++q) {
        const int buf = q & 1;
        const uint32_t bar_empty = buf ? bar_empty1 : bar_empty0;
        if (q >= 2 && alive && !mbar_wait(bar_empty, ((q >> 1) - 1) & 1)) alive = false;
        const float4 mu = *reinterpret_cast<const float4*>(s_mu + kc * KC + c4 * 4);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 x = xr[kc][i];
          const float a0 = x.x - mu.x, a1 = x.y - mu.y, a2 = x.z - mu.z, a3 = x.w - mu.w;
          const float h0 = tf32_head(a0), h1 = tf32_head(a1), h2 = tf32_head(a2), h3 = tf32_head(a3);
          const int off = buf * SLAB + x_off + i * 4096;
          *reinterpret_cast<float4*>(sm + OFF_XH + off) = make_float4(h0, h1, h2, h3);
          *reinterpret_cast<float4*>(sm + OFF_XL + off) = make_float4(tf32_head(a0 - h0), tf32_head(a1 - h1), tf32_head(a2 - h2), tf32_head(a3 - h3));
        }
        load_tile(tile + 1, kc);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t xh = sm_base + OFF_XH + buf * SLAB, xl = sm_base + OFF_XL + buf * SLAB;
          const uint32_t vh = sm_base + OFF_VH + kc * SLAB, vl = sm_base + OFF_VL + kc * SLAB;
#pragma unroll
          for (int ks = 0; ks < KC / UMMA_K; ++ks) {
            const uint32_t ko = ks * UMMA_K * 4;
            umma_tf32(acc_col, umma_desc(xl + ko), umma_desc(vh + ko), (kc | ks) ? 1u : 0u);
            umma_tf32(acc_col, umma_desc(xh + ko), umma_desc(vl + ko), 1u);
            umma_tf32(acc_col, umma_desc(xh + ko), umma_desc(vh + ko), 1u);
          }
          umma_commit(bar_empty);
          if (kc == NCHUNK - 1) umma_commit(sub ? bar_acc1 : bar_acc0);
        }
      }
    }
    // ---- quantising epilogue, tile by tile.  Warp w: tokens 32 (w & 3) .. + 31 of the tile, channels 64 (w >> 2) .. + 63.
    const int lq = warp & 3, blk = lq >> 1, half = lq & 1, cb = (warp >> 2) * 64;
#pragma unroll 1
    for (int sub = 0; sub < 2; ++sub) {
      if (alive && !mbar_wait(sub ? bar_acc1 : bar_acc0, ucount & 1)) alive = false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const long long tok = (2 * u + sub) * TILE_M + lq * 32 + lane;          // this lane's token
      const bool present = tok < n;
      const uint32_t keep = __ballot_sync(0xffffffffu, present);             // absent tail tokens carry 0 bits
      uint32_t r[2][32];
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const uint32_t taddr = tmem_d + ((uint32_t)(lq * 32) << 16) + (uint32_t)sub * 128u + (uint32_t)(cb + p * 32);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
            : "=r"(r[p][0]), "=r"(r[p][1]), "=r"(r[p][2]), "=r"(r[p][3]), "=r"(r[p][4]), "=r"(r[p][5]), "=r"(r[p][6]), "=r"(r[p][7]),
              "=r"(r[p][8]), "=r"(r[p][9]), "=r"(r[p][10]), "=r"(r[p][11]), "=r"(r[p][12]), "=r"(r[p][13]), "=r"(r[p][14]),
              "=r"(r[p][15]), "=r"(r[p][16]), "=r"(r[p][17]), "=r"(r[p][18]), "=r"(r[p][19]), "=r"(r[p][20]), "=r"(r[p][21]),
              "=r"(r[p][22]), "=r"(r[p][23]), "=r"(r[p][24]), "=r"(r[p][25]), "=r"(r[p][26]), "=r"(r[p][27]), "=r"(r[p][28]),
              "=r"(r[p][29]), "=r"(r[p][30]), "=r"(r[p][31])
            : "r"(taddr) : "memory");
      }
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      // block maximum per channel: |k'| of non-negative floats orders like its bit pattern, so one integer redux per
      // channel gives the warp's maximum; lane c keeps channel c's
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        uint32_t mine = 0u;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          if (!present) r[p][c] = 0u;                         // an absent token counts as 0 everywhere
          const uint32_t m = __reduce_max_sync(0xffffffffu, r[p][c] & 0x7fffffffu);
          if (lane == c) mine = m;
        }
        s_amax[(blk * 2 + half) * FATHOM_D + cb + p * 32 + lane] = __uint_as_float(mine);
      }
      __syncthreads();                                        // the two halves of every block have met
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const int ch = cb + p * 32 + lane;                    // the channel whose scale and plane words this lane keeps
        const float a = fmaxf(s_amax[(blk * 2 + 0) * FATHOM_D + ch], s_amax[(blk * 2 + 1) * FATHOM_D + ch]);
        const __half sh = __float2half_rn(a * 0.125f);        // a/8 is exact; one rounding to fp16
        const float my_sc = __half2float(sh);
        uint32_t w0 = 0u, w1 = 0u, w2 = 0u, w3 = 0u;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const float sc = __shfl_sync(0xffffffffu, my_sc, c);               // scale of channel cb + 32 p + c
          const float k = __uint_as_float(r[p][c]);
          const float s2 = sc * 2.0f, s4 = sc * 4.0f;
          const bool c0 = k >= 0.0f;
          float thr = c0 ? s4 : -s4;
          const bool c1 = k >= thr;
          thr += c1 ? s2 : -s2;
          const bool c2 = k >= thr;
          thr += c2 ? sc : -sc;
          const bool c3 = k >= thr;
          const uint32_t b0 = __ballot_sync(0xffffffffu, c0), b1 = __ballot_sync(0xffffffffu, c1);
          const uint32_t b2 = __ballot_sync(0xffffffffu, c2), b3 = __ballot_sync(0xffffffffu, c3);
          if (lane == c) { w0 = b0; w1 = b1; w2 = b2; w3 = b3; }
        }
        if (my_sc > 0.0f) { w0 &= keep; w1 &= keep; w2 &= keep; w3 &= keep; }
        else { w0 = keep; w1 = 0u; w2 = 0u; w3 = 0u; }        // zero scale: every code is 8 = 0b1000
        const int bu = 2 * sub + blk;                         // block within the 256-token unit
        uint32_t* o = s_out + ch * FB_PITCH;
        o[(0 * 4 + bu) * 2 + half] = w0;
        o[(1 * 4 + bu) * 2 + half] = w1;
        o[(2 * 4 + bu) * 2 + half] = w2;
        o[(3 * 4 + bu) * 2 + half] = w3;
        if (half == 0) s_scale[ch * 4 + bu] = __half_as_ushort(sh);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();                                        // s_amax is reused by the next tile
    }
    // ---- flush: the unit's four blocks of every (channel, plane) row are 32 contiguous bytes
    {
      const long long b0 = 4 * u;
      const int nblk = (int)min((long long)4, nb - b0);
      uint64_t* planes64 = reinterpret_cast<uint64_t*>(planes32);
      for (int e = tid; e < FATHOM_D * FATHOM_NPLANES; e += TC_THREADS) {
        const int ch = e >> 2, p = e & 3;
        const uint32_t* src = s_out + ch * FB_PITCH + p * 8;
        uint64_t* dst = planes64 + (((size_t)kv * FATHOM_D + ch) * FATHOM_NPLANES + p) * (size_t)plane_stride + b0;
#pragma unroll
        for (int pair = 0; pair < 2; ++pair) {
          if (2 * pair + 1 < nblk) {
            *reinterpret_cast<uint4*>(dst + 2 * pair) = make_uint4(src[4 * pair], src[4 * pair + 1], src[4 * pair + 2], src[4 * pair + 3]);
          } else if (2 * pair < nblk) {
            dst[2 * pair] = ((uint64_t)src[4 * pair + 1] << 32) | src[4 * pair];
          }
        }
      }
      if (tid < FATHOM_D) {
        uint16_t* dst = scales + ((size_t)kv * FATHOM_D + tid) * (size_t)scale_stride + b0;
        for (int x = 0; x < nblk; ++x) dst[x] = s_scale[tid * 4 + x];
      }
    }
    __syncthreads();                                          // the staging is rewritten by the next unit
  }

  if (!alive && dev_status) atomicOr(dev_status, FATHOM_DEV_WAIT_EXPIRED);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"(TMEM_COLS) : "memory");
  }
}

// ---- covariance partials on the tensor cores: C = sum_t (x_t - mu)(x_t - mu)^T ----------------------------------------
// D[i][j] += sum_t A[i][t] B[j][t] with A = B = (X - mu)^T, i.e. M = N = 128 channels and K = tokens.  X is stored token
// by token with the channels contiguous, which is the MN-major operand form: a slab holds 64 tokens x 32 channels in
// rows of 128 bytes (row = token; swizzled in 32-byte pieces over groups of four rows, the only form MN-major tf32
// operands take), four slabs side by side cover the 128 channels (leading offset = slab size), eight token rows
// (1024 bytes) are one K step.  Head and tail of the split keys serve as both operands:
// xh xh^T + xh xl^T + xl xh^T.  A CTA accumulates a contiguous token range of one KV head in tensor memory and writes
// one 128 x 128 partial at the end; the partials are summed in fp64 by the caller's reduction kernel.
constexpr int CV_TOK = 64;                                   // tokens per stage
constexpr int CV_SLAB = CV_TOK * 128;                        // 8 KB: 64 token rows of 128 bytes (32 channels)
constexpr int CV_PART = NCHUNK * CV_SLAB;                    // 32 KB: head (or tail) of one stage, 128 channels
constexpr int CV_OFF_STAGE = 4 * CV_PART;                    // two stages x (head, tail), then the epilogue staging
constexpr int CV_OFF_MU = CV_OFF_STAGE + 8 * 32 * 32 * 4;
constexpr int CV_OFF_BAR = CV_OFF_MU + FATHOM_D * 4;
constexpr int CV_SMEM = CV_OFF_BAR + 64 + 1024;
// MN-major operands of 32-bit elements take the 128-byte swizzle with a 32-byte base: rows of 128 bytes (32 channels) in
// groups of FOUR, and inside a group the 32-byte piece p of row r sits at position p ^ (r & 3).
__device__ __forceinline__ int slab_offset_mn(int row, int c4) { return row * 128 + (((((c4 >> 1) ^ (row & 3)) << 1) | (c4 & 1)) << 4); }
// descriptor: leading offset = bytes between 32-channel slabs, stride offset = bytes between 4-token groups, layout type 1
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3ffffu) >> 4) | ((uint64_t)(CV_SLAB >> 4) << 16) | ((uint64_t)(512 >> 4) << 32) | (1ull << 46) | (1ull << 61);
}
constexpr uint32_t UMMA_IDESC_MN = UMMA_IDESC | (1u << 15) | (1u << 16);   // A and B MN-major
__device__ __forceinline__ void umma_tf32_mn(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
      :: "r"(tmem_d), "l"(a), "l"(b), "r"(UMMA_IDESC_MN), "r"(accumulate), "r"(0u) : "memory");
}

// shift[kv][c] = mean of channel c over 64 keys spread evenly over the head's sequence (any value near the data would
// do; it only has to keep S S^T / n small against the sum of squares - keys from one place, e.g. the first tokens of a
// prompt, may sit far from the rest)
template <typename T>
__global__ void __launch_bounds__(FATHOM_D)
cov_shift_kernel(const T* __restrict__ K, long long n, float* __restrict__ shift) {
  const int kv = blockIdx.x, c = threadIdx.x;
  const T* Kh = K + (size_t)kv * (size_t)n * FATHOM_D;
  const int rows = (int)min((long long)64, n);
  const long long step = n / rows;                            // >= 1
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int r = 0; r < rows; r += 8)
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (r + u < rows) acc[u] += (float)Kh[(size_t)((r + u) * step) * FATHOM_D + c];
  shift[(size_t)kv * FATHOM_D + c] = (((acc[0] + acc[1]) + (acc[2] + acc[3])) + ((acc[4] + acc[5]) + (acc[6] + acc[7]))) / (float)rows;
}

template <typename T>
__global__ void __launch_bounds__(TC_THREADS, 1)
cov_partial_tc_kernel(const T* __restrict__ K, const float* __restrict__ shift, float* __restrict__ partial,
                      float* __restrict__ partial_sum, long long n, uint32_t* __restrict__ dev_status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sm_base = smem_u32(sm);
  float* s_mu = reinterpret_cast<float*>(sm + CV_OFF_MU);
  float* s_stage = reinterpret_cast<float*>(sm + CV_OFF_STAGE);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm + CV_OFF_BAR + 32);
  const uint32_t bar_empty0 = sm_base + CV_OFF_BAR, bar_empty1 = sm_base + CV_OFF_BAR + 8, bar_acc = sm_base + CV_OFF_BAR + 16;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, kv = blockIdx.y;
  // this CTA's tokens: stages of 64 tokens, split evenly over the CTAs of the head
  const long long stages_total = (n + CV_TOK - 1) / CV_TOK;
  const long long s0 = stages_total * blockIdx.x / gridDim.x, s1 = stages_total * (blockIdx.x + 1) / gridDim.x;
  const T* Kh = K + (size_t)kv * (size_t)n * FATHOM_D;

  if (tid == 0) {
    mbar_init(bar_empty0, 1);
    mbar_init(bar_empty1, 1);
    mbar_init(bar_acc, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(s_tmem)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid < FATHOM_D) s_mu[tid] = shift[(size_t)kv * FATHOM_D + tid];
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = *s_tmem;

  // the thread's share of a stage: eight 16-byte pieces; piece f = tid + 256 i is token f / 32, channels 4 (f % 32)..
  const int q4 = tid & 31, kc = q4 >> 3, c4 = q4 & 7, tok0 = tid >> 5;      // token tok0 + 8 i
  const int x_off = kc * CV_SLAB + slab_offset_mn(tok0, c4);                 // + 1024 i (tokens 8 apart: eight rows further)
  const float4 mu = *reinterpret_cast<const float4*>(s_mu + 4 * q4);
  float4 xr[8];
  auto load_stage = [&](long long st) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const long long t = st * CV_TOK + tok0 + 8 * i;
      xr[i] = (st < s1 && t < n) ? load_row4<T>(Kh + (size_t)t * FATHOM_D + 4 * q4) : make_float4(mu.x, mu.y, mu.z, mu.w);
    }
  };
  load_stage(s0);
  bool alive = true;
  uint32_t q = 0;
  float4 sum4 = make_float4(0.f, 0.f, 0.f, 0.f);              // sum of (x - shift) over this thread's tokens, 4 channels
  for (long long st = s0; st < s1; ++st, ++q) {
    const int buf = q & 1;
    const uint32_t bar_empty = buf ? bar_empty1 : bar_empty0;
    if (q >= 2 && alive && !mbar_wait(bar_empty, ((q >> 1) - 1) & 1)) alive = false;
#pragma unroll
    for (int i = 0; i < 8; ++i) {                             // tokens past the end were loaded as the shift: they add nothing
      const float a0 = xr[i].x - mu.x, a1 = xr[i].y - mu.y, a2 = xr[i].z - mu.z, a3 = xr[i].w - mu.w;
      sum4.x += a0; sum4.y += a1; sum4.z += a2; sum4.w += a3;
      const float h0 = tf32_head(a0), h1 = tf32_head(a1), h2 = tf32_head(a2), h3 = tf32_head(a3);
      const int off = buf * 2 * CV_PART + x_off + i * 1024;
      *reinterpret_cast<float4*>(sm + off) = make_float4(h0, h1, h2, h3);
      *reinterpret_cast<float4*>(sm + off + CV_PART) = make_float4(tf32_head(a0 - h0), tf32_head(a1 - h1), tf32_head(a2 - h2), tf32_head(a3 - h3));
    }
    load_stage(st + 1);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t xh = sm_base + buf * 2 * CV_PART, xl = xh + CV_PART;
#pragma unroll
      for (int ks = 0; ks < CV_TOK / UMMA_K; ++ks) {          // eight tokens per MMA = one 1024-byte group of rows
        const uint64_t dh = umma_desc_mn(xh + ks * 1024), dl = umma_desc_mn(xl + ks * 1024);
        const uint32_t accumulate = (q | (uint32_t)ks) ? 1u : 0u;
        umma_tf32_mn(tmem_d, dh, dh, accumulate);             // first accumulator:  sum xh xh^T
        umma_tf32_mn(tmem_d + 128u, dh, dl, accumulate);      // second accumulator: sum xh xl^T (its transpose is xl xh^T)
      }
      umma_commit(bar_empty);
      if (st == s1 - 1) umma_commit(bar_acc);
    }
  }
  // ---- per-channel sums of (x - shift): the eight threads of a channel quad (one per warp) are added in warp order
  {
    float4* red = reinterpret_cast<float4*>(s_stage);         // [8 warps][32 quads]
    red[warp * 32 + q4] = sum4;
    __syncthreads();
    if (warp == 0) {
      float4 t = red[q4];
#pragma unroll
      for (int w = 1; w < 8; ++w) { const float4 u = red[w * 32 + q4]; t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w; }
      *reinterpret_cast<float4*>(partial_sum + ((size_t)kv * gridDim.x + blockIdx.x) * FATHOM_D + 4 * q4) = t;
    }
    __syncthreads();                                          // the staging area is reused by the epilogue below
  }
  // ---- the partial: accumulator -> registers -> staging -> global memory (zeros if the CTA had no tokens)
  float* out_base = partial + ((size_t)kv * gridDim.x + blockIdx.x) * 2 * FATHOM_D * FATHOM_D;   // two matrices per CTA
  if (s0 < s1) {
    if (alive && !mbar_wait(bar_acc, 0)) alive = false;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  }
#pragma unroll 1
  for (int which = 0; which < 2; ++which) {
    const int lq = warp & 3, cb = (warp >> 2) * 64;
    float4* st4 = reinterpret_cast<float4*>(s_stage + warp * 1024);
    float* out = out_base + (size_t)which * FATHOM_D * FATHOM_D + (size_t)(lq * 32) * FATHOM_D + cb;
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      uint32_t r[32];
      if (s0 < s1) {
        const uint32_t taddr = tmem_d + ((uint32_t)(lq * 32) << 16) + (uint32_t)(which * 128 + cb + p * 32);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
              "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
              "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
              "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
            : "r"(taddr) : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) r[c] = 0u;
      }
      __syncwarp();
#pragma unroll
      for (int f = 0; f < 8; ++f)
        st4[lane * 8 + (f ^ (lane & 7))] = make_float4(__uint_as_float(r[4 * f]), __uint_as_float(r[4 * f + 1]),
                                                        __uint_as_float(r[4 * f + 2]), __uint_as_float(r[4 * f + 3]));
      __syncwarp();
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int rr = it * 4 + (lane >> 3), f = lane & 7;
        *reinterpret_cast<float4*>(out + (size_t)rr * FATHOM_D + p * 32 + f * 4) = st4[rr * 8 + (f ^ (rr & 7))];
      }
    }
  }
  if (!alive && dev_status) atomicOr(dev_status, FATHOM_DEV_WAIT_EXPIRED);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"(256u) : "memory");
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

// CTAs per KV head of the tensor-core covariance pass (one 128 x 128 partial each)
int fathom_cov_tc_ctas_per_head(int Hkv) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int c = sms / (Hkv > 0 ? Hkv : 1);
  return c < 1 ? 1 : c;
}

// Enqueues the shift, the covariance partials [Hkv][ctas][2][128][128] (sum xh xh^T and sum xh xl^T of the shifted
// keys, per CTA) and the per-channel sums [Hkv][ctas][128].
int fathom_launch_cov_tc(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, float* shift, float* partial,
                         float* partial_sum, int ctas_per_head, cudaStream_t st) {
  dim3 grid((unsigned)ctas_per_head, (unsigned)L->n_kv_heads);
  if (k_dtype == FATHOM_F32) {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(cov_partial_tc_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, CV_SMEM));
    cov_shift_kernel<float><<<L->n_kv_heads, FATHOM_D, 0, st>>>(static_cast<const float*>(K), L->n, shift);
    cov_partial_tc_kernel<float><<<grid, TC_THREADS, CV_SMEM, st>>>(static_cast<const float*>(K), shift, partial, partial_sum, L->n,
                                                                     ctx->dev_status);
  } else {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(cov_partial_tc_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, CV_SMEM));
    cov_shift_kernel<__nv_bfloat16><<<L->n_kv_heads, FATHOM_D, 0, st>>>(static_cast<const __nv_bfloat16*>(K), L->n, shift);
    cov_partial_tc_kernel<__nv_bfloat16><<<grid, TC_THREADS, CV_SMEM, st>>>(static_cast<const __nv_bfloat16*>(K), shift, partial,
                                                                             partial_sum, L->n, ctx->dev_status);
  }
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

// Enqueues the fused rotation + plane builder; scratch holds the split, transposed basis (fathom_rotate_tc_scratch_bytes).
int fathom_launch_rotate_build_tc(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, const float* mean,
                                  const float* basis, uint64_t* planes, uint16_t* scales, void* scratch, cudaStream_t st) {
  const int Hkv = L->n_kv_heads;
  const long long n = L->n;
  float* vh_t = static_cast<float*>(scratch);
  float* vl_t = vh_t + (size_t)Hkv * FATHOM_D * FATHOM_D;
  split_basis_kernel<<<dim3(FATHOM_D, Hkv), FATHOM_D, 0, st>>>(basis, vh_t, vl_t);
  int dev = 0, sms = 0;
  FATHOM_CUDA_TRY(ctx, cudaGetDevice(&dev));
  FATHOM_CUDA_TRY(ctx, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const long long supers = (n + 255) / 256;
  long long per_head = sms / Hkv > 0 ? sms / Hkv : 1;
  if (per_head > supers) per_head = supers;
  dim3 grid((unsigned)per_head, (unsigned)Hkv);
  uint32_t* p32 = reinterpret_cast<uint32_t*>(planes);
  if (k_dtype == FATHOM_F32) {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(rotate_build_tc_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, FB_SMEM));
    rotate_build_tc_kernel<float><<<grid, TC_THREADS, FB_SMEM, st>>>(static_cast<const float*>(K), mean, vh_t, vl_t, p32, scales, n,
                                                                      L->plane_stride_words, L->scale_stride, ctx->dev_status);
  } else {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(rotate_build_tc_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, FB_SMEM));
    rotate_build_tc_kernel<__nv_bfloat16><<<grid, TC_THREADS, FB_SMEM, st>>>(static_cast<const __nv_bfloat16*>(K), mean, vh_t, vl_t, p32,
                                                                              scales, n, L->plane_stride_words, L->scale_stride,
                                                                              ctx->dev_status);
  }
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

extern "C" int fathom_selftest_wait_expiry(fathom_ctx* ctx, int tries, void* stream) {
  if (!ctx || tries < 1 || tries > 4096) return FATHOM_ERR_INVALID_ARG;
  wait_expiry_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->dev_status, (uint32_t)tries);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
