// Pieces shared by the two scan kernels (scan.cu: tensor-core accumulate, the default; scan_simt.cu: one predicated
// fp32 add per plane bit, kept selectable) and by the host code that launches them.  Internal, not part of the C ABI.
#pragma once
#include "fathom_common.cuh"

constexpr int FATHOM_SCAN_TILE_BLOCKS = 16;                  // a tile = 16 blocks = 1024 tokens of one plan

// ---- the sessions of one launch: their tiles are laid end to end (fathom_scan has one item)
struct ScanBatch {
  static constexpr int MAX_ITEMS = 32;
  const uint64_t* planes[MAX_ITEMS];
  const uint16_t* scales[MAX_ITEMS];
  const float* q[MAX_ITEMS];
  const uint8_t* depth[MAX_ITEMS];
  float* scores[MAX_ITEMS];
  long long n[MAX_ITEMS], plane_stride[MAX_ITEMS], scale_stride[MAX_ITEMS], score_stride[MAX_ITEMS];
  long long tile_end[MAX_ITEMS];                              // tiles of items 0 .. i, inclusive prefix
  int items;
};

// fp32 value whose order-preserving integer image (see topk.cu) has `bin` as its 12 leading bits and zeros below:
// the lower edge of that histogram bin
__device__ __forceinline__ float fathom_bin_lower_edge(uint32_t bin) {
  if (bin >= FATHOM_TOPK_BINS) return __uint_as_float(0x7fc00000u);   // past the last bin: nothing reaches it (NaN compares false)
  if (bin <= 7u) return -INFINITY;                                    // bins below -inf's hold no finite score: everything reaches them
  const uint32_t key = bin << 20;
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// BYTES (8 or 16) asynchronous copy global -> shared; `valid` false writes zeros and reads nothing.  past_l1: a 16-byte
// copy of data read once from device memory goes past the L1 (less work for its data path: 1.4 us of the 47 us of a scan);
// data read over the host link must go through it, where the 16-byte pieces of a row are gathered into 128-byte requests
// (past it the same scan takes 2.9 ms instead of 1.25 ms).
template <int BYTES>
__device__ __forceinline__ void fathom_copy_async(void* dst, const void* src, bool valid, bool past_l1 = false) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  const int bytes = valid ? BYTES : 0;
  if (BYTES == 16 && past_l1)
    asm volatile("cp.async.cg.shared.global [%0], [%1], %2, %3;" ::"r"(d), "l"(src), "n"(BYTES), "r"(bytes) : "memory");
  else
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;" ::"r"(d), "l"(src), "n"(BYTES), "r"(bytes) : "memory");
}
__device__ __forceinline__ void fathom_copies_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void fathom_copies_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

// CTAs per plan of a scan launch: planes in device memory - as many CTAs as are resident at once (ctas_per_sm per SM,
// and no more than there are tiles), each walking several tiles; planes read over the host link - one CTA per tile, so
// that CTAs become resident in block order and the link sees a few long sequential streams.  A positive
// fathom_scan_ctas_override() (set through fathom_scan_set_ctas_per_plan) replaces both.
int fathom_scan_grid_ctas(long long tiles, int plans, bool host_planes, int ctas_per_sm);
int fathom_scan_ctas_override();
bool fathom_planes_in_host_memory(const void* planes);

// The legacy kernel (scan_simt.cu).  mode 0: all scores written; 1: sampled tiles, compact; 2: candidates above a threshold.
int fathom_scan_simt_dispatch(int mode, const ScanBatch& B, int Hkv, int Hq, int heads_per_plan, const fathom_scan_fuse& fz,
                              bool dependent, cudaStream_t st);
