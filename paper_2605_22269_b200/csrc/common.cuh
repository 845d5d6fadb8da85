// Shared device helpers of the MuKV kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/mukv.h"

namespace mukv {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// ---------------------------------------------------------------- element access
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <typename T> struct ElemTraits;
template <> struct ElemTraits<__nv_bfloat16> {
  static constexpr int kPerWord = 2;      // elements in one 32-bit word
  static constexpr int kPad = 2;          // row padding (elements) that makes the word stride odd
};
template <> struct ElemTraits<float> {
  static constexpr int kPerWord = 1;
  static constexpr int kPad = 1;
};

template <typename T> __device__ __forceinline__ float elem_to_float(T x);
template <> __device__ __forceinline__ float elem_to_float<float>(float x) { return x; }
template <> __device__ __forceinline__ float elem_to_float<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}

// acc += q.k over the elements packed in one 32-bit word
template <typename T, typename A> __device__ __forceinline__ A dot_word(uint32_t q, uint32_t k, A acc);
template <> __device__ __forceinline__ float dot_word<__nv_bfloat16, float>(uint32_t q, uint32_t k, float acc) {
  acc = fmaf(bf16_lo(q), bf16_lo(k), acc);
  return fmaf(bf16_hi(q), bf16_hi(k), acc);
}
template <> __device__ __forceinline__ double dot_word<__nv_bfloat16, double>(uint32_t q, uint32_t k, double acc) {
  acc = fma((double)bf16_lo(q), (double)bf16_lo(k), acc);
  return fma((double)bf16_hi(q), (double)bf16_hi(k), acc);
}
template <> __device__ __forceinline__ float dot_word<float, float>(uint32_t q, uint32_t k, float acc) {
  return fmaf(__uint_as_float(q), __uint_as_float(k), acc);
}
template <> __device__ __forceinline__ double dot_word<float, double>(uint32_t q, uint32_t k, double acc) {
  return fma((double)__uint_as_float(q), (double)__uint_as_float(k), acc);
}

// ---------------------------------------------------------------- math in the accumulation type
__device__ __forceinline__ float exp_acc(float x) { return expf(x); }
__device__ __forceinline__ double exp_acc(double x) { return exp(x); }
__device__ __forceinline__ float fma_acc(float a, float b, float c) { return fmaf(a, b, c); }
__device__ __forceinline__ double fma_acc(double a, double b, double c) { return fma(a, b, c); }
__device__ __forceinline__ float sqrt_acc(float x) { return sqrtf(x); }
__device__ __forceinline__ double sqrt_acc(double x) { return sqrt(x); }
template <typename A> __device__ __forceinline__ A neg_inf();
template <> __device__ __forceinline__ float neg_inf<float>() { return -INFINITY; }
template <> __device__ __forceinline__ double neg_inf<double>() { return -(double)INFINITY; }

// ---------------------------------------------------------------- warp / block reductions
template <typename A> __device__ __forceinline__ A warp_sum(A v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}
template <typename A> __device__ __forceinline__ A warp_max(A v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    A u = __shfl_xor_sync(kFull, v, o);
    v = u > v ? u : v;
  }
  return v;
}
template <typename A> __device__ __forceinline__ A warp_min(A v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    A u = __shfl_xor_sync(kFull, v, o);
    v = u < v ? u : v;
  }
  return v;
}

// A set of threads that synchronise together: the whole block, or a fixed sub-range of its
// threads on a named barrier (warp-specialised kernels, where other warps never join).
struct BlockGroup {
  __device__ __forceinline__ static int tid() { return threadIdx.x; }
  __device__ __forceinline__ static int size() { return blockDim.x; }
  __device__ __forceinline__ static void sync() { __syncthreads(); }
};
template <int ID, int NT, int OFF> struct NamedGroup {
  __device__ __forceinline__ static int tid() { return (int)threadIdx.x - OFF; }
  __device__ __forceinline__ static int size() { return NT; }
  __device__ __forceinline__ static void sync() { asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(NT) : "memory"); }
};

// Exclusive prefix count of `flag` over the group in thread order, plus the group total.
// scratch: at least (size/32 + 1) ints of shared memory.  Contains two barriers.
template <class Grp>
__device__ __forceinline__ int group_excl_count(bool flag, int* scratch, int& total) {
  const int t = Grp::tid();
  const int lane = t & 31, warp = t >> 5, nwarp = (Grp::size() + 31) >> 5;
  const unsigned b = __ballot_sync(kFull, flag);
  const int in_warp = __popc(b & ((1u << lane) - 1u));
  Grp::sync();                           // scratch may still be read from a previous call
  if (lane == 0) scratch[warp] = __popc(b);
  Grp::sync();
  int before = 0, sum = 0;
  for (int w = 0; w < nwarp; ++w) {
    const int c = scratch[w];
    if (w < warp) before += c;
    sum += c;
  }
  total = sum;
  return before + in_warp;
}
__device__ __forceinline__ int block_excl_count(bool flag, int* scratch, int& total) {
  return group_excl_count<BlockGroup>(flag, scratch, total);
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialisation attribute may
// start while its predecessor in the stream still runs; pdl_wait() returns once that predecessor
// has completed and its writes are visible (a no-op for a normally launched kernel), pdl_trigger()
// tells the runtime that this block no longer minds the successor being scheduled.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// super patch (row-major, split x split) of token id j in a frame of P tokens laid out as a grid
// with grid_width tokens per row: rectangles of ceil(rows/split) x ceil(grid_width/split) tokens
__device__ __forceinline__ int super_patch_index(int j, int P, int grid_width, int split) {
  const int rows = P / grid_width;
  const int rh = (rows + split - 1) / split, cw = (grid_width + split - 1) / split;
  return (j / grid_width) / rh * split + (j % grid_width) / cw;
}

// owner of item i when n items are split into contiguous shares [c*n/nb, (c+1)*n/nb) (the blocks of
// the persistent scoring kernel take such shares of its item list)
__device__ __forceinline__ int share_owner(unsigned i, unsigned n, unsigned nb) { return (int)(((i + 1u) * nb - 1u) / n); }

// ---------------------------------------------------------------- segment entries (Eq. 5 at segment level)
// What the pooling of segment entries needs, small enough to travel in registers (compact_segment_plane
// is kept out of line so that its 32 loads in flight do not set the register count of the kernels that
// call it; a reference to a kernel's parameter block would force a per-thread copy of the block instead).
struct SegmentArgs {
  int L, kappa, C, fseg, n_frames;
  long long first_frame;
  const float* frame_entry;
  const double* frame_ksum;
  float* seg_entry;
  float* seg_key;
  const int* kept_count;          // [max_frames] tokens kept per frame, or null: kappa in every frame
};

// 16-byte streaming copies
__device__ __forceinline__ uint4 ld_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(void* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

}  // namespace mukv
