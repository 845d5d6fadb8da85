// KV compaction into the paged store and block pooling (Sec. 3.3 "selected KV slices ... are
// stored", Sec. 3.4 Eq. 5).
//
// compact_kernel<T>: one thread block per (layer, K|V, frame).  The kappa kept rows of that
// plane (C = Hkv*D elements each, one contiguous run in the input) are copied, in ascending
// token order, to the frame's page; the same registers feed the mean over the kept rows.
// The last-layer key plane is summed in double: its mean is the retrieval key (Eq. 5) that
// later ranks blocks, so it is kept free of accumulation-order noise.
// segment_kernel: refreshes every segment entry the chunk touches: mean over the frames present.
#pragma once
#include "common.cuh"

namespace mukv {

constexpr int kCompactThreads = 256;

struct CompactParams {
  int L, kappa, C, P;             // C = Hkv*D elements per row
  int n_frames;
  long long first_frame;
  const void* k;                  // [L][n][P][C]
  const void* v;
  const int* kept_store;          // [max_frames][kappa]
  unsigned char* store;           // store base
  const long long* page_table;    // [max_frames] byte offsets
  float* frame_entry;             // [max_frames][L][2][C]
  float* frame_key;               // [max_frames][C]
  double* frame_ksum;             // [max_frames][C]  exact sums of the last-layer kept keys
  int* n_flagged;                 // reset here for the next chunk
  long long* stat_refined;        // device counter
  // segment entries (Eq. 5 at segment level)
  int fseg;                       // frames per segment
  float* seg_entry;               // [max_segs][L][2][C]
  float* seg_key;                 // [max_segs][C]
};

// Segment entries (Eq. 5 at segment level) of one (layer, K|V) plane for every segment the chunk
// touches: mean over the frames present.  Run by one whole block.
__device__ inline void compact_segment_plane(const CompactParams& p, int l, int kv) {
  const int tid = threadIdx.x;
  const int C = p.C, kappa = p.kappa;
  const bool exact = (l == p.L - 1) && (kv == 0);
  const long long frames_total = p.first_frame + p.n_frames;
  const long long first_seg = p.first_frame / p.fseg, last_seg = (frames_total - 1) / p.fseg;
  for (long long u = first_seg; u <= last_seg; ++u) {
    const long long t0 = u * p.fseg;
    long long t1 = t0 + p.fseg;
    if (t1 > frames_total) t1 = frames_total;
    const int nf = (int)(t1 - t0);
    for (int col = tid; col < C; col += kCompactThreads) {
      float m;
      // eight loads in flight at a time, added in frame order
      if (exact) {
        double t = 0.0;
        for (long long ff = t0; ff < t1; ff += 8) {
          double x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) x[i] = ff + i < t1 ? __ldcg(p.frame_ksum + (ff + i) * C + col) : 0.0;
#pragma unroll
          for (int i = 0; i < 8; ++i) t += x[i];
        }
        m = (float)(t / ((double)nf * (double)kappa));
        p.seg_key[u * C + col] = m;
      } else {
        float t = 0.f;
        for (long long ff = t0; ff < t1; ff += 8) {
          float x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)
            x[i] = ff + i < t1 ? __ldcg(p.frame_entry + (((ff + i) * p.L + l) * 2 + kv) * C + col) : 0.f;
#pragma unroll
          for (int i = 0; i < 8; ++i) t += x[i];
        }
        m = t / (float)nf;
      }
      p.seg_entry[((u * p.L + l) * 2 + kv) * C + col] = m;
    }
  }
}

// NV = 16-byte vectors per row; the block covers 256/NV rows per pass.
template <typename T>
__global__ void __launch_bounds__(kCompactThreads) compact_kernel(const CompactParams p) {
  constexpr int VE = 16 / sizeof(T);
  __shared__ float s_red[kCompactThreads * VE];
  __shared__ double s_red64[kCompactThreads * VE];
  __shared__ int s_kept[MUKV_MAX_TOKENS];
  const int tid = threadIdx.x;
  const int plane = blockIdx.x;                 // l*2 + kv
  const int l = plane >> 1, kv = plane & 1;
  const int f = blockIdx.y;
  const long long f_abs = p.first_frame + f;
  pdl_wait();
  pdl_trigger();
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) {
    *p.stat_refined += *p.n_flagged;
    *p.n_flagged = 0;
  }
  const int kappa = p.kappa, C = p.C;
  const int NV = C / VE;                        // vectors per row (power of two, <= 256)
  const int rows_per_pass = kCompactThreads / NV;
  for (int r = tid; r < kappa; r += kCompactThreads) s_kept[r] = p.kept_store[f_abs * kappa + r];
  __syncthreads();
  const T* src_base = reinterpret_cast<const T*>(kv ? p.v : p.k) + ((long long)l * p.n_frames + f) * p.P * C;
  unsigned char* page = p.store + p.page_table[f_abs];
  T* dst_base = reinterpret_cast<T*>(page) + (long long)plane * kappa * C;
  const int c = tid % NV, r0 = tid / NV;
  const bool exact = (l == p.L - 1) && (kv == 0);
  float acc[VE];
  double acc64[VE];
#pragma unroll
  for (int e = 0; e < VE; ++e) { acc[e] = 0.f; acc64[e] = 0.0; }
  constexpr int kUnroll = 4;
  for (int r = r0; r < kappa; r += rows_per_pass * kUnroll) {
    uint4 x[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int rr = r + u * rows_per_pass;
      if (rr < kappa) x[u] = ld_stream(src_base + (long long)s_kept[rr] * C + c * VE);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int rr = r + u * rows_per_pass;
      if (rr < kappa) {
        st_stream(dst_base + (long long)rr * C + c * VE, x[u]);
        const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
        float e[VE];
        if constexpr (sizeof(T) == 2) {
#pragma unroll
          for (int i = 0; i < 4; ++i) { e[(2 * i) % VE] = bf16_lo(w[i]); e[(2 * i + 1) % VE] = bf16_hi(w[i]); }
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) e[i % VE] = __uint_as_float(w[i]);
        }
        if (exact) {
#pragma unroll
          for (int i = 0; i < VE; ++i) acc64[i] += (double)e[i];
        } else {
#pragma unroll
          for (int i = 0; i < VE; ++i) acc[i] += e[i];
        }
      }
    }
  }
  // reduce the row groups (fixed order) and write the mean
  if (exact) {
#pragma unroll
    for (int i = 0; i < VE; ++i) s_red64[tid * VE + i] = acc64[i];
  } else {
#pragma unroll
    for (int i = 0; i < VE; ++i) s_red[tid * VE + i] = acc[i];
  }
  __syncthreads();
  float* fe = p.frame_entry + ((f_abs * p.L + l) * 2 + kv) * C;
  for (int col = tid; col < C; col += kCompactThreads) {
    const int cv = col / VE, ce = col % VE;
    if (exact) {
      double t = 0.0;
      for (int g = 0; g < rows_per_pass; ++g) t += s_red64[(g * NV + cv) * VE + ce];
      p.frame_ksum[f_abs * C + col] = t;
      const float m = (float)(t / (double)kappa);
      fe[col] = m;
      p.frame_key[f_abs * C + col] = m;
    } else {
      float t = 0.f;
      for (int g = 0; g < rows_per_pass; ++g) t += s_red[(g * NV + cv) * VE + ce];
      fe[col] = t / (float)kappa;
    }
  }
}

// segment_kernel: one block per (layer, K|V) plane; refreshes that plane of every segment entry the
// chunk touches.  Launched right after compact_kernel (programmatic dependent launch).
__global__ void __launch_bounds__(kCompactThreads) segment_kernel(const CompactParams p) {
  pdl_wait();
  compact_segment_plane(p, blockIdx.x >> 1, blockIdx.x & 1);
}

}  // namespace mukv
