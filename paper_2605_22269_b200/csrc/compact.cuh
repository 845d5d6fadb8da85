// KV compaction into the paged store and block pooling (Sec. 3.3 "selected KV slices ... are
// stored", Sec. 3.4 Eq. 5).
//
// compact_kernel<T>: one thread block per (layer, K|V, frame).  The kappa kept rows of that
// plane (C = Hkv*D elements each, one contiguous run in the input) are copied, in ascending
// token order, to the frame's page; the same registers feed the mean over the kept rows.
// The last-layer key plane is summed in double: its mean is the retrieval key (Eq. 5) that
// later ranks blocks, so it is kept free of accumulation-order noise.
// The block that finishes a (layer, K|V) plane of the chunk last (arrival counter, nobody waits)
// refreshes that plane of every segment entry the chunk touches: mean over the frames present.
#pragma once
#include "common.cuh"
#include "tc.cuh"

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
  int* plane_counter;             // [L*2] arrivals per plane, zero between launches
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

  // ---- segment entries of this plane, by the block that completes the plane
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int old = atomicAdd(p.plane_counter + plane, 1);
    s_last = (old == p.n_frames - 1);
    if (s_last) p.plane_counter[plane] = 0;            // ready for the next launch
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  compact_segment_plane(p, l, kv);
}

// compact_stream_kernel<T>: the same work as a persistent, pipelined stream through the bulk-copy
// engine.  One block per SM walks its share of the (layer, K|V, frame) planes.  The kappa kept rows
// of a plane are fetched with one bulk copy each into one of `n_buf` shared-memory buffers, leave as
// ONE contiguous bulk store into the frame's page, and are summed for the pooled entry out of shared
// memory meanwhile; the rows of the next planes are already in flight.  Used when at least two
// planes fit in shared memory.
constexpr int kStreamScratchBytes = 8192;        // cross-group partial sums
constexpr int kStreamMaxBufs = 4;
constexpr int kStreamMaxItems = 64;              // planes per block
constexpr int kStreamSmemLimit = 226 * 1024;     // dynamic shared memory (the kernel also has a little static)

struct StreamShape {
  int n_buf;                                     // 0: does not fit
  int grid;
  size_t smem;
};

__host__ inline StreamShape compact_stream_shape(int kappa, int C, int esize, int n_planes, int n_sms, size_t limit) {
  StreamShape sh;
  sh.n_buf = 0; sh.grid = 0; sh.smem = 0;
  const size_t rows = ((size_t)kappa * C * esize + 127) / 128 * 128;
  int grid = n_sms < n_planes ? n_sms : n_planes;
  if (grid < 1) grid = 1;
  const int per_block = (n_planes + grid - 1) / grid;
  if (per_block > kStreamMaxItems) return sh;
  const size_t fixed = kStreamScratchBytes + (size_t)per_block * kappa * sizeof(int) + 256 + 128;
  for (int nb = kStreamMaxBufs; nb >= 2; --nb) {
    if (nb * rows + fixed <= limit) { sh.n_buf = nb; sh.grid = grid; sh.smem = nb * rows + fixed; return sh; }
  }
  return sh;
}

template <typename T>
__global__ void __launch_bounds__(kCompactThreads, 1) compact_stream_kernel(const CompactParams p, int n_buf,
                                                                           int* status) {
  constexpr int VE = 16 / sizeof(T);
  extern __shared__ unsigned char smem_raw[];
  __shared__ int s_done[kStreamMaxItems];           // planes whose last frame this block finished
  __shared__ int s_ndone;
  const uint32_t raw = tc::smem_u32(smem_raw);
  const uint32_t base = (raw + 127u) & ~127u;
  unsigned char* sm = smem_raw + (base - raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kappa = p.kappa, C = p.C;
  const int n_planes = p.L * 2 * p.n_frames;
  const uint32_t row_bytes = (uint32_t)C * sizeof(T);
  const uint32_t rows_bytes = ((uint32_t)kappa * row_bytes + 127u) / 128u * 128u;
  const int n_my = (n_planes - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // items b, b+grid, ...
  unsigned char* s_scratch = sm + (size_t)n_buf * rows_bytes;
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(s_scratch + kStreamScratchBytes);        // [kStreamMaxBufs]
  int* s_kept = reinterpret_cast<int*>(s_scratch + kStreamScratchBytes + 256);           // [n_my][kappa]
  pdl_wait();
  if (blockIdx.x == 0 && tid == 0) {
    *p.stat_refined += *p.n_flagged;
    *p.n_flagged = 0;
  }
  if (tid == 0) {
    for (int b = 0; b < kStreamMaxBufs; ++b) tc::mbar_init(tc::smem_u32(&s_bar[b]), 1);
    tc::fence_mbar_init();
    s_ndone = 0;
  }
  // item k of this block is plane (blockIdx.x + k*gridDim.x): frame-major, so neighbouring blocks
  // work on the same frame
  for (int i = tid; i < n_my * kappa; i += kCompactThreads) {
    const int k = i / kappa, r = i % kappa;
    const int item = blockIdx.x + k * gridDim.x;
    const int f = item / (p.L * 2);
    s_kept[i] = p.kept_store[(p.first_frame + f) * kappa + r];
  }
  __syncthreads();

  // warp 0 issues the row copies of item k into buffer k % n_buf
  auto issue_loads = [&](int k) {
    const int item = blockIdx.x + k * gridDim.x;
    const int f = item / (p.L * 2), plane = item % (p.L * 2);
    const int l = plane >> 1, kv = plane & 1;
    const uint32_t bar = tc::smem_u32(&s_bar[k % n_buf]);
    const uint32_t dst = base + (uint32_t)(k % n_buf) * rows_bytes;
    const unsigned char* src_base = reinterpret_cast<const unsigned char*>(kv ? p.v : p.k) +
                                    ((long long)l * p.n_frames + f) * p.P * (long long)row_bytes;
    if (lane == 0) tc::mbar_expect_tx(bar, (uint32_t)kappa * row_bytes);
    __syncwarp();
    for (int r = lane; r < kappa; r += 32)
      tc::bulk_load(dst + (uint32_t)r * row_bytes, src_base + (long long)s_kept[k * kappa + r] * row_bytes, row_bytes, bar);
  };
  if (warp == 0)
    for (int k = 0; k < n_buf && k < n_my; ++k) issue_loads(k);

  const int NV = C / VE;                        // 16-byte vectors per row (power of two, <= 256)
  const int rows_per_pass = kCompactThreads / NV;
  const int c = tid % NV, r0 = tid / NV;
  bool failed = false;
  int pend_plane = -1, pend_old = 0;            // arrival of the previous item, looked at one item later
  for (int k = 0; k < n_my; ++k) {
    const int item = blockIdx.x + k * gridDim.x;
    const int f = item / (p.L * 2), plane = item % (p.L * 2);
    const int l = plane >> 1, kv = plane & 1;
    const long long f_abs = p.first_frame + f;
    const int b = k % n_buf;
    const uint32_t ph = (uint32_t)((k / n_buf) & 1);
    const bool landed = tc::mbar_wait(tc::smem_u32(&s_bar[b]), ph) || tc::mbar_wait(tc::smem_u32(&s_bar[b]), ph);
    if (__syncthreads_or(landed ? 0 : 1)) { failed = true; break; }
    const unsigned char* s_rows = sm + (size_t)b * rows_bytes;
    if (tid == 0)
      tc::bulk_store(p.store + p.page_table[f_abs] + (long long)plane * kappa * row_bytes,
                     base + (uint32_t)b * rows_bytes, (uint32_t)kappa * row_bytes);
    // ---- pooled entry out of shared memory: thread = (row group, 16-byte column)
    const bool exact = (l == p.L - 1) && (kv == 0);
    float acc[VE];
    double acc64[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) { acc[e] = 0.f; acc64[e] = 0.0; }
    for (int r = r0; r < kappa; r += rows_per_pass) {
      const uint4 x = *reinterpret_cast<const uint4*>(s_rows + (size_t)r * row_bytes + (size_t)c * 16);
      const uint32_t w[4] = {x.x, x.y, x.z, x.w};
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
    float* fe = p.frame_entry + ((f_abs * p.L + l) * 2 + kv) * C;
    if (!exact) {
      float* s_red = reinterpret_cast<float*>(s_scratch);           // [256 threads][VE] <= 8 KB
#pragma unroll
      for (int i = 0; i < VE; ++i) s_red[tid * VE + i] = acc[i];
      __syncthreads();
      for (int col = tid; col < C; col += kCompactThreads) {
        const int cv = col / VE, ce = col % VE;
        float t = 0.f;
        for (int g = 0; g < rows_per_pass; ++g) t += s_red[(g * NV + cv) * VE + ce];
        fe[col] = t / (float)kappa;
      }
    } else {
      // the last-layer keys are summed in double (their mean ranks blocks later); the scratch holds
      // half of the threads' partial sums at a time
      double* s_red64 = reinterpret_cast<double*>(s_scratch);       // [128 threads][VE] <= 8 KB
      for (int half = 0; half < 2; ++half) {
        if ((tid & 1) == half) {
#pragma unroll
          for (int i = 0; i < VE; ++i) s_red64[(tid >> 1) * VE + i] = acc64[i];
        }
        __syncthreads();
        // thread t = g*NV + cv wrote slot t>>1 when (t & 1) == half: columns with (cv & 1) == half
        for (int col = tid; col < C; col += kCompactThreads) {
          const int cv = col / VE, ce = col % VE;
          if ((cv & 1) != half) continue;
          double t = 0.0;
          for (int g = 0; g < rows_per_pass; ++g) t += s_red64[((g * NV + cv) >> 1) * VE + ce];
          p.frame_ksum[f_abs * C + col] = t;
          const float m = (float)(t / (double)kappa);
          fe[col] = m;
          p.frame_key[f_abs * C + col] = m;
        }
        __syncthreads();
      }
    }
    // ---- the plane's arrival counter (the result is looked at during the next item)
    __threadfence();
    __syncthreads();                            // every thread has read the buffer and written its entries
    if (tid == 0) {
      if (pend_plane >= 0 && pend_old == p.n_frames - 1) s_done[s_ndone++] = pend_plane;
      pend_old = atomicAdd(p.plane_counter + plane, 1);
      pend_plane = plane;
      // refill the buffer once the store has read it
      tc::bulk_store_wait_read();
    }
    if (k + n_buf < n_my) {
      __syncthreads();                          // thread 0 has seen the store leave shared memory
      if (warp == 0) issue_loads(k + n_buf);
    }
  }
  if (tid == 0) {
    if (failed) atomicCAS(status, 0, 6);
    if (pend_plane >= 0 && pend_old == p.n_frames - 1) s_done[s_ndone++] = pend_plane;
    tc::bulk_store_wait_read();
  }
  __syncthreads();
  // ---- segment entries of the planes this block completed
  const int nd = s_ndone;
  if (nd > 0) __threadfence();
  for (int i = 0; i < nd; ++i) {
    const int plane = s_done[i];
    if (tid == 0) p.plane_counter[plane] = 0;          // ready for the next launch
    compact_segment_plane(p, plane >> 1, plane & 1);
  }
}

}  // namespace mukv
