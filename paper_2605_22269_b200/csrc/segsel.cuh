// Segment-level dual-signal selection (Sec. 3.3: the indicator "I_v in R^O" of a whole segment and
// its budget kappa_v = floor(rho_v * O)).
//
// The indicators of every frame are computed as for frame-level selection (attention inside the
// frame); segsel_kernel then normalises both signals over all O = F * P tokens of a segment (Eq. 4),
// keeps the kappa_v best of them and splits the result by frame: a frame keeps a variable number of
// tokens, its page has that many rows, and the pages of a segment lie one behind the other in the
// segment's share of the page region.  One block per segment of the chunk.
// Two sources of the indicators:
//   src32 = 0  the double-precision partial sums of score_kernel; everything in double precision,
//              the ranking by the radix select of the retrieval kernels (block_topk_set);
//   src32 = 1  the single-precision partial sums of the persistent tensor-core kernel; Eq. 4 and the
//              ranking in single precision (segment_select32: the scheme of the frame-level selection,
//              a 256-bin histogram and an exact rank inside the bin of the kappa_v-th score).  The
//              ranking then stands only when the lowest kept and the highest dropped score are further
//              apart than tie_eps + flag_margin and neither signal is flat (the rule of the
//              frame-level selection); otherwise the kernel writes nothing but the segment's word in
//              seg_flag, and the double-precision pass that follows (score_kernel gated by that word,
//              then this kernel with src32 = 0 and only_flagged = 1) redoes the segment.
#pragma once
#include "common.cuh"
#include "retrieve.cuh"
#include "score.cuh"

namespace mukv {

constexpr int kSegSelThreads = 1024;
constexpr int kSegSelWarps = kSegSelThreads / 32;
constexpr int kSegSelMaxTokens = 4096;        // F * P of one segment
constexpr int kSegSelList = 512;              // scores of one histogram bin that are ranked directly
static_assert(kSegSelMaxTokens <= 4 * kSegSelThreads, "a thread emits at most four consecutive tokens");

struct SegSelParams {
  ScoreParams sp;               // partial sums of the scoring kernel, Eq. 4 parameters, outputs
  int fseg;                     // frames per segment
  int kappa_v;                  // tokens kept in a full segment
  long long token_bytes;        // bytes one kept token takes in a page: 2 * L * C * sizeof(element)
  int* kept_count;              // [max_frames]
  int src32;                    // see the head of this file
  int only_flagged;             // 1: segments whose seg_flag word is 0 are left alone
  int* seg_flag;                // [segments of the chunk]; written with src32 = 1, read with only_flagged
  int ps_grid, ps_items, ps_ipf;  // the persistent scoring launch: blocks, items, items per frame (src32 = 1)
  unsigned long long* stat_refined;  // frames ranked by the gated double-precision pass are added here
  // Blocks n_seg, n_seg + 1, ... of the grid (one per (layer, K|V) plane, present when prev.n_frames > 0)
  // pool the segment entries the previous call left to this one, on SMs this kernel leaves idle
  int n_seg;
  SegmentArgs prev;
};

__host__ inline size_t segsel_smem_bytes(int tokens) {
  return (size_t)tokens * (2 * sizeof(double) + sizeof(int)) + 64 * sizeof(int);
}

struct SegSel32Scratch {
  unsigned mm[kSegSelWarps][4];   // per-warp min / max keys of the two signals
  unsigned ab[kSegSelWarps][2];   // per-warp lowest kept / highest dropped key
  int warp_tot[kSegSelWarps];
  int hist[256];
  int list[kSegSelList];
  int bin, rank, n_list;
  float tau;
};

// Exclusive prefix of v over the block in thread order, and the block total.  Two barriers.
__device__ __forceinline__ int segsel_scan_excl(int v, int* warp_tot, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int u = __shfl_up_sync(kFull, incl, o);
    if (lane >= o) incl += u;
  }
  __syncthreads();                                       // warp_tot may still be read from a previous call
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  const int wt = lane < kSegSelWarps ? warp_tot[lane] : 0;
  total = warp_sum(wt);
  return warp_sum(lane < warp ? wt : 0) + incl - v;
}

// The single-precision selection of one segment (src32 = 1).  Fills oi with the kept tokens in
// ascending order and returns their number, or -1 when single precision cannot decide the segment
// (the segment's word in seg_flag is then 1, else 0).  att / fft / s32: [O] floats of scratch.
__device__ inline int segment_select32(const SegSelParams& p, int f0, int O, int k, float* att, float* fft,
                                       float* s32, int* oi, SegSel32Scratch* sc) {
  const ScoreParams& sp = p.sp;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = sp.P, HkvV = sp.Ls * sp.Hkv;
  // ---- the indicators, from the scoring blocks' column sums (added in block order)
  const float na = 1.f / (float)((long long)sp.Ls * sp.Hq * P), nf = 1.f / (float)((long long)HkvV * sp.D);
  unsigned k0 = 0xffffffffu, k1 = 0u, k2 = 0xffffffffu, k3 = 0u;
  bool bad = false;
  // (with P a multiple of four a thread takes four neighbouring tokens of a frame with 16-byte loads, so that
  // one trip covers a 16-frame segment: the loads of this one block are what the kernel spends most time on)
  const bool vec4 = (P & 3) == 0;
  for (int i = tid * 4; vec4 && i < O; i += 4 * kSegSelThreads) {
    const int f = f0 + i / P, j = i % P;
    const int c_first = share_owner((unsigned)(f * p.ps_ipf), (unsigned)p.ps_items, (unsigned)p.ps_grid);
    const int c_last = share_owner((unsigned)((f + 1) * p.ps_ipf - 1), (unsigned)p.ps_items, (unsigned)p.ps_grid);
    const float* cp = reinterpret_cast<const float*>(sp.colsum_part) + j;
    const float* fp = reinterpret_cast<const float*>(sp.ifft_part) + (long long)f * HkvV * P + j;
    float4 a4 = make_float4(0.f, 0.f, 0.f, 0.f), f4 = a4;
    for (int c0 = c_first; c0 <= c_last; c0 += 8) {
      float4 x[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        x[u] = c0 + u <= c_last ? __ldcg(reinterpret_cast<const float4*>(cp + (long long)(c0 + u + f) * P))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 8; ++u) { a4.x += x[u].x; a4.y += x[u].y; a4.z += x[u].z; a4.w += x[u].w; }
    }
    for (int g0 = 0; g0 < HkvV; g0 += 8) {
      float4 y[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        y[u] = g0 + u < HkvV ? __ldcg(reinterpret_cast<const float4*>(fp + (long long)(g0 + u) * P))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 8; ++u) { f4.x += y[u].x; f4.y += y[u].y; f4.z += y[u].z; f4.w += y[u].w; }
    }
    const float av[4] = {a4.x * na, a4.y * na, a4.z * na, a4.w * na};
    const float bv[4] = {f4.x * nf, f4.y * nf, f4.z * nf, f4.w * nf};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      att[i + e] = av[e];
      fft[i + e] = bv[e];
      bad |= !(isfinite(av[e]) && isfinite(bv[e]));
      const unsigned ka = __float_as_uint(av[e]), kf = __float_as_uint(bv[e]);
      k0 = min(k0, ka); k1 = max(k1, ka); k2 = min(k2, kf); k3 = max(k3, kf);
    }
  }
  for (int i = tid; !vec4 && i < O; i += kSegSelThreads) {
    const int f = f0 + i / P, j = i % P;
    const int c_first = share_owner((unsigned)(f * p.ps_ipf), (unsigned)p.ps_items, (unsigned)p.ps_grid);
    const int c_last = share_owner((unsigned)((f + 1) * p.ps_ipf - 1), (unsigned)p.ps_items, (unsigned)p.ps_grid);
    const float* cp = reinterpret_cast<const float*>(sp.colsum_part) + j;
    const float* fp = reinterpret_cast<const float*>(sp.ifft_part) + (long long)f * HkvV * P + j;
    // all loads of the common case (up to 16 blocks per frame, up to 8 key heads) are in flight together
    float x[16], y[8];
#pragma unroll
    for (int u = 0; u < 16; ++u) x[u] = c_first + u <= c_last ? __ldcg(cp + (long long)(c_first + u + f) * P) : 0.f;
#pragma unroll
    for (int u = 0; u < 8; ++u) y[u] = u < HkvV ? __ldcg(fp + (long long)u * P) : 0.f;
    float a32 = 0.f, f32 = 0.f;
#pragma unroll
    for (int u = 0; u < 16; ++u) a32 += x[u];
#pragma unroll
    for (int u = 0; u < 8; ++u) f32 += y[u];
    for (int cc = c_first + 16; cc <= c_last; ++cc) a32 += __ldcg(cp + (long long)(cc + f) * P);
    for (int gg = 8; gg < HkvV; ++gg) f32 += __ldcg(fp + (long long)gg * P);
    const float a = a32 * na, b = f32 * nf;
    att[i] = a;
    fft[i] = b;
    bad |= !(isfinite(a) && isfinite(b));
    // both signals are sums of non-negative terms: their bit patterns order like the values
    const unsigned ka = __float_as_uint(a), kf = __float_as_uint(b);
    k0 = min(k0, ka); k1 = max(k1, ka); k2 = min(k2, kf); k3 = max(k3, kf);
  }
  k0 = __reduce_min_sync(kFull, k0); k1 = __reduce_max_sync(kFull, k1);
  k2 = __reduce_min_sync(kFull, k2); k3 = __reduce_max_sync(kFull, k3);
  if (lane == 0) { sc->mm[warp][0] = k0; sc->mm[warp][1] = k1; sc->mm[warp][2] = k2; sc->mm[warp][3] = k3; }
  if (tid < 256) sc->hist[tid] = 0;
  if (tid == 0) sc->n_list = 0;
  const bool any_bad = __syncthreads_or(bad) != 0;
  const float amin = __uint_as_float(__reduce_min_sync(kFull, sc->mm[lane][0]));
  const float amax = __uint_as_float(__reduce_max_sync(kFull, sc->mm[lane][1]));
  const float fmin_ = __uint_as_float(__reduce_min_sync(kFull, sc->mm[lane][2]));
  const float fmax_ = __uint_as_float(__reduce_max_sync(kFull, sc->mm[lane][3]));
  // ---- Eq. 4 (a segment with a score that is not a number has no ranking: every score counts as 0)
  const float inv_a = (amax == amin) ? 0.f : 1.f / (amax - amin);
  const float inv_f = (fmax_ == fmin_) ? 0.f : 1.f / (fmax_ - fmin_);
  const long long np = (long long)sp.n_frames * P;
  for (int i = tid; i < O; i += kSegSelThreads) {
    const float a = att[i], b = fft[i];
    const float an = (a - amin) * inv_a;
    float fn = (b - fmin_) * inv_f;
    if (sp.keep_low) fn = 1.f - fn;
    const float s = any_bad ? 0.f : sp.alpha * an + (1.f - sp.alpha) * fn;
    s32[i] = s;
    int bin = (int)(s * 256.f);
    bin = bin < 0 ? 0 : (bin > 255 ? 255 : bin);
    atomicAdd(&sc->hist[bin], 1);
    if (sp.scores_out) {
      const long long o = (long long)f0 * P + i;
      sp.scores_out[o] = a;
      sp.scores_out[np + o] = b;
      sp.scores_out[2 * np + o] = s;
    }
  }
  if (tid == 0 && any_bad && sp.status) atomicCAS(sp.status, 0, kStatusNonFinite);
  __syncthreads();
  // ---- tau = k-th largest score: the histogram finds its bin, the scores of that bin are ranked
  // among themselves
  bool overflow = false;
  float tau = 3.0e38f;                                     // k = 0: nothing is taken
  if (any_bad) {
    tau = 0.f;                                             // every score is 0: the k lowest ids are taken
  } else if (k >= O) {
    tau = -3.0e38f;                                        // everything is taken
  } else if (k > 0) {
    if (warp == 0) {
      int c[8], T = 0;                                     // lane l owns bins 8l .. 8l+7
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = sc->hist[8 * lane + i]; T += c[i]; }
      int incl = T;                                        // scores in this lane's bins and all higher ones
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_down_sync(kFull, incl, o);
        if (lane + o < 32) incl += v;
      }
      const int above = incl - T;
      if (above < k && k <= above + T) {                   // true for exactly one lane
        int r = k - above, b = 7;
        for (; b > 0; --b) {
          if (r <= c[b]) break;
          r -= c[b];
        }
        sc->bin = 8 * lane + b;
        sc->rank = r;
      }
    }
    __syncthreads();
    const int the_bin = sc->bin;
    for (int i = tid; i < O; i += kSegSelThreads) {
      const float s = s32[i];
      int bin = (int)(s * 256.f);
      bin = bin < 0 ? 0 : (bin > 255 ? 255 : bin);
      if (bin == the_bin) {
        const int at = atomicAdd(&sc->n_list, 1);
        if (at < kSegSelList) sc->list[at] = __float_as_int(s);
      }
    }
    __syncthreads();
    const int n = sc->n_list, r = sc->rank;
    overflow = n > kSegSelList;                            // a crowded bin: left to the double-precision pass
    if (!overflow && tid < n) {
      const int key = sc->list[tid];
      int gt = 0, ge = 0;
      for (int i = 0; i < n; ++i) {
        const int o = sc->list[i];
        gt += (o > key);
        ge += (o >= key);
      }
      if (gt < r && r <= ge) sc->tau = __int_as_float(key);   // every writer holds the same value
    }
    __syncthreads();
    tau = overflow ? 3.0e38f : sc->tau;
  }
  // ---- the tie band and the kept list in ascending order: a thread owns consecutive tokens
  const float delta = sp.tie_eps;
  const int per = (O + kSegSelThreads - 1) / kSegSelThreads;   // <= 4
  const int i0 = tid * per;
  bool sure[4], band[4];
  int n_sure_t = 0, n_band_t = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int i = i0 + e;
    const bool in = e < per && i < O;
    const float s = in ? s32[i] : 0.f;
    sure[e] = in && s > tau + delta;
    band[e] = in && !sure[e] && s >= tau - delta;
    n_sure_t += sure[e] ? 1 : 0;
    n_band_t += band[e] ? 1 : 0;
  }
  int total = 0;
  const int before = segsel_scan_excl(n_sure_t | (n_band_t << 16), sc->warp_tot, total);
  const int need = k - (total & 0xffff);
  int band_rank = before >> 16, n_keep_t = 0;
  bool keep[4];
  unsigned lo_kept = 0xffffffffu, hi_drop = 0u;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int i = i0 + e;
    const bool in = e < per && i < O;
    keep[e] = sure[e] || (band[e] && band_rank < need);
    band_rank += band[e] ? 1 : 0;
    n_keep_t += keep[e] ? 1 : 0;
    if (in) {
      const unsigned key = __float_as_uint(s32[i]);
      if (keep[e]) lo_kept = min(lo_kept, key);
      else hi_drop = max(hi_drop, key);
    }
  }
  int n_kept = 0;
  int pos = segsel_scan_excl(n_keep_t, sc->warp_tot, n_kept);
#pragma unroll
  for (int e = 0; e < 4; ++e)
    if (keep[e]) oi[pos++] = i0 + e;
  lo_kept = __reduce_min_sync(kFull, lo_kept);
  hi_drop = __reduce_max_sync(kFull, hi_drop);
  if (lane == 0) { sc->ab[warp][0] = lo_kept; sc->ab[warp][1] = hi_drop; }
  __syncthreads();
  const float a = __uint_as_float(__reduce_min_sync(kFull, sc->ab[lane][0]));
  const float b = __uint_as_float(__reduce_max_sync(kFull, sc->ab[lane][1]));
  // ---- does single precision decide this segment safely?  (see select_frame)
  bool risky = n_kept < O && n_kept > 0 && (a - b <= delta + sp.flag_margin);
  const float aabs = fmaxf(amax, -amin), fabs_ = fmaxf(fmax_, -fmin_);
  if (amax != amin && (amax - amin) < sp.flat_ratio * aabs && sp.alpha != 0.f) risky = true;
  if (fmax_ != fmin_ && (fmax_ - fmin_) < sp.flat_ratio * fabs_ && sp.alpha != 1.f) risky = true;
  if (overflow) risky = true;
  if (any_bad) risky = false;                              // double precision would not rank it either
  if (tid == 0) p.seg_flag[blockIdx.x] = risky ? 1 : 0;
  return risky ? -1 : n_kept;                              // (the same decision in every thread)
}

// Segment entries (Eq. 5 at segment level) of one (layer, K|V) plane for every segment that frames
// a.first_frame .. a.first_frame + a.n_frames - 1 touch: the same sums in the same frame order as
// compact_segment_plane, one channel per thread at a time, eight loads in flight.
__device__ inline void pool_plane_entries(const SegmentArgs& a, int plane) {
  const int C = a.C, l = plane >> 1, kv = plane & 1;
  const bool exact = (l == a.L - 1) && (kv == 0);
  const long long frames_total = a.first_frame + a.n_frames;
  const long long first_seg = a.first_frame / a.fseg, last_seg = (frames_total - 1) / a.fseg;
  const long long fstride = 2LL * a.L * C;                  // floats between the entries of two frames
  for (long long u = first_seg; u <= last_seg; ++u) {
    const long long t0 = u * a.fseg;
    const long long t1 = t0 + a.fseg < frames_total ? t0 + a.fseg : frames_total;
    const int nf = (int)(t1 - t0);
    for (int col = threadIdx.x; col < C; col += blockDim.x) {
      float* dst = a.seg_entry + ((u * a.L + l) * 2 + kv) * C + col;
      const float* src = a.frame_entry + ((t0 * a.L + l) * 2 + kv) * C + col;
      const double* srck = a.frame_ksum + t0 * C + col;
      double td = 0.0;
      float tf = 0.f;
      long long n_tok = 0;
      for (int i0 = 0; i0 < nf; i0 += 8) {
        int cn[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) cn[i] = (a.kept_count && i0 + i < nf) ? __ldcg(a.kept_count + t0 + i0 + i) : 0;
        if (exact) {
          double x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) x[i] = i0 + i < nf ? __ldcg(srck + (long long)(i0 + i) * C) : 0.0;
#pragma unroll
          for (int i = 0; i < 8; ++i) td += x[i];
        } else {
          float x[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) x[i] = i0 + i < nf ? __ldcg(src + (i0 + i) * fstride) : 0.f;
#pragma unroll
          for (int i = 0; i < 8; ++i) tf += a.kept_count ? (float)cn[i] * x[i] : x[i];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) n_tok += cn[i];
      }
      float m;
      if (a.kept_count)                                       // frames keep different numbers of tokens: count-weighted
        m = exact ? (n_tok ? (float)(td / (double)n_tok) : 0.f) : (n_tok ? tf / (float)n_tok : 0.f);
      else
        m = exact ? (float)(td / ((double)nf * (double)a.kappa)) : tf / (float)nf;
      if (exact) a.seg_key[u * C + col] = m;
      *dst = m;
    }
  }
}

__global__ void __launch_bounds__(kSegSelThreads) segsel_kernel(const SegSelParams p) {
  if (p.prev.n_frames > 0 && (int)blockIdx.x >= p.n_seg) {
    // nothing of this call is needed for the previous call's entries: no wait for the scoring kernel
    for (int plane = (int)blockIdx.x - p.n_seg; plane < 2 * p.prev.L; plane += (int)gridDim.x - p.n_seg)
      pool_plane_entries(p.prev, plane);
    return;
  }
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ RankScratch sc;
  __shared__ SegSel32Scratch sc32;
  __shared__ double s_red[kSegSelWarps][4];
  const ScoreParams& sp = p.sp;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = sp.P;
  const int f0 = blockIdx.x * p.fseg;                                     // first chunk frame of this segment
  const int m = min(p.fseg, sp.n_frames - f0);                            // frames of it that are present
  const int O = m * P;
  double* sa = reinterpret_cast<double*>(smem_raw);                       // [O] I_att, later the fused score
  double* sf = sa + O;                                                    // [O] I_fft
  int* oi = reinterpret_cast<int*>(sf + O);                               // [O] kept tokens, ascending
  int* s_start = oi + O;                                                  // [m + 1]
  pdl_wait();
  if (p.only_flagged && __ldcg(p.seg_flag + blockIdx.x) == 0) return;
  if (p.only_flagged && tid == 0) atomicAdd(p.stat_refined, (unsigned long long)m);
  // the kappa best of the segment (kappa_v scaled to the frames present)
  const int k = (int)(((long long)p.kappa_v * m) / p.fseg);
  int n_kept;
  if (p.src32) {
    float* att = reinterpret_cast<float*>(smem_raw);                      // three float arrays in front of oi
    n_kept = segment_select32(p, f0, O, k, att, att + O, att + 2 * O, oi, &sc32);
    if (n_kept < 0) return;                                               // left to the double-precision pass
    __syncthreads();
  } else {
    // ---- the indicators of every token of the segment, from the scoring kernel's partial sums
    const int HqV = sp.Ls * sp.Hq * sp.row_split, HkvV = sp.Ls * sp.Hkv;
    const double na = 1.0 / (double)((long long)sp.Ls * sp.Hq * P), nf = 1.0 / (double)((long long)HkvV * sp.D);
    const double big = 3.0e38;
    double v0 = big, v1 = -big, v2 = big, v3 = -big;
    bool bad = false;
    for (int i = tid; i < O; i += kSegSelThreads) {
      const int f = f0 + i / P, j = i % P;
      const double* cp = reinterpret_cast<const double*>(sp.colsum_part) + (long long)f * HqV * P + j;
      const double* fp = reinterpret_cast<const double*>(sp.ifft_part) + (long long)f * HkvV * P + j;
      double a = 0.0, b = 0.0;
      for (int hh = 0; hh < HqV; ++hh) a += __ldcg(cp + (long long)hh * P);
      for (int gg = 0; gg < HkvV; ++gg) b += __ldcg(fp + (long long)gg * P);
      a *= na;
      b *= nf;
      sa[i] = a;
      sf[i] = b;
      bad |= !(isfinite(a) && isfinite(b));
      v0 = a < v0 ? a : v0; v1 = a > v1 ? a : v1;
      v2 = b < v2 ? b : v2; v3 = b > v3 ? b : v3;
    }
    v0 = warp_min(v0); v1 = warp_max(v1); v2 = warp_min(v2); v3 = warp_max(v3);
    if (lane == 0) { s_red[warp][0] = v0; s_red[warp][1] = v1; s_red[warp][2] = v2; s_red[warp][3] = v3; }
    const bool any_bad = __syncthreads_or(bad) != 0;
    double amin = big, amax = -big, fmin_ = big, fmax_ = -big;
    for (int w = 0; w < kSegSelWarps; ++w) {
      amin = s_red[w][0] < amin ? s_red[w][0] : amin;
      amax = s_red[w][1] > amax ? s_red[w][1] : amax;
      fmin_ = s_red[w][2] < fmin_ ? s_red[w][2] : fmin_;
      fmax_ = s_red[w][3] > fmax_ ? s_red[w][3] : fmax_;
    }
    // ---- Eq. 4 over the segment (a segment with a score that is not a number has no ranking: all 0)
    const double alpha = (double)sp.alpha;
    const long long np = (long long)sp.n_frames * P;
    for (int i = tid; i < O; i += kSegSelThreads) {
      const double a = sa[i], b = sf[i];
      const double an = (amax == amin) ? 0.0 : (a - amin) / (amax - amin);
      double fn = (fmax_ == fmin_) ? 0.0 : (b - fmin_) / (fmax_ - fmin_);
      if (sp.keep_low) fn = 1.0 - fn;
      const double s = any_bad ? 0.0 : alpha * an + (1.0 - alpha) * fn;
      sa[i] = s;
      if (sp.scores_out) {
        const long long o = (long long)f0 * P + i;
        sp.scores_out[o] = (float)a;
        sp.scores_out[np + o] = (float)b;
        sp.scores_out[2 * np + o] = (float)s;
      }
    }
    if (tid == 0 && any_bad && sp.status) atomicCAS(sp.status, 0, kStatusNonFinite);
    __syncthreads();
    // ---- ascending
    const ArrScore score{sa};
    const AllMembers always;
    n_kept = block_topk_set(score, always, O, k, (double)sp.tie_eps, oi, (double*)nullptr, &sc);
    __syncthreads();
  }
  // first kept token of every frame: lower bound of f * P in the ascending list
  for (int f = tid; f <= m; f += kSegSelThreads) {
    int lo = 0, hi = n_kept;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (oi[mid] < f * P) lo = mid + 1; else hi = mid;
    }
    s_start[f] = lo;
  }
  __syncthreads();
  const long long t0 = sp.first_frame + f0;
  const long long seg = t0 / p.fseg;
  for (int f = tid; f < m; f += kSegSelThreads) {
    const long long t = t0 + f;
    p.kept_count[t] = s_start[f + 1] - s_start[f];
    sp.frame_ts[t] = t;
    sp.page_table[t] = sp.pages_off + (seg * p.kappa_v + s_start[f]) * p.token_bytes;
  }
  for (int i = tid; i < O; i += kSegSelThreads) {
    // slot r of frame f: its r-th kept token, -1 behind the last one
    const int f = i / P, r = i % P;
    const int cnt = s_start[f + 1] - s_start[f];
    const int id = r < cnt ? oi[s_start[f] + r] - f * P : -1;
    sp.kept_store[(t0 + f) * P + r] = id;
    if (sp.kept_out) sp.kept_out[(long long)(f0 + f) * P + r] = id;
  }
}

}  // namespace mukv
