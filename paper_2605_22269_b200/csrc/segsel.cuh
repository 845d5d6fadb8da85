// Segment-level dual-signal selection (Sec. 3.3: the indicator "I_v in R^O" of a whole segment and
// its budget kappa_v = floor(rho_v * O)).
//
// The indicators of every frame are computed as for frame-level selection (score_kernel in double
// precision, attention inside the frame); segsel_kernel then normalises both signals over all
// O = F * P tokens of a segment (Eq. 4), keeps the kappa_v best of them and splits the result by
// frame: a frame keeps a variable number of tokens, its page has that many rows, and the pages of
// a segment lie one behind the other in the segment's share of the page region.
// One block per segment of the chunk; everything is double precision (the whole segment is ranked
// at once, so there is no cheap way to tell which frames would be safe in single precision).
#pragma once
#include "common.cuh"
#include "retrieve.cuh"
#include "score.cuh"

namespace mukv {

constexpr int kSegSelThreads = 512;
constexpr int kSegSelMaxTokens = 4096;        // F * P of one segment

struct SegSelParams {
  ScoreParams sp;               // double partial sums of score_kernel, Eq. 4 parameters, outputs
  int fseg;                     // frames per segment
  int kappa_v;                  // tokens kept in a full segment
  long long token_bytes;        // bytes one kept token takes in a page: 2 * L * C * sizeof(element)
  int* kept_count;              // [max_frames]
};

__host__ inline size_t segsel_smem_bytes(int tokens) {
  return (size_t)tokens * (2 * sizeof(double) + sizeof(int)) + 64 * sizeof(int);
}

__global__ void __launch_bounds__(kSegSelThreads) segsel_kernel(const SegSelParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ RankScratch sc;
  __shared__ double s_red[kSegSelThreads / 32][4];
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
  for (int w = 0; w < kSegSelThreads / 32; ++w) {
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

  // ---- the kappa best of the segment (kappa_v scaled to the frames present), ascending
  const int k = (int)(((long long)p.kappa_v * m) / p.fseg);
  const ArrScore score{sa};
  const AllMembers always;
  const int n_kept = block_topk_set(score, always, O, k, (double)sp.tie_eps, oi, (double*)nullptr, &sc);
  __syncthreads();
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
