// Per-frame token scoring and selection (Sec. 3.3, Eq. 1-4 and the top-kappa rule).
//
// score_kernel<T, A, NC>: one thread block per (query head h, frame f).
//   * Eq. 1: S = Q_h K_g^T / sqrt(D) over the frame's P tokens, row softmax, column sums.
//     Lanes own key columns (j = lane + 32c), a warp walks the query rows four at a time, so
//     the column sums stay in registers and only the row maximum / row sum cross lanes.
//     The attention matrix is never written anywhere.
//   * Eq. 2-3: the G query-head blocks that share key head g split that head's tokens and
//     transform each key vector along the feature axis; sum of the D bin magnitudes per token.
//   * The block that finishes a frame last (arrival counter, nobody waits) reduces the
//     per-head partials in a fixed order, applies Eq. 4 and selects the kappa tokens.
// T is the input element type, A the arithmetic type: float for the normal path, double for
// the frames whose selection is too close to a tie boundary to trust single precision.
#pragma once
#include "common.cuh"

namespace mukv {

constexpr int kScoreThreads = 256;
constexpr int kStatusNonFinite = 7;   // a frame's scores were not finite: its lowest kappa ids were kept
constexpr int kScoreWarps = kScoreThreads / 32;
constexpr int kRowsPerStep = 4;

struct ScoreParams {
  int P, Hq, Hkv, D, G, kappa;
  int Ls;                       // scoring layers (Eq. 1-3 are averaged over them); >= 1
  long long q_layer_stride;     // elements between the queries of two scoring layers (n * P * Hq * D)
  long long k_layer_stride;     // elements between the keys of two layers (n * P * Hkv * D)
  int n_frames;                 // frames in this chunk
  int causal, keep_low;
  float alpha, tie_eps, flag_margin, flat_ratio;
  long long first_frame;
  // inputs
  const void* q;                // [Ls][n][P][Hq][D]
  const void* k_last;           // [Ls][n][P][Hkv][D]  (the scoring layers of K; by default the last layer)
  // scratch
  void* colsum_part;            // A [F][Ls * Hq * row_split][P]
  void* ifft_part;              // A [F][Ls * Hkv][P]
  int* frame_counter;           // [F], zero between launches
  int* flagged;                 // [F] frame slots needing the double pass
  int* n_flagged;               // count (written by the float pass, read by the double pass)
  // outputs
  int* kept_store;              // [max_frames][kappa]
  int* kept_out;                // [n][kappa] or null
  float* scores_out;            // [3][n][P] or null
  long long* frame_ts;          // [max_frames]
  long long* page_table;        // [max_frames]
  long long pages_off, page_bytes;
  int* status;                  // device event word (0 = nothing recorded); see mukv_stats.device_status
  // cached keys the queries also attend to (Sec. 3.2): the kept keys of the n_past_frames frames stored
  // just before the chunk, kappa rows each, read from their pages; n_past_frames = 0: none
  int n_past_frames;
  long long past_first;         // absolute index of the first of those frames
  int first_score_layer;        // layer of the model the first scoring layer is
  const unsigned char* store;   // store base (page_table holds byte offsets from it)
  int no_select;                // 1: only the partial sums are wanted (the selection runs over a whole segment elsewhere)
  int refine;                   // 1: frames come from the flagged list, no further flagging
  int row_split;                // blocks that share a query head, each a range of query rows (>= 1)
  // segment-level selection, double-precision pass: only the frames of segments whose word is non-zero
  // are scored (segment of chunk frame f: f / gate_fseg); null: every frame
  const int* seg_gate;
  int gate_fseg;
};

template <typename T>
__host__ __device__ constexpr int score_row_stride(int D) { return D + ElemTraits<T>::kPad; }

// P: key rows held in shared memory (the frame's tokens plus the past keys)
template <typename T, typename A>
__host__ inline size_t score_smem_bytes(int P, int D) {
  size_t ks = (size_t)P * score_row_stride<T>(D) * sizeof(T);
  size_t qs = (size_t)kScoreWarps * kRowsPerStep * D * sizeof(T);
  size_t tw = (size_t)D * 2 * sizeof(A);
  size_t red = (size_t)kScoreWarps * 256 * sizeof(A);
  size_t sel = (size_t)256 * sizeof(double) + 64 * sizeof(double) + 64 * sizeof(int);
  return ((ks + 15) / 16) * 16 + qs + tw + red + sel + 64;
}

// The top-kappa rule for one frame on final scores s (double), run by all threads of the group Grp.
// Thread tid owns the tokens tid + k*size, k < TOK (TOK*size >= P).  tau is the kappa-th largest
// score (rank counting: P <= 256); scores above tau + tie_eps are kept, the scores within tie_eps
// of tau share the remaining places by lowest token id.  keep[k] says which of the thread's tokens
// stay; the kept ids go, ascending, to s_kept (shared memory, may be null) and, with `write`, to
// the store, to the caller's output and the frame's time stamp and page-table entry are set.
// s_sc (P doubles), s_int (one int per warp + 1), s_misc (4 doubles per warp) are shared scratch.
template <int TOK, class Grp = BlockGroup>
__device__ inline void select_by_score(const ScoreParams& p, int f, const double (&s)[TOK], bool write, int* s_kept,
                                       bool (&keep)[TOK], double* s_sc, int* s_int, double* s_misc) {
  const int tid = Grp::tid();
  const int nt = Grp::size();
  const int P = p.P;
  int tok[TOK];
  bool valid[TOK];
#pragma unroll
  for (int k = 0; k < TOK; ++k) {
    tok[k] = tid + k * nt;
    valid[k] = tok[k] < P;
    if (valid[k]) s_sc[tok[k]] = s[k];
  }
  Grp::sync();
  const int kappa = p.kappa;
#pragma unroll
  for (int k = 0; k < TOK; ++k) {
    if (valid[k]) {
      int gt = 0, ge = 0;
      for (int i = 0; i < P; ++i) {
        const double o = s_sc[i];
        gt += (o > s[k]);
        ge += (o >= s[k]);
      }
      if (gt < kappa && kappa <= ge) s_misc[0] = s[k];      // every writer holds the same value
    }
  }
  Grp::sync();
  const double tau = s_misc[0];
  const double delta = (double)p.tie_eps;
  bool sure[TOK], band[TOK];
  int n_sure = 0;
#pragma unroll
  for (int k = 0; k < TOK; ++k) {
    sure[k] = valid[k] && (s[k] > tau + delta);
    band[k] = valid[k] && !sure[k] && (s[k] >= tau - delta);
    int t;
    group_excl_count<Grp>(sure[k], s_int, t);
    n_sure += t;
  }
  int band_before = 0;
#pragma unroll
  for (int k = 0; k < TOK; ++k) {
    int t;
    const int band_rank = band_before + group_excl_count<Grp>(band[k], s_int, t);
    band_before += t;
    keep[k] = sure[k] || (band[k] && band_rank < kappa - n_sure);
  }
  const long long f_abs = p.first_frame + f;
  int out_before = 0;
#pragma unroll
  for (int k = 0; k < TOK; ++k) {
    int t;
    const int pos = out_before + group_excl_count<Grp>(keep[k], s_int, t);
    out_before += t;
    if (keep[k]) {
      if (s_kept) s_kept[pos] = tok[k];
      if (write) {
        p.kept_store[f_abs * kappa + pos] = tok[k];
        if (p.kept_out) p.kept_out[(long long)f * kappa + pos] = tok[k];
      }
    }
  }
  if (write && tid == 0) {
    p.frame_ts[f_abs] = f_abs;
    p.page_table[f_abs] = p.pages_off + f_abs * p.page_bytes;
  }
}

// Eq. 4 and the top-kappa rule for one frame, run by all threads of the group Grp.  Thread tid owns
// the tokens tid + k*size, k < TOK (TOK*size >= P); att_raw / fft_raw are their I_att and I_fft;
// s_sc (P doubles), s_int (one int per warp + 1), s_misc (4 doubles per warp) are shared scratch.
// The arithmetic here is always double: it is a few hundred operations per frame and keeps
// the normalisation from adding rounding noise of its own to the scores.
template <int TOK, class Grp = BlockGroup>
__device__ inline void select_frame(const ScoreParams& p, int f, const double (&att_raw)[TOK],
                                    const double (&fft_raw)[TOK], double* s_sc, int* s_int, double* s_misc) {
  typedef double A;
  const int tid = Grp::tid(), lane = tid & 31, warp = tid >> 5;
  const int nt = Grp::size(), nwarp = nt >> 5;
  const int P = p.P;
  const A big = (A)3.0e38;
  int tok[TOK];
  bool valid[TOK];
#pragma unroll
  for (int k = 0; k < TOK; ++k) { tok[k] = tid + k * nt; valid[k] = tok[k] < P; }
  // ---- a frame with a score that is not a number has no ranking: every score counts as 0 below,
  // so that the lowest kappa ids are kept, and the event is recorded
  bool bad_here = false;
#pragma unroll
  for (int k = 0; k < TOK; ++k) bad_here |= valid[k] && !(isfinite(att_raw[k]) && isfinite(fft_raw[k]));
  int n_bad;
  group_excl_count<Grp>(bad_here, s_int, n_bad);
  const bool bad = n_bad != 0;
  // ---- min / max of both signals over the frame
  A v[4] = {big, -big, big, -big};
#pragma unroll
  for (int k = 0; k < TOK; ++k) {
    if (valid[k]) {
      v[0] = att_raw[k] < v[0] ? att_raw[k] : v[0];
      v[1] = att_raw[k] > v[1] ? att_raw[k] : v[1];
      v[2] = fft_raw[k] < v[2] ? fft_raw[k] : v[2];
      v[3] = fft_raw[k] > v[3] ? fft_raw[k] : v[3];
    }
  }
  v[0] = warp_min(v[0]); v[1] = warp_max(v[1]); v[2] = warp_min(v[2]); v[3] = warp_max(v[3]);
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) s_misc[warp * 4 + i] = v[i];
  }
  Grp::sync();
  A amin = big, amax = -big, fmin_ = big, fmax_ = -big;
  for (int w = 0; w < nwarp; ++w) {
    amin = s_misc[w * 4 + 0] < amin ? s_misc[w * 4 + 0] : amin;
    amax = s_misc[w * 4 + 1] > amax ? s_misc[w * 4 + 1] : amax;
    fmin_ = s_misc[w * 4 + 2] < fmin_ ? s_misc[w * 4 + 2] : fmin_;
    fmax_ = s_misc[w * 4 + 3] > fmax_ ? s_misc[w * 4 + 3] : fmax_;
  }
  Grp::sync();
  // ---- Eq. 4
  const A alpha = (A)p.alpha;
  A s[TOK];
#pragma unroll
  for (int k = 0; k < TOK; ++k) {
    A an = (amax == amin) ? (A)0 : (att_raw[k] - amin) / (amax - amin);
    A fn = (fmax_ == fmin_) ? (A)0 : (fft_raw[k] - fmin_) / (fmax_ - fmin_);
    if (p.keep_low) fn = (A)1 - fn;
    s[k] = bad ? (A)0 : alpha * an + ((A)1 - alpha) * fn;
  }
  bool keep[TOK];
  select_by_score<TOK, Grp>(p, f, s, true, nullptr, keep, s_sc, s_int, s_misc);
  if (p.scores_out) {
    const long long np = (long long)p.n_frames * P;
#pragma unroll
    for (int k = 0; k < TOK; ++k) {
      if (valid[k]) {
        p.scores_out[0 * np + (long long)f * P + tok[k]] = (float)att_raw[k];
        p.scores_out[1 * np + (long long)f * P + tok[k]] = (float)fft_raw[k];
        p.scores_out[2 * np + (long long)f * P + tok[k]] = (float)s[k];
      }
    }
  }
  if (tid == 0 && bad && p.status) atomicCAS(p.status, 0, kStatusNonFinite);
  // ---- does single precision decide this frame safely?
  // With a = lowest kept score and b = highest dropped score, the kept set is the same for every
  // perturbation of the scores below flag_margin / 2 as long as a - b > tie_eps + flag_margin: no
  // dropped token can then enter the tie band of the kappa-th score.  Anything closer is redone
  // in double precision.
  if (!p.refine && !bad) {
    const int kappa = p.kappa;
    const A delta = (A)p.tie_eps;
    A a = big, b = -big;
#pragma unroll
    for (int k = 0; k < TOK; ++k) {
      if (valid[k]) {
        if (keep[k]) a = s[k] < a ? s[k] : a;
        else b = s[k] > b ? s[k] : b;
      }
    }
    a = warp_min(a);
    b = warp_max(b);
    Grp::sync();
    if (lane == 0) { s_misc[warp * 4] = a; s_misc[warp * 4 + 1] = b; }
    Grp::sync();
    if (tid == 0) {
      for (int w = 1; w < nwarp; ++w) {
        a = s_misc[w * 4] < a ? s_misc[w * 4] : a;
        b = s_misc[w * 4 + 1] > b ? s_misc[w * 4 + 1] : b;
      }
      bool risky = (kappa < P) && (a - b <= delta + (A)p.flag_margin);
      // a nearly flat signal amplifies rounding noise through the min-max division
      const A fr = (A)p.flat_ratio;
      const A aabs = amax > -amin ? amax : -amin, fabs_ = fmax_ > -fmin_ ? fmax_ : -fmin_;
      if (amax != amin && (amax - amin) < fr * aabs && p.alpha != 0.f) risky = true;
      if (fmax_ != fmin_ && (fmax_ - fmin_) < fr * fabs_ && p.alpha != 1.f) risky = true;
      if (risky) {
        const int slot = atomicAdd(p.n_flagged, 1);
        p.flagged[slot] = f;
      }
    }
  }
}

// The work of one block: part q (of p.row_split) of the query rows of head hv of frame f (a frame
// slot of the chunk); hv counts the query heads of all scoring layers, layer-major.
template <typename T, typename A, int NC>
__device__ __forceinline__ void score_frame_block(const ScoreParams& p, int hv, int q, int f,
                                                  unsigned char* smem_raw) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = p.P, D = p.D, Hq = p.Hq, Hkv = p.Hkv, G = p.G;
  const int layer = hv / Hq, h = hv - layer * Hq;
  const int HqV = p.Ls * Hq, HkvV = p.Ls * Hkv;
  const int g = h / G;
  constexpr int EPW = ElemTraits<T>::kPerWord;
  const int DS = score_row_stride<T>(D);
  const int WS = DS / EPW;                         // words per padded K row
  const int DW = D / EPW;                          // words per vector

  // key rows: the past keys first, then the frame's own tokens
  const int n_past = p.n_past_frames * p.kappa, Pk = n_past + P;

  // ---- shared memory carve-up
  size_t off = 0;
  T* Ks = reinterpret_cast<T*>(smem_raw);
  off = (((size_t)Pk * DS * sizeof(T)) + 15) / 16 * 16;
  T* Qs = reinterpret_cast<T*>(smem_raw + off);
  off += (size_t)kScoreWarps * kRowsPerStep * D * sizeof(T);
  A* tw = reinterpret_cast<A*>(smem_raw + off);
  off += (size_t)D * 2 * sizeof(A);
  A* red = reinterpret_cast<A*>(smem_raw + off);
  off += (size_t)kScoreWarps * 256 * sizeof(A);
  double* s_sc = reinterpret_cast<double*>(smem_raw + off);
  off += (size_t)256 * sizeof(double);
  double* s_misc = reinterpret_cast<double*>(smem_raw + off);
  off += 64 * sizeof(double);
  int* s_int = reinterpret_cast<int*>(smem_raw + off);

  // ---- stage K_g of this frame (rows padded so that 32 consecutive rows hit 32 banks)
  const T* Kg = reinterpret_cast<const T*>(p.k_last) + layer * p.k_layer_stride + ((long long)f * P * Hkv + g) * D;
  {
    constexpr int VE = 16 / sizeof(T);             // elements per 16-byte vector
    const int vec_per_row = D / VE;
    for (int v = tid; v < n_past * vec_per_row; v += kScoreThreads) {
      // row r of the past: kept row r % kappa of frame past_first + r / kappa, this layer's K plane of its page
      const int r = v / vec_per_row, c = v % vec_per_row;
      const long long t = p.past_first + r / p.kappa;
      const T* page = reinterpret_cast<const T*>(p.store + p.page_table[t]);
      const T* src = page + ((long long)(p.first_score_layer + layer) * 2 * p.kappa + r % p.kappa) * Hkv * D + g * D;
      const uint4 x = *reinterpret_cast<const uint4*>(src + c * VE);
      uint32_t* dst = reinterpret_cast<uint32_t*>(Ks + (size_t)r * DS + c * VE);
      dst[0] = x.x; dst[1] = x.y; dst[2] = x.z; dst[3] = x.w;
    }
    for (int v = tid; v < P * vec_per_row; v += kScoreThreads) {
      const int j = v / vec_per_row, c = v % vec_per_row;
      const uint4 x = *reinterpret_cast<const uint4*>(Kg + (long long)j * Hkv * D + c * VE);
      uint32_t* dst = reinterpret_cast<uint32_t*>(Ks + (size_t)(n_past + j) * DS + c * VE);
      dst[0] = x.x; dst[1] = x.y; dst[2] = x.z; dst[3] = x.w;
    }
    for (int d = tid; d < D; d += kScoreThreads) {
      double sn, cs;
      sincospi(2.0 * (double)d / (double)D, &sn, &cs);
      tw[2 * d] = (A)cs;
      tw[2 * d + 1] = (A)sn;
    }
  }
  __syncthreads();

  // ---- Eq. 1: column sums of the row softmax
  const uint32_t* Kw = reinterpret_cast<const uint32_t*>(Ks);
  uint32_t* Qw = reinterpret_cast<uint32_t*>(Qs) + (size_t)warp * kRowsPerStep * DW;
  const T* Qh = reinterpret_cast<const T*>(p.q) + layer * p.q_layer_stride + ((long long)f * P * Hq + h) * D;
  // 1/sqrt(D) as a two-term constant, so that single precision scales the logits without a
  // systematic relative error shared by every element
  const double scale_d = 1.0 / sqrt((double)D);
  const A scale = (A)scale_d;
  const A scale_lo = (A)(scale_d - (double)scale);
  A csum[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) csum[c] = (A)0;
  int jrow[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) jrow[c] = min(lane + 32 * c, Pk - 1) * WS;

  const int RS = p.row_split;
  const int n_steps = (P + kRowsPerStep - 1) / kRowsPerStep;
  const int n_per = (n_steps + RS - 1) / RS;
  const int rb_end = (q + 1) * n_per < n_steps ? (q + 1) * n_per : n_steps;
  for (int rb = q * n_per + warp; rb < rb_end; rb += kScoreWarps) {
    __syncwarp();
#pragma unroll
    for (int r = 0; r < kRowsPerStep; ++r) {
      const int i = rb * kRowsPerStep + r;
      const uint32_t* src = reinterpret_cast<const uint32_t*>(Qh + (long long)min(i, P - 1) * Hq * D);
      for (int w = lane; w < DW; w += 32) Qw[r * DW + w] = (i < P) ? __ldg(src + w) : 0u;
    }
    __syncwarp();
    A acc[kRowsPerStep][NC];
#pragma unroll
    for (int r = 0; r < kRowsPerStep; ++r)
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[r][c] = (A)0;
#pragma unroll 2
    for (int w = 0; w < DW; ++w) {
      uint32_t qw[kRowsPerStep];
#pragma unroll
      for (int r = 0; r < kRowsPerStep; ++r) qw[r] = Qw[r * DW + w];
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const uint32_t kw = Kw[jrow[c] + w];
#pragma unroll
        for (int r = 0; r < kRowsPerStep; ++r) acc[r][c] = dot_word<T, A>(qw[r], kw, acc[r][c]);
      }
    }
#pragma unroll
    for (int r = 0; r < kRowsPerStep; ++r) {
      const int i = rb * kRowsPerStep + r;
      A z[NC];
      A m = neg_inf<A>();
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const int j = lane + 32 * c;                     // past keys are visible to every query
        const bool ok = (j < Pk) && (!p.causal || j - n_past <= i);
        z[c] = ok ? fma_acc(acc[r][c], scale, acc[r][c] * scale_lo) : neg_inf<A>();
        m = z[c] > m ? z[c] : m;
      }
      m = warp_max(m);
      A l = (A)0;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        z[c] = (z[c] == neg_inf<A>()) ? (A)0 : exp_acc(z[c] - m);
        l += z[c];
      }
      l = warp_sum(l);
      const A inv = (i < P) ? (A)1 / l : (A)0;
#pragma unroll
      for (int c = 0; c < NC; ++c) csum[c] += z[c] * inv;
    }
  }
  // cross-warp reduction in a fixed order
#pragma unroll
  for (int c = 0; c < NC; ++c) red[warp * 256 + lane + 32 * c] = csum[c];
  __syncthreads();
  if (tid < P) {                                       // the importance is that of the frame's own tokens
    A t = (A)0;
    for (int w = 0; w < kScoreWarps; ++w) t += red[w * 256 + n_past + tid];
    reinterpret_cast<A*>(p.colsum_part)[(((long long)f * HqV + hv) * RS + q) * P + tid] = t;
  }

  // ---- Eq. 2-3: sum over the D bins of |DFT(k_j)| for this block's share of head g's tokens
  {
    const int hg = (h % G) * RS + q;                 // the G * RS blocks that hold key head g share its tokens
    const int half = D / 2;
    for (int j = hg + warp * G * RS; j < P; j += kScoreWarps * G * RS) {
      const T* kr = Ks + (size_t)(n_past + j) * DS;
      A total = (A)0;
      // bins 1 .. D/2-1 (twice, by conjugate symmetry) and bin 0
      for (int b = lane; b < half; b += 32) {
        A re = (A)0, im = (A)0;
        for (int d = 0; d < D; ++d) {
          const A x = (A)elem_to_float<T>(kr[d]);
          const int m = (b * d) & (D - 1);
          re += x * tw[2 * m];
          im -= x * tw[2 * m + 1];
        }
        const A mag = sqrt_acc(re * re + im * im);
        total += (b == 0) ? mag : (A)2 * mag;
      }
      // bin D/2: alternating sum
      A alt = (A)0;
      for (int d = lane; d < D; d += 32) {
        const A x = (A)elem_to_float<T>(kr[d]);
        alt += (d & 1) ? -x : x;
      }
      total = warp_sum(total);
      alt = warp_sum(alt);
      if (lane == 0)
        reinterpret_cast<A*>(p.ifft_part)[((long long)f * HkvV + layer * Hkv + g) * P + j] = total + (alt < (A)0 ? -alt : alt);
    }
  }

  // ---- last block of the frame finishes Eq. 1 / Eq. 3 and selects
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int old = atomicAdd(p.frame_counter + f, 1);
    s_int[63] = (old == HqV * RS - 1);
    if (old == HqV * RS - 1) p.frame_counter[f] = 0;  // ready for the next launch
  }
  __syncthreads();
  if (!s_int[63] || p.no_select) return;
  __threadfence();
  double att[1] = {0.0}, fft[1] = {0.0};
  if (tid < P) {
    const A* cp = reinterpret_cast<const A*>(p.colsum_part) + (long long)f * HqV * RS * P + tid;
    for (int hh = 0; hh < HqV * RS; ++hh) att[0] += (double)__ldcg(cp + (long long)hh * P);
    att[0] = att[0] / (double)((long long)HqV * P);
    const A* fp = reinterpret_cast<const A*>(p.ifft_part) + (long long)f * HkvV * P + tid;
    for (int gg = 0; gg < HkvV; ++gg) fft[0] += (double)__ldcg(fp + (long long)gg * P);
    fft[0] = fft[0] / (double)((long long)HkvV * D);
  }
  __syncthreads();
  select_frame<1>(p, f, att, fft, s_sc, s_int, s_misc);
}

// Grid (Hq * row_split, frames).  Normal pass: block row = frame slot of the chunk.  Double-precision
// pass (p.refine): the grid has few rows of blocks, which walk the list of flagged frames; with
// nothing flagged they return at once.
template <typename T, typename A, int NC>
__global__ void __launch_bounds__(kScoreThreads) score_kernel(const ScoreParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_wait();
  pdl_trigger();
  if (!p.refine) {
    if (p.seg_gate) {
      // a small one-dimensional grid walks the frames and scores those of flagged segments (rarely any)
      const int units = p.Ls * p.Hq * p.row_split;
      for (int f = 0; f < p.n_frames; ++f) {
        if (__ldcg(p.seg_gate + f / p.gate_fseg) == 0) continue;
        for (int u = blockIdx.x; u < units; u += gridDim.x) {
          score_frame_block<T, A, NC>(p, u / p.row_split, u % p.row_split, f, smem_raw);
          __syncthreads();
        }
      }
      return;
    }
    score_frame_block<T, A, NC>(p, blockIdx.x / p.row_split, blockIdx.x % p.row_split, blockIdx.y, smem_raw);
    return;
  }
  const int n = *p.n_flagged;
  for (int slot = blockIdx.y; slot < n; slot += gridDim.y) {
    score_frame_block<T, A, NC>(p, blockIdx.x / p.row_split, blockIdx.x % p.row_split, p.flagged[slot], smem_raw);
    __syncthreads();
  }
}

}  // namespace mukv
