// Semi-hierarchical retrieval (Sec. 3.4, Eq. 6-8) and the gather of the retrieved context
// (Sec. 3.5, Eq. 9).
//
// All ranking arithmetic is double precision: the work is a few hundred MFLOP per batch of
// questions, tiny next to the gather, and it makes the selected indices independent of
// summation order.  Kernels:
//   qpool_kernel    Eq. 6   one block per (question, key head)
//   scan_kernel     Eq. 7   cosine of every question with every frame key and segment key (a skinny
//                           double-precision product on the fp64 tensor-core instruction)
//   rank_kernel     stage-1 candidates, Eq. 8 rerank, final top-k; one block per question
//   gather_kernel   Eq. 9   copies the selected pages into the per-question decode buffers
#pragma once
#include "common.cuh"

namespace mukv {

struct QMeta {
  int off[MUKV_MAX_QUESTIONS + 1];
  long long t_limit[MUKV_MAX_QUESTIONS];
};

// ------------------------------------------------------------------------------ Eq. 6
// One block per (question, key head).  Thread (slice, vector) sums one 16-byte vector of the head's
// channels over the tokens n = slice, slice + slices, ... and the G query heads of the group: every
// load is a full 16-byte vector and all of a thread's loads are independent.  The slices are added
// in a fixed order.  The pooled query is written transposed, q64t[c][question] (row stride
// MUKV_MAX_QUESTIONS), the layout scan_kernel stages; the head's share of the squared norm goes to
// qn2[question][key head] (scan_kernel adds the shares in head order).
constexpr int kPoolThreads = 512;
constexpr int kPoolSmemDoubles = 4096;

template <typename T>
__global__ void __launch_bounds__(kPoolThreads) qpool_kernel(const T* __restrict__ qtok, const QMeta meta, int Hq,
                                                             int Hkv, int D, double* __restrict__ q64t,
                                                             double* __restrict__ qn2) {
  constexpr int VE = 16 / sizeof(T);
  __shared__ double s_acc[kPoolSmemDoubles];
  __shared__ double s_part[kPoolThreads / 32];
  const int qi = blockIdx.x, g = blockIdx.y;
  const int G = Hq / Hkv;
  const int n0 = meta.off[qi], n1 = meta.off[qi + 1];
  const int DV = D / VE;                                    // vectors per head
  int nsl = kPoolThreads / DV;                              // token slices whose partial sums fit
  if (nsl > kPoolSmemDoubles / D) nsl = kPoolSmemDoubles / D;
  const int sl = threadIdx.x / DV, dv = threadIdx.x % DV;
  if (sl < nsl) {
    double tot[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) tot[e] = 0.0;
    for (int n = n0 + sl; n < n1; n += nsl) {
      const T* row = qtok + ((long long)n * Hq + (long long)g * G) * D + dv * VE;
#pragma unroll 1
      for (int j0 = 0; j0 < G; j0 += 8) {
        uint4 x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
          x[j] = j0 + j < G ? *reinterpret_cast<const uint4*>(row + (long long)(j0 + j) * D) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t w[4] = {x[j].x, x[j].y, x[j].z, x[j].w};
          if constexpr (sizeof(T) == 2) {
#pragma unroll
            for (int i = 0; i < 4; ++i) { tot[2 * i] += (double)bf16_lo(w[i]); tot[2 * i + 1] += (double)bf16_hi(w[i]); }
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) tot[i] += (double)__uint_as_float(w[i]);
          }
        }
      }
    }
#pragma unroll
    for (int e = 0; e < VE; ++e) s_acc[sl * D + dv * VE + e] = tot[e];
  }
  __syncthreads();
  double sq = 0.0;
  for (int col = threadIdx.x; col < D; col += kPoolThreads) {
    double t = 0.0;
    for (int k = 0; k < nsl; ++k) t += s_acc[k * D + col];
    t = t / (double)((long long)(n1 - n0) * G);
    q64t[(long long)(g * D + col) * MUKV_MAX_QUESTIONS + qi] = t;
    sq += t * t;
  }
  sq = warp_sum(sq);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = sq;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < kPoolThreads / 32; ++w) t += s_part[w];
    qn2[(long long)qi * Hkv + g] = t;
  }
}

// ------------------------------------------------------------------------------ Eq. 7
// Rows 0..n_frm-1 are frame keys, rows n_frm..n_frm+n_seg-1 segment keys, then n_pat patch-level
// keys (n_pat = 0 without a patch level).  A block owns
// kScanRows rows and walks the feature axis in chunks of kScanCC: the rows' chunk (float) and the
// chunk of up to kScanQB pooled queries (double) are staged in shared memory.  The product itself
// is a dense double-precision contraction [rows x C] . [C x questions] and runs on the
// double-precision tensor-core instruction (mma.sync m8n8k4 f64): warp w owns rows 8*(w%4).. and
// questions 32*(w/4).., four 8 x 8 accumulator tiles.  (Plain double-precision FMAs are slow on
// this part; the scores have to be double because indices are ranked on them.)
constexpr int kScanRows = 32;
constexpr int kScanCC = 64;
constexpr int kScanQB = 64;
constexpr int kScanQPad = kScanQB + 4;

__device__ __forceinline__ void dmma_m8n8k4(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(c[0]), "+d"(c[1])
               : "d"(a), "d"(b));
}

struct ScanParams {
  const float* frame_key; const float* seg_key; const float* patch_key;
  long long n_frm, n_seg, n_pat;
  int C, nq, Hkv;
  const double* q64t; const double* qn2;
  double* s_frm; double* s_seg; double* s_pat;
  long long frm_stride, seg_stride, pat_stride;
};

__global__ void __launch_bounds__(256) scan_kernel(const ScanParams sp) {
  const float* __restrict__ frame_key = sp.frame_key;
  const float* __restrict__ seg_key = sp.seg_key;
  const long long n_frm = sp.n_frm, n_seg = sp.n_seg;
  const int C = sp.C, nq = sp.nq, Hkv = sp.Hkv;
  const double* __restrict__ q64t = sp.q64t;
  const double* __restrict__ qn2 = sp.qn2;
  double* __restrict__ s_frm = sp.s_frm;
  double* __restrict__ s_seg = sp.s_seg;
  const long long frm_stride = sp.frm_stride, seg_stride = sp.seg_stride;
  __shared__ float rows[kScanRows][kScanCC + 1];
  __shared__ __align__(16) double qs[kScanCC][kScanQPad];
  __shared__ double s_knorm[kScanRows];
  __shared__ double s_qn[MUKV_MAX_QUESTIONS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();                                                // the pooled questions are complete
  pdl_trigger();
  for (int qq = tid; qq < nq; qq += 256) {                   // norms of the pooled questions (read after the barriers below)
    double t = 0.0;
    for (int gg = 0; gg < Hkv; ++gg) t += qn2[(long long)qq * Hkv + gg];
    s_qn[qq] = sqrt(t);
  }
  const long long row0 = (long long)blockIdx.x * kScanRows;
  const long long n_rows = n_frm + n_seg + sp.n_pat;
  const int lr = tid >> 3, lc = (tid & 7) * 8;               // staging: row, first column of 8
  const long long my_row = row0 + lr;
  const float* src = my_row < n_frm ? frame_key + my_row * C
                     : (my_row < n_frm + n_seg ? seg_key + (my_row - n_frm) * C
                     : (my_row < n_rows ? sp.patch_key + (my_row - n_frm - n_seg) * C : nullptr));
  const int wr = (warp & 3) * 8, wq = (warp >> 2) * 32;      // this warp's rows and questions
  const int fr = lane >> 2, fk = lane & 3;                   // fragment row / k (A), k / column (B)
  for (int qb = 0; qb < nq; qb += kScanQB) {
    double acc[4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i) { acc[i][0] = 0.0; acc[i][1] = 0.0; }
    double kk = 0.0;
    // the chunk after the one being multiplied is already on its way into registers
    float xr[8];
    double xq[kScanCC * kScanQB / 256];
    auto fetch = [&](int c0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int cc = lc + i;
        xr[i] = (src && c0 + cc < C) ? src[c0 + cc] : 0.f;
      }
#pragma unroll
      for (int i = 0; i < kScanCC * kScanQB / 256; ++i) {
        const int idx = tid + i * 256;
        const int cc = idx / kScanQB, qq = idx % kScanQB;
        xq[i] = (c0 + cc < C && qb + qq < nq) ? q64t[(long long)(c0 + cc) * MUKV_MAX_QUESTIONS + qb + qq] : 0.0;
      }
    };
    fetch(0);
    for (int c0 = 0; c0 < C; c0 += kScanCC) {
      __syncthreads();                                       // the previous chunk has been consumed
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        rows[lr][lc + i] = xr[i];
        kk = fma((double)xr[i], (double)xr[i], kk);
      }
#pragma unroll
      for (int i = 0; i < kScanCC * kScanQB / 256; ++i) {
        const int idx = tid + i * 256;
        qs[idx / kScanQB][idx % kScanQB] = xq[i];
      }
      __syncthreads();
      if (c0 + kScanCC < C) fetch(c0 + kScanCC);
#pragma unroll 4
      for (int cc = 0; cc < kScanCC; cc += 4) {
        const double a = (double)rows[wr + fr][cc + fk];     // A[row fr][k fk]
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) dmma_m8n8k4(acc[nt], a, qs[cc + fk][wq + nt * 8 + fr]);   // B[k fk][col fr]
      }
    }
    if (qb == 0) {
      // the 8 staging threads of a row hold the parts of its squared norm
      kk += __shfl_xor_sync(kFull, kk, 1);
      kk += __shfl_xor_sync(kFull, kk, 2);
      kk += __shfl_xor_sync(kFull, kk, 4);
      if ((tid & 7) == 0) s_knorm[lr] = sqrt(kk);
    }
    __syncthreads();
    // accumulator tile: row fr, columns 2*fk and 2*fk + 1
    const int r = wr + fr;
    const long long row = row0 + r;
    if (row < n_rows) {
      const double knorm = s_knorm[r];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int qi = qb + wq + nt * 8 + 2 * fk + j;
          if (qi >= nq) continue;
          double den = knorm * s_qn[qi];
          den = den > 1e-12 ? den : 1e-12;
          const double sc = acc[nt][j] / den;
          if (row < n_frm) s_frm[(long long)qi * frm_stride + row] = sc;
          else if (row < n_frm + n_seg) s_seg[(long long)qi * seg_stride + (row - n_frm)] = sc;
          else sp.s_pat[(long long)qi * sp.pat_stride + (row - n_frm - n_seg)] = sc;
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------ ranking
__device__ __forceinline__ unsigned long long order_key(double x) {
  const unsigned long long b = (unsigned long long)__double_as_longlong(x);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}
__device__ __forceinline__ double order_key_inv(unsigned long long k) {
  const unsigned long long b = (k >> 63) ? (k & 0x7fffffffffffffffull) : ~k;
  return __longlong_as_double((long long)b);
}

constexpr int kRankList = 64;      // keys left in the radix select below which they are ranked directly
constexpr int kRankCand = 256;     // scores at or above the tie band that the short emission path can hold

struct RankScratch {
  unsigned int hist[256];
  int scan[40];
  unsigned long long prefix;
  int remaining;
  int bin_count, list_n, cand_n;
  unsigned long long list[kRankList];
  int cand_idx[kRankCand];
  double cand_s[kRankCand];
  unsigned char cand_band[kRankCand], cand_keep[kRankCand];
};

// Indices of the k highest scores among i in [0,n) with member(i) true, ascending by index, with
// the tie band: tau = k-th largest; scores above tau+delta are taken; those within delta of tau
// share the remaining places by lowest index.  Run by the whole block; returns the count
// (= min(k, number of members)).  score(i) must be cheap and pure.
// score(i) read from an array; every index a member.  One pair of types for the selections over
// segments, frames and candidates, so that they share one copy of block_topk_set (kept out of
// line: the ranking kernel is bound by instruction fetch, not by arithmetic).
struct ArrScore {
  const double* p;
  __device__ double operator()(int i) const { return p[i]; }
};
struct AllMembers {
  __device__ bool operator()(int) const { return true; }
};

template <typename ScoreFn, typename MemberFn>
__device__ __noinline__ int block_topk_set(ScoreFn score, MemberFn member, int n, int k, double delta, int* out_idx,
                              double* out_score, RankScratch* sc) {
  const int tid = threadIdx.x, nt = blockDim.x;
  // how many members are there at all
  int local = 0;
  for (int i = tid; i < n; i += nt) local += member(i) ? 1 : 0;
  __syncthreads();
  if (tid == 0) sc->remaining = 0;
  __syncthreads();
  local = warp_sum(local);
  if ((tid & 31) == 0 && local) atomicAdd(&sc->remaining, local);
  __syncthreads();
  const int n_mem = sc->remaining;
  __syncthreads();
  if (k > n_mem) k = n_mem;
  if (k <= 0) return 0;
  double tau;
  if (k == n_mem) {
    tau = -1.0e300;     // everything is taken; handled below by the "all" flag
  } else {
    // radix select of the k-th largest order key, 8 bits per pass from the top
    if (tid == 0) { sc->prefix = 0ull; sc->remaining = k; }
    for (int pass = 0; pass < 8; ++pass) {
      const int shift = 56 - 8 * pass;
      for (int b = tid; b < 256; b += nt) sc->hist[b] = 0u;
      __syncthreads();
      const unsigned long long prefix = sc->prefix;
      const unsigned long long himask = pass == 0 ? 0ull : (~0ull << (shift + 8));
      for (int i = tid; i < n; i += nt) {
        if (!member(i)) continue;
        const unsigned long long key = order_key(score(i));
        if ((key & himask) == prefix) atomicAdd(&sc->hist[(unsigned)(key >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (tid < 32) {
        // warp 0 finds the bin that holds the remaining-th largest key: lane l owns bins 8l .. 8l+7
        int c[8], T = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { c[i] = (int)sc->hist[8 * tid + i]; T += c[i]; }
        int incl = T;                                   // keys in this lane's bins and all higher ones
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_down_sync(kFull, incl, o);
          if (tid + o < 32) incl += v;
        }
        const int above = incl - T;
        const int rem = sc->remaining;
        __syncwarp();
        if (above < rem && rem <= above + T) {          // true for exactly one lane
          int r = rem - above, b = 7;
          for (; b > 0; --b) {
            if (r <= c[b]) break;
            r -= c[b];
          }
          sc->prefix = prefix | ((unsigned long long)(8 * tid + b) << shift);
          sc->remaining = r;
          sc->bin_count = c[b];
        }
      }
      __syncthreads();
      if (pass < 7 && sc->bin_count <= kRankList) {
        // few keys share the prefix found so far: collect them and rank them directly
        const unsigned long long pre = sc->prefix, mask = ~0ull << shift;
        if (tid == 0) sc->list_n = 0;
        __syncthreads();
        for (int i = tid; i < n; i += nt) {
          if (!member(i)) continue;
          const unsigned long long key = order_key(score(i));
          if ((key & mask) == pre) sc->list[atomicAdd(&sc->list_n, 1)] = key;
        }
        __syncthreads();
        const int m = sc->list_n, r = sc->remaining;
        if (tid < m) {
          const unsigned long long key = sc->list[tid];
          int gt = 0, ge = 0;
          for (int t = 0; t < m; ++t) {
            gt += (sc->list[t] > key);
            ge += (sc->list[t] >= key);
          }
          if (gt < r && r <= ge) sc->prefix = key;      // every writer holds the same value
        }
        __syncthreads();
        break;
      }
    }
    tau = order_key_inv(sc->prefix);
  }
  const bool all = (k == n_mem);
  // Everything at or above the tie band, collected in any order.  When that is a short list (it
  // holds k entries plus the ties), the band rule and the ascending output order are worked out
  // on the list; the ordered walk over all n scores below is the fallback for a crowded band.
  if (tid == 0) sc->cand_n = 0;
  __syncthreads();
  for (int i = tid; i < n; i += nt) {
    if (!member(i)) continue;
    const double s = score(i);
    const bool sure = all || s > tau + delta;
    const bool band = !sure && s >= tau - delta;
    if (sure || band) {
      const int c = atomicAdd(&sc->cand_n, 1);
      if (c < kRankCand) {
        sc->cand_idx[c] = i;
        sc->cand_s[c] = s;
        sc->cand_band[c] = band ? 1 : 0;
      }
    }
  }
  __syncthreads();
  const int n_cand = sc->cand_n;
  if (n_cand <= kRankCand) {
    bool keep = false;
    int my_idx = 0;
    if (tid < n_cand) {
      my_idx = sc->cand_idx[tid];
      int n_sure = 0, band_before = 0;
      for (int t = 0; t < n_cand; ++t) {
        const bool bt = sc->cand_band[t] != 0;
        n_sure += bt ? 0 : 1;
        band_before += (bt && sc->cand_idx[t] < my_idx) ? 1 : 0;
      }
      keep = !sc->cand_band[tid] || band_before < k - n_sure;
      sc->cand_keep[tid] = keep ? 1 : 0;
    }
    __syncthreads();
    if (keep) {
      int pos = 0;
      for (int t = 0; t < n_cand; ++t) pos += (sc->cand_keep[t] && sc->cand_idx[t] < my_idx) ? 1 : 0;
      out_idx[pos] = my_idx;
      if (out_score) out_score[pos] = sc->cand_s[tid];
    }
    __syncthreads();
    return k;
  }
  // count the sure ones
  int cnt = 0;
  for (int i = tid; i < n; i += nt)
    if (member(i) && !all && score(i) > tau + delta) ++cnt;
  __syncthreads();
  if (tid == 0) sc->remaining = 0;
  __syncthreads();
  cnt = warp_sum(cnt);
  if ((tid & 31) == 0 && cnt) atomicAdd(&sc->remaining, cnt);
  __syncthreads();
  const int need = k - sc->remaining;
  __syncthreads();
  // ordered emission
  int band_before = 0, out_before = 0;
  for (int base = 0; base < n; base += nt) {
    const int i = base + tid;
    bool sure = false, band = false;
    double s = 0.0;
    if (i < n && member(i)) {
      s = score(i);
      if (all) sure = true;
      else {
        sure = s > tau + delta;
        band = !sure && s >= tau - delta;
      }
    }
    int n_band, n_out;
    const int br = band_before + block_excl_count(band, sc->scan, n_band);
    const bool keep = sure || (band && br < need);
    const int pos = out_before + block_excl_count(keep, sc->scan, n_out);
    if (keep) {
      out_idx[pos] = i;
      if (out_score) out_score[pos] = s;
    }
    band_before += n_band;
    out_before += n_out;
  }
  __syncthreads();
  return k;
}

struct RankParams {
  int nq, C, fseg;
  int k_seg, k_frm, k_pat, top_n, mode;
  int S;                                  // patch-level blocks per frame (0: none)
  double lam_seg, lam_frm, lam_pat, delta;
  long long n_frm, n_seg;                 // stored
  const double* s_frm;                    // [nq][frm_stride]
  const double* s_seg;
  const double* s_pat;                    // [nq][pat_stride]
  long long frm_stride, seg_stride, pat_stride;
  const float* frame_key;
  const float* seg_key;
  const float* patch_key;
  const int* patch_cnt;                   // [frames][S]
  int* seg_idx; int* frm_idx; int* pat_idx; float* seg_score; float* frm_score; float* pat_score;
  int* counts; int counts_stride;         // 2 or 3 ints per question
  int stage;                              // 1: the question's frame and segment scores are copied to shared memory first
};

constexpr int kRankThreads = 512;
constexpr int kRankStageBytes = 192 * 1024;       // dynamic shared memory the kernel may be given
constexpr int kMaxCand = 2 * MUKV_MAX_TOPK;

struct RankShared {
  RankScratch sc;
  int sel_seg[MUKV_MAX_TOPK];
  double sel_seg_score[MUKV_MAX_TOPK];
  int top[MUKV_MAX_TOPK];
  int cand[kMaxCand];
  double cand_score[kMaxCand];
  double s_new[kMaxCand];
  int pick[MUKV_MAX_TOPK];
  double pick_score[MUKV_MAX_TOPK];
  double gn;
};

// Stage 1 + stage 2 of one granularity for one question, run by the whole block: top-2k candidates
// by cosine among the members, Eq. 8 against the global query gq (norm gnorm; have_g false: gamma = 0),
// then the k best by the calibrated score.  PARALLEL / HIER callers pass semi = false: the k best by
// cosine among the members.  Results (ascending ids) in sh->pick / sh->pick_score; returns the count.
template <typename MemberFn>
__device__ __noinline__ int rank_level(const double* scores, MemberFn member, int n, int k, bool semi, double lambda,
                                       double delta, const float* keys, int C, const double* gq, double gnorm,
                                       bool have_g, RankShared* sh) {
  const int tid = threadIdx.x;
  const ArrScore s1{scores};
  if (!semi) return block_topk_set(s1, member, n, k, delta, sh->pick, sh->pick_score, &sh->sc);
  const int n_cand = block_topk_set(s1, member, n, 2 * k, delta, sh->cand, sh->cand_score, &sh->sc);
  // Eq. 8 for every candidate: one warp per candidate
  const int lane = tid & 31, warp = tid >> 5;
  for (int ci = warp; ci < n_cand; ci += kRankThreads / 32) {
    const float* kr = keys + (long long)sh->cand[ci] * C;
    double dot = 0.0, kk = 0.0;
    for (int c = lane; c < C; c += 32) {
      const double x = (double)kr[c];
      dot = fma(x, gq[c], dot);
      kk = fma(x, x, kk);
    }
    dot = warp_sum(dot);
    kk = warp_sum(kk);
    if (lane == 0) {
      double gamma = 0.0;
      if (have_g) {
        double den = sqrt(kk) * gnorm;
        den = den > 1e-12 ? den : 1e-12;
        gamma = dot / den;
      }
      sh->s_new[ci] = (1.0 - lambda) * sh->cand_score[ci] + lambda * gamma;
    }
  }
  __syncthreads();
  const ArrScore new_score{sh->s_new};
  const AllMembers always;
  const int c = block_topk_set(new_score, always, n_cand, k, delta, sh->pick, sh->pick_score, &sh->sc);
  // pick holds positions in the candidate list (ascending position = ascending block id)
  for (int i = tid; i < c; i += kRankThreads) sh->pick[i] = sh->cand[sh->pick[i]];
  __syncthreads();
  return c;
}

__device__ __forceinline__ void rank_emit(int* idx, float* score, long long base, int k, int c, const RankShared* sh) {
  for (int i = threadIdx.x; i < k; i += kRankThreads) {
    idx[base + i] = i < c ? sh->pick[i] : -1;
    if (score) score[base + i] = i < c ? (float)sh->pick_score[i] : 0.f;
  }
}

__global__ void __launch_bounds__(kRankThreads) rank_kernel(const RankParams p, const QMeta meta) {
  __shared__ RankShared sh;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* gq = reinterpret_cast<double*>(smem_raw);               // [C] global query

  const int qi = blockIdx.x, tid = threadIdx.x;
  pdl_wait();                                                // the scores of the scan are complete
  const int C = p.C;
  long long tl = meta.t_limit[qi];
  if (tl > p.n_frm) tl = p.n_frm;
  if (tl < 0) tl = 0;
  const int n_frm = (int)tl;
  // segment u is visible when its last stored frame is: min((u+1)*fseg, n_stored) <= t_limit
  int n_seg = (int)(tl / p.fseg);
  if (tl == p.n_frm && (p.n_frm % p.fseg) != 0) n_seg += 1;
  if (n_seg > p.n_seg) n_seg = (int)p.n_seg;
  const double* sf = p.s_frm + (long long)qi * p.frm_stride;
  const double* ss = p.s_seg + (long long)qi * p.seg_stride;
  if (p.stage) {
    // every selection below scans the scores several times: do that out of shared memory
    double* st_f = gq + C;
    double* st_s = st_f + n_frm;
    for (int i = tid; i < n_frm; i += kRankThreads) st_f[i] = sf[i];
    for (int i = tid; i < n_seg; i += kRankThreads) st_s[i] = ss[i];
    __syncthreads();
    sf = st_f;
    ss = st_s;
  }
  const ArrScore seg_score{ss};
  const AllMembers always;
  const bool semi = p.mode == MUKV_RETR_SEMI;

  // ---- global query = mean of the top-N segment keys (stage 1 order)
  bool have_g = false;
  double gnorm = 0.0;
  if (semi) {
    const int N = p.top_n > 0 ? p.top_n : p.k_seg;
    const int n_top = block_topk_set(seg_score, always, n_seg, N, p.delta, sh.top, (double*)nullptr, &sh.sc);
    double part = 0.0;
    for (int c = tid; c < C; c += kRankThreads) {
      double t = 0.0;
      for (int i = 0; i < n_top; ++i) t += (double)p.seg_key[(long long)sh.top[i] * C + c];
      t = n_top > 0 ? t / (double)n_top : 0.0;
      gq[c] = t;
      part += t * t;
    }
    if (tid == 0) sh.gn = 0.0;
    __syncthreads();
    part = warp_sum(part);
    if ((tid & 31) == 0) atomicAdd(&sh.gn, part);
    __syncthreads();
    gnorm = sqrt(sh.gn);
    have_g = n_top > 0;
  }

  // ---- segments (the paper's lambda for them is 0: final = stage-1 top-k)
  const int c_seg = rank_level(ss, always, n_seg, p.k_seg, semi && p.lam_seg > 0.0, p.lam_seg, p.delta, p.seg_key, C, gq,
                               gnorm, have_g, &sh);
  rank_emit(p.seg_idx, p.seg_score, (long long)qi * p.k_seg, p.k_seg, c_seg, &sh);
  for (int i = tid; i < c_seg; i += kRankThreads) sh.sel_seg[i] = sh.pick[i];
  __syncthreads();

  // ---- frames
  // HIER: only what lies inside the selected segments is a candidate.  Those are few, so the ranking
  // runs over positions in the list "selected segments (ascending) x their frames" and maps the
  // winners back (ascending position = ascending frame).
  const int fseg = p.fseg;
  int c_frm;
  if (p.mode == MUKV_RETR_HIER) {
    auto frame_of = [&](int i) { return sh.sel_seg[i / fseg] * fseg + i % fseg; };
    auto score_h = [&](int i) { return sf[frame_of(i)]; };
    auto member_h = [&](int i) { return frame_of(i) < n_frm; };
    c_frm = block_topk_set(score_h, member_h, c_seg * fseg, p.k_frm, p.delta, sh.pick, sh.pick_score, &sh.sc);
    for (int i = tid; i < c_frm; i += kRankThreads) sh.pick[i] = frame_of(sh.pick[i]);
    __syncthreads();
  } else {
    c_frm = rank_level(sf, always, n_frm, p.k_frm, semi, p.lam_frm, p.delta, p.frame_key, C, gq, gnorm, have_g, &sh);
  }
  rank_emit(p.frm_idx, p.frm_score, (long long)qi * p.k_frm, p.k_frm, c_frm, &sh);
  __syncthreads();

  // ---- patch-level blocks: (frame, super patch) pairs that kept at least one token
  int c_pat = 0;
  if (p.k_pat > 0) {
    const int S = p.S;
    const int* cnt = p.patch_cnt;
    const double* spat = p.s_pat + (long long)qi * p.pat_stride;
    if (S > 0) {
      if (p.mode == MUKV_RETR_HIER) {
        const int per_seg = fseg * S;
        auto block_of = [&](int i) { return sh.sel_seg[i / per_seg] * per_seg + i % per_seg; };
        auto score_h = [&](int i) { return spat[block_of(i)]; };
        auto member_h = [&](int i) {
          const int b = block_of(i);
          return b < n_frm * S && cnt[b] > 0;
        };
        c_pat = block_topk_set(score_h, member_h, c_seg * per_seg, p.k_pat, p.delta, sh.pick, sh.pick_score, &sh.sc);
        for (int i = tid; i < c_pat; i += kRankThreads) sh.pick[i] = block_of(sh.pick[i]);
        __syncthreads();
      } else {
        auto member = [&](int b) { return cnt[b] > 0; };
        c_pat = rank_level(spat, member, n_frm * S, p.k_pat, semi, p.lam_pat, p.delta, p.patch_key, C, gq, gnorm, have_g,
                           &sh);
      }
    }
    rank_emit(p.pat_idx, p.pat_score, (long long)qi * p.k_pat, p.k_pat, c_pat, &sh);
  }
  if (tid == 0) {
    p.counts[p.counts_stride * qi] = c_seg;
    p.counts[p.counts_stride * qi + 1] = c_frm;
    if (p.counts_stride > 2) p.counts[p.counts_stride * qi + 2] = c_pat;
  }
}

// ------------------------------------------------------------------------------ Eq. 9
struct GatherParams {
  int nq, k_frm, L, kappa;
  long long run_bytes;                     // kappa * C * sizeof(T): one (frame, layer, K|V) run
  const int* frm_idx; const int* counts;
  const unsigned char* store; const long long* page_table; const int* kept_store;
  unsigned char* decode; long long decode_stride;
  int* tok_meta;
};

// unit = (question, plane = l*2+kv, slot): one contiguous run of the page goes to one contiguous
// run of the decode buffer.
__global__ void __launch_bounds__(256) gather_kernel(const GatherParams p) {
  const long long planes = (long long)p.L * 2;
  const long long n_units = (long long)p.nq * planes * p.k_frm;
  for (long long u = blockIdx.x; u < n_units; u += gridDim.x) {
    const int slot = (int)(u % p.k_frm);
    const long long r = u / p.k_frm;
    const int plane = (int)(r % planes);
    const int qi = (int)(r / planes);
    if (slot >= p.counts[2 * qi + 1]) continue;
    const int f = p.frm_idx[(long long)qi * p.k_frm + slot];
    const unsigned char* src = p.store + p.page_table[f] + (long long)plane * p.run_bytes;
    unsigned char* dst = p.decode + (long long)qi * p.decode_stride +
                         ((long long)plane * p.k_frm + slot) * p.run_bytes;
    const long long nvec = p.run_bytes >> 4;
    long long v = threadIdx.x;
    for (; v + 3 * 256 < nvec; v += 4 * 256) {
      uint4 x0 = ld_stream(src + (v << 4));
      uint4 x1 = ld_stream(src + ((v + 256) << 4));
      uint4 x2 = ld_stream(src + ((v + 512) << 4));
      uint4 x3 = ld_stream(src + ((v + 768) << 4));
      st_stream(dst + (v << 4), x0);
      st_stream(dst + ((v + 256) << 4), x1);
      st_stream(dst + ((v + 512) << 4), x2);
      st_stream(dst + ((v + 768) << 4), x3);
    }
    for (; v < nvec; v += 256) st_stream(dst + (v << 4), ld_stream(src + (v << 4)));
    if (plane == 0 && p.tok_meta) {
      for (int t = threadIdx.x; t < p.kappa; t += 256) {
        int* m = p.tok_meta + (((long long)qi * p.k_frm + slot) * p.kappa + t) * 2;
        m[0] = f;
        m[1] = p.kept_store[(long long)f * p.kappa + t];
      }
    }
  }
}

// ------------------------------------------------------------------------------ Eq. 9, all granularities
struct Gather3Params {
  int nq, k_seg, k_frm, k_pat, L, kappa, C, P, S, grid_width, patch_split;
  int tok_cap;                             // token slots per (layer, K|V) plane of a decode buffer
  int esize;                               // bytes per element of the store dtype
  const int* seg_idx; const int* frm_idx; const int* pat_idx; const int* counts;   // counts [nq][3]
  const unsigned char* store; const long long* page_table; const int* kept_store;
  const float* seg_entry;                  // [segments][L][2][C]
  const int* patch_cnt;                    // [frames][S]
  const int* kept_count;                   // [frames] tokens in a frame's page, or null: kappa in every page
  int kept_stride;                         // ints per frame in kept_store
  unsigned char* decode; long long decode_stride;
  int* ntok; int* tok_meta;
};

// one contiguous run, copied by a block of 256 threads with four 16-byte vectors in flight per thread
__device__ __forceinline__ void copy_run16(unsigned char* dst, const unsigned char* src, long long bytes) {
  const long long nvec = bytes >> 4;
  long long v = threadIdx.x;
  for (; v + 3 * 256 < nvec; v += 4 * 256) {
    const uint4 x0 = ld_stream(src + (v << 4));
    const uint4 x1 = ld_stream(src + ((v + 256) << 4));
    const uint4 x2 = ld_stream(src + ((v + 512) << 4));
    const uint4 x3 = ld_stream(src + ((v + 768) << 4));
    st_stream(dst + (v << 4), x0);
    st_stream(dst + ((v + 256) << 4), x1);
    st_stream(dst + ((v + 512) << 4), x2);
    st_stream(dst + ((v + 768) << 4), x3);
  }
  for (; v < nvec; v += 256) st_stream(dst + (v << 4), ld_stream(src + (v << 4)));
}

constexpr int kGatherListCap = 1024;       // rows of patch-level blocks listed at a time (>= MUKV_MAX_TOKENS)

// Units, per question and (layer, K|V) plane: k_frm frame runs (one contiguous run of the page each),
// then one unit for the summary tokens and the patch-level rows.  Token slots of a plane: summary
// tokens of the selected segments, kept tokens of the selected frames, kept tokens of the selected
// patch-level blocks.
template <typename T>
__global__ void __launch_bounds__(256) gather3_kernel(const Gather3Params p) {
  __shared__ int s_off[MUKV_MAX_TOPK + 1];                 // first row of each selected patch block
  __shared__ long long s_src[kGatherListCap];              // byte offset in the store of each listed row
  __shared__ int s_row0;
  const long long planes = (long long)p.L * 2;
  const int upp = p.k_frm + 1;                             // units per (question, plane)
  const long long n_units = (long long)p.nq * planes * upp;
  const long long row_bytes = (long long)p.C * p.esize;
  const long long run_bytes = (long long)p.kappa * row_bytes;
  for (long long u = blockIdx.x; u < n_units; u += gridDim.x) {
    const int slot = (int)(u % upp);
    const long long r = u / upp;
    const int plane = (int)(r % planes);
    const int qi = (int)(r / planes);
    const int c_seg = p.counts[3 * qi], c_frm = p.counts[3 * qi + 1], c_pat = p.counts[3 * qi + 2];
    unsigned char* dplane = p.decode + (long long)qi * p.decode_stride + (long long)plane * p.tok_cap * row_bytes;
    int* meta = p.tok_meta ? p.tok_meta + (long long)qi * p.tok_cap * 2 : nullptr;
    if (slot < p.k_frm) {
      if (slot >= c_frm) continue;
      const int f = p.frm_idx[(long long)qi * p.k_frm + slot];
      int row0 = c_seg + slot * p.kappa, rows = p.kappa;
      if (p.kept_count) {
        // pages of different lengths: this frame's rows start behind those of the frames before it
        __syncthreads();
        if (threadIdx.x == 0) {
          int off = c_seg;
          for (int i = 0; i < slot; ++i) off += p.kept_count[p.frm_idx[(long long)qi * p.k_frm + i]];
          s_row0 = off;
        }
        __syncthreads();
        row0 = s_row0;
        rows = p.kept_count[f];
      }
      const long long fbytes = (long long)rows * row_bytes;
      copy_run16(dplane + (long long)row0 * row_bytes, p.store + p.page_table[f] + (long long)plane * fbytes, fbytes);
      if (plane == 0 && meta) {
        for (int t = threadIdx.x; t < rows; t += blockDim.x) {
          meta[(row0 + t) * 2] = f;
          meta[(row0 + t) * 2 + 1] = p.kept_store[(long long)f * p.kept_stride + t];
        }
      }
      continue;
    }
    // ---- summary tokens: the segment's pooled entry of this plane, rounded to the store dtype
    for (int i = 0; i < c_seg; ++i) {
      const int useg = p.seg_idx[(long long)qi * p.k_seg + i];
      const float* e = p.seg_entry + ((long long)useg * planes + plane) * p.C;
      T* d = reinterpret_cast<T*>(dplane + (long long)i * row_bytes);
      for (int c = threadIdx.x; c < p.C; c += blockDim.x) {
        if constexpr (sizeof(T) == 2) d[c] = __float2bfloat16_rn(e[c]);
        else d[c] = e[c];
      }
      if (plane == 0 && meta && threadIdx.x == 0) { meta[i * 2] = -1 - useg; meta[i * 2 + 1] = -1; }
    }
    // ---- patch-level rows: block b = frame * S + super patch holds the frame's kept rows inside it
    __syncthreads();
    if (threadIdx.x == 0) {
      int off = c_seg + c_frm * p.kappa;
      if (p.kept_count) {
        off = c_seg;
        for (int i = 0; i < c_frm; ++i) off += p.kept_count[p.frm_idx[(long long)qi * p.k_frm + i]];
      }
      for (int i = 0; i < c_pat; ++i) {
        s_off[i] = off;
        off += p.patch_cnt[p.pat_idx[(long long)qi * p.k_pat + i]];
      }
      s_off[c_pat] = off;
      if (plane == 0 && p.ntok) p.ntok[qi] = off;
    }
    __syncthreads();
    // Patch blocks in batches whose rows fit the list.  One warp per block walks the frame's kept
    // list and notes where the rows of its super patch lie; then the whole block copies the rows.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    const int vpr = (int)(row_bytes >> 4);                 // 16-byte vectors per row
    for (int b0 = 0; b0 < c_pat;) {
      int b1 = b0 + 1;                                     // (one block has at most kappa <= list capacity rows)
      while (b1 < c_pat && s_off[b1 + 1] - s_off[b0] <= kGatherListCap) ++b1;
      for (int i = b0 + warp; i < b1; i += nwarp) {
        const int b = p.pat_idx[(long long)qi * p.k_pat + i];
        const int f = b / p.S, sp = b % p.S;
        const long long page = p.page_table[f] + (long long)plane * run_bytes;
        const int base = s_off[i] - s_off[b0], room = min(s_off[i + 1] - s_off[i], kGatherListCap - base);
        int pos = 0;
        for (int t0 = 0; t0 < p.kappa; t0 += 32) {
          const int t = t0 + lane;
          int tok = 0;
          bool hit = false;
          if (t < p.kappa) {
            tok = p.kept_store[(long long)f * p.kappa + t];
            hit = super_patch_index(tok, p.P, p.grid_width, p.patch_split) == sp;
          }
          const unsigned bal = __ballot_sync(kFull, hit);
          const int at = pos + __popc(bal & ((1u << lane) - 1u));
          if (hit && at < room) {
            s_src[base + at] = page + (long long)t * row_bytes;
            if (plane == 0 && meta) { meta[(s_off[i] + at) * 2] = f; meta[(s_off[i] + at) * 2 + 1] = tok; }
          }
          pos += __popc(bal);
        }
        // (a block with fewer rows than its count says, which a consistent store never has, repeats its first row)
        for (int at = pos + lane; at < room; at += 32) s_src[base + at] = page;
      }
      __syncthreads();
      const int nvec = min(s_off[b1] - s_off[b0], kGatherListCap) * vpr;
      unsigned char* dst = dplane + (long long)s_off[b0] * row_bytes;
      int v = threadIdx.x;
      for (; v + 3 * 256 < nvec; v += 4 * 256) {
        uint4 x[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int vv = v + k * 256;
          x[k] = ld_stream(p.store + s_src[vv / vpr] + ((long long)(vv % vpr) << 4));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) st_stream(dst + ((long long)(v + k * 256) << 4), x[k]);
      }
      for (; v < nvec; v += 256)
        st_stream(dst + ((long long)v << 4), ld_stream(p.store + s_src[v / vpr] + ((long long)(v % vpr) << 4)));
      __syncthreads();                                     // the list is rewritten by the next batch
      b0 = b1;
    }
    __syncthreads();
  }
}

}  // namespace mukv
