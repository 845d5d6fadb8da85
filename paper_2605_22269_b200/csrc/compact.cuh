// KV compaction into the paged store and block pooling (Sec. 3.3 "selected KV slices ... are
// stored", Sec. 3.4 Eq. 5), and the in-block selection that feeds it (Eq. 4 and the top-kappa rule).
//
// compact_kernel<T>: one thread block per (layer, K|V, frame).  The kappa kept rows of that
// plane (C = Hkv*D elements each, one contiguous run in the input) are copied, in ascending
// token order, to the frame's page; the same registers feed the mean over the kept rows.
// The last-layer key plane is summed in double: its mean is the retrieval key (Eq. 5) that
// later ranks blocks, so it is kept free of accumulation-order noise.
//
// Where do the kept ids come from?  After the persistent tensor-core scoring kernel every block
// works them out itself (sel_mode 1): it adds the scoring blocks' partial column sums of its frame
// in a fixed order, applies Eq. 4 and selects, all in single precision; the blocks of a frame run
// the same arithmetic on the same numbers, so they agree, and the one with plane 0 writes the ids
// and the index.  That costs a few microseconds at the start of each block, in parallel on the
// whole device, where a selection inside the scoring kernel left one block per frame working while
// all others had finished.  After the other scoring kernels the ids are read from the store
// (sel_mode 0).  Either way a frame whose lowest kept and highest dropped score are closer than
// tie_eps + flag_margin is skipped here: tail_kernel decides it in double precision and compacts it.
//
// What has to wait for every frame of the chunk:
// tail_kernel<T, NC>, launched behind compact_kernel: returns at once unless frames were flagged (about
// one chunk in fifty on the synthetic streams); then all its blocks first score those frames in double
// precision and select; once every block has finished that, the flagged frames are compacted and then
// the segment entries written, one plane per block.
// The segment entries (Eq. 5 at segment level; one (layer, K|V) plane per block, mean over the frames
// present) of the common case are not written by the call itself.  The next call pools them with a row
// of compact_kernel blocks that does not wait for its scoring kernel (CompactParams::prev), or the first
// reader launches segment_kernel for them.  (As the last launch of every call that kernel cost 6 us;
// pooling by the compaction block that finishes a plane last was measured too: the fence every block
// then needs before it signs off costs more than a launch.)
#pragma once
#include "common.cuh"
#include "score.cuh"

namespace mukv {

constexpr int kCompactThreads = 256;
static_assert(kCompactThreads == kScoreThreads, "tail_kernel runs the scoring and the compaction code in one block");

struct CompactParams {
  int L, kappa, C, P;             // C = Hkv*D elements per row
  int n_frames;
  long long first_frame;
  const void* k;                  // [L][n][P][C]
  const void* v;
  unsigned char* store;           // store base
  float* frame_entry;             // [max_frames][L][2][C]
  float* frame_key;               // [max_frames][C]
  double* frame_ksum;             // [max_frames][C]  exact sums of the last-layer kept keys
  long long* stat_refined;        // device counter
  int* n_flagged_next;            // the flagged count of the next chunk (the two chunks' counts alternate)
  int* tail_ctr;                  // [2] tail_kernel: blocks done with the double-precision scores / with everything
  // segment entries (Eq. 5 at segment level)
  int fseg;                       // frames per segment
  float* seg_entry;               // [max_segs][L][2][C]
  float* seg_key;                 // [max_segs][C]
  // selection
  // patch-level blocks (Sec. 3.2; Eq. 5 "similarly"): S = patch_split^2 super patches per frame
  int patch_split, grid_width;    // 0: no patch level
  float* patch_key;               // [max_frames][S][C]
  int* patch_cnt;                 // [max_frames][S]
  int pool_always;                // segment_kernel: pool whatever the flagged count says (the entries of an earlier call)
  // compact_kernel: with prev.n_frames > 0 the grid has one more row of blocks (the second one), which pools
  // the segment entries the previous call left to this one
  SegmentArgs prev;
  int sel_mode;                   // 0: kept ids are in the store; 1: select here from the partial sums;
                                  // 2: select here by the caller's scores; 3: ids and counts are in the store
                                  // (segment-level selection)
  const float* ext_scores;        // [n_frames][P] (sel_mode 2)
  const int* kept_count;          // [max_frames] (sel_mode 3: a frame's page holds that many tokens; ids in
                                  // kept_store with a stride of P), else null
  int ps_grid, ps_items, ps_ipf;  // the scoring launch: blocks, items, items per frame
  unsigned* sel_flag;             // [F] (epoch << 1 | risky) once the plane-0 block has published its frame's ids
  unsigned epoch;                 // number of this call, never repeated
  ScoreParams sp;                 // partial sums, Eq. 4 parameters, index and flag outputs
};

// a token id read back from memory, forced into the frame (row addresses are computed from it)
__device__ __forceinline__ int token_id(int id, int P) { return (unsigned)id < (unsigned)P ? id : 0; }

struct SelectScratch {
  unsigned mm[kCompactThreads / 32][4];   // per-warp min / max keys of the two signals
  int hist[256];
  int list[256];                  // keys of the scores in the bin that holds the kappa-th largest
  int cnt[kCompactThreads / 32][4];
  unsigned ab[kCompactThreads / 32][2];
  int bin, rank, n_list;
  float tau;
  // scratch of select_by_score (ranking by the caller's scores)
  double sc64[MUKV_MAX_TOKENS];
  double misc64[4 * (kCompactThreads / 32)];
  int cnt64[kCompactThreads / 32 + 1];
};

// Eq. 4 and the top-kappa rule for frame f from the partial sums of the persistent scoring kernel,
// run by a whole block of kCompactThreads threads (thread t owns token t; P <= 256).  The kept ids
// go to s_kept in ascending order; with `write` also to the store and to the caller's outputs.
// Returns true when single precision cannot decide the frame safely (see select_frame): nothing
// of the frame may then be used, and with `write` the frame has been put on the flagged list.
// Everything is single precision; scores lie in [0, 1], so their bit patterns order like the
// values and the reductions run on them as integers.
__device__ inline bool select_from_partials(const CompactParams& p, int f, bool write, int* s_kept, SelectScratch* sc) {
  const ScoreParams& sp = p.sp;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NW = kCompactThreads / 32;
  const int P = sp.P, Hkv = sp.Hkv * sp.Ls, kappa = sp.kappa;   // key heads of all scoring layers
  const bool valid = tid < P;
  float att = 0.f, fft = 0.f;
  if (valid) {
    // the scoring blocks' column sums, added in block order
    const int c_first = share_owner((unsigned)(f * p.ps_ipf), (unsigned)p.ps_items, (unsigned)p.ps_grid);
    const int c_last = share_owner((unsigned)((f + 1) * p.ps_ipf - 1), (unsigned)p.ps_items, (unsigned)p.ps_grid);
    const float* cp = reinterpret_cast<const float*>(sp.colsum_part) + tid;
    const float* fp = reinterpret_cast<const float*>(sp.ifft_part) + (long long)f * Hkv * P + tid;
    // all loads of the common case (up to 16 blocks per frame, up to 8 key heads) are in flight together
    float x[16], y[8];
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = c_first + i <= c_last ? __ldcg(cp + (long long)(c_first + i + f) * P) : 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = i < Hkv ? __ldcg(fp + (long long)i * P) : 0.f;
#pragma unroll
    for (int w = 8; w >= 1; w >>= 1)
#pragma unroll
      for (int i = 0; i < w; ++i) x[i] += x[i + w];
#pragma unroll
    for (int w = 4; w >= 1; w >>= 1)
#pragma unroll
      for (int i = 0; i < w; ++i) y[i] += y[i + w];
    float a32 = x[0], f32 = y[0];
    for (int cc = c_first + 16; cc <= c_last; ++cc) a32 += __ldcg(cp + (long long)(cc + f) * P);
    for (int g = 8; g < Hkv; ++g) f32 += __ldcg(fp + (long long)g * P);
    att = a32 * (1.f / (float)((long long)sp.Hq * sp.Ls * P));
    fft = f32 * (1.f / (float)((long long)Hkv * sp.D));
  }
  // ---- min / max of both signals over the frame (both are sums of non-negative terms)
  {
    const unsigned ka = __float_as_uint(att), kf = __float_as_uint(fft);
    const unsigned v0 = __reduce_min_sync(kFull, valid ? ka : 0xffffffffu), v1 = __reduce_max_sync(kFull, valid ? ka : 0u);
    const unsigned v2 = __reduce_min_sync(kFull, valid ? kf : 0xffffffffu), v3 = __reduce_max_sync(kFull, valid ? kf : 0u);
    if (lane == 0) { sc->mm[warp][0] = v0; sc->mm[warp][1] = v1; sc->mm[warp][2] = v2; sc->mm[warp][3] = v3; }
    sc->hist[tid] = 0;
    if (tid == 0) sc->n_list = 0;
  }
  // a frame with a score that is not a number has no ranking: every score counts as 0 below, so
  // that the lowest kappa ids are kept (every block of the frame sees the same sums and agrees)
  const bool bad = __syncthreads_or(valid && !(isfinite(att) && isfinite(fft))) != 0;
  const int wl = lane < NW ? lane : 0;                     // lanes past the warp count repeat warp 0
  const unsigned m0 = __reduce_min_sync(kFull, sc->mm[wl][0]), m1 = __reduce_max_sync(kFull, sc->mm[wl][1]);
  const unsigned m2 = __reduce_min_sync(kFull, sc->mm[wl][2]), m3 = __reduce_max_sync(kFull, sc->mm[wl][3]);
  const float amin = __uint_as_float(m0), amax = __uint_as_float(m1);
  const float fmin_ = __uint_as_float(m2), fmax_ = __uint_as_float(m3);
  // ---- Eq. 4
  // (one reciprocal per signal, the same in every thread, instead of a division per token)
  const float inv_a = (amax == amin) ? 0.f : 1.f / (amax - amin);
  const float inv_f = (fmax_ == fmin_) ? 0.f : 1.f / (fmax_ - fmin_);
  const float an = (att - amin) * inv_a;
  float fn = (fft - fmin_) * inv_f;
  if (sp.keep_low) fn = 1.f - fn;
  const float s = bad ? 0.f : sp.alpha * an + (1.f - sp.alpha) * fn;
  const int key = __float_as_int(s);
  // ---- tau = kappa-th largest score: a 256-bin histogram finds its bin, the scores of that bin
  // are ranked among themselves
  int bin = (int)(s * 256.f);
  bin = bin < 0 ? 0 : (bin > 255 ? 255 : bin);
  if (valid) atomicAdd(&sc->hist[bin], 1);
  __syncthreads();
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
    if (above < kappa && kappa <= above + T) {           // true for exactly one lane
      int r = kappa - above, b = 7;
      for (; b > 0; --b) {
        if (r <= c[b]) break;
        r -= c[b];
      }
      sc->bin = 8 * lane + b;
      sc->rank = r;
    }
  }
  __syncthreads();
  const bool member = valid && bin == sc->bin;
  if (member) sc->list[atomicAdd(&sc->n_list, 1)] = key;
  __syncthreads();
  if (member) {
    const int n = sc->n_list, r = sc->rank;
    int gt = 0, ge = 0;
    for (int i = 0; i < n; ++i) {
      const int o = sc->list[i];
      gt += (o > key);
      ge += (o >= key);
    }
    if (gt < r && r <= ge) sc->tau = s;                  // every writer holds the same value
  }
  __syncthreads();
  const float tau = sc->tau;
  const float delta = sp.tie_eps;
  const bool sure = valid && (s > tau + delta);
  const bool band = valid && !sure && (s >= tau - delta);
  const unsigned lt = (1u << lane) - 1u;
  const unsigned b_sure = __ballot_sync(kFull, sure), b_band = __ballot_sync(kFull, band);
  if (lane == 0) { sc->cnt[warp][0] = __popc(b_sure); sc->cnt[warp][1] = __popc(b_band); }
  __syncthreads();
  int n_sure = 0, band_rank = __popc(b_band & lt);
#pragma unroll
  for (int w = 0; w < NW; ++w) {
    n_sure += sc->cnt[w][0];
    if (w < warp) band_rank += sc->cnt[w][1];
  }
  const bool keep = sure || (band && band_rank < kappa - n_sure);
  const unsigned b_keep = __ballot_sync(kFull, keep);
  {
    // lowest kept and highest dropped score, for the safety test below
    const unsigned ks = (unsigned)key;
    const unsigned a = __reduce_min_sync(kFull, keep ? ks : 0xffffffffu);
    const unsigned b = __reduce_max_sync(kFull, (valid && !keep) ? ks : 0u);
    if (lane == 0) { sc->cnt[warp][2] = __popc(b_keep); sc->ab[warp][0] = a; sc->ab[warp][1] = b; }
  }
  __syncthreads();
  int pos = __popc(b_keep & lt);
  unsigned ka = 0xffffffffu, kb = 0u;
  bool any_dropped = false;
#pragma unroll
  for (int w = 0; w < NW; ++w) {
    if (w < warp) pos += sc->cnt[w][2];
    ka = min(ka, sc->ab[w][0]);
    kb = max(kb, sc->ab[w][1]);
  }
  any_dropped = kappa < P;
  // does single precision decide this frame safely?  (see select_frame)
  const float a = __uint_as_float(ka), b = any_dropped ? __uint_as_float(kb) : -3.0e38f;
  bool risky = any_dropped && (a - b <= delta + sp.flag_margin);
  const float aabs = fmaxf(amax, -amin), fabs_ = fmaxf(fmax_, -fmin_);
  if (amax != amin && (amax - amin) < sp.flat_ratio * aabs && sp.alpha != 0.f) risky = true;
  if (fmax_ != fmin_ && (fmax_ - fmin_) < sp.flat_ratio * fabs_ && sp.alpha != 1.f) risky = true;
  if (bad) risky = false;                                 // double precision would not rank it either
  if (keep) s_kept[pos] = tid;
  if (write) {
    const long long f_abs = sp.first_frame + f;
    if (keep) {
      sp.kept_store[f_abs * kappa + pos] = tid;
      if (sp.kept_out) sp.kept_out[(long long)f * kappa + pos] = tid;
    }
    if (sp.scores_out && valid) {
      const long long np = (long long)sp.n_frames * P;
      sp.scores_out[0 * np + (long long)f * P + tid] = att;
      sp.scores_out[1 * np + (long long)f * P + tid] = fft;
      sp.scores_out[2 * np + (long long)f * P + tid] = s;
    }
    if (tid == 0) {
      sp.frame_ts[f_abs] = f_abs;
      sp.page_table[f_abs] = sp.pages_off + f_abs * sp.page_bytes;
      if (risky) sp.flagged[atomicAdd(sp.n_flagged, 1)] = f;
      if (bad && sp.status) atomicCAS(sp.status, 0, kStatusNonFinite);
    }
  }
  __syncthreads();
  return risky;
}

__device__ __forceinline__ SegmentArgs segment_args(const CompactParams& p) {
  SegmentArgs a;
  a.L = p.L; a.kappa = p.kappa; a.C = p.C; a.fseg = p.fseg; a.n_frames = p.n_frames; a.first_frame = p.first_frame;
  a.frame_entry = p.frame_entry; a.frame_ksum = p.frame_ksum; a.seg_entry = p.seg_entry; a.seg_key = p.seg_key;
  a.kept_count = p.kept_count;
  return a;
}

// Segment entries (Eq. 5 at segment level) of one (layer, K|V) plane for every segment the chunk
// touches: mean over the frames present, added in frame order.  Run by one whole block.  The loads
// of up to 16 frames (and, in single precision, of two columns) are in flight together: the
// work is a chain of L2 round trips and little else.
__device__ __noinline__ void compact_segment_plane(const SegmentArgs p, int l, int kv) {
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
    if (p.kept_count) {
      // frames keep different numbers of tokens (segment-level selection): the mean over all kept
      // tokens of the segment is the count-weighted mean of the frame entries
      for (int col = tid; col < C; col += kCompactThreads) {
        long long n_tok = 0;
        double td = 0.0;
        float tf = 0.f;
        for (long long ff = t0; ff < t1; ff += 16) {
          int cn[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) cn[i] = ff + i < t1 ? __ldcg(p.kept_count + ff + i) : 0;
          if (exact) {
            double x[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) x[i] = ff + i < t1 ? __ldcg(p.frame_ksum + (ff + i) * C + col) : 0.0;
#pragma unroll
            for (int i = 0; i < 16; ++i) td += x[i];
          } else {
            float x[16];
#pragma unroll
            for (int i = 0; i < 16; ++i)
              x[i] = ff + i < t1 ? __ldcg(p.frame_entry + (((ff + i) * p.L + l) * 2 + kv) * C + col) : 0.f;
#pragma unroll
            for (int i = 0; i < 16; ++i) tf += (float)cn[i] * x[i];
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) n_tok += cn[i];
        }
        if (exact) {
          const float m = n_tok ? (float)(td / (double)n_tok) : 0.f;
          p.seg_key[u * C + col] = m;
          p.seg_entry[((u * p.L + l) * 2 + kv) * C + col] = m;
        } else {
          p.seg_entry[((u * p.L + l) * 2 + kv) * C + col] = n_tok ? tf / (float)n_tok : 0.f;
        }
      }
      continue;
    }
    if (exact) {
      for (int col = tid; col < C; col += kCompactThreads) {
        double t = 0.0;
        for (long long ff = t0; ff < t1; ff += 16) {
          double x[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) x[i] = ff + i < t1 ? __ldcg(p.frame_ksum + (ff + i) * C + col) : 0.0;
#pragma unroll
          for (int i = 0; i < 16; ++i) t += x[i];
        }
        const float m = (float)(t / ((double)nf * (double)kappa));
        p.seg_key[u * C + col] = m;
        p.seg_entry[((u * p.L + l) * 2 + kv) * C + col] = m;
      }
    } else {
      for (int col = tid; col < C; col += 2 * kCompactThreads) {
        const int col1 = col + kCompactThreads;
        const bool two = col1 < C;
        float ta = 0.f, tb = 0.f;
        for (long long ff = t0; ff < t1; ff += 16) {
          float xa[16], xb[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float* src = p.frame_entry + (((ff + i) * p.L + l) * 2 + kv) * C;
            xa[i] = ff + i < t1 ? __ldcg(src + col) : 0.f;
            xb[i] = (two && ff + i < t1) ? __ldcg(src + col1) : 0.f;
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) { ta += xa[i]; tb += xb[i]; }
        }
        float* dst = p.seg_entry + ((u * p.L + l) * 2 + kv) * C;
        dst[col] = ta / (float)nf;
        if (two) dst[col1] = tb / (float)nf;
      }
    }
  }
}

struct CompactScratch {
  float red[kCompactThreads * 8];
  double red64[kCompactThreads * 8];
  int kept[MUKV_MAX_TOKENS];
};

// Copies the kappa kept rows (ids in sc->kept, ascending) of plane (l, kv) of chunk frame f to the
// frame's page (planes of kappa rows each, starting at `page`) and writes the plane's frame entry
// (Eq. 5; zeros for a frame that keeps nothing).  Run by a whole block.
// NV = 16-byte vectors per row; the block covers 256/NV rows per pass.
template <typename T>
__device__ inline void compact_plane(const CompactParams& p, int plane, int f, CompactScratch* sc, int kappa,
                                     unsigned char* page) {
  constexpr int VE = 16 / sizeof(T);
  const int tid = threadIdx.x;
  const int l = plane >> 1, kv = plane & 1;
  const long long f_abs = p.first_frame + f;
  const int C = p.C;
  const int NV = C / VE;                        // vectors per row (power of two, <= 256)
  const int rows_per_pass = kCompactThreads / NV;
  const T* src_base = reinterpret_cast<const T*>(kv ? p.v : p.k) + ((long long)l * p.n_frames + f) * p.P * C;
  T* dst_base = reinterpret_cast<T*>(page) + (long long)plane * kappa * C;
  const int c = tid % NV, r0 = tid / NV;
  const bool exact = (l == p.L - 1) && (kv == 0);
  float acc[VE];
  double acc64[VE];
#pragma unroll
  for (int e = 0; e < VE; ++e) { acc[e] = 0.f; acc64[e] = 0.0; }
  // Rows in flight per thread.  With 4 row groups per pass, 5 covers the 49 kept rows of the 7B shape in
  // three trips (20 + 20 + 9) where 4 needs a fourth trip for a single row; the kernel then takes 80
  // registers and three blocks per SM instead of four, which measured faster all the same.
  constexpr int kUnroll = 5;
  for (int r = r0; r < kappa; r += rows_per_pass * kUnroll) {
    uint4 x[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int rr = r + u * rows_per_pass;
      if (rr < kappa) x[u] = ld_stream(src_base + (long long)sc->kept[rr] * C + c * VE);
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
    for (int i = 0; i < VE; ++i) sc->red64[tid * VE + i] = acc64[i];
  } else {
#pragma unroll
    for (int i = 0; i < VE; ++i) sc->red[tid * VE + i] = acc[i];
  }
  __syncthreads();
  float* fe = p.frame_entry + ((f_abs * p.L + l) * 2 + kv) * C;
  for (int col = tid; col < C; col += kCompactThreads) {
    const int cv = col / VE, ce = col % VE;
    if (exact) {
      double t = 0.0;
      for (int g = 0; g < rows_per_pass; ++g) t += sc->red64[(g * NV + cv) * VE + ce];
      p.frame_ksum[f_abs * C + col] = t;
      const float m = kappa ? (float)(t / (double)kappa) : 0.f;
      fe[col] = m;
      p.frame_key[f_abs * C + col] = m;
    } else {
      float t = 0.f;
      for (int g = 0; g < rows_per_pass; ++g) t += sc->red[(g * NV + cv) * VE + ce];
      fe[col] = kappa ? t / (float)kappa : 0.f;
    }
  }
}

// Patch-level block keys of chunk frame f (Eq. 5 on the kept tokens of each super patch): mean of
// their last-layer keys, summed in double like the frame key; kept ids in sc->kept.  Run by a
// whole block; the kept rows are first grouped by super patch, then every thread sums its channels
// of each group in ascending row order.  sc->red is used as scratch.
template <typename T>
__device__ inline void pool_patches(const CompactParams& p, int f, CompactScratch* sc) {
  constexpr int EW = ElemTraits<T>::kPerWord;
  const int tid = threadIdx.x;
  const int S = p.patch_split * p.patch_split, C = p.C, kappa = p.kappa;
  const long long f_abs = p.first_frame + f;
  int* order = reinterpret_cast<int*>(sc->red);          // kept ids grouped by super patch, ascending inside a group
  int* start = order + MUKV_MAX_TOKENS;                  // [S + 1] first entry of every group
  int* sp_of = start + 32;                               // [kappa] super patch of each kept row
  static_assert(sizeof(sc->red) >= (2 * MUKV_MAX_TOKENS + 32) * sizeof(int), "scratch too small");
  static_assert(MUKV_MAX_PATCH_SPLIT * MUKV_MAX_PATCH_SPLIT < 32, "group starts do not fit");
  __syncthreads();
  for (int r = tid; r < kappa; r += kCompactThreads) sp_of[r] = super_patch_index(sc->kept[r], p.P, p.grid_width, p.patch_split);
  __syncthreads();
  if (tid <= S) {
    int c = 0;
    for (int r = 0; r < kappa; ++r) c += (sp_of[r] < tid);
    start[tid] = c;
  }
  __syncthreads();
  for (int r = tid; r < kappa; r += kCompactThreads) {
    const int s = sp_of[r];
    int pos = start[s];
    for (int q = 0; q < r; ++q) pos += (sp_of[q] == s);
    order[pos] = sc->kept[r];
  }
  __syncthreads();
  // a thread owns one 32-bit word of the row (one or two channels); eight rows are in flight at a time
  const int wpr = C / EW;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(reinterpret_cast<const T*>(p.k) +
                                                          ((long long)(p.L - 1) * p.n_frames + f) * p.P * C);
  for (int w = tid; w < wpr; w += kCompactThreads) {
    for (int sp = 0; sp < S; ++sp) {
      const int b = start[sp], e = start[sp + 1];
      double t0 = 0.0, t1 = 0.0;
      for (int i = b; i < e; i += 8) {
        uint32_t x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = i + u < e ? __ldg(src + (long long)order[i + u] * wpr + w) : 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) {                      // (a zero word adds +0.0)
          if (EW == 2) {
            t0 += (double)bf16_lo(x[u]);
            t1 += (double)bf16_hi(x[u]);
          } else {
            t0 += (double)__uint_as_float(x[u]);
          }
        }
      }
      const int cnt = e - b;
      float* dst = p.patch_key + ((f_abs * S) + sp) * C + (long long)w * EW;
      dst[0] = cnt ? (float)(t0 / (double)cnt) : 0.f;
      if (EW == 2) dst[1] = cnt ? (float)(t1 / (double)cnt) : 0.f;
    }
  }
  if (tid < S) p.patch_cnt[f_abs * S + tid] = start[tid + 1] - start[tid];
}

// is chunk frame f on the flagged list (of n entries)?
__device__ __forceinline__ bool frame_is_flagged(const int* flagged, int n, int f) {
  bool hit = false;
  for (int i = 0; i < n; ++i) hit |= (__ldcg(flagged + i) == f);
  return hit;
}

template <typename T>
__global__ void __launch_bounds__(kCompactThreads, 3) compact_kernel(const CompactParams p) {
  __shared__ CompactScratch cs;
  __shared__ SelectScratch ss;
  __shared__ unsigned s_seen;
  const int tid = threadIdx.x;
  // frame is the fast block index: the blocks that start first cover the low planes of every frame,
  // the plane-0 blocks among them
  const int f = blockIdx.x;
  // block row -> plane l*2 + kv; with a patch level its blocks (plane 2L) sit in row 1, so that they run
  // in the first wave beside the copy blocks instead of alone at the end
  int row = blockIdx.y;
  if (p.prev.n_frames > 0) {
    if (row == 1) {
      // nothing of this call is needed for the entries of the previous one: no wait for the scoring kernel
      for (int pl = blockIdx.x; pl < 2 * p.prev.L; pl += gridDim.x) compact_segment_plane(p.prev, pl >> 1, pl & 1);
      return;
    }
    if (row > 1) --row;
  }
  const int plane = p.patch_split > 0 && row >= 1 ? (row == 1 ? 2 * p.L : row - 1) : row;
  pdl_wait();
  pdl_trigger();
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) *p.n_flagged_next = 0;
  const long long f_abs = p.first_frame + f;
  int kappa_f = p.kappa;
  unsigned char* page = p.store + p.sp.pages_off + f_abs * p.sp.page_bytes;
  bool risky;
  if (p.sel_mode == 1) {
    // A block that starts after its frame's plane-0 block has published the ids (the blocks beyond
    // the first wave do) reads them; every other block selects itself.  Nobody waits.
    if (tid == 0) {
      unsigned v = 0u;
      if (plane != 0) {
        v = *reinterpret_cast<volatile unsigned*>(p.sel_flag + f);
        __threadfence();
      }
      s_seen = v;
    }
    __syncthreads();
    const unsigned seen = s_seen;
    if ((seen >> 1) == p.epoch) {
      risky = (seen & 1u) != 0u;
      for (int r = tid; r < p.kappa; r += kCompactThreads) cs.kept[r] = token_id(__ldcg(p.sp.kept_store + f_abs * p.kappa + r), p.P);
      __syncthreads();
    } else {
      risky = select_from_partials(p, f, plane == 0, cs.kept, &ss);
      if (plane == 0) {
        __threadfence();                        // this thread's ids are visible before the flag is
        __syncthreads();
        if (tid == 0) *reinterpret_cast<volatile unsigned*>(p.sel_flag + f) = (p.epoch << 1) | (risky ? 1u : 0u);
      }
    }
  } else if (p.sel_mode == 2) {
    // Ranking by numbers the caller supplies (no Eq. 1-4): every block ranks its frame itself, in
    // double precision on exact inputs, so nothing is ever too close to call; plane 0 writes the ids.
    double sx[1] = {tid < p.P ? (double)__ldg(p.ext_scores + (long long)f * p.P + tid) : 0.0};
    const bool bad = __syncthreads_or(tid < p.P && !isfinite(sx[0])) != 0;
    if (bad) sx[0] = 0.0;
    bool keep[1];
    select_by_score<1>(p.sp, f, sx, plane == 0, cs.kept, keep, ss.sc64, ss.cnt64, ss.misc64);
    if (bad && plane == 0 && tid == 0 && p.sp.status) atomicCAS(p.sp.status, 0, kStatusNonFinite);
    risky = false;
    __syncthreads();
  } else if (p.sel_mode == 3) {
    kappa_f = __ldcg(p.kept_count + f_abs);
    kappa_f = kappa_f < 0 ? 0 : (kappa_f > p.P ? p.P : kappa_f);
    page = p.store + __ldcg(p.sp.page_table + f_abs);
    for (int r = tid; r < kappa_f; r += kCompactThreads) cs.kept[r] = token_id(__ldcg(p.sp.kept_store + f_abs * p.P + r), p.P);
    risky = false;
    __syncthreads();
  } else {
    risky = frame_is_flagged(p.sp.flagged, *p.sp.n_flagged, f);
    for (int r = tid; r < p.kappa; r += kCompactThreads) cs.kept[r] = token_id(p.sp.kept_store[f_abs * p.kappa + r], p.P);
    __syncthreads();
  }
  if (risky) return;
  if (plane < 2 * p.L) compact_plane<T>(p, plane, f, &cs, kappa_f, page);
  else pool_patches<T>(p, f, &cs);
}

// Bounded wait until *ctr reaches `target` (other blocks of the same grid add to it; the grid is
// sized so that all its blocks are resident).  False after about 1.5 s.
__device__ inline bool wait_counter(const int* ctr, int target) {
  const volatile int* c = ctr;
  unsigned long long t0 = 0;
  for (long long spin = 0;; ++spin) {
    if (*c >= target) return true;
    if ((spin & 63) == 63) {
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (t0 == 0) t0 = now;
      else if (now - t0 > 1500000000ull) return false;
    }
    __nanosleep(200);
  }
}

constexpr int kStatusTailWait = 6;   // tail_kernel: the wait for the double-precision scores ran out

// tail_kernel: see the head of this file.  sp is the scoring configuration of the double-precision
// pass (its partial-sum buffers, refine = 1); the grid is a multiple of nothing in particular: blocks
// stride over the work, and the host keeps the grid within what is resident at once.
// segment_kernel: one block per (layer, K|V) plane writes that plane of every segment entry the frames
// first_frame .. first_frame + n_frames - 1 touch.  Launched for the chunk of an earlier call when
// something is about to read its segment entries (pool_always = 1); without pool_always it leaves
// everything to tail_kernel when frames were flagged.
__global__ void __launch_bounds__(kCompactThreads) segment_kernel(const CompactParams p) {
  pdl_wait();
  pdl_trigger();
  if (!p.pool_always && *p.sp.n_flagged != 0) return;
  for (int plane = blockIdx.x; plane < 2 * p.L; plane += gridDim.x)
    compact_segment_plane(segment_args(p), plane >> 1, plane & 1);
}

template <typename T, int NC>
__global__ void __launch_bounds__(kScoreThreads, 2) tail_kernel(const ScoreParams sp, const CompactParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ CompactScratch cs;
  __shared__ int s_ok;
  const int tid = threadIdx.x;
  pdl_wait();
  const int n_fl = *sp.n_flagged;
  if (n_fl == 0) return;                        // the common case: the next call pools this chunk's segment entries
  // ---- scores of the flagged frames in double precision; the block that finishes a frame last selects
  const int units = sp.Ls * sp.Hq * sp.row_split;
  for (int w = blockIdx.x; w < n_fl * units; w += gridDim.x) {
    const int u = w % units;
    score_frame_block<T, double, NC>(sp, u / sp.row_split, u % sp.row_split, sp.flagged[w / units], smem_raw);
    __syncthreads();
  }
  // ---- every block waits for all selections
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    atomicAdd(p.tail_ctr, 1);
    s_ok = wait_counter(p.tail_ctr, (int)gridDim.x) ? 1 : 0;
    __threadfence();
  }
  __syncthreads();
  if (!s_ok) {
    if (tid == 0 && sp.status) atomicCAS(sp.status, 0, kStatusTailWait);
  } else {
    // ---- the flagged frames' compaction, then the segment entries, plane by plane
    const int n_planes = 2 * p.L + (p.patch_split > 0 ? 1 : 0);
    for (int plane = blockIdx.x; plane < n_planes; plane += gridDim.x) {
      for (int i = 0; i < n_fl; ++i) {
        const int f = sp.flagged[i];
        const long long f_abs = p.first_frame + f;
        __syncthreads();
        for (int r = tid; r < p.kappa; r += kCompactThreads) cs.kept[r] = token_id(__ldcg(sp.kept_store + f_abs * p.kappa + r), p.P);
        __syncthreads();
        if (plane < 2 * p.L) compact_plane<T>(p, plane, f, &cs, p.kappa, p.store + sp.pages_off + f_abs * sp.page_bytes);
        else pool_patches<T>(p, f, &cs);
      }
      if (plane >= 2 * p.L) continue;
      __threadfence();                          // the frame entries just written are read below by other threads
      __syncthreads();
      compact_segment_plane(segment_args(p), plane >> 1, plane & 1);
    }
  }
  // ---- the block that leaves last resets the counters and adds to the statistics
  __syncthreads();
  if (tid == 0) {
    const int old = atomicAdd(p.tail_ctr + 1, 1);
    if (old == (int)gridDim.x - 1) {
      *p.stat_refined += n_fl;
      p.tail_ctr[0] = 0;
      p.tail_ctr[1] = 0;
    }
  }
}

}  // namespace mukv
