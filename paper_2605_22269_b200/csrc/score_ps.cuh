// Persistent, warp-specialised tensor-core scoring of a bf16 chunk (Sec. 3.3, Eq. 1-4).
//
// score_ps_kernel: one block of 640 threads per SM.  The chunk is a list of items, ordered by
// (frame, scoring layer, key head): first the DFT row tiles of that head's keys (Eq. 2-3), then the attention
// row tiles (Eq. 1; the G query heads of the group are flattened with the tokens into rows: one
// TMA box of tpt = 128/G tokens x G heads x 64 channels lands as up to 128 rows of a K-major,
// 128-byte-swizzled operand).  Each block takes a contiguous share of the list.
//
//   warp 0      TMA producer.  The key tile K_g of a (frame, head) goes to one of two buffers when
//               the head changes; everything else streams through a ring of 32 KB operand stages:
//               one Q row tile per attention item, the three bf16 terms of the DFT matrix (read
//               from L2) per DFT item.
//   warp 1      issues tcgen05.mma into one of two 256-column accumulators in tensor memory and
//               commits to the barriers that free the stages and the key buffers.
//   warps 4-19  epilogue (warps 2-3 only hand their registers over).  Four warps share each 32-lane quarter of the accumulator and split its
//               columns.  Attention item: one sweep takes a running row maximum, writes
//               exp(z - running max) back into tensor memory and keeps the row sum (rescaled when
//               the maximum grows); the warps of a row exchange (max, sum) through shared
//               memory; a second sweep adds e * 2^(ref - max) / sum to per-column accumulators in
//               registers.  The 32 rows of a warp are added only when the block leaves a frame
//               (shuffle butterfly), so the per-tile cost is one fused multiply-add per logit.
//               DFT item: magnitudes of the D bins of each key vector, summed.
//
// Per frame, every block that worked on it stores its column sums in a slot of its own (slot
// index = block + frame).  Eq. 4 and the selection are left to the kernel that follows
// (compact_kernel adds the slots in a fixed order): done here, by the block that finishes a frame
// last, they kept one block per frame busy for microseconds after all others had finished.
// All mbarrier waits are bounded; a wait that runs out makes the role record a code in the status
// word; the producer and the MMA issuer then leave their loops, the epilogue warps go on without
// waiting (their reads stay inside the accumulators).
#pragma once
#include "common.cuh"
#include "score.cuh"
#include "tc.cuh"

namespace mukv {

constexpr int kPsThreads = 640;           // warpgroup 0: control, warpgroups 1-4: epilogue
constexpr int kPsEpiThreads = 512;
constexpr int kPsSplit = 4;                // warps that share a row (32-lane quarter), each a column range
constexpr int kPsEpiOff = 128;             // first epilogue thread
constexpr int kPsMiscBytes = 12800 + 8192;
constexpr int kPsMaxBlocks = 256;          // bound on the grid (slots of partial sums)
constexpr int kPsAccCols = 64;             // accumulator columns per epilogue thread: P <= 4 * 64
// Twenty warps put five on each scheduler, whose 16 K registers allow 96 per thread at launch.
// The control warpgroup then gives registers back (setmaxnreg.dec) and the four epilogue warpgroups
// take them.  The hand-over has to balance: what the control warpgroup releases, 128 * (96 - 32),
// is all the epilogue warpgroups can claim, 512 * (112 - 96); a larger claim would block forever.
constexpr int kPsCtrlRegs = 32;
constexpr int kPsEpiRegs = 112;
static_assert(128 * (96 - kPsCtrlRegs) >= 512 * (kPsEpiRegs - 96), "register hand-over does not balance");
typedef NamedGroup<5, kPsEpiThreads, kPsEpiOff> PsEpiGroup;

struct ScorePsParams {
  ScoreParams sp;            // colsum_part: float [grid + n_frames][P] slots, ifft_part: float [F][Hkv][P]
  int tiles, tpt, npad, n_mt;  // npad: rows of a key tile = columns of an attention product
  // cached keys the queries also attend to (Sec. 3.2): rows own_rows + w * past_pad .. + kappa of the key
  // tile hold the kept keys of frame past_first + w (w < n_past), read from that frame's page
  int own_rows;              // rows the box of the frame's own keys covers (P rounded up to 8 with cached keys, else npad)
  int n_past, past_pad, kappa;
  int past_plane0;           // plane (layer * 2) of the first scoring layer's keys in a page
  long long past_first;
  int n_stages;              // operand stages in the ring (2 .. kPsMaxStages)
  int n_items;               // n_frames * Ls * Hkv * (n_mt + tiles)
  float exp2_scale;          // log2(e) / sqrt(D)
  int* status;
};

constexpr int kPsMaxStages = 6;
// two key buffers + n_stages operand stages + scratch (+ slack to align the tiles to 1024 bytes)
__host__ inline size_t score_ps_smem_bytes(int npad, int D, int n_stages) {
  const size_t KB = D / 64;
  return 2 * KB * (size_t)npad * 128 + (size_t)n_stages * KB * 128 * 128 + kPsMiscBytes + 1024;
}
__host__ inline int score_ps_stages(int npad, int D, size_t limit) {
  int n = kPsMaxStages;
  while (n >= 2 && score_ps_smem_bytes(npad, D, n) > limit) --n;
  return n;                  // < 2: the kernel does not fit
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// v[c] summed over the 32 lanes of the warp, for 32 columns c at once: lane c ends with column c.
__device__ __forceinline__ float warp_column_sums(float (&v)[32], int lane) {
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) {
    const bool up = (lane & s) != 0;
#pragma unroll
    for (int k = 0; k < s; ++k) {
      const float send = up ? v[k] : v[k + s];
      const float keep = up ? v[k + s] : v[k];
      v[k] = keep + __shfl_xor_sync(kFull, send, s);
    }
  }
  return v[0];
}

// square root to about one unit in the last place (one special-function instruction and a multiply)
__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// vm: bit k set when column col0 + k of the key tile holds a key (an own token or a cached past key);
// with a causal mask an own token j (j < P) also needs j <= i_tok
// (PAST = false: the tile holds the frame's own keys only and vm is not looked at: column j holds a key when j < P)
template <bool PAST>
__device__ __forceinline__ float ps_chunk_max(const uint32_t (&r)[16], int col0, int P, uint32_t vm, bool causal,
                                              int i_tok) {
  if (!causal && (PAST ? vm == 0xffffu : col0 + 16 <= P)) {
    const float a = tc::fmax3(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]));
    const float b = tc::fmax3(__uint_as_float(r[3]), __uint_as_float(r[4]), __uint_as_float(r[5]));
    const float c = tc::fmax3(__uint_as_float(r[6]), __uint_as_float(r[7]), __uint_as_float(r[8]));
    const float d = tc::fmax3(__uint_as_float(r[9]), __uint_as_float(r[10]), __uint_as_float(r[11]));
    const float e = tc::fmax3(__uint_as_float(r[12]), __uint_as_float(r[13]), __uint_as_float(r[14]));
    return fmaxf(tc::fmax3(a, b, c), tc::fmax3(d, e, __uint_as_float(r[15])));
  }
  float m = -INFINITY;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const int j = col0 + k;
    const bool ok = PAST ? ((vm >> k) & 1u) && (!causal || j >= P || j <= i_tok) : (j < P) && (!causal || j <= i_tok);
    m = ok ? fmaxf(m, __uint_as_float(r[k])) : m;
  }
  return m;
}

// r <- exp2(r * c - mc) (0 where masked); returns the sum
template <bool PAST>
__device__ __forceinline__ float ps_chunk_exp(uint32_t (&r)[16], float c, float mc, int col0, int P, uint32_t vm,
                                              bool causal, int i_tok) {
  float l0 = 0.f, l1 = 0.f;
  if (!causal && (PAST ? vm == 0xffffu : col0 + 16 <= P)) {
#pragma unroll
    for (int k = 0; k < 16; k += 2) {
      const float e0 = ex2_approx(fmaf(__uint_as_float(r[k]), c, -mc));
      const float e1 = ex2_approx(fmaf(__uint_as_float(r[k + 1]), c, -mc));
      l0 += e0;
      l1 += e1;
      r[k] = __float_as_uint(e0);
      r[k + 1] = __float_as_uint(e1);
    }
  } else {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const int j = col0 + k;
      const bool ok = PAST ? ((vm >> k) & 1u) && (!causal || j >= P || j <= i_tok) : (j < P) && (!causal || j <= i_tok);
      const float e = ok ? ex2_approx(fmaf(__uint_as_float(r[k]), c, -mc)) : 0.f;
      l0 += e;
      r[k] = __float_as_uint(e);
    }
  }
  return l0 + l1;
}

// PAST: the key tile also holds cached keys of past frames (a second instantiation, so that the common
// case keeps its shorter inner loop: the epilogue is bound by instruction issue)
template <bool PAST>
__global__ void __maxnreg__(96) score_ps_kernel(const ScorePsParams p,
                                                 const __grid_constant__ CUtensorMap qmap,
                                                 const __grid_constant__ CUtensorMap kmap,
                                                 const __grid_constant__ CUtensorMap wmap,
                                                 const __grid_constant__ CUtensorMap pmap) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = tc::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const ScoreParams& sp = p.sp;
  const int P = sp.P, D = sp.D, G = sp.G, Hkv = sp.Hkv, KB = D >> 6, Ls = sp.Ls;
  // a unit is (frame, scoring layer, key head), in that order; its rows in the K / Q maps (layer-major tensors)
  auto unit_row = [&](int unit) {
    const int fl = unit / Hkv;
    return ((fl % Ls) * sp.n_frames + fl / Ls) * P;
  };
  const int NS = p.n_stages;
  const int ipu = p.n_mt + p.tiles;                      // items per (frame, key head)
  const int n_cta = gridDim.x, cta = blockIdx.x;
  // contiguous shares [c*n/nb, (c+1)*n/nb); the compaction kernel finds the blocks of a frame from the same rule
  const int i0 = (int)((unsigned)cta * (unsigned)p.n_items / (unsigned)n_cta);
  const int i1 = (int)((unsigned)(cta + 1) * (unsigned)p.n_items / (unsigned)n_cta);
  const int rows_q = p.tpt * G;

  const uint32_t k_kb = (uint32_t)p.npad * 128u, st_kb = 128u * 128u;
  const uint32_t k_buf = (uint32_t)KB * k_kb, st_buf = (uint32_t)KB * st_kb;
  const uint32_t sK = base;                              // two key buffers
  const uint32_t sS = sK + 2u * k_buf;                   // NS operand stages
  const uint32_t misc_off = 2u * k_buf + (uint32_t)NS * st_buf;
  float* s_col = reinterpret_cast<float*>(sm + misc_off);                     // [4][256]
  // (reference, sum) of a row's four warps, one copy per accumulator: a copy is rewritten two items
  // later, after the row's warps have met again at the barrier of the item in between
  float* s_mx = reinterpret_cast<float*>(sm + misc_off + 4096);               // [2][kPsSplit][128]
  float* s_sum = s_mx + 2 * kPsSplit * 128;                                   // [2][kPsSplit][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + misc_off + 12288);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + misc_off + 12288 + 192);
  float* s_mref = reinterpret_cast<float*>(sm + misc_off + 12800);            // [4 chunks][512 threads]
  const uint32_t b0 = tc::smem_u32(bars);
  // key buffer full / empty, accumulator full / empty (2 each), stage full / empty (kPsMaxStages each)
#define PS_BAR_KF(s) (b0 + 8u * (uint32_t)(s))
#define PS_BAR_KE(s) (b0 + 16u + 8u * (uint32_t)(s))
#define PS_BAR_AF(s) (b0 + 32u + 8u * (uint32_t)(s))
#define PS_BAR_AE(s) (b0 + 48u + 8u * (uint32_t)(s))
#define PS_BAR_SF(s) (b0 + 64u + 8u * (uint32_t)(s))
#define PS_BAR_SE(s) (b0 + 64u + 8u * (uint32_t)kPsMaxStages + 8u * (uint32_t)(s))

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(PS_BAR_KF(s), 1);
      tc::mbar_init(PS_BAR_KE(s), 1);
      tc::mbar_init(PS_BAR_AF(s), 1);
      tc::mbar_init(PS_BAR_AE(s), kPsEpiThreads / 32);   // one arrival per epilogue warp
    }
    for (int s = 0; s < kPsMaxStages; ++s) {
      tc::mbar_init(PS_BAR_SF(s), 1);
      tc::mbar_init(PS_BAR_SE(s), 1);
    }
    tc::fence_mbar_init();
    tc::prefetch_tmap(&qmap);
    tc::prefetch_tmap(&kmap);
    tc::prefetch_tmap(&wmap);
    if (PAST) tc::prefetch_tmap(&pmap);
  }
  // ---- TMA producer (thread 0).  The key tile of the block's first (frame, head) and its first
  // operand stage are requested here, before the block-wide barrier and with as little code in
  // front of them as possible (the first instructions of a launch come from device memory), so
  // that they are on their way while tensor memory is being allocated; produce() issues the rest.
  int pr_i = i0, pr_t = 0, pr_nk = 0, pr_ns = 0, pr_unit = -1;
  bool pr_ok = true;
  // the key tile of a unit into key buffer kb_i: the frame's own keys, then the cached keys of the past frames
  const uint32_t k_tx = (uint32_t)KB * 128u * (uint32_t)(p.own_rows + (PAST ? p.n_past * p.kappa : 0));
  auto load_keys = [&](int unit, int kb_i) {
    const uint32_t dst = sK + (uint32_t)kb_i * k_buf, bar = PS_BAR_KF(kb_i);
    const int g = unit % Hkv;
    tc::mbar_expect_tx(bar, k_tx);
    for (int kb = 0; kb < KB; ++kb) tc::tma_load_3d(dst + kb * k_kb, &kmap, kb * 64, g, unit_row(unit), bar);
    if constexpr (PAST) {
      const int plane = p.past_plane0 + 2 * ((unit / Hkv) % Ls);
      for (int w = 0; w < p.n_past; ++w)
        for (int kb = 0; kb < KB; ++kb)
          tc::tma_load_5d(dst + kb * k_kb + (uint32_t)(p.own_rows + w * p.past_pad) * 128u, &pmap, kb * 64, g, 0, plane,
                          (int)(p.past_first + w), bar);
    }
  };
  if (tid == 0) {
    const int unit0 = i0 / ipu, x0 = i0 - unit0 * ipu;
    const int g0 = unit0 % Hkv, r0 = unit_row(unit0);
    load_keys(unit0, 0);
    if (x0 < p.n_mt) {
      tc::mbar_expect_tx(PS_BAR_SF(0), (uint32_t)KB * (uint32_t)D * 128u);
      for (int kb = 0; kb < KB; ++kb) tc::tma_load_2d(sS + kb * st_kb, &wmap, kb * 64, 2 * D, PS_BAR_SF(0));
    } else {
      tc::mbar_expect_tx(PS_BAR_SF(0), (uint32_t)KB * (uint32_t)rows_q * 128u);
      for (int kb = 0; kb < KB; ++kb)
        tc::tma_load_3d(sS + kb * st_kb, &qmap, kb * 64, g0 * G, r0 + (x0 - p.n_mt) * p.tpt, PS_BAR_SF(0));
    }
    pr_nk = 1; pr_unit = unit0; pr_ns = 1; pr_t = 1;
    if (x0 >= p.n_mt) { pr_i = i0 + 1; pr_t = 0; }         // an attention item has this one operand load
  }
  auto produce = [&]() {
    while (pr_i < i1 && pr_ok) {
      const int unit = pr_i / ipu, x = pr_i % ipu;
      const int g = unit % Hkv, urow = unit_row(unit);
      if (unit != pr_unit) {
        const int kb_i = pr_nk & 1;
        pr_ok = tc::mbar_wait(PS_BAR_KE(kb_i), (uint32_t)(((pr_nk >> 1) & 1) ^ 1));
        if (!pr_ok) break;
        load_keys(unit, kb_i);
        ++pr_nk;
        pr_unit = unit;
      }
      const int n_ld = x < p.n_mt ? 3 : 1;               // DFT item: the three matrix terms, smallest first
      while (pr_t < n_ld) {
        const int s = pr_ns % NS;
        pr_ok = tc::mbar_wait(PS_BAR_SE(s), (uint32_t)(((pr_ns / NS) & 1) ^ 1));
        if (!pr_ok) break;
        const uint32_t dst = sS + (uint32_t)s * st_buf;
        if (x < p.n_mt) {
          tc::mbar_expect_tx(PS_BAR_SF(s), (uint32_t)KB * (uint32_t)D * 128u);
          for (int kb = 0; kb < KB; ++kb)
            tc::tma_load_2d(dst + kb * st_kb, &wmap, kb * 64, (2 - pr_t) * D, PS_BAR_SF(s));
        } else {
          tc::mbar_expect_tx(PS_BAR_SF(s), (uint32_t)KB * (uint32_t)rows_q * 128u);
          for (int kb = 0; kb < KB; ++kb)
            tc::tma_load_3d(dst + kb * st_kb, &qmap, kb * 64, g * G, urow + (x - p.n_mt) * p.tpt, PS_BAR_SF(s));
        }
        ++pr_ns;
        ++pr_t;
      }
      if (!pr_ok) break;
      ++pr_i;
      pr_t = 0;
    }
  };
  if (warp == 1) {
    __syncwarp();
    tc::tmem_alloc(tc::smem_u32(tmem_slot), 512u);
  }
  // Rows of a stage that a Q box never writes (rows_q .. 127) hold whatever the stage held before.
  // The MMA reads them as rows of the tile: they only produce rows of the product that belong to
  // no token, and the epilogue discards those rows whatever their bits are.
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp < 4) {
    // the control warpgroup (warps 2 and 3 have no other job) hands its registers over
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kPsCtrlRegs));
  if (warp == 0) {
    // ================================================================== TMA producer (continued)
    if (lane == 0) {
      produce();
      if (!pr_ok) atomicCAS(p.status, 0, 3);
      pdl_trigger();                                     // the next kernel of the call may be scheduled
      // copies of this thread still in flight land before the block goes away
      for (int s = 0; s < 2; ++s) {
        const int cnt = (pr_nk + 1 - s) >> 1;
        if (cnt) tc::mbar_wait(PS_BAR_KF(s), (uint32_t)((cnt - 1) & 1));
      }
      for (int s = 0; s < NS; ++s) {
        const int cnt = (pr_ns + NS - 1 - s) / NS;
        if (cnt) tc::mbar_wait(PS_BAR_SF(s), (uint32_t)((cnt - 1) & 1));
      }
    }
  } else if (warp == 1) {
    // ================================================================== MMA issuer
    if (lane == 0) {
      bool ok = true;
      const uint32_t idesc_att = tc::idesc_bf16_f32(128, p.npad), idesc_dft = tc::idesc_bf16_f32(128, D);
      int nk = 0, ns = 0, it = 0, last_unit = -1, kb_i = 0;
      for (int i = i0; i < i1 && ok; ++i, ++it) {
        const int unit = i / ipu, x = i % ipu;
        if (unit != last_unit) {
          kb_i = nk & 1;
          ok = tc::mbar_wait(PS_BAR_KF(kb_i), (uint32_t)((nk >> 1) & 1));
          if (!ok) break;
          ++nk;
          last_unit = unit;
        }
        const int b = it & 1;
        ok = tc::mbar_wait(PS_BAR_AE(b), (uint32_t)(((it >> 1) & 1) ^ 1));
        if (!ok) break;
        tc::tc_fence_after_sync();
        const uint32_t d_tmem = tmem + (uint32_t)b * 256u;
        const uint32_t kbase = sK + (uint32_t)kb_i * k_buf;
        const int n_ld = x < p.n_mt ? 3 : 1;
        for (int t = 0; t < n_ld && ok; ++t) {
          const int s = ns % NS;
          ok = tc::mbar_wait(PS_BAR_SF(s), (uint32_t)((ns / NS) & 1));
          if (!ok) break;
          tc::tc_fence_after_sync();
          const uint32_t sbase = sS + (uint32_t)s * st_buf;
          if (x < p.n_mt) {
            // rows x*128 .. of the key tile times one term of the DFT matrix
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                tc::mma_bf16_ss(d_tmem, tc::smem_desc_sw128(kbase + kb * k_kb + (uint32_t)x * st_kb + k * 32),
                                tc::smem_desc_sw128(sbase + kb * st_kb + k * 32), idesc_dft, (t | kb | k) != 0);
          } else {
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                tc::mma_bf16_ss(d_tmem, tc::smem_desc_sw128(sbase + kb * st_kb + k * 32),
                                tc::smem_desc_sw128(kbase + kb * k_kb + k * 32), idesc_att, (kb | k) != 0);
          }
          tc::mma_commit(PS_BAR_SE(s));
          ++ns;
        }
        if (!ok) break;
        tc::mma_commit(PS_BAR_AF(b));
        if (i + 1 == i1 || (i + 1) / ipu != unit) tc::mma_commit(PS_BAR_KE(kb_i));
      }
      if (!ok) atomicCAS(p.status, 0, 4);
    }
  }
  } else {
    // ================================================================== epilogue
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kPsEpiRegs));
    const int et = tid - kPsEpiOff, ew = et >> 5;
    const int q = warp & 3, h = ew >> 2;                 // TMEM lane quarter, column range
    const int row = q * 32 + lane;
    const int row_tok = row / G;                         // token of this row inside its tile
    const uint32_t tlane = (uint32_t)(q * 32) << 16;
    // the columns of a row go to its four warps in chunks of 16
    const int nch16 = p.npad >> 4, ch_base = nch16 / kPsSplit, ch_rem = nch16 % kPsSplit;
    const int my_c0 = h * ch_base + (h < ch_rem ? h : ch_rem), my_nch = ch_base + (h < ch_rem ? 1 : 0);
    const bool causal = sp.causal != 0;
    const float c = p.exp2_scale;
    constexpr int kMaxCh = kPsAccCols / 16;
    // which of the 16 columns from col0 on hold a key: the frame's own tokens, and behind them the
    // kappa cached keys at the front of every past frame's share of the tile
    const int past_end = p.own_rows + p.n_past * p.past_pad;
    auto chunk_mask = [&](int col0) -> uint32_t {
      const int nv = P - col0;
      uint32_t vm = nv >= 16 ? 0xffffu : (nv <= 0 ? 0u : (1u << nv) - 1u);
      if (col0 + 16 > p.own_rows && col0 < past_end) {
        int r = col0 - p.own_rows, rem = r >= 0 ? r % p.past_pad : 0;
#pragma unroll
        for (int k = 0; k < 16; ++k, ++r) {
          if (r >= 0 && r < past_end - p.own_rows) {
            if (rem < p.kappa) vm |= 1u << k;
            rem = rem + 1 == p.past_pad ? 0 : rem + 1;
          }
        }
      }
      return vm;
    };
    // (the masks of this thread's chunks, 16 bits each, worked out once)
    unsigned long long vmask = 0ull;
    if constexpr (PAST) {
      for (int ch = 0; ch < my_nch; ++ch) vmask |= (unsigned long long)chunk_mask((my_c0 + ch) * 16) << (16 * ch);
    }
    float acc[kPsAccCols];                               // column sums of this thread's row, over tiles
#pragma unroll
    for (int k = 0; k < kPsAccCols; ++k) acc[k] = 0.f;
    bool ok = true;
    int it = 0;
    int x = i0 % ipu, g = (i0 / ipu) % Hkv, ly = ((i0 / ipu) / Hkv) % Ls, f = ((i0 / ipu) / Hkv) / Ls;
    for (int i = i0; i < i1; ++i, ++it) {
      const int b = it & 1;
      // A wait that runs out is recorded; the warp then goes on without waiting (every read
      // below stays inside the accumulators), so that the warps of a row keep meeting at their barrier.
      if (ok) ok = __all_sync(kFull, tc::mbar_wait(PS_BAR_AF(b), (uint32_t)((it >> 1) & 1)));
      tc::tc_fence_after_sync();
      const uint32_t tb = tmem + (uint32_t)b * 256u + tlane;
      if (x < p.n_mt) {
        // ---- Eq. 2-3: this thread's share of the bins of its token
        const int H2 = D >> 1;
        const int bins = H2 / kPsSplit >= 16 ? H2 / kPsSplit : 16;   // per warp of the row, a multiple of 16
        const int bin0 = h * bins;
        float tot = 0.f;
        if (bin0 < H2) {
#pragma unroll 1
          for (int cc = 0; cc < bins; cc += 8) {
            uint32_t re[8], im[8];
            tc::tmem_ld8(tb + bin0 + cc, re);
            tc::tmem_ld8(tb + H2 + bin0 + cc, im);
            tc::tmem_wait_ld8x2(re, im);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const float a = __uint_as_float(re[k]), bb = __uint_as_float(im[k]);
              const float mag = sqrt_approx(fmaf(a, a, bb * bb));
              // bins 0 and D/2 are real: their two values sit in the re/im slots of "bin 0"
              tot += (bin0 + cc + k == 0) ? fabsf(a) + fabsf(bb) : 2.f * mag;
            }
          }
        }
        float* xs = s_sum + b * kPsSplit * 128;
        xs[h * 128 + row] = tot;
        tc::named_sync(1 + q, 32 * kPsSplit);
        const int token = x * 128 + row;
        if (h == 0 && token < P) {
          float t4 = 0.f;
#pragma unroll
          for (int hh = 0; hh < kPsSplit; ++hh) t4 += xs[hh * 128 + row];
          reinterpret_cast<float*>(sp.ifft_part)[(((long long)f * Ls + ly) * Hkv + g) * P + token] = t4;
        }
      } else {
        // ---- Eq. 1
        const int i_tok = (x - p.n_mt) * p.tpt + row_tok;
        const bool valid = (row < rows_q) && (i_tok < P);
        // sweep 1: running maximum, e = exp(z - running max) back into tensor memory, row sum.
        // One 16-column chunk per trip; the other warps of the scheduler cover the load latency.
        // The loop is kept rolled: many warps walking a long unrolled body starve on instruction fetch.
        float m_run = -INFINITY, l = 0.f;
#pragma unroll 1
        for (int ch = 0; ch < my_nch; ++ch) {
          const int col = (my_c0 + ch) * 16;
          uint32_t ra[16];
          tc::tmem_ld16(tb + col, ra);
          tc::tmem_wait_ld16(ra);
          const uint32_t vm = PAST ? (uint32_t)(vmask >> (16 * ch)) & 0xffffu : 0u;
          const float m_new = fmaxf(m_run, ps_chunk_max<PAST>(ra, col, P, vm, causal, i_tok));
          const float resc = (m_new == m_run) ? 1.f : ex2_approx((m_run - m_new) * c);
          l = l * resc + ps_chunk_exp<PAST>(ra, c, m_new * c, col, P, vm, causal, i_tok);
          tc::tmem_st16(tb + col, ra);
          s_mref[ch * kPsEpiThreads + et] = m_new;
          m_run = m_new;
        }
        tc::tmem_wait_st();
        float* xm = s_mx + b * kPsSplit * 128;
        float* xs = s_sum + b * kPsSplit * 128;
        xm[h * 128 + row] = m_run;
        xs[h * 128 + row] = l;
        tc::named_sync(1 + q, 32 * kPsSplit);
        float m = xm[row];
#pragma unroll
        for (int hh = 1; hh < kPsSplit; ++hh) m = fmaxf(m, xm[hh * 128 + row]);
        float lsum = 0.f;
#pragma unroll
        for (int hh = 0; hh < kPsSplit; ++hh) lsum += xs[hh * 128 + row] * ex2_approx((xm[hh * 128 + row] - m) * c);
        const float inv = valid ? __fdividef(1.f, lsum) : 0.f;
        // sweep 2: acc[column] += e * 2^(ref - max) / sum
#pragma unroll
        for (int ch = 0; ch < kMaxCh; ++ch) {
          if (ch < my_nch) {
            uint32_t ra[16];
            tc::tmem_ld16(tb + (my_c0 + ch) * 16, ra);
            // rows outside the frame contribute nothing, whatever bits they hold
            const float w = valid ? ex2_approx((s_mref[ch * kPsEpiThreads + et] - m) * c) * inv : 0.f;
            tc::tmem_wait_ld16(ra);
#pragma unroll
            for (int k = 0; k < 16; ++k)
              acc[ch * 16 + k] = valid ? fmaf(__uint_as_float(ra[k]), w, acc[ch * 16 + k]) : acc[ch * 16 + k];
          }
        }
      }
      // the accumulator may be overwritten
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(PS_BAR_AE(b));

      const bool frame_ends = (i + 1 == i1) || (x == ipu - 1 && g == Hkv - 1 && ly == Ls - 1);
      if (frame_ends) {
        // ---- leaving frame f: this block's column sums go to its slot of the frame
#pragma unroll
        for (int pp = 0; pp < (kPsAccCols + 31) / 32; ++pp) {
          float v[32];
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            if (pp * 32 + k < kPsAccCols) { v[k] = acc[pp * 32 + k]; acc[pp * 32 + k] = 0.f; }
            else v[k] = 0.f;
          }
          const float s = warp_column_sums(v, lane);
          if (pp * 32 + lane < my_nch * 16) s_col[q * 256 + my_c0 * 16 + pp * 32 + lane] = s;
        }
        PsEpiGroup::sync();
        float* slot = reinterpret_cast<float*>(sp.colsum_part) + (long long)(cta + f) * P;
        for (int t = et; t < P; t += kPsEpiThreads)
          slot[t] = (s_col[t] + s_col[256 + t]) + (s_col[512 + t] + s_col[768 + t]);
        PsEpiGroup::sync();                                // the sums may be overwritten
      }
      if (++x == ipu) {
        x = 0;
        if (++g == Hkv) {
          g = 0;
          if (++ly == Ls) { ly = 0; ++f; }
        }
      }
    }
    if (!ok && lane == 0) atomicCAS(p.status, 0, 5);
  }
#undef PS_BAR_KF
#undef PS_BAR_KE
#undef PS_BAR_AF
#undef PS_BAR_AE
#undef PS_BAR_SF
#undef PS_BAR_SE

  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::tmem_dealloc(tmem, 512u);
  }
}

}  // namespace mukv
