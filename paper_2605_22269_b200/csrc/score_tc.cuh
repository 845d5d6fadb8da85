// Tensor-core scoring of a chunk (Sec. 3.3, Eq. 1-4) for bf16 inputs: tcgen05.mma with the
// accumulator in tensor memory, operands brought in by TMA.
//
// score_tc_kernel: grid (n_mt + tiles, Hkv, n_frames), 128 threads, two blocks per SM.
//
//   attention blocks (blockIdx.x >= n_mt), Eq. 1.  The G query heads that share key head g are
//   flattened with the tokens into rows (token, head): one TMA box of tpt = 128/G tokens x G
//   heads x 64 channels lands as up to 128 rows of a K-major, 128-byte-swizzled operand.  One
//   block computes S = Q_tile K_g^T (128 x npad, K = D) into tensor memory.  Thread r owns row r
//   (its TMEM lane): pass A takes the row maximum, pass B writes exp(z - max) back into tensor
//   memory and sums the row, pass C scales by 1/sum and adds the 32 rows of a warp column by
//   column with a shuffle butterfly.  The attention matrix never leaves the SM.
//
//   DFT blocks (blockIdx.x < n_mt), Eq. 2-3.  The D-point transform of every key vector of 128
//   tokens is the dense product K_tile W with W[d][n] = cos(2 pi n d / D) for n <= D/2 and
//   -sin(2 pi (n - D/2) d / D) above: columns 0..D/2 are the real parts of bins 0..D/2, the rest
//   the imaginary parts of bins 1..D/2-1 (the upper bins mirror them).  W is held as three bf16
//   terms (hi + mid + lo reproduce the float value), the keys are bf16 already, so the products
//   are exact and the sum is accumulated in float.  Thread r then adds the D bin magnitudes.
//
//   The block that finishes a frame last (arrival counter, nobody waits) adds the per-tile
//   partial sums in a fixed order, applies Eq. 4 and selects the kappa tokens.
#pragma once
#include "common.cuh"
#include "score.cuh"
#include "tc.cuh"

namespace mukv {

constexpr int kTcThreads = 128;
constexpr int kTcScratchBytes = 4096;     // column partials / selection scratch
constexpr int kTcTailBytes = 128;         // barriers, TMEM slot

struct ScoreTcParams {
  ScoreParams sp;            // colsum_part: float [F][Hkv*tiles][P], ifft_part: float [F][Hkv][P]
  int tiles;                 // attention row tiles per (frame, key head)
  int tpt;                   // tokens per attention tile = 128 / G
  int npad;                  // P rounded up to a multiple of 16 (the MMA's N)
  int n_mt;                  // DFT row tiles per (frame, key head) = ceil(P / 128)
  int tmem_cols;             // power of two >= max(npad, D)
  uint32_t op_bytes;         // bytes reserved for the operand tiles
  float exp2_scale;          // log2(e) / sqrt(D)
  int* status;               // device error word (0 = fine)
};

__host__ inline uint32_t score_tc_op_bytes(int P, int D) {
  const uint32_t KB = D / 64, npad = (P + 15) / 16 * 16;
  const uint32_t att = KB * npad * 128 + KB * 128 * 128;
  const uint32_t dft = KB * 128 * 128 + 2 * KB * D * 128;
  return att > dft ? att : dft;
}
__host__ inline size_t score_tc_smem_bytes(int P, int D) {
  return (size_t)score_tc_op_bytes(P, D) + kTcScratchBytes + kTcTailBytes + 1024;   // 1024: alignment slack
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

__global__ void __launch_bounds__(kTcThreads) score_tc_kernel(const ScoreTcParams p,
                                                              const __grid_constant__ CUtensorMap qmap,
                                                              const __grid_constant__ CUtensorMap kmap,
                                                              const __grid_constant__ CUtensorMap kmap_dft,
                                                              const __grid_constant__ CUtensorMap wmap) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = tc::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;          // swizzled operand tiles start on 1024 bytes
  unsigned char* sm = smem_raw + (base - raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const ScoreParams& sp = p.sp;
  const int P = sp.P, D = sp.D, G = sp.G, Hkv = sp.Hkv, KB = D >> 6;
  const int g = blockIdx.y, f = blockIdx.z, x = blockIdx.x;
  const bool dft = x < p.n_mt;

  float* s_part = reinterpret_cast<float*>(sm + p.op_bytes);                     // [4][256]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + p.op_bytes + kTcScratchBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
  const uint32_t bar_full = tc::smem_u32(&bars[0]), bar_mma = tc::smem_u32(&bars[1]);
  const uint32_t bar_w = tc::smem_u32(&bars[2]), bar_mma2 = tc::smem_u32(&bars[3]);

  if (tid == 0) {
    tc::mbar_init(bar_full, 1);
    tc::mbar_init(bar_mma, 1);
    tc::mbar_init(bar_w, 1);
    tc::mbar_init(bar_mma2, 1);
    tc::fence_mbar_init();
    if (dft) { tc::prefetch_tmap(&kmap_dft); tc::prefetch_tmap(&wmap); }
    else { tc::prefetch_tmap(&kmap); tc::prefetch_tmap(&qmap); }
  }
  if (warp == 0) {
    __syncwarp();
    tc::tmem_alloc(tc::smem_u32(tmem_slot), (uint32_t)p.tmem_cols);
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);      // this warp's 32 TMEM lanes
  bool failed = false;                                              // meaningful in thread 0 only

  if (!dft) {
    // ------------------------------------------------------------------ Eq. 1
    const int tile = x - p.n_mt;
    const int rows_q = p.tpt * G;                                   // rows the Q box fills
    const uint32_t k_kb = (uint32_t)p.npad * 128u, q_kb = 128u * 128u;
    const uint32_t sK = base, sQ = base + (uint32_t)KB * k_kb;
    // rows of the Q operand that the box does not cover must not hold stale bits
    {
      const int pad_rows = 128 - rows_q;
      uint4* q4 = reinterpret_cast<uint4*>(sm + (size_t)KB * k_kb);
      for (int i = tid; i < KB * pad_rows * 8; i += kTcThreads) {
        const int kb = i / (pad_rows * 8), rem = i % (pad_rows * 8);
        q4[(size_t)kb * (q_kb / 16) + (size_t)rows_q * 8 + rem] = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    tc::fence_proxy_async_smem();
    __syncthreads();
    if (tid == 0) {
      tc::mbar_expect_tx(bar_full, (uint32_t)KB * (uint32_t)(p.npad + rows_q) * 128u);
      for (int kb = 0; kb < KB; ++kb) tc::tma_load_3d(sK + kb * k_kb, &kmap, kb * 64, g, f * P, bar_full);
      for (int kb = 0; kb < KB; ++kb)
        tc::tma_load_3d(sQ + kb * q_kb, &qmap, kb * 64, g * G, f * P + tile * p.tpt, bar_full);
      const bool ok = tc::mbar_wait(bar_full, 0) || tc::mbar_wait(bar_full, 0);
      tc::tc_fence_after_sync();
      if (ok) {
        const uint32_t idesc = tc::idesc_bf16_f32(128, p.npad);
        for (int kb = 0; kb < KB; ++kb)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc::mma_bf16_ss(tmem, tc::smem_desc_sw128(sQ + kb * q_kb + k * 32),
                            tc::smem_desc_sw128(sK + kb * k_kb + k * 32), idesc, (kb | k) != 0);
      }
      failed = !ok;
      tc::mma_commit(bar_mma);
    }
    const bool done = tc::mbar_wait(bar_mma, 0);
    tc::tc_fence_after_sync();
    const int bad = __syncthreads_or((!done || failed) ? 1 : 0);
    if (bad) {
      if (tid == 0) atomicCAS(p.status, 0, 1);
    } else {
      const int r = tid;                                            // row of the tile = TMEM lane
      const int i_tok = tile * p.tpt + r / G;
      const bool valid = (r < rows_q) && (i_tok < P);
      const bool causal = sp.causal != 0;
      const int nch = (p.npad + 31) >> 5;
      const float c = p.exp2_scale;
      // pass A: row maximum
      float m = -INFINITY;
      for (int ch = 0; ch < nch; ++ch) {
        float v[32];
        tc::tmem_ld32(trow + ch * 32, v);
        const int j0 = ch * 32;
        if (!causal && j0 + 32 <= P) {
#pragma unroll
          for (int k = 0; k < 32; ++k) m = fmaxf(m, v[k]);
        } else {
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            const int j = j0 + k;
            const bool ok = (j < P) && (!causal || j <= i_tok);
            m = ok ? fmaxf(m, v[k]) : m;
          }
        }
      }
      // pass B: e = exp(z - max) back into tensor memory, row sum
      const float mc = m * c;
      float l = 0.f;
      for (int ch = 0; ch < nch; ++ch) {
        float v[32];
        tc::tmem_ld32(trow + ch * 32, v);
        const int j0 = ch * 32;
        if (!causal && j0 + 32 <= P) {
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            v[k] = ex2_approx(fmaf(v[k], c, -mc));
            l += v[k];
          }
        } else {
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            const int j = j0 + k;
            const bool ok = (j < P) && (!causal || j <= i_tok);
            v[k] = ok ? ex2_approx(fmaf(v[k], c, -mc)) : 0.f;
            l += v[k];
          }
        }
        tc::tmem_st32(trow + ch * 32, v);
      }
      tc::tmem_wait_st();
      // pass C: normalise and add the rows column by column
      const float inv = valid ? 1.f / l : 0.f;
      const bool all_valid = __all_sync(kFull, valid);
      for (int ch = 0; ch < nch; ++ch) {
        float v[32];
        tc::tmem_ld32(trow + ch * 32, v);
        if (all_valid) {
#pragma unroll
          for (int k = 0; k < 32; ++k) v[k] *= inv;
        } else {
#pragma unroll
          for (int k = 0; k < 32; ++k) v[k] = valid ? v[k] * inv : 0.f;
        }
        s_part[warp * 256 + ch * 32 + lane] = warp_column_sums(v, lane);
      }
      __syncthreads();
      float* out = reinterpret_cast<float*>(sp.colsum_part) +
                   ((long long)f * Hkv * p.tiles + (long long)g * p.tiles + tile) * P;
      for (int j = tid; j < P; j += kTcThreads)
        out[j] = (s_part[j] + s_part[256 + j]) + (s_part[512 + j] + s_part[768 + j]);
    }
  } else {
    // ------------------------------------------------------------------ Eq. 2-3
    const int mt = x;
    const uint32_t a_kb = 128u * 128u, w_kb = (uint32_t)D * 128u;
    const uint32_t sA = base, sW0 = base + (uint32_t)KB * a_kb, sW1 = sW0 + (uint32_t)KB * w_kb;
    if (tid == 0) {
      tc::mbar_expect_tx(bar_full, (uint32_t)KB * (a_kb + 2u * w_kb));
      for (int kb = 0; kb < KB; ++kb)
        tc::tma_load_3d(sA + kb * a_kb, &kmap_dft, kb * 64, g, f * P + mt * 128, bar_full);
      for (int kb = 0; kb < KB; ++kb) tc::tma_load_2d(sW0 + kb * w_kb, &wmap, kb * 64, 2 * D, bar_full);   // lo
      for (int kb = 0; kb < KB; ++kb) tc::tma_load_2d(sW1 + kb * w_kb, &wmap, kb * 64, D, bar_full);       // mid
      bool ok = tc::mbar_wait(bar_full, 0) || tc::mbar_wait(bar_full, 0);
      tc::tc_fence_after_sync();
      const uint32_t idesc = tc::idesc_bf16_f32(128, D);
      if (ok) {
        for (int t = 0; t < 2; ++t) {
          const uint32_t sW = t ? sW1 : sW0;
          for (int kb = 0; kb < KB; ++kb)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              tc::mma_bf16_ss(tmem, tc::smem_desc_sw128(sA + kb * a_kb + k * 32),
                              tc::smem_desc_sw128(sW + kb * w_kb + k * 32), idesc, (t | kb | k) != 0);
        }
      }
      tc::mma_commit(bar_mma);
      ok = tc::mbar_wait(bar_mma, 0) && ok;                         // the lo term's buffer is free again
      if (ok) {
        tc::mbar_expect_tx(bar_w, (uint32_t)KB * w_kb);
        for (int kb = 0; kb < KB; ++kb) tc::tma_load_2d(sW0 + kb * w_kb, &wmap, kb * 64, 0, bar_w);        // hi
        ok = tc::mbar_wait(bar_w, 0) || tc::mbar_wait(bar_w, 0);
        tc::tc_fence_after_sync();
      }
      if (ok) {
        for (int kb = 0; kb < KB; ++kb)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc::mma_bf16_ss(tmem, tc::smem_desc_sw128(sA + kb * a_kb + k * 32),
                            tc::smem_desc_sw128(sW0 + kb * w_kb + k * 32), idesc, 1u);
      }
      failed = !ok;
      tc::mma_commit(bar_mma2);
    }
    const bool done = tc::mbar_wait(bar_mma2, 0);
    tc::tc_fence_after_sync();
    const int bad = __syncthreads_or((!done || failed) ? 1 : 0);
    if (bad) {
      if (tid == 0) atomicCAS(p.status, 0, 2);
    } else {
      const int token = mt * 128 + tid;
      const int H2 = D >> 1;
      float total = 0.f;
      for (int b0 = 0; b0 < H2; b0 += 32) {
        float re[32], im[32];
        tc::tmem_ld32(trow + b0, re);
        tc::tmem_ld32(trow + H2 + b0, im);
#pragma unroll
        for (int k = 0; k < 32; ++k) {
          if (b0 + k == 0) total += fabsf(re[k]) + fabsf(im[k]);   // bins 0 and D/2 are real
          else total += 2.f * sqrtf(fmaf(re[k], re[k], im[k] * im[k]));
        }
      }
      if (token < P) reinterpret_cast<float*>(sp.ifft_part)[((long long)f * Hkv + g) * P + token] = total;
    }
  }

  // ------------------------------------------------------------------ last block of the frame: Eq. 4, selection
  int* s_int = reinterpret_cast<int*>(sm + p.op_bytes + 2048 + 512);
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int total_blocks = Hkv * (p.tiles + p.n_mt);
    const int old = atomicAdd(sp.frame_counter + f, 1);
    s_int[63] = (old == total_blocks - 1);
    if (old == total_blocks - 1) sp.frame_counter[f] = 0;          // ready for the next launch
  }
  __syncthreads();
  if (s_int[63]) {
    __threadfence();
    double* s_sc = reinterpret_cast<double*>(sm + p.op_bytes);
    double* s_misc = reinterpret_cast<double*>(sm + p.op_bytes + 2048);
    double att[2] = {0.0, 0.0}, fft[2] = {0.0, 0.0};
    const int U = Hkv * p.tiles;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int t = tid + k * kTcThreads;
      if (t < P) {
        const float* cp = reinterpret_cast<const float*>(sp.colsum_part) + (long long)f * U * P + t;
        for (int u = 0; u < U; ++u) att[k] += (double)__ldcg(cp + (long long)u * P);
        att[k] = att[k] / (double)((long long)sp.Hq * P);
        const float* fp = reinterpret_cast<const float*>(sp.ifft_part) + (long long)f * Hkv * P + t;
        for (int gg = 0; gg < Hkv; ++gg) fft[k] += (double)__ldcg(fp + (long long)gg * P);
        fft[k] = fft[k] / (double)((long long)Hkv * D);
      }
    }
    __syncthreads();
    select_frame<2>(sp, f, att, fft, s_sc, s_int, s_misc);
  }

  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tc::tmem_dealloc(tmem, (uint32_t)p.tmem_cols);
  }
}

}  // namespace mukv
