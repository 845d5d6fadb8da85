// Seeded synthetic K/V/Q streams, device side.  Produces the same bytes as synth/cpu.py:
// integer hashing, a quantile-table lookup and IEEE float32 multiplies/adds in a fixed order
// (the _rn intrinsics keep the compiler from contracting them into fused multiply-adds).
// This file holds no part of the compression or retrieval arithmetic.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr unsigned long long kGold = 0x9E3779B97F4A7C15ull;
constexpr unsigned long long kM1 = 0xBF58476D1CE4E5B9ull;
constexpr unsigned long long kM2 = 0x94D049BB133111EBull;

__host__ __device__ inline unsigned long long mix64(unsigned long long x) {
  x ^= x >> 30; x *= kM1;
  x ^= x >> 27; x *= kM2;
  x ^= x >> 31;
  return x;
}
__host__ __device__ inline unsigned long long stream_key(unsigned long long seed, unsigned long long tag,
                                                         unsigned long long sub) {
  return mix64(mix64(seed * kGold + tag) + (sub + 1) * kGold);
}

struct SynthParams {
  unsigned long long seed;
  int L, Hq, Hkv, D, P;
  int bf16;
  int has_scenes;
  float scene_sigma, frame_sigma;
};

// four consecutive normals of stream `key` starting at element e4*4
__device__ inline void normals4(unsigned long long key, unsigned long long word, const float* __restrict__ table,
                                float out[4]) {
  unsigned long long h = mix64(key + (word + 1) * kGold);
#pragma unroll
  for (int i = 0; i < 4; ++i) out[i] = __ldg(table + ((h >> (16 * i)) & 0xFFFFull));
}

template <typename T> __device__ inline void store4(T* dst, const float v[4]);
template <> __device__ inline void store4<float>(float* dst, const float v[4]) {
  *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ inline void store4<__nv_bfloat16>(__nv_bfloat16* dst, const float v[4]) {
  __nv_bfloat162 a = __halves2bfloat162(__float2bfloat16_rn(v[0]), __float2bfloat16_rn(v[1]));
  __nv_bfloat162 b = __halves2bfloat162(__float2bfloat16_rn(v[2]), __float2bfloat16_rn(v[3]));
  uint2 u;
  u.x = *reinterpret_cast<unsigned*>(&a);
  u.y = *reinterpret_cast<unsigned*>(&b);
  *reinterpret_cast<uint2*>(dst) = u;
}

// K and V of frames t0..t0+n-1, layout [L][n][P][Hkv][D]; one thread per 4 channels.
template <typename T>
__global__ void synth_kv_kernel(SynthParams sp, const float* __restrict__ table, const float* __restrict__ out_scale,
                                const int* __restrict__ scene_of_frame, long long t0, int n, T* __restrict__ K,
                                T* __restrict__ V) {
  const long long per_frame_layer = (long long)sp.P * sp.Hkv * sp.D;       // elements of one [P][Hkv][D] block
  const long long total4 = (long long)sp.L * n * per_frame_layer / 4;
  const int D4 = sp.D / 4;
  for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < total4;
       w += (long long)gridDim.x * blockDim.x) {
    long long r = w;
    const int d4 = (int)(r % D4); r /= D4;
    const int g = (int)(r % sp.Hkv); r /= sp.Hkv;
    const int p = (int)(r % sp.P); r /= sp.P;
    const int f = (int)(r % n); r /= n;
    const int l = (int)r;
    const long long t = t0 + f;
    // element index inside the frame's own stream: ((l*P + p)*Hkv + g)*D + d
    const unsigned long long e = (((unsigned long long)l * sp.P + p) * sp.Hkv + g) * sp.D + d4 * 4;
    float nk[4], nv[4], sc[4];
    normals4(stream_key(sp.seed, 1, (unsigned long long)t), e >> 2, table, nk);
    normals4(stream_key(sp.seed, 2, (unsigned long long)t), e >> 2, table, nv);
    const long long ch = ((long long)l * sp.Hkv + g) * sp.D + d4 * 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) sc[i] = __ldg(out_scale + ch + i);
    float kk[4], vv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      kk[i] = __fmul_rn(nk[i], sc[i]);
      vv[i] = __fmul_rn(nv[i], sc[i]);
    }
    if (sp.has_scenes) {
      float mu[4], nu[4];
      const int c = scene_of_frame[t];
      normals4(stream_key(sp.seed, 5, (unsigned long long)c), (unsigned long long)ch >> 2, table, mu);
      normals4(stream_key(sp.seed, 6, (unsigned long long)t), (unsigned long long)ch >> 2, table, nu);
#pragma unroll
      for (int i = 0; i < 4; ++i)
        kk[i] = __fadd_rn(__fadd_rn(kk[i], __fmul_rn(mu[i], sp.scene_sigma)), __fmul_rn(nu[i], sp.frame_sigma));
    }
    const long long off = (((long long)l * n + f) * sp.P + p) * sp.Hkv * sp.D + (long long)g * sp.D + d4 * 4;
    store4<T>(K + off, kk);
    store4<T>(V + off, vv);
  }
}

// Q of frames t0..t0+n-1, layout [n][P][Hq][D]
template <typename T>
__global__ void synth_q_kernel(SynthParams sp, const float* __restrict__ table, long long t0, int n,
                               T* __restrict__ Q) {
  const long long per_frame = (long long)sp.P * sp.Hq * sp.D;
  const long long total4 = (long long)n * per_frame / 4;
  for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < total4;
       w += (long long)gridDim.x * blockDim.x) {
    const int f = (int)(w / (per_frame / 4));
    const unsigned long long e4 = (unsigned long long)(w % (per_frame / 4));
    float q[4];
    normals4(stream_key(sp.seed, 3, (unsigned long long)(t0 + f)), e4, table, q);
    store4<T>(Q + (long long)f * per_frame + e4 * 4, q);
  }
}

}  // namespace

extern "C" {

// Fills Q[n][P][Hq][D] and K,V[L][n][P][Hkv][D] for absolute frames t0..t0+n-1 on `stream`.
// d_table: 65,536 float32 quantiles; d_out_scale: float32 [L][Hkv][D];
// d_scene_of_frame: int32 scene id of every frame of the stream (may be NULL without scenes).
// Returns 0, or a cudaError_t value.
int mukv_synth_chunk(unsigned long long seed, int L, int Hq, int Hkv, int D, int P, int bf16, float scene_sigma,
                     float frame_sigma, const float* d_table, const float* d_out_scale,
                     const int* d_scene_of_frame, long long t0, int n, void* d_q, void* d_k, void* d_v,
                     void* stream) {
  if (D % 4 != 0 || n <= 0) return (int)cudaErrorInvalidValue;
  SynthParams sp;
  sp.seed = seed; sp.L = L; sp.Hq = Hq; sp.Hkv = Hkv; sp.D = D; sp.P = P; sp.bf16 = bf16;
  sp.has_scenes = (scene_sigma != 0.f || frame_sigma != 0.f) ? 1 : 0;
  sp.scene_sigma = scene_sigma; sp.frame_sigma = frame_sigma;
  if (sp.has_scenes && d_scene_of_frame == nullptr) return (int)cudaErrorInvalidValue;
  cudaStream_t st = (cudaStream_t)stream;
  const int threads = 256;
  const int blocks = 148 * 16;
  if (bf16) {
    synth_kv_kernel<__nv_bfloat16><<<blocks, threads, 0, st>>>(sp, d_table, d_out_scale, d_scene_of_frame, t0, n,
                                                               (__nv_bfloat16*)d_k, (__nv_bfloat16*)d_v);
    synth_q_kernel<__nv_bfloat16><<<blocks, threads, 0, st>>>(sp, d_table, t0, n, (__nv_bfloat16*)d_q);
  } else {
    synth_kv_kernel<float><<<blocks, threads, 0, st>>>(sp, d_table, d_out_scale, d_scene_of_frame, t0, n,
                                                       (float*)d_k, (float*)d_v);
    synth_q_kernel<float><<<blocks, threads, 0, st>>>(sp, d_table, t0, n, (float*)d_q);
  }
  return (int)cudaGetLastError();
}

}  // extern "C"
