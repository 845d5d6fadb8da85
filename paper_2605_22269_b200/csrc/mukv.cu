// Host side of the MuKV library: context, store layout, argument checks, kernel launches.
// Built for sm_100a only.  No device memory is allocated here: the store and the workspace
// belong to the caller.
#include "../../include/mukv.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "compact.cuh"
#include "retrieve.cuh"
#include "score.cuh"
#include "score_ps.cuh"
#include "segsel.cuh"

using namespace mukv;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct StoreLayout {
  size_t pages, kept, frame_entry, seg_entry, frame_key, seg_key, frame_ts, page_table, frame_ksum, patch_key, patch_cnt,
      kept_count, total;
  size_t pages_bytes, kept_stride;
  size_t page_bytes;
  long long max_segs;
};

struct WorkLayout {
  size_t colsum_f, colsum_p, ifft_f, colsum_d, ifft_d, frame_counter, flagged, n_flagged, tail_ctr, sel_flag,
      seg_flag, stat_refined, dev_status;
  size_t q64, qnorm, s_frm, s_seg, s_pat, wtab, total;
  size_t zero_begin, zero_end;          // region that must start as zeros
};

// Tiling of the tensor-core scoring kernel (bf16 inputs only).
struct TcShape {
  bool ok;                 // bf16 chunk scored on the tensor cores (every supported bf16 shape fits)
  int tpt, tiles, npad, n_mt, ps_stages;
  int own_rows, past_pad;  // key-tile rows of the frame's own keys; rows reserved per cached past frame (0: none)
  size_t smem_ps;
};

thread_local std::string g_create_error;

}  // namespace

struct mukv_ctx {
  mukv_config cfg;
  StoreLayout sl;
  WorkLayout wl;
  unsigned char* store;
  unsigned char* ws;
  long long frames;
  long long launches;
  int parity = 0;                        // which of the two flagged counters this chunk uses
  unsigned epoch = 0;                    // compress calls so far (tags the per-frame selection flags)
  int C, G, esize, nc, Ls;
  int key_rows;                          // key rows of the multiply-add scoring kernel: P + past_frames * kappa
  float flag_margin, flat_ratio;
  bool force_fma = false;                // MUKV_OPT_SCORE_PATH 1: multiply-add scoring for every dtype
  bool failed = false;                   // a compress call broke off half way: only reset / stats / destroy
  TcShape tcs;                           // tcs.ok: the chunk is scored on the tensor cores
  int n_sms;
  int tail_capacity = 1;                 // blocks of tail_kernel that are resident at once on this device
  CUtensorMap wmap;                      // DFT matrix terms [3*D][D] bf16
  CUtensorMap pmap;                      // the page region as [frame][plane][kept row][key head][D] (past_frames > 0)
  // Segment entries a compress call left to whoever comes next (see flush_segments): the frames whose
  // segments still have to be pooled, and the stream that call ran on
  mutable bool seg_pending = false;
  mutable long long seg_first = 0;
  mutable int seg_n = 0;
  mutable cudaStream_t seg_stream = nullptr;
  std::string err;
  // optional per-kernel timing (host objects only)
  bool prof_on = false;
  std::vector<cudaEvent_t> prof_ev;      // pairs: start, stop
  std::vector<int> prof_kind;            // kind of each used pair
};

namespace {

mukv_status fail(mukv_ctx* ctx, mukv_status st, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (ctx) ctx->err = buf; else g_create_error = buf;
  return st;
}

// A launch failed after part of a compress call was enqueued: the chunk is half stored and the
// device-side counters no longer match the host's, so the context stops until mukv_reset.
mukv_status broke_off(mukv_ctx* ctx, const char* what, cudaError_t e) {
  ctx->failed = true;
  return fail(ctx, MUKV_E_CUDA, "%s: %s (the chunk is half stored: call mukv_reset)", what, cudaGetErrorString(e));
}

// Brackets one kernel launch with a pair of events when profiling is on.
struct ProfScope {
  mukv_ctx* c;
  cudaStream_t st;
  cudaEvent_t stop = nullptr;
  ProfScope(mukv_ctx* ctx, int kind, cudaStream_t s) : c(ctx), st(s) {
    if (!c->prof_on) return;
    const size_t used = c->prof_kind.size();
    while (c->prof_ev.size() < 2 * (used + 1)) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      c->prof_ev.push_back(e);
    }
    c->prof_kind.push_back(kind);
    cudaEventRecord(c->prof_ev[2 * used], st);
    stop = c->prof_ev[2 * used + 1];
  }
  ~ProfScope() {
    if (stop) cudaEventRecord(stop, st);
  }
};

bool is_pow2(long long x) { return x > 0 && (x & (x - 1)) == 0; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

// Returns nullptr if the configuration is supported, else the reason.
const char* check_config(const mukv_config* c) {
  if (!c) return "null config";
  if (c->dtype != MUKV_BF16 && c->dtype != MUKV_FP32) return "dtype must be MUKV_BF16 or MUKV_FP32";
  if (c->n_layers < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return "layer/head counts must be positive";
  if (c->n_q_heads % c->n_kv_heads != 0) return "n_q_heads must be a multiple of n_kv_heads";
  if (c->head_dim != 64 && c->head_dim != 128) return "head_dim must be 64 or 128";
  if (c->tokens_per_frame < 1 || c->tokens_per_frame > MUKV_MAX_TOKENS) return "tokens_per_frame out of range";
  if (c->keep_per_frame < 1 || c->keep_per_frame > c->tokens_per_frame) return "keep_per_frame out of range";
  if (c->frames_per_segment < 1) return "frames_per_segment must be positive";
  if (c->max_frames_per_chunk < 1 || c->max_frames_per_chunk > 4096) return "max_frames_per_chunk out of range";
  if (c->max_frames < 1) return "max_frames must be positive";
  if (!(c->alpha >= 0.f && c->alpha <= 1.f)) return "alpha must lie in [0, 1]";
  if (!(c->tie_eps >= 0.f)) return "tie_eps must be >= 0";
  if (c->patch_split < 0 || c->patch_split > MUKV_MAX_PATCH_SPLIT) return "patch_split out of range";
  if (c->patch_split > 0 && (c->grid_width < 1 || c->tokens_per_frame % c->grid_width != 0))
    return "grid_width must divide tokens_per_frame when patch_split > 0";
  if (c->reserved != 0) return "reserved fields must be 0";
  if (c->past_frames < 0) return "past_frames must be >= 0";
  if (c->past_frames > 0) {
    if (c->keep_per_segment > 0) return "past keys are not combined with segment-level selection";
    if ((long long)c->past_frames * c->keep_per_frame + c->tokens_per_frame > MUKV_MAX_TOKENS)
      return "past_frames * keep_per_frame + tokens_per_frame must be <= 256";
  }
  if (c->keep_per_segment < 0) return "keep_per_segment must be >= 0";
  if (c->keep_per_segment > 0) {
    if (c->patch_split != 0) return "segment-level selection has no patch level";
    if ((long long)c->frames_per_segment * c->tokens_per_frame > kSegSelMaxTokens)
      return "segment-level selection: frames_per_segment * tokens_per_frame must be <= 4096";
    if (c->keep_per_segment > c->frames_per_segment * c->tokens_per_frame) return "keep_per_segment out of range";
  }
  if (c->n_score_layers < 0 || c->score_layer_offset < 0 ||
      (c->n_score_layers > 1 ? c->n_score_layers : 1) + c->score_layer_offset > c->n_layers)
    return "scoring layers must lie inside the model: n_score_layers + score_layer_offset <= n_layers";
  if ((long long)(c->n_score_layers > 1 ? c->n_score_layers : 1) * c->n_q_heads > 4096) return "too many scoring layers";
  const long long esize = c->dtype == MUKV_BF16 ? 2 : 4;
  const long long row_vec = (long long)c->n_kv_heads * c->head_dim * esize / 16;
  if (!is_pow2(row_vec) || row_vec > 256) return "Hkv*D*sizeof(element)/16 must be a power of two <= 256";
  // the scoring kernel keeps one key head of a frame in shared memory
  const int key_rows = c->tokens_per_frame + c->past_frames * c->keep_per_frame;
  const size_t smem = c->dtype == MUKV_BF16 ? score_smem_bytes<__nv_bfloat16, double>(key_rows, c->head_dim)
                                            : score_smem_bytes<float, double>(key_rows, c->head_dim);
  if (smem > 227 * 1024) return "tokens_per_frame * head_dim too large for shared memory";
  return nullptr;
}

StoreLayout store_layout(const mukv_config& c) {
  StoreLayout s;
  const size_t esize = c.dtype == MUKV_BF16 ? 2 : 4;
  const size_t C = (size_t)c.n_kv_heads * c.head_dim;
  const size_t T = (size_t)c.max_frames;
  s.max_segs = (c.max_frames + c.frames_per_segment - 1) / c.frames_per_segment;
  s.page_bytes = (size_t)c.n_layers * 2 * c.keep_per_frame * C * esize;
  size_t off = 0;
  // segment-level selection: a segment's pages share kappa_v token slots; kept ids are padded to P per frame
  const bool seg_scope = c.keep_per_segment > 0;
  s.pages_bytes = seg_scope ? (size_t)s.max_segs * c.keep_per_segment * c.n_layers * 2 * C * esize : T * s.page_bytes;
  s.kept_stride = seg_scope ? (size_t)c.tokens_per_frame : (size_t)c.keep_per_frame;
  s.pages = off;        off = align_up(off + s.pages_bytes);
  s.kept = off;         off = align_up(off + T * s.kept_stride * sizeof(int));
  s.frame_entry = off;  off = align_up(off + T * c.n_layers * 2 * C * sizeof(float));
  s.seg_entry = off;    off = align_up(off + (size_t)s.max_segs * c.n_layers * 2 * C * sizeof(float));
  s.frame_key = off;    off = align_up(off + T * C * sizeof(float));
  s.seg_key = off;      off = align_up(off + (size_t)s.max_segs * C * sizeof(float));
  s.frame_ts = off;     off = align_up(off + T * sizeof(long long));
  s.page_table = off;   off = align_up(off + T * sizeof(long long));
  s.frame_ksum = off;   off = align_up(off + T * C * sizeof(double));
  const size_t S = (size_t)c.patch_split * c.patch_split;
  s.patch_key = off;    off = align_up(off + T * S * C * sizeof(float));
  s.patch_cnt = off;    off = align_up(off + T * S * sizeof(int));
  s.kept_count = off;   off = align_up(off + (seg_scope ? T * sizeof(int) : 0));
  s.total = off;
  return s;
}

TcShape tc_shape(const mukv_config& c) {
  TcShape t;
  memset(&t, 0, sizeof t);
  const int G = c.n_q_heads / c.n_kv_heads;
  if (c.dtype != MUKV_BF16 || G > 128) return t;
  t.tpt = 128 / G;
  t.tiles = (c.tokens_per_frame + t.tpt - 1) / t.tpt;
  t.npad = (c.tokens_per_frame + 15) / 16 * 16;
  t.own_rows = t.npad;
  if (c.past_frames > 0) {
    // the cached keys of a past frame start on a multiple of eight rows of the key tile (one swizzle
    // atom), behind the frame's own keys
    t.own_rows = (c.tokens_per_frame + 7) / 8 * 8;
    t.past_pad = (c.keep_per_frame + 7) / 8 * 8;
    t.npad = (t.own_rows + c.past_frames * t.past_pad + 15) / 16 * 16;
    if (c.keep_per_segment > 0) return t;               // pages of different lengths are not one regular tensor
  }
  t.n_mt = (c.tokens_per_frame + 127) / 128;
  t.ps_stages = score_ps_stages(t.npad, c.head_dim, 227 * 1024);
  t.smem_ps = score_ps_smem_bytes(t.npad, c.head_dim, t.ps_stages < 2 ? 2 : t.ps_stages);
  t.ok = t.ps_stages >= 2 && t.npad <= kPsSplit * kPsAccCols;
  return t;
}

constexpr int kRefineSplit = 4;     // blocks per query head in the double-precision pass
// Single precision decides a frame only when its lowest kept and highest dropped fused score are
// further apart than tie_eps + kFlagMargin; a signal whose range is below kFlatRatio of its
// magnitude (the min-max division then amplifies rounding noise) also sends the frame to the
// double-precision pass.
constexpr float kFlagMargin = 3e-6f;
constexpr float kFlatRatio = 1e-3f;

WorkLayout work_layout(const mukv_config& c) {
  WorkLayout w;
  const size_t F = c.max_frames_per_chunk, P = c.tokens_per_frame;
  const size_t C = (size_t)c.n_kv_heads * c.head_dim;
  const size_t max_segs = (c.max_frames + c.frames_per_segment - 1) / c.frames_per_segment;
  size_t off = 0;
  const TcShape ts = tc_shape(c);
  const size_t Ls = c.n_score_layers > 1 ? c.n_score_layers : 1;
  w.colsum_f = off;       off = align_up(off + F * Ls * (size_t)c.n_q_heads * P * sizeof(float));
  w.colsum_p = off;       off = align_up(off + (ts.ok ? (kPsMaxBlocks + F) * P * sizeof(float) : 0));
  w.ifft_f = off;         off = align_up(off + F * Ls * c.n_kv_heads * P * sizeof(float));
  w.colsum_d = off;       off = align_up(off + F * Ls * c.n_q_heads * kRefineSplit * P * sizeof(double));
  w.ifft_d = off;         off = align_up(off + F * Ls * c.n_kv_heads * P * sizeof(double));
  w.zero_begin = off;
  w.frame_counter = off;  off = align_up(off + F * sizeof(int));
  w.flagged = off;        off = align_up(off + F * sizeof(int));
  w.n_flagged = off;      off = align_up(off + 2 * sizeof(int));   // alternate between chunks
  w.tail_ctr = off;       off = align_up(off + 2 * sizeof(int));
  w.sel_flag = off;       off = align_up(off + F * sizeof(unsigned));
  w.seg_flag = off;       off = align_up(off + F * sizeof(int));
  w.stat_refined = off;   off = align_up(off + sizeof(long long));
  w.dev_status = off;     off = align_up(off + sizeof(int));
  w.zero_end = off;
  w.q64 = off;            off = align_up(off + (size_t)MUKV_MAX_QUESTIONS * C * sizeof(double));
  w.qnorm = off;          off = align_up(off + (size_t)MUKV_MAX_QUESTIONS * c.n_kv_heads * sizeof(double));
  w.s_frm = off;          off = align_up(off + (size_t)MUKV_MAX_QUESTIONS * c.max_frames * sizeof(double));
  w.s_seg = off;          off = align_up(off + (size_t)MUKV_MAX_QUESTIONS * max_segs * sizeof(double));
  w.s_pat = off;          off = align_up(off + (size_t)MUKV_MAX_QUESTIONS * c.max_frames * c.patch_split * c.patch_split *
                                               sizeof(double));
  w.wtab = off;           off = align_up(off + (ts.ok ? (size_t)3 * c.head_dim * c.head_dim * 2 : 0));
  w.total = off;
  return w;
}

int pick_nc(int P) { return P <= 64 ? 2 : P <= 128 ? 4 : P <= 224 ? 7 : 8; }

// Launches a kernel; with `dependent` it may be scheduled while the previous kernel of the stream
// still runs (programmatic dependent launch: the kernel itself waits in pdl_wait()).
template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, unsigned block, size_t smem, cudaStream_t st,
                     bool dependent, Args... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = grid;
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <typename T>
const void* tail_fn(int nc) {
  switch (nc) {
    case 2: return (const void*)tail_kernel<T, 2>;
    case 4: return (const void*)tail_kernel<T, 4>;
    case 7: return (const void*)tail_kernel<T, 7>;
    default: return (const void*)tail_kernel<T, 8>;
  }
}

template <typename T>
cudaError_t launch_tail(const ScoreParams& sp, const CompactParams& cp, int nc, int grid, size_t smem, cudaStream_t st,
                        bool dependent) {
  switch (nc) {
    case 2: return launch_k(tail_kernel<T, 2>, dim3(grid), kScoreThreads, smem, st, dependent, sp, cp);
    case 4: return launch_k(tail_kernel<T, 4>, dim3(grid), kScoreThreads, smem, st, dependent, sp, cp);
    case 7: return launch_k(tail_kernel<T, 7>, dim3(grid), kScoreThreads, smem, st, dependent, sp, cp);
    default: return launch_k(tail_kernel<T, 8>, dim3(grid), kScoreThreads, smem, st, dependent, sp, cp);
  }
}

template <typename T, typename A>
cudaError_t launch_score(const ScoreParams& sp, int nc, dim3 grid, size_t smem, cudaStream_t st,
                         bool dependent = false) {
  switch (nc) {
    case 2: return launch_k(score_kernel<T, A, 2>, grid, kScoreThreads, smem, st, dependent, sp);
    case 4: return launch_k(score_kernel<T, A, 4>, grid, kScoreThreads, smem, st, dependent, sp);
    case 7: return launch_k(score_kernel<T, A, 7>, grid, kScoreThreads, smem, st, dependent, sp);
    default: return launch_k(score_kernel<T, A, 8>, grid, kScoreThreads, smem, st, dependent, sp);
  }
}

// Raises a kernel's dynamic shared-memory limit to everything the device allows beside the
// kernel's static shared memory.
cudaError_t raise_smem_limit(const void* fn, int optin) {
  cudaFuncAttributes fa;
  cudaError_t e = cudaFuncGetAttributes(&fa, fn);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - (int)fa.sharedSizeBytes);
}

template <typename T, typename A>
cudaError_t raise_score_limits(int optin) {
  cudaError_t e = raise_smem_limit((const void*)score_kernel<T, A, 2>, optin);
  if (e == cudaSuccess) e = raise_smem_limit((const void*)score_kernel<T, A, 4>, optin);
  if (e == cudaSuccess) e = raise_smem_limit((const void*)score_kernel<T, A, 7>, optin);
  if (e == cudaSuccess) e = raise_smem_limit((const void*)score_kernel<T, A, 8>, optin);
  return e;
}

constexpr int kMaxDevices = 64;
std::mutex g_dev_mutex;
bool g_limits_raised[kMaxDevices];

// Once per device (that device current): the dynamic shared-memory limit of every kernel that
// needs more than the default goes to the device's maximum.  The limit belongs to the kernel,
// not to a context, so it is never set to one context's need: a second context of another
// shape, or the allocation-free entry point, would otherwise find it too low.
cudaError_t raise_kernel_limits(int* n_sms) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (n_sms) {
    e = cudaDeviceGetAttribute(n_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_dev_mutex);
  if (g_limits_raised[dev]) return cudaSuccess;
  int optin = 0;
  e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e == cudaSuccess) e = raise_score_limits<__nv_bfloat16, float>(optin);
  if (e == cudaSuccess) e = raise_score_limits<__nv_bfloat16, double>(optin);
  if (e == cudaSuccess) e = raise_score_limits<float, float>(optin);
  if (e == cudaSuccess) e = raise_score_limits<float, double>(optin);
  const int ncs[4] = {2, 4, 7, 8};
  for (int i = 0; i < 4 && e == cudaSuccess; ++i) {
    e = raise_smem_limit(tail_fn<__nv_bfloat16>(ncs[i]), optin);
    if (e == cudaSuccess) e = raise_smem_limit(tail_fn<float>(ncs[i]), optin);
  }
  if (e == cudaSuccess) e = raise_smem_limit((const void*)rank_kernel, optin);
  if (e == cudaSuccess) e = raise_smem_limit((const void*)segsel_kernel, optin);
  if (e == cudaSuccess) e = raise_smem_limit((const void*)score_ps_kernel<false>, optin);
  if (e == cudaSuccess) e = raise_smem_limit((const void*)score_ps_kernel<true>, optin);
  if (e == cudaSuccess) g_limits_raised[dev] = true;
  return e;
}

// ---------------------------------------------------------------- TMA descriptors
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// bf16 tensor [rows][mid][D] (D contiguous) seen as a rank-3 map; the box is box_rows x box_mid x 64
// channels, written to shared memory with the 128-byte swizzle.  Out-of-range rows read as zero.
bool encode_map3(CUtensorMap* m, const void* base, int D, int mid, long long rows, int box_mid, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)mid, (cuuint64_t)rows};
  const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)mid * D * 2};
  const cuuint32_t box[3] = {64u, (cuuint32_t)box_mid, (cuuint32_t)box_rows};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The pages of a store with frame-level selection, bf16: [frames][2L planes][kappa rows][Hkv][D] as a
// rank-5 map; the box is the kappa rows of one key head in one plane of one page, 64 channels wide.
bool encode_map_pages(CUtensorMap* m, const void* pages, int D, int Hkv, int kappa, int planes, long long frames,
                      long long page_bytes) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t row = (cuuint64_t)Hkv * D * 2;
  const cuuint64_t dims[5] = {(cuuint64_t)D, (cuuint64_t)Hkv, (cuuint64_t)kappa, (cuuint64_t)planes, (cuuint64_t)frames};
  const cuuint64_t strides[4] = {(cuuint64_t)D * 2, row, row * kappa, (cuuint64_t)page_bytes};
  const cuuint32_t box[5] = {64u, 1u, (cuuint32_t)kappa, 1u, 1u};
  const cuuint32_t estr[5] = {1u, 1u, 1u, 1u, 1u};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(pages), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_map2(CUtensorMap* m, const void* base, int cols, long long rows, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

uint16_t bf16_rne(float x) {
  uint32_t b;
  memcpy(&b, &x, 4);
  b += 0x7FFFu + ((b >> 16) & 1u);
  return (uint16_t)(b >> 16);
}
float bf16_val(uint16_t h) {
  const uint32_t b = (uint32_t)h << 16;
  float x;
  memcpy(&x, &b, 4);
  return x;
}

// The D-point DFT as a matrix, rows = output column n, columns = input channel d (the layout of
// a K-major B operand): n <= D/2 holds cos(2 pi n d / D), n > D/2 holds -sin(2 pi (n - D/2) d / D).
// Each entry is split into three bf16 terms, hi + mid + lo, stored as [3][D][D].
std::vector<uint16_t> dft_terms(int D) {
  std::vector<uint16_t> w((size_t)3 * D * D);
  const double pi = 3.14159265358979323846;
  for (int n = 0; n < D; ++n)
    for (int d = 0; d < D; ++d) {
      const int b = n <= D / 2 ? n : n - D / 2;
      const int m = (int)(((long long)b * d) % D);
      const double ang = 2.0 * pi * (double)m / (double)D;
      const double x = n <= D / 2 ? std::cos(ang) : -std::sin(ang);
      const uint16_t hi = bf16_rne((float)x);
      const double r1 = x - (double)bf16_val(hi);
      const uint16_t mid = bf16_rne((float)r1);
      const double r2 = r1 - (double)bf16_val(mid);
      const uint16_t lo = bf16_rne((float)r2);
      w[((size_t)0 * D + n) * D + d] = hi;
      w[((size_t)1 * D + n) * D + d] = mid;
      w[((size_t)2 * D + n) * D + d] = lo;
    }
  return w;
}

// The pooling of segment entries (Eq. 5 at segment level) for frames first .. first + n - 1.
SegmentArgs segment_args_of(const mukv_ctx* ctx, long long first, int n) {
  const mukv_config& c = ctx->cfg;
  SegmentArgs a;
  memset(&a, 0, sizeof a);
  a.L = c.n_layers; a.kappa = c.keep_per_frame; a.C = ctx->C; a.fseg = c.frames_per_segment;
  a.n_frames = n; a.first_frame = first;
  a.frame_entry = reinterpret_cast<const float*>(ctx->store + ctx->sl.frame_entry);
  a.frame_ksum = reinterpret_cast<const double*>(ctx->store + ctx->sl.frame_ksum);
  a.seg_entry = reinterpret_cast<float*>(ctx->store + ctx->sl.seg_entry);
  a.seg_key = reinterpret_cast<float*>(ctx->store + ctx->sl.seg_key);
  if (c.keep_per_segment > 0) a.kept_count = reinterpret_cast<const int*>(ctx->store + ctx->sl.kept_count);
  return a;
}

// A compress call does not pool the segment entries of its chunk itself (unless frames were flagged:
// tail_kernel then does): the next compress call does it with blocks that do not wait for that call's
// scoring kernel (one more row in its compaction kernel; with segment-level selection, extra blocks of its
// first segsel_kernel launch).  Whoever else needs the entries first
// (retrieval, a gather with summary tokens, a view of the store, an export) pools them with one launch here.
cudaError_t flush_segments(const mukv_ctx* ctx, cudaStream_t st) {
  if (!ctx->seg_pending) return cudaSuccess;
  CompactParams cp;
  memset(&cp, 0, sizeof cp);
  const SegmentArgs a = segment_args_of(ctx, ctx->seg_first, ctx->seg_n);
  cp.L = a.L; cp.kappa = a.kappa; cp.C = a.C; cp.fseg = a.fseg; cp.n_frames = a.n_frames; cp.first_frame = a.first_frame;
  cp.frame_entry = const_cast<float*>(a.frame_entry); cp.frame_ksum = const_cast<double*>(a.frame_ksum);
  cp.seg_entry = a.seg_entry; cp.seg_key = a.seg_key; cp.kept_count = a.kept_count;
  cp.pool_always = 1;
  const cudaError_t e = launch_k(segment_kernel, dim3(2 * a.L), kCompactThreads, 0, st, false, cp);
  if (e == cudaSuccess) ctx->seg_pending = false;
  return e;
}

// Scores a bf16 chunk on the tensor cores (Eq. 1-3; Eq. 4 and the selection follow in compact_kernel).
cudaError_t launch_score_ps(mukv_ctx* ctx, const ScoreParams& sp, const void* d_q, const void* k_last, int n,
                            cudaStream_t st, const char** why, int* ps_grid, int* ps_items, int* ps_ipf) {
  *ps_grid = 0;
  const mukv_config& c = ctx->cfg;
  const TcShape& t = ctx->tcs;
  const int P = c.tokens_per_frame, D = c.head_dim;
  CUtensorMap qmap, kmap;
  const long long rows = (long long)ctx->Ls * n * P;
  if (!encode_map3(&qmap, d_q, D, c.n_q_heads, rows, ctx->G, t.tpt) ||
      !encode_map3(&kmap, k_last, D, c.n_kv_heads, rows, 1, t.own_rows)) {
    *why = "cuTensorMapEncodeTiled failed";
    return cudaErrorInvalidValue;
  }
  ScorePsParams pp;
  memset(&pp, 0, sizeof pp);
  pp.sp = sp;
  pp.sp.colsum_part = ctx->ws + ctx->wl.colsum_p;
  pp.tiles = t.tiles; pp.tpt = t.tpt; pp.npad = t.npad; pp.n_mt = t.n_mt; pp.n_stages = t.ps_stages;
  pp.own_rows = t.own_rows; pp.n_past = sp.n_past_frames; pp.past_pad = t.past_pad; pp.kappa = c.keep_per_frame;
  pp.past_plane0 = 2 * sp.first_score_layer; pp.past_first = sp.past_first;
  pp.n_items = n * ctx->Ls * c.n_kv_heads * (t.n_mt + t.tiles);
  pp.exp2_scale = (float)(1.4426950408889634 / std::sqrt((double)D));
  pp.status = reinterpret_cast<int*>(ctx->ws + ctx->wl.dev_status);
  int blocks = ctx->n_sms < kPsMaxBlocks ? ctx->n_sms : kPsMaxBlocks;
  if (blocks > pp.n_items) blocks = pp.n_items;
  *ps_grid = blocks; *ps_items = pp.n_items; *ps_ipf = ctx->Ls * c.n_kv_heads * (t.n_mt + t.tiles);
  if (sp.n_past_frames)
    score_ps_kernel<true><<<blocks, kPsThreads, t.smem_ps, st>>>(pp, qmap, kmap, ctx->wmap, ctx->pmap);
  else
    score_ps_kernel<false><<<blocks, kPsThreads, t.smem_ps, st>>>(pp, qmap, kmap, ctx->wmap, kmap);
  *why = "score_ps kernel";
  return cudaGetLastError();
}

template <typename T>
mukv_status compress_impl(mukv_ctx* ctx, const void* d_q, const float* d_ext, const void* d_k, const void* d_v, int n,
                          long long t0, int* d_kept_out, float* d_scores_out, cudaStream_t st) {
  const mukv_config& c = ctx->cfg;
  const int P = c.tokens_per_frame, L = c.n_layers, C = ctx->C;
  const bool seg_scope = c.keep_per_segment > 0;
  if (seg_scope) {
    if (d_ext) return fail(ctx, MUKV_E_UNSUPPORTED, "caller-supplied scores are ranked per frame only");
    if (t0 % c.frames_per_segment != 0)
      return fail(ctx, MUKV_E_STATE, "segment-level selection: first_frame must be a multiple of frames_per_segment");
  }
  ScoreParams sp;
  memset(&sp, 0, sizeof sp);
  sp.P = P; sp.Hq = c.n_q_heads; sp.Hkv = c.n_kv_heads; sp.D = c.head_dim; sp.G = ctx->G;
  sp.kappa = c.keep_per_frame; sp.n_frames = n; sp.causal = c.attn_causal; sp.keep_low = c.keep_low_freq;
  sp.alpha = c.alpha; sp.tie_eps = c.tie_eps; sp.flag_margin = ctx->flag_margin; sp.flat_ratio = ctx->flat_ratio;
  sp.first_frame = t0;
  sp.q = d_q;
  sp.Ls = ctx->Ls;
  sp.q_layer_stride = (long long)n * P * c.n_q_heads * c.head_dim;
  sp.k_layer_stride = (long long)n * P * C;
  sp.k_last = reinterpret_cast<const T*>(d_k) + (long long)(L - c.score_layer_offset - ctx->Ls) * n * P * C;
  sp.colsum_part = ctx->ws + ctx->wl.colsum_f;
  sp.ifft_part = ctx->ws + ctx->wl.ifft_f;
  sp.frame_counter = reinterpret_cast<int*>(ctx->ws + ctx->wl.frame_counter);
  sp.flagged = reinterpret_cast<int*>(ctx->ws + ctx->wl.flagged);
  sp.n_flagged = reinterpret_cast<int*>(ctx->ws + ctx->wl.n_flagged) + ctx->parity;
  sp.kept_store = reinterpret_cast<int*>(ctx->store + ctx->sl.kept);
  sp.kept_out = d_kept_out;
  sp.scores_out = d_scores_out;
  sp.frame_ts = reinterpret_cast<long long*>(ctx->store + ctx->sl.frame_ts);
  sp.page_table = reinterpret_cast<long long*>(ctx->store + ctx->sl.page_table);
  sp.pages_off = (long long)ctx->sl.pages;
  sp.page_bytes = (long long)ctx->sl.page_bytes;
  sp.status = reinterpret_cast<int*>(ctx->ws + ctx->wl.dev_status);
  sp.store = ctx->store;
  sp.first_score_layer = L - c.score_layer_offset - ctx->Ls;
  sp.past_first = t0 - c.past_frames > 0 ? t0 - c.past_frames : 0;
  sp.n_past_frames = c.past_frames > 0 ? (int)(t0 - sp.past_first) : 0;
  sp.refine = 0;
  sp.row_split = 1;
  const dim3 grid(ctx->Ls * c.n_q_heads, n);
  cudaError_t e = cudaSuccess;
  const char* what = "score kernel";
  int ps_grid = 0, ps_items = 0, ps_ipf = 0;
  int n_launch = 0;
  if (seg_scope) {
    // One block per segment ranks all its tokens.  A bf16 chunk is first scored on the tensor cores and
    // ranked from those single-precision sums; segments that are too close to call are scored and
    // ranked again in double precision (both launches of that pass return at once for the others).
    // Any other chunk goes through the double-precision pass as a whole.
    const bool tc_first = ctx->tcs.ok && !ctx->force_fma;
    const int n_seg = (n + c.frames_per_segment - 1) / c.frames_per_segment;
    const int seg_tokens = (n < c.frames_per_segment ? n : c.frames_per_segment) * P;
    const bool dep = !ctx->prof_on;
    SegSelParams gp;
    memset(&gp, 0, sizeof gp);
    gp.fseg = c.frames_per_segment; gp.kappa_v = c.keep_per_segment;
    gp.token_bytes = (long long)L * 2 * C * ctx->esize;
    gp.kept_count = reinterpret_cast<int*>(ctx->store + ctx->sl.kept_count);
    gp.seg_flag = reinterpret_cast<int*>(ctx->ws + ctx->wl.seg_flag);
    gp.n_seg = n_seg;
    // Segment entries the previous call left behind: pooled by extra blocks of the first segsel_kernel launch
    // (that kernel uses one SM per segment); with per-kernel timing on, by a launch of their own
    if (ctx->seg_pending && ctx->prof_on) {
      ProfScope ps(ctx, 3, st);
      e = flush_segments(ctx, st);
      if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "segment kernel: %s", cudaGetErrorString(e));
      ++n_launch;
    }
    int extra = 0;
    if (ctx->seg_pending) {
      gp.prev = segment_args_of(ctx, ctx->seg_first, ctx->seg_n);
      extra = 2 * L;
    }
    gp.stat_refined = reinterpret_cast<unsigned long long*>(ctx->ws + ctx->wl.stat_refined);
    if (tc_first) {
      int ps_grid1 = 0, ps_items1 = 0, ps_ipf1 = 0;
      {
        ProfScope ps(ctx, 0, st);
        e = launch_score_ps(ctx, sp, d_q, sp.k_last, n, st, &what, &ps_grid1, &ps_items1, &ps_ipf1);
      }
      if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "%s: %s", what, cudaGetErrorString(e));
      n_launch += 2;
      gp.sp = sp;
      gp.sp.colsum_part = ctx->ws + ctx->wl.colsum_p;
      gp.src32 = 1;
      gp.ps_grid = ps_grid1; gp.ps_items = ps_items1; gp.ps_ipf = ps_ipf1;
      {
        ProfScope ps(ctx, 1, st);
        e = launch_k(segsel_kernel, dim3(n_seg + extra), kSegSelThreads, segsel_smem_bytes(seg_tokens), st, dep, gp);
      }
      if (e != cudaSuccess) return broke_off(ctx, "segment selection kernel", e);
      ctx->seg_pending = false;
      extra = 0;
      memset(&gp.prev, 0, sizeof gp.prev);
    }
    ScoreParams sd = sp;
    sd.no_select = 1;
    sd.row_split = kRefineSplit;
    sd.colsum_part = ctx->ws + ctx->wl.colsum_d;
    sd.ifft_part = ctx->ws + ctx->wl.ifft_d;
    if (tc_first) {
      sd.seg_gate = gp.seg_flag;
      sd.gate_fseg = c.frames_per_segment;
    }
    {
      ProfScope ps(ctx, tc_first ? 1 : 0, st);
      const int units = ctx->Ls * c.n_q_heads * kRefineSplit;
      const dim3 grid_d = tc_first ? dim3(units < 2 * ctx->n_sms ? units : 2 * ctx->n_sms) : dim3(units, n);
      e = launch_score<T, double>(sd, ctx->nc, grid_d,
                                  score_smem_bytes<T, double>(P, c.head_dim), st, tc_first && dep);
    }
    if (e != cudaSuccess) {
      if (tc_first) return broke_off(ctx, "score kernel", e);
      return fail(ctx, MUKV_E_CUDA, "score kernel: %s", cudaGetErrorString(e));
    }
    gp.sp = sd;
    gp.src32 = 0;
    gp.only_flagged = tc_first ? 1 : 0;
    {
      ProfScope ps(ctx, 1, st);
      e = launch_k(segsel_kernel, dim3(n_seg + extra), kSegSelThreads, segsel_smem_bytes(seg_tokens), st, tc_first && dep,
                   gp);
    }
    if (e != cudaSuccess) return broke_off(ctx, "segment selection kernel", e);
    ctx->seg_pending = false;
    n_launch += 2;
  } else if (!d_ext) {
    ProfScope ps(ctx, 0, st);
    if (ctx->tcs.ok && !ctx->force_fma)
      e = launch_score_ps(ctx, sp, d_q, sp.k_last, n, st, &what, &ps_grid, &ps_items, &ps_ipf);
    else
      e = launch_score<T, float>(sp, ctx->nc, grid, score_smem_bytes<T, float>(ctx->key_rows, c.head_dim), st);
    ++n_launch;
  }
  if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "%s: %s", what, cudaGetErrorString(e));

  // Compaction of every frame that single precision decides; after the persistent scoring kernel
  // its blocks also do the selection (Eq. 4, top-kappa) from that kernel's partial sums.
  CompactParams cp;
  memset(&cp, 0, sizeof cp);
  cp.L = L; cp.kappa = c.keep_per_frame; cp.C = C; cp.P = P; cp.n_frames = n; cp.first_frame = t0;
  cp.k = d_k; cp.v = d_v;
  cp.store = ctx->store;
  cp.frame_entry = reinterpret_cast<float*>(ctx->store + ctx->sl.frame_entry);
  cp.frame_key = reinterpret_cast<float*>(ctx->store + ctx->sl.frame_key);
  cp.frame_ksum = reinterpret_cast<double*>(ctx->store + ctx->sl.frame_ksum);
  cp.stat_refined = reinterpret_cast<long long*>(ctx->ws + ctx->wl.stat_refined);
  cp.tail_ctr = reinterpret_cast<int*>(ctx->ws + ctx->wl.tail_ctr);
  cp.sel_flag = reinterpret_cast<unsigned*>(ctx->ws + ctx->wl.sel_flag);
  cp.epoch = (++ctx->epoch) & 0x7fffffffu;
  cp.n_flagged_next = reinterpret_cast<int*>(ctx->ws + ctx->wl.n_flagged) + (ctx->parity ^ 1);
  cp.fseg = c.frames_per_segment;
  cp.seg_entry = reinterpret_cast<float*>(ctx->store + ctx->sl.seg_entry);
  cp.seg_key = reinterpret_cast<float*>(ctx->store + ctx->sl.seg_key);
  cp.patch_split = c.patch_split; cp.grid_width = c.grid_width;
  cp.patch_key = reinterpret_cast<float*>(ctx->store + ctx->sl.patch_key);
  cp.patch_cnt = reinterpret_cast<int*>(ctx->store + ctx->sl.patch_cnt);
  cp.sel_mode = seg_scope ? 3 : d_ext ? 2 : ps_grid > 0 ? 1 : 0;
  cp.kept_count = seg_scope ? reinterpret_cast<const int*>(ctx->store + ctx->sl.kept_count) : nullptr;
  cp.ext_scores = d_ext;
  cp.ps_grid = ps_grid; cp.ps_items = ps_items; cp.ps_ipf = ps_ipf;
  cp.sp = sp;
  if (ps_grid > 0) cp.sp.colsum_part = ctx->ws + ctx->wl.colsum_p;
  // segment entries the previous call left behind: one more row of blocks (with per-kernel timing on,
  // a launch of their own, so that each kernel is timed doing its own work only)
  if (ctx->seg_pending && ctx->prof_on) {
    ProfScope ps(ctx, 3, st);
    e = flush_segments(ctx, st);
    if (e != cudaSuccess) return broke_off(ctx, "segment kernel", e);
    ++n_launch;
  }
  if (ctx->seg_pending) cp.prev = segment_args_of(ctx, ctx->seg_first, ctx->seg_n);
  {
    ProfScope ps(ctx, 2, st);
    e = launch_k(compact_kernel<T>, dim3(n, L * 2 + (c.patch_split > 0 ? 1 : 0) + (ctx->seg_pending ? 1 : 0)),
                 kCompactThreads, 0, st, !ctx->prof_on, cp);
  }
  if (e != cudaSuccess) return broke_off(ctx, "compact kernel", e);
  ctx->seg_pending = false;

  // The segment entries need every frame of the chunk.  They are left to the next call (flush_segments);
  // when frames were flagged, tail_kernel pools them after it has redone those frames.
  cp.sp.n_flagged = sp.n_flagged;
  sp.refine = 1;
  sp.row_split = kRefineSplit;
  sp.colsum_part = ctx->ws + ctx->wl.colsum_d;
  sp.ifft_part = ctx->ws + ctx->wl.ifft_d;
  if (!seg_scope) {                                      // (segment-level selection flags nothing)
    ProfScope ps(ctx, 1, st);
    int grid_t = ctx->Ls * c.n_q_heads * kRefineSplit * (n < 2 ? n : 2);
    if (grid_t < 2 * L + 1) grid_t = 2 * L + 1;
    if (grid_t > ctx->tail_capacity) grid_t = ctx->tail_capacity;
    e = launch_tail<T>(sp, cp, ctx->nc, grid_t, score_smem_bytes<T, double>(ctx->key_rows, c.head_dim), st, !ctx->prof_on);
    ++n_launch;
  }
  if (e != cudaSuccess) return broke_off(ctx, "tail kernel", e);
  ctx->seg_pending = true;
  ctx->seg_first = t0;
  ctx->seg_n = n;
  ctx->seg_stream = st;

  ctx->launches += n_launch + 1;                          // + compact_kernel
  ctx->parity ^= 1;
  ctx->frames = t0 + n;
  return MUKV_OK;
}

mukv_status create_impl(const mukv_config* cfg, void* d_store, size_t store_bytes, void* d_workspace,
                        size_t workspace_bytes, long long frames0, mukv_ctx** out);

mukv_status retrieve_impl(mukv_ctx* ctx, const void* d_qtok, const int32_t* h_q_offsets, const int64_t* h_t_limit,
                          int32_t nq, const mukv_retr_params& prm, int32_t* d_seg_idx, int32_t* d_frm_idx,
                          int32_t* d_pat_idx, float* d_seg_score, float* d_frm_score, float* d_pat_score,
                          int32_t* d_counts, int counts_stride, mukv_stream stream) {
  try {
    const int k_seg = prm.k_seg, k_frm = prm.k_frm, k_pat = prm.k_patch, top_n = prm.top_n, mode = prm.mode;
    if (ctx->failed) return fail(ctx, MUKV_E_STATE, "an earlier call broke off half way: call mukv_reset");
    if (!d_qtok || !h_q_offsets || !d_seg_idx || !d_frm_idx || !d_counts)
      return fail(ctx, MUKV_E_INVALID, "null argument");
    if (!aligned16(d_qtok) || !aligned4(d_seg_idx) || !aligned4(d_frm_idx) || !aligned4(d_seg_score) ||
        !aligned4(d_frm_score) || !aligned4(d_counts))
      return fail(ctx, MUKV_E_ALIGN, "d_qtok must be 16-byte aligned, the outputs 4-byte aligned");
    if (nq < 1) return fail(ctx, MUKV_E_INVALID, "nq must be >= 1");
    if (nq > MUKV_MAX_QUESTIONS) return fail(ctx, MUKV_E_CAPACITY, "nq %d exceeds %d", nq, MUKV_MAX_QUESTIONS);
    if (k_seg < 1 || k_frm < 1 || k_pat < 0 || top_n < 0)
      return fail(ctx, MUKV_E_INVALID, "k_seg, k_frm must be >= 1, k_patch and top_n >= 0");
    if (k_seg > MUKV_MAX_TOPK || k_frm > MUKV_MAX_TOPK || k_pat > MUKV_MAX_TOPK || top_n > MUKV_MAX_TOPK)
      return fail(ctx, MUKV_E_CAPACITY, "k_seg / k_frm / k_patch / top_n exceed %d", MUKV_MAX_TOPK);
    if (k_pat > 0 && ctx->cfg.patch_split == 0) return fail(ctx, MUKV_E_STATE, "the store has no patch level");
    if (k_pat > 0 && !d_pat_idx) return fail(ctx, MUKV_E_INVALID, "d_patch_idx is null");
    if (!aligned4(d_pat_idx) || !aligned4(d_pat_score)) return fail(ctx, MUKV_E_ALIGN, "outputs must be 4-byte aligned");
    if (mode != MUKV_RETR_PARALLEL && mode != MUKV_RETR_HIER && mode != MUKV_RETR_SEMI)
      return fail(ctx, MUKV_E_INVALID, "unknown retrieval mode %d", mode);
    for (float lam : {prm.lambda_patch, prm.lambda_frm, prm.lambda_seg})
      if (!(lam >= 0.f && lam <= 1.f)) return fail(ctx, MUKV_E_INVALID, "every lambda must lie in [0, 1]");
    if (ctx->frames < 1) return fail(ctx, MUKV_E_STATE, "the store is empty");
    if (ctx->seg_pending) {                                // the last chunk's segment entries are read below
      const cudaError_t ef = flush_segments(ctx, static_cast<cudaStream_t>(stream));
      if (ef != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "segment kernel: %s", cudaGetErrorString(ef));
      ctx->launches += 1;
    }
    QMeta meta;
    if (h_q_offsets[0] != 0) return fail(ctx, MUKV_E_INVALID, "q_offsets[0] must be 0");
    for (int i = 0; i < nq; ++i) {
      if (h_q_offsets[i + 1] <= h_q_offsets[i])
        return fail(ctx, MUKV_E_INVALID, "question %d has no tokens (offsets must ascend)", i);
      if (h_t_limit && h_t_limit[i] < 0) return fail(ctx, MUKV_E_INVALID, "t_limit[%d] is negative", i);
    }
    for (int i = 0; i <= nq; ++i) meta.off[i] = h_q_offsets[i];
    for (int i = 0; i < nq; ++i) meta.t_limit[i] = h_t_limit ? (long long)h_t_limit[i] : ctx->frames;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const mukv_config& c = ctx->cfg;
    const int C = ctx->C;
    double* q64 = reinterpret_cast<double*>(ctx->ws + ctx->wl.q64);
    double* qnorm = reinterpret_cast<double*>(ctx->ws + ctx->wl.qnorm);
    double* s_frm = reinterpret_cast<double*>(ctx->ws + ctx->wl.s_frm);
    double* s_seg = reinterpret_cast<double*>(ctx->ws + ctx->wl.s_seg);
    const float* frame_key = reinterpret_cast<const float*>(ctx->store + ctx->sl.frame_key);
    const float* seg_key = reinterpret_cast<const float*>(ctx->store + ctx->sl.seg_key);
    const long long n_frm = ctx->frames;
    const long long n_seg = (n_frm + c.frames_per_segment - 1) / c.frames_per_segment;
    {
      ProfScope ps(ctx, 4, st);
      if (c.dtype == MUKV_BF16)
        qpool_kernel<__nv_bfloat16><<<dim3(nq, c.n_kv_heads), kPoolThreads, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(d_qtok), meta,
                                                       c.n_q_heads, c.n_kv_heads, c.head_dim, q64, qnorm);
      else
        qpool_kernel<float><<<dim3(nq, c.n_kv_heads), kPoolThreads, 0, st>>>(reinterpret_cast<const float*>(d_qtok), meta, c.n_q_heads,
                                               c.n_kv_heads, c.head_dim, q64, qnorm);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "qpool kernel: %s", cudaGetErrorString(e));
    const int S = c.patch_split * c.patch_split;
    const long long n_pat = k_pat > 0 ? n_frm * S : 0;
    const long long rows = n_frm + n_seg + n_pat;
    const unsigned blocks = (unsigned)((rows + kScanRows - 1) / kScanRows);
    double* s_pat = reinterpret_cast<double*>(ctx->ws + ctx->wl.s_pat);
    const float* patch_key = reinterpret_cast<const float*>(ctx->store + ctx->sl.patch_key);
    {
      ProfScope ps(ctx, 5, st);
      ScanParams sc;
      memset(&sc, 0, sizeof sc);
      sc.frame_key = frame_key; sc.seg_key = seg_key; sc.patch_key = patch_key;
      sc.n_frm = n_frm; sc.n_seg = n_seg; sc.n_pat = n_pat;
      sc.C = C; sc.nq = nq; sc.Hkv = c.n_kv_heads; sc.q64t = q64; sc.qn2 = qnorm;
      sc.s_frm = s_frm; sc.s_seg = s_seg; sc.s_pat = s_pat;
      sc.frm_stride = c.max_frames; sc.seg_stride = ctx->sl.max_segs; sc.pat_stride = (long long)c.max_frames * S;
      e = launch_k(scan_kernel, dim3(blocks), 256, 0, st, !ctx->prof_on, sc);
    }
    if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "scan kernel: %s", cudaGetErrorString(e));
    RankParams rp;
    memset(&rp, 0, sizeof rp);
    rp.nq = nq; rp.C = C; rp.fseg = c.frames_per_segment;
    rp.k_seg = k_seg; rp.k_frm = k_frm; rp.k_pat = k_pat; rp.top_n = top_n; rp.mode = mode; rp.S = S;
    rp.lam_seg = (double)prm.lambda_seg; rp.lam_frm = (double)prm.lambda_frm; rp.lam_pat = (double)prm.lambda_patch;
    rp.delta = (double)c.tie_eps;
    rp.n_frm = n_frm; rp.n_seg = n_seg;
    rp.s_frm = s_frm; rp.s_seg = s_seg; rp.s_pat = s_pat;
    rp.frm_stride = c.max_frames; rp.seg_stride = ctx->sl.max_segs; rp.pat_stride = (long long)c.max_frames * S;
    rp.frame_key = frame_key; rp.seg_key = seg_key; rp.patch_key = patch_key;
    rp.patch_cnt = reinterpret_cast<const int*>(ctx->store + ctx->sl.patch_cnt);
    rp.seg_idx = d_seg_idx; rp.frm_idx = d_frm_idx; rp.pat_idx = d_pat_idx;
    rp.seg_score = d_seg_score; rp.frm_score = d_frm_score; rp.pat_score = d_pat_score;
    rp.counts = d_counts; rp.counts_stride = counts_stride;
    {
      ProfScope ps(ctx, 6, st);
      size_t rank_smem = (size_t)C * sizeof(double);
      const size_t staged = rank_smem + (size_t)(n_frm + n_seg) * sizeof(double);
      rp.stage = staged <= (size_t)kRankStageBytes ? 1 : 0;
      if (rp.stage) rank_smem = staged;
      e = launch_k(rank_kernel, dim3(nq), kRankThreads, rank_smem, st, !ctx->prof_on, rp, meta);
    }
    if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "rank kernel: %s", cudaGetErrorString(e));
    ctx->launches += 4;
    return MUKV_OK;
  } catch (...) {
    return fail(ctx, MUKV_E_INVALID, "unexpected exception");
  }
}



mukv_status check_chunk_args(mukv_ctx* ctx, int n_frames, long long first_frame) {
  if (n_frames < 1) return fail(ctx, MUKV_E_INVALID, "n_frames must be >= 1");
  if (n_frames > ctx->cfg.max_frames_per_chunk)
    return fail(ctx, MUKV_E_CAPACITY, "n_frames %d exceeds max_frames_per_chunk %d", n_frames,
                ctx->cfg.max_frames_per_chunk);
  if (first_frame != ctx->frames)
    return fail(ctx, MUKV_E_STATE, "first_frame %lld does not continue the stream (%lld frames stored)", first_frame,
                ctx->frames);
  if (first_frame + n_frames > ctx->cfg.max_frames)
    return fail(ctx, MUKV_E_CAPACITY, "store full: %lld + %d frames > max_frames %lld", ctx->frames, n_frames,
                (long long)ctx->cfg.max_frames);
  return MUKV_OK;
}

}  // namespace

extern "C" {

size_t mukv_store_bytes(const mukv_config* cfg) {
  if (check_config(cfg)) return 0;
  return store_layout(*cfg).total;
}

size_t mukv_workspace_bytes(const mukv_config* cfg) {
  if (check_config(cfg)) return 0;
  return work_layout(*cfg).total;
}

mukv_status mukv_create(const mukv_config* cfg, void* d_store, size_t store_bytes, void* d_workspace,
                        size_t workspace_bytes, mukv_ctx** out) {
  return create_impl(cfg, d_store, store_bytes, d_workspace, workspace_bytes, 0, out);
}

// Host readers of the store (a view of a region, an export): segment entries still owed by the last
// compress call are pooled on that call's stream, and the stream is waited for.
static cudaError_t settle_store(const mukv_ctx* ctx) {
  if (!ctx->seg_pending) return cudaSuccess;
  const cudaStream_t st = ctx->seg_stream;
  cudaError_t e = flush_segments(ctx, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  return e;
}

mukv_status mukv_export_header(const mukv_ctx* ctx, mukv_store_header* out) {
  if (!ctx || !out) return MUKV_E_INVALID;
  if (settle_store(ctx) != cudaSuccess) return MUKV_E_CUDA;
  memset(out, 0, sizeof *out);
  out->magic = MUKV_STORE_MAGIC;
  out->version = MUKV_STORE_VERSION;
  out->cfg = ctx->cfg;
  out->frames = ctx->frames;
  out->store_bytes = ctx->sl.total;
  return MUKV_OK;
}

mukv_status mukv_import(const mukv_store_header* header, void* d_store, size_t store_bytes, void* d_workspace,
                        size_t workspace_bytes, mukv_ctx** out) {
  if (!out) return fail(nullptr, MUKV_E_INVALID, "out is null");
  *out = nullptr;
  if (!header) return fail(nullptr, MUKV_E_INVALID, "null header");
  if (header->magic != MUKV_STORE_MAGIC || header->version != MUKV_STORE_VERSION)
    return fail(nullptr, MUKV_E_INVALID, "not a store header of this library version");
  if (header->frames < 0 || header->frames > header->cfg.max_frames)
    return fail(nullptr, MUKV_E_INVALID, "header: frame count out of range");
  if (check_config(&header->cfg) == nullptr && header->store_bytes != store_layout(header->cfg).total)
    return fail(nullptr, MUKV_E_INVALID, "header: store size does not match its configuration");
  return create_impl(&header->cfg, d_store, store_bytes, d_workspace, workspace_bytes, header->frames, out);
}

}  // extern "C"

namespace {
mukv_status create_impl(const mukv_config* cfg, void* d_store, size_t store_bytes, void* d_workspace,
                        size_t workspace_bytes, long long frames0, mukv_ctx** out) {
  if (!out) return fail(nullptr, MUKV_E_INVALID, "out is null");
  *out = nullptr;
  if (!cfg || !d_store || !d_workspace) return fail(nullptr, MUKV_E_INVALID, "null argument");
  if (const char* why = check_config(cfg))
    return fail(nullptr, (cfg->dtype != MUKV_BF16 && cfg->dtype != MUKV_FP32) ? MUKV_E_DTYPE : MUKV_E_SHAPE, "%s", why);
  if (!aligned16(d_store) || !aligned16(d_workspace))
    return fail(nullptr, MUKV_E_ALIGN, "store and workspace must be 16-byte aligned");
  mukv_ctx* ctx = new (std::nothrow) mukv_ctx();
  if (!ctx) return fail(nullptr, MUKV_E_INVALID, "out of host memory");
  ctx->cfg = *cfg;
  ctx->sl = store_layout(*cfg);
  ctx->wl = work_layout(*cfg);
  if (store_bytes < ctx->sl.total || workspace_bytes < ctx->wl.total) {
    const size_t need_s = ctx->sl.total, need_w = ctx->wl.total;
    delete ctx;
    return fail(nullptr, MUKV_E_CAPACITY, "store needs %zu bytes (got %zu), workspace needs %zu bytes (got %zu)",
                need_s, store_bytes, need_w, workspace_bytes);
  }
  ctx->store = static_cast<unsigned char*>(d_store);
  ctx->ws = static_cast<unsigned char*>(d_workspace);
  ctx->frames = frames0;
  ctx->launches = 0;
  ctx->C = cfg->n_kv_heads * cfg->head_dim;
  ctx->G = cfg->n_q_heads / cfg->n_kv_heads;
  ctx->Ls = cfg->n_score_layers > 1 ? cfg->n_score_layers : 1;
  ctx->esize = cfg->dtype == MUKV_BF16 ? 2 : 4;
  ctx->key_rows = cfg->tokens_per_frame + cfg->past_frames * cfg->keep_per_frame;
  ctx->nc = pick_nc(ctx->key_rows);
  ctx->tcs = tc_shape(*cfg);
  ctx->n_sms = 1;
  ctx->flag_margin = kFlagMargin;
  ctx->flat_ratio = kFlatRatio;
  const int D = cfg->head_dim;
  cudaError_t e = raise_kernel_limits(&ctx->n_sms);
  if (e == cudaSuccess) {
    // the blocks of tail_kernel wait for one another: its grid must be resident as a whole
    int per_sm = 0;
    const bool bf = cfg->dtype == MUKV_BF16;
    const size_t dyn = bf ? score_smem_bytes<__nv_bfloat16, double>(ctx->key_rows, D)
                          : score_smem_bytes<float, double>(ctx->key_rows, D);
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bf ? tail_fn<__nv_bfloat16>(ctx->nc) : tail_fn<float>(ctx->nc),
                                                      kScoreThreads, dyn);
    if (e == cudaSuccess && per_sm < 1) e = cudaErrorInvalidConfiguration;
    ctx->tail_capacity = per_sm * ctx->n_sms;
  }
  if (e == cudaSuccess && ctx->tcs.ok) {
    const std::vector<uint16_t> w = dft_terms(D);
    e = cudaMemcpy(ctx->ws + ctx->wl.wtab, w.data(), w.size() * 2, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !encode_map2(&ctx->wmap, ctx->ws + ctx->wl.wtab, D, 3LL * D, D)) e = cudaErrorInvalidValue;
    if (e == cudaSuccess && cfg->past_frames > 0 &&
        !encode_map_pages(&ctx->pmap, ctx->store + ctx->sl.pages, D, cfg->n_kv_heads, cfg->keep_per_frame, 2 * cfg->n_layers,
                          cfg->max_frames, (long long)ctx->sl.page_bytes))
      e = cudaErrorInvalidValue;
  }
  if (e == cudaSuccess)
    e = cudaMemset(ctx->ws + ctx->wl.zero_begin, 0, ctx->wl.zero_end - ctx->wl.zero_begin);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    fail(nullptr, MUKV_E_CUDA, "mukv_create: %s", cudaGetErrorString(e));
    delete ctx;
    return MUKV_E_CUDA;
  }
  *out = ctx;
  return MUKV_OK;
}
}  // namespace

extern "C" {

void mukv_destroy(mukv_ctx* ctx) {
  if (!ctx) return;
  for (cudaEvent_t e : ctx->prof_ev) cudaEventDestroy(e);
  delete ctx;
}

mukv_status mukv_profile_enable(mukv_ctx* ctx, int32_t on) {
  if (!ctx) return MUKV_E_INVALID;
  ctx->prof_on = on != 0;
  ctx->prof_kind.clear();
  return MUKV_OK;
}

mukv_status mukv_profile_read(mukv_ctx* ctx, double* ms, int64_t* launches) {
  if (!ctx || !ms || !launches) return MUKV_E_INVALID;
  for (int i = 0; i < MUKV_PROF_KINDS; ++i) { ms[i] = 0.0; launches[i] = 0; }
  for (size_t i = 0; i < ctx->prof_kind.size(); ++i) {
    float t = 0.f;
    cudaError_t e = cudaEventSynchronize(ctx->prof_ev[2 * i + 1]);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&t, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]);
    if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "mukv_profile_read: %s", cudaGetErrorString(e));
    ms[ctx->prof_kind[i]] += (double)t;
    launches[ctx->prof_kind[i]] += 1;
  }
  ctx->prof_kind.clear();
  return MUKV_OK;
}

mukv_status mukv_reset(mukv_ctx* ctx, mukv_stream stream) {
  if (!ctx) return MUKV_E_INVALID;
  // arrival counters, flagged lists, selection flags, statistics and the event word start over
  cudaError_t e = cudaMemsetAsync(ctx->ws + ctx->wl.zero_begin, 0, ctx->wl.zero_end - ctx->wl.zero_begin,
                                  static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "mukv_reset: %s", cudaGetErrorString(e));
  ctx->frames = 0;
  ctx->parity = 0;
  ctx->failed = false;
  ctx->seg_pending = false;
  return MUKV_OK;
}

mukv_status mukv_set_option(mukv_ctx* ctx, int32_t option, double value) {
  if (!ctx) return MUKV_E_INVALID;
  switch (option) {
    case MUKV_OPT_FLAG_MARGIN:
      if (!(value >= (double)kFlagMargin) || !(value <= 4.0))
        return fail(ctx, MUKV_E_INVALID, "the safety margin can only be raised above %g (got %g)", (double)kFlagMargin, value);
      ctx->flag_margin = (float)value;
      return MUKV_OK;
    case MUKV_OPT_SCORE_PATH:
      if (value != 0.0 && value != 1.0) return fail(ctx, MUKV_E_INVALID, "score path must be 0 or 1");
      ctx->force_fma = value == 1.0;
      return MUKV_OK;
    default:
      return fail(ctx, MUKV_E_INVALID, "unknown option %d", option);
  }
}

mukv_status mukv_compress_chunk(mukv_ctx* ctx, const void* d_q, const void* d_k, const void* d_v, int32_t n_frames,
                                int64_t first_frame, int32_t* d_kept_out, float* d_scores_out,
                                mukv_stream stream) {
  if (!ctx) return MUKV_E_INVALID;
  try {
    if (ctx->failed) return fail(ctx, MUKV_E_STATE, "an earlier call broke off half way: call mukv_reset");
    if (!d_q || !d_k || !d_v) return fail(ctx, MUKV_E_INVALID, "null input pointer");
    if (!aligned16(d_q) || !aligned16(d_k) || !aligned16(d_v) || !aligned4(d_kept_out) || !aligned4(d_scores_out))
      return fail(ctx, MUKV_E_ALIGN, "d_q, d_k, d_v must be 16-byte aligned, the outputs 4-byte aligned");
    if (const mukv_status st = check_chunk_args(ctx, n_frames, first_frame)) return st;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->cfg.dtype == MUKV_BF16)
      return compress_impl<__nv_bfloat16>(ctx, d_q, nullptr, d_k, d_v, n_frames, first_frame, d_kept_out, d_scores_out, st);
    return compress_impl<float>(ctx, d_q, nullptr, d_k, d_v, n_frames, first_frame, d_kept_out, d_scores_out, st);
  } catch (...) {
    return fail(ctx, MUKV_E_INVALID, "unexpected exception");
  }
}

mukv_status mukv_compress_chunk_scored(mukv_ctx* ctx, const float* d_select_scores, const void* d_k, const void* d_v,
                                       int32_t n_frames, int64_t first_frame, int32_t* d_kept_out,
                                       mukv_stream stream) {
  if (!ctx) return MUKV_E_INVALID;
  try {
    if (ctx->failed) return fail(ctx, MUKV_E_STATE, "an earlier call broke off half way: call mukv_reset");
    if (!d_select_scores || !d_k || !d_v) return fail(ctx, MUKV_E_INVALID, "null input pointer");
    if (!aligned4(d_select_scores) || !aligned16(d_k) || !aligned16(d_v) || !aligned4(d_kept_out))
      return fail(ctx, MUKV_E_ALIGN, "d_k, d_v must be 16-byte aligned, scores and outputs 4-byte aligned");
    if (const mukv_status st = check_chunk_args(ctx, n_frames, first_frame)) return st;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->cfg.dtype == MUKV_BF16)
      return compress_impl<__nv_bfloat16>(ctx, nullptr, d_select_scores, d_k, d_v, n_frames, first_frame, d_kept_out,
                                          nullptr, st);
    return compress_impl<float>(ctx, nullptr, d_select_scores, d_k, d_v, n_frames, first_frame, d_kept_out, nullptr, st);
  } catch (...) {
    return fail(ctx, MUKV_E_INVALID, "unexpected exception");
  }
}

mukv_status mukv_retrieve(mukv_ctx* ctx, const void* d_qtok, const int32_t* h_q_offsets, const int64_t* h_t_limit,
                          int32_t nq, int32_t k_seg, int32_t k_frm, int32_t top_n, float lambda_frm, int32_t mode,
                          int32_t* d_seg_idx, int32_t* d_frm_idx, float* d_seg_score, float* d_frm_score,
                          int32_t* d_counts, mukv_stream stream) {
  if (!ctx) return MUKV_E_INVALID;
  mukv_retr_params rp;
  memset(&rp, 0, sizeof rp);
  rp.k_seg = k_seg; rp.k_frm = k_frm; rp.k_patch = 0;
  rp.lambda_frm = lambda_frm; rp.top_n = top_n; rp.mode = mode;
  return retrieve_impl(ctx, d_qtok, h_q_offsets, h_t_limit, nq, rp, d_seg_idx, d_frm_idx, nullptr, d_seg_score,
                       d_frm_score, nullptr, d_counts, 2, stream);
}

mukv_status mukv_retrieve3(mukv_ctx* ctx, const void* d_qtok, const int32_t* h_q_offsets, const int64_t* h_t_limit,
                           int32_t nq, const mukv_retr_params* params, int32_t* d_seg_idx, int32_t* d_frm_idx,
                           int32_t* d_patch_idx, float* d_seg_score, float* d_frm_score, float* d_patch_score,
                           int32_t* d_counts, mukv_stream stream) {
  if (!ctx) return MUKV_E_INVALID;
  if (!params) return fail(ctx, MUKV_E_INVALID, "null params");
  return retrieve_impl(ctx, d_qtok, h_q_offsets, h_t_limit, nq, *params, d_seg_idx, d_frm_idx, d_patch_idx, d_seg_score,
                       d_frm_score, d_patch_score, d_counts, 3, stream);
}

int64_t mukv_decode3_tokens(const mukv_ctx* ctx, int32_t k_seg, int32_t k_frm, int32_t k_patch) {
  if (!ctx || k_seg < 0 || k_frm < 0 || k_patch < 0) return 0;
  const mukv_config& c = ctx->cfg;
  long long pmax = 0;
  if (c.patch_split > 0) {
    const int rows = c.tokens_per_frame / c.grid_width;
    pmax = (long long)((rows + c.patch_split - 1) / c.patch_split) * ((c.grid_width + c.patch_split - 1) / c.patch_split);
    if (pmax > c.keep_per_frame) pmax = c.keep_per_frame;
  }
  long long per_frame = c.keep_per_frame;
  if (c.keep_per_segment > 0)                            // a frame may hold up to a whole segment's budget
    per_frame = c.keep_per_segment < c.tokens_per_frame ? c.keep_per_segment : c.tokens_per_frame;
  return (long long)k_seg + (long long)k_frm * per_frame + (long long)k_patch * pmax;
}

mukv_status mukv_gather3(mukv_ctx* ctx, const int32_t* d_seg_idx, const int32_t* d_frm_idx, const int32_t* d_patch_idx,
                         const int32_t* d_counts, int32_t nq, int32_t k_seg, int32_t k_frm, int32_t k_patch,
                         void* d_decode, int64_t decode_stride_bytes, int32_t* d_ntok, int32_t* d_tok_meta,
                         mukv_stream stream) {
  if (!ctx) return MUKV_E_INVALID;
  try {
    if (ctx->failed) return fail(ctx, MUKV_E_STATE, "an earlier call broke off half way: call mukv_reset");
    if (!d_seg_idx || !d_frm_idx || !d_counts || !d_decode || !d_ntok) return fail(ctx, MUKV_E_INVALID, "null argument");
    if (k_patch > 0 && !d_patch_idx) return fail(ctx, MUKV_E_INVALID, "d_patch_idx is null");
    if (!aligned4(d_seg_idx) || !aligned4(d_frm_idx) || !aligned4(d_patch_idx) || !aligned4(d_counts) ||
        !aligned16(d_decode) || !aligned4(d_ntok) || !aligned4(d_tok_meta))
      return fail(ctx, MUKV_E_ALIGN, "d_decode must be 16-byte aligned, index arrays 4-byte aligned");
    if (nq < 1 || k_seg < 1 || k_frm < 1 || k_patch < 0) return fail(ctx, MUKV_E_INVALID, "nq, k_seg, k_frm must be >= 1");
    if (nq > MUKV_MAX_QUESTIONS || k_seg > MUKV_MAX_TOPK || k_frm > MUKV_MAX_TOPK || k_patch > MUKV_MAX_TOPK)
      return fail(ctx, MUKV_E_CAPACITY, "nq or a k too large");
    const mukv_config& c = ctx->cfg;
    if (k_patch > 0 && c.patch_split == 0) return fail(ctx, MUKV_E_STATE, "the store has no patch level");
    const long long tok_cap = mukv_decode3_tokens(ctx, k_seg, k_frm, k_patch);
    const long long need = (long long)c.n_layers * 2 * tok_cap * ctx->C * ctx->esize;
    if (decode_stride_bytes < need)
      return fail(ctx, MUKV_E_CAPACITY, "decode_stride_bytes %lld < %lld needed per question",
                  (long long)decode_stride_bytes, need);
    if (decode_stride_bytes % 16 != 0) return fail(ctx, MUKV_E_ALIGN, "decode_stride_bytes must be a multiple of 16");
    if (ctx->seg_pending) {                                // the summary tokens are segment entries
      const cudaError_t ef = flush_segments(ctx, static_cast<cudaStream_t>(stream));
      if (ef != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "segment kernel: %s", cudaGetErrorString(ef));
      ctx->launches += 1;
    }
    Gather3Params gp;
    memset(&gp, 0, sizeof gp);
    gp.nq = nq; gp.k_seg = k_seg; gp.k_frm = k_frm; gp.k_pat = k_patch; gp.L = c.n_layers; gp.kappa = c.keep_per_frame;
    gp.C = ctx->C; gp.P = c.tokens_per_frame; gp.S = c.patch_split * c.patch_split; gp.grid_width = c.grid_width;
    gp.patch_split = c.patch_split; gp.tok_cap = (int)tok_cap; gp.esize = ctx->esize;
    gp.seg_idx = d_seg_idx; gp.frm_idx = d_frm_idx; gp.pat_idx = d_patch_idx; gp.counts = d_counts;
    gp.store = ctx->store;
    gp.page_table = reinterpret_cast<const long long*>(ctx->store + ctx->sl.page_table);
    gp.kept_store = reinterpret_cast<const int*>(ctx->store + ctx->sl.kept);
    gp.seg_entry = reinterpret_cast<const float*>(ctx->store + ctx->sl.seg_entry);
    gp.patch_cnt = reinterpret_cast<const int*>(ctx->store + ctx->sl.patch_cnt);
    gp.kept_count = c.keep_per_segment > 0 ? reinterpret_cast<const int*>(ctx->store + ctx->sl.kept_count) : nullptr;
    gp.kept_stride = (int)ctx->sl.kept_stride;
    gp.decode = static_cast<unsigned char*>(d_decode);
    gp.decode_stride = decode_stride_bytes;
    gp.ntok = d_ntok; gp.tok_meta = d_tok_meta;
    const long long units = (long long)nq * c.n_layers * 2 * (k_frm + 1);
    const unsigned blocks = (unsigned)(units < 148 * 8 ? units : 148 * 8);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
      ProfScope ps(ctx, 7, st);
      if (c.dtype == MUKV_BF16) gather3_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(gp);
      else gather3_kernel<float><<<blocks, 256, 0, st>>>(gp);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "gather3 kernel: %s", cudaGetErrorString(e));
    ctx->launches += 1;
    return MUKV_OK;
  } catch (...) {
    return fail(ctx, MUKV_E_INVALID, "unexpected exception");
  }
}

mukv_status mukv_gather(mukv_ctx* ctx, const int32_t* d_frm_idx, const int32_t* d_counts, int32_t nq, int32_t k_frm,
                        void* d_decode, int64_t decode_stride_bytes, int32_t* d_tok_meta, mukv_stream stream) {
  if (!ctx) return MUKV_E_INVALID;
  try {
    if (ctx->failed) return fail(ctx, MUKV_E_STATE, "an earlier call broke off half way: call mukv_reset");
    if (!d_frm_idx || !d_counts || !d_decode) return fail(ctx, MUKV_E_INVALID, "null argument");
    if (!aligned4(d_frm_idx) || !aligned4(d_counts) || !aligned16(d_decode) || !aligned4(d_tok_meta))
      return fail(ctx, MUKV_E_ALIGN, "d_decode must be 16-byte aligned, index arrays 4-byte aligned");
    if (ctx->cfg.keep_per_segment > 0)
      return fail(ctx, MUKV_E_UNSUPPORTED, "pages have different lengths (segment-level selection): use mukv_gather3");
    if (nq < 1 || k_frm < 1) return fail(ctx, MUKV_E_INVALID, "nq and k_frm must be >= 1");
    if (nq > MUKV_MAX_QUESTIONS || k_frm > MUKV_MAX_TOPK)
      return fail(ctx, MUKV_E_CAPACITY, "nq or k_frm too large");
    const mukv_config& c = ctx->cfg;
    const long long run = (long long)c.keep_per_frame * ctx->C * ctx->esize;
    const long long need = (long long)c.n_layers * 2 * k_frm * run;
    if (decode_stride_bytes < need)
      return fail(ctx, MUKV_E_CAPACITY, "decode_stride_bytes %lld < %lld needed per question",
                  (long long)decode_stride_bytes, need);
    if (decode_stride_bytes % 16 != 0) return fail(ctx, MUKV_E_ALIGN, "decode_stride_bytes must be a multiple of 16");
    GatherParams gp;
    gp.nq = nq; gp.k_frm = k_frm; gp.L = c.n_layers; gp.kappa = c.keep_per_frame;
    gp.run_bytes = run;
    gp.frm_idx = d_frm_idx; gp.counts = d_counts;
    gp.store = ctx->store;
    gp.page_table = reinterpret_cast<const long long*>(ctx->store + ctx->sl.page_table);
    gp.kept_store = reinterpret_cast<const int*>(ctx->store + ctx->sl.kept);
    gp.decode = static_cast<unsigned char*>(d_decode);
    gp.decode_stride = decode_stride_bytes;
    gp.tok_meta = d_tok_meta;
    const long long units = (long long)nq * c.n_layers * 2 * k_frm;
    const unsigned blocks = (unsigned)(units < 148 * 8 ? units : 148 * 8);
    {
      ProfScope ps(ctx, 7, static_cast<cudaStream_t>(stream));
      gather_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(gp);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "gather kernel: %s", cudaGetErrorString(e));
    ctx->launches += 1;
    return MUKV_OK;
  } catch (...) {
    return fail(ctx, MUKV_E_INVALID, "unexpected exception");
  }
}

void* mukv_store_region(const mukv_ctx* ctx, int32_t which, size_t* bytes) {
  if (!ctx) return nullptr;
  if (settle_store(ctx) != cudaSuccess) return nullptr;
  const mukv_config& c = ctx->cfg;
  const StoreLayout& s = ctx->sl;
  const size_t T = (size_t)c.max_frames, C = (size_t)ctx->C;
  size_t off = 0, sz = 0;
  switch (which) {
    case 0: off = s.pages; sz = s.pages_bytes; break;
    case 1: off = s.kept; sz = T * s.kept_stride * sizeof(int); break;
    case 10: if (c.keep_per_segment <= 0) return nullptr; off = s.kept_count; sz = T * sizeof(int); break;
    case 2: off = s.frame_entry; sz = T * c.n_layers * 2 * C * sizeof(float); break;
    case 3: off = s.seg_entry; sz = (size_t)s.max_segs * c.n_layers * 2 * C * sizeof(float); break;
    case 4: off = s.frame_key; sz = T * C * sizeof(float); break;
    case 5: off = s.seg_key; sz = (size_t)s.max_segs * C * sizeof(float); break;
    case 6: off = s.frame_ts; sz = T * sizeof(long long); break;
    case 7: off = s.page_table; sz = T * sizeof(long long); break;
    case 8: off = s.patch_key; sz = T * c.patch_split * c.patch_split * C * sizeof(float); break;
    case 9: off = s.patch_cnt; sz = T * c.patch_split * c.patch_split * sizeof(int); break;
    default: return nullptr;
  }
  if (bytes) *bytes = sz;
  return ctx->store + off;
}

mukv_status mukv_get_stats(mukv_ctx* ctx, mukv_stats* out, mukv_stream stream) {
  if (!ctx || !out) return MUKV_E_INVALID;
  memset(out, 0, sizeof *out);
  long long refined = 0;
  int dev_status = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(&refined, ctx->ws + ctx->wl.stat_refined, sizeof refined, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(&dev_status, ctx->ws + ctx->wl.dev_status, sizeof dev_status, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(ctx, MUKV_E_CUDA, "mukv_get_stats: %s", cudaGetErrorString(e));
  const mukv_config& c = ctx->cfg;
  out->frames = ctx->frames;
  out->segments = (ctx->frames + c.frames_per_segment - 1) / c.frames_per_segment;
  out->kept_tokens = ctx->frames * c.keep_per_frame;
  out->page_bytes = (long long)ctx->sl.page_bytes;
  out->store_bytes_used = ctx->frames * (long long)ctx->sl.page_bytes;
  if (c.keep_per_segment > 0) {
    const long long fs = c.frames_per_segment, full = ctx->frames / fs, rest = ctx->frames % fs;
    out->kept_tokens = full * c.keep_per_segment + (long long)c.keep_per_segment * rest / fs;
    out->page_bytes = 0;                                 // pages have different lengths
    out->store_bytes_used = out->kept_tokens * c.n_layers * 2 * ctx->C * ctx->esize;
  }
  out->refined_frames = refined;
  out->kernel_launches = ctx->launches;
  out->device_status = dev_status;
  return MUKV_OK;
}

const char* mukv_last_error(const mukv_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

}  // extern "C"

// =====================================================================================
// Scoring without a workspace.
//
// Everything above works in memory the caller hands over (store, workspace).  Some callers
// cannot produce such a buffer: a plug-in that runs inside a serving process whose start-up
// code has already given the whole device to its KV-cache pool, or a control loop that is
// forbidden to touch the allocator once it is running (cudaMalloc may fail there, and it
// synchronises the device when it does not).  For them the scratch of the scoring kernel lives
// in the array below, which is part of the loaded library image on every device.
// =====================================================================================
namespace {

constexpr int kNaFrames = MUKV_NOALLOC_MAX_FRAMES, kNaHq = MUKV_NOALLOC_MAX_Q_HEADS;
constexpr int kNaHkv = MUKV_NOALLOC_MAX_KV_HEADS, kNaP = MUKV_MAX_TOKENS;
constexpr size_t kNaColF = 0;
constexpr size_t kNaFftF = kNaColF + (size_t)kNaFrames * kNaHq * kNaP * sizeof(float);
constexpr size_t kNaColD = kNaFftF + (size_t)kNaFrames * kNaHkv * kNaP * sizeof(float);
constexpr size_t kNaFftD = kNaColD + (size_t)kNaFrames * kNaHq * kNaP * sizeof(double);
constexpr size_t kNaKept = kNaFftD + (size_t)kNaFrames * kNaHkv * kNaP * sizeof(double);
constexpr size_t kNaTs = kNaKept + (size_t)kNaFrames * kNaP * sizeof(int);
constexpr size_t kNaPt = kNaTs + 256;
constexpr size_t kNaCtrl = kNaPt + 256;                  // frame_counter[16], flagged[16], n_flagged
constexpr size_t kNaCtrlBytes = 256;
constexpr size_t kNaTotal = kNaCtrl + kNaCtrlBytes;

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaTotal];

unsigned char* g_noalloc_ptr[kMaxDevices];               // device address of the array, per device

// Once per device, with that device current: resolves the array's device address and makes sure the
// scoring kernels may use the shared memory the largest supported frame needs.  Allocates nothing.
cudaError_t noalloc_setup(int dev, unsigned char** out) {
  cudaError_t e = raise_kernel_limits(nullptr);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(g_dev_mutex);
  if (!g_noalloc_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[dev] = static_cast<unsigned char*>(ptr);
  }
  *out = g_noalloc_ptr[dev];
  return cudaSuccess;
}

template <typename T>
mukv_status noalloc_impl(const mukv_config& c, const void* d_q, const void* d_k_last, int n, int* d_kept_out,
                         float* d_scores_out, cudaStream_t st) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(nullptr, MUKV_E_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(nullptr, MUKV_E_CAPACITY, "device index %d not supported", dev);
  const int P = c.tokens_per_frame, D = c.head_dim, nc = pick_nc(P);
  unsigned char* base = nullptr;
  e = noalloc_setup(dev, &base);
  if (e != cudaSuccess) return fail(nullptr, MUKV_E_CUDA, "set-up of the static scratch: %s", cudaGetErrorString(e));
  // the array keeps what the last call left: the arrival counters and the flagged list start at zero
  e = cudaMemsetAsync(base + kNaCtrl, 0, kNaCtrlBytes, st);
  if (e != cudaSuccess) return fail(nullptr, MUKV_E_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
  ScoreParams sp;
  memset(&sp, 0, sizeof sp);
  sp.P = P; sp.Hq = c.n_q_heads; sp.Hkv = c.n_kv_heads; sp.D = D; sp.G = c.n_q_heads / c.n_kv_heads;
  sp.kappa = c.keep_per_frame; sp.n_frames = n; sp.causal = c.attn_causal; sp.keep_low = c.keep_low_freq;
  sp.alpha = c.alpha; sp.tie_eps = c.tie_eps; sp.flag_margin = kFlagMargin; sp.flat_ratio = kFlatRatio;
  sp.Ls = 1;                                             // one scoring layer: the one the caller passes
  sp.first_frame = 0;
  sp.q = d_q;
  sp.k_last = d_k_last;
  sp.colsum_part = base + kNaColF;
  sp.ifft_part = base + kNaFftF;
  sp.frame_counter = reinterpret_cast<int*>(base + kNaCtrl);
  sp.flagged = reinterpret_cast<int*>(base + kNaCtrl) + kNaFrames;
  sp.n_flagged = reinterpret_cast<int*>(base + kNaCtrl) + 2 * kNaFrames;
  sp.kept_store = d_kept_out ? d_kept_out : reinterpret_cast<int*>(base + kNaKept);
  sp.kept_out = nullptr;
  sp.scores_out = d_scores_out;
  sp.frame_ts = reinterpret_cast<long long*>(base + kNaTs);
  sp.page_table = reinterpret_cast<long long*>(base + kNaPt);
  sp.refine = 0;
  sp.row_split = 1;
  const dim3 grid(c.n_q_heads, n);
  e = launch_score<T, float>(sp, nc, grid, score_smem_bytes<T, float>(P, D), st);
  if (e != cudaSuccess) return fail(nullptr, MUKV_E_CUDA, "score kernel: %s", cudaGetErrorString(e));
  sp.refine = 1;
  sp.colsum_part = base + kNaColD;
  sp.ifft_part = base + kNaFftD;
  e = launch_score<T, double>(sp, nc, grid, score_smem_bytes<T, double>(P, D), st);
  if (e != cudaSuccess) return fail(nullptr, MUKV_E_CUDA, "refine kernel: %s", cudaGetErrorString(e));
  return MUKV_OK;
}

}  // namespace

extern "C" mukv_status mukv_score_frames_noalloc(const mukv_config* cfg, const void* d_q, const void* d_k_last,
                                                 int32_t n_frames, int32_t* d_kept_out, float* d_scores_out,
                                                 mukv_stream stream) {
  try {
    if (!cfg || !d_q || !d_k_last) return fail(nullptr, MUKV_E_INVALID, "null argument");
    if (!d_kept_out && !d_scores_out) return fail(nullptr, MUKV_E_INVALID, "no output requested");
    mukv_config c = *cfg;
    c.max_frames = 1;                                            // fields this entry point ignores
    c.max_frames_per_chunk = 1;
    c.n_layers = 1;
    c.frames_per_segment = 1;
    c.n_score_layers = 0;
    c.score_layer_offset = 0;
    c.patch_split = 0;
    c.keep_per_segment = 0;
    c.past_frames = 0;
    c.reserved = 0;
    if (const char* why = check_config(&c))
      return fail(nullptr, (c.dtype != MUKV_BF16 && c.dtype != MUKV_FP32) ? MUKV_E_DTYPE : MUKV_E_SHAPE, "%s", why);
    if (n_frames < 1) return fail(nullptr, MUKV_E_INVALID, "n_frames must be >= 1");
    if (n_frames > kNaFrames || c.n_q_heads > kNaHq || c.n_kv_heads > kNaHkv)
      return fail(nullptr, MUKV_E_CAPACITY,
                  "the static scratch holds at most %d frames, %d query heads and %d key heads per call "
                  "(got %d, %d, %d)", kNaFrames, kNaHq, kNaHkv, n_frames, c.n_q_heads, c.n_kv_heads);
    if (!aligned16(d_q) || !aligned16(d_k_last) || !aligned4(d_kept_out) || !aligned4(d_scores_out))
      return fail(nullptr, MUKV_E_ALIGN, "d_q, d_k_last must be 16-byte aligned, the outputs 4-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (c.dtype == MUKV_BF16)
      return noalloc_impl<__nv_bfloat16>(c, d_q, d_k_last, n_frames, d_kept_out, d_scores_out, st);
    return noalloc_impl<float>(c, d_q, d_k_last, n_frames, d_kept_out, d_scores_out, st);
  } catch (...) {
    return fail(nullptr, MUKV_E_INVALID, "unexpected exception");
  }
}
