// C ABI of the rolling-KV chunk-attention library: host-side cache metadata, argument checks,
// tensor-map construction and kernel launches.  Declarations and semantics: include/astro.h.
#include "astro.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstring>
#include <mutex>
#include <new>

#include "attn_bwd.cuh"
#include "attn_fwd.cuh"
#include "attn_fwd_pair.cuh"
#include "kv_ring.cuh"
#include "nft_loss.cuh"

using namespace astro;

struct astro_kvcache {
  astro_kvcache_desc_t d;
  void* k;
  void* v;
  int sink_held;   // frames in sink slots [0, S)
  int win_head;    // ring index (0..L-1) of the oldest window frame
  int win_held;    // frames in the window ring, slots S + (head + i) % L
  int64_t frames_seen;
  // Tensor maps of the storage: built once (by create when a driver is present, else by the first attention
  // call) under a once-flag, read-only afterwards, so attention calls from several threads may share a handle.
  mutable std::once_flag maps_once;
  mutable astro_status_t maps_status;
  mutable CUtensorMap tm_k, tm_v;
};

namespace astro {
// Self-test of the bounded wait: one warp waits on an mbarrier that nothing will ever complete.  The wait
// gives up after `cycle_limit` clocks, records the time-out in the device status word and the kernel ends
// normally, which is exactly the path a broken hand-off in the attention kernels would take.
__global__ void wait_timeout_selftest_kernel(long long cycle_limit) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  mbar_wait_spin(&bar, 0, &abort_flag, cycle_limit);
}
}  // namespace astro

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool desc_ok(const astro_kvcache_desc_t* d) {
  return d && d->cache_batch >= 1 && d->heads >= 1 && (d->head_dim == 64 || d->head_dim == 128) &&
         d->tokens_per_frame >= 1 && d->sink_frames >= 0 && d->window_frames >= 1;
}

// ---- device / driver helpers -------------------------------------------------------------------
// Per-device facts are cached in atomics: several host threads may make their first call at the same time,
// and all of them would store the same value.
constexpr int kMaxDevices = 64;

astro_status_t check_arch() {
  static std::atomic<int> ok_device[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ASTRO_ERR_CUDA;
  if (dev >= 0 && dev < kMaxDevices && ok_device[dev].load(std::memory_order_acquire)) return ASTRO_OK;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ASTRO_ERR_CUDA;
  if (major != 10) return ASTRO_ERR_ARCH;
  if (dev >= 0 && dev < kMaxDevices) ok_device[dev].store(1, std::memory_order_release);
  return ASTRO_OK;
}

// Number of SMs of the current device (0 if it cannot be read).
int sm_count() {
  static std::atomic<int> count[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (dev >= 0 && dev < kMaxDevices) {
    const int c = count[dev].load(std::memory_order_acquire);
    if (c > 0) return c;
  }
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (dev >= 0 && dev < kMaxDevices) count[dev].store(n, std::memory_order_release);
  return n;
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_fn() {
  static encode_tiled_fn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<encode_tiled_fn>(p);
  });
  return fn;
}

// bf16 tensor seen as {d, token, head, batch} with byte strides; box = 64 columns x 128 tokens, 128-byte
// swizzle, zero fill outside the tensor.
astro_status_t make_tmap(CUtensorMap* out, const void* base, int head_dim, long long n_tok, int heads, int batch,
                         unsigned long long stride_tok, unsigned long long stride_head,
                         unsigned long long stride_batch, int box_rows = kTile) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return ASTRO_ERR_CUDA;
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(head_dim), static_cast<cuuint64_t>(n_tok),
                        static_cast<cuuint64_t>(heads), static_cast<cuuint64_t>(batch)};
  cuuint64_t strides[3] = {stride_tok, stride_head, stride_batch};
  cuuint32_t box[4] = {64, static_cast<cuuint32_t>(box_rows), 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ASTRO_OK : ASTRO_ERR_CUDA;
}

// Caller tensor [batch, n_tok, H, D].
astro_status_t make_tmap_user(CUtensorMap* out, const void* base, int head_dim, int n_tok, int heads, int batch,
                              int box_rows = kTile) {
  const unsigned long long row = static_cast<unsigned long long>(head_dim) * 2;
  return make_tmap(out, base, head_dim, n_tok, heads, batch, row * heads, row, row * heads * n_tok, box_rows);
}

// Cache storage seen up to token `end_tok` only (rows from there on read as zeros), box of `box_rows` tokens.
astro_status_t make_tmap_cache_range(CUtensorMap* out, const astro_kvcache* c, const void* base, long long end_tok,
                                     int box_rows) {
  const auto& d = c->d;
  const long long tok = static_cast<long long>(d.sink_frames + d.window_frames) * d.tokens_per_frame;
  const unsigned long long row = static_cast<unsigned long long>(d.head_dim) * 2;
  return make_tmap(out, base, d.head_dim, end_tok, d.heads, d.cache_batch, row, row * tok, row * tok * d.heads,
                   box_rows);
}

astro_status_t build_cache_maps(const astro_kvcache* c) {
  const auto& d = c->d;
  const long long tok = static_cast<long long>(d.sink_frames + d.window_frames) * d.tokens_per_frame;
  const unsigned long long row = static_cast<unsigned long long>(d.head_dim) * 2;
  astro_status_t s = make_tmap(&c->tm_k, c->k, d.head_dim, tok, d.heads, d.cache_batch, row, row * tok,
                               row * tok * d.heads);
  if (s != ASTRO_OK) return s;
  s = make_tmap(&c->tm_v, c->v, d.head_dim, tok, d.heads, d.cache_batch, row, row * tok, row * tok * d.heads);
  return s;
}

astro_status_t cache_maps(const astro_kvcache* c) {
  std::call_once(c->maps_once, [c] { c->maps_status = build_cache_maps(c); });
  return c->maps_status;
}

// Physical token ranges of the held frames, merged where adjacent, followed by the chunk's keys.
KeySegs build_segments(const astro_kvcache* c, int n_kc) {
  KeySegs s;
  std::memset(&s, 0, sizeof(s));
  auto push = [&s](long long start, long long count, int from_chunk) {
    if (count <= 0) return;
    if (s.n > 0 && !from_chunk && !s.from_chunk[s.n - 1] && s.start[s.n - 1] + s.count[s.n - 1] == start) {
      s.count[s.n - 1] += static_cast<int>(count);
      return;
    }
    s.start[s.n] = static_cast<int>(start);
    s.count[s.n] = static_cast<int>(count);
    s.from_chunk[s.n] = from_chunk;
    ++s.n;
  };
  if (c) {
    const int T = c->d.tokens_per_frame, S = c->d.sink_frames, L = c->d.window_frames;
    const int first = c->win_held < L - c->win_head ? c->win_held : L - c->win_head;  // frames before the wrap
    const int wrapped = c->win_held - first;
    push(0, static_cast<long long>(c->sink_held) * T, 0);
    push(static_cast<long long>(S) * T, static_cast<long long>(wrapped) * T, 0);
    push(static_cast<long long>(S + c->win_head) * T, static_cast<long long>(first) * T, 0);
  }
  push(0, n_kc, 1);
  return s;
}

template <typename K> astro_status_t set_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess
             ? ASTRO_OK
             : ASTRO_ERR_CUDA;
}

template <typename K> astro_status_t set_smem_once(K kernel, int bytes, std::atomic<int> (&done)[kMaxDevices]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ASTRO_ERR_CUDA;
  if (dev >= 0 && dev < kMaxDevices && done[dev].load(std::memory_order_acquire)) return ASTRO_OK;
  astro_status_t s = set_smem(kernel, bytes);   // idempotent: a second thread repeating it does no harm
  if (s == ASTRO_OK && dev >= 0 && dev < kMaxDevices) done[dev].store(1, std::memory_order_release);
  return s;
}

astro_status_t launch_status() { return cudaGetLastError() == cudaSuccess ? ASTRO_OK : ASTRO_ERR_CUDA; }

struct AttnArgs {
  const astro_kvcache* cache;
  int batch, heads, head_dim, n_q, n_kc;
};

astro_status_t check_attn_args(const AttnArgs& a, float scale) {
  if (a.batch < 1 || a.heads < 1 || a.n_q < 1 || a.n_kc < 0) return ASTRO_ERR_SHAPE;
  if (a.head_dim != 64 && a.head_dim != 128) return ASTRO_ERR_SHAPE;
  if (!(scale >= 0.f) || !(scale < 3.0e38f)) return ASTRO_ERR_SHAPE;
  if (a.batch > 65535 || a.heads > 65535) return ASTRO_ERR_SHAPE;
  int held = 0;
  if (a.cache) {
    const auto& d = a.cache->d;
    if (d.heads != a.heads || d.head_dim != a.head_dim) return ASTRO_ERR_SHAPE;
    if (d.cache_batch != a.batch && d.cache_batch != 1) return ASTRO_ERR_SHAPE;
    held = a.cache->sink_held + a.cache->win_held;
  }
  if (held == 0 && a.n_kc == 0) return ASTRO_ERR_SHAPE;  // no key at all: softmax undefined
  return ASTRO_OK;
}

// 0: fast pass with the safe pass as fallback (normal operation); 1: safe pass only; 2: CTA-pair kernel where the
// shape allows it (head_dim 128).  Diagnostics and tests.
std::atomic<int> g_fwd_mode{0};

// Set by the CTA-pair kernel when a row needs the running-reference pass; read back by astro_debug_pair_flag.
__device__ int g_pair_needs_safe = 0;

astro_status_t launch_fwd_pair(const AttnArgs& a, const astro_kvcache* cache, bool have_ctx, const void* q,
                               const void* k_chunk, const void* v_chunk, const KeySegs& segs, float scale, void* o,
                               float* lse, cudaStream_t st) {
  static std::atomic<int> done[kMaxDevices];
  astro_status_t s = set_smem_once(chunk_attn_fwd_pair_kernel, PairSmem::kTotal, done);
  if (s != ASTRO_OK) return s;
  PairMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  if (a.n_kc > 0) {
    if ((s = make_tmap_user(&maps.kc, k_chunk, 128, a.n_kc, a.heads, a.batch, 64)) != ASTRO_OK) return s;
    if ((s = make_tmap_user(&maps.vc, v_chunk, 128, a.n_kc, a.heads, a.batch)) != ASTRO_OK) return s;
  }
  if (have_ctx) {
    int ci = 0;
    for (int i = 0; i < segs.n; ++i) {
      if (segs.from_chunk[i]) continue;
      const long long end = static_cast<long long>(segs.start[i]) + segs.count[i];
      if ((s = make_tmap_cache_range(&maps.kx[ci], cache, cache->k, end, 64)) != ASTRO_OK) return s;
      if ((s = make_tmap_cache_range(&maps.vx[ci], cache, cache->v, end, kTile)) != ASTRO_OK) return s;
      ++ci;
    }
  }
  int* flag = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&flag), g_pair_needs_safe) != cudaSuccess) return ASTRO_ERR_CUDA;
  const int shared = (cache && cache->d.cache_batch == 1 && a.batch > 1) ? 1 : 0;
  const int tiles = (a.n_q + kTile - 1) / kTile;
  dim3 grid((tiles + 1) / 2 * 2, shared ? a.batch : a.heads, shared ? a.heads : a.batch);
  chunk_attn_fwd_pair_kernel<<<grid, kPairThreads, PairSmem::kTotal, st>>>(
      static_cast<const __nv_bfloat16*>(q), maps, segs, a.n_q, a.heads, shared, scale * kLog2e,
      static_cast<__nv_bfloat16*>(o), lse, flag);
  return launch_status();
}

template <int D>
astro_status_t launch_fwd(const AttnArgs& a, const __nv_bfloat16* q, const CUtensorMap& tkc, const CUtensorMap& tvc,
                          const CUtensorMap& tkx, const CUtensorMap (&tvx)[2], const KeySegs& segs, float scale,
                          void* o, float* lse, cudaStream_t st) {
  static std::atomic<int> done[kMaxDevices];
  astro_status_t s = set_smem_once(chunk_attn_fwd_kernel<D>, FwdSmem<D>::kTotal, done);
  if (s != ASTRO_OK) return s;
  const int shared = (a.cache && a.cache->d.cache_batch == 1 && a.batch > 1) ? 1 : 0;
  // One CTA per SM, each walking over its share of the (query tile, head, sample) units; more CTAs only when a
  // CTA would get more units than it has redo bits for.
  const long long units = static_cast<long long>((a.n_q + kTile - 1) / kTile) * a.heads * a.batch;
  const int sms = sm_count();
  if (sms <= 0) return ASTRO_ERR_CUDA;
  if (units > 0x7fffffffLL) return ASTRO_ERR_SHAPE;
  long long ctas = units < sms ? units : sms;
  if (units > ctas * kFwdMaxUnits) ctas = sms * ((units + static_cast<long long>(sms) * kFwdMaxUnits - 1) / (static_cast<long long>(sms) * kFwdMaxUnits));
  chunk_attn_fwd_kernel<D><<<static_cast<unsigned>(ctas), kFwdThreads, FwdSmem<D>::kTotal, st>>>(
      q, tkc, tvc, tkx, tvx[0], tvx[1], segs, a.batch, a.n_q, a.heads, shared,
      scale * kLog2e, g_fwd_mode.load(std::memory_order_relaxed) == 1 ? 1 : 0, static_cast<__nv_bfloat16*>(o), lse);
  return launch_status();
}

template <int D>
astro_status_t launch_bwd_delta(const void* o, const void* d_o, int batch, int heads, int n_q, float* delta,
                                cudaStream_t st) {
  const long long rows = static_cast<long long>(batch) * n_q * heads;
  const unsigned blocks = static_cast<unsigned>((rows * 32 + 255) / 256);
  bwd_delta_kernel<D><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(o),
                                             static_cast<const __nv_bfloat16*>(d_o), delta, batch, n_q, heads);
  return launch_status();
}

template <int D>
astro_status_t launch_bwd_dq(const AttnArgs& a, const __nv_bfloat16* q, const CUtensorMap& tdo, const CUtensorMap& tkc,
                             const CUtensorMap& tvc, const CUtensorMap (&tkx)[2], const CUtensorMap& tvx,
                             const KeySegs& segs, float scale, const float* lse, const float* delta, void* dq,
                             cudaStream_t st) {
  static std::atomic<int> done[kMaxDevices];
  astro_status_t s = set_smem_once(chunk_attn_bwd_dq_kernel<D>, DqSmem<D>::kTotal, done);
  if (s != ASTRO_OK) return s;
  const int shared = (a.cache && a.cache->d.cache_batch == 1 && a.batch > 1) ? 1 : 0;
  dim3 grid_q((a.n_q + kTile - 1) / kTile, shared ? a.batch : a.heads, shared ? a.heads : a.batch);
  chunk_attn_bwd_dq_kernel<D><<<grid_q, kDqThreads, DqSmem<D>::kTotal, st>>>(
      q, tdo, tkc, tvc, tkx[0], tkx[1], tvx, segs, a.n_q, a.heads, shared, scale, lse, delta,
      static_cast<__nv_bfloat16*>(dq));
  return launch_status();
}

template <int D>
astro_status_t launch_bwd_dkv(const AttnArgs& a, const CUtensorMap& tq, const CUtensorMap& tdo,
                              const CUtensorMap& tkc, const CUtensorMap& tvc, float scale, const float* lse,
                              const float* delta, void* dk, void* dv, cudaStream_t st) {
  static std::atomic<int> done[kMaxDevices];
  astro_status_t s = set_smem_once(chunk_attn_bwd_dkv_kernel<D>, DkvSmem<D>::kTotal, done);
  if (s != ASTRO_OK) return s;
  dim3 grid_k((a.n_kc + kTile - 1) / kTile, a.heads, a.batch);
  chunk_attn_bwd_dkv_kernel<D><<<grid_k, kDkvThreads, DkvSmem<D>::kTotal, st>>>(
      tq, tdo, tkc, tvc, a.n_q, a.n_kc, a.heads, scale, lse, delta, static_cast<__nv_bfloat16*>(dk),
      static_cast<__nv_bfloat16*>(dv));
  return launch_status();
}

// Copies frames between a caller tensor and the storage slots listed in `slots` (logical order).
template <bool ToCache>
astro_status_t launch_ring_copy(const astro_kvcache* c, void* k_user, void* v_user, const int* slots, int n_frames,
                                cudaStream_t st) {
  const auto& d = c->d;
  const int vpr = d.head_dim * 2 / 16;
  const int row_vecs = d.heads * vpr;
  const int threads = row_vecs >= 256 ? 256 : ((row_vecs + 31) / 32) * 32;
  const int chunks_per_frame = (d.tokens_per_frame + kRingTokensPerThread - 1) / kRingTokensPerThread;
  if (d.cache_batch > 32767 || static_cast<long long>(chunks_per_frame) * kMaxFramesPerCopy > 65535)
    return ASTRO_ERR_SHAPE;
  for (int f0 = 0; f0 < n_frames; f0 += kMaxFramesPerCopy) {
    SlotMap map;
    map.n = n_frames - f0 < kMaxFramesPerCopy ? n_frames - f0 : kMaxFramesPerCopy;
    for (int j = 0; j < map.n; ++j) map.slot[j] = slots[f0 + j];
    dim3 grid((row_vecs + threads - 1) / threads, map.n * chunks_per_frame, 2 * d.cache_batch);
    ring_copy_kernel<ToCache><<<grid, threads, 0, st>>>(
        static_cast<uint4*>(k_user), static_cast<uint4*>(v_user), static_cast<uint4*>(c->k),
        static_cast<uint4*>(c->v), map, d.heads, d.tokens_per_frame, vpr, d.sink_frames + d.window_frames, f0,
        n_frames, chunks_per_frame);
  }
  return launch_status();
}

}  // namespace

extern "C" {

size_t astro_kvcache_storage_bytes(const astro_kvcache_desc_t* d) {
  if (!desc_ok(d)) return 0;
  return static_cast<size_t>(d->cache_batch) * d->heads * (d->sink_frames + d->window_frames) *
         d->tokens_per_frame * d->head_dim * 2;
}

astro_status_t astro_kvcache_create(const astro_kvcache_desc_t* desc, void* k_storage, void* v_storage,
                                    size_t bytes_each, astro_kvcache_t** out) {
  if (!desc || !k_storage || !v_storage || !out) return ASTRO_ERR_NULL;
  if (!desc_ok(desc)) return ASTRO_ERR_SHAPE;
  if (!aligned16(k_storage) || !aligned16(v_storage)) return ASTRO_ERR_ALIGN;
  if (bytes_each < astro_kvcache_storage_bytes(desc)) return ASTRO_ERR_CAPACITY;
  const long long tok = static_cast<long long>(desc->sink_frames + desc->window_frames) * desc->tokens_per_frame;
  if (tok >= (1ll << 31) - kTile) return ASTRO_ERR_SHAPE;
  astro_kvcache* c = new (std::nothrow) astro_kvcache();
  if (!c) return ASTRO_ERR_CUDA;
  c->d = *desc;
  c->k = k_storage;
  c->v = v_storage;
  c->sink_held = c->win_head = c->win_held = 0;
  c->frames_seen = 0;
  c->maps_status = ASTRO_ERR_CUDA;
  if (get_encode_fn() != nullptr) {   // a driver is present: build the maps now, so attention calls only read them
    const astro_status_t ms = cache_maps(c);
    if (ms != ASTRO_OK) { delete c; return ms; }
  }
  *out = c;
  return ASTRO_OK;
}

astro_status_t astro_kvcache_destroy(astro_kvcache_t* cache) {
  if (!cache) return ASTRO_ERR_NULL;
  delete cache;
  return ASTRO_OK;
}

astro_status_t astro_kvcache_reset(astro_kvcache_t* c) {
  if (!c) return ASTRO_ERR_NULL;
  c->sink_held = c->win_head = c->win_held = 0;
  c->frames_seen = 0;
  return ASTRO_OK;
}

astro_status_t astro_kvcache_append(astro_kvcache_t* c, const void* k, const void* v, int n_frames, void* stream) {
  if (!c || !k || !v) return ASTRO_ERR_NULL;
  if (n_frames < 0) return ASTRO_ERR_SHAPE;
  if (!aligned16(k) || !aligned16(v)) return ASTRO_ERR_ALIGN;
  const int S = c->d.sink_frames, L = c->d.window_frames;
  const int room = (S - c->sink_held) + (L - c->win_held);
  if (n_frames > room) return ASTRO_ERR_CAPACITY;
  if (n_frames == 0) return ASTRO_OK;
  astro_status_t s = check_arch();
  if (s != ASTRO_OK) return s;
  int* slots = new (std::nothrow) int[n_frames];
  if (!slots) return ASTRO_ERR_CUDA;
  int sink = c->sink_held, held = c->win_held;
  for (int j = 0; j < n_frames; ++j) {
    if (sink < S) slots[j] = sink++;
    else { slots[j] = S + (c->win_head + held) % L; ++held; }
  }
  s = launch_ring_copy<true>(c, const_cast<void*>(k), const_cast<void*>(v), slots, n_frames,
                             static_cast<cudaStream_t>(stream));
  delete[] slots;
  if (s != ASTRO_OK) return s;
  c->sink_held = sink;
  c->win_held = held;
  c->frames_seen += n_frames;
  return ASTRO_OK;
}

astro_status_t astro_kvcache_evict(astro_kvcache_t* c, int n_frames, void* /*stream*/) {
  if (!c) return ASTRO_ERR_NULL;
  if (n_frames < 0) return ASTRO_ERR_SHAPE;
  if (n_frames > c->win_held) return ASTRO_ERR_UNDERFLOW;
  c->win_head = (c->win_head + n_frames) % c->d.window_frames;
  c->win_held -= n_frames;
  if (c->win_held == 0) c->win_head = 0;
  return ASTRO_OK;
}

astro_status_t astro_kvcache_query(const astro_kvcache_t* c, int* sink_held, int* window_held, int64_t* frames_seen) {
  if (!c) return ASTRO_ERR_NULL;
  if (sink_held) *sink_held = c->sink_held;
  if (window_held) *window_held = c->win_held;
  if (frames_seen) *frames_seen = c->frames_seen;
  return ASTRO_OK;
}

astro_status_t astro_kvcache_get_state(const astro_kvcache_t* c, astro_kvcache_state_t* state) {
  if (!c || !state) return ASTRO_ERR_NULL;
  state->sink_held = c->sink_held;
  state->window_head = c->win_head;
  state->window_held = c->win_held;
  state->frames_seen = c->frames_seen;
  return ASTRO_OK;
}

astro_status_t astro_kvcache_set_state(astro_kvcache_t* c, const astro_kvcache_state_t* state) {
  if (!c || !state) return ASTRO_ERR_NULL;
  const int S = c->d.sink_frames, L = c->d.window_frames;
  if (state->sink_held < 0 || state->sink_held > S || state->window_held < 0 || state->window_held > L ||
      state->window_head < 0 || state->window_head >= L || state->frames_seen < state->sink_held + state->window_held)
    return ASTRO_ERR_SHAPE;
  if (state->window_held > 0 && state->sink_held != S) return ASTRO_ERR_SHAPE;  // the sink fills first
  c->sink_held = state->sink_held;
  c->win_head = state->window_held == 0 ? 0 : state->window_head;
  c->win_held = state->window_held;
  c->frames_seen = state->frames_seen;
  return ASTRO_OK;
}

astro_status_t astro_kvcache_key_segments(const astro_kvcache_t* c, int n_kc, int* n_segments, int* first_token,
                                          int* token_count, int* from_chunk) {
  if (!n_segments || !first_token || !token_count || !from_chunk) return ASTRO_ERR_NULL;
  if (n_kc < 0) return ASTRO_ERR_SHAPE;
  const bool have_ctx = c && (c->sink_held + c->win_held) > 0;
  const KeySegs s = build_segments(have_ctx ? c : nullptr, n_kc);
  *n_segments = s.n;
  for (int i = 0; i < s.n; ++i) {
    first_token[i] = s.start[i];
    token_count[i] = s.count[i];
    from_chunk[i] = s.from_chunk[i];
  }
  return ASTRO_OK;
}

astro_status_t astro_kvcache_export(const astro_kvcache_t* c, void* k_out, void* v_out, void* stream) {
  if (!c || !k_out || !v_out) return ASTRO_ERR_NULL;
  if (!aligned16(k_out) || !aligned16(v_out)) return ASTRO_ERR_ALIGN;
  const int n = c->sink_held + c->win_held;
  if (n == 0) return ASTRO_OK;
  astro_status_t s = check_arch();
  if (s != ASTRO_OK) return s;
  int* slots = new (std::nothrow) int[n];
  if (!slots) return ASTRO_ERR_CUDA;
  for (int j = 0; j < c->sink_held; ++j) slots[j] = j;
  for (int j = 0; j < c->win_held; ++j)
    slots[c->sink_held + j] = c->d.sink_frames + (c->win_head + j) % c->d.window_frames;
  s = launch_ring_copy<false>(c, k_out, v_out, slots, n, static_cast<cudaStream_t>(stream));
  delete[] slots;
  return s;
}

astro_status_t astro_chunk_attn_fwd(const astro_kvcache_t* cache, const void* q, const void* k_chunk,
                                    const void* v_chunk, int batch, int heads, int head_dim, int n_q, int n_kc,
                                    float scale, void* o, float* lse, void* stream) {
  if (!q || !o) return ASTRO_ERR_NULL;
  if (n_kc > 0 && (!k_chunk || !v_chunk)) return ASTRO_ERR_NULL;
  const AttnArgs a{cache, batch, heads, head_dim, n_q, n_kc};
  astro_status_t s = check_attn_args(a, scale);
  if (s != ASTRO_OK) return s;
  if (!aligned16(q) || !aligned16(o) || (n_kc > 0 && (!aligned16(k_chunk) || !aligned16(v_chunk))) ||
      (reinterpret_cast<uintptr_t>(lse) & 3u))
    return ASTRO_ERR_ALIGN;
  s = check_arch();
  if (s != ASTRO_OK) return s;
  const bool have_ctx = cache && (cache->sink_held + cache->win_held) > 0;
  CUtensorMap tkc, tvc, tkx, tvx[2];
  std::memset(&tkc, 0, sizeof(tkc)); std::memset(&tvc, 0, sizeof(tvc));
  std::memset(&tkx, 0, sizeof(tkx)); std::memset(tvx, 0, sizeof(tvx));
  if (n_kc > 0) {
    if ((s = make_tmap_user(&tkc, k_chunk, head_dim, n_kc, heads, batch)) != ASTRO_OK) return s;
    if ((s = make_tmap_user(&tvc, v_chunk, head_dim, n_kc, heads, batch)) != ASTRO_OK) return s;
  }
  const KeySegs segs = build_segments(have_ctx ? cache : nullptr, n_kc);
  if (have_ctx) {
    if ((s = cache_maps(cache)) != ASTRO_OK) return s;
    tkx = cache->tm_k;
    // V of each cache key range through a map that ends where the range ends: rows past it are zero-filled by
    // TMA instead of carrying whatever an evicted or never written slot holds (0 * NaN would reach O)
    for (int i = 0, ci = 0; i < segs.n; ++i) {
      if (segs.from_chunk[i]) continue;
      const long long end = static_cast<long long>(segs.start[i]) + segs.count[i];
      if ((s = make_tmap_cache_range(&tvx[ci++], cache, cache->v, end, kTile)) != ASTRO_OK) return s;
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16* qp = static_cast<const __nv_bfloat16*>(q);
  if (head_dim == 128 && g_fwd_mode.load(std::memory_order_relaxed) == 2)
    return launch_fwd_pair(a, cache, have_ctx, q, k_chunk, v_chunk, segs, scale, o, lse, st);
  return head_dim == 128 ? launch_fwd<128>(a, qp, tkc, tvc, tkx, tvx, segs, scale, o, lse, st)
                         : launch_fwd<64>(a, qp, tkc, tvc, tkx, tvx, segs, scale, o, lse, st);
}

size_t astro_chunk_attn_bwd_workspace_bytes(int batch, int heads, int n_q, int head_dim) {
  if (batch < 1 || heads < 1 || n_q < 1 || (head_dim != 64 && head_dim != 128)) return 0;
  const size_t b = static_cast<size_t>(batch) * heads * n_q * sizeof(float);
  return (b + 255) & ~static_cast<size_t>(255);
}

astro_status_t astro_chunk_attn_bwd_delta(const void* o, const void* d_o, int batch, int heads, int head_dim, int n_q,
                                          float* delta, void* stream) {
  if (!o || !d_o || !delta) return ASTRO_ERR_NULL;
  if (batch < 1 || heads < 1 || n_q < 1 || (head_dim != 64 && head_dim != 128)) return ASTRO_ERR_SHAPE;
  if (!aligned16(o) || !aligned16(d_o) || !aligned16(delta)) return ASTRO_ERR_ALIGN;
  astro_status_t s = check_arch();
  if (s != ASTRO_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return head_dim == 128 ? launch_bwd_delta<128>(o, d_o, batch, heads, n_q, delta, st)
                         : launch_bwd_delta<64>(o, d_o, batch, heads, n_q, delta, st);
}

astro_status_t astro_chunk_attn_bwd_dq(const astro_kvcache_t* cache, const void* q, const void* k_chunk,
                                       const void* v_chunk, const float* lse, const float* delta, const void* d_o,
                                       int batch, int heads, int head_dim, int n_q, int n_kc, float scale, void* dq,
                                       void* stream) {
  if (!q || !lse || !delta || !d_o || !dq) return ASTRO_ERR_NULL;
  if (n_kc > 0 && (!k_chunk || !v_chunk)) return ASTRO_ERR_NULL;
  const AttnArgs a{cache, batch, heads, head_dim, n_q, n_kc};
  astro_status_t s = check_attn_args(a, scale);
  if (s != ASTRO_OK) return s;
  if (!aligned16(q) || !aligned16(d_o) || !aligned16(dq) || (reinterpret_cast<uintptr_t>(lse) & 3u) ||
      (reinterpret_cast<uintptr_t>(delta) & 3u) || (n_kc > 0 && (!aligned16(k_chunk) || !aligned16(v_chunk))))
    return ASTRO_ERR_ALIGN;
  s = check_arch();
  if (s != ASTRO_OK) return s;
  const bool have_ctx = cache && (cache->sink_held + cache->win_held) > 0;
  CUtensorMap tdo, tkc, tvc, tkx[2], tvx;
  std::memset(&tkc, 0, sizeof(tkc)); std::memset(&tvc, 0, sizeof(tvc));
  std::memset(tkx, 0, sizeof(tkx)); std::memset(&tvx, 0, sizeof(tvx));
  if ((s = make_tmap_user(&tdo, d_o, head_dim, n_q, heads, batch)) != ASTRO_OK) return s;
  if (n_kc > 0) {
    if ((s = make_tmap_user(&tkc, k_chunk, head_dim, n_kc, heads, batch)) != ASTRO_OK) return s;
    if ((s = make_tmap_user(&tvc, v_chunk, head_dim, n_kc, heads, batch)) != ASTRO_OK) return s;
  }
  const KeySegs segs = build_segments(have_ctx ? cache : nullptr, n_kc);
  if (have_ctx) {
    if ((s = cache_maps(cache)) != ASTRO_OK) return s;
    tvx = cache->tm_v;
    // K of each cache key range through a map that ends where the range ends (rows past it are zeros: dS is 0
    // there, but 0 * NaN from a stale slot would reach dQ)
    for (int i = 0, ci = 0; i < segs.n; ++i) {
      if (segs.from_chunk[i]) continue;
      const long long end = static_cast<long long>(segs.start[i]) + segs.count[i];
      if ((s = make_tmap_cache_range(&tkx[ci++], cache, cache->k, end, kTile)) != ASTRO_OK) return s;
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16* qp = static_cast<const __nv_bfloat16*>(q);
  return head_dim == 128 ? launch_bwd_dq<128>(a, qp, tdo, tkc, tvc, tkx, tvx, segs, scale, lse, delta, dq, st)
                         : launch_bwd_dq<64>(a, qp, tdo, tkc, tvc, tkx, tvx, segs, scale, lse, delta, dq, st);
}

astro_status_t astro_chunk_attn_bwd_dkv(const void* q, const void* k_chunk, const void* v_chunk, const float* lse,
                                        const float* delta, const void* d_o, int batch, int heads, int head_dim,
                                        int n_q, int n_kc, float scale, void* dk_chunk, void* dv_chunk, void* stream) {
  if (!q || !k_chunk || !v_chunk || !lse || !delta || !d_o || !dk_chunk || !dv_chunk) return ASTRO_ERR_NULL;
  const AttnArgs a{nullptr, batch, heads, head_dim, n_q, n_kc};
  astro_status_t s = check_attn_args(a, scale);
  if (s != ASTRO_OK) return s;
  if (!aligned16(q) || !aligned16(d_o) || !aligned16(k_chunk) || !aligned16(v_chunk) || !aligned16(dk_chunk) ||
      !aligned16(dv_chunk) || (reinterpret_cast<uintptr_t>(lse) & 3u) || (reinterpret_cast<uintptr_t>(delta) & 3u))
    return ASTRO_ERR_ALIGN;
  s = check_arch();
  if (s != ASTRO_OK) return s;
  CUtensorMap tq, tdo, tkc, tvc;
  if ((s = make_tmap_user(&tq, q, head_dim, n_q, heads, batch)) != ASTRO_OK) return s;
  if ((s = make_tmap_user(&tdo, d_o, head_dim, n_q, heads, batch)) != ASTRO_OK) return s;
  if ((s = make_tmap_user(&tkc, k_chunk, head_dim, n_kc, heads, batch)) != ASTRO_OK) return s;
  if ((s = make_tmap_user(&tvc, v_chunk, head_dim, n_kc, heads, batch)) != ASTRO_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return head_dim == 128 ? launch_bwd_dkv<128>(a, tq, tdo, tkc, tvc, scale, lse, delta, dk_chunk, dv_chunk, st)
                         : launch_bwd_dkv<64>(a, tq, tdo, tkc, tvc, scale, lse, delta, dk_chunk, dv_chunk, st);
}

astro_status_t astro_chunk_attn_bwd(const astro_kvcache_t* cache, const void* q, const void* k_chunk,
                                    const void* v_chunk, const void* o, const float* lse, const void* d_o, int batch,
                                    int heads, int head_dim, int n_q, int n_kc, float scale, void* dq, void* dk_chunk,
                                    void* dv_chunk, void* workspace, size_t workspace_bytes, void* stream) {
  if (!q || !o || !lse || !d_o || !dq || !workspace) return ASTRO_ERR_NULL;
  if (n_kc > 0 && (!k_chunk || !v_chunk || !dk_chunk || !dv_chunk)) return ASTRO_ERR_NULL;
  const AttnArgs a{cache, batch, heads, head_dim, n_q, n_kc};
  astro_status_t s = check_attn_args(a, scale);
  if (s != ASTRO_OK) return s;
  if (workspace_bytes < astro_chunk_attn_bwd_workspace_bytes(batch, heads, n_q, head_dim)) return ASTRO_ERR_CAPACITY;
  if (!aligned16(q) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) || !aligned16(workspace) ||
      (reinterpret_cast<uintptr_t>(lse) & 3u) ||
      (n_kc > 0 && (!aligned16(k_chunk) || !aligned16(v_chunk) || !aligned16(dk_chunk) || !aligned16(dv_chunk))))
    return ASTRO_ERR_ALIGN;
  float* delta = static_cast<float*>(workspace);
  s = astro_chunk_attn_bwd_delta(o, d_o, batch, heads, head_dim, n_q, delta, stream);
  if (s != ASTRO_OK) return s;
  s = astro_chunk_attn_bwd_dq(cache, q, k_chunk, v_chunk, lse, delta, d_o, batch, heads, head_dim, n_q, n_kc, scale,
                              dq, stream);
  if (s != ASTRO_OK || n_kc == 0) return s;
  return astro_chunk_attn_bwd_dkv(q, k_chunk, v_chunk, lse, delta, d_o, batch, heads, head_dim, n_q, n_kc, scale,
                                  dk_chunk, dv_chunk, stream);
}

astro_status_t astro_nft_loss(const void* v_theta, const void* v_old, const void* v_ref, const void* v_target,
                              const float* r_tilde, const float* w_policy, const float* w_kl, int batch,
                              long long elems, float beta, float* policy_out, float* kl_out, void* grad,
                              void* stream) {
  if (!v_theta || !v_old || !v_target || !r_tilde || !policy_out) return ASTRO_ERR_NULL;
  if ((v_ref == nullptr) != (kl_out == nullptr)) return ASTRO_ERR_NULL;
  if (batch < 1 || batch > 65535 || elems < 8 || (elems & 7)) return ASTRO_ERR_SHAPE;
  if (!aligned16(v_theta) || !aligned16(v_old) || !aligned16(v_target) || (v_ref && !aligned16(v_ref)) ||
      (grad && !aligned16(grad)))
    return ASTRO_ERR_ALIGN;
  astro_status_t s = check_arch();
  if (s != ASTRO_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(policy_out, 0, sizeof(float) * batch, st) != cudaSuccess) return ASTRO_ERR_CUDA;
  if (kl_out && cudaMemsetAsync(kl_out, 0, sizeof(float) * batch, st) != cudaSuccess) return ASTRO_ERR_CUDA;
  const long long vecs = elems / 8;
  const long long per_block = static_cast<long long>(kNftThreads) * kNftVecsPerThread;
  long long blocks = (vecs + per_block - 1) / per_block;
  if (blocks > 4096) blocks = 4096;
  dim3 grid(static_cast<unsigned>(blocks), batch);
  nft_loss_kernel<<<grid, kNftThreads, 0, st>>>(
      static_cast<const uint4*>(v_theta), static_cast<const uint4*>(v_old), static_cast<const uint4*>(v_ref),
      static_cast<const uint4*>(v_target), r_tilde, w_policy, w_kl, vecs, beta, policy_out, kl_out,
      static_cast<uint4*>(grad));
  return launch_status();
}

// ---- backward without caller scratch ---------------------------------------------------------------
// delta lives in this fixed device array.  In host code `g_bwd_static_delta` is only a stand-in for the
// symbol, not a device address: the address each GPU gives it is looked up once per device below.
static __device__ __align__(256) float g_bwd_static_delta[ASTRO_BWD_STATIC_MAX_ROWS];

static astro_status_t bwd_static_scratch(float** out) {
  static std::atomic<float*> addr[kMaxDevices];   // every thread that races here stores the same address
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ASTRO_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return ASTRO_ERR_CUDA;
  float* p = addr[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_bwd_static_delta) != cudaSuccess || !p)
      return ASTRO_ERR_CUDA;
    addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return ASTRO_OK;
}

astro_status_t astro_chunk_attn_bwd_static(const astro_kvcache_t* cache, const void* q, const void* k_chunk,
                                           const void* v_chunk, const void* o, const float* lse, const void* d_o,
                                           int batch, int heads, int head_dim, int n_q, int n_kc, float scale,
                                           void* dq, void* dk_chunk, void* dv_chunk, void* stream) {
  if (!q || !o || !lse || !d_o || !dq) return ASTRO_ERR_NULL;
  if (n_kc > 0 && (!k_chunk || !v_chunk || !dk_chunk || !dv_chunk)) return ASTRO_ERR_NULL;
  const AttnArgs a{cache, batch, heads, head_dim, n_q, n_kc};
  astro_status_t s = check_attn_args(a, scale);
  if (s != ASTRO_OK) return s;
  if (!aligned16(q) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
      (reinterpret_cast<uintptr_t>(lse) & 3u) ||
      (n_kc > 0 && (!aligned16(k_chunk) || !aligned16(v_chunk) || !aligned16(dk_chunk) || !aligned16(dv_chunk))))
    return ASTRO_ERR_ALIGN;
  if (static_cast<long long>(batch) * heads * n_q > ASTRO_BWD_STATIC_MAX_ROWS) return ASTRO_ERR_CAPACITY;
  s = check_arch();
  if (s != ASTRO_OK) return s;
  float* delta = nullptr;
  if ((s = bwd_static_scratch(&delta)) != ASTRO_OK) return s;
  s = astro_chunk_attn_bwd_delta(o, d_o, batch, heads, head_dim, n_q, delta, stream);
  if (s != ASTRO_OK) return s;
  s = astro_chunk_attn_bwd_dq(cache, q, k_chunk, v_chunk, lse, delta, d_o, batch, heads, head_dim, n_q, n_kc, scale,
                              dq, stream);
  if (s != ASTRO_OK || n_kc == 0) return s;
  return astro_chunk_attn_bwd_dkv(q, k_chunk, v_chunk, lse, delta, d_o, batch, heads, head_dim, n_q, n_kc, scale,
                                  dk_chunk, dv_chunk, stream);
}

astro_status_t astro_debug_forward_mode(int mode) {
  if (mode < 0 || mode > 2) return ASTRO_ERR_SHAPE;
  g_fwd_mode.store(mode, std::memory_order_relaxed);
  return ASTRO_OK;
}

astro_status_t astro_debug_pair_flag(int* flag) {
  if (!flag) return ASTRO_ERR_NULL;
  if (cudaDeviceSynchronize() != cudaSuccess) return ASTRO_ERR_CUDA;
  if (cudaMemcpyFromSymbol(flag, g_pair_needs_safe, sizeof(int)) != cudaSuccess) return ASTRO_ERR_CUDA;
  const int zero = 0;
  if (cudaMemcpyToSymbol(g_pair_needs_safe, &zero, sizeof(zero)) != cudaSuccess) return ASTRO_ERR_CUDA;
  return ASTRO_OK;
}

astro_status_t astro_selftest_wait_timeout(void* stream) {
  astro_status_t s = check_arch();
  if (s != ASTRO_OK) return s;
  wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(2000000LL);  // about 1 ms
  return launch_status();
}

astro_status_t astro_last_device_status(uint32_t* detail) {
  if (cudaDeviceSynchronize() != cudaSuccess) return ASTRO_ERR_CUDA;
  uint32_t word = 0;
  if (cudaMemcpyFromSymbol(&word, g_device_status, sizeof(word)) != cudaSuccess) return ASTRO_ERR_CUDA;
  if (detail) *detail = word;
  if (word == 0) return ASTRO_OK;
  const uint32_t zero = 0;
  if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero)) != cudaSuccess) return ASTRO_ERR_CUDA;
  return ASTRO_ERR_TIMEOUT;
}

const char* astro_status_string(astro_status_t s) {
  switch (s) {
    case ASTRO_OK: return "ok";
    case ASTRO_ERR_NULL: return "null pointer";
    case ASTRO_ERR_SHAPE: return "unsupported or inconsistent shape";
    case ASTRO_ERR_ALIGN: return "pointer not 16-byte aligned";
    case ASTRO_ERR_CAPACITY: return "capacity exceeded";
    case ASTRO_ERR_UNDERFLOW: return "evict exceeds window frames held";
    case ASTRO_ERR_ARCH: return "device is not compute capability 10.x";
    case ASTRO_ERR_CUDA: return "CUDA call failed";
    case ASTRO_ERR_TIMEOUT: return "a bounded device-side wait ran out";
  }
  return "unknown status";
}

}  // extern "C"
