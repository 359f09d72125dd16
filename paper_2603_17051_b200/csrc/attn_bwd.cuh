// Backward of chunk attention with the cached context detached.
//   delta kernel : delta_i = dO_i . O_i
//   dQ kernel    : query tile stationary, loops over ALL key tiles (cache + chunk):
//                  S = Q K^T, dP = dO V^T, dS = P o (dP - delta), dQ += dS K
//   dK/dV kernel : chunk key tile stationary, loops over query tiles:
//                  S^T = K Q^T, dP^T = V dO^T, dV += P^T dO, dK += dS^T Q   (chunk keys only)
// P is rebuilt from LSE; fp32 accumulators live in tensor memory; no atomics.
#pragma once
#include "attn_common.cuh"

namespace astro {

constexpr float kLog2e = 1.4426950408889634f;

// One warp per (b, token, h) row: delta[b, h, i] = sum_d dO * O.
template <int D>
__global__ void __launch_bounds__(256) bwd_delta_kernel(const __nv_bfloat16* __restrict__ o,
                                                        const __nv_bfloat16* __restrict__ d_o,
                                                        float* __restrict__ delta, int batch, int n_q, int heads) {
  const long long row = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const long long rows = static_cast<long long>(batch) * n_q * heads;
  if (row >= rows) return;
  constexpr int kPerLane = D / 32;  // 2 or 4 bf16
  const __nv_bfloat16* po = o + row * D + lane * kPerLane;
  const __nv_bfloat16* pd = d_o + row * D + lane * kPerLane;
  float acc = 0.f;
  if constexpr (kPerLane == 4) {
    const uint2 a = *reinterpret_cast<const uint2*>(po), c = *reinterpret_cast<const uint2*>(pd);
    const __nv_bfloat162* a2 = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* c2 = reinterpret_cast<const __nv_bfloat162*>(&c);
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float2 x = __bfloat1622float2(a2[i]), y = __bfloat1622float2(c2[i]);
      acc = fmaf(x.x, y.x, acc);
      acc = fmaf(x.y, y.y, acc);
    }
  } else {
    const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(po));
    const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(pd));
    acc = fmaf(x.x, y.x, fmaf(x.y, y.y, 0.f));
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if (lane == 0) {
    const long long bi = row / heads;  // b * n_q + i
    const int h = static_cast<int>(row - bi * heads);
    const long long b = bi / n_q;
    const long long i = bi - b * n_q;
    delta[(b * heads + h) * n_q + i] = acc;
  }
}

template <int D> struct BwdSmem {
  static constexpr int kT0 = 0;                              // Q   (dQ kernel) | K (dK/dV kernel)
  static constexpr int kT1 = TileGeom<D>::kBytes;            // dO               | V
  static constexpr int kT2 = 2 * TileGeom<D>::kBytes;        // K tile           | Q tile
  static constexpr int kT3 = 3 * TileGeom<D>::kBytes;        // V tile           | dO tile
  static constexpr int kRowStats = 4 * TileGeom<D>::kBytes;  // 2 x 128 floats (dK/dV kernel)
  static constexpr int kBars = kRowStats + 1024;
  static constexpr int kTotal = kBars + 64 + 1024;
};

// ------------------------------------------------------------------------------------------ dQ
template <int D>
__global__ void __launch_bounds__(128, 1)
chunk_attn_bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
                         const __grid_constant__ CUtensorMap tm_kc, const __grid_constant__ CUtensorMap tm_vc,
                         const __grid_constant__ CUtensorMap tm_kx, const __grid_constant__ CUtensorMap tm_vx,
                         const KeySegs segs, const int n_q, const int heads, const int cache_shared,
                         const float scale, const float* __restrict__ lse, const float* __restrict__ delta,
                         __nv_bfloat16* __restrict__ dq) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sQ = smem + BwdSmem<D>::kT0;
  uint8_t* sdO = smem + BwdSmem<D>::kT1;
  uint8_t* sK = smem + BwdSmem<D>::kT2;
  uint8_t* sV = smem + BwdSmem<D>::kT3;
  uint64_t* bar_q = reinterpret_cast<uint64_t*>(smem + BwdSmem<D>::kBars);
  uint64_t* bar_kv = bar_q + 1;
  uint64_t* bar_mma = bar_q + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_q + 3);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int q0 = blockIdx.x * kTile, h = blockIdx.y, b = blockIdx.z;
  const int bx = cache_shared ? 0 : b;
  constexpr uint32_t kTmemCols = 512;
  constexpr uint32_t kColS = 0, kColdP = 128, kColdQ = 256, kColdS = 384;

  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_kv, 1);
    mbar_init(bar_mma, 1);
    *abort_flag = 0;
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 0) {
    tmem_alloc(tmem_holder, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);

  if (tid == 0) {
    mbar_arrive_expect_tx(bar_q, 2 * TileGeom<D>::kBytes);
    tma_load_tile<D>(sQ, &tm_q, bar_q, q0, h, b);
    tma_load_tile<D>(sdO, &tm_do, bar_q, q0, h, b);
  }
  const int row = q0 + tid;
  const bool in_range = row < n_q;
  const size_t stat_idx = (static_cast<size_t>(b) * heads + h) * n_q + (in_range ? row : 0);
  const float lse2 = in_range ? lse[stat_idx] * kLog2e : 0.f;
  const float delta_r = in_range ? delta[stat_idx] : 0.f;
  const float scale_log2 = scale * kLog2e;

  uint32_t ph_kv = 0, ph_mma = 0;
  bool first = true;
  for (KeyTileIter it; !it.done(segs); it.next(segs)) {
    const int valid = it.valid(segs);
    if (tid == 0) {
      mbar_arrive_expect_tx(bar_kv, 2 * TileGeom<D>::kBytes);
      const bool fc = it.from_chunk(segs);
      tma_load_tile<D>(sK, fc ? &tm_kc : &tm_kx, bar_kv, it.row0(segs), h, fc ? b : bx);
      tma_load_tile<D>(sV, fc ? &tm_vc : &tm_vx, bar_kv, it.row0(segs), h, fc ? b : bx);
    }
    if (first) mbar_wait(bar_q, 0, abort_flag);
    mbar_wait(bar_kv, ph_kv, abort_flag);
    ph_kv ^= 1;
    if (valid < kTile) zero_tile_rows_from<D>(sK, valid, tid);  // dS is 0 there, but 0 * NaN is NaN
    __syncthreads();

    if (tid == 0) {
      tc_fence_after_sync();
      mma_abT<D>(tmem_base + kColS, smem_u32(sQ), smem_u32(sK));
      mma_abT<D>(tmem_base + kColdP, smem_u32(sdO), smem_u32(sV));
      mma_commit(bar_mma);
    }
    mbar_wait(bar_mma, ph_mma, abort_flag);
    ph_mma ^= 1;
    tc_fence_after_sync();

#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t s[32], dp[32], ds[16];
      tmem_ld32(tmem_lane + kColS + j * 32, s);
      tmem_ld32(tmem_lane + kColdP + j * 32, dp);
      tmem_wait_ld();
#pragma unroll
      for (int c = 0; c < 32; c += 2) {
        const float p0 = fast_exp2(fmaf(__uint_as_float(s[c]), scale_log2, -lse2));
        const float p1 = fast_exp2(fmaf(__uint_as_float(s[c + 1]), scale_log2, -lse2));
        float d0 = p0 * (__uint_as_float(dp[c]) - delta_r);
        float d1 = p1 * (__uint_as_float(dp[c + 1]) - delta_r);
        if (valid < kTile) {
          if (j * 32 + c >= valid) d0 = 0.f;
          if (j * 32 + c + 1 >= valid) d1 = 0.f;
        }
        ds[c >> 1] = pack_bf16(d0, d1);
      }
      tmem_st16(tmem_lane + kColdS + j * 16, ds);
    }
    tmem_wait_st();
    tc_fence_before_sync();
    __syncthreads();

    if (tid == 0) {
      tc_fence_after_sync();
      mma_pb<D>(tmem_base + kColdQ, tmem_base + kColdS, smem_u32(sK), !first);
      mma_commit(bar_mma);
    }
    mbar_wait(bar_mma, ph_mma, abort_flag);
    ph_mma ^= 1;
    tc_fence_after_sync();
    first = false;
  }

  const size_t row_off = ((static_cast<size_t>(b) * n_q + (in_range ? row : 0)) * heads + h) * D;
  store_row_from_tmem<D>(tmem_lane + kColdQ, scale, dq + row_off, in_range);

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------------------------------ dK, dV
template <int D>
__global__ void __launch_bounds__(128, 1)
chunk_attn_bwd_dkv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
                          const __grid_constant__ CUtensorMap tm_kc, const __grid_constant__ CUtensorMap tm_vc,
                          const int n_q, const int n_kc, const int heads, const float scale,
                          const float* __restrict__ lse, const float* __restrict__ delta,
                          __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sK = smem + BwdSmem<D>::kT0;
  uint8_t* sV = smem + BwdSmem<D>::kT1;
  uint8_t* sQ = smem + BwdSmem<D>::kT2;
  uint8_t* sdO = smem + BwdSmem<D>::kT3;
  float* sLse2 = reinterpret_cast<float*>(smem + BwdSmem<D>::kRowStats);
  float* sDelta = sLse2 + kTile;
  uint64_t* bar_kv = reinterpret_cast<uint64_t*>(smem + BwdSmem<D>::kBars);
  uint64_t* bar_q = bar_kv + 1;
  uint64_t* bar_mma = bar_kv + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_kv + 3);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int k0 = blockIdx.x * kTile, h = blockIdx.y, b = blockIdx.z;
  constexpr uint32_t kTmemCols = 512;
  // P^T overlays S^T and dS^T overlays dP^T: a thread rewrites only columns it has already read.
  constexpr uint32_t kColSt = 0, kColPt = 0, kColdPt = 128, kColdSt = 128, kColdK = 256, kColdV = 384;

  if (tid == 0) {
    mbar_init(bar_kv, 1);
    mbar_init(bar_q, 1);
    mbar_init(bar_mma, 1);
    *abort_flag = 0;
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == 0) {
    tmem_alloc(tmem_holder, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);

  if (tid == 0) {
    mbar_arrive_expect_tx(bar_kv, 2 * TileGeom<D>::kBytes);
    tma_load_tile<D>(sK, &tm_kc, bar_kv, k0, h, b);
    tma_load_tile<D>(sV, &tm_vc, bar_kv, k0, h, b);
  }
  const float scale_log2 = scale * kLog2e;
  const size_t stat_base = (static_cast<size_t>(b) * heads + h) * n_q;

  uint32_t ph_q = 0, ph_mma = 0;
  bool first = true;
  for (int q0 = 0; q0 < n_q; q0 += kTile) {
    const int valid = min(kTile, n_q - q0);
    if (tid == 0) {
      mbar_arrive_expect_tx(bar_q, 2 * TileGeom<D>::kBytes);
      tma_load_tile<D>(sQ, &tm_q, bar_q, q0, h, b);
      tma_load_tile<D>(sdO, &tm_do, bar_q, q0, h, b);
    }
    sLse2[tid] = (tid < valid) ? lse[stat_base + q0 + tid] * kLog2e : 0.f;
    sDelta[tid] = (tid < valid) ? delta[stat_base + q0 + tid] : 0.f;
    if (first) mbar_wait(bar_kv, 0, abort_flag);
    mbar_wait(bar_q, ph_q, abort_flag);
    ph_q ^= 1;
    __syncthreads();

    if (tid == 0) {
      tc_fence_after_sync();
      mma_abT<D>(tmem_base + kColSt, smem_u32(sK), smem_u32(sQ));
      mma_abT<D>(tmem_base + kColdPt, smem_u32(sV), smem_u32(sdO));
      mma_commit(bar_mma);
    }
    mbar_wait(bar_mma, ph_mma, abort_flag);
    ph_mma ^= 1;
    tc_fence_after_sync();

#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t s[32], dp[32], pt[16], ds[16];
      tmem_ld32(tmem_lane + kColSt + j * 32, s);
      tmem_ld32(tmem_lane + kColdPt + j * 32, dp);
      tmem_wait_ld();
#pragma unroll
      for (int c = 0; c < 32; c += 2) {
        const int qa = j * 32 + c;
        float p0 = fast_exp2(fmaf(__uint_as_float(s[c]), scale_log2, -sLse2[qa]));
        float p1 = fast_exp2(fmaf(__uint_as_float(s[c + 1]), scale_log2, -sLse2[qa + 1]));
        if (valid < kTile) {  // query rows past n_q: zero Q and dO rows, no LSE
          if (qa >= valid) p0 = 0.f;
          if (qa + 1 >= valid) p1 = 0.f;
        }
        const float d0 = p0 * (__uint_as_float(dp[c]) - sDelta[qa]);
        const float d1 = p1 * (__uint_as_float(dp[c + 1]) - sDelta[qa + 1]);
        pt[c >> 1] = pack_bf16(p0, p1);
        ds[c >> 1] = pack_bf16(d0, d1);
      }
      tmem_st16(tmem_lane + kColPt + j * 16, pt);
      tmem_st16(tmem_lane + kColdSt + j * 16, ds);
    }
    tmem_wait_st();
    tc_fence_before_sync();
    __syncthreads();

    if (tid == 0) {
      tc_fence_after_sync();
      mma_pb<D>(tmem_base + kColdV, tmem_base + kColPt, smem_u32(sdO), !first);
      mma_pb<D>(tmem_base + kColdK, tmem_base + kColdSt, smem_u32(sQ), !first);
      mma_commit(bar_mma);
    }
    mbar_wait(bar_mma, ph_mma, abort_flag);
    ph_mma ^= 1;
    tc_fence_after_sync();
    first = false;
  }

  const int krow = k0 + tid;
  const bool in_range = krow < n_kc;
  const size_t row_off = ((static_cast<size_t>(b) * n_kc + (in_range ? krow : 0)) * heads + h) * D;
  store_row_from_tmem<D>(tmem_lane + kColdK, scale, dk + row_off, in_range);
  store_row_from_tmem<D>(tmem_lane + kColdV, 1.f, dv + row_off, in_range);

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace astro
