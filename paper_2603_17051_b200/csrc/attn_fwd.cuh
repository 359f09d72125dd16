// Forward of chunk attention over the rolling cache: O and LSE for one 128-query tile per CTA.
// TMA brings Q once and one K/V key tile at a time; tcgen05 MMAs form S = Q K^T and O += P V with
// accumulators in tensor memory; each of the 128 threads owns one query row for the online softmax.
// Two CTAs share an SM, so one CTA's softmax overlaps the other's MMAs.
#pragma once
#include "attn_common.cuh"

namespace astro {

template <int D> struct FwdSmem {
  static constexpr int kQ = 0;
  static constexpr int kK = TileGeom<D>::kBytes;
  static constexpr int kV = 2 * TileGeom<D>::kBytes;
  static constexpr int kBars = 3 * TileGeom<D>::kBytes;  // 3 mbarriers, tmem holder, abort flag
  static constexpr int kTotal = kBars + 64 + 1024;       // + slack to align the base to 1024
};

constexpr float kRescaleThreshold = 8.0f;  // log2 units: stale row max tolerated before O is rescaled

template <int D>
__global__ void __launch_bounds__(128, 2)
chunk_attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kc,
                      const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kx,
                      const __grid_constant__ CUtensorMap tm_vx, const KeySegs segs, const int n_q, const int heads,
                      const int cache_shared, const float scale_log2, __nv_bfloat16* __restrict__ o,
                      float* __restrict__ lse) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sQ = smem + FwdSmem<D>::kQ;
  uint8_t* sK = smem + FwdSmem<D>::kK;
  uint8_t* sV = smem + FwdSmem<D>::kV;
  uint64_t* bar_q = reinterpret_cast<uint64_t*>(smem + FwdSmem<D>::kBars);
  uint64_t* bar_kv = bar_q + 1;
  uint64_t* bar_mma = bar_q + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_q + 3);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int q0 = blockIdx.x * kTile, h = blockIdx.y, b = blockIdx.z;
  const int bx = cache_shared ? 0 : b;
  constexpr uint32_t kTmemCols = 256;
  constexpr uint32_t kColS = 0, kColP = 0, kColO = 128;

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
    mbar_arrive_expect_tx(bar_q, TileGeom<D>::kBytes);
    tma_load_tile<D>(sQ, &tm_q, bar_q, q0, h, b);
  }
  uint32_t ph_kv = 0, ph_mma = 0;
  float m_run = -INFINITY, l_run = 0.f;
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
    // Rows past the segment's end may hold stale cache contents: P is 0 there, but 0 * NaN is NaN.
    if (valid < kTile) zero_tile_rows_from<D>(sV, valid, tid);

    if (tid == 0) {
      tc_fence_after_sync();
      mma_abT<D>(tmem_base + kColS, smem_u32(sQ), smem_u32(sK));
      mma_commit(bar_mma);
    }
    mbar_wait(bar_mma, ph_mma, abort_flag);
    ph_mma ^= 1;
    tc_fence_after_sync();

    // ---- online softmax on this thread's row
    uint32_t s[4][32];
#pragma unroll
    for (int j = 0; j < 4; ++j) tmem_ld32(tmem_lane + kColS + j * 32, s[j]);
    tmem_wait_ld();
    float mx = -INFINITY;
    if (valid < kTile) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int c = 0; c < 32; ++c)
          if (j * 32 + c < valid) mx = fmaxf(mx, __uint_as_float(s[j][c]));
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int c = 0; c < 32; ++c) mx = fmaxf(mx, __uint_as_float(s[j][c]));
    }
    const float m_new = mx * scale_log2;
    float alpha = 1.f;
    bool rescale = false;
    if (first) {
      m_run = m_new;
    } else if (m_new - m_run > kRescaleThreshold) {
      alpha = fast_exp2(m_run - m_new);
      m_run = m_new;
      rescale = true;
    }
    float rowsum = 0.f;
    uint32_t pk[2][32];
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int c = 0; c < 32; c += 2) {
        float p0 = fast_exp2(fmaf(__uint_as_float(s[j][c]), scale_log2, -m_run));
        float p1 = fast_exp2(fmaf(__uint_as_float(s[j][c + 1]), scale_log2, -m_run));
        if (valid < kTile) {
          if (j * 32 + c >= valid) p0 = 0.f;
          if (j * 32 + c + 1 >= valid) p1 = 0.f;
        }
        rowsum += p0 + p1;
        pk[j >> 1][(j & 1) * 16 + (c >> 1)] = pack_bf16(p0, p1);
      }
    l_run = l_run * alpha + rowsum;
    tmem_st32(tmem_lane + kColP, pk[0]);
    tmem_st32(tmem_lane + kColP + 32, pk[1]);
    if (!first && __any_sync(0xffffffffu, rescale)) {
#pragma unroll
      for (int j = 0; j < D / 32; ++j) {
        uint32_t r[32];
        tmem_ld32(tmem_lane + kColO + j * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
        tmem_st32(tmem_lane + kColO + j * 32, r);
      }
    }
    tmem_wait_st();
    tc_fence_before_sync();
    __syncthreads();

    if (tid == 0) {
      tc_fence_after_sync();
      mma_pb<D>(tmem_base + kColO, tmem_base + kColP, smem_u32(sV), !first);
      mma_commit(bar_mma);
    }
    mbar_wait(bar_mma, ph_mma, abort_flag);
    ph_mma ^= 1;
    tc_fence_after_sync();
    first = false;
  }

  // ---- epilogue: O / l as bf16, LSE in natural log
  const int row = q0 + tid;
  const bool in_range = row < n_q;
  const float inv_l = 1.f / l_run;
  const size_t row_off = ((static_cast<size_t>(b) * n_q + (in_range ? row : 0)) * heads + h) * D;
  store_row_from_tmem<D>(tmem_lane + kColO, inv_l, o + row_off, in_range);
  if (in_range && lse != nullptr)
    lse[(static_cast<size_t>(b) * heads + h) * n_q + row] = (m_run + log2f(l_run)) * 0.6931471805599453f;

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace astro
