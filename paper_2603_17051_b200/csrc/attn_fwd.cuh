// Forward of chunk attention over the rolling cache: O and LSE for one 128-query tile per CTA.
//
// Warp-specialised, one CTA per SM:
//   warps 0-3  softmax group 0: key tiles 0, 2, 4, ...   (one query row per thread)
//   warps 4-7  softmax group 1: key tiles 1, 3, 5, ...
//   warp  8    one thread issues every tcgen05 MMA        warp 9   one thread issues every TMA load
// Each group keeps its own running max / sum and its own O accumulator in tensor memory, so while one
// group exponentiates its S tile the tensor core works on the other group's tiles; the two partial
// results are merged by their log-sum-exp at the end.  K and V tiles travel through 3-deep rings.
//   TMEM columns: S0 [0,128) S1 [128,256) O0 [256,256+D) O1 [384,384+D); P overlays S as bf16 pairs.
#pragma once
#include "attn_common.cuh"

namespace astro {

constexpr int kFwdStages = 3;
constexpr int kFwdThreads = 320;

template <int D> struct FwdSmem {
  static constexpr int kQ = 0;
  static constexpr int kK = TileGeom<D>::kBytes;
  static constexpr int kV = kK + kFwdStages * TileGeom<D>::kBytes;
  static constexpr int kBars = kV + kFwdStages * TileGeom<D>::kBytes;
  static constexpr int kTotal = kBars + 256 + 1024;  // barriers, tmem holder, abort flag + slack to align to 1024
};

constexpr float kRescaleThreshold = 8.0f;  // log2 units: stale row max tolerated before O is rescaled

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
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
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + FwdSmem<D>::kBars);
  uint64_t* q_full = bars;
  uint64_t* k_full = bars + 1;                    // [kFwdStages]
  uint64_t* k_empty = k_full + kFwdStages;
  uint64_t* v_full = k_empty + kFwdStages;
  uint64_t* v_empty = v_full + kFwdStages;
  uint64_t* s_full = v_empty + kFwdStages;        // [2]
  uint64_t* p_full = s_full + 2;                  // [2]
  uint64_t* o_full = p_full + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(o_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q0 = blockIdx.x * kTile, h = blockIdx.y, b = blockIdx.z;
  const int bx = cache_shared ? 0 : b;
  constexpr uint32_t kTmemCols = 512;
  constexpr uint32_t kColS = 0, kColO = 256;  // + 128 * group
  constexpr int kMmaWarp = 8, kTmaWarp = 9;

  if (tid == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < kFwdStages; ++i) {
      mbar_init(k_full + i, 1);
      mbar_init(k_empty + i, 1);
      mbar_init(v_full + i, 1);
      mbar_init(v_empty + i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(s_full + i, 1);
      mbar_init(p_full + i, 128);
    }
    mbar_init(o_full, 1);
    *abort_flag = 0;
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(tmem_holder, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == kTmaWarp) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_arrive_expect_tx(q_full, TileGeom<D>::kBytes);
      tma_load_tile<D>(sQ, &tm_q, q_full, q0, h, b);
      int j = 0;
      for (KeyTileIter it; !it.done(segs); it.next(segs), ++j) {
        const int st = j % kFwdStages;
        const uint32_t ph = ((j / kFwdStages) & 1) ^ 1;
        const bool fc = it.from_chunk(segs);
        mbar_wait_spin(k_empty + st, ph, abort_flag);
        mbar_arrive_expect_tx(k_full + st, TileGeom<D>::kBytes);
        tma_load_tile<D>(sK + st * TileGeom<D>::kBytes, fc ? &tm_kc : &tm_kx, k_full + st, it.row0(segs), h,
                         fc ? b : bx);
        mbar_wait_spin(v_empty + st, ph, abort_flag);
        mbar_arrive_expect_tx(v_full + st, TileGeom<D>::kBytes);
        tma_load_tile<D>(sV + st * TileGeom<D>::kBytes, fc ? &tm_vc : &tm_vx, v_full + st, it.row0(segs), h,
                         fc ? b : bx);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const int n_tiles = seg_tiles(segs);
      auto issue_pv = [&](int jj) {
        const int g = jj & 1, st = jj % kFwdStages;
        mbar_wait_spin(p_full + g, (jj >> 1) & 1, abort_flag);
        mbar_wait_spin(v_full + st, (jj / kFwdStages) & 1, abort_flag);
        tc_fence_after_sync();
        mma_pb<D>(tmem_base + kColO + g * 128, tmem_base + kColS + g * 128, smem_u32(sV + st * TileGeom<D>::kBytes),
                  jj >= 2);
        mma_commit(v_empty + st);
      };
      mbar_wait_spin(q_full, 0, abort_flag);
      for (int j = 0; j < n_tiles; ++j) {
        const int g = j & 1, st = j % kFwdStages;
        mbar_wait_spin(k_full + st, (j / kFwdStages) & 1, abort_flag);
        tc_fence_after_sync();
        // S_g is free: the PV that read P_g two tiles ago was issued before this point and MMAs run in order
        mma_abT<D>(tmem_base + kColS + g * 128, smem_u32(sQ), smem_u32(sK + st * TileGeom<D>::kBytes));
        mma_commit(k_empty + st);
        mma_commit(s_full + g);
        if (j >= 1) issue_pv(j - 1);
      }
      issue_pv(n_tiles - 1);
      mma_commit(o_full);
    }
  } else {
    // ------------------------------------------------------------------ softmax groups
    const int g = warp >> 2;           // group 0 or 1
    const int r = tid & 127;           // query row inside the tile = TMEM lane
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint32_t colS = kColS + g * 128, colO = kColO + g * 128;
    float m_run = -INFINITY, l_run = 0.f;
    int cnt = 0, j = 0;
    for (KeyTileIter it; !it.done(segs); it.next(segs), ++j) {
      if ((j & 1) != g) continue;
      const int valid = it.valid(segs);
      const bool first = cnt == 0;
      mbar_wait(s_full + g, cnt & 1, abort_flag);
      tc_fence_after_sync();

      uint32_t s[4][32];
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) tmem_ld32(tmem_lane + colS + c4 * 32, s[c4]);
      tmem_wait_ld();
      float mx = -INFINITY;
      if (valid < kTile) {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4)
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c4 * 32 + c < valid) mx = fmaxf(mx, __uint_as_float(s[c4][c]));
      } else {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4)
#pragma unroll
          for (int c = 0; c < 32; ++c) mx = fmaxf(mx, __uint_as_float(s[c4][c]));
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
      for (int c4 = 0; c4 < 4; ++c4)
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float p0 = fast_exp2(fmaf(__uint_as_float(s[c4][c]), scale_log2, -m_run));
          float p1 = fast_exp2(fmaf(__uint_as_float(s[c4][c + 1]), scale_log2, -m_run));
          if (valid < kTile) {
            if (c4 * 32 + c >= valid) p0 = 0.f;
            if (c4 * 32 + c + 1 >= valid) p1 = 0.f;
          }
          rowsum += p0 + p1;
          pk[c4 >> 1][(c4 & 1) * 16 + (c >> 1)] = pack_bf16(p0, p1);
        }
      l_run = l_run * alpha + rowsum;
      tmem_st32(tmem_lane + colS, pk[0]);
      tmem_st32(tmem_lane + colS + 32, pk[1]);
      // O_g is quiescent here: its last PV was issued before this tile's S, which has completed.
      if (!first && __any_sync(0xffffffffu, rescale)) {
#pragma unroll
        for (int c4 = 0; c4 < D / 32; ++c4) {
          uint32_t acc[32];
          tmem_ld32(tmem_lane + colO + c4 * 32, acc);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) acc[c] = __float_as_uint(__uint_as_float(acc[c]) * alpha);
          tmem_st32(tmem_lane + colO + c4 * 32, acc);
        }
      }
      if (valid < kTile) {
        // Rows past the segment's end may hold stale cache contents: P is 0 there, but 0 * NaN is NaN.
        const int st = j % kFwdStages;
        mbar_wait(v_full + st, (j / kFwdStages) & 1, abort_flag);
        zero_tile_rows_from<D>(sV + st * TileGeom<D>::kBytes, valid, r);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(p_full + g);
      ++cnt;
    }

    // ---- merge the two groups' partial results; group g writes columns [g D/2, (g+1) D/2)
    mbar_wait(o_full, 0, abort_flag);
    tc_fence_after_sync();
    float* ex = reinterpret_cast<float*>(sQ);  // Q is no longer read: every MMA has completed
    ex[(g * 2 + 0) * kTile + r] = cnt ? m_run : -INFINITY;
    ex[(g * 2 + 1) * kTile + r] = cnt ? l_run : 0.f;
    named_barrier_sync(1, 256);
    const float m0 = ex[0 * kTile + r], l0 = ex[1 * kTile + r], m1 = ex[2 * kTile + r], l1 = ex[3 * kTile + r];
    const bool two = seg_tiles(segs) >= 2;  // group 1 saw at least one tile (uniform over the CTA)
    const float m = fmaxf(m0, m1);
    const float a0 = fast_exp2(m0 - m), a1 = two ? fast_exp2(m1 - m) : 0.f;
    const float l = l0 * a0 + l1 * a1;
    const float inv_l = 1.f / l;
    const float w0 = a0 * inv_l, w1 = a1 * inv_l;
    const int row = q0 + r;
    const bool in_range = row < n_q;
    __nv_bfloat16* dst = o + ((static_cast<size_t>(b) * n_q + (in_range ? row : 0)) * heads + h) * D + g * (D / 2);
#pragma unroll
    for (int c4 = 0; c4 < D / 64; ++c4) {
      uint32_t x0[32], x1[32];
      tmem_ld32(tmem_lane + kColO + g * (D / 2) + c4 * 32, x0);
      if (two) tmem_ld32(tmem_lane + kColO + 128 + g * (D / 2) + c4 * 32, x1);
      tmem_wait_ld();
      if (in_range) {
        uint4* out = reinterpret_cast<uint4*>(dst + c4 * 32);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            f[e] = __uint_as_float(x0[8 * v + e]) * w0;
            if (two) f[e] = fmaf(__uint_as_float(x1[8 * v + e]), w1, f[e]);
          }
          uint4 w;
          w.x = pack_bf16(f[0], f[1]);
          w.y = pack_bf16(f[2], f[3]);
          w.z = pack_bf16(f[4], f[5]);
          w.w = pack_bf16(f[6], f[7]);
          out[v] = w;
        }
      }
    }
    if (g == 0 && in_range && lse != nullptr)
      lse[(static_cast<size_t>(b) * heads + h) * n_q + row] = (m + log2f(l)) * 0.6931471805599453f;
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace astro
