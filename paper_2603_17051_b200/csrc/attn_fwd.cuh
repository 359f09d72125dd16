// Forward of chunk attention over the rolling cache: O and LSE for one 128-query tile per CTA.
//
// Warp-specialised, one CTA per SM:
//   warps 0-3  softmax group 0: keys  0..63  of every key tile (one query row per thread)
//   warps 4-7  softmax group 1: keys 64..127 of every key tile
//   warp  8    one thread issues every tcgen05 MMA        warp 9   one thread issues every TMA load
// S = Q K^T of a whole key tile is one 128x128 MMA into one of two S buffers, issued two tiles ahead.
// Each group is an independent softmax stream over its half of the keys: own running max / sum, own O
// accumulator (O_g += P_g V[64g..64g+63]); the two partial results are merged by their log-sum-exp at the
// end.  P_g is written as bf16 pairs over the group's own S columns.  K and V tiles travel through
// 3-deep rings.  Part of the exponentials is evaluated by a polynomial on the FMA pipe, because the
// special-function unit (16 exp2 per clock per SM) is as busy as the tensor core at head_dim 128.
//   TMEM columns: S buffer 0 [0,128)  S buffer 1 [128,256)  O_0 [256,256+D)  O_1 [384,384+D)
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

constexpr int kPolyOf8 = 3;  // of every 8 pairs of exponentials, how many use the polynomial on the FMA pipe
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
  uint64_t* s_full = v_empty + kFwdStages;        // [2] per S buffer
  // A group may publish P of tile j+1 before the MMA thread has looked at tile j (it only needs S(j+1),
  // issued long before), so one barrier per group would let a phase go by unseen: alternate two per group.
  uint64_t* p_full = s_full + 2;                  // [2 groups][2 tile parities]
  uint64_t* pv_done = p_full + 4;                 // [2] per group
  uint64_t* o_full = pv_done + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(o_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // With one shared cache (frozen prefix of a sample group) the samples of a head are launched next to each
  // other, so the head's cached K/V is fetched from HBM once and served to the whole group out of L2.
  const int q0 = blockIdx.x * kTile;
  const int h = cache_shared ? blockIdx.z : blockIdx.y, b = cache_shared ? blockIdx.y : blockIdx.z;
  const int bx = cache_shared ? 0 : b;
  constexpr uint32_t kTmemCols = 512;
  constexpr uint32_t kColS = 0 /* + 128 * buffer */, kColO = 256 /* + 128 * group */;
  constexpr int kMmaWarp = 8, kTmaWarp = 9;
  constexpr int kHalfBytes = 64 * 128;  // 64 rows of a block
  const int n_tiles = seg_tiles(segs);

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
      mbar_init(p_full + 2 * i, 128);
      mbar_init(p_full + 2 * i + 1, 128);
      mbar_init(pv_done + i, 1);
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
      // K runs two tiles ahead of V: order the loads K0 K1 | V0 K2 | V1 K3 | ...
      KeyTileIter itk, itv;
      auto load_k = [&](int j) {
        const int st = j % kFwdStages;
        const bool fc = itk.from_chunk(segs);
        mbar_wait_spin(k_empty + st, ((j / kFwdStages) & 1) ^ 1, abort_flag);
        mbar_arrive_expect_tx(k_full + st, TileGeom<D>::kBytes);
        tma_load_tile<D>(sK + st * TileGeom<D>::kBytes, fc ? &tm_kc : &tm_kx, k_full + st, itk.row0(segs), h,
                         fc ? b : bx);
        itk.next(segs);
      };
      auto load_v = [&](int j) {
        const int st = j % kFwdStages;
        const bool fc = itv.from_chunk(segs);
        mbar_wait_spin(v_empty + st, ((j / kFwdStages) & 1) ^ 1, abort_flag);
        mbar_arrive_expect_tx(v_full + st, TileGeom<D>::kBytes);
        tma_load_tile<D>(sV + st * TileGeom<D>::kBytes, fc ? &tm_vc : &tm_vx, v_full + st, itv.row0(segs), h,
                         fc ? b : bx);
        itv.next(segs);
      };
      load_k(0);
      if (n_tiles > 1) load_k(1);
      for (int j = 0; j < n_tiles; ++j) {
        load_v(j);
        if (j + 2 < n_tiles) load_k(j + 2);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      auto issue_s = [&](int j) {  // S(j) -> buffer j & 1; free because both PVs of tile j-2 were issued before
        const int st = j % kFwdStages;
        mbar_wait_spin(k_full + st, (j / kFwdStages) & 1, abort_flag);
        tc_fence_after_sync();
        mma_abT<D>(tmem_base + kColS + (j & 1) * 128, smem_u32(sQ), smem_u32(sK + st * TileGeom<D>::kBytes));
        mma_commit(k_empty + st);
        mma_commit(s_full + (j & 1));
      };
      mbar_wait_spin(q_full, 0, abort_flag);
      issue_s(0);
      if (n_tiles > 1) issue_s(1);
      for (int j = 0; j < n_tiles; ++j) {
        const int st = j % kFwdStages;
        const uint32_t vt = smem_u32(sV + st * TileGeom<D>::kBytes);
        const uint32_t pcol = tmem_base + kColS + (j & 1) * 128;
        mbar_wait_spin(v_full + st, (j / kFwdStages) & 1, abort_flag);
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          mbar_wait_spin(p_full + 2 * g + (j & 1), (j >> 1) & 1, abort_flag);
          tc_fence_after_sync();
          mma_pb<D, 64>(tmem_base + kColO + g * 128, pcol + g * 64, vt + g * kHalfBytes, j > 0);
          mma_commit(pv_done + g);
        }
        mma_commit(v_empty + st);
        if (j + 2 < n_tiles) issue_s(j + 2);
      }
      mma_commit(o_full);
    }
  } else {
    // ------------------------------------------------------------------ softmax groups
    const int g = warp >> 2;           // group: keys 64g..64g+63 of every tile
    const int r = tid & 127;           // query row inside the tile = TMEM lane
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint32_t colO = kColO + g * 128;
    float m_run = -INFINITY, l_run = 0.f;
    int j = 0;
    for (KeyTileIter it; !it.done(segs); it.next(segs), ++j) {
      const int tile_valid = it.valid(segs);
      const int valid = tile_valid - 64 * g;  // valid keys of this group's half (may be <= 0)
      const uint32_t colS = kColS + (j & 1) * 128 + g * 64;
      mbar_wait(s_full + (j & 1), (j >> 1) & 1, abort_flag);
      tc_fence_after_sync();

      uint32_t s[2][32];
      tmem_ld32(tmem_lane + colS, s[0]);
      tmem_ld32(tmem_lane + colS + 32, s[1]);
      tmem_wait_ld();
      float mx;
      if (valid < 64) {
        mx = -INFINITY;
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2)
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c2 * 32 + c < valid) mx = fmaxf(mx, __uint_as_float(s[c2][c]));
      } else {
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2)
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            mx0 = max3(mx0, __uint_as_float(s[c2][c]), __uint_as_float(s[c2][c + 1]));
            mx1 = max3(mx1, __uint_as_float(s[c2][c + 2]), __uint_as_float(s[c2][c + 3]));
            mx2 = max3(mx2, __uint_as_float(s[c2][c + 4]), __uint_as_float(s[c2][c + 5]));
            mx3 = max3(mx3, __uint_as_float(s[c2][c + 6]), __uint_as_float(s[c2][c + 7]));
          }
        mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      }
      const bool any_valid = valid > 0;
      float alpha = 1.f;
      bool rescale = false;
      if (any_valid) {
        const float m_new = mx * scale_log2;
        if (m_run == -INFINITY) {
          m_run = m_new;                      // first keys of this stream: O_g holds nothing but zeros so far
        } else if (m_new - m_run > kRescaleThreshold) {
          alpha = fast_exp2(m_run - m_new);
          m_run = m_new;
          rescale = true;
        }
      }
      const float neg_m = any_valid ? -m_run : 0.f;
      float rowsum;
      uint32_t pk[32];
      if (valid < 64) {
        rowsum = 0.f;
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2)
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            float p0 = fast_exp2(fmaf(__uint_as_float(s[c2][c]), scale_log2, neg_m));
            float p1 = fast_exp2(fmaf(__uint_as_float(s[c2][c + 1]), scale_log2, neg_m));
            if (c2 * 32 + c >= valid) p0 = 0.f;
            if (c2 * 32 + c + 1 >= valid) p1 = 0.f;
            rowsum += p0 + p1;
            pk[c2 * 16 + (c >> 1)] = pack_bf16(p0, p1);
          }
      } else {
        // full tile: packed fp32 arithmetic; kPolyOf8 of every 8 pairs take the polynomial exp2 so that the
        // special-function unit and the FMA pipe share the exponentials
        const uint64_t sc2 = f32x2(scale_log2, scale_log2), nm2 = f32x2(neg_m, neg_m);
        uint64_t acc_a = f32x2(0.f, 0.f), acc_b = f32x2(0.f, 0.f);
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2)
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const uint64_t x2 = fma2(f32x2(__uint_as_float(s[c2][c]), __uint_as_float(s[c2][c + 1])), sc2, nm2);
            float p0, p1;
            if (((c >> 1) & 7) < kPolyOf8) {
              exp2_poly_pair(x2, p0, p1);
            } else {
              float x0, x1;
              f32x2_split(x2, x0, x1);
              p0 = fast_exp2(x0);
              p1 = fast_exp2(x1);
            }
            if ((c >> 1) & 1) acc_a = add2(acc_a, f32x2(p0, p1));
            else acc_b = add2(acc_b, f32x2(p0, p1));
            pk[c2 * 16 + (c >> 1)] = pack_bf16(p0, p1);
          }
        float r0, r1;
        f32x2_split(add2(acc_a, acc_b), r0, r1);
        rowsum = r0 + r1;
      }
      l_run = l_run * alpha + rowsum;
      tmem_st32(tmem_lane + colS, pk);  // in place: this thread has read all 64 of its S columns
      if (__any_sync(0xffffffffu, rescale)) {
        // O_g must be at rest: wait for the PV of the previous tile (rescale implies j >= 1).  The barrier
        // has completed j-1 or j phases here, so the parity of phase j-1 is unambiguous.
        mbar_wait(pv_done + g, (j - 1) & 1, abort_flag);
        tc_fence_after_sync();
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
      if (g == 0 && tile_valid < kTile) {
        // Rows past the segment's end may hold stale cache contents: P is 0 there, but 0 * NaN is NaN.
        // Group 0 clears them before publishing P_0, which both PV MMAs of the tile are issued after.
        const int st = j % kFwdStages;
        mbar_wait(v_full + st, (j / kFwdStages) & 1, abort_flag);
        zero_tile_rows_from<D>(sV + st * TileGeom<D>::kBytes, tile_valid, r);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(p_full + 2 * g + (j & 1));
    }

    // ---- merge the two streams; group g writes columns [g D/2, (g+1) D/2)
    mbar_wait(o_full, 0, abort_flag);
    tc_fence_after_sync();
    float* ex = reinterpret_cast<float*>(sQ);  // Q is no longer read: every MMA has completed
    ex[(g * 2 + 0) * kTile + r] = m_run;
    ex[(g * 2 + 1) * kTile + r] = l_run;
    named_barrier_sync(1, 256);
    const float m0 = ex[0 * kTile + r], l0 = ex[1 * kTile + r], m1 = ex[2 * kTile + r], l1 = ex[3 * kTile + r];
    const float m = fmaxf(m0, m1);  // finite: the first key tile has at least one key in group 0's half
    const float a0 = l0 > 0.f ? fast_exp2(m0 - m) : 0.f, a1 = l1 > 0.f ? fast_exp2(m1 - m) : 0.f;
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
      tmem_ld32(tmem_lane + kColO + 128 + g * (D / 2) + c4 * 32, x1);
      tmem_wait_ld();
      if (in_range) {
        uint4* out = reinterpret_cast<uint4*>(dst + c4 * 32);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e)
            f[e] = fmaf(__uint_as_float(x1[8 * v + e]), w1, __uint_as_float(x0[8 * v + e]) * w0);
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
