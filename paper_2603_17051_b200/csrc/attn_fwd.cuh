// Forward of chunk attention over the rolling cache: O and LSE for one 128-query tile per CTA.
//
// Warp-specialised, one CTA per SM:
//   kFwdGroups softmax groups of 4 warps: group g owns keys [g, g+1) * 128 / kFwdGroups of every key tile,
//   one query row per thread; then one warp whose first thread issues every tcgen05 MMA, one for TMA loads
// Q lives in tensor memory (bf16 pairs, written once by the softmax threads) and is the A operand of
// S = Q K^T, so shared memory only carries K and V: an MMA with both operands in shared memory reads
// 128 B/clk, the whole shared-memory bandwidth, and then competes with the TMA writes of the next tiles.
// S of a whole key tile is one 128x128 MMA into one of two S buffers, issued two tiles ahead.
// The threads that share a query row (one per group) keep the same reference exponent for the row, so all
// parts of P V accumulate into ONE O accumulator; each keeps its own partial row sum.  The fast path takes
// no row maximum: a row re-references itself (true tile maximum, O and row sums rescaled) only when a tile's
// row sum leaves the safe range.  P is written as bf16 pairs over the thread's own S columns.  K and V tiles
// travel through 3-deep rings.
// Part of the exponentials is evaluated by a polynomial on the FMA pipe, because the special-function
// unit (16 exp2 per clock per SM) is as busy as the tensor core at head_dim 128.
//   TMEM columns: S buffers [0,128) [128,256)   O [256,256+D)   Q [384,384+D/2)
#pragma once
#include "attn_common.cuh"

namespace astro {

constexpr int kFwdKStages = 3, kFwdVStages = 3, kFwdSBufs = 2;
constexpr int kFwdGroups = 2;                    // more warps per scheduler hide the exp2 latency
constexpr int kFwdCols = kTile / kFwdGroups;     // keys per group and tile
constexpr int kFwdThreads = 128 * kFwdGroups + 64;

template <int D> struct FwdSmem {
  static constexpr int kK = 0;
  static constexpr int kV = kK + kFwdKStages * TileGeom<D>::kBytes;
  static constexpr int kMax = kV + kFwdVStages * TileGeom<D>::kBytes;  // float [2 parities + 1][groups][128]
  static constexpr int kBars = kMax + 3 * kFwdGroups * kTile * 4;
  static constexpr int kTotal = kBars + 256 + 1024;  // barriers, tmem holder, abort flag + slack to align to 1024
};

constexpr int kPolyOf8 = 2;  // of every 8 pairs of exponentials, how many use the polynomial on the FMA pipe
constexpr float kRowSumLimit = 1073741824.f;  // 2^30: a tile row sum beyond it makes the row re-reference itself

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
chunk_attn_fwd_kernel(const __nv_bfloat16* __restrict__ q, const __grid_constant__ CUtensorMap tm_kc,
                      const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kx,
                      const __grid_constant__ CUtensorMap tm_vx, const KeySegs segs, const int n_q, const int heads,
                      const int cache_shared, const float scale_log2, __nv_bfloat16* __restrict__ o,
                      float* __restrict__ lse) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sK = smem + FwdSmem<D>::kK;
  uint8_t* sV = smem + FwdSmem<D>::kV;
  float* smax = reinterpret_cast<float*>(smem + FwdSmem<D>::kMax);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + FwdSmem<D>::kBars);
  uint64_t* q_full = bars;
  uint64_t* k_full = bars + 1;                    // [kFwdKStages]
  uint64_t* k_empty = k_full + kFwdKStages;
  uint64_t* v_full = k_empty + kFwdKStages;       // [kFwdVStages]
  uint64_t* v_empty = v_full + kFwdVStages;
  uint64_t* s_full = v_empty + kFwdVStages;       // [kFwdSBufs]
  // The groups may run up to two tiles ahead of the MMA thread (S is ready that far), so the P barriers
  // rotate with the S buffers: a barrier is reused only after the MMA thread has consumed its last phase.
  uint64_t* p_full = s_full + kFwdSBufs;          // [kFwdGroups][kFwdSBufs]
  uint64_t* pv_done = p_full + kFwdGroups * kFwdSBufs;  // [2] by tile parity
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
  constexpr uint32_t kColS = 0 /* + 128 * buffer */, kColO = 256, kColQ = 384;
  constexpr int kMmaWarp = 4 * kFwdGroups, kTmaWarp = 4 * kFwdGroups + 1;
  const int n_tiles = seg_tiles(segs);

  if (tid == 0) {
    mbar_init(q_full, 128 * (D / 64));  // the threads that write Q into tensor memory
    for (int i = 0; i < kFwdKStages; ++i) { mbar_init(k_full + i, 1); mbar_init(k_empty + i, 1); }
    for (int i = 0; i < kFwdVStages; ++i) { mbar_init(v_full + i, 1); mbar_init(v_empty + i, 1); }
    for (int i = 0; i < kFwdSBufs; ++i) {
      mbar_init(s_full + i, 1);
      for (int g = 0; g < kFwdGroups; ++g) mbar_init(p_full + g * kFwdSBufs + i, 128);
    }
    mbar_init(pv_done, 1);
    mbar_init(pv_done + 1, 1);
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
      // K runs ahead of V by the S look-ahead: order the loads K0 K1 | V0 K2 | V1 K3 | ...
      KeyTileIter itk, itv;
      auto load_k = [&](int j) {
        const int st = j % kFwdKStages;
        const bool fc = itk.from_chunk(segs);
        mbar_wait_spin(k_empty + st, ((j / kFwdKStages) & 1) ^ 1, abort_flag);
        mbar_arrive_expect_tx(k_full + st, TileGeom<D>::kBytes);
        tma_load_tile<D>(sK + st * TileGeom<D>::kBytes, fc ? &tm_kc : &tm_kx, k_full + st, itk.row0(segs), h,
                         fc ? b : bx);
        itk.next(segs);
      };
      auto load_v = [&](int j) {
        const int st = j % kFwdVStages;
        const bool fc = itv.from_chunk(segs);
        mbar_wait_spin(v_empty + st, ((j / kFwdVStages) & 1) ^ 1, abort_flag);
        mbar_arrive_expect_tx(v_full + st, TileGeom<D>::kBytes);
        tma_load_tile<D>(sV + st * TileGeom<D>::kBytes, fc ? &tm_vc : &tm_vx, v_full + st, itv.row0(segs), h,
                         fc ? b : bx);
        itv.next(segs);
      };
      for (int j = 0; j < kFwdSBufs && j < n_tiles; ++j) load_k(j);
      for (int j = 0; j < n_tiles; ++j) {
        load_v(j);
        if (j + kFwdSBufs < n_tiles) load_k(j + kFwdSBufs);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint64_t k_desc0 = desc_kmajor(smem_u32(sK));
      constexpr uint32_t idesc_s = make_idesc_bf16(kTile, kTile, false, false);
      auto issue_s = [&](int j) {  // S(j) -> buffer j % 2; free because the PV of tile j-2 was issued before
        const int st = j % kFwdKStages;
        mbar_wait_spin(k_full + st, (j / kFwdKStages) & 1, abort_flag);
        tc_fence_after_sync();
        const uint64_t k_desc = desc_step(k_desc0, st * TileGeom<D>::kBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)  // 16 elements of the head dimension = 8 packed Q columns
          mma_ts(tmem_base + kColS + (j % kFwdSBufs) * 128, tmem_base + kColQ + k * 8,
                 desc_step(k_desc, (k >> 2) * TileGeom<D>::kBlockBytes + (k & 3) * 32), idesc_s, k > 0);
        mma_commit(k_empty + st);
        mma_commit(s_full + j % kFwdSBufs);
      };
      mbar_wait_spin(q_full, 0, abort_flag);
      tc_fence_after_sync();
      for (int j = 0; j < kFwdSBufs && j < n_tiles; ++j) issue_s(j);
      for (int j = 0; j < n_tiles; ++j) {
        const int st = j % kFwdVStages, buf = j % kFwdSBufs;
        const uint32_t vt = smem_u32(sV + st * TileGeom<D>::kBytes);
        const uint32_t pcol = tmem_base + kColS + buf * 128;
        mbar_wait_spin(v_full + st, (j / kFwdVStages) & 1, abort_flag);
        // every group first: any of them may have rescaled its part of O, which all MMAs below accumulate into
#pragma unroll
        for (int g = 0; g < kFwdGroups; ++g)
          mbar_wait_spin(p_full + g * kFwdSBufs + buf, (j / kFwdSBufs) & 1, abort_flag);
        tc_fence_after_sync();
        // P of 16 keys = 8 packed columns; group g's pairs start at its own S columns
        constexpr uint32_t idesc = make_idesc_bf16(kTile, D, false, true);
        const uint64_t v_desc = desc_mnmajor(vt, TileGeom<D>::kBlockBytes);
#pragma unroll
        for (int kb = 0; kb < kTile / 16; ++kb) {
          const uint32_t a = pcol + (kb * 16 / kFwdCols) * kFwdCols + (kb * 16 % kFwdCols) / 2;
          mma_ts(tmem_base + kColO, a, desc_step(v_desc, kb * 2048), idesc, (j > 0 || kb > 0) ? 1u : 0u);
        }
        mma_commit(pv_done + (j & 1));
        mma_commit(v_empty + st);
        if (j + kFwdSBufs < n_tiles) issue_s(j + kFwdSBufs);
      }
      mma_commit(o_full);
    }
  } else {
    // ------------------------------------------------------------------ softmax groups
    const int g = warp >> 2;           // group: keys kFwdCols * g .. of every tile
    constexpr int NL = kFwdCols / 32;  // 32-column TMEM loads per thread and tile
    const int r = tid & 127;           // query row inside the tile = TMEM lane
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const int row = q0 + r;
    const bool in_range = row < n_q;
    // Q row -> tensor memory: 64-element halves of the row (32 packed columns each) are dealt to the groups
#pragma unroll
    for (int hq = 0; hq < D / 64; ++hq) {
      if (hq % kFwdGroups != g) continue;
      uint32_t qr[32];
      const uint4* src = reinterpret_cast<const uint4*>(q + ((static_cast<size_t>(b) * n_q + (in_range ? row : 0)) * heads + h) * D + hq * 64);
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        const uint4 t = in_range ? src[v] : make_uint4(0, 0, 0, 0);
        qr[4 * v] = t.x; qr[4 * v + 1] = t.y; qr[4 * v + 2] = t.z; qr[4 * v + 3] = t.w;
      }
      tmem_st32(tmem_lane + kColQ + hq * 32, qr);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(q_full);
    }
    float m_run = -INFINITY, l_run = 0.f;
    int j = 0;
    for (KeyTileIter it; !it.done(segs); it.next(segs), ++j) {
      const int tile_valid = it.valid(segs);
      const int valid = tile_valid - kFwdCols * g;  // valid keys of this group's share (may be <= 0)
      const int buf = j % kFwdSBufs;
      const uint32_t colS = kColS + buf * 128 + g * kFwdCols;
      mbar_wait(s_full + buf, (j / kFwdSBufs) & 1, abort_flag);
      tc_fence_after_sync();

      // P = exp2(s * scale * log2e - m_run) for this thread's keys, with the row sum; m_run is whatever
      // reference the row has had so far (any reference is exact as long as nothing overflows)
      auto exponentiate = [&](uint32_t (&pk)[NL][16]) -> float {
        uint32_t s[NL][32];
#pragma unroll
        for (int c2 = 0; c2 < NL; ++c2) tmem_ld32(tmem_lane + colS + c2 * 32, s[c2]);
        tmem_wait_ld();
        const float neg_m = -m_run;
        float rowsum;
        if (valid < kFwdCols) {
          rowsum = 0.f;
#pragma unroll
          for (int c2 = 0; c2 < NL; ++c2)
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              float p0 = fast_exp2(fmaf(__uint_as_float(s[c2][c]), scale_log2, neg_m));
              float p1 = fast_exp2(fmaf(__uint_as_float(s[c2][c + 1]), scale_log2, neg_m));
              if (c2 * 32 + c >= valid) p0 = 0.f;
              if (c2 * 32 + c + 1 >= valid) p1 = 0.f;
              rowsum += p0 + p1;
              pk[c2][c >> 1] = pack_bf16(p0, p1);
            }
        } else {
          // full tile: packed fp32 arithmetic; kPolyOf8 of every 8 pairs take the polynomial exp2
          const uint64_t sc2 = f32x2(scale_log2, scale_log2), nm2 = f32x2(neg_m, neg_m);
          uint64_t acc_a = f32x2(0.f, 0.f), acc_b = f32x2(0.f, 0.f);
#pragma unroll
          for (int c2 = 0; c2 < NL; ++c2)
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
              pk[c2][c >> 1] = pack_bf16(p0, p1);
            }
          float r0, r1;
          f32x2_split(add2(acc_a, acc_b), r0, r1);
          rowsum = r0 + r1;
        }
        return rowsum;
      };

      // Fast path: no row maximum at all.  The tile is exponentiated against the row's current reference;
      // only if a row sum leaves the safe range (or the row has no reference yet: first tile) does the row take
      // the true maximum of the tile as its new reference.  The two threads of a row must agree, so each
      // publishes its decision and reads the other's (one 64-thread barrier per warp pair and tile).
      uint32_t pk[NL][16];
      float rowsum = 0.f;
      bool redo = m_run == -INFINITY;
      if (!__all_sync(0xffffffffu, redo)) {
        rowsum = exponentiate(pk);
        redo = redo || !(rowsum < kRowSumLimit);   // also true for inf and NaN
      }
      float* fslot = smax + (j & 1) * kFwdGroups * kTile;
      fslot[g * kTile + r] = redo ? 1.f : 0.f;
      named_barrier_sync(1 + (warp & 3), 32 * kFwdGroups);
#pragma unroll
      for (int og = 0; og < kFwdGroups; ++og) redo = redo || fslot[og * kTile + r] != 0.f;
      float alpha = 1.f;
      if (__any_sync(0xffffffffu, redo)) {
        // Slow path (first tile, or scores far above everything seen so far): exact tile maximum, shared
        // between the threads of the row; rows of the warp that did not ask for it keep their reference.
        uint32_t s[NL][32];
#pragma unroll
        for (int c2 = 0; c2 < NL; ++c2) tmem_ld32(tmem_lane + colS + c2 * 32, s[c2]);   // S is still intact
        tmem_wait_ld();
        float mx = -INFINITY;
#pragma unroll
        for (int c2 = 0; c2 < NL; ++c2)
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c2 * 32 + c < valid) mx = fmaxf(mx, __uint_as_float(s[c2][c]));
        float* mslot = smax + 2 * kFwdGroups * kTile;
        mslot[g * kTile + r] = mx;
        named_barrier_sync(1 + (warp & 3), 32 * kFwdGroups);
#pragma unroll
        for (int og = 0; og < kFwdGroups; ++og) mx = fmaxf(mx, mslot[og * kTile + r]);  // finite: >= 1 valid key
        if (redo) {
          const float m_new = mx * scale_log2;
          if (m_run != -INFINITY) alpha = fast_exp2(m_run - m_new);   // may be > 1 if the max went down: exact too
          m_run = m_new;
        }
        if (j > 0) {
          // O must be at rest: wait for the P V of the previous tile.  The barriers alternate with the tile
          // parity, so the awaited phase is at most one completion away.
          mbar_wait(pv_done + ((j - 1) & 1), ((j - 1) >> 1) & 1, abort_flag);
          tc_fence_after_sync();
          // 32-column slices of the row are dealt round-robin to the groups
#pragma unroll
          for (int c4 = 0; c4 < D / 32; ++c4) {
            if (c4 % kFwdGroups != g) continue;
            uint32_t acc[32];
            tmem_ld32(tmem_lane + kColO + c4 * 32, acc);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) acc[c] = __float_as_uint(__uint_as_float(acc[c]) * alpha);
            tmem_st32(tmem_lane + kColO + c4 * 32, acc);
          }
        }
        l_run *= alpha;
        rowsum = exponentiate(pk);
      }
      l_run += rowsum;
#pragma unroll
      for (int c2 = 0; c2 < NL; ++c2)   // in place: this thread has read all of its S columns
        tmem_st16(tmem_lane + colS + c2 * 16, pk[c2]);
      if (g == 0 && tile_valid < kTile) {
        // Rows past the segment's end may hold stale cache contents: P is 0 there, but 0 * NaN is NaN.
        // Group 0 clears them before publishing P_0, which both PV MMAs of the tile are issued after.
        const int st = j % kFwdVStages;
        mbar_wait(v_full + st, (j / kFwdVStages) & 1, abort_flag);
        zero_tile_rows_from<D>(sV + st * TileGeom<D>::kBytes, tile_valid, r);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(p_full + g * kFwdSBufs + buf);
    }

    // ---- epilogue: all groups hold the same running max; row sum = sum of the partial sums;
    //      32-column slices of the output row are dealt round-robin to the groups
    mbar_wait(o_full, 0, abort_flag);
    tc_fence_after_sync();
    float* ex = smax;  // the last tile's maxima were consumed before its P was published
    ex[g * kTile + r] = l_run;
    named_barrier_sync(5, 128 * kFwdGroups);
    float l = 0.f;
#pragma unroll
    for (int og = 0; og < kFwdGroups; ++og) l += ex[og * kTile + r];
    const float inv_l = 1.f / l;
    __nv_bfloat16* dst = o + ((static_cast<size_t>(b) * n_q + (in_range ? row : 0)) * heads + h) * D;
#pragma unroll
    for (int c4 = 0; c4 < D / 32; ++c4)
      if (c4 % kFwdGroups == g) store_row_from_tmem<32>(tmem_lane + kColO + c4 * 32, inv_l, dst + c4 * 32, in_range);
    if (g == 0 && in_range && lse != nullptr)
      lse[(static_cast<size_t>(b) * heads + h) * n_q + row] = (m_run + log2f(l)) * 0.6931471805599453f;
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace astro
