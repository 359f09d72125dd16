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

// ------------------------------------------------------------------------------------------ dQ
// Warp-specialised, one CTA (one 128-query tile) per SM:
//   kDqGroups groups of 4 warps; group g owns keys [g, g+1) * 128 / kDqGroups of every key tile, one query
//   row per thread; then one warp whose first thread issues every tcgen05 MMA and one for every TMA load
// Per key tile j: S(j) = Q K^T and dP(j) = dO V^T are full 128x128 MMAs into single buffers that the
// groups hand back as soon as their values are in registers, so S(j+1) and dP(j+1) are computed while the
// groups still work on tile j.  dS = P o (dP - delta) goes to a bf16 buffer and dQ += dS K follows.  Q lives
// in tensor memory (bf16 pairs, written once by the softmax threads) as the A operand of S, which takes a
// quarter of the operand traffic off shared memory.
// The MMA-issuing thread sets the pace of the kernel, so it gets two waits and two commits per key tile:
//   rs[j % 4]  every thread has S(j) in registers AND the bytes of K(j+1) have landed -> S(j+1), commit s_full
//   rb[j % 4]  every thread has stored dS(j) (so it has dP(j) in registers too) AND the bytes of V(j+1) have
//              landed -> dP(j+1) and dQ(j) as one burst, commit b_done
// b_done is committed once before the loop (behind dP(0)) and once per tile: commit number j+1 says dP(j) is
// ready and dQ(j-1) is done, which frees the dS buffer, the K stage of tile j-1 and the V stage of tile j.  The
// commits alternate between two barriers (commit k goes to b_done[k & 1]), because the producer may be asked
// for commit k only after commit k+1 has happened, and a single barrier cannot be two phases ahead of a waiter.
// Cache K goes through tensor maps that end where a key range ends, so rows past it are zeros, never stale data
// (dS is 0 there, but 0 * NaN would reach dQ).
//   TMEM columns: S [0,128)  dP [128,256)  dS [256,320)  Q [320,320+D/2)  dQ [384,384+D)
constexpr int kDqKStages = 3, kDqVStages = 2;
constexpr int kDqGroups = 2;                      // softmax groups: more warps per scheduler hide the
constexpr int kDqCols = kTile / kDqGroups;         // exp2 latency behind the arithmetic of the other warps
constexpr int kDqSoftmaxThreads = 128 * kDqGroups;
constexpr int kDqThreads = kDqSoftmaxThreads + 64;
constexpr int kDqPolyOf8 = 0;  // share of the exponentials on the FMA pipe: none pays (1.122 ms with 2/8 vs 1.086)

template <int D> struct DqSmem {
  static constexpr int kdO = 0;
  static constexpr int kK = TileGeom<D>::kBytes;
  static constexpr int kV = kK + kDqKStages * TileGeom<D>::kBytes;
  static constexpr int kBars = kV + kDqVStages * TileGeom<D>::kBytes;
  static constexpr int kTotal = kBars + 256 + 1024;
};

template <int D>
__global__ void __launch_bounds__(kDqThreads, 1)
chunk_attn_bwd_dq_kernel(const __nv_bfloat16* __restrict__ q, const __grid_constant__ CUtensorMap tm_do,
                         const __grid_constant__ CUtensorMap tm_kc, const __grid_constant__ CUtensorMap tm_vc,
                         const __grid_constant__ CUtensorMap tm_kx0, const __grid_constant__ CUtensorMap tm_kx1,
                         const __grid_constant__ CUtensorMap tm_vx, const __grid_constant__ KeySegs segs, const int n_q,
                         const int heads, const int cache_shared, const float scale, const float* __restrict__ lse,
                         const float* __restrict__ delta, __nv_bfloat16* __restrict__ dq) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sdO = smem + DqSmem<D>::kdO;
  uint8_t* sK = smem + DqSmem<D>::kK;
  uint8_t* sV = smem + DqSmem<D>::kV;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + DqSmem<D>::kBars);
  uint64_t* kv0_full = bars;                   // dO, K(0), V(0) have landed
  uint64_t* qt_full = bars + 1;                // Q is in tensor memory
  uint64_t* rs = bars + 2;                     // [4]
  uint64_t* rb = bars + 6;                     // [4]
  uint64_t* s_full = bars + 10;                // S(j) computed
  uint64_t* b_done = bars + 11;                // [2], see above
  uint64_t* dq_full = bars + 13;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 14);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // With one shared cache (frozen prefix of a sample group) the samples of a head are launched next to each
  // other, so the head's cached K/V is fetched from HBM once and served to the whole group out of L2.
  const int q0 = blockIdx.x * kTile;
  const int h = cache_shared ? blockIdx.z : blockIdx.y, b = cache_shared ? blockIdx.y : blockIdx.z;
  const int bx = cache_shared ? 0 : b;
  constexpr uint32_t kTmemCols = 512;
  constexpr uint32_t kColS = 0, kColdP = 128, kColdS = 256, kColQ = 320, kColdQ = 384;
  constexpr int kMmaWarp = 4 * kDqGroups, kTmaWarp = 4 * kDqGroups + 1;
  const int n_tiles = seg_tiles(segs);

  if (tid == 0) {
    mbar_init(kv0_full, 1);
    mbar_init(qt_full, 128 * (D / 64));
    for (int i = 0; i < 4; ++i) { mbar_init(rs + i, 1 + kDqSoftmaxThreads); mbar_init(rb + i, 1 + kDqSoftmaxThreads); }
    mbar_init(s_full, 1);
    mbar_init(b_done, 1);
    mbar_init(b_done + 1, 1);
    mbar_init(dq_full, 1);
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
    if (lane == 0) {
      KeyTileIter it;
      auto load_kv = [&](int t, uint64_t* k_bar, uint64_t* v_bar) {   // K(t), V(t) of the tile the iterator is on
        const bool fc = it.from_chunk(segs);
        const CUtensorMap* tk = fc ? &tm_kc : (it.seg == 0 ? &tm_kx0 : &tm_kx1);
        tma_load_tile<D>(sK + (t % kDqKStages) * TileGeom<D>::kBytes, tk, k_bar, it.row0(segs), h, fc ? b : bx);
        tma_load_tile<D>(sV + (t % kDqVStages) * TileGeom<D>::kBytes, fc ? &tm_vc : &tm_vx, v_bar, it.row0(segs), h,
                         fc ? b : bx);
        it.next(segs);
      };
      mbar_arrive_expect_tx(kv0_full, 3 * TileGeom<D>::kBytes);
      tma_load_tile<D>(sdO, &tm_do, kv0_full, q0, h, b);
      load_kv(0, kv0_full, kv0_full);
      for (int t = 1; t <= n_tiles; ++t) {
        // commit t-1 of b_done: dQ(t-3) and dP(t-2) are done, the K stage and the V stage of tile t are free
        if (t >= 2 && !mbar_wait_spin(b_done + ((t - 1) & 1), ((t - 2) >> 1) & 1, abort_flag)) break;
        if (t < n_tiles) {
          mbar_arrive_expect_tx(rs + (t - 1) % 4, TileGeom<D>::kBytes);
          mbar_arrive_expect_tx(rb + (t - 1) % 4, TileGeom<D>::kBytes);
          load_kv(t, rs + (t - 1) % 4, rb + (t - 1) % 4);
        } else {
          mbar_arrive(rb + (t - 1) % 4);   // the last tile's burst waits for no bytes (its rs is never awaited)
        }
      }
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kTile, kTile, false, false);
      const uint64_t k_desc0 = desc_kmajor(smem_u32(sK));
      auto issue_s = [&](int j) {
        const uint64_t k_desc = desc_step(k_desc0, (j % kDqKStages) * TileGeom<D>::kBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)  // 16 elements of the head dimension = 8 packed Q columns
          mma_ts(tmem_base + kColS, tmem_base + kColQ + k * 8,
                 desc_step(k_desc, (k >> 2) * TileGeom<D>::kBlockBytes + (k & 3) * 32), idesc_s, k > 0);
        mma_commit(s_full);
      };
      auto issue_dp = [&](int j) {
        mma_abT<D>(tmem_base + kColdP, smem_u32(sdO), smem_u32(sV + (j % kDqVStages) * TileGeom<D>::kBytes));
      };
      mbar_wait_spin(qt_full, 0, abort_flag);
      mbar_wait_spin(kv0_full, 0, abort_flag);
      tc_fence_after_sync();
      issue_s(0);
      issue_dp(0);
      mma_commit(b_done + 1);                       // commit 1
      for (int j = 0; j < n_tiles; ++j) {
        const bool more = j + 1 < n_tiles;
        if (more) {
          mbar_wait_spin(rs + j % 4, (j / 4) & 1, abort_flag);
          tc_fence_after_sync();
          issue_s(j + 1);
        }
        mbar_wait_spin(rb + j % 4, (j / 4) & 1, abort_flag);
        tc_fence_after_sync();
        if (more) issue_dp(j + 1);
        mma_pb<D, kTile>(tmem_base + kColdQ, tmem_base + kColdS, smem_u32(sK + (j % kDqKStages) * TileGeom<D>::kBytes), j > 0);
        mma_commit(b_done + (j & 1));                 // commit j + 2
      }
      mma_commit(dq_full);
    }
  } else {
    const int g = warp >> 2;
    const int r = tid & 127;
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const int row = q0 + r;
    const bool in_range = row < n_q;
    const size_t stat_idx = (static_cast<size_t>(b) * heads + h) * n_q + (in_range ? row : 0);
    const float lse2 = in_range ? lse[stat_idx] * kLog2e : 0.f;
    const float delta_r = in_range ? delta[stat_idx] : 0.f;
    const float scale_log2 = scale * kLog2e;
    const uint64_t sc2 = f32x2(scale_log2, scale_log2), nl2 = f32x2(-lse2, -lse2), nd2 = f32x2(-delta_r, -delta_r);
    // Q row -> tensor memory: group g writes elements [64g, 64g+64) of its row as 32 packed columns
    if (g * 64 < D) {
      uint32_t qr[32];
      const QuadRows q_rows = quad_rows(q, b, h, n_q, heads, D, row);   // the quads of a warp fetch their rows together
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint4 ch[4];
        load_quad_rows(ch, q_rows, g * 64 + half * 32, tid & 31);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          qr[16 * half + 4 * v] = ch[v].x; qr[16 * half + 4 * v + 1] = ch[v].y;
          qr[16 * half + 4 * v + 2] = ch[v].z; qr[16 * half + 4 * v + 3] = ch[v].w;
        }
      }
      tmem_st32(tmem_lane + kColQ + g * 32, qr);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(qt_full);
    }
    constexpr int NL = kDqCols / 32;
    // One key tile; `valid` = valid keys of this group's share (may be <= 0).  Full tiles pass the constant
    // kDqCols, which leaves nothing about key validity in their code.
    auto tile = [&](int j, int valid) {
      mbar_wait(s_full, j & 1, abort_flag);
      tc_fence_after_sync();
      uint32_t s[NL][32];
#pragma unroll
      for (int c2 = 0; c2 < NL; ++c2) tmem_ld32(tmem_lane + kColS + g * kDqCols + c2 * 32, s[c2]);
      tmem_wait_ld();
      tc_fence_before_sync();
      mbar_arrive(rs + j % 4);
      // P = exp2(s * scale * log2e - LSE * log2e), kept as packed fp32 pairs
      uint64_t p2[NL][16];
#pragma unroll
      for (int c2 = 0; c2 < NL; ++c2)
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const uint64_t x2 = fma2(f32x2(__uint_as_float(s[c2][c]), __uint_as_float(s[c2][c + 1])), sc2, nl2);
          float p0, p1;
          if (((c >> 1) & 7) < kDqPolyOf8) {
            exp2_poly_pair(x2, p0, p1);
          } else {
            float x0, x1;
            f32x2_split(x2, x0, x1);
            p0 = fast_exp2(x0);
            p1 = fast_exp2(x1);
          }
          p2[c2][c >> 1] = f32x2(p0, p1);
        }
      // commit j+1 of b_done: dP(j) is there, and dQ(j-1) has consumed the one dS buffer
      mbar_wait(b_done + ((j + 1) & 1), (j >> 1) & 1, abort_flag);
      tc_fence_after_sync();
      uint32_t dp[NL][32], ds[NL][16];
#pragma unroll
      for (int c2 = 0; c2 < NL; ++c2) tmem_ld32(tmem_lane + kColdP + g * kDqCols + c2 * 32, dp[c2]);
      tmem_wait_ld();
      if (valid >= kDqCols) {   // the usual tile: no key to mask, nothing but the algebra in the loop
#pragma unroll
        for (int c2 = 0; c2 < NL; ++c2)
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const uint64_t d2 = mul2(p2[c2][c >> 1],
                                     add2(f32x2(__uint_as_float(dp[c2][c]), __uint_as_float(dp[c2][c + 1])), nd2));
            float d0, d1;
            f32x2_split(d2, d0, d1);
            ds[c2][c >> 1] = pack_bf16(d0, d1);
          }
      } else {                  // keys past the segment's end: S and dP hold anything, dS must be 0
#pragma unroll
        for (int c2 = 0; c2 < NL; ++c2)
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const uint64_t d2 = mul2(p2[c2][c >> 1],
                                     add2(f32x2(__uint_as_float(dp[c2][c]), __uint_as_float(dp[c2][c + 1])), nd2));
            float d0, d1;
            f32x2_split(d2, d0, d1);
            if (c2 * 32 + c >= valid) d0 = 0.f;
            if (c2 * 32 + c + 1 >= valid) d1 = 0.f;
            ds[c2][c >> 1] = pack_bf16(d0, d1);
          }
      }
#pragma unroll
      for (int c2 = 0; c2 < NL; ++c2)
        tmem_st16(tmem_lane + kColdS + g * (kDqCols / 2) + c2 * 16, ds[c2]);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(rb + j % 4);   // dS(j) stored; dP(j) was read before it, so its buffer is free as well
    };
    // key ranges one after the other: their full tiles in a loop of their own, then the ragged last tile if any
    int j = 0;
    for (int sg = 0; sg < segs.n; ++sg) {
      const int full = segs.count[sg] / kTile, rest = segs.count[sg] % kTile;
      for (int t = 0; t < full; ++t, ++j) tile(j, kDqCols);
      if (rest) { tile(j, rest - kDqCols * g); ++j; }
    }
    // ---- epilogue: groups 0 and 1 write columns [g D/2, (g+1) D/2) of dQ
    mbar_wait(dq_full, 0, abort_flag);
    tc_fence_after_sync();
    if (g < 2)
      store_rows_from_tmem<D / 2>(tmem_lane + kColdQ + g * (D / 2), scale, quad_rows(dq, b, h, n_q, heads, D, row),
                                  g * (D / 2), tid & 31);
  }

  settle_after_abort(abort_flag);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------------------------------ dK, dV
// Warp-specialised, one CTA (one 128-key tile of the chunk) per SM; K and V of the tile stay in shared
// memory and the query tiles stream through a 2-deep ring of (Q, dO) pairs:
//   warps 0-3  group 0: queries  0..63 of every query tile (one key row per thread)
//   warps 4-7  group 1: queries 64..127
//   warp  8    MMA issuer                                       warp  9    TMA producer
// Per query tile i: S^T = K Q^T and dP^T = V dO^T are full 128x128 MMAs (keys x queries).  A thread turns its
// 64 S^T values into P^T (bf16 pairs written over its own S^T columns) -> dV += P^T dO and S^T(i+1) follow;
// then dP^T into dS^T = P^T o (dP^T - delta) in place -> dK += dS^T Q and dP^T(i+1) follow.
//   TMEM columns: S^T / P^T [0,128)  dP^T / dS^T [128,256)  dK [256,256+D)  dV [384,384+D)
constexpr int kDkvStages = 2;
constexpr int kDkvThreads = 320;
constexpr int kDkvPolyOf8 = 2;

template <int D> struct DkvSmem {
  static constexpr int kK = 0;
  static constexpr int kV = TileGeom<D>::kBytes;
  static constexpr int kQ = 2 * TileGeom<D>::kBytes;                      // [kDkvStages]
  static constexpr int kdO = kQ + kDkvStages * TileGeom<D>::kBytes;       // [kDkvStages]
  static constexpr int kStats = kdO + kDkvStages * TileGeom<D>::kBytes;   // float [stages][2][128]: -lse*log2e, -delta
  static constexpr int kBars = kStats + 2 * kTile * 8;
  static constexpr int kTotal = kBars + 256 + 1024;
};

template <int D>
__global__ void __launch_bounds__(kDkvThreads, 1)
chunk_attn_bwd_dkv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
                          const __grid_constant__ CUtensorMap tm_kc, const __grid_constant__ CUtensorMap tm_vc,
                          const int n_q, const int n_kc, const int heads, const float scale,
                          const float* __restrict__ lse, const float* __restrict__ delta,
                          __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sK = smem + DkvSmem<D>::kK;
  uint8_t* sV = smem + DkvSmem<D>::kV;
  uint8_t* sQ = smem + DkvSmem<D>::kQ;
  uint8_t* sdO = smem + DkvSmem<D>::kdO;
  float* sStat = reinterpret_cast<float*>(smem + DkvSmem<D>::kStats);   // [stage][-LSE*log2e | -delta][128 queries]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + DkvSmem<D>::kBars);
  uint64_t* kv_full = bars;
  uint64_t* q_full = bars + 1;                 // [kDkvStages]
  uint64_t* q_empty = q_full + kDkvStages;
  uint64_t* s_full = q_empty + kDkvStages;
  uint64_t* dp_full = s_full + 1;
  uint64_t* p_full = dp_full + 1;              // 256 arrivals
  uint64_t* ds_full = p_full + 1;              // 256 arrivals
  uint64_t* acc_full = ds_full + 1;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k0 = blockIdx.x * kTile, h = blockIdx.y, b = blockIdx.z;
  constexpr uint32_t kTmemCols = 512;
  constexpr uint32_t kColSt = 0, kColdPt = 128, kColdK = 256, kColdV = 384;
  constexpr int kMmaWarp = 8, kTmaWarp = 9;
  constexpr int kHalfBytes = 64 * 128;
  const int n_tiles = (n_q + kTile - 1) / kTile;

  if (tid == 0) {
    mbar_init(kv_full, 1);
    // a (Q, dO) stage is full when its TMA bytes have landed and the producer warp has staged the per-query
    // constants of the tile beside it: two arrivals
    for (int i = 0; i < kDkvStages; ++i) { mbar_init(q_full + i, 2); mbar_init(q_empty + i, 1); }
    mbar_init(s_full, 1);
    mbar_init(dp_full, 1);
    mbar_init(p_full, 256);
    mbar_init(ds_full, 256);
    mbar_init(acc_full, 1);
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
    // the whole warp: lane 0 issues the TMA loads, every lane stages the (LSE * log2e, delta) pairs of four
    // queries of the tile; +inf as LSE turns query rows past n_q into P = 0
    const size_t stat_base = (static_cast<size_t>(b) * heads + h) * n_q;
    if (lane == 0) {
      mbar_arrive_expect_tx(kv_full, 2 * TileGeom<D>::kBytes);
      tma_load_tile<D>(sK, &tm_kc, kv_full, k0, h, b);
      tma_load_tile<D>(sV, &tm_vc, kv_full, k0, h, b);
    }
    for (int i = 0; i < n_tiles; ++i) {
      const int st = i % kDkvStages;
      const bool go = mbar_wait(q_empty + st, ((i / kDkvStages) & 1) ^ 1, abort_flag);
      if (lane == 0 && go) {   // no copies once a wait has run out
        mbar_arrive_expect_tx(q_full + st, 2 * TileGeom<D>::kBytes);
        tma_load_tile<D>(sQ + st * TileGeom<D>::kBytes, &tm_q, q_full + st, i * kTile, h, b);
        tma_load_tile<D>(sdO + st * TileGeom<D>::kBytes, &tm_do, q_full + st, i * kTile, h, b);
      }
      float* stat = sStat + st * 2 * kTile;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int qi = i * kTile + lane * 4 + e;
        // negated once here, so that the consumers' loops add them as they come; +inf as LSE turns rows past n_q into P = 0
        stat[lane * 4 + e] = qi < n_q ? -lse[stat_base + qi] * kLog2e : -INFINITY;
        stat[kTile + lane * 4 + e] = qi < n_q ? -delta[stat_base + qi] : 0.f;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(q_full + st);
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      auto q_tile = [&](int i) { return smem_u32(sQ + (i % kDkvStages) * TileGeom<D>::kBytes); };
      auto do_tile = [&](int i) { return smem_u32(sdO + (i % kDkvStages) * TileGeom<D>::kBytes); };
      auto wait_q = [&](int i) {
        mbar_wait_spin(q_full + i % kDkvStages, (i / kDkvStages) & 1, abort_flag);
        tc_fence_after_sync();
      };
      mbar_wait_spin(kv_full, 0, abort_flag);
      wait_q(0);
      mma_abT<D>(tmem_base + kColSt, smem_u32(sK), q_tile(0));
      mma_commit(s_full);
      mma_abT<D>(tmem_base + kColdPt, smem_u32(sV), do_tile(0));
      mma_commit(dp_full);
      for (int i = 0; i < n_tiles; ++i) {
        mbar_wait_spin(p_full, i & 1, abort_flag);
        tc_fence_after_sync();
        mma_pb<D, 64>(tmem_base + kColdV, tmem_base + kColSt, do_tile(i), i > 0);
        mma_pb<D, 64>(tmem_base + kColdV, tmem_base + kColSt + 64, do_tile(i) + kHalfBytes, true);
        if (i + 1 < n_tiles) {  // overwrites P^T(i) after the dV MMAs that read it (MMAs run in order)
          wait_q(i + 1);
          mma_abT<D>(tmem_base + kColSt, smem_u32(sK), q_tile(i + 1));
          mma_commit(s_full);
        }
        mbar_wait_spin(ds_full, i & 1, abort_flag);
        tc_fence_after_sync();
        mma_pb<D, 64>(tmem_base + kColdK, tmem_base + kColdPt, q_tile(i), i > 0);
        mma_pb<D, 64>(tmem_base + kColdK, tmem_base + kColdPt + 64, q_tile(i) + kHalfBytes, true);
        mma_commit(q_empty + i % kDkvStages);
        if (i + 1 < n_tiles) {
          mma_abT<D>(tmem_base + kColdPt, smem_u32(sV), do_tile(i + 1));
          mma_commit(dp_full);
        }
      }
      mma_commit(acc_full);
    }
  } else {
    const int g = warp >> 2;
    const int r = tid & 127;  // key row inside the tile = TMEM lane
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const float scale_log2 = scale * kLog2e;
    const uint64_t sc2 = f32x2(scale_log2, scale_log2);
    for (int i = 0; i < n_tiles; ++i) {
      // per-query constants of this group's 64 queries, staged by the producer warp with the tile
      const float* stat = sStat + (i % kDkvStages) * 2 * kTile + g * 64;
      mbar_wait(q_full + i % kDkvStages, (i / kDkvStages) & 1, abort_flag);
      mbar_wait(s_full, i & 1, abort_flag);
      tc_fence_after_sync();
      uint32_t s[2][32], pt[32];
      tmem_ld32(tmem_lane + kColSt + g * 64, s[0]);
      tmem_ld32(tmem_lane + kColSt + g * 64 + 32, s[1]);
      tmem_wait_ld();
      uint64_t p2[2][16];
#pragma unroll
      for (int c2 = 0; c2 < 2; ++c2)
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const uint64_t nl2 = *reinterpret_cast<const uint64_t*>(stat + c2 * 32 + c);   // -LSE*log2e of 2 queries
          const uint64_t x2 = fma2(f32x2(__uint_as_float(s[c2][c]), __uint_as_float(s[c2][c + 1])), sc2, nl2);
          float p0, p1;
          if (((c >> 1) & 7) < kDkvPolyOf8) {
            exp2_poly_pair(x2, p0, p1);
          } else {
            float x0, x1;
            f32x2_split(x2, x0, x1);
            p0 = fast_exp2(x0);
            p1 = fast_exp2(x1);
          }
          p2[c2][c >> 1] = f32x2(p0, p1);
          pt[c2 * 16 + (c >> 1)] = pack_bf16(p0, p1);
        }
      // in place: every S^T column this thread owns is already in registers
      tmem_st32(tmem_lane + kColSt + g * 64, pt);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(p_full);

      mbar_wait(dp_full, i & 1, abort_flag);
      tc_fence_after_sync();
#pragma unroll
      for (int c2 = 0; c2 < 2; ++c2) {
        uint32_t dp[32], ds[16];
        tmem_ld32(tmem_lane + kColdPt + g * 64 + c2 * 32, dp);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const uint64_t nd2 = *reinterpret_cast<const uint64_t*>(stat + kTile + c2 * 32 + c);   // -delta of 2 queries
          const uint64_t d2 = mul2(p2[c2][c >> 1], add2(f32x2(__uint_as_float(dp[c]), __uint_as_float(dp[c + 1])), nd2));
          float d0, d1;
          f32x2_split(d2, d0, d1);
          ds[c >> 1] = pack_bf16(d0, d1);
        }
        tmem_st16(tmem_lane + kColdPt + g * 64 + c2 * 16, ds);
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(ds_full);
    }
    mbar_wait(acc_full, 0, abort_flag);
    tc_fence_after_sync();
    const int krow = k0 + r;
    store_rows_from_tmem<D / 2>(tmem_lane + kColdK + g * (D / 2), scale, quad_rows(dk, b, h, n_kc, heads, D, krow),
                                g * (D / 2), tid & 31);
    store_rows_from_tmem<D / 2>(tmem_lane + kColdV + g * (D / 2), 1.f, quad_rows(dv, b, h, n_kc, heads, D, krow),
                                g * (D / 2), tid & 31);
  }

  settle_after_abort(abort_flag);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace astro
