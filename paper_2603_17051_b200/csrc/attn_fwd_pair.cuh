// Forward of chunk attention on CTA pairs (head_dim 128): two 128-query tiles of one (sample, head) share every
// K and V tile.  The two CTAs of a cluster each keep their own Q (tensor memory), S, P and O for 128 query rows
// and load only HALF of every key tile -- the CTA of rank r takes keys [64 r, 64 r + 64) of K (the B operand of
// S = Q K^T, split along N) and head-dim columns [64 r, 64 r + 64) of V (the B operand of O += P V, split along N)
// -- with plain tiled TMA loads into its own shared memory; one tcgen05.mma.cta_group::2 with M = 256 then reads
// both halves.  Per flop this halves the shared-memory fill, the L2 -> SM traffic and the shared-memory reads of
// B.  This is the work unit for a group of candidates decoding against one prefix as well: the tiles of a pair
// belong to one sample, and the samples of a head are launched next to each other so that L2 serves the prefix.
//
// Structure per CTA as in the single-CTA kernel's fast pass (two softmax groups, one row reference per row, P in
// place over S, S two tiles ahead); only the leader's MMA thread issues, its commits arrive in both CTAs, and
// the softmax threads of both CTAs arrive on the leader's barriers.  Key ranges of the cache get tensor maps that
// end where the range ends, so rows past a range's end are zero-filled by TMA and never stale.
// A row whose sums leave the range fp32 can hold sets `*needs_safe`; the host then repeats the call with the
// single-CTA kernel's safe pass.
#pragma once
#include "attn_fwd.cuh"

namespace astro {

constexpr int kPairStages = 4;
constexpr int kPairGroups = 2;                       // softmax groups per CTA: 64 keys of a tile each
constexpr int kPairCols = kTile / kPairGroups;
constexpr int kPairThreads = 128 * kPairGroups + 64;
constexpr int kPairHalfBytes = 64 * 128 * 2;   // 64 keys x 128 d of K (2 blocks of 64 rows), or 128 keys x 64 d of V

struct PairSmem {
  static constexpr int kK = 0;
  static constexpr int kV = kK + kPairStages * kPairHalfBytes;
  static constexpr int kMax = kV + kPairStages * kPairHalfBytes;   // float [3][groups][128]
  static constexpr int kBars = kMax + 3 * kPairGroups * kTile * 4;
  static constexpr int kTotal = kBars + 32 * 8 + 64 + 1024;
};

// Barriers, at the same offsets in both CTAs.  "leader": only the copy in the CTA of cluster rank 0 is used.
struct PairBars {
  uint64_t *q_full;    // leader: Q of both CTAs is in tensor memory (512 arrivals)
  uint64_t *k_full;    // leader [stage]: both halves of a K tile have landed (1 arrival + bytes of both CTAs)
  uint64_t *v_full;    // leader [stage]
  uint64_t *k_empty;   // each CTA [stage]: the MMAs that read the stage are done (commit arrives in both CTAs)
  uint64_t *v_empty;   // each CTA [stage]
  uint64_t *s_full;    // each CTA [S buffer]
  uint64_t *p_full;    // leader [S buffer]: P of both CTAs is in tensor memory (one arrival per softmax warp: 16)
  uint64_t *o_full;    // each CTA
  __device__ explicit PairBars(uint64_t* b)
      : q_full(b), k_full(b + 1), v_full(k_full + kPairStages), k_empty(v_full + kPairStages),
        v_empty(k_empty + kPairStages), s_full(v_empty + kPairStages), p_full(s_full + kFwdSBufs),
        o_full(p_full + kFwdSBufs) {}
  __device__ void init() const {
    mbar_init(q_full, 2 * 128 * kPairGroups);
    for (int i = 0; i < kPairStages; ++i) {
      mbar_init(k_full + i, 1); mbar_init(v_full + i, 1); mbar_init(k_empty + i, 1); mbar_init(v_empty + i, 1);
    }
    for (int i = 0; i < kFwdSBufs; ++i) { mbar_init(s_full + i, 1); mbar_init(p_full + i, 2 * 4 * kPairGroups); }
    mbar_init(o_full, 1);
  }
};

struct PairMaps {
  CUtensorMap kc, vc;        // chunk K (box 64 d x 64 tokens) and V (box 64 d x 128 tokens)
  CUtensorMap kx[2], vx[2];  // the cache key ranges, each map ending where its range ends
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
chunk_attn_fwd_pair_kernel(const __nv_bfloat16* __restrict__ q, const __grid_constant__ PairMaps maps,
                           const __grid_constant__ KeySegs segs, const int n_q, const int heads, const int cache_shared,
                           const float scale_log2, __nv_bfloat16* __restrict__ o, float* __restrict__ lse,
                           int* __restrict__ needs_safe) {
  constexpr int D = 128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint8_t* sK = smem + PairSmem::kK;
  uint8_t* sV = smem + PairSmem::kV;
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(smem + PairSmem::kBars);
  const PairBars bar(bar_mem);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_mem + 32);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();            // 0: leader
  const int q0 = blockIdx.x * kTile;                   // the pair covers query tiles 2i and 2i+1
  const int h = cache_shared ? blockIdx.z : blockIdx.y, b = cache_shared ? blockIdx.y : blockIdx.z;
  const int bx = cache_shared ? 0 : b;
  constexpr uint32_t kTmemCols = 512;
  constexpr int kMmaWarp = 4 * kPairGroups, kTmaWarp = 4 * kPairGroups + 1;
  const int n_tiles = seg_tiles(segs);

  if (tid == 0) {
    bar.init();
    *abort_flag = 0;
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (warp == kMmaWarp) {          // one warp of each CTA: the allocation is made for the pair
    tmem_alloc_pair(tmem_holder, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();              // both CTAs' barriers exist before anything arrives on them from the peer
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == kTmaWarp) {
    // ------------------------------------------------------------------ TMA producer: this CTA's halves
    if (lane == 0) {
      KeyTileIter itk, itv;
      auto load_k = [&](int j) {
        const int st = j % kPairStages;
        const bool fc = itk.from_chunk(segs);
        mbar_wait_spin(bar.k_empty + st, ((j / kPairStages) & 1) ^ 1, abort_flag);
        if (rank == 0) mbar_arrive_expect_tx(bar.k_full + st, 2 * kPairHalfBytes);
        const uint32_t full = cluster_map(smem_u32(bar.k_full + st), 0);
        const CUtensorMap* tm = fc ? &maps.kc : &maps.kx[itk.seg];   // cache ranges come first in the list
        uint8_t* dst = sK + st * kPairHalfBytes;
        const int row = itk.row0(segs) + 64 * static_cast<int>(rank);
        tma_load_4d_pair(dst, tm, full, 0, row, h, fc ? b : bx);
        tma_load_4d_pair(dst + 64 * 128, tm, full, 64, row, h, fc ? b : bx);
        itk.next(segs);
      };
      auto load_v = [&](int j) {
        const int st = j % kPairStages;
        const bool fc = itv.from_chunk(segs);
        mbar_wait_spin(bar.v_empty + st, ((j / kPairStages) & 1) ^ 1, abort_flag);
        if (rank == 0) mbar_arrive_expect_tx(bar.v_full + st, 2 * kPairHalfBytes);
        const uint32_t full = cluster_map(smem_u32(bar.v_full + st), 0);
        const CUtensorMap* tm = fc ? &maps.vc : &maps.vx[itv.seg];
        tma_load_4d_pair(sV + st * kPairHalfBytes, tm, full, 64 * static_cast<int>(rank), itv.row0(segs), h,
                         fc ? b : bx);
        itv.next(segs);
      };
      for (int j = 0; j < kFwdSBufs && j < n_tiles; ++j) load_k(j);
      for (int j = 0; j < n_tiles; ++j) {
        if (*abort_flag) break;
        load_v(j);
        if (j + kFwdSBufs < n_tiles) load_k(j + kFwdSBufs);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer: the leader's first thread
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc_s = make_idesc_bf16(2 * kTile, kTile, false, false);
      constexpr uint32_t idesc_pv = make_idesc_bf16(2 * kTile, D, false, true);
      const uint64_t k_desc0 = desc_kmajor(smem_u32(sK));
      auto issue_s = [&](int j) {
        const uint64_t k_desc = desc_step(k_desc0, (j % kPairStages) * kPairHalfBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          mma_ts_pair(tmem_base + kFwdColS + (j % kFwdSBufs) * 128, tmem_base + kFwdColQ + k * 8,
                      desc_step(k_desc, (k >> 2) * (64 * 128) + (k & 3) * 32), idesc_s, k > 0);
      };
      mbar_wait_spin_cluster(bar.q_full, 0, abort_flag);
      for (int j = 0; j < kFwdSBufs && j < n_tiles; ++j) {
        mbar_wait_spin(bar.k_full + j % kPairStages, (j / kPairStages) & 1, abort_flag);
        tc_fence_after_sync();
        issue_s(j);
        mma_commit_pair(bar.k_empty + j % kPairStages);
        mma_commit_pair(bar.s_full + j % kFwdSBufs);
      }
      for (int j = 0; j < n_tiles; ++j) {
        const int st = j % kPairStages, buf = j % kFwdSBufs, jn = j + kFwdSBufs;
        const bool more = jn < n_tiles;
        const uint32_t pcol = tmem_base + kFwdColS + buf * 128;
        const uint64_t v_desc = desc_mnmajor(smem_u32(sV + st * kPairHalfBytes), kPairHalfBytes);
        mbar_wait_spin(bar.v_full + st, (j / kPairStages) & 1, abort_flag);
        if (more) mbar_wait_spin(bar.k_full + jn % kPairStages, (jn / kPairStages) & 1, abort_flag);
        mbar_wait_spin_cluster(bar.p_full + buf, (j / kFwdSBufs) & 1, abort_flag);
        tc_fence_after_sync();
#pragma unroll
        for (int kb = 0; kb < kTile / 16; ++kb) {
          const uint32_t a = pcol + (kb * 16 / kPairCols) * kPairCols + (kb * 16 % kPairCols) / 2;
          mma_ts_pair(tmem_base + kFwdColO, a, desc_step(v_desc, kb * 2048), idesc_pv, (j > 0 || kb > 0) ? 1u : 0u);
        }
        if (more) issue_s(jn);
        mma_commit_pair(bar.v_empty + st);
        if (more) {
          mma_commit_pair(bar.k_empty + jn % kPairStages);
          mma_commit_pair(bar.s_full + buf);
        }
      }
      mma_commit_pair(bar.o_full);
    }
  } else {
    // ------------------------------------------------------------------ softmax groups (both CTAs)
    const int g = warp >> 2;
    const int r = tid & 127;
    const uint32_t tmem_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const int row = q0 + r;
    const bool in_range = row < n_q;
    float* smax = reinterpret_cast<float*>(smem + PairSmem::kMax);
    {   // Q row -> tensor memory: group g writes elements [64 g, 64 g + 64) as 32 packed columns
      uint32_t qr[32];
      const uint4* src = reinterpret_cast<const uint4*>(q + ((static_cast<size_t>(b) * n_q + (in_range ? row : 0)) * heads + h) * D + g * 64);
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        const uint4 t = in_range ? src[v] : make_uint4(0, 0, 0, 0);
        qr[4 * v] = t.x; qr[4 * v + 1] = t.y; qr[4 * v + 2] = t.z; qr[4 * v + 3] = t.w;
      }
      tmem_st32(tmem_lane + kFwdColQ + g * 32, qr);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive_cluster(cluster_map(smem_u32(bar.q_full), 0));
    }
    const uint32_t p_full0 = cluster_map(smem_u32(bar.p_full), 0);
    float m_ref = 0.f, l_run = 0.f, poly_max = -INFINITY;
    int j = 0;
    for (KeyTileIter it; !it.done(segs); it.next(segs), ++j) {
      const int valid = it.valid(segs) - kPairCols * g;
      const int buf = j % kFwdSBufs;
      const uint32_t colS = kFwdColS + buf * 128 + g * kPairCols;
      mbar_wait(bar.s_full + buf, (j / kFwdSBufs) & 1, abort_flag);
      tc_fence_after_sync();
      uint32_t s[2][32];
      tmem_ld32(tmem_lane + colS, s[0]);
      tmem_ld32(tmem_lane + colS + 32, s[1]);
      tmem_wait_ld();
      if (j == 0) {
        float mx = -INFINITY;
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2)
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c2 * 32 + c < valid) mx = fmaxf(mx, __uint_as_float(s[c2][c]));
        float* mslot = smax + 2 * kPairGroups * kTile;
        mslot[g * kTile + r] = mx;
        named_barrier_sync(1 + (warp & 3), 32 * kPairGroups);
        mx = fmaxf(mx, mslot[(g ^ 1) * kTile + r]);
        m_ref = mx * scale_log2;
      }
      const float neg_m = -m_ref;
      uint32_t pk[2][16];
#pragma unroll
      for (int half = 0; half < 2; ++half)
        l_run += fwd_exp32(s[half], valid - 32 * half, scale_log2, neg_m, pk[half], poly_max);
      tmem_st16(tmem_lane + colS, pk[0]);
      tmem_st16(tmem_lane + colS + 16, pk[1]);
      tmem_wait_st();
      tc_fence_before_sync();
      __syncwarp();                  // one arrival per warp: an arrival in the peer CTA's shared memory is not cheap
      if (lane == 0) mbar_arrive_cluster(p_full0 + 8 * buf);
    }
    bool ok = (l_run < kFastSumLimit) && !(poly_max > kPolyArgLimit);
    FwdUnit<D> u;
    u.smax = smax;
    u.abort_flag = abort_flag;
    const QuadRows out = quad_rows(o, b, h, n_q, heads, D, row);
    float* lse_dst = lse ? lse + (static_cast<size_t>(b) * heads + h) * n_q + (in_range ? row : 0) : nullptr;
    ok = fwd_epilogue<D, kPairGroups>(u, bar.o_full, 0, nullptr, u.smax, g, r, tmem_lane, m_ref, l_run, out, in_range, lse_dst) && ok;
    if (!ok) *needs_safe = 1;
  }

  settle_after_abort(abort_flag);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();              // the peer may still read this CTA's shared memory and arrive on its barriers
  if (warp == kMmaWarp) tmem_dealloc_pair(tmem_base, kTmemCols);
}

}  // namespace astro
