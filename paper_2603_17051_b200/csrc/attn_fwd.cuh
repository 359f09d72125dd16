// Forward of chunk attention over the rolling cache: O and LSE.  A work unit is one 128-query tile of one head of
// one sample; one CTA per SM walks over its share of the units.
//
// Warp-specialised:
//   four softmax groups of 4 warps: group g owns keys [32 g, 32 g + 32) of every key tile, one query row
//   per thread (four warps per scheduler: while one waits for tensor memory or a barrier the others keep the
//   special-function unit busy); then one warp whose first thread issues every tcgen05 MMA, one for TMA loads, and
//   (fast pass) eight epilogue warps that write O and LSE out and bring the Q rows of the units to come in.
// Q lives in tensor memory (bf16 pairs, two buffers: the unit at hand and the next) and is the A operand of
// S = Q K^T, so shared memory only carries K and V: an MMA with both operands in shared memory reads
// 128 B/clk, the whole shared-memory bandwidth, and then competes with the TMA writes of the next tiles.
// S of a whole key tile is one 128x128 MMA into one of two S buffers, issued two tiles ahead.  P is written
// as bf16 pairs over the thread's own S columns and feeds P V from tensor memory.  K and V tiles travel
// through 3-deep rings.  A share of the exponentials can be evaluated by a polynomial on the FMA pipe instead of
// the special-function unit (16 exp2 per clock per SM, as busy as the tensor core at head_dim 128); measured, the
// polynomial's own FMA and integer work costs more than it saves, so the share is zero.
//
// The kernel makes up to two passes:
//   fast pass  over all the CTA's units.  Every row keeps ONE reference exponent, the maximum of its first key
//              tile.  exp2(s - m) is exact for any reference as long as nothing overflows (bf16 and fp32 share the
//              exponent range, so later scores may exceed the reference by ~100 in log2 units), so O is never
//              rescaled and the threads of a row never have to agree on anything after the first tile.  The
//              MMA-issuing thread sets the pace, so everything a tile needs (the bytes of V(J) and K(J+2), every
//              thread's P(J)) arrives on ONE barrier and every burst of 16 MMAs (P V of tile J, S of tile J+2) is
//              followed by ONE commit.  The key tiles of all the CTA's units form one stream: look-ahead, rings
//              and barriers run on across unit boundaries, where the softmax threads only leave their row sums
//              and references in shared memory; the epilogue warps do everything else there (O out of tensor
//              memory, normalised, stored; LSE; the Q rows of the unit after the next into the free Q buffer).
//   safe pass  unit by unit, only for units one of whose rows saw a sum beyond 2^100, an infinity or a NaN in the
//              fast pass: the unit is recomputed with a running reference that follows the row maximum (rescaling
//              O and the row sums when a tile's row sum leaves the safe range).
//   TMEM columns: S buffers [0,128) [128,256)   O [256,256+D)   Q buffers [384,384+D/2) [448,448+D/2)
#pragma once
#include <type_traits>

#include "attn_common.cuh"

namespace astro {

constexpr int kFwdKStages = 3, kFwdVStages = 3, kFwdSBufs = 2;
constexpr int kFwdGroups = 4;                    // layer shape, forward alone: 2 groups 0.741 ms, 4 groups 0.713 ms
constexpr int kFwdCols = kTile / kFwdGroups;     // keys per group and tile
constexpr int kFwdEpiWarps = 8;                  // fast pass: warps that write O and LSE out and stage Q
constexpr int kFwdThreads = 128 * kFwdGroups + 64 + 32 * kFwdEpiWarps;
constexpr int kFwdBarSlots = 32;                 // mbarriers of one pass
constexpr int kFwdMaxUnits = 1024;               // work units one CTA may walk (one redo bit each)

template <int D> struct FwdSmem {
  static constexpr int kK = 0;
  static constexpr int kV = kK + kFwdKStages * TileGeom<D>::kBytes;
  static constexpr int kMax = kV + kFwdVStages * TileGeom<D>::kBytes;  // float [4][groups][128] + [2][128]: exchange slots
  static constexpr int kBars = kMax + (4 * kFwdGroups + 2) * kTile * 4;  // two sets of barriers, 3 words, redo bits
  static constexpr int kTotal = kBars + 2 * kFwdBarSlots * 8 + 64 + kFwdMaxUnits / 8 + 1024;  // + slack to align to 1024
};

// Of every 8 pairs of exponentials, how many use the polynomial on the FMA pipe.  Layer shape, forward alone:
// 0 -> 0.776 ms, 1 -> 0.781, 2 -> 0.802, 3 -> 0.828 in bursts; the same order under the power limit.  The same
// again with four softmax groups and the CTAs walking over their units: 0 -> 0.662 ms, 1 -> 0.689, 2 -> 0.719.
constexpr int kPolyOf8 = 0;
constexpr float kRowSumLimit = 1073741824.f;        // safe pass: a tile row sum beyond 2^30 re-references the row
constexpr float kFastSumLimit = 1.2676506e30f;      // fast pass: a row sum beyond 2^100 sends the unit to the safe pass
constexpr float kPolyArgLimit = 126.f;              // largest exponent the polynomial exp2 may be handed

// The mbarriers of the safe pass.  The two passes use separate sets, so a late arrival of the first pass can
// never land in a phase of the second.
struct FwdBars {
  uint64_t *q_full, *k_full, *k_empty, *v_full, *v_empty, *s_full, *p_full, *pv_done, *o_full;
  __device__ explicit FwdBars(uint64_t* b)
      : q_full(b), k_full(b + 1), k_empty(k_full + kFwdKStages), v_full(k_empty + kFwdKStages),
        v_empty(v_full + kFwdVStages), s_full(v_empty + kFwdVStages), p_full(s_full + kFwdSBufs),
        pv_done(p_full + kFwdGroups * kFwdSBufs), o_full(pv_done + 2) {}
  // p_full [group][S buffer], 128 arrivals each: the groups may run up to two tiles ahead of the MMA thread, so
  // the barriers rotate with the S buffers.
  __device__ void init(int q_count, int p_count) const {
    mbar_init(q_full, q_count);
    for (int i = 0; i < kFwdKStages; ++i) { mbar_init(k_full + i, 1); mbar_init(k_empty + i, 1); }
    for (int i = 0; i < kFwdVStages; ++i) { mbar_init(v_full + i, 1); mbar_init(v_empty + i, 1); }
    for (int i = 0; i < kFwdSBufs; ++i) mbar_init(s_full + i, 1);
    for (int i = 0; i < kFwdGroups * kFwdSBufs; ++i) mbar_init(p_full + i, p_count);
    mbar_init(pv_done, 1);
    mbar_init(pv_done + 1, 1);
    mbar_init(o_full, 1);
  }
  // Fresh phases for another run of the pass; every thread of the CTA is past its last use of the barriers.
  __device__ void rearm(int q_count, int p_count) const {
    for (uint64_t* b = q_full; b <= o_full; ++b) mbar_inval(b);
    init(q_count, p_count);
  }
};

// What every role of the CTA needs to know about its work unit.
template <int D> struct FwdUnit {
  const CUtensorMap *tm_kc, *tm_vc, *tm_kx;
  const CUtensorMap *tm_vx0, *tm_vx1;   // one per cache key range, each ending where its range ends (rows past it read as 0)
  __device__ const CUtensorMap* vx(int seg) const { return seg == 0 ? tm_vx0 : tm_vx1; }
  const KeySegs* segs;
  uint8_t *sK, *sV;
  float* smax;
  volatile int* abort_flag;
  uint32_t tmem_base;
  int n_tiles, h, b, bx;
};

constexpr uint32_t kFwdColS = 0 /* + 128 * buffer */, kFwdColO = 256, kFwdColQ = 384 /* + 64 * buffer */;
constexpr uint32_t kFwdQCols = 64;

// ---------------------------------------------------------------------------------- TMA producer (one thread)
// K runs ahead of V by the S look-ahead: order the loads K0 K1 | V0 K2 | V1 K3 | ...
template <int D>
__device__ __forceinline__ void fwd_produce(const FwdUnit<D>& u, const FwdBars& bar) {
  const KeySegs& segs = *u.segs;
  KeyTileIter itk, itv;
  auto load_k = [&](int j) {
    const int st = j % kFwdKStages;
    const bool fc = itk.from_chunk(segs);
    mbar_wait_spin(bar.k_empty + st, ((j / kFwdKStages) & 1) ^ 1, u.abort_flag);
    mbar_arrive_expect_tx(bar.k_full + st, TileGeom<D>::kBytes);
    tma_load_tile<D>(u.sK + st * TileGeom<D>::kBytes, fc ? u.tm_kc : u.tm_kx, bar.k_full + st, itk.row0(segs), u.h,
                     fc ? u.b : u.bx);
    itk.next(segs);
  };
  auto load_v = [&](int j) {
    const int st = j % kFwdVStages;
    const bool fc = itv.from_chunk(segs);
    mbar_wait_spin(bar.v_empty + st, ((j / kFwdVStages) & 1) ^ 1, u.abort_flag);
    mbar_arrive_expect_tx(bar.v_full + st, TileGeom<D>::kBytes);
    tma_load_tile<D>(u.sV + st * TileGeom<D>::kBytes, fc ? u.tm_vc : u.vx(itv.seg), bar.v_full + st, itv.row0(segs), u.h,
                     fc ? u.b : u.bx);
    itv.next(segs);
  };
  for (int j = 0; j < kFwdSBufs && j < u.n_tiles; ++j) load_k(j);
  for (int j = 0; j < u.n_tiles; ++j) {
    if (*u.abort_flag) break;
    load_v(j);
    if (j + kFwdSBufs < u.n_tiles) load_k(j + kFwdSBufs);
  }
}

// ---------------------------------------------------------------------------------- fast pass: schedule
// A CTA walks over work units (one 128-query tile of one head of one sample each): first, first + stride, ...
// Unit ids count the query tiles fastest, then y, then z, where (y, z) = (head, sample), or (sample, head) when one
// stored prefix serves every sample: then the samples of a head sit next to each other, and the CTAs that run at
// the same time read the same cached K/V, which is fetched from HBM once and served out of L2.
struct FwdSched {
  int first, stride, total, q_tiles, dim_y, cache_shared;
  __device__ int count() const { return (total - first + stride - 1) / stride; }
  __device__ void decode(int unit, int& q_tile, int& h, int& b) const {
    q_tile = unit % q_tiles;
    const int yz = unit / q_tiles, y = yz % dim_y, z = yz / dim_y;
    h = cache_shared ? z : y;
    b = cache_shared ? y : z;
  }
};

// A unit as (query tile, y, z), stepped from one unit of the CTA to the next or the previous one without divisions.
struct FwdPos {
  int qt, y, z;
  int dq, dy, dz;   // the CTA's stride, taken apart the same way
  __device__ FwdPos(const FwdSched& s, int unit) {
    qt = unit % s.q_tiles;
    const int yz = unit / s.q_tiles;
    y = yz % s.dim_y;
    z = yz / s.dim_y;
    dq = s.stride % s.q_tiles;
    const int syz = s.stride / s.q_tiles;
    dy = syz % s.dim_y;
    dz = syz / s.dim_y;
  }
  __device__ void forward(const FwdSched& s) {
    qt += dq;
    int carry = 0;
    if (qt >= s.q_tiles) { qt -= s.q_tiles; carry = 1; }
    y += dy + carry;
    carry = 0;
    if (y >= s.dim_y) { y -= s.dim_y; carry = 1; }
    z += dz + carry;
  }
  __device__ void back(const FwdSched& s) {
    qt -= dq;
    int borrow = 0;
    if (qt < 0) { qt += s.q_tiles; borrow = 1; }
    y -= dy + borrow;
    borrow = 0;
    if (y < 0) { y += s.dim_y; borrow = 1; }
    z -= dz + borrow;
  }
  __device__ int h(const FwdSched& s) const { return s.cache_shared ? z : y; }
  __device__ int b(const FwdSched& s) const { return s.cache_shared ? y : z; }
};

// Position in the CTA's stream of key tiles: the tiles of its first unit, then those of the next, ...
struct FwdCursor {
  KeyTileIter it;
  int unit, h, b, bx;
  __device__ void set(const FwdSched& s) {
    int qt;
    s.decode(unit, qt, h, b);
    bx = s.cache_shared ? 0 : b;
  }
  __device__ void start(const FwdSched& s) { unit = s.first; set(s); }
  __device__ void next(const KeySegs& segs, const FwdSched& s) {
    it.next(segs);
    if (it.done(segs)) {
      it = KeyTileIter();
      unit += s.stride;
      if (unit < s.total) set(s);
    }
  }
};

// ---------------------------------------------------------------------------------- fast pass: barriers
// The MMA-issuing thread is the pace-maker of the kernel, so the fast pass gives it ONE wait and ONE commit per key
// tile, and the key tiles of all the CTA's units form ONE stream (tile J of the stream; S two tiles ahead of P V
// across unit boundaries as well), so the tensor pipe does not drain between units.
// ready[J % 4] collects everything tile J needs: the bytes of V(J) and K(J+2) (the producer's arrive with the
// byte count plus the TMA completions) and the arrival of every softmax thread that has stored its P(J).
// sdone[J % 4] is committed behind S(J): S(J) is ready for the softmax threads, and -- MMAs complete in order --
// the P V of tile J-2 is done too, so the producer may refill the K stage of tile J and the V stage of tile J-2.
// Per unit: q_full[n % 2] (the unit's Q rows are in tensor memory buffer n % 2), stats_full[n % 2] (every softmax
// thread has left its row sum, and the row's reference, in shared memory), o_full (the unit's last P V is done),
// o_free (the epilogue warps have read O out of tensor memory: the next unit's first P V may overwrite it).
// kFwdHalves = 2 splits the hand-offs of a tile in two: keys [0, 64) (softmax groups 0 and 1) and keys [64, 128)
// (groups 2 and 3) get barriers of their own (ready[4 h + J % 4], sdone[4 h + J % 4]) and S(J+2) is issued as two
// groups of N = 64 MMAs, each behind the P V MMAs of its own half, so that a half of S(J+2) is on its way as soon as
// the half of P(J) that shares its columns has been consumed (the bytes of a tile's loads count on the first
// half).  Measured on the layer shape: 0.793 ms against 0.669 ms with whole tiles -- the 16 narrower S MMAs and the
// second wait and commit cost the issuing thread more than the finer hand-off wins -- so tiles stay whole.
constexpr int kFwdHalves = 1;
struct FwdFastBars {
  uint64_t *q_full, *k01, *ready, *sdone, *o_full, *o_free, *stats_full;
  __device__ explicit FwdFastBars(uint64_t* b)
      : q_full(b), k01(b + 2), ready(b + 3), sdone(b + 11), o_full(b + 19), o_free(b + 20), stats_full(b + 21) {}
  __device__ void init(int q_count) const {
    mbar_init(q_full, q_count);
    mbar_init(q_full + 1, q_count);
    mbar_init(k01, 1);
    for (int h = 0; h < kFwdHalves; ++h)
      for (int i = 0; i < 4; ++i) {
        mbar_init(ready + 4 * h + i, (h == 0 ? 1 : 0) + 128 * kFwdGroups / kFwdHalves);
        mbar_init(sdone + 4 * h + i, 1);
      }
    mbar_init(o_full, 1);
    mbar_init(o_free, 32 * kFwdEpiWarps);
    mbar_init(stats_full, 128 * kFwdGroups);
    mbar_init(stats_full + 1, 128 * kFwdGroups);
  }
};

// The loops of the three roles work from local copies of what they need: nothing in them reads `u`, `sch` or `bar`
// again, whatever the compiler decides about where those structures live.
template <int D>
__device__ __forceinline__ void fwd_produce_fast(const FwdUnit<D>& u, const FwdSched& sch_in, const FwdFastBars& bar) {
  const KeySegs& segs = *u.segs;
  const FwdSched sch = sch_in;
  const int total = u.n_tiles * sch.count();
  const CUtensorMap *tm_kc = u.tm_kc, *tm_vc = u.tm_vc, *tm_kx = u.tm_kx, *tm_vx0 = u.tm_vx0, *tm_vx1 = u.tm_vx1;
  uint8_t *sK = u.sK, *sV = u.sV;
  uint64_t *ready = bar.ready, *sdone = bar.sdone;
  volatile int* abort_flag = u.abort_flag;
  FwdCursor ck, cv;   // K runs two tiles ahead of V
  ck.start(sch);
  cv.start(sch);
  auto load_k = [&](int J, uint64_t* full) {
    const bool fc = ck.it.from_chunk(segs);
    tma_load_tile<D>(sK + (J % kFwdKStages) * TileGeom<D>::kBytes, fc ? tm_kc : tm_kx, full, ck.it.row0(segs),
                     ck.h, fc ? ck.b : ck.bx);
    ck.next(segs, sch);
  };
  const int n01 = total < kFwdSBufs ? total : kFwdSBufs;
  mbar_arrive_expect_tx(bar.k01, n01 * TileGeom<D>::kBytes);
  for (int J = 0; J < n01; ++J) load_k(J, bar.k01);
  for (int J = 0; J < total; ++J) {
    // S(J-1) done: the K stage of tile J+2 (that of tile J-1) and the V stage of tile J (that of tile J-3) are free
    if (J >= 1 && !mbar_wait_spin(sdone + 4 * (kFwdHalves - 1) + (J - 1) % 4, ((J - 1) / 4) & 1, abort_flag)) break;
    const bool more = J + kFwdSBufs < total;
    uint64_t* full = ready + J % 4;
    mbar_arrive_expect_tx(full, (more ? 2 : 1) * TileGeom<D>::kBytes);
    const bool fc = cv.it.from_chunk(segs);
    tma_load_tile<D>(sV + (J % kFwdVStages) * TileGeom<D>::kBytes, fc ? tm_vc : (cv.it.seg == 0 ? tm_vx0 : tm_vx1), full,
                     cv.it.row0(segs), cv.h, fc ? cv.b : cv.bx);
    cv.next(segs, sch);
    if (more) load_k(J + kFwdSBufs, full);
  }
}

template <int D>
__device__ __forceinline__ void fwd_issue_fast(const FwdUnit<D>& u, const FwdSched& sch, const FwdFastBars& bar) {
  const uint64_t k_desc0 = desc_kmajor(smem_u32(u.sK));
  const uint32_t sV_addr = smem_u32(u.sV);
  constexpr uint32_t idesc_pv = make_idesc_bf16(kTile, D, false, true);
  const uint32_t tmem_base = u.tmem_base;
  const int T = u.n_tiles, total = T * sch.count();
  uint64_t *q_full = bar.q_full, *ready = bar.ready, *sdone = bar.sdone, *o_full = bar.o_full, *o_free = bar.o_free;
  volatile int* abort_flag = u.abort_flag;
  constexpr int kHalfKeys = kTile / kFwdHalves;
  constexpr uint32_t idesc_sh = make_idesc_bf16(kTile, kHalfKeys, false, false);
  // Half h of S(J) -> columns [h kHalfKeys, +kHalfKeys) of buffer J % 2 (free: the P V MMAs that read the P in those
  // columns, tile J-2's, were issued before), from the Q buffer `qbuf` and rows [h kHalfKeys, +kHalfKeys) of K(J)
  auto issue_s = [&](int J, int qbuf, int h) {
    const uint32_t qcol = tmem_base + kFwdColQ + qbuf * kFwdQCols;
    const uint64_t k_desc = desc_step(k_desc0, (J % kFwdKStages) * TileGeom<D>::kBytes + h * kHalfKeys * 128);
#pragma unroll
    for (int k = 0; k < D / 16; ++k)  // 16 elements of the head dimension = 8 packed Q columns
      mma_ts(tmem_base + kFwdColS + (J % kFwdSBufs) * 128 + h * kHalfKeys, qcol + k * 8,
             desc_step(k_desc, (k >> 2) * TileGeom<D>::kBlockBytes + (k & 3) * 32), idesc_sh, k > 0);
    mma_commit(sdone + 4 * h + J % 4);
  };
  // Half h of P V of tile J; `first`: the unit's first tile, which starts O afresh
  auto issue_pv = [&](int J, bool first, int h) {
    const uint32_t pcol = tmem_base + kFwdColS + (J % kFwdSBufs) * 128;
    const uint64_t v_desc = desc_mnmajor(sV_addr + (J % kFwdVStages) * TileGeom<D>::kBytes, TileGeom<D>::kBlockBytes);
#pragma unroll
    for (int i = 0; i < kHalfKeys / 16; ++i) {
      const int kb = h * (kHalfKeys / 16) + i;
      // P of 16 keys = 8 packed columns; group g's pairs start at its own S columns
      const uint32_t a = pcol + (kb * 16 / kFwdCols) * kFwdCols + (kb * 16 % kFwdCols) / 2;
      mma_ts(tmem_base + kFwdColO, a, desc_step(v_desc, kb * 2048), idesc_pv, (!first || kb > 0) ? 1u : 0u);
    }
  };
  // One tile of the stream: per half, wait for its P (and, with the first half, for the tile's bytes), issue its
  // P V MMAs and the same half of S two tiles ahead.  s_mode 0: no S left to issue; 1: S of a tile inside the unit
  // at hand; 2: S of a tile that may open a unit, whose Q rows must then be in tensor memory.
  int s_n = 0, s_t = 0;        // unit (counted within the CTA) and tile within it of the next S to issue
  auto s_opens_unit = [&]() {
    if (s_t == 0) {
      mbar_wait_spin(q_full + (s_n & 1), (s_n >> 1) & 1, abort_flag);
      tc_fence_after_sync();
    }
  };
  auto s_issued = [&]() { if (++s_t == T) { s_t = 0; ++s_n; } };
  auto tile = [&](int J, int n, bool first, bool last, int s_mode) {
#pragma unroll
    for (int h = 0; h < kFwdHalves; ++h) {
      mbar_wait_spin(ready + 4 * h + J % 4, (J / 4) & 1, abort_flag);
      if (h == 0 && first && n > 0) mbar_wait_spin(o_free, (n - 1) & 1, abort_flag);   // the previous unit's O is out
      tc_fence_after_sync();
      issue_pv(J, first, h);
      if (h == kFwdHalves - 1 && last) mma_commit(o_full);
      if (s_mode != 0) {
        if (s_mode == 2 && h == 0) s_opens_unit();
        issue_s(J + kFwdSBufs, s_mode == 2 ? (s_n & 1) : (n & 1), h);
        if (s_mode == 2 && h == kFwdHalves - 1) s_issued();
      }
    }
  };
  mbar_wait_spin(bar.k01, 0, abort_flag);
  tc_fence_after_sync();
  for (int J = 0; J < kFwdSBufs && J < total; ++J) {
    s_opens_unit();
    for (int h = 0; h < kFwdHalves; ++h) issue_s(J, s_n & 1, h);
    s_issued();
  }
  int J = 0;
  for (int n = 0; J < total; ++n) {
    // first tile of the unit
    tile(J, n, true, T == 1, J + kFwdSBufs < total ? 2 : 0);
    ++J;
    // interior tiles: S two tiles ahead stays inside the unit, nothing to check
    for (int t = 1; t + kFwdSBufs < T; ++t, ++J) tile(J, n, false, false, 1);
    if (T > kFwdSBufs + 1) {   // what the interior loop issued: the unit's tiles 3 .. T-1, which end the unit
      s_t += T - 1 - kFwdSBufs;
      if (s_t >= T) { s_t -= T; ++s_n; }
    }
    // last tiles of the unit (not the first): their S look-ahead belongs to the next unit
    for (int t = (T - kFwdSBufs > 1 ? T - kFwdSBufs : 1); t < T; ++t, ++J)
      tile(J, n, false, t == T - 1, J + kFwdSBufs < total ? 2 : 0);
  }
}

// ---------------------------------------------------------------------------------- MMA issuer (one thread)
// The tensor pipe runs only while this thread keeps handing it MMAs (an issue blocks for about as long as an MMA
// executes, the queue behind it is short), so every clock this thread spends on anything else is an idle clock of
// the pipe.  Per key tile it therefore first makes sure of everything the tile needs (V(j), K(j+2), P(j)), then
// issues P V of tile j and S of tile j+2 as one uninterrupted burst of 16 MMAs, then commits.
// Safe pass: P arrives per group (p_full[group][buffer]); any of the groups may have rescaled its part of O before
// it published, so all of them are awaited first.
template <int D>
__device__ __forceinline__ void fwd_issue(const FwdUnit<D>& u, const FwdBars& bar) {
  const uint64_t k_desc0 = desc_kmajor(smem_u32(u.sK));
  constexpr uint32_t idesc_s = make_idesc_bf16(kTile, kTile, false, false);
  constexpr uint32_t idesc_pv = make_idesc_bf16(kTile, D, false, true);
  const uint32_t tmem_base = u.tmem_base;
  auto wait_k = [&](int j) {
    mbar_wait_spin(bar.k_full + j % kFwdKStages, (j / kFwdKStages) & 1, u.abort_flag);
  };
  auto issue_s = [&](int j) {  // S(j) -> buffer j % 2; free because the PV of tile j-2 was issued before
    const uint64_t k_desc = desc_step(k_desc0, (j % kFwdKStages) * TileGeom<D>::kBytes);
#pragma unroll
    for (int k = 0; k < D / 16; ++k)  // 16 elements of the head dimension = 8 packed Q columns
      mma_ts(tmem_base + kFwdColS + (j % kFwdSBufs) * 128, tmem_base + kFwdColQ + k * 8,
             desc_step(k_desc, (k >> 2) * TileGeom<D>::kBlockBytes + (k & 3) * 32), idesc_s, k > 0);
  };
  auto commit_s = [&](int j) {
    mma_commit(bar.k_empty + j % kFwdKStages);
    mma_commit(bar.s_full + j % kFwdSBufs);
  };
  for (int j = 0; j < kFwdSBufs && j < u.n_tiles; ++j) {
    wait_k(j);
    tc_fence_after_sync();
    issue_s(j);
    commit_s(j);
  }
  for (int j = 0; j < u.n_tiles; ++j) {
    const int st = j % kFwdVStages, buf = j % kFwdSBufs;
    const bool more = j + kFwdSBufs < u.n_tiles;
    const uint32_t pcol = tmem_base + kFwdColS + buf * 128;
    const uint64_t v_desc = desc_mnmajor(smem_u32(u.sV + st * TileGeom<D>::kBytes), TileGeom<D>::kBlockBytes);
    mbar_wait_spin(bar.v_full + st, (j / kFwdVStages) & 1, u.abort_flag);
    if (more) wait_k(j + kFwdSBufs);
#pragma unroll
    for (int g = 0; g < kFwdGroups; ++g)
      mbar_wait_spin(bar.p_full + g * kFwdSBufs + buf, (j / kFwdSBufs) & 1, u.abort_flag);
    tc_fence_after_sync();
#pragma unroll
    for (int kb = 0; kb < kTile / 16; ++kb) {
      // P of 16 keys = 8 packed columns; group g's pairs start at its own S columns
      const uint32_t a = pcol + (kb * 16 / kFwdCols) * kFwdCols + (kb * 16 % kFwdCols) / 2;
      mma_ts(tmem_base + kFwdColO, a, desc_step(v_desc, kb * 2048), idesc_pv, (j > 0 || kb > 0) ? 1u : 0u);
    }
    if (more) issue_s(j + kFwdSBufs);
    mma_commit(bar.pv_done + (j & 1));   // tracks the S MMAs too: they are long done when O is needed
    mma_commit(bar.v_empty + st);
    if (more) commit_s(j + kFwdSBufs);
  }
  mma_commit(bar.o_full);
}

// exp2(s * scale_log2 - m) for 32 consecutive keys of one row, as 16 bf16 pairs; returns their sum.
// `valid` = how many of the 32 keys exist (the rest get P = 0 whatever their S, which may be stale data).
// kPolyOf8 of every 8 pairs take the polynomial; the largest argument it was handed is folded into poly_max.
__device__ __forceinline__ float fwd_exp32(const uint32_t (&s)[32], int valid, float scale_log2, float neg_m,
                                           uint32_t (&pk)[16], float& poly_max) {
  if (valid < 32) {
    float sum = 0.f;
#pragma unroll
    for (int c = 0; c < 32; c += 2) {
      float p0 = fast_exp2(fmaf(__uint_as_float(s[c]), scale_log2, neg_m));
      float p1 = fast_exp2(fmaf(__uint_as_float(s[c + 1]), scale_log2, neg_m));
      if (c >= valid) p0 = 0.f;
      if (c + 1 >= valid) p1 = 0.f;
      sum += p0 + p1;
      pk[c >> 1] = pack_bf16(p0, p1);
    }
    return sum;
  }
  const uint64_t sc2 = f32x2(scale_log2, scale_log2), nm2 = f32x2(neg_m, neg_m);
  uint64_t acc_a = f32x2(0.f, 0.f), acc_b = f32x2(0.f, 0.f);
#pragma unroll
  for (int c = 0; c < 32; c += 2) {
    const uint64_t x2 = fma2(f32x2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, nm2);
    float p0, p1, x0, x1;
    f32x2_split(x2, x0, x1);
    if (((c >> 1) & 7) < kPolyOf8) {
      poly_max = max3(poly_max, x0, x1);
      exp2_poly_pair(x2, p0, p1);
    } else {
      p0 = fast_exp2(x0);
      p1 = fast_exp2(x1);
    }
    if ((c >> 1) & 1) acc_a = add2(acc_a, f32x2(p0, p1));
    else acc_b = add2(acc_b, f32x2(p0, p1));
    pk[c >> 1] = pack_bf16(p0, p1);
  }
  float r0, r1;
  f32x2_split(add2(acc_a, acc_b), r0, r1);
  return r0 + r1;
}

// 32 accumulator columns of the lane's row -> times 1/l -> bf16 -> columns [col0, col0 + 32) of the output row, the
// quads of the warp storing their rows together.  chk2 stays 0 while every value times 0 is 0, i.e. is finite.
__device__ __forceinline__ void fwd_store_slice(const uint32_t (&acc)[32], uint64_t inv2, uint64_t& chk2,
                                                const QuadRows& out, int col0, int lane) {
  const uint64_t zero2 = f32x2(0.f, 0.f);
  uint4 ch[4];
#pragma unroll
  for (int v = 0; v < 4; ++v) {
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint64_t f2 = mul2(f32x2(__uint_as_float(acc[8 * v + 2 * e]), __uint_as_float(acc[8 * v + 2 * e + 1])), inv2);
      chk2 = fma2(f2, zero2, chk2);
      float f0, f1;
      f32x2_split(f2, f0, f1);
      w[e] = pack_bf16(f0, f1);
    }
    ch[v] = make_uint4(w[0], w[1], w[2], w[3]);
  }
  store_quad_rows(ch, out, col0, lane);
}
__device__ __forceinline__ bool fwd_all_finite(uint64_t chk2) {
  float chk0, chk1;
  f32x2_split(chk2, chk0, chk1);
  return chk0 == 0.f && chk1 == 0.f;
}

// Epilogue shared by the safe pass and the CTA-pair kernel: row sum = sum of the groups' partial sums; 32-column slices of the output
// row are dealt round-robin to the groups.  The slices are read out of tensor memory first; `o_free`, if given,
// gets this thread's arrival right after that (O may be overwritten from then on).  `ex` = [G][128] floats for the
// exchange of the partial sums.  The quads of a warp store their rows together (64 contiguous bytes per row).
// Returns false if a stored value was not finite.
template <int D, int G = kFwdGroups>
__device__ __forceinline__ bool fwd_epilogue(const FwdUnit<D>& u, uint64_t* o_full, uint32_t o_parity,
                                             uint64_t* o_free, float* ex, int g, int r, uint32_t tmem_lane,
                                             float m_run, float l_run, const QuadRows& out, bool in_range,
                                             float* lse_dst) {
  constexpr int kSlices = D / 32, kOwn = (kSlices + G - 1) / G;
  mbar_wait(o_full, o_parity, u.abort_flag);
  tc_fence_after_sync();
  uint32_t acc[kOwn][32];
#pragma unroll
  for (int i = 0; i < kOwn; ++i)
    if (g + i * G < kSlices) tmem_ld32(tmem_lane + kFwdColO + (g + i * G) * 32, acc[i]);
  tmem_wait_ld();
  if (o_free != nullptr) {
    tc_fence_before_sync();
    mbar_arrive(o_free);
  }
  ex[g * kTile + r] = l_run;
  named_barrier_sync(5, 128 * G);
  float l = 0.f;
#pragma unroll
  for (int og = 0; og < G; ++og) l += ex[og * kTile + r];
  const float inv_l = 1.f / l;
  const uint64_t inv2 = f32x2(inv_l, inv_l);
  uint64_t chk2 = f32x2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < kOwn; ++i) {
    const int c4 = g + i * G;
    if (c4 >= kSlices) continue;   // the same for the whole warp
    fwd_store_slice(acc[i], inv2, chk2, out, c4 * 32, r & 31);
  }
  if (g == G - 1 && in_range && lse_dst != nullptr) *lse_dst = (m_run + log2f(l)) * 0.6931471805599453f;
  return fwd_all_finite(chk2);
}

// Where the rows of a unit are: the lane's own row for LSE, its quad's rows for O and Q.
template <int D> struct FwdRow {
  bool in_range;
  float* lse_dst;
  QuadRows out, q_rows;
  __device__ FwdRow(const FwdSched& sch, int unit, int r, const __nv_bfloat16* q, int n_q, int heads,
                    __nv_bfloat16* o, float* lse) {
    int qt, h, b;
    sch.decode(unit, qt, h, b);
    init(qt, h, b, r, q, n_q, heads, o, lse);
  }
  __device__ FwdRow(const FwdSched& sch, const FwdPos& pos, int r, const __nv_bfloat16* q, int n_q, int heads,
                    __nv_bfloat16* o, float* lse) {
    init(pos.qt, pos.h(sch), pos.b(sch), r, q, n_q, heads, o, lse);
  }
  __device__ void init(int qt, int h, int b, int r, const __nv_bfloat16* q, int n_q, int heads, __nv_bfloat16* o,
                       float* lse) {
    const int row = qt * kTile + r;
    in_range = row < n_q;
    lse_dst = lse ? lse + (static_cast<size_t>(b) * heads + h) * n_q + (in_range ? row : 0) : nullptr;
    out = quad_rows(o, b, h, n_q, heads, D, row);
    q_rows = quad_rows(q, b, h, n_q, heads, D, row);
  }
  // elements [64 q_part, 64 q_part + 64) of the lane's own Q row, as the 32 packed words tensor memory takes
  __device__ void load_q(uint32_t (&qr)[32], int q_part, int lane) const {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint4 ch[4];
      load_quad_rows(ch, q_rows, q_part * 64 + half * 32, lane);
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        qr[16 * half + 4 * v] = ch[v].x; qr[16 * half + 4 * v + 1] = ch[v].y;
        qr[16 * half + 4 * v + 2] = ch[v].z; qr[16 * half + 4 * v + 3] = ch[v].w;
      }
    }
  }
};

// ---------------------------------------------------------------------------------- softmax, fast pass
// What a softmax thread needs for one key tile of the fast pass.
struct FwdTileCtx {
  uint32_t tmem_lane;
  int g, r, warp;
  float scale_log2;
  uint64_t *sdone, *ready;
  volatile int* abort_flag;
  float* mslot;   // [groups][128] floats for the exchange of the first tile's row maxima
};

// One key tile J of the CTA's stream; `valid` = valid keys of this group's share (may be <= 0).  Full tiles pass the
// constant kFwdCols, so that nothing about key validity is left in their code.  kFirst: the unit's first tile, which
// fixes the rows' reference.
template <bool kFirst>
__device__ __forceinline__ void fwd_fast_tile(const FwdTileCtx& c, int J, int valid, float& m_ref, float& l_run,
                                              float& poly_max) {
  constexpr int NL = kFwdCols / 32;  // 32-column TMEM loads per thread and tile
  const uint32_t colS = kFwdColS + (J % kFwdSBufs) * 128 + c.g * kFwdCols;
  mbar_wait(c.sdone + J % 4, (J / 4) & 1, c.abort_flag);
  tc_fence_after_sync();
  uint32_t s[NL][32];
#pragma unroll
  for (int c2 = 0; c2 < NL; ++c2) tmem_ld32(c.tmem_lane + colS + c2 * 32, s[c2]);
  tmem_wait_ld();
  if (kFirst) {
    // the row's one reference: the maximum of the first tile, agreed between the threads of the row
    float mx = -INFINITY;
#pragma unroll
    for (int c2 = 0; c2 < NL; ++c2)
#pragma unroll
      for (int k = 0; k < 32; ++k)
        if (c2 * 32 + k < valid) mx = fmaxf(mx, __uint_as_float(s[c2][k]));
    c.mslot[c.g * kTile + c.r] = mx;
    named_barrier_sync(1 + (c.warp & 3), 32 * kFwdGroups);
#pragma unroll
    for (int og = 0; og < kFwdGroups; ++og) mx = fmaxf(mx, c.mslot[og * kTile + c.r]);  // finite: >= 1 valid key
    m_ref = mx * c.scale_log2;
  }
  const float neg_m = -m_ref;
  // V rows past a key range's end never hold stale data here: the cache ranges' tensor maps end with the range,
  // the chunk's with the chunk, and TMA fills what lies beyond with zeros
#pragma unroll
  for (int c2 = 0; c2 < NL; ++c2) {
    uint32_t pk[16];
    l_run += fwd_exp32(s[c2], valid - 32 * c2, c.scale_log2, neg_m, pk, poly_max);
    tmem_st16(c.tmem_lane + colS + c2 * 16, pk);   // in place: this thread has read all of its S columns
  }
  tmem_wait_st();
  tc_fence_before_sync();
  mbar_arrive(c.ready + J % 4);
}

// A run of `count` full key tiles that do not open a unit, from tile J of the stream on: the loop in which the
// kernel spends its time.  Compiled out of line and handed plain values only (shared-memory addresses as 32-bit
// numbers), so that its code does not depend on what the bookkeeping between units needs around it.
// Returns the row sum.
__device__ __noinline__ float fwd_fast_run(uint32_t tmem_lane_g, uint32_t sdone, uint32_t ready, uint32_t abort_flag,
                                           float scale_log2, float neg_m, float l_run, int J, int count) {
  static_assert(kFwdCols == 32, "one 32-column load per thread and tile");
  float poly_max = -INFINITY;
  for (int i = 0; i < count; ++i, ++J) {
    const uint32_t colS = tmem_lane_g + kFwdColS + (J % kFwdSBufs) * 128;
    mbar_wait_at(sdone + 8 * (J % 4), (J / 4) & 1, abort_flag);
    tc_fence_after_sync();
    uint32_t sv[32], pk[16];
    tmem_ld32(colS, sv);
    tmem_wait_ld();
    l_run += fwd_exp32(sv, 32, scale_log2, neg_m, pk, poly_max);
    tmem_st16(colS, pk);   // in place: this thread has read all of its S columns
    tmem_wait_st();
    tc_fence_before_sync();
    mbar_arrive_at(ready + 8 * (J % 4));
  }
  if (poly_max > kPolyArgLimit) l_run = INFINITY;   // the polynomial was handed an argument beyond its range: redo the unit
  return l_run;
}

// Where the fast pass leaves a unit's row statistics for the epilogue warps: per unit parity, the groups' partial
// row sums [groups][128] and the rows' reference exponents [128].
template <int D> struct FwdStats {
  float* smax;
  __device__ float* sums(int n) const { return smax + (n & 1) * kFwdGroups * kTile; }
  __device__ float* refs(int n) const { return smax + 4 * kFwdGroups * kTile + (n & 1) * kTile; }
  __device__ float* maxima(int n) const { return smax + (2 + (n & 1)) * kFwdGroups * kTile; }   // first-tile exchange
};

// Walks the CTA's units: per unit the first key tile (which fixes the rows' reference), the others, then the row
// sum and the reference go to shared memory for the epilogue warps.  Nothing else happens between the last tile of a
// unit and the first of the next, whose S was issued two tiles earlier.
// A unit one of whose rows must be redone by the safe pass gets its bit set in `redo_bits`.
template <int D>
__device__ __forceinline__ void fwd_softmax_fast(const FwdUnit<D>& u, const FwdSched& sch, const FwdFastBars& bar,
                                                 int warp, int r, float scale_log2, uint32_t* redo_bits) {
  const KeySegs& segs = *u.segs;
  const int g = warp >> 2;
  const FwdStats<D> stats{u.smax};
  FwdTileCtx c;
  c.tmem_lane = u.tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
  c.g = g; c.r = r; c.warp = warp;
  c.scale_log2 = scale_log2;
  const int half = g * kFwdHalves / kFwdGroups;   // which half of a tile's keys the group works on
  c.sdone = bar.sdone + 4 * half; c.ready = bar.ready + 4 * half;
  c.abort_flag = u.abort_flag;
  const int c0 = segs.count[0], T = u.n_tiles;
  const uint32_t lane_g = c.tmem_lane + g * kFwdCols;
  const uint32_t sdone_at = smem_u32(c.sdone), ready_at = smem_u32(c.ready);
  const uint32_t abort_at = smem_u32(const_cast<int*>(u.abort_flag));
  int n = 0;
  for (int unit = sch.first; unit < sch.total; unit += sch.stride, ++n) {
    const int J = n * T;
    float m_ref = 0.f, l_run = 0.f, poly_max = -INFINITY;
    c.mslot = stats.maxima(n);   // alternates: a fast thread may be a unit ahead of the others
    if (c0 >= kTile) fwd_fast_tile<true>(c, J, kFwdCols, m_ref, l_run, poly_max);
    else fwd_fast_tile<true>(c, J, c0 - kFwdCols * g, m_ref, l_run, poly_max);
    // the other tiles: key ranges one after the other, their full tiles in one run, then the ragged last tile if any
    int Jr = J + 1;
    for (int sg = 0; sg < segs.n; ++sg) {
      int full = segs.count[sg] / kTile, rest = segs.count[sg] % kTile;
      if (sg == 0) {   // minus the first tile
        if (full > 0) --full; else rest = 0;
      }
      if (full > 0) {
        l_run = fwd_fast_run(lane_g, sdone_at, ready_at, abort_at, scale_log2, -m_ref, l_run, Jr, full);
        Jr += full;
      }
      if (rest) { fwd_fast_tile<false>(c, Jr, rest - kFwdCols * g, m_ref, l_run, poly_max); ++Jr; }
    }
    // The slots of unit n - 2 are free: the epilogue warps read them before they let go of that unit's O, which the
    // first P V of unit n - 1 waited for.
    stats.sums(n)[g * kTile + r] = l_run;
    if (g == 0) stats.refs(n)[r] = m_ref;
    if (!((l_run < kFastSumLimit) && !(poly_max > kPolyArgLimit)))   // true for inf and NaN too
      atomicOr(redo_bits + (n >> 5), 1u << (n & 31));
    mbar_arrive(bar.stats_full + (n & 1));
  }
}

// ---------------------------------------------------------------------------------- epilogue warps, fast pass
// Eight warps: one per quarter of the tensor-memory lanes (lane = query row of the tile) and half of the head
// dimension.  Per unit: wait for the row statistics and for the last P V, read the warp's half of O out of tensor
// memory in one go (o_free right after), normalise, store O (and LSE: the first half's warps); then fetch the warp's
// 64-element part of the Q rows of the unit after the next into the Q buffer this unit used.
// They keep every load from and store to global memory away from the softmax threads.
template <int D>
__device__ __forceinline__ void fwd_epilogue_fast(const FwdUnit<D>& u, const FwdSched& sch, const FwdFastBars& bar,
                                                  int warp, int lane, const __nv_bfloat16* q, int n_q, int heads,
                                                  __nv_bfloat16* o, float* lse, uint32_t* redo_bits) {
  constexpr int kSlices = D / 32, kOwn = kSlices / 2;   // 32-column slices of O: all, and this warp's
  constexpr int kMmaWarp = 4 * kFwdGroups;
  const FwdStats<D> stats{u.smax};
  const int half = (warp - kMmaWarp - 2) >> 2;          // 0: columns [0, D/2), 1: the others
  const int r = (warp & 3) * 32 + lane;
  const uint32_t tmem_lane = u.tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
  const bool stages_q = half < D / 64;                  // part `half` of the Q rows
  auto stage_q = [&](const FwdPos& pos, int buf) {
    if (!stages_q) return;
    const FwdRow<D> row(sch, pos, r, q, n_q, heads, o, lse);
    uint32_t qr[32];
    row.load_q(qr, half, lane);
    tmem_st32(tmem_lane + kFwdColQ + buf * kFwdQCols + half * 32, qr);
    tmem_wait_st();
    tc_fence_before_sync();
    mbar_arrive(bar.q_full + buf);
  };
  FwdPos pos(sch, sch.first);
  {   // the first two units' Q
    stage_q(pos, 0);
    if (sch.first + sch.stride < sch.total) {
      FwdPos next = pos;
      next.forward(sch);
      stage_q(next, 1);
    }
  }
  int n = 0;
  for (int unit = sch.first; unit < sch.total; unit += sch.stride, ++n) {
    const FwdRow<D> row(sch, pos, r, q, n_q, heads, o, lse);
    mbar_wait_relaxed(bar.stats_full + (n & 1), (n >> 1) & 1, u.abort_flag);
    float l = 0.f;
#pragma unroll
    for (int g = 0; g < kFwdGroups; ++g) l += stats.sums(n)[g * kTile + r];
    const float m = stats.refs(n)[r];
    const float inv_l = 1.f / l;
    const uint64_t inv2 = f32x2(inv_l, inv_l);
    uint64_t chk2 = f32x2(0.f, 0.f);
    mbar_wait(bar.o_full, n & 1, u.abort_flag);
    tc_fence_after_sync();
    uint32_t acc[kOwn][32];
#pragma unroll
    for (int i = 0; i < kOwn; ++i) tmem_ld32(tmem_lane + kFwdColO + (half * kOwn + i) * 32, acc[i]);
    tmem_wait_ld();
    tc_fence_before_sync();
    mbar_arrive(bar.o_free);   // this warp's part of O is in registers: the next unit may start on it
#pragma unroll
    for (int i = 0; i < kOwn; ++i) fwd_store_slice(acc[i], inv2, chk2, row.out, (half * kOwn + i) * 32, lane);
    if (half == 0 && row.in_range && row.lse_dst != nullptr) *row.lse_dst = (m + log2f(l)) * 0.6931471805599453f;
    if (!fwd_all_finite(chk2)) atomicOr(redo_bits + (n >> 5), 1u << (n & 31));
    // Q of the unit after the next, into this unit's buffer: every S of this unit is complete (o_full)
    if (unit + 2 * sch.stride < sch.total) {
      FwdPos later = pos;
      later.forward(sch);
      later.forward(sch);
      stage_q(later, n & 1);
    }
    pos.forward(sch);
  }
}

// ---------------------------------------------------------------------------------- softmax, safe pass
// The threads that share a query row (one per group) keep the same running reference for the row, so all
// parts of P V accumulate into ONE O accumulator; each keeps its own partial row sum.  No row maximum while
// nothing happens: a tile is exponentiated against the row's current reference; only when a tile's row sum
// leaves the safe range (>= 2^30, inf or NaN, or the polynomial was handed an argument beyond its range), or
// on the first tile, do the two threads agree (one 64-thread named barrier per warp pair and tile carries the
// decision) to take the tile's true maximum as the new reference, rescaling O and the row sums.
template <int D>
__device__ __forceinline__ void fwd_softmax_safe(const FwdUnit<D>& u, const FwdBars& bar, int warp, int r,
                                                 float scale_log2, const QuadRows& out, bool in_range,
                                                 float* lse_dst) {
  const KeySegs& segs = *u.segs;
  const int g = warp >> 2;
  constexpr int NL = kFwdCols / 32;  // 32-column TMEM loads per thread and tile
  const uint32_t tmem_lane = u.tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
  float m_run = -INFINITY, l_run = 0.f;
  int j = 0;
  for (KeyTileIter it; !it.done(segs); it.next(segs), ++j) {
    const int tile_valid = it.valid(segs);
    const int valid = tile_valid - kFwdCols * g;
    const int buf = j % kFwdSBufs;
    const uint32_t colS = kFwdColS + buf * 128 + g * kFwdCols;
    mbar_wait(bar.s_full + buf, (j / kFwdSBufs) & 1, u.abort_flag);
    tc_fence_after_sync();

    uint32_t pk[NL][16];
    auto exponentiate = [&](bool& overflow) -> float {
      uint32_t s[NL][32];
#pragma unroll
      for (int c2 = 0; c2 < NL; ++c2) tmem_ld32(tmem_lane + colS + c2 * 32, s[c2]);
      tmem_wait_ld();
      float sum = 0.f, poly_max = -INFINITY;
#pragma unroll
      for (int c2 = 0; c2 < NL; ++c2) sum += fwd_exp32(s[c2], valid - 32 * c2, scale_log2, -m_run, pk[c2], poly_max);
      overflow = !(sum < kRowSumLimit) || poly_max > kPolyArgLimit;   // also true for inf and NaN
      return sum;
    };

    float rowsum = 0.f;
    bool redo = m_run == -INFINITY;
    if (!__all_sync(0xffffffffu, redo)) {
      bool overflow;
      rowsum = exponentiate(overflow);
      redo = redo || overflow;
    }
    float* fslot = u.smax + (j & 1) * kFwdGroups * kTile;
    fslot[g * kTile + r] = redo ? 1.f : 0.f;
    named_barrier_sync(1 + (warp & 3), 32 * kFwdGroups);
#pragma unroll
    for (int og = 0; og < kFwdGroups; ++og) redo = redo || fslot[og * kTile + r] != 0.f;
    float alpha = 1.f;
    if (__any_sync(0xffffffffu, redo)) {
      // exact tile maximum, shared between the threads of the row; rows of the warp that did not ask for it
      // keep their reference
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
      float* mslot = u.smax + 2 * kFwdGroups * kTile;
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
        mbar_wait(bar.pv_done + ((j - 1) & 1), ((j - 1) >> 1) & 1, u.abort_flag);
        tc_fence_after_sync();
        // 32-column slices of the row are dealt round-robin to the groups
#pragma unroll
        for (int c4 = 0; c4 < D / 32; ++c4) {
          if (c4 % kFwdGroups != g) continue;
          uint32_t acc[32];
          tmem_ld32(tmem_lane + kFwdColO + c4 * 32, acc);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) acc[c] = __float_as_uint(__uint_as_float(acc[c]) * alpha);
          tmem_st32(tmem_lane + kFwdColO + c4 * 32, acc);
        }
      }
      l_run *= alpha;
      bool overflow;
      rowsum = exponentiate(overflow);
    }
    l_run += rowsum;
#pragma unroll
    for (int c2 = 0; c2 < NL; ++c2) tmem_st16(tmem_lane + colS + c2 * 16, pk[c2]);
    if (g == 0 && tile_valid < kTile) {
      const int st = j % kFwdVStages;
      mbar_wait(bar.v_full + st, (j / kFwdVStages) & 1, u.abort_flag);
      zero_tile_rows_from<D>(u.sV + st * TileGeom<D>::kBytes, tile_valid, r);
    }
    tmem_wait_st();
    tc_fence_before_sync();
    mbar_arrive(bar.p_full + g * kFwdSBufs + buf);
  }
  fwd_epilogue<D>(u, bar.o_full, 0, nullptr, u.smax, g, r, tmem_lane, m_run, l_run, out, in_range, lse_dst);
}

// The safe pass of one unit, all roles.  Kept out of line: it is the rare path, and the registers it needs must not
// weigh on the allocation of the fast pass around it.
template <int D>
__device__ __noinline__ void fwd_safe_unit(const FwdUnit<D>& u, const FwdBars& bar, int warp, int lane, int r,
                                           float scale_log2, const QuadRows& out, bool in_range, float* lse_dst) {
  constexpr int kMmaWarp = 4 * kFwdGroups, kTmaWarp = 4 * kFwdGroups + 1;
  if (warp == kTmaWarp) {
    if (lane == 0) fwd_produce<D>(u, bar);
  } else if (warp == kMmaWarp) {
    if (lane == 0) fwd_issue<D>(u, bar);
  } else if (warp < kMmaWarp) {
    fwd_softmax_safe<D>(u, bar, warp, r, scale_log2, out, in_range, lse_dst);
  }
}

// grid.x CTAs share `batch * heads * ceil(n_q / 128)` work units (at most kFwdMaxUnits each): CTA i takes units
// i, i + grid.x, ...  Launched with one CTA per SM the CTAs are all resident and each streams through its units.
template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
chunk_attn_fwd_kernel(const __nv_bfloat16* __restrict__ q, const __grid_constant__ CUtensorMap tm_kc,
                      const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kx,
                      const __grid_constant__ CUtensorMap tm_vx0, const __grid_constant__ CUtensorMap tm_vx1,
                      const __grid_constant__ KeySegs segs, const int batch, const int n_q,
                      const int heads, const int cache_shared, const float scale_log2, const int force_safe,
                      __nv_bfloat16* __restrict__ o, float* __restrict__ lse) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align_1024(smem_raw);
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(smem + FwdSmem<D>::kBars);
  const FwdFastBars bar_fast(bar_mem);
  const FwdBars bar_safe(bar_mem + kFwdBarSlots);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_mem + 2 * kFwdBarSlots);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  uint32_t* redo_bits = tmem_holder + 16;   // one bit per unit of this CTA

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr uint32_t kTmemCols = 512;
  constexpr int kMmaWarp = 4 * kFwdGroups, kTmaWarp = 4 * kFwdGroups + 1;
  FwdSched sch;
  sch.q_tiles = (n_q + kTile - 1) / kTile;
  sch.dim_y = cache_shared ? batch : heads;
  sch.cache_shared = cache_shared;
  sch.first = blockIdx.x;
  sch.stride = gridDim.x;
  sch.total = sch.q_tiles * heads * batch;

  const int r = tid & 127;           // query row inside the tile = TMEM lane (softmax warps)
  const bool stages_q = warp < kMmaWarp && (warp >> 2) < D / 64;   // safe pass: who writes Q into tensor memory
  if (warp == kTmaWarp && lane == 0) {
    tma_prefetch_desc(&tm_kc); tma_prefetch_desc(&tm_vc); tma_prefetch_desc(&tm_kx); tma_prefetch_desc(&tm_vx0);
  }
  if (tid == 0) {
    bar_fast.init(128 * (D / 64));   // q_full: one arrival per row and 64-element part
    bar_safe.init(1, 128);
    *abort_flag = 0;
    fence_mbar_init();
    fence_proxy_async_smem();
  }
  if (tid < kFwdMaxUnits / 32) redo_bits[tid] = 0;
  if (warp == kMmaWarp) {
    tmem_alloc(tmem_holder, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  FwdUnit<D> u;
  u.tm_kc = &tm_kc; u.tm_vc = &tm_vc; u.tm_kx = &tm_kx; u.tm_vx0 = &tm_vx0; u.tm_vx1 = &tm_vx1;
  u.segs = &segs;
  u.sK = smem + FwdSmem<D>::kK;
  u.sV = smem + FwdSmem<D>::kV;
  u.smax = reinterpret_cast<float*>(smem + FwdSmem<D>::kMax);
  u.abort_flag = abort_flag;
  u.tmem_base = *tmem_holder;
  u.n_tiles = seg_tiles(segs);
  u.h = u.b = u.bx = 0;   // set per unit by the safe pass; the fast pass follows its cursors
  const uint32_t tmem_lane = u.tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);

  // ---- fast pass over all the CTA's units
  if (!force_safe) {
    if (warp == kTmaWarp) {
      if (lane == 0) fwd_produce_fast<D>(u, sch, bar_fast);
    } else if (warp == kMmaWarp) {
      if (lane == 0) fwd_issue_fast<D>(u, sch, bar_fast);
    } else if (warp < kMmaWarp) {
      fwd_softmax_fast<D>(u, sch, bar_fast, warp, r, scale_log2, redo_bits);
    } else {
      fwd_epilogue_fast<D>(u, sch, bar_fast, warp, lane, q, n_q, heads, o, lse, redo_bits);
    }
  }

  // ---- safe pass, unit by unit, for the units one of whose rows asked for it (every MMA of the fast pass has
  //      finished by now: the epilogue warps waited for the last one)
  int n = 0;
  for (int unit = sch.first; unit < sch.total; unit += sch.stride, ++n) {
    tc_fence_before_sync();
    __syncthreads();   // the fast pass, or the unit before, is over for every thread: redo bits and barriers at rest
    tc_fence_after_sync();
    if (*abort_flag) break;
    if (!force_safe && !((redo_bits[n >> 5] >> (n & 31)) & 1u)) continue;
    int qt;
    sch.decode(unit, qt, u.h, u.b);
    u.bx = cache_shared ? 0 : u.b;
    const FwdRow<D> row(sch, unit, r, q, n_q, heads, o, lse);
    if (tid == 0) {
      bar_safe.rearm(1, 128);
      fence_mbar_init();
    }
    if (stages_q) {
      uint32_t qr[32];
      row.load_q(qr, warp >> 2, lane);
      tmem_st32(tmem_lane + kFwdColQ + (warp >> 2) * 32, qr);
      tmem_wait_st();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const FwdUnit<D> su = u;   // a copy: `u` itself never leaves the registers of the fast pass
    fwd_safe_unit<D>(su, bar_safe, warp, lane, r, scale_log2, row.out, row.in_range, row.lse_dst);
  }
  settle_after_abort(abort_flag);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(u.tmem_base, kTmemCols);
}

}  // namespace astro
