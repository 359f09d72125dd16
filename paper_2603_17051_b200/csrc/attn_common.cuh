// Shared pieces of the chunk-attention kernels: the list of key segments a call attends to,
// the shared-memory tile geometry, and small TMEM/epilogue helpers.
#pragma once
#include "sm100_ptx.cuh"

namespace astro {

constexpr int kTile = 128;  // query rows per CTA tile and keys per key tile

// The keys of one call: up to two contiguous token ranges of the cache storage (the ring can be
// split by its wrap-around or by a hole left by evict) and the chunk's own keys.
struct KeySegs {
  int n;
  int start[3];     // first token (row of the source tensor)
  int count[3];     // tokens in the segment (> 0)
  int from_chunk[3];  // 1: rows of K_chunk/V_chunk, 0: rows of the cache storage
};

__host__ __device__ inline int seg_tiles(const KeySegs& s) {
  int t = 0;
  for (int i = 0; i < s.n; ++i) t += (s.count[i] + kTile - 1) / kTile;
  return t;
}

// Walks key tiles segment by segment.
struct KeyTileIter {
  int seg, off;
  __device__ KeyTileIter() : seg(0), off(0) {}
  __device__ bool done(const KeySegs& s) const { return seg >= s.n; }
  __device__ int row0(const KeySegs& s) const { return s.start[seg] + off; }
  __device__ int valid(const KeySegs& s) const { return min(kTile, s.count[seg] - off); }
  __device__ int from_chunk(const KeySegs& s) const { return s.from_chunk[seg]; }
  __device__ void next(const KeySegs& s) {
    off += kTile;
    if (off >= s.count[seg]) { ++seg; off = 0; }
  }
};

// Rows of a row-major tensor seen by a warp whose lane L owns row L of 32 consecutive rows: the four lanes of a quad
// (lanes 4m .. 4m+3) move the 64-byte pieces of their four rows together, each lane one 16-byte chunk of every row,
// so that one warp-wide access touches 8 rows x 64 contiguous bytes instead of 32 rows x 16 bytes.
// transpose4x4 turns "lane l of the quad holds chunks 0..3 of row l" into "lane l holds chunk l of rows 0..3"
// (slot j = row j), and back: the exchange is its own inverse.
__device__ __forceinline__ void quad_exchange(uint4& a, uint4& b, bool bit, int mask) {
  // lanes with the bit clear keep a and swap b for the partner's a; lanes with it set keep b and swap a
  const uint4 send = bit ? a : b;
  uint4 recv;
  recv.x = __shfl_xor_sync(0xffffffffu, send.x, mask);
  recv.y = __shfl_xor_sync(0xffffffffu, send.y, mask);
  recv.z = __shfl_xor_sync(0xffffffffu, send.z, mask);
  recv.w = __shfl_xor_sync(0xffffffffu, send.w, mask);
  if (bit) a = recv; else b = recv;
}
__device__ __forceinline__ void transpose4x4(uint4 (&c)[4], int lane) {
  const bool b0 = lane & 1, b1 = lane & 2;
  quad_exchange(c[0], c[1], b0, 1);
  quad_exchange(c[2], c[3], b0, 1);
  quad_exchange(c[0], c[2], b1, 2);
  quad_exchange(c[1], c[3], b1, 2);
}

// The four rows of a lane's quad in a [.., rows, heads, D] bf16 tensor: `first` points at element 0 of the quad's
// first row (for the head and sample at hand), rows are `stride` elements apart, `valid` of the four exist.
struct QuadRows {
  __nv_bfloat16* first;
  size_t stride;
  int valid;
};
__device__ __forceinline__ QuadRows quad_rows(const __nv_bfloat16* base, int b, int h, int n_rows, int heads, int D,
                                              int own_row) {
  QuadRows q;
  const int row_first = own_row & ~3;
  q.stride = static_cast<size_t>(heads) * D;
  q.first = const_cast<__nv_bfloat16*>(base) + (static_cast<size_t>(b) * n_rows + row_first) * q.stride +
            static_cast<size_t>(h) * D;
  q.valid = n_rows - row_first;   // may be <= 0 or > 4
  return q;
}
// Lane L holds 32 bf16 (64 bytes, as 4 chunks) of row L, destined for columns [col0, col0 + 32) of its row.
__device__ __forceinline__ void store_quad_rows(uint4 (&c)[4], const QuadRows& q, int col0, int lane) {
  transpose4x4(c, lane);
#pragma unroll
  for (int j = 0; j < 4; ++j)
    if (j < q.valid) *reinterpret_cast<uint4*>(q.first + j * q.stride + col0 + (lane & 3) * 8) = c[j];
}
// The reverse: 32 bf16 of columns [col0, col0 + 32) of the lane's own row (zeros for rows that do not exist).
__device__ __forceinline__ void load_quad_rows(uint4 (&c)[4], const QuadRows& q, int col0, int lane) {
#pragma unroll
  for (int j = 0; j < 4; ++j)
    c[j] = j < q.valid ? *reinterpret_cast<const uint4*>(q.first + j * q.stride + col0 + (lane & 3) * 8)
                       : make_uint4(0, 0, 0, 0);
  transpose4x4(c, lane);
}

// A [128 x D] bf16 tile sits in shared memory as D/64 blocks of [128 rows x 128 bytes], 128-byte
// swizzled by TMA; block h holds columns 64h..64h+63.
template <int D> struct TileGeom {
  static constexpr int kBlocks = D / 64;
  static constexpr int kBlockBytes = kTile * 128;
  static constexpr int kBytes = kBlocks * kBlockBytes;
};

template <int D>
__device__ __forceinline__ void tma_load_tile(uint8_t* smem_tile, const CUtensorMap* tm, uint64_t* bar, int row0,
                                              int h, int b) {
#pragma unroll
  for (int blk = 0; blk < TileGeom<D>::kBlocks; ++blk)
    tma_load_4d(smem_tile + blk * TileGeom<D>::kBlockBytes, tm, bar, blk * 64, row0, h, b);
}

// The single MMA-issuing thread is latency bound on scalar work, so descriptors are built once per tile
// operand and stepped by adding to the start-address field (bits 0-13, units of 16 bytes; tiles live below
// 256 KB, so the field never overflows into its neighbours).
__device__ __forceinline__ uint64_t desc_step(uint64_t desc, uint32_t byte_offset) { return desc + (byte_offset >> 4); }

// acc[128 x N] = A[128 x D] * B[N x D]^T, both tiles K-major (contraction over D), given the descriptors of
// the tiles' first bytes.  B may start at any multiple of 8 rows inside a 128-row tile (+ rows * 128 bytes).
template <int D, int N = kTile>
__device__ __forceinline__ void mma_abT_desc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc) {
  constexpr uint32_t idesc = make_idesc_bf16(kTile, N, false, false);
#pragma unroll
  for (int k = 0; k < D / 16; ++k) {
    const uint32_t off = (k >> 2) * TileGeom<D>::kBlockBytes + (k & 3) * 32;
    mma_ss(d_tmem, desc_step(a_desc, off), desc_step(b_desc, off), idesc, k > 0);
  }
}
template <int D, int N = kTile>
__device__ __forceinline__ void mma_abT(uint32_t d_tmem, uint32_t a_smem, uint32_t b_smem) {
  mma_abT_desc<D, N>(d_tmem, desc_kmajor(a_smem), desc_kmajor(b_smem));
}

// acc[128 x D] (+)= A_tmem[128 x KROWS bf16] * B[KROWS x D] with the contraction over B's rows (MN-major
// B); B starts at row (b_smem - tile base) / 128 of a 128-row tile, a multiple of 16.
template <int D, int KROWS = kTile>
__device__ __forceinline__ void mma_pb(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_smem, bool accumulate) {
  constexpr uint32_t idesc = make_idesc_bf16(kTile, D, false, true);
  const uint64_t b_desc = desc_mnmajor(b_smem, TileGeom<D>::kBlockBytes);
#pragma unroll
  for (int k = 0; k < KROWS / 16; ++k)
    mma_ts(d_tmem, a_tmem + k * 8, desc_step(b_desc, k * 2048), idesc, (accumulate || k > 0) ? 1u : 0u);
}

// Zero rows [first_row, 128) of a tile in shared memory (every block), then publish to the async proxy.
// Row r of a block occupies bytes [128 r, 128 r + 128) whatever the swizzle.  Called by 128 threads.
template <int D>
__device__ __forceinline__ void zero_tile_rows_from(uint8_t* smem_tile, int first_row, int tid) {
  if (tid >= first_row) {
#pragma unroll
    for (int blk = 0; blk < TileGeom<D>::kBlocks; ++blk) {
      uint4* p = reinterpret_cast<uint4*>(smem_tile + blk * TileGeom<D>::kBlockBytes + tid * 128);
#pragma unroll
      for (int i = 0; i < 8; ++i) p[i] = make_uint4(0, 0, 0, 0);
    }
  }
  fence_proxy_async_smem();
}

// Write N fp32 accumulators of this thread's row (TMEM columns [taddr, taddr + N) of its lane), times `mult`, as
// bf16 into columns [col0, col0 + N) of the row; the quads of the warp store their rows together (64 contiguous
// bytes per row and access).  Warp-collective.
template <int N>
__device__ __forceinline__ void store_rows_from_tmem(uint32_t taddr_lane_col0, float mult, const QuadRows& rows,
                                                     int col0, int lane) {
  const uint64_t m2 = f32x2(mult, mult);
#pragma unroll
  for (int j = 0; j < N / 32; ++j) {
    uint32_t r[32];
    tmem_ld32(taddr_lane_col0 + j * 32, r);
    tmem_wait_ld();
    uint4 ch[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      uint32_t w[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float f0, f1;
        f32x2_split(mul2(f32x2(__uint_as_float(r[8 * v + 2 * e]), __uint_as_float(r[8 * v + 2 * e + 1])), m2), f0, f1);
        w[e] = pack_bf16(f0, f1);
      }
      ch[v] = make_uint4(w[0], w[1], w[2], w[3]);
    }
    store_quad_rows(ch, rows, col0 + j * 32, lane);
  }
}

__device__ __forceinline__ uint8_t* align_1024(uint8_t* p) {
  const uint32_t a = smem_u32(p);
  return p + ((1024u - (a & 1023u)) & 1023u);
}

}  // namespace astro
