// Ring-buffer KV storage: bit-exact copies between the caller's [B_c, frames*T, H, D] layout and the
// private cache layout [B_c, H, slot*T + t, D].  Pure bandwidth work.  A thread owns one 16-byte vector
// position (head, d) and walks kTokens consecutive tokens of one frame, so its addresses advance by a
// constant on both sides and no per-element index division is needed; a warp covers 512 contiguous bytes
// of the caller tensor and two 256-byte token rows of the storage per step.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace astro {

constexpr int kMaxFramesPerCopy = 32;
constexpr int kRingTokensPerThread = 8;

struct SlotMap {
  int n;                         // frames in this launch
  int slot[kMaxFramesPerCopy];   // storage slot of the j-th frame of this launch
};

// ToCache: caller tensor -> storage (append); otherwise storage -> caller tensor (export).
// grid.x covers the H * vec_per_row vector positions of a token row, grid.y = frame * token chunks,
// grid.z = 2 * b + (0: K, 1: V).  `frame0` is the first frame of the caller tensor handled by this launch,
// `frames_total` the frame count of the caller tensor.
template <bool ToCache>
__global__ void __launch_bounds__(256)
ring_copy_kernel(uint4* __restrict__ k_user, uint4* __restrict__ v_user, uint4* __restrict__ k_store,
                 uint4* __restrict__ v_store, const SlotMap map, const int heads, const int tokens_per_frame,
                 const int vec_per_row, const int slots, const int frame0, const int frames_total,
                 const int chunks_per_frame) {
  const int hv = blockIdx.x * blockDim.x + threadIdx.x;  // head * vec_per_row + vec
  const int row_vecs = heads * vec_per_row;
  if (hv >= row_vecs) return;
  const int j = blockIdx.y / chunks_per_frame;
  const int t0 = (blockIdx.y - j * chunks_per_frame) * kRingTokensPerThread;
  const int b = blockIdx.z >> 1;
  uint4* user = (blockIdx.z & 1) ? v_user : k_user;
  uint4* store = (blockIdx.z & 1) ? v_store : k_store;
  const int h = hv / vec_per_row, vec = hv - h * vec_per_row;
  const long long u0 = ((static_cast<long long>(b) * frames_total + frame0 + j) * tokens_per_frame + t0) * row_vecs + hv;
  const long long s0 =
      ((static_cast<long long>(b) * heads + h) * slots + map.slot[j]) * tokens_per_frame * vec_per_row +
      static_cast<long long>(t0) * vec_per_row + vec;
  const uint4* src = ToCache ? user + u0 : store + s0;
  uint4* dst = ToCache ? store + s0 : user + u0;
  const int src_step = ToCache ? row_vecs : vec_per_row, dst_step = ToCache ? vec_per_row : row_vecs;
  const int n = min(kRingTokensPerThread, tokens_per_frame - t0);
  uint4 val[kRingTokensPerThread];
#pragma unroll
  for (int i = 0; i < kRingTokensPerThread; ++i)
    if (i < n) val[i] = src[static_cast<long long>(i) * src_step];
#pragma unroll
  for (int i = 0; i < kRingTokensPerThread; ++i)
    if (i < n) dst[static_cast<long long>(i) * dst_step] = val[i];
}

}  // namespace astro
