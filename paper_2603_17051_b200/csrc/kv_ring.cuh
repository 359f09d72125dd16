// Ring-buffer KV storage: bit-exact copies between the caller's [B_c, frames*T, H, D] layout and the
// private cache layout [B_c, H, slot*T + t, D].  Pure bandwidth work: one 16-byte vector per thread
// per step, 256-byte token rows contiguous on both sides.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace astro {

constexpr int kMaxFramesPerCopy = 32;

struct SlotMap {
  int n;                         // frames in this launch
  int slot[kMaxFramesPerCopy];   // storage slot of the j-th frame of the caller's tensor
};

// ToCache: caller tensor -> storage (append); otherwise storage -> caller tensor (export).
// blockIdx.y selects K (0) or V (1).  `frame0` is the first frame of the caller tensor handled here,
// `frames_total` the frame count of the caller tensor (its token stride per batch entry).
template <bool ToCache>
__global__ void __launch_bounds__(256)
ring_copy_kernel(uint4* __restrict__ k_user, uint4* __restrict__ v_user, uint4* __restrict__ k_store,
                 uint4* __restrict__ v_store, const SlotMap map, const int heads, const int tokens_per_frame,
                 const int vec_per_row, const int slots, const int frame0, const int frames_total,
                 const long long vec_per_batch /* map.n * T * H * vec_per_row */, const long long total) {
  uint4* user = blockIdx.y == 0 ? k_user : v_user;
  uint4* store = blockIdx.y == 0 ? k_store : v_store;
  constexpr int kItems = 4;
  const long long base = static_cast<long long>(blockIdx.x) * (blockDim.x * kItems) + threadIdx.x;
  long long src_idx[kItems], dst_idx[kItems];
  bool ok[kItems];
#pragma unroll
  for (int i = 0; i < kItems; ++i) {
    const long long idx = base + static_cast<long long>(i) * blockDim.x;
    ok[i] = idx < total;
    const long long b = ok[i] ? idx / vec_per_batch : 0;
    uint32_t r = ok[i] ? static_cast<uint32_t>(idx - b * vec_per_batch) : 0u;  // (j, t, h, vec) in caller order
    const uint32_t vec = r % vec_per_row;
    r /= vec_per_row;
    const uint32_t h = r % heads;
    r /= heads;
    const uint32_t t = r % tokens_per_frame;
    const uint32_t j = r / tokens_per_frame;
    const long long u = ((b * frames_total + frame0 + j) * tokens_per_frame + t) * heads + h;
    const long long s = ((b * heads + h) * slots + map.slot[j]) * tokens_per_frame + t;
    const long long ui = u * vec_per_row + vec, si = s * vec_per_row + vec;
    src_idx[i] = ToCache ? ui : si;
    dst_idx[i] = ToCache ? si : ui;
  }
  const uint4* src = ToCache ? user : store;
  uint4* dst = ToCache ? store : user;
  uint4 val[kItems];
#pragma unroll
  for (int i = 0; i < kItems; ++i)
    if (ok[i]) val[i] = src[src_idx[i]];
#pragma unroll
  for (int i = 0; i < kItems; ++i)
    if (ok[i]) dst[dst_idx[i]] = val[i];
}

}  // namespace astro
