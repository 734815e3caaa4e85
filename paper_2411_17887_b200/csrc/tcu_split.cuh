// Radix sort by repeated splits, every split built on the tensor-core-unit scan (Blelloch's reduction
// of radix sort to prefix sums, which the paper's introduction cites as the way a TCU can sort).
//
// One pass per key bit b, least significant first:
//   e[i] = 1 if bit b of key[i] is 0, else 0                       (int8 flags)
//   f    = exclusive scan of e                                      (tcu scan, int8 -> int32, exact)
//   key[i] goes to f[i] if e[i] = 1, else to i - f[i] + (number of zeros)
// The split is stable, so after 32 passes the keys are sorted.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace tcu {

__global__ void split_flags_kernel(const uint32_t *__restrict__ keys, int8_t *__restrict__ flags, size_t n, int bit) {
    // four keys per thread: one 16-byte load, one 4-byte store
    const size_t i4 = (size_t(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
    if (i4 + 3 < n) {
        const uint4 k = *reinterpret_cast<const uint4 *>(keys + i4);
        const uint32_t packed = (((k.x >> bit) & 1u) ^ 1u) | ((((k.y >> bit) & 1u) ^ 1u) << 8) |
                                ((((k.z >> bit) & 1u) ^ 1u) << 16) | ((((k.w >> bit) & 1u) ^ 1u) << 24);
        *reinterpret_cast<uint32_t *>(flags + i4) = packed;
    } else {
        for (size_t i = i4; i < n; ++i) flags[i] = int8_t(((keys[i] >> bit) & 1u) ^ 1u);
    }
}

__global__ void split_scatter_kernel(const uint32_t *__restrict__ keys, const int8_t *__restrict__ flags,
                                     const int32_t *__restrict__ f, uint32_t *__restrict__ out, size_t n) {
    const size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint32_t zeros = uint32_t(f[n - 1]) + uint32_t(flags[n - 1]);   // total number of keys whose bit is 0
    const uint32_t fi = uint32_t(f[i]);
    const size_t dest = flags[i] ? size_t(fi) : size_t(i) - fi + zeros;
    out[dest] = keys[i];
}

}  // namespace tcu
