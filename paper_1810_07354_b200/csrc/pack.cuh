// Gather-pack of the selected blocks plus refresh of the running checkpoint
// (Section 4.3, checkpoint step 4): payload[poff[j] ...] := x over block sel[j],
// and z := x on the same block.  Pure byte movement, so elements travel as
// 32-bit patterns and NaN payloads survive bit-exactly.
#pragma once
#include "block_pass.cuh"

namespace scar {

// A group of G lanes copies one selected block, four units per lane and batch,
// with the loads of the next batch issued before the stores of the current one
// (see block_distance for why).
template <typename U, int G>
__device__ __forceinline__ void copy_block_2dst(const U *__restrict__ src, U *__restrict__ d0, U *__restrict__ d1,
                                                uint64_t n, int lane) {
    constexpr uint64_t step = 4 * (uint64_t)G;
    U c[4], nx[4];
    uint64_t u = lane;
    bool have = u < n;
    // Loads are unconditional (a unit past the end re-reads the block's last unit; it is never stored), so that the
    // four of a batch are issued back to back instead of one per branch.
    if (have) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint64_t i = u + (uint64_t)j * G;
            c[j] = ld_stream(src + (i < n ? i : n - 1));
        }
    }
    while (have) {
        const uint64_t un = u + step;
        const bool more = un < n;
        if (more) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint64_t i = un + (uint64_t)j * G;
                nx[j] = ld_stream(src + (i < n ? i : n - 1));
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint64_t i = u + (uint64_t)j * G;
            if (i < n) {
                st_stream(d0 + i, c[j]);
                st_stream(d1 + i, c[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) c[j] = nx[j];
        u = un;
        have = more;
    }
}

template <int G, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_pack_update(const uint32_t *__restrict__ x, uint32_t *__restrict__ z, uint32_t *__restrict__ payload, Geom g,
              const uint32_t *__restrict__ sel, const unsigned long long *__restrict__ poff, unsigned long long k,
              const SaveInfoDev *info) {
    const int lane = threadIdx.x & (G - 1);
    const uint64_t j = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    if (j >= k) return;
    griddep_wait();  // the selection that wrote sel / poff may still be running
    if (info->error || j >= info->k) return;  // a selection that gave up selected nothing that may be copied
    uint64_t beg, len;
    g.range(sel[j], beg, len);
    const uint64_t dst = poff[j];
    if (VEC)
        copy_block_2dst<uint4, G>(reinterpret_cast<const uint4 *>(x + beg), reinterpret_cast<uint4 *>(payload + dst),
                                  reinterpret_cast<uint4 *>(z + beg), len >> 2, lane);
    else
        copy_block_2dst<uint32_t, G>(x + beg, payload + dst, z + beg, len, lane);
}

}  // namespace scar
