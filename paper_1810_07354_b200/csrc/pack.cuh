// Gather-pack of the selected blocks plus refresh of the running checkpoint
// (Section 4.3, checkpoint step 4): payload[poff[j] ...] := x over block sel[j],
// and z := x on the same block.  Pure byte movement, so elements travel as
// 32-bit patterns and NaN payloads survive bit-exactly.
#pragma once
#include "block_pass.cuh"

namespace scar {

template <int G, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_pack_update(const uint32_t *__restrict__ x, uint32_t *__restrict__ z, uint32_t *__restrict__ payload, Geom g,
              const uint32_t *__restrict__ sel, const unsigned long long *__restrict__ poff, unsigned long long k) {
    const int lane = threadIdx.x & (G - 1);
    const uint64_t j = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    if (j >= k) return;
    uint64_t beg, len;
    g.range(sel[j], beg, len);
    const uint64_t dst = poff[j];
    if (VEC) {
        const uint4 *xv = reinterpret_cast<const uint4 *>(x + beg);
        uint4 *zv = reinterpret_cast<uint4 *>(z + beg);
        uint4 *pv = reinterpret_cast<uint4 *>(payload + dst);
        const uint64_t nvec = len >> 2;
        uint64_t v = lane;
        for (; v + 3 * G < nvec; v += 4 * G) {
            uint4 a = ld_stream(xv + v), b = ld_stream(xv + v + G), c = ld_stream(xv + v + 2 * G),
                  d = ld_stream(xv + v + 3 * G);
            st_stream(pv + v, a); st_stream(pv + v + G, b); st_stream(pv + v + 2 * G, c); st_stream(pv + v + 3 * G, d);
            st_stream(zv + v, a); st_stream(zv + v + G, b); st_stream(zv + v + 2 * G, c); st_stream(zv + v + 3 * G, d);
        }
        for (; v < nvec; v += G) {
            uint4 a = ld_stream(xv + v);
            st_stream(pv + v, a);
            st_stream(zv + v, a);
        }
    } else {
        const uint32_t *xs = x + beg;
        uint32_t *zs = z + beg, *ps = payload + dst;
        uint64_t i = lane;
        for (; i + 3 * G < len; i += 4 * G) {
            uint32_t a = ld_stream(xs + i), b = ld_stream(xs + i + G), c = ld_stream(xs + i + 2 * G),
                     d = ld_stream(xs + i + 3 * G);
            ps[i] = a; ps[i + G] = b; ps[i + 2 * G] = c; ps[i + 3 * G] = d;
            zs[i] = a; zs[i + G] = b; zs[i + 2 * G] = c; zs[i + 3 * G] = d;
        }
        for (; i < len; i += G) {
            uint32_t a = ld_stream(xs + i);
            ps[i] = a;
            zs[i] = a;
        }
    }
}

}  // namespace scar
