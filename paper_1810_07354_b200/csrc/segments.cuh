// Layouts with very long blocks (Section 5.1's by-layer partitioning of a
// network: one block per weight or bias tensor, from a few dozen elements to
// many millions).  One group per block would stream a whole layer through a
// single warp, so such layouts are cut into segments of at most kSegElems
// elements: the streaming kernels take one warp per segment and a second, tiny
// kernel adds each block's segment sums in segment order.  The cut depends only
// on the layout, so scores and recovery partials of a block are bit-identical
// and reproducible.
#pragma once
#include "block_pass.cuh"
#include "pack.cuh"
#include "select.cuh"

namespace scar {

constexpr uint64_t kSegElems = 4096;  // 16 KiB per stream and segment (measured: 6.7 TB/s, against 6.1 TB/s with 64 KiB); a multiple of 4 keeps segments 16-byte aligned

struct Segs {
    const uint32_t *block;  // block a segment belongs to
    const uint64_t *beg;    // first element of the segment
    const uint64_t *first;  // B + 1: first segment of every block (blocks own consecutive segments)
    uint64_t n;
};

__device__ __forceinline__ uint64_t seg_len(const Geom &g, uint32_t b, uint64_t sbeg) {
    uint64_t bbeg, blen;
    g.range(b, bbeg, blen);
    const uint64_t rest = bbeg + blen - sbeg;
    return rest < kSegElems ? rest : kSegElems;
}

// Distance sum of every segment (of every lost segment when a block mask is
// given; the others get 0), optionally restoring x := z on it.
template <typename T, int NORM, bool VEC, bool WRITE>
__global__ void __launch_bounds__(kThreads)
k_segment_pass(T *__restrict__ x, const T *__restrict__ z, Geom g, Segs sg, const uint8_t *__restrict__ lost_blocks,
               typename Elem<T, NORM>::wide_t *__restrict__ seg_part) {
    const int lane = threadIdx.x & 31;
    const uint64_t s = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const bool valid = s < sg.n;
    uint64_t beg = 0, len = 0;
    if (valid) {
        const uint32_t b = sg.block[s];
        if (!lost_blocks || lost_blocks[b] != 0) {
            beg = sg.beg[s];
            len = seg_len(g, b, beg);
        }
    }
    typename Elem<T, NORM>::wide_t t = block_distance<T, NORM, 32, VEC, WRITE>(x, z, beg, len, lane);
    if (valid && lane == 0) seg_part[s] = t;
}

// Adds the segment sums of each block in a fixed order and writes the
// (weighted) block score or recovery partial; for scores also records which
// uint64 key bits occur and clears the first radix histogram, as k_block_scores
// does.  Two launches share this code: WIDE = false takes one warp per block
// (lanes add segments l, l + 32, ... in order, then a fixed xor tree) and skips
// blocks with more than kWideSegs segments; WIDE = true takes one CTA per such
// block (threads add segments t, t + 256, ..., then the same tree per warp and
// the warps in order), listed in wide_blocks.
constexpr uint64_t kWideSegs = 256;

template <typename E>
__device__ __forceinline__ void store_block_total(typename E::wide_t t, uint64_t b, const float *__restrict__ weight,
                                                  typename E::score_t *__restrict__ out, unsigned long long *key_or) {
    const typename E::score_t sc = weighted<E>(t, weight, b);
    out[b] = sc;
    if (key_or && sizeof(typename E::score_t) == 8) {
        const unsigned long long bits = (unsigned long long)sc;
        const unsigned long long seen = *reinterpret_cast<volatile unsigned long long *>(key_or);
        if (bits & ~seen) atomicOr(key_or, bits);
    }
}

template <typename T, int NORM, bool WIDE>
__global__ void __launch_bounds__(kThreads)
k_combine_segments(Segs sg, uint64_t n_blocks, const uint32_t *__restrict__ wide_blocks,
                   const typename Elem<T, NORM>::wide_t *__restrict__ seg_part, const float *__restrict__ weight,
                   const uint8_t *__restrict__ lost_blocks, typename Elem<T, NORM>::score_t *__restrict__ out,
                   unsigned long long *key_or, unsigned *hist0, int hist0_len) {
    using E = Elem<T, NORM>;
    using W = typename E::wide_t;
    if (WIDE) {
        __shared__ W sh[kThreads / 32];
        const uint64_t b = wide_blocks[blockIdx.x];
        if (lost_blocks && lost_blocks[b] == 0) return;
        const uint64_t s0 = sg.first[b], s1 = sg.first[b + 1];
        W t = 0;
        for (uint64_t s = s0 + threadIdx.x; s < s1; s += kThreads) t += seg_part[s];
        t = cta_sum<W>(t, sh);
        if (threadIdx.x == 0) store_block_total<E>(t, b, weight, out, key_or);
        return;
    }
    const int lane = threadIdx.x & 31;
    const uint64_t b = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    if (b < n_blocks && (!lost_blocks || lost_blocks[b] != 0)) {
        const uint64_t s0 = sg.first[b], s1 = sg.first[b + 1];
        if (s1 - s0 <= kWideSegs) {
            W t = 0;
            for (uint64_t s = s0 + lane; s < s1; s += 32) t += seg_part[s];
            t = group_sum<32, W>(t);
            if (lane == 0) store_block_total<E>(t, b, weight, out, key_or);
        }
    }
    if (hist0 && blockIdx.x == 0)
        for (int i = threadIdx.x; i < hist0_len; i += kThreads) hist0[i] = 0;
}

// selpos[b] = position of block b in the id list, for the blocks that were selected
// (the rest keep the 0xffffffff the array was filled with).
static __global__ void __launch_bounds__(kThreads)
k_mark_selected(const uint32_t *__restrict__ sel, const SaveInfoDev *info, uint32_t *__restrict__ selpos) {
    const unsigned long long j = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
    if (j < info->k) selpos[sel[j]] = (uint32_t)j;
}

// Gather-pack + cache refresh, one warp per segment of a selected block.
template <bool VEC>
__global__ void __launch_bounds__(kThreads)
k_pack_segments(const uint32_t *__restrict__ x, uint32_t *__restrict__ z, uint32_t *__restrict__ payload, Geom g,
                Segs sg, const uint32_t *__restrict__ selpos, const unsigned long long *__restrict__ poff) {
    const int lane = threadIdx.x & 31;
    const uint64_t s = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    if (s >= sg.n) return;
    const uint32_t b = sg.block[s];
    const uint32_t j = selpos[b];
    if (j == 0xffffffffu) return;
    uint64_t bbeg, blen;
    g.range(b, bbeg, blen);
    const uint64_t beg = sg.beg[s];
    const uint64_t rest = bbeg + blen - beg;
    const uint64_t len = rest < kSegElems ? rest : kSegElems;
    const uint64_t dst = poff[j] + (beg - bbeg);
    if (VEC)
        copy_block_2dst<uint4, 32>(reinterpret_cast<const uint4 *>(x + beg), reinterpret_cast<uint4 *>(payload + dst),
                                   reinterpret_cast<uint4 *>(z + beg), len >> 2, lane);
    else
        copy_block_2dst<uint32_t, 32>(x + beg, payload + dst, z + beg, len, lane);
}

}  // namespace scar
