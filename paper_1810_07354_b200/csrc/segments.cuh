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
// uint64 key bits occur and clears the selection's state, as k_block_scores
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
                   unsigned long long *key_or, SelState *sel_state, SaveInfoDev *info) {
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
    if (sel_state) sel_state_clear(sel_state, info);
}

// Position of block b in the ascending id list sel[0..k), or -1 when it is not there: a 32-way search, one probe
// per lane and round (every lane of the warp gets the answer).
__device__ __forceinline__ long long find_selected(const uint32_t *__restrict__ sel, unsigned long long k, uint32_t b,
                                                   int lane) {
    unsigned long long lo = 0, n = k;  // candidates sel[lo .. lo + n)
    while (n > 32) {
        const unsigned long long step = (n + 31) / 32, idx = lo + (unsigned long long)lane * step;
        const bool le = idx < lo + n && sel[idx] <= b;  // true for a prefix of the lanes: the list ascends
        const unsigned bal = __ballot_sync(0xffffffffu, le);
        if (bal == 0) return -1;
        const unsigned long long nlo = lo + (unsigned long long)(__popc(bal) - 1) * step;
        n = lo + n - nlo < step ? lo + n - nlo : step;
        lo = nlo;
    }
    const bool eq = (unsigned long long)lane < n && sel[lo + lane] == b;
    const unsigned bal = __ballot_sync(0xffffffffu, eq);
    return bal ? (long long)(lo + __ffs(bal) - 1) : -1;
}

// Gather-pack + cache refresh of the selected blocks of a segmented layout: the warps of a fixed-size grid walk
// the segment table with a grid stride, look every segment's block up in the id list and copy the segments of
// selected blocks.  Unselected segments cost two small loads, and no CTA is launched only to find that it
// has nothing to do.
template <bool VEC>
__global__ void __launch_bounds__(kThreads)
k_pack_segments(const uint32_t *__restrict__ x, uint32_t *__restrict__ z, uint32_t *__restrict__ payload, Geom g,
                Segs sg, const uint32_t *__restrict__ sel, const unsigned long long *__restrict__ poff,
                const SaveInfoDev *info) {
    griddep_wait();  // the selection that wrote sel / poff may still be running
    if (info->error) return;
    const unsigned long long k = info->k;
    const int lane = threadIdx.x & 31;
    const uint64_t n_warps = (uint64_t)gridDim.x * (kThreads / 32);
    for (uint64_t s = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) >> 5; s < sg.n; s += n_warps) {
        const uint32_t b = sg.block[s];
        const long long j = find_selected(sel, k, b, lane);
        if (j < 0) continue;
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
}

// ---- the traditional full checkpoint (k == B) of a segmented layout ---------------
// As k_full_save: every block is saved, so the scoring pass itself writes x to the payload (at the element's own
// offset) and over z, segment by segment; the combine kernel then forms the scores, and one small kernel writes
// the identity id list, the offsets and the result record.  4 N elements move instead of 5 N.
template <typename T, int NORM, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_segment_full_save(const T *__restrict__ x, T *__restrict__ z, T *__restrict__ payload, Geom g, Segs sg,
                    typename Elem<T, NORM>::wide_t *__restrict__ seg_part) {
    const int lane = threadIdx.x & 31;
    const uint64_t s = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const bool valid = s < sg.n;
    uint64_t beg = 0, len = 0;
    if (valid) {
        beg = sg.beg[s];
        len = seg_len(g, sg.block[s], beg);
    }
    typename Elem<T, NORM>::wide_t t = block_distance_save<T, NORM, 32, VEC>(x, z, payload, beg, len, lane);
    if (valid && lane == 0) seg_part[s] = t;
}

// info must have been cleared before the launch (the non-finite count is added up with atomics).
template <typename Sc>
__global__ void __launch_bounds__(kThreads)
k_full_save_ids(Geom g, const Sc *__restrict__ score, uint32_t *__restrict__ sel, unsigned long long *__restrict__ poff,
                SaveInfoDev *info) {
    using SK = ScoreKey<Sc>;
    const uint64_t b = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    if (b >= g.n_blocks) return;
    uint64_t beg, len;
    g.range((uint32_t)b, beg, len);
    sel[b] = (uint32_t)b;
    poff[b] = beg;
    if (SK::nonfinite(SK::key(score[b]))) atomicAdd(&info->nonfinite_blocks, 1ull);
    if (b == g.n_blocks - 1) {
        poff[g.n_blocks] = g.n_elems;
        info->k = g.n_blocks;
        info->payload_elems = g.n_elems;
    }
}

}  // namespace scar
