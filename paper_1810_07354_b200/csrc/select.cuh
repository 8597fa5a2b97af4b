// Top-k block selection (Section 4.3, checkpoint step 3: the fraction r of
// parameters with the largest distances) as an exact radix select with a
// deterministic tie-break: among blocks whose score equals the k-th largest,
// the lowest block ids win.  Output is the ascending id list sel[k] and the
// payload offsets poff[k+1].
//
// Keys are order-preserving unsigned integers: the bit pattern of a
// non-negative float32 score (NaN and +Inf both map to the +Inf pattern, so
// such blocks rank first), or the uint64 l1 score itself.
//
// The whole selection is ONE kernel, because the score array is small (4-8 bytes per block) and a chain of
// dependent launches costs more than the work itself.  Each CTA owns a contiguous range of 4096-key tiles.
// Three forms:
//   k_select_tile<S, true>    at most one tile in all: a single CTA, launched plainly, whose histograms never
//                             leave shared memory
//   k_select_tile<S, false>   one tile per CTA (up to about 600 000 blocks on a 148-SM device), launched
//                             cooperatively so that every CTA is resident; keys are loaded once and stay in
//                             shared memory
//   k_select<S>               several tiles per CTA, also cooperative; keys are re-read from the score array
// The CTAs meet at few points, and at each of them a CTA pays for as few dependent trips to the L2 cache as
// possible:
//
//   digit passes   most-significant digit first: shared-memory histogram of the keys that match the prefix so
//                  far, flushed with integer reductions; every CTA resolves the digit from the global
//                  histogram (the same small scan in every CTA).  k_select_tile knows how many keys a pass
//                  counts and simply re-reads the histogram until its bins add up to that number; k_select
//                  meets at one arrival counter per pass (fire-and-forget increment, then an acquiring poll).
//                  Digits that are zero in every uint64 key are skipped.
//   exchange       with the threshold key tau and `need` (how many keys equal to tau are taken) every CTA
//                  publishes one record: how many of its keys lie above / at tau and their summed lengths.
//                  A record's words hold value + 1, so a word that reads non-zero has arrived: no fence, no
//                  flag.  Thread c of every CTA waits for the record of CTA c, and a CTA-wide scan of the
//                  records gives the CTA its output bases and the totals.  This one step stands for a
//                  barrier, the per-CTA counts and their prefix sums.
//   boundary       only when the tau-keys run out inside one CTA's range and block lengths differ: the CTAs
//                  after it recompute, from that CTA's keys, the summed length of the tau-blocks it takes
//   emit           ordered compaction into sel[] / poff[]
//
// Every wait is bounded: a CTA that gives up records an error and leaves, the others see it and leave too, and
// the host reports SCAR_ERR_TIMEOUT.  The counters, histograms and records must be zero when the kernel starts
// (sel_state_clear, run by the kernel that precedes it on the stream, or a memset); the kernel never has to put
// them back.
#pragma once
#include "block_pass.cuh"
#include "sel_state.cuh"

namespace scar {

// Digit plan per key width: 11/11/10 bits for 32-bit keys, 11/11/11/11/10/10 for 64-bit keys.
template <typename K> struct KeyTraits;
template <> struct KeyTraits<unsigned> {
    static constexpr int kPasses = 3;
    static constexpr bool kSkippable = false;
    __host__ __device__ static constexpr int shift(int p) { return p == 0 ? 21 : (p == 1 ? 10 : 0); }
    __host__ __device__ static constexpr int width(int p) { return p == 2 ? 10 : 11; }
};
template <> struct KeyTraits<unsigned long long> {
    static constexpr int kPasses = 6;
    static constexpr bool kSkippable = true;
    __host__ __device__ static constexpr int shift(int p) {
        return p == 0 ? 53 : p == 1 ? 42 : p == 2 ? 31 : p == 3 ? 20 : p == 4 ? 10 : 0;
    }
    __host__ __device__ static constexpr int width(int p) { return p >= 4 ? 10 : 11; }
};

// What is ranked -> its order-preserving unsigned key.
template <typename S> struct ScoreKey;
template <> struct ScoreKey<float> {  // squared l2 scores
    using K = unsigned;
    static __device__ __forceinline__ K key(float s) {
        unsigned u = __float_as_uint(s) & 0x7fffffffu;
        return u > 0x7f800000u ? 0x7f800000u : u;
    }
    static __device__ __forceinline__ bool nonfinite(K k) { return k == 0x7f800000u; }
};
template <> struct ScoreKey<unsigned long long> {  // integer l1 scores
    using K = unsigned long long;
    static __device__ __forceinline__ K key(unsigned long long s) { return s; }
    static __device__ __forceinline__ bool nonfinite(K) { return false; }
};
template <> struct ScoreKey<unsigned> {  // caller-supplied 32-bit priorities (random strategy)
    using K = unsigned;
    static __device__ __forceinline__ K key(unsigned s) { return s; }
    static __device__ __forceinline__ bool nonfinite(K) { return false; }
};

// The selection kernels run every instruction once, and their time is close to the number of instructions a warp
// issues.  Combining the per-warp partials of a CTA-wide sum or scan with a loop over shared memory costs four
// instructions per warp of the CTA; here every warp takes one partial per lane and combines them with shuffles.
//
// Exclusive prefix, for the calling thread's warp, of the NW per-warp partials in sh[]; *total gets their sum.
template <typename W, int NW>
__device__ __forceinline__ W warp_partials(const W *sh, W *total) {
    static_assert(NW <= 32 && (NW & (NW - 1)) == 0, "one partial per lane");
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const W v = lane < NW ? sh[lane] : W(0);
    W inc = v;
#pragma unroll
    for (int o = 1; o < NW; o <<= 1) {
        const W n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (total) *total = __shfl_sync(0xffffffffu, inc, NW - 1);
    return __shfl_sync(0xffffffffu, inc - v, w);
}

// Exclusive prefix sum of one value per thread over a CTA of kSelThreads threads; *total gets the sum.
template <typename W>
__device__ __forceinline__ W sel_excl_scan(W v, W *sh /*kSelThreads / 32*/, W *total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    W inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const W n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();
    if (lane == 31) sh[w] = inc;
    __syncthreads();
    return warp_partials<W, kSelThreads / 32>(sh, total) + inc - v;
}

// Sums N values per thread over the CTA with one pair of barriers.  sh holds N * NT / 32 words.
template <int N, int NT = kThreads>
__device__ __forceinline__ void cta_sum_n(unsigned long long (&v)[N], unsigned long long *sh) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = group_sum<32, unsigned long long>(v[i]);
    __syncthreads();
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < N; ++i) sh[w * N + i] = v[i];
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = group_sum<32, unsigned long long>(lane < NT / 32 ? sh[lane * N + i] : 0ull);
}

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(__cvta_generic_to_global(p)) : "memory");
    return v;
}

// Polls *word until it reaches target.  False when the wait was abandoned: after kSpinLimit polls, or as soon
// as another CTA has recorded an error.
__device__ __forceinline__ bool spin_until_at_least(const unsigned *word, unsigned target, const SelState *st) {
    unsigned tries = 0;
    while (ld_acquire(word) < target) {
        ++tries;
        if (tries > kSpinLimit || ((tries & 255u) == 0 && ld_acquire(&st->error) != 0)) return false;
        if (tries > 16) __nanosleep(tries > 4096 ? 256 : 32);
    }
    return true;
}

// Publishes this CTA's record (see SelRecord: value + 1 per word, no fence).
__device__ __forceinline__ void rec_publish(SelRecord *r, unsigned c_gt, unsigned c_eq, unsigned c_nf,
                                            unsigned long long len_gt, unsigned long long len_eq) {
    *reinterpret_cast<volatile unsigned long long *>(&r->len_gt) = len_gt + 1;
    *reinterpret_cast<volatile unsigned long long *>(&r->len_eq) = len_eq + 1;
    *reinterpret_cast<volatile unsigned *>(&r->c_gt) = c_gt + 1;
    *reinterpret_cast<volatile unsigned *>(&r->c_eq) = c_eq + 1;
    *reinterpret_cast<volatile unsigned *>(&r->c_nf) = c_nf + 1;
}

// Waits (with the usual bound) until the record of a CTA has arrived and returns its values; the lengths only when
// asked for.  False when the wait was abandoned.
__device__ __forceinline__ bool rec_take(const SelRecord *r, bool want_lens, const SelState *st, unsigned &c_gt,
                                         unsigned &c_eq, unsigned &c_nf, unsigned long long &len_gt,
                                         unsigned long long &len_eq) {
    unsigned tries = 0;
    for (;;) {
        unsigned x, y, z;  // the fourth word of the vector is padding
        asm volatile("{ .reg .u32 pad; ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, pad}, [%3]; }"
                     : "=r"(x), "=r"(y), "=r"(z)
                     : "l"(__cvta_generic_to_global(r))
                     : "memory");
        unsigned long long lg = 1, le = 1;
        if (want_lens) {
            lg = *reinterpret_cast<const volatile unsigned long long *>(&r->len_gt);
            le = *reinterpret_cast<const volatile unsigned long long *>(&r->len_eq);
        }
        if (x && y && z && lg && le) {
            c_gt = x - 1, c_eq = y - 1, c_nf = z - 1, len_gt = lg - 1, len_eq = le - 1;
            return true;
        }
        ++tries;
        if (tries > kSpinLimit || ((tries & 255u) == 0 && ld_acquire(&st->error) != 0)) return false;
        if (tries > 16) __nanosleep(tries > 4096 ? 256 : 32);
    }
}

__device__ __forceinline__ void sel_fail(SelState *st, SaveInfoDev *info) {
    atomicExch(&st->error, 1u);
    *reinterpret_cast<volatile unsigned long long *>(&info->error) = 1ull;
    __threadfence();
}

// Arrival at the meeting point after a digit pass: every CTA adds one to *ctr and waits until `target` CTAs
// have.  What the CTA's threads wrote before (their histogram updates) is visible to every CTA that gets past
// the wait.  Returns false when the wait was abandoned (it cannot happen while all CTAs are resident, which a
// cooperative launch guarantees; the bound is there so that nothing can hang).
__device__ __forceinline__ bool sel_arrive_wait(unsigned *ctr, unsigned target, SelState *st, SaveInfoDev *info,
                                                int *sh_ok) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(ctr, 1u);  // result unused: a reduction, nothing to wait for
        const bool good = spin_until_at_least(ctr, target, st);
        if (!good) sel_fail(st, info);
        *sh_ok = good;
    }
    __syncthreads();
    return *sh_ok != 0;
}

// Resolves one digit: scanning bins from the highest down, finds the bin d with
//   count(bins > d) < remaining <= count(bins >= d)
// and returns it; remaining becomes the rank wanted inside bin d.
template <int WIDTH>
__device__ __forceinline__ unsigned resolve_digit_w(const unsigned *hist, unsigned long long &remaining,
                                                    unsigned long long *sh_scan, unsigned long long *sh_out) {
    constexpr int nb = 1 << WIDTH;
    constexpr int per = nb / kSelThreads;  // 4 or 2 consecutive bins per thread, highest bins in thread 0
    static_assert(per == 4 || per == 2, "one vector load per thread");
    unsigned local[per];
    const unsigned *src = hist + (nb - (int)(threadIdx.x + 1) * per);
    if (per == 4) {
        const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(src));
        local[0] = v.w; local[1] = v.z; local[per - 2] = v.y; local[per - 1] = v.x;
    } else {
        const uint2 v = __ldcg(reinterpret_cast<const uint2 *>(src));
        local[0] = v.y; local[1] = v.x;
    }
    unsigned long long sum = 0;
#pragma unroll
    for (int i = 0; i < per; ++i) sum += local[i];
    unsigned long long cum = sel_excl_scan<unsigned long long>(sum, sh_scan, nullptr);
#pragma unroll
    for (int i = 0; i < per; ++i) {
        unsigned long long h = local[i];
        if (cum < remaining && remaining <= cum + h) {
            sh_out[0] = (unsigned long long)(nb - 1 - ((int)threadIdx.x * per + i));
            sh_out[1] = remaining - cum;
        }
        cum += h;
    }
    __syncthreads();
    remaining = sh_out[1];
    unsigned d = (unsigned)sh_out[0];
    __syncthreads();
    return d;
}

__device__ __forceinline__ unsigned resolve_digit(const unsigned *hist, int width, unsigned long long &remaining,
                                                  unsigned long long *sh_scan, unsigned long long *sh_out) {
    return width == 11 ? resolve_digit_w<11>(hist, remaining, sh_scan, sh_out)
                       : resolve_digit_w<10>(hist, remaining, sh_scan, sh_out);
}

// Keys of the kSelPerThread consecutive blocks a thread owns in a tile (first = index of the first of them);
// bit j of valid says block first + j exists.
template <typename S>
__device__ __forceinline__ void load_keys(const S *__restrict__ score, unsigned long long n_blocks,
                                          unsigned long long first, typename ScoreKey<S>::K (&key)[kSelPerThread],
                                          unsigned &valid) {
    using SK = ScoreKey<S>;
    static_assert(kSelPerThread == 8 && (sizeof(S) == 4 || sizeof(S) == 8), "vector loads below");
    if (first + kSelPerThread <= n_blocks && (reinterpret_cast<uintptr_t>(score) & 15) == 0) {
        S raw[kSelPerThread];
        uint4 *dst = reinterpret_cast<uint4 *>(raw);
        const uint4 *src = reinterpret_cast<const uint4 *>(score + first);
#pragma unroll
        for (int i = 0; i < (int)(sizeof(S) * kSelPerThread / 16); ++i) dst[i] = src[i];
#pragma unroll
        for (int j = 0; j < kSelPerThread; ++j) key[j] = SK::key(raw[j]);
        valid = 0xffu;
        return;
    }
    valid = 0;
#pragma unroll
    for (int j = 0; j < kSelPerThread; ++j) {
        key[j] = 0;
        if (first + j < n_blocks) {
            key[j] = SK::key(score[first + j]);
            valid |= 1u << j;
        }
    }
}

// Length of every block of an implicit layout when they are all the same, else 0.
__device__ __forceinline__ unsigned long long uniform_block_len(const Geom &g) {
    if (g.boff) return 0;
    if (g.blocks_per_row == 1) return g.row_len;
    return g.row_len % g.block_elems == 0 ? (unsigned long long)g.block_elems : 0ull;
}

// Summed length of the first `take` blocks (in id order) of CTA cb's tile range whose key equals tau.
template <typename S>
__device__ __forceinline__ unsigned long long boundary_len(const S *__restrict__ score, const Geom &g, unsigned cb,
                                                           unsigned tiles_per_cta, unsigned n_tiles,
                                                           typename ScoreKey<S>::K tau, unsigned long long take,
                                                           unsigned long long *sh_scan, unsigned long long *sh_red) {
    typedef unsigned long long u64;
    using K = typename ScoreKey<S>::K;
    const u64 ulen = uniform_block_len(g);
    if (ulen) return take * ulen;
    const unsigned t_lo = cb * tiles_per_cta;
    const unsigned t_hi = t_lo + tiles_per_cta < n_tiles ? t_lo + tiles_per_cta : n_tiles;
    u64 run = 0;
    u64 pl[1] = {0};
    for (unsigned t = t_lo; t < t_hi; ++t) {
        K key[kSelPerThread];
        unsigned valid;
        const u64 first = (u64)t * kSelTile + (u64)threadIdx.x * kSelPerThread;
        load_keys<S>(score, g.n_blocks, first, key, valid);
        unsigned eq_bits = 0;
#pragma unroll
        for (int j = 0; j < kSelPerThread; ++j)
            if ((valid >> j & 1u) && key[j] == tau) eq_bits |= 1u << j;
        u64 tot;
        u64 rank = run + sel_excl_scan<u64>(__popc(eq_bits), sh_scan, &tot);
        run += tot;
        for (int j = 0; j < kSelPerThread; ++j)
            if (eq_bits >> j & 1u) {
                if (rank < take) {
                    uint64_t beg, len;
                    g.range((uint32_t)(first + j), beg, len);
                    pl[0] += len;
                }
                ++rank;
            }
    }
    cta_sum_n<1, kSelThreads>(pl, sh_red);
    return pl[0];
}

// The general form: every CTA owns a contiguous range of tiles and re-reads their keys in every phase (used when
// there are more tiles than SMs; k_select_tile below is the form for one tile per CTA).  never != 0 (self-test
// only) makes every wait expect one arrival more than there are CTAs, so that it runs out.
template <typename S>
__global__ void __launch_bounds__(kSelThreads, 1)
k_select(const S *__restrict__ score, Geom g, unsigned long long k, SelState *st, SaveInfoDev *info,
         uint32_t *__restrict__ sel, unsigned long long *__restrict__ poff, unsigned n_tiles, unsigned tiles_per_cta,
         unsigned never) {
    using SK = ScoreKey<S>;
    using K = typename SK::K;
    using KT = KeyTraits<K>;
    typedef unsigned long long u64;
    __shared__ unsigned sh_hist[kHistBins];
    __shared__ u64 sh_scan[kSelThreads / 32];
    __shared__ u64 sh_out[2];
    __shared__ u64 sh_red[6 * kSelThreads / 32];
    __shared__ int sh_boundary;
    __shared__ u64 sh_boundary_take;
    __shared__ int sh_ok;

    griddep_launch();  // the pack kernel may be scheduled while this one runs; it waits before reading sel / poff
    SEL_STAMP(st, 0);
    const u64 B = g.n_blocks;
    const unsigned t_lo = blockIdx.x * tiles_per_cta;
    const unsigned t_hi = t_lo + tiles_per_cta < n_tiles ? t_lo + tiles_per_cta : n_tiles;
    const bool none = k == 0;
    const u64 key_or = KT::kSkippable ? st->key_or : ~0ull;  // put back to 0 after the exchange
    const u64 ulen = uniform_block_len(g);
    // Every walk over the CTA's tiles has the next tile's keys on their way while this tile's are worked on: one
    // CTA per SM keeps few loads in flight otherwise.
    K key[kSelPerThread], ahead[kSelPerThread];
    unsigned valid = 0, valid_ahead = 0;
    const u64 mine0 = (u64)threadIdx.x * kSelPerThread;
    for (int i = threadIdx.x; i < kHistBins; i += kSelThreads) sh_hist[i] = 0;
    if (threadIdx.x == 0) {
        sh_boundary = -1;
        sh_boundary_take = 0;
    }
    __syncthreads();
    SEL_STAMP(st, 1);  // keys loaded
    bool alive = true;

    // ---- digit passes: tau = the k-th largest key, need = how many keys equal to tau are taken
    u64 prefix = 0, need = k;
    if (!none) {
        for (int p = 0; p < KT::kPasses && alive; ++p) {
            const int shift = KT::shift(p), width = KT::width(p);
            const u64 mask = (1ull << width) - 1;
            if (KT::kSkippable && ((key_or >> shift) & mask) == 0) {  // this digit is 0 in every key
                prefix <<= width;
                continue;
            }
            if (t_lo < t_hi) load_keys<S>(score, B, (u64)t_lo * kSelTile + mine0, ahead, valid_ahead);
            for (unsigned t = t_lo; t < t_hi; ++t) {
#pragma unroll
                for (int j = 0; j < kSelPerThread; ++j) key[j] = ahead[j];
                valid = valid_ahead;
                if (t + 1 < t_hi) load_keys<S>(score, B, (u64)(t + 1) * kSelTile + mine0, ahead, valid_ahead);
#pragma unroll
                for (int j = 0; j < kSelPerThread; ++j) {
                    const bool match = p == 0 || ((u64)key[j] >> (shift + width)) == prefix;
                    if ((valid >> j & 1u) && match) atomicAdd(&sh_hist[(unsigned)(((u64)key[j] >> shift) & mask)], 1u);
                }
            }
            __syncthreads();
            SEL_STAMP(st, 2 + 4 * p);  // pass p: shared histogram built
            for (int i = threadIdx.x; i < (1 << width); i += kSelThreads) {
                const unsigned c = sh_hist[i];
                if (c) {
                    atomicAdd(&st->hist[p][i], c);
                    sh_hist[i] = 0;  // ready for the next pass
                }
            }
            SEL_STAMP(st, 3 + 4 * p);  // flushed
            alive = sel_arrive_wait(&st->arrive[p], gridDim.x + never, st, info, &sh_ok);
            SEL_STAMP(st, 4 + 4 * p);  // every CTA has arrived
            if (alive) prefix = (prefix << width) | resolve_digit(st->hist[p], width, need, sh_scan, sh_out);
            SEL_STAMP(st, 5 + 4 * p);  // digit resolved
        }
    }
    const K tau = (K)prefix;

    // ---- this CTA's record: counts and summed lengths of its keys above / at tau
    u64 my_eq = 0;
    if (alive) {
        u64 five[5] = {0, 0, 0, 0, 0};  // c_gt, c_eq, c_nf, len_gt, len_eq
        if (t_lo < t_hi) load_keys<S>(score, B, (u64)t_lo * kSelTile + mine0, ahead, valid_ahead);
        for (unsigned t = t_lo; t < t_hi; ++t) {
            const u64 first = (u64)t * kSelTile + mine0;
#pragma unroll
            for (int j = 0; j < kSelPerThread; ++j) key[j] = ahead[j];
            valid = valid_ahead;
            if (t + 1 < t_hi) load_keys<S>(score, B, (u64)(t + 1) * kSelTile + mine0, ahead, valid_ahead);
#pragma unroll
            for (int j = 0; j < kSelPerThread; ++j) {
                if (!(valid >> j & 1u)) continue;
                if (SK::nonfinite(key[j])) ++five[2];
                if (none || key[j] < tau) continue;
                uint64_t beg, len = 0;
                if (!ulen) g.range((uint32_t)(first + j), beg, len);  // one block length: lengths are counts
                if (key[j] > tau) {
                    ++five[0];
                    five[3] += len;
                } else {
                    ++five[1];
                    five[4] += len;
                }
            }
        }
        cta_sum_n<5, kSelThreads>(five, sh_red);
        if (ulen) five[3] = five[0] * ulen, five[4] = five[1] * ulen;
        my_eq = five[1];
        SEL_STAMP(st, 26);  // own counts known
        if (threadIdx.x == 0) {
            rec_publish(&st->rec[blockIdx.x], (unsigned)five[0], (unsigned)five[1], (unsigned)five[2], five[3], five[4]);
        }
    }

    // ---- exchange: thread c takes the record of CTA c; one scan gives this CTA its bases and the totals
    u64 my_eq_before = 0, my_sel_base = 0, my_len_base = 0, total_n = 0, total_l = 0, total_nf = 0;
    int cb = -1;
    if (alive) {
        const unsigned c = threadIdx.x;
        u64 e = 0, gt = 0, nf = 0, lg = 0, le = 0;
        bool ok = true;
        if (c < gridDim.x + never) {
            unsigned e32 = 0, gt32 = 0, nf32 = 0;
            ok = rec_take(&st->rec[c], true, st, gt32, e32, nf32, lg, le);
            e = e32, gt = gt32, nf = nf32;
            if (!ok) sel_fail(st, info);
        }
        alive = __syncthreads_and(ok) != 0;
        SEL_STAMP(st, 27);  // every CTA's record read
        if (alive) {
            const u64 ex = sel_excl_scan<u64>(e, sh_scan, nullptr);
            u64 take = need > ex ? need - ex : 0;
            if (take > e) take = e;
            if (take != 0 && take != e) {  // the tau-keys run out inside CTA c's range
                sh_boundary = (int)c;
                sh_boundary_take = take;
            }
            const u64 n = gt + take;
            const u64 l = lg + (take == e ? le : 0);
            const bool mine = c < blockIdx.x;
            u64 six[6] = {mine ? e : 0, mine ? n : 0, mine ? l : 0, n, l, nf};
            cta_sum_n<6, kSelThreads>(six, sh_red);
            my_eq_before = six[0], my_sel_base = six[1], my_len_base = six[2];
            total_n = six[3], total_l = six[4], total_nf = six[5];
            cb = sh_boundary;  // written before the barriers inside cta_sum_n
        }
    }

    // ---- boundary: the CTAs behind the one where the tau-keys run out need the length of what it takes
    if (alive && cb >= 0 && (int)blockIdx.x >= cb) {
        const u64 pl = boundary_len<S>(score, g, (unsigned)cb, tiles_per_cta, n_tiles, tau, sh_boundary_take, sh_scan,
                                       sh_red);
        total_l += pl;
        if ((int)blockIdx.x > cb) my_len_base += pl;
    }

    SEL_STAMP(st, 28);  // bases known
    // ---- emit: ordered compaction of this CTA's tiles
    if (alive && !none) {
        // Keys equal to tau: this CTA takes all of its own, none of them, or (one CTA at most) the first few; only
        // that CTA has to rank them tile by tile.
        const bool take_none = need <= my_eq_before, take_all = need >= my_eq_before + my_eq;
        u64 run_eq = my_eq_before, pos_base = my_sel_base, off_base = my_len_base;
        if (t_lo < t_hi) load_keys<S>(score, B, (u64)t_lo * kSelTile + mine0, ahead, valid_ahead);
        for (unsigned t = t_lo; t < t_hi; ++t) {
            const u64 first = (u64)t * kSelTile + mine0;
#pragma unroll
            for (int j = 0; j < kSelPerThread; ++j) key[j] = ahead[j];
            valid = valid_ahead;
            if (t + 1 < t_hi) load_keys<S>(score, B, (u64)(t + 1) * kSelTile + mine0, ahead, valid_ahead);
            unsigned gt_bits = 0, eq_bits = 0;
#pragma unroll
            for (int j = 0; j < kSelPerThread; ++j)
                if (valid >> j & 1u) {
                    if (key[j] > tau) gt_bits |= 1u << j;
                    else if (key[j] == tau) eq_bits |= 1u << j;
                }
            unsigned take_bits = gt_bits;
            if (take_all) {
                take_bits |= eq_bits;
            } else if (!take_none) {
                u64 tot_eq;
                u64 rank = run_eq + sel_excl_scan<u64>(__popc(eq_bits), sh_scan, &tot_eq);
                for (int j = 0; j < kSelPerThread; ++j)
                    if (eq_bits >> j & 1u) {
                        if (rank < need) take_bits |= 1u << j;
                        ++rank;
                    }
                run_eq += tot_eq;
            }
            if (ulen) {  // one block length: an offset is a position times that length
                u64 tot;
                u64 pos = pos_base + sel_excl_scan<u64>(__popc(take_bits), sh_scan, &tot);
#pragma unroll
                for (int j = 0; j < kSelPerThread; ++j)
                    if (take_bits >> j & 1u) {
                        sel[pos] = (uint32_t)(first + j);
                        poff[pos] = pos * ulen;
                        ++pos;
                    }
                pos_base += tot;
                continue;
            }
            u64 lens[kSelPerThread];
            u64 lsum = 0;
#pragma unroll
            for (int j = 0; j < kSelPerThread; ++j) {
                lens[j] = 0;
                if (take_bits >> j & 1u) {
                    uint64_t beg, len;
                    g.range((uint32_t)(first + j), beg, len);
                    lens[j] = len;
                    lsum += len;
                }
            }
            // one scan for both outputs: block counts in the top 16 bits (at most 4096 per tile), summed
            // lengths below (a buffer has fewer than 2^48 elements: init rejects more)
            u64 tot_both;
            const u64 both =
                sel_excl_scan<u64>(((u64)__popc(take_bits) << 48) | lsum, sh_scan, &tot_both);
            u64 pos = pos_base + (both >> 48);
            u64 off = off_base + (both & ((1ull << 48) - 1));
#pragma unroll
            for (int j = 0; j < kSelPerThread; ++j)
                if (take_bits >> j & 1u) {
                    sel[pos] = (uint32_t)(first + j);
                    poff[pos] = off;
                    ++pos;
                    off += lens[j];
                }
            pos_base += tot_both >> 48;
            off_base += tot_both & ((1ull << 48) - 1);
        }
    }
    SEL_STAMP(st, 29);  // emitted
    // The last CTA lies behind every boundary, so its totals are complete.  By now every CTA has read key_or.
    if (alive && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
        info->k = total_n;
        info->payload_elems = total_l;
        info->nonfinite_blocks = total_nf;
        poff[total_n] = total_l;
        if (KT::kSkippable) st->key_or = 0;  // forget which uint64 key bits were seen
    }
}

// ---- the same selection when every CTA owns exactly one tile -----------------------
//
// This is the form that runs for up to kSelTile * (number of SMs) blocks.  The kernel is a chain of short
// phases that each run once, so its time is latency: trips to L2, CTA barriers, and fetching code that has not
// run yet.  Hence: a thread's keys sit in (padded, conflict-free) shared memory and the loops over them are not
// unrolled, which keeps the code short; counts travel as 32-bit words and are added with the warp-reduce
// instruction; one packed scan over the CTAs' records gives all prefix sums; and layouts whose blocks all have
// one length skip every sum of lengths.
//
// A digit pass needs no arrival counter here.  Every CTA knows how many keys take part in the pass (all of them in
// the first, afterwards the count of the bin resolved before), and the global histogram only grows: a CTA re-reads
// the histogram until its bins add up to that number, and then every bin it read has its final value.  The
// reading that finds the histogram complete is also the one the digit is resolved from, so the wait costs no
// fence, no atomic with a dependent poll and no second read.  expected + 1 can never be reached (self-test).
constexpr unsigned kHistPollLimit = 1u << 19;  // polls of about half a microsecond each, sleeping 64 ns between them

//
// LOCAL: the histogram is the CTA's own, in shared memory and already complete (a selection that one CTA does
// alone); the first reading resolves the digit, and the bins are put back to zero for the next pass.
template <int WIDTH, bool LOCAL>
__device__ __forceinline__ bool resolve_digit_when_complete(unsigned *hist, unsigned expected, unsigned &remaining,
                                                            unsigned &digit, unsigned &bin_count, const SelState *st,
                                                            unsigned (*sh_w)[kSelThreads / 32], unsigned *sh_out,
                                                            int *sh_stop) {
    constexpr int nb = 1 << WIDTH;
    constexpr int per = nb / kSelThreads;  // 4 or 2 consecutive bins per thread, highest bins in thread 0
    constexpr int kWarps = kSelThreads / 32;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned *src = hist + (nb - (int)(threadIdx.x + 1) * per);
    unsigned local[4] = {0, 0, 0, 0};
    unsigned sum = 0;
    for (unsigned iter = 0;; ++iter) {
        if (LOCAL) {
            if (per == 4) {
                const uint4 v = *reinterpret_cast<const uint4 *>(src);
                local[0] = v.w, local[1] = v.z, local[2] = v.y, local[3] = v.x;
                *reinterpret_cast<uint4 *>(src) = make_uint4(0u, 0u, 0u, 0u);
            } else {
                const uint2 v = *reinterpret_cast<const uint2 *>(src);
                local[0] = v.y, local[1] = v.x;
                *reinterpret_cast<uint2 *>(src) = make_uint2(0u, 0u);
            }
        } else if (per == 4) {
            unsigned a, b, c, d;
            asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(a), "=r"(b), "=r"(c), "=r"(d)
                         : "l"(__cvta_generic_to_global(src))
                         : "memory");
            local[0] = d, local[1] = c, local[2] = b, local[3] = a;
        } else {
            unsigned a, b;
            asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];"
                         : "=r"(a), "=r"(b)
                         : "l"(__cvta_generic_to_global(src))
                         : "memory");
            local[0] = b, local[1] = a;
        }
        sum = (local[0] + local[1]) + (local[2] + local[3]);
        const unsigned wsum = __reduce_add_sync(0xffffffffu, sum);
        unsigned *buf = sh_w[iter & 1];  // two buffers: a fast warp may already write the next round's sums
        if (lane == 0) buf[w] = wsum;
        if (threadIdx.x == 0)
            sh_stop[iter & 1] = iter > kHistPollLimit || ((iter & 63u) == 63u && ld_acquire(&st->error) != 0);
        __syncthreads();
        unsigned total;
        const unsigned before = warp_partials<unsigned, kWarps>(buf, &total);
        if (total == expected) {
            // exclusive prefix of this thread's bins, highest bins first: warps before, lanes before
            unsigned inc = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += n;
            }
            unsigned cum = before + inc - sum;
#pragma unroll
            for (int i = 0; i < per; ++i) {
                const unsigned h = local[i];
                if (cum < remaining && remaining <= cum + h) {
                    sh_out[0] = (unsigned)(nb - 1 - ((int)threadIdx.x * per + i));
                    sh_out[1] = remaining - cum;
                    sh_out[2] = h;
                }
                cum += h;
            }
            __syncthreads();
            digit = sh_out[0];
            remaining = sh_out[1];
            bin_count = sh_out[2];
            return true;  // the next write to sh_out / sh_w comes after further barriers
        }
        if (sh_stop[iter & 1]) return false;  // two buffers, as for the sums
        if (iter > 8) __nanosleep(64);
    }
}

// SOLO: the whole selection is this one CTA's (at most kSelTile blocks): histograms stay in shared memory and
// nothing is exchanged through global memory.
template <typename S, bool SOLO>
__global__ void __launch_bounds__(kSelThreads, 1)
k_select_tile(const S *__restrict__ score, Geom g, unsigned k, SelState *st, SaveInfoDev *info,
              uint32_t *__restrict__ sel, unsigned long long *__restrict__ poff, unsigned never) {
    using SK = ScoreKey<S>;
    using K = typename SK::K;
    using KT = KeyTraits<K>;
    typedef unsigned long long u64;
    constexpr int P = kSelPerThread, kPad = P + 1;  // odd stride: the threads of a warp hit 32 different banks
    constexpr int kWarps = kSelThreads / 32;
    __shared__ K sh_key[kSelThreads * kPad];
    __shared__ __align__(16) unsigned sh_hist[kHistBins];
    __shared__ unsigned sh_scan[kWarps];
    __shared__ unsigned sh_poll[2][kWarps];
    __shared__ int sh_stop[2];
    __shared__ u64 sh_scan64[kWarps];
    __shared__ unsigned sh_out[3];
    __shared__ unsigned sh_w[kWarps];
    __shared__ u64 sh_wl[2 * kWarps];
    __shared__ u64 sh_mine[3];
    __shared__ int sh_boundary;
    __shared__ unsigned sh_boundary_take;

    griddep_launch();  // the pack kernel may be scheduled while this one runs; it waits before reading sel / poff
    SEL_STAMP(st, 0);
    const unsigned B = (unsigned)g.n_blocks;  // fewer than 2^32 blocks: init rejects more
    const unsigned first = blockIdx.x * kSelTile + threadIdx.x * P;
    const bool none = k == 0;
    const u64 key_or = KT::kSkippable ? st->key_or : ~0ull;  // put back to 0 after the exchange
    const u64 ulen = uniform_block_len(g);
    K *my = sh_key + threadIdx.x * kPad;
    // 32-bit keys always start with digit pass 0, so its histogram is built here, from the registers the keys were
    // loaded into: no second walk over them.  (64-bit keys usually skip their first passes.)
    constexpr bool kFusedFirstPass = !KT::kSkippable;
    int nv;  // how many of this thread's P blocks exist
    {
        K key[P];
        unsigned valid;
        load_keys<S>(score, B, first, key, valid);  // on their way while the histogram is cleared
        for (int i = threadIdx.x; i < kHistBins; i += kSelThreads) sh_hist[i] = 0;
        if (threadIdx.x == 0) {
            sh_boundary = -1;
            sh_boundary_take = 0;
        }
        __syncthreads();
        nv = __popc(valid);  // the valid ones come first
#pragma unroll
        for (int j = 0; j < P; ++j) {
            my[j] = key[j];
            if (kFusedFirstPass && !none && j < nv)
                atomicAdd(&sh_hist[(unsigned)((key[j] >> KT::shift(0)) & ((1ull << KT::width(0)) - 1))], 1u);
        }
    }
    // Rows that end in a shorter block give an implicit layout two block lengths.  Which of this thread's blocks
    // are the short ones is worked out once; every sum of lengths is then two population counts.
    const bool two_len = !ulen && !g.boff;
    const u64 len_full = g.block_elems;
    u64 len_short = 0;
    unsigned short_bits = 0;
    if (two_len) {
        len_short = g.row_len - (u64)(g.blocks_per_row - 1) * g.block_elems;
        unsigned j = first % g.blocks_per_row;
        for (int i = 0; i < P; ++i) {
            if (j == g.blocks_per_row - 1) short_bits |= 1u << i;
            if (++j == g.blocks_per_row) j = 0;
        }
    }
    __syncthreads();
    SEL_STAMP(st, 1);  // keys loaded
    bool alive = true;

    // ---- digit passes: tau = the k-th largest key, need = how many keys equal to tau are taken
    u64 prefix = 0;
    unsigned need = k, taking_part = B;  // keys that enter the next histogram: all, then those of the resolved bin
    if (!none) {
        for (int p = 0; p < KT::kPasses && alive; ++p) {
            const int shift = KT::shift(p), width = KT::width(p);
            const u64 mask = (1ull << width) - 1;
            if (KT::kSkippable && ((key_or >> shift) & mask) == 0) {  // this digit is 0 in every key
                prefix <<= width;
                continue;
            }
            // A handful of keys left (the usual state of the last pass) go to the global histogram one by one: the
            // shared histogram, its barrier and the sweep over its bins would cost more.  taking_part is the same
            // number in every CTA, so all of them take the same branch.
            const bool direct = !SOLO && p != 0 && taking_part <= kSelDirectKeys;
            if (kFusedFirstPass && p == 0) {
                // counted while the keys were loaded
            } else {
#pragma unroll 2
                for (int j = 0; j < nv; ++j) {
                    const u64 key = my[j];
                    if (p == 0 || (key >> (shift + width)) == prefix) {
                        const unsigned bin = (unsigned)((key >> shift) & mask);
                        if (direct) atomicAdd(&st->hist[p][bin], 1u);
                        else atomicAdd(&sh_hist[bin], 1u);
                    }
                }
            }
            if (!direct) __syncthreads();
            SEL_STAMP(st, 2 + 4 * p);  // pass p: histogram built
            if (!direct && !SOLO) {
                // two neighbouring bins per reduction (a count never carries into its neighbour: a histogram holds
                // fewer than 2^32 keys): half as many updates meet in L2
                u64 *pairs = reinterpret_cast<u64 *>(st->hist[p]);
                uint2 *mine = reinterpret_cast<uint2 *>(sh_hist);
                for (int i = threadIdx.x; i < (1 << (width - 1)); i += kSelThreads) {
                    const uint2 c = mine[i];
                    if (c.x | c.y) {
                        atomicAdd(&pairs[i], (u64)c.x | ((u64)c.y << 32));
                        mine[i] = make_uint2(0u, 0u);  // ready for the next pass
                    }
                }
            }
            SEL_STAMP(st, 3 + 4 * p);  // flushed
            SEL_STAMP(st, 4 + 4 * p);
            unsigned d = 0, h = 0;
            unsigned *hist = SOLO ? sh_hist : st->hist[p];
            const unsigned expected = SOLO ? taking_part : taking_part + never;
            // one instantiation for both digit widths: a 10-bit pass leaves the upper half of its 2048-bin row at
            // zero, and code that has already run once is cheaper than a second copy that has not
            alive = resolve_digit_when_complete<11, SOLO>(hist, expected, need, d, h, st, sh_poll, sh_out, sh_stop);
            if (alive) {
                prefix = (prefix << width) | d;
                taking_part = h;  // the keys of the resolved bin are the ones the next pass counts
            } else if (threadIdx.x == 0) {
                sel_fail(st, info);
            }
            SEL_STAMP(st, 5 + 4 * p);  // histogram complete and digit resolved
        }
    }
    const K tau = (K)prefix;

    // ---- this CTA's record
    unsigned gt_bits = 0, eq_bits = 0, my_gt = 0, my_eq = 0, my_nf = 0;
    u64 my_lgt = 0, my_leq = 0;
    if (alive) {
        unsigned c_nf = 0;
#pragma unroll 2
        for (int j = 0; j < nv; ++j) {
            const K key = my[j];
            if (SK::nonfinite(key)) ++c_nf;
            if (none) continue;
            if (key > tau) gt_bits |= 1u << j;
            else if (key == tau) eq_bits |= 1u << j;
        }
        // per warp at most 256 of each: three 10-bit fields in one word, one warp-reduce instruction
        const unsigned packed = __reduce_add_sync(0xffffffffu, __popc(gt_bits) | (__popc(eq_bits) << 10) | (c_nf << 20));
        u64 lgt = 0, leq = 0;
        if (two_len) {
            const unsigned shorts = __reduce_add_sync(0xffffffffu, __popc(gt_bits & short_bits) |
                                                                       (__popc(eq_bits & short_bits) << 10));
            const unsigned s_gt = shorts & 1023u, s_eq = shorts >> 10;
            lgt = (u64)((packed & 1023u) - s_gt) * len_full + (u64)s_gt * len_short;
            leq = (u64)(((packed >> 10) & 1023u) - s_eq) * len_full + (u64)s_eq * len_short;
        } else if (!ulen) {
            BlockLens bl(g, first);
            for (int j = 0; j < nv; ++j) {
                const u64 len = bl.next();
                if (gt_bits >> j & 1u) lgt += len;
                else if (eq_bits >> j & 1u) leq += len;
            }
            lgt = group_sum<32, u64>(lgt);
            leq = group_sum<32, u64>(leq);
        }
        if ((threadIdx.x & 31) == 0) {
            sh_w[threadIdx.x >> 5] = packed;
            sh_wl[2 * (threadIdx.x >> 5)] = lgt;
            sh_wl[2 * (threadIdx.x >> 5) + 1] = leq;
        }
        __syncthreads();
        // one warp's partial per lane (the fields of different warps cannot be added inside one word: up to 4096)
        const int ln = threadIdx.x & 31;
        const unsigned pv = ln < kWarps ? sh_w[ln] : 0u;
        const unsigned c_gt = __reduce_add_sync(0xffffffffu, pv & 1023u);
        const unsigned c_eq = __reduce_add_sync(0xffffffffu, (pv >> 10) & 1023u);
        const unsigned t_nf = __reduce_add_sync(0xffffffffu, pv >> 20);
        lgt = leq = 0;
        if (!ulen) {
            lgt = group_sum<32, u64>(ln < kWarps ? sh_wl[2 * ln] : 0ull);
            leq = group_sum<32, u64>(ln < kWarps ? sh_wl[2 * ln + 1] : 0ull);
        }
        my_gt = c_gt, my_eq = c_eq, my_nf = t_nf, my_lgt = lgt, my_leq = leq;
        SEL_STAMP(st, 26);  // own counts known
        if (!SOLO && threadIdx.x == 0) rec_publish(&st->rec[blockIdx.x], c_gt, c_eq, t_nf, lgt, leq);
    }

    // ---- exchange: thread c takes the record of CTA c; one packed scan gives every prefix sum
    unsigned my_eq_before = 0, my_sel_base = 0, total_n = 0, total_nf = 0;
    u64 my_len_base = 0, total_l = 0;
    int cb = -1;
    if (alive) {
        const unsigned c = threadIdx.x;
        unsigned e = 0, gt = 0, nf = 0;
        u64 lg = 0, le = 0;
        bool ok = true;
        if (SOLO) {
            if (c == 0) gt = my_gt, e = my_eq, nf = my_nf, lg = my_lgt, le = my_leq;
        } else if (c < gridDim.x + never) {
            ok = rec_take(&st->rec[c], !ulen, st, gt, e, nf, lg, le);
            if (!ok) sel_fail(st, info);
        }
        alive = __syncthreads_and(ok) != 0;
        SEL_STAMP(st, 27);  // every CTA's record read
        if (alive) {
            // fewer than 2^21 keys in the whole grid (one tile of 4096 per CTA, fewer than 512 CTAs): three
            // 21-bit fields
            u64 tot;
            const u64 ex = sel_excl_scan<u64>((u64)gt | ((u64)e << 21) | ((u64)nf << 42), sh_scan64, &tot);
            const unsigned ex_gt = (unsigned)(ex & 0x1fffffu), ex_e = (unsigned)((ex >> 21) & 0x1fffffu);
            const unsigned tot_gt = (unsigned)(tot & 0x1fffffu), tot_e = (unsigned)((tot >> 21) & 0x1fffffu);
            total_nf = (unsigned)(tot >> 42);
            // the keys equal to tau are taken in id order, so the CTAs before c take min(need, ex_e) of them
            const unsigned taken_before = need < ex_e ? need : ex_e;
            unsigned take = need - taken_before;
            if (take > e) take = e;
            if (take != 0 && take != e) {  // the tau-keys run out inside CTA c's range
                sh_boundary = (int)c;
                sh_boundary_take = take;
            }
            total_n = tot_gt + (need < tot_e ? need : tot_e);
            if (c == blockIdx.x) {
                sh_mine[0] = ex_e;
                sh_mine[1] = ex_gt + taken_before;
            }
            if (!ulen) {
                const u64 l = lg + (take == e ? le : 0);
                u64 two[2] = {c < blockIdx.x ? l : 0, l};
                cta_sum_n<2, kSelThreads>(two, sh_wl);
                my_len_base = two[0], total_l = two[1];
            } else {
                __syncthreads();
            }
            my_eq_before = (unsigned)sh_mine[0];
            my_sel_base = (unsigned)sh_mine[1];
            cb = sh_boundary;
            if (ulen) {
                my_len_base = (u64)my_sel_base * ulen;
                total_l = (u64)total_n * ulen;
            }
        }
    }

    // ---- boundary: with blocks of different lengths, the CTAs behind the one where the tau-keys run out need
    // the length of what it takes
    if (alive && !ulen && cb >= 0 && (int)blockIdx.x >= cb) {
        u64 *scan2 = sh_wl;  // free again
        const u64 pl = boundary_len<S>(score, g, (unsigned)cb, 1u, gridDim.x, tau, sh_boundary_take, sh_scan64, scan2);
        total_l += pl;
        if ((int)blockIdx.x > cb) my_len_base += pl;
    }
    SEL_STAMP(st, 28);  // bases known

    // ---- emit: ordered compaction of this CTA's tile
    if (alive && !none) {
        unsigned my_take = need > my_eq_before ? need - my_eq_before : 0;
        if (my_take > my_eq) my_take = my_eq;
        unsigned take_bits = gt_bits;
        if (my_take == my_eq) {
            take_bits |= eq_bits;
        } else if (my_take != 0) {  // only in the CTA where the tau-keys run out (the same decision in all its threads)
            unsigned rank = sel_excl_scan<unsigned>(__popc(eq_bits), sh_scan, nullptr);
            for (int j = 0; j < nv; ++j)
                if (eq_bits >> j & 1u) {
                    if (rank < my_take) take_bits |= 1u << j;
                    ++rank;
                }
        }
        if (ulen) {
            unsigned pos = my_sel_base + sel_excl_scan<unsigned>(__popc(take_bits), sh_scan, nullptr);
            for (int j = 0; j < nv; ++j)
                if (take_bits >> j & 1u) {
                    sel[pos] = first + j;
                    poff[pos] = (u64)pos * ulen;
                    ++pos;
                }
        } else {
            u64 lsum = 0;
            if (two_len) {
                lsum = (u64)__popc(take_bits & ~short_bits) * len_full + (u64)__popc(take_bits & short_bits) * len_short;
            } else {
                BlockLens bl(g, first);
                for (int j = 0; j < nv; ++j) {
                    const u64 len = bl.next();
                    if (take_bits >> j & 1u) lsum += len;
                }
            }
            // one scan for both outputs: block counts in the top 16 bits (at most 4096 per tile), summed
            // lengths below (a buffer has fewer than 2^48 elements: init rejects more)
            const u64 both = sel_excl_scan<u64>(((u64)__popc(take_bits) << 48) | lsum, sh_scan64, nullptr);
            unsigned pos = my_sel_base + (unsigned)(both >> 48);
            u64 off = my_len_base + (both & ((1ull << 48) - 1));
            if (two_len) {
                for (int j = 0; j < nv; ++j)
                    if (take_bits >> j & 1u) {
                        sel[pos] = first + j;
                        poff[pos] = off;
                        ++pos;
                        off += (short_bits >> j & 1u) ? len_short : len_full;
                    }
            } else {
                BlockLens bl(g, first);
                for (int j = 0; j < nv; ++j) {
                    const u64 len = bl.next();
                    if (take_bits >> j & 1u) {
                        sel[pos] = first + j;
                        poff[pos] = off;
                        ++pos;
                        off += len;
                    }
                }
            }
        }
    }
    SEL_STAMP(st, 29);  // emitted
    // The last CTA lies behind every boundary, so its totals are complete.  By now every CTA has read key_or.
    if (alive && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
        info->k = total_n;
        info->payload_elems = total_l;
        info->nonfinite_blocks = total_nf;
        poff[total_n] = total_l;
        if (KT::kSkippable) st->key_or = 0;  // forget which uint64 key bits were seen
    }
}

// ---- the traditional full checkpoint (k == B) -----------------------------------
//
// When every block is saved the selection is known beforehand (all ids, in
// order, each block's payload offset equal to its own offset), so scoring and
// packing fuse into one pass: x and z are read once for the distance, and x is
// written to the payload and over z from the registers it already sits in.
// That moves 4 N elements instead of the 5 N of score pass + pack pass.
// Same traversal and accumulation order as block_distance, so the scores are
// bit-identical to a partial save's.
template <typename T, int NORM, int G, bool VEC>
__device__ __forceinline__ typename Elem<T, NORM>::wide_t block_distance_save(const T *__restrict__ x, T *__restrict__ z,
                                                                              T *__restrict__ payload, uint64_t beg,
                                                                              uint64_t len, int lane) {
    using E = Elem<T, NORM>;
    using U = typename std::conditional<VEC, typename E::vec_t, T>::type;
    using acc_t = typename E::acc_t;
    using wide_t = typename E::wide_t;
    constexpr unsigned kFlushMask = VEC ? 63u : 255u;
    const U *xs = reinterpret_cast<const U *>(x + beg);
    U *zs = reinterpret_cast<U *>(z + beg);
    U *ps = reinterpret_cast<U *>(payload + beg);
    const uint64_t n = VEC ? (len >> 2) : len;
    constexpr uint64_t step = 4 * (uint64_t)G;
    acc_t a[4] = {0, 0, 0, 0};
    wide_t total = 0;
    U xc[4], zc[4], xn[4], zn[4];
    uint64_t u = lane;
    unsigned it = 0;
    bool have = u < n;
    if (have) load_batch<U, G>(xs, zs, u, n, xc, zc);
    while (have) {  // loads of the next batch are issued before the stores of this one (see block_distance)
        const uint64_t un = u + step;
        const bool more = un < n;
        if (more) load_batch<U, G>(xs, zs, un, n, xn, zn);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            E::addu(a[j], xc[j], zc[j]);
            const uint64_t i = u + (uint64_t)j * G;
            if (i < n) {
                st_stream(ps + i, xc[j]);
                st_stream(zs + i, xc[j]);
            }
        }
        if (E::kFlush && (++it & kFlushMask) == 0) {
            total += ((wide_t)a[0] + (wide_t)a[1]) + ((wide_t)a[2] + (wide_t)a[3]);
            a[0] = a[1] = a[2] = a[3] = 0;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            xc[j] = xn[j];
            zc[j] = zn[j];
        }
        u = un;
        have = more;
    }
    total += ((wide_t)a[0] + (wide_t)a[1]) + ((wide_t)a[2] + (wide_t)a[3]);
    return group_sum<G, wide_t>(total);
}

// info must have been cleared before the launch (the non-finite count is added up with atomics).
template <typename T, int NORM, int G, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_full_save(const T *__restrict__ x, T *__restrict__ z, T *__restrict__ payload, Geom g, const float *__restrict__ weight,
            typename Elem<T, NORM>::score_t *__restrict__ score, uint32_t *__restrict__ sel,
            unsigned long long *__restrict__ poff, SaveInfoDev *info) {
    using E = Elem<T, NORM>;
    using SK = ScoreKey<typename E::score_t>;
    const int lane = threadIdx.x & (G - 1);
    const uint64_t grp = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    const bool valid = grp < g.n_blocks;
    uint64_t beg = 0, len = 0;
    if (valid) g.range((uint32_t)grp, beg, len);
    typename E::wide_t s = block_distance_save<T, NORM, G, VEC>(x, z, payload, beg, len, lane);
    if (valid && lane == 0) {
        const typename E::score_t sc = weighted<E>(s, weight, grp);
        score[grp] = sc;
        sel[grp] = (uint32_t)grp;
        poff[grp] = beg;
        if (SK::nonfinite(SK::key(sc))) atomicAdd(&info->nonfinite_blocks, 1ull);
        if (grp == g.n_blocks - 1) {
            poff[g.n_blocks] = g.n_elems;
            info->k = g.n_blocks;
            info->payload_elems = g.n_elems;
        }
    }
}

// ---- multi-GPU form of a save: which of the globally selected blocks are this rank's ---------------
//
// sel_g holds the ascending global ids chosen among all ranks' scores.  Marks, in member[0..n_local), the ones in
// [first, first + n_local) (member must be zero before) and counts them; rec = {count, error of the global
// selection, non-finite scores over all ranks} for the host.
static __global__ void __launch_bounds__(kThreads)
k_mark_members(const uint32_t *__restrict__ sel_g, const SaveInfoDev *info_g, unsigned long long first,
               unsigned long long n_local, uint32_t *__restrict__ member, unsigned long long *rec) {
    const unsigned long long j = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
    const bool failed = info_g->error != 0;
    bool mine = false;
    if (!failed && j < info_g->k) {
        const unsigned long long id = sel_g[j];
        if (id >= first && id - first < n_local) {
            member[id - first] = 1u;
            mine = true;
        }
    }
    const unsigned bal = __ballot_sync(0xffffffffu, mine);
    if ((threadIdx.x & 31) == 0 && bal) atomicAdd(&rec[0], (unsigned long long)__popc(bal));
    if (j == 0) {
        rec[1] = info_g->error;
        rec[2] = info_g->nonfinite_blocks;
    }
}

// ---- baseline strategies of Section 5.4 -------------------------------------
//
// `round`: the k blocks that follow a cursor, wrapping at the end of the buffer.
// The id list stays ascending, so a wrapped selection is the run [0, wrap)
// followed by the run [cursor, B); offsets inside a run of consecutive blocks
// are differences of block start offsets, so no scan is needed.
static __global__ void __launch_bounds__(kThreads)
k_select_round(Geom g, unsigned long long cursor, unsigned long long k, uint32_t *__restrict__ sel,
               unsigned long long *__restrict__ poff, SaveInfoDev *info) {
    const unsigned long long j = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
    if (k == 0) {
        if (j == 0) {
            poff[0] = 0;
            info->k = 0;
            info->payload_elems = 0;
            info->nonfinite_blocks = 0;
            info->error = 0;
        }
        return;
    }
    if (j >= k) return;
    const unsigned long long B = g.n_blocks;
    const unsigned long long wrap = cursor + k > B ? cursor + k - B : 0;  // ids below the cursor that are taken
    uint64_t beg, len, first_beg, first_len, base = 0;
    uint32_t b;
    if (j < wrap) {
        b = (uint32_t)j;
        first_beg = 0;
    } else {
        b = (uint32_t)(cursor + (j - wrap));
        g.range((uint32_t)cursor, first_beg, first_len);
        if (wrap) g.range((uint32_t)wrap, base, first_len);  // elements of blocks [0, wrap)
    }
    g.range(b, beg, len);
    const unsigned long long off = base + (beg - first_beg);
    sel[j] = b;
    poff[j] = off;
    if (j == k - 1) {
        poff[k] = off + len;
        info->k = k;
        info->payload_elems = off + len;
        info->nonfinite_blocks = 0;
        info->error = 0;
    }
}

}  // namespace scar
