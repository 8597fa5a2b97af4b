// Streaming pass over the two parameter streams x (live) and z (running
// checkpoint), block by block: per-block distance for the checkpoint scores
// (Section 4.3, checkpoint step 1) and, for recovery, the same sum over the lost
// blocks fused with x_b := z_b (Section 4.1; appendix proof of Theorem 4.1).
//
// A group of G consecutive lanes (G = 4..32, a power of two) owns one block at
// a time.  Each lane issues 16-byte loads G vectors apart, four per stream per
// batch with the next batch already in flight, and keeps four independent
// accumulators; the group total is formed with xor-shuffles, so the summation
// order depends only on G and the block length, never on scheduling: results
// are bit-reproducible run to run.
#pragma once
#include <type_traits>

#include "geom.cuh"
#include "sel_state.cuh"

namespace scar {

constexpr int kThreads = 256;

// Distance of one block: NORM 0 is the default of the element type (squared l2
// for float32, l1 for int32); NORM 1 is the l1 distance of float32 data, which
// with per-block weights gives the length-scaled total variation that Appendix C
// uses for topic distributions.
constexpr int kNormDefault = 0;
constexpr int kNormL1 = 1;

template <typename T, int NORM = kNormDefault> struct Elem;

// float32 elements: squared l2 distance.  Inner chains are fp32 (at most 64
// vectors per accumulator between flushes), the outer sum and the cross-lane
// reduction are fp64, so long blocks do not lose accuracy.
template <> struct Elem<float, kNormDefault> {
    using vec_t = float4;
    using wide_t = double;   // what a group reduces to
    using score_t = float;   // what is stored per block
    using acc_t = float;
    static __device__ __forceinline__ void add(acc_t &a, float x, float z) {
        float d = x - z;
        a = fmaf(d, d, a);
    }
    static __device__ __forceinline__ void addu(acc_t &a, float x, float z) { add(a, x, z); }
    static __device__ __forceinline__ void addu(acc_t &a, const vec_t &x, const vec_t &z) {
        add(a, x.x, z.x); add(a, x.y, z.y); add(a, x.z, z.z); add(a, x.w, z.w);
    }
    static constexpr bool kFlush = true;
};

// float32 elements, l1 distance: same accumulation scheme with |x - z| in place of (x - z)^2.
template <> struct Elem<float, kNormL1> {
    using vec_t = float4;
    using wide_t = double;
    using score_t = float;
    using acc_t = float;
    static __device__ __forceinline__ void add(acc_t &a, float x, float z) { a += fabsf(x - z); }
    static __device__ __forceinline__ void addu(acc_t &a, float x, float z) { add(a, x, z); }
    static __device__ __forceinline__ void addu(acc_t &a, const vec_t &x, const vec_t &z) {
        add(a, x.x, z.x); add(a, x.y, z.y); add(a, x.z, z.z); add(a, x.w, z.w);
    }
    static constexpr bool kFlush = true;
};

// int32 elements: integer l1 distance, exact in 64 bits (|x - z| < 2^32).
template <> struct Elem<int, kNormDefault> {
    using vec_t = int4;
    using wide_t = unsigned long long;
    using score_t = unsigned long long;
    using acc_t = unsigned long long;
    static __device__ __forceinline__ void add(acc_t &a, int x, int z) {
        a += __sad(x, z, 0u);  // |x - z| as an unsigned 32-bit value, exact for any pair of int32
    }
    static __device__ __forceinline__ void addu(acc_t &a, int x, int z) { add(a, x, z); }
    static __device__ __forceinline__ void addu(acc_t &a, const vec_t &x, const vec_t &z) {
        add(a, x.x, z.x); add(a, x.y, z.y); add(a, x.z, z.z); add(a, x.w, z.w);
    }
    static constexpr bool kFlush = false;
};

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may start while
// the kernel before it is still running; it must call griddep_wait() before touching anything that kernel
// writes.  griddep_launch() in the earlier kernel lets the later one be scheduled as soon as every CTA of the
// earlier one has started.  Both are no-ops for launches without the attribute.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename V> __device__ __forceinline__ V ld_stream(const V *p) { return __ldcs(p); }
template <typename V> __device__ __forceinline__ void st_stream(V *p, const V &v) { __stcs(p, v); }

// Keeps the compiler from moving a store above a load that precedes it in the source.  In the restoring pass a
// batch's stores depend on its loads; when the compiler interleaves them to save registers ("load, store, load,
// store"), each load waits behind a store that waits for the load before it, and a batch costs four round
// trips to memory instead of one (measured: a 3x slower pass, depending on what else the kernel contained).
__device__ __forceinline__ void loads_before_stores() { asm volatile("" ::: "memory"); }

template <int G, typename W> __device__ __forceinline__ W group_sum(W v) {
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One batch = four units (16-byte vectors, or single elements on the
// element-wise path) per stream and lane, G units apart.  Units past the end of
// the block count as zero, which adds nothing to either distance.  Requires
// n > 0.  The loads themselves are unconditional (a unit past the end reads the
// block's last unit instead and the value is dropped): eight loads in one
// straight line are issued back to back, whereas loads under eight branches
// were, in some builds, each waited for before the next was issued, which made
// a pass over short blocks three times slower.
template <typename U, int G>
__device__ __forceinline__ void load_batch(const U *__restrict__ xs, const U *__restrict__ zs, uint64_t u, uint64_t n,
                                           U (&xr)[4], U (&zr)[4]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint64_t i = u + (uint64_t)j * G;
        const uint64_t at = i < n ? i : n - 1;
        xr[j] = ld_stream(xs + at);
        zr[j] = ld_stream(zs + at);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (u + (uint64_t)j * G >= n) {
            xr[j] = U{};
            zr[j] = U{};
        }
    }
}

// Distance sum of one block over the lanes of a group; every lane returns the
// group total.  len == 0 is allowed (the lane then only takes part in the
// shuffles).  WRITE: also store z over x.  VEC: block starts/ends are 16-byte
// aligned, so the whole block moves as 16-byte vectors; otherwise element-wise.
//
// The loop is software-pipelined: the loads of batch i+1 are issued before the
// stores of batch i.  Issue is in order, so a store that waits for its data
// would otherwise hold back the next loads and leave the memory system idle for
// one round trip per batch (measured: 3.1 TB/s without, 6.8 TB/s with, on the
// in-place restore).  Accumulator slot j always takes unit lane + (4i + j) * G,
// with or without WRITE, so the score pass and the recovery pass produce
// bit-identical per-block sums.
template <typename T, int NORM, int G, bool VEC, bool WRITE>
__device__ __forceinline__ typename Elem<T, NORM>::wide_t block_distance(T *__restrict__ x, const T *__restrict__ z,
                                                                         uint64_t beg, uint64_t len, int lane) {
    using E = Elem<T, NORM>;
    using U = typename std::conditional<VEC, typename E::vec_t, T>::type;
    using acc_t = typename E::acc_t;
    using wide_t = typename E::wide_t;
    constexpr unsigned kFlushMask = VEC ? 63u : 255u;
    U *xs = reinterpret_cast<U *>(x + beg);
    const U *zs = reinterpret_cast<const U *>(z + beg);
    const uint64_t n = VEC ? (len >> 2) : len;
    constexpr uint64_t step = 4 * (uint64_t)G;
    acc_t a[4] = {0, 0, 0, 0};
    wide_t total = 0;
    U xc[4], zc[4], xn[4], zn[4];
    uint64_t u = lane;
    unsigned it = 0;
    if (!WRITE || G < 32) {
        // Plain loop (full batches unguarded, then one guarded batch).  For the
        // read-only pass nothing can hold back the loads, so this is the faster
        // form.  It is also the form of the restoring pass over short blocks
        // (G < 32: a block is about one batch, so there is no next batch to
        // load ahead, and the registers of the pipelined form below would only
        // cost occupancy: 16 resident warps per SM instead of 48).  A batch
        // counts as full only when it is full for every lane of the group, so
        // the lanes of a group never diverge between the two forms.
        for (; u - lane + step <= n; u += step) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                xc[j] = ld_stream(xs + u + (uint64_t)j * G);
                zc[j] = ld_stream(zs + u + (uint64_t)j * G);
            }
            if (WRITE) loads_before_stores();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                E::addu(a[j], xc[j], zc[j]);
                if (WRITE) st_stream(xs + u + (uint64_t)j * G, zc[j]);
            }
            if (E::kFlush && (++it & kFlushMask) == 0) {
                total += ((wide_t)a[0] + (wide_t)a[1]) + ((wide_t)a[2] + (wide_t)a[3]);
                a[0] = a[1] = a[2] = a[3] = 0;
            }
        }
        if (u < n) {
            load_batch<U, G>(xs, zs, u, n, xc, zc);
            if (WRITE) loads_before_stores();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                E::addu(a[j], xc[j], zc[j]);
                if (WRITE && u + (uint64_t)j * G < n) st_stream(xs + u + (uint64_t)j * G, zc[j]);
            }
        }
        total += ((wide_t)a[0] + (wide_t)a[1]) + ((wide_t)a[2] + (wide_t)a[3]);
        return group_sum<G, wide_t>(total);
    }
    bool have = u < n;
    if (have) load_batch<U, G>(xs, zs, u, n, xc, zc);
    while (have) {
        const uint64_t un = u + step;
        const bool more = un < n;
        if (more) load_batch<U, G>(xs, zs, un, n, xn, zn);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            E::addu(a[j], xc[j], zc[j]);
            if (WRITE && u + (uint64_t)j * G < n) st_stream(xs + u + (uint64_t)j * G, zc[j]);
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

// ---- a1: score of every block ----------------------------------------------

// Block total -> stored score, times the block's weight when the caller set
// weights (float data only; Appendix C: a positive combination of block norms
// is still a norm).
template <typename E>
__device__ __forceinline__ typename E::score_t weighted(typename E::wide_t s, const float *__restrict__ weight,
                                                        uint64_t b) {
    if (std::is_same<typename E::wide_t, double>::value && weight) s = (typename E::wide_t)((double)s * (double)weight[b]);
    return (typename E::score_t)s;
}

// sel_state / info: the scoring pass is what runs before a selection, so its first CTAs clear the selection's
// counters, histograms and records and the save's result record (both may be nullptr: nothing is cleared).
template <typename T, int NORM, int G, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_block_scores(const T *__restrict__ x, const T *__restrict__ z, Geom g, const float *__restrict__ weight,
               typename Elem<T, NORM>::score_t *__restrict__ score, SelState *sel_state, SaveInfoDev *info) {
    using E = Elem<T, NORM>;
    if (sel_state) sel_state_clear(sel_state, info);
    const int lane = threadIdx.x & (G - 1);
    const uint64_t grp = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    const bool valid = grp < g.n_blocks;
    uint64_t beg = 0, len = 0;
    if (valid) g.range((uint32_t)grp, beg, len);
    typename E::wide_t s = block_distance<T, NORM, G, VEC, false>(const_cast<T *>(x), z, beg, len, lane);
    if (valid && lane == 0) {
        typename E::score_t sc = weighted<E>(s, weight, grp);
        score[grp] = sc;
        if (sel_state && sizeof(typename E::score_t) == 8) {
            // Remember which key bits occur at all, so that radix passes over
            // digits that are zero in every key can be skipped.
            unsigned long long bits = (unsigned long long)sc;
            unsigned long long seen = *reinterpret_cast<volatile unsigned long long *>(&sel_state->key_or);
            if (bits & ~seen) atomicOr(&sel_state->key_or, bits);
        }
    }
}

// ---- final reduction of a recovery / norm pass, in a fixed order ------------------

struct NormInfoDev {
    double l2;
    unsigned long long l1;
    unsigned long long lost_blocks;
    unsigned long long lost_elems;
};

template <typename W> __device__ __forceinline__ W cta_sum(W v, W *sh) {
    v = group_sum<32, W>(v);
    const int w = threadIdx.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[w] = v;
    __syncthreads();
    W t = 0;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) t += sh[i];
    return t;
}

// Scratch of the reduction: two slots per CTA of the pass and three per watcher.  A slot holds kSlotEmpty except
// between its owner's store and the watcher's read, so the value itself tells the reader that it has arrived
// (an aligned 8-byte store is seen whole or not at all); no fence, ticket or atomic is involved.
constexpr unsigned long long kSlotEmpty = ~0ull;
constexpr unsigned kMaxWatchers = kThreads;
struct NormScratch {
    unsigned long long *cta_val;   // per CTA: sum of its blocks' partials (bits of a double, or a uint64)
    unsigned long long *cta_cnt;   // per CTA: lost blocks it covered (top 16 bits) and their elements (low 48)
    unsigned long long *tile_val;  // per watcher, kMaxWatchers of each: the sum over its CTAs,
    unsigned long long *tile_blocks;  // their lost blocks,
    unsigned long long *tile_elems;   // and elements
};
// 8-byte words a launch of n_ctas CTAs needs: two arrays of n_ctas, then three of kMaxWatchers.
inline size_t norm_scratch_words(uint64_t n_ctas) { return 2 * (size_t)n_ctas + 3 * kMaxWatchers; }
inline NormScratch norm_scratch_at(unsigned long long *base, uint64_t n_ctas) {
    NormScratch rs;
    rs.cta_val = base;
    rs.cta_cnt = base + n_ctas;
    rs.tile_val = base + 2 * n_ctas;
    rs.tile_blocks = rs.tile_val + kMaxWatchers;
    rs.tile_elems = rs.tile_val + 2 * kMaxWatchers;
    return rs;
}

// How many CTAs at the end of a grid add up the others' slots.
__host__ __device__ inline unsigned norm_watchers(unsigned grid) {
    const unsigned n = grid / 1024;
    return n < 1 ? 1 : (n > kMaxWatchers ? kMaxWatchers : n);
}

constexpr unsigned kSlotSpinLimit = 1u << 20;  // a quarter of a second at the earliest

__device__ __forceinline__ unsigned long long slot_peek(const unsigned long long *slot) {
    return *reinterpret_cast<const volatile unsigned long long *>(slot);
}
// v: what slot_peek saw.  Waits (with a bound) until the slot's owner has filled it, and empties it again for the
// next launch.  false: gave up.
__device__ __forceinline__ bool slot_take(unsigned long long *slot, unsigned long long &v) {
    volatile unsigned long long *p = slot;
    unsigned tries = 0;
    while (v == kSlotEmpty) {
        if (++tries > kSlotSpinLimit) return false;
        if (tries > 16) __nanosleep(tries > 4096 ? 256 : 32);
        v = *p;
    }
    *p = kSlotEmpty;
    return true;
}

__device__ __forceinline__ void norm_write(NormInfoDev *out, bool is_float, bool take_sqrt, bool ok, double fs,
                                           unsigned long long is, unsigned long long nb, unsigned long long ne) {
    if (!ok) {  // a slot never arrived: the result says so (lost_blocks can never be this large)
        out->l2 = __longlong_as_double(0x7ff8000000000000ll);
        out->l1 = 0;
        out->lost_blocks = kSlotEmpty;
        out->lost_elems = 0;
        return;
    }
    out->l2 = is_float ? (take_sqrt ? sqrt(fs) : fs) : 0.0;  // l2 norms sum squares; l1 / weighted-l1 norms sum as they are
    out->l1 = is_float ? 0ull : is;
    out->lost_blocks = nb;
    out->lost_elems = ne;
}

// Sums a value (double for float data, else uint64) and a uint64 per thread over the CTA with one pair of
// barriers, in a fixed order: xor tree inside each warp, then the warps in order.
template <bool kF>
__device__ __forceinline__ void cta_sum_pair(double &fs, unsigned long long &is, unsigned long long &cnt, double *shd,
                                             unsigned long long *shu, unsigned long long *shc) {
    if (kF) fs = group_sum<32, double>(fs);
    else is = group_sum<32, unsigned long long>(is);
    cnt = group_sum<32, unsigned long long>(cnt);
    const int w = threadIdx.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) {
        if (kF) shd[w] = fs;
        else shu[w] = is;
        shc[w] = cnt;
    }
    __syncthreads();
    fs = 0.0, is = 0, cnt = 0;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) {
        if (kF) fs += shd[i];
        else is += shu[i];
        cnt += shc[i];
    }
}

// Called by every thread of every CTA of a recovery / norm pass with the thread's own share (fs for float data,
// is for integer data, lost blocks, lost elements; a CTA covers fewer than 2^16 blocks and a buffer has fewer
// than 2^48 elements, so the two counts travel in one word).  The CTA's total goes to its two slots with plain
// stores, and the CTA is done: nothing in the streaming part of the pass waits for the memory system on behalf
// of the reduction.  The last CTAs of the grid (the watchers: one per 1024 CTAs) do the adding: watcher t
// collects the slots of its contiguous share of the CTAs, thread i taking slots i, i + 256, ... in that order,
// then the fixed tree of cta_sum; the last CTA collects the watchers' totals the same way and writes the result.
// A watcher only ever waits for CTAs with a lower index than its own, which were dispatched before it and wait
// for nobody, and every wait is bounded.  The order of every addition depends only on the grid size, so the
// result is the same bits on every run.  This replaces a second launch: the pass and its reduction are one kernel.
template <typename T>
__device__ __forceinline__ void norm_epilogue(double fs, unsigned long long is, unsigned long long nb,
                                              unsigned long long ne, const NormScratch &rs, NormInfoDev *out,
                                              bool take_sqrt) {
    typedef unsigned long long u64;
    constexpr bool kF = std::is_same<T, float>::value;
    constexpr u64 kElemMask = (1ull << 48) - 1;
    __shared__ double shd[kThreads / 32];
    __shared__ u64 shu[kThreads / 32];
    __shared__ u64 shc[kThreads / 32];
    u64 cnt = (nb << 48) | ne;
    cta_sum_pair<kF>(fs, is, cnt, shd, shu, shc);
    const unsigned grid = gridDim.x;
    if (grid == 1) {
        if (threadIdx.x == 0) norm_write(out, kF, take_sqrt, true, fs, is, cnt >> 48, cnt & kElemMask);
        return;
    }
    if (threadIdx.x == 0) {
        u64 v = is;
        if (kF) v = fs != fs ? 0x7ff8000000000000ull : (u64)__double_as_longlong(fs);  // never the empty pattern
        *reinterpret_cast<volatile u64 *>(rs.cta_val + blockIdx.x) = v;
        *reinterpret_cast<volatile u64 *>(rs.cta_cnt + blockIdx.x) = cnt;
    }
    const unsigned n_watch = norm_watchers(grid);
    if (blockIdx.x < grid - n_watch) return;

    // ---- watcher t: the slots of CTAs [lo, hi)
    const unsigned t = blockIdx.x - (grid - n_watch);
    const unsigned share = (grid + n_watch - 1) / n_watch;
    const unsigned lo = t * share, hi = lo + share < grid ? lo + share : grid;
    bool ok = true;
    fs = 0.0, is = 0, nb = 0, ne = 0;
    constexpr int kAhead = 4;  // slots per thread whose loads are in flight together
    for (unsigned base = lo + threadIdx.x; base < hi; base += kAhead * kThreads) {
        u64 v[kAhead], c[kAhead];
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            const unsigned i = base + j * kThreads;
            if (i < hi) {
                v[j] = slot_peek(rs.cta_val + i);
                c[j] = slot_peek(rs.cta_cnt + i);
            }
        }
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            const unsigned i = base + j * kThreads;
            if (i < hi) {
                ok = slot_take(rs.cta_val + i, v[j]) && ok;
                ok = slot_take(rs.cta_cnt + i, c[j]) && ok;
                if (kF) fs += __longlong_as_double((long long)v[j]);
                else is += v[j];
                nb += c[j] >> 48;
                ne += c[j] & kElemMask;
            }
        }
    }
    ok = __syncthreads_and(ok) != 0;
    if (kF) fs = cta_sum<double>(fs, shd);
    else is = cta_sum<u64>(is, shu);
    nb = cta_sum<u64>(nb, shu);
    ne = cta_sum<u64>(ne, shu);
    if (n_watch == 1) {
        if (threadIdx.x == 0) norm_write(out, kF, take_sqrt, ok, fs, is, nb, ne);
        return;
    }
    if (threadIdx.x == 0) {
        u64 v = is;
        if (kF) v = fs != fs ? 0x7ff8000000000000ull : (u64)__double_as_longlong(fs);
        *reinterpret_cast<volatile u64 *>(rs.tile_val + t) = v;
        *reinterpret_cast<volatile u64 *>(rs.tile_blocks + t) = ok ? nb : kSlotEmpty - 1;  // passes a failure on
        *reinterpret_cast<volatile u64 *>(rs.tile_elems + t) = ne;
    }
    if (blockIdx.x != grid - 1) return;

    // ---- the last CTA: the watchers' totals, in watcher order
    fs = 0.0, is = 0, nb = 0, ne = 0;
    if (threadIdx.x < n_watch) {
        u64 v = slot_peek(rs.tile_val + threadIdx.x), b = slot_peek(rs.tile_blocks + threadIdx.x),
            e = slot_peek(rs.tile_elems + threadIdx.x);
        ok = slot_take(rs.tile_val + threadIdx.x, v) && ok;
        ok = slot_take(rs.tile_blocks + threadIdx.x, b) && ok;
        ok = slot_take(rs.tile_elems + threadIdx.x, e) && ok;
        if (b == kSlotEmpty - 1) ok = false, b = 0;
        if (kF) fs = __longlong_as_double((long long)v);
        else is = v;
        nb = b;
        ne = e;
    }
    ok = __syncthreads_and(ok) != 0;
    if (kF) fs = cta_sum<double>(fs, shd);
    else is = cta_sum<u64>(is, shu);
    nb = cta_sum<u64>(nb, shu);
    ne = cta_sum<u64>(ne, shu);
    if (threadIdx.x == 0) norm_write(out, kF, take_sqrt, ok, fs, is, nb, ne);
}

// ---- a4 / a5: perturbation over the lost set, optional restore, and its norm: one launch -----------

// Exclusive prefix sum of one value per thread over a CTA of NT threads; *total gets the sum.
template <typename W, int NT = kThreads>
__device__ __forceinline__ W cta_excl_scan(W v, W *sh /*NT/32*/, W *total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    W inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        W n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();
    if (lane == 31) sh[w] = inc;
    __syncthreads();
    W before = 0, all = 0;
#pragma unroll
    for (int i = 0; i < NT / 32; ++i) {
        W t = sh[i];
        if (i < w) before += t;
        all += t;
    }
    if (total) *total = all;
    return before + inc - v;
}

// Launch shape of the pass: one group of lanes per lost block; a per-block mask is cut into chunks of `chunk`
// mask entries (a multiple of kThreads), one CTA each.
constexpr unsigned kMaxMaskChunk = 4 * kThreads;
constexpr uint64_t kTwoRoundsFrom = 4096;  // CTAs a one-round launch would have
struct RecoverShape {
    unsigned grid;
    unsigned chunk;
};
inline RecoverShape recover_shape(int mode, uint64_t n_work, int group_lanes, bool write) {
    RecoverShape r{1, (unsigned)kThreads};
    uint64_t want;
    if (mode == 2) {
        r.chunk = group_lanes < 32 ? 2 * kThreads : kThreads;  // short blocks: more of them per CTA
        want = (n_work + r.chunk - 1) / r.chunk;
    } else {
        // One work item per group; two, one after the other, when a read-only pass over short blocks would
        // otherwise need thousands of CTAs that live for one batch of loads and then pay for the CTA-wide sum
        // (400-byte rows: 68 us instead of 73 us; four and more lost what two gained, and small launches lost
        // at any number above one).
        const uint64_t groups = kThreads / group_lanes;
        const bool twice = !write && group_lanes < 32 && n_work >= kTwoRoundsFrom * groups;
        r.chunk = (unsigned)(groups * (twice ? 2 : 1));
        want = (n_work + r.chunk - 1) / r.chunk;
    }
    r.grid = (unsigned)(want < 1 ? 1 : want);
    return r;
}
// CTAs of the largest launch recover_shape can give for a layout of n_blocks blocks.
inline uint64_t recover_max_ctas(uint64_t n_blocks, int group_lanes) {
    return (n_blocks + kThreads / group_lanes - 1) / (kThreads / group_lanes) + 1;
}

// What a streaming pass has in flight is the number of resident warps times what a warp has in flight, so the
// kernels are held to the registers that let four CTAs share an SM (64 per thread), except the restoring pass
// over long blocks, whose hand-pipelined loop keeps two batches per lane in registers and settles for two.
// Asking for five or six CTAs made the compiler spill and the short-block passes 1.4 to 3 times slower; leaving
// the bound open let it take 96 registers for the read-only pass and lose a fifth of its speed (both measured).
constexpr int kStreamCtasPerSm = 4;

// A block's partial enters the sum as the value a score would store (rounded to float32 for float data), so that
// the squared perturbation of a lost set is exactly the sum of the scores of its blocks.
// MASK: the lost set is a per-block mask (S.mode == 2); otherwise all blocks or runs of blocks.  A template
// parameter rather than a branch, so that each kernel holds one copy of the streaming loop: with both forms in one
// kernel the compiler's schedule of that loop changed from build to build (10 to 20 % on the norm pass).
template <typename T, int NORM, int G, bool VEC, bool WRITE, bool MASK>
__global__ void __launch_bounds__(kThreads, (WRITE && G == 32 ? 2 : kStreamCtasPerSm))
k_recover_blocks(T *__restrict__ x, const T *__restrict__ z, Geom g, LostSet S, unsigned chunk,
                 const float *__restrict__ weight, NormScratch rs, NormInfoDev *out) {
    using E = Elem<T, NORM>;
    typedef unsigned long long u64;
    constexpr int kGroups = kThreads / G;
    constexpr bool kF = std::is_same<T, float>::value;
    const int lane = threadIdx.x & (G - 1), gi = threadIdx.x / G;
    double fs = 0.0;
    u64 is = 0, nb = 0, ne = 0;
    if (MASK) {
        // Per-block mask: the CTA takes `chunk` consecutive mask entries, writes the ids of the lost blocks
        // among them, in order, to a list in shared memory, and its groups walk that list side by side, so
        // that every group has a lost block to work on however sparse the mask is.
        __shared__ uint32_t sh_list[kMaxMaskChunk];
        __shared__ unsigned sh_scan[kThreads / 32];
        const unsigned per = chunk / kThreads;  // consecutive entries per thread, 1..4
        const u64 first = (u64)blockIdx.x * chunk + (u64)threadIdx.x * per;
        unsigned bits = 0;
        for (unsigned j = 0; j < per; ++j)
            if (first + j < g.n_blocks && S.mask[first + j] != 0) bits |= 1u << j;
        unsigned total;
        unsigned pos = cta_excl_scan<unsigned, kThreads>(__popc(bits), sh_scan, &total);
        for (unsigned j = 0; j < per; ++j)
            if (bits >> j & 1u) sh_list[pos++] = (uint32_t)(first + j);
        __syncthreads();
        for (unsigned i0 = 0; i0 < total; i0 += kGroups) {  // same trip count for every thread of the CTA
            const unsigned i = i0 + gi;
            const bool valid = i < total;
            uint32_t b = 0;
            uint64_t beg = 0, len = 0;
            if (valid) {
                b = sh_list[i];
                g.range(b, beg, len);
            }
            const typename E::wide_t s = block_distance<T, NORM, G, VEC, WRITE>(x, z, beg, len, lane);
            if (valid && lane == 0) {
                const typename E::score_t sc = weighted<E>(s, weight, b);
                if (kF) fs += (double)sc;
                else is += (u64)sc;
                ++nb;
                ne += len;
            }
        }
    } else {
        // chunk work items per CTA: one or two per group (recover_shape)
        for (unsigned w0 = 0; w0 < chunk; w0 += kGroups) {  // same trip count for every thread of the CTA
            const uint64_t w = (uint64_t)blockIdx.x * chunk + w0 + gi;
            uint32_t b = 0;
            const bool valid = S.block_of(w, b);
            uint64_t beg = 0, len = 0;
            if (valid) g.range(b, beg, len);
            const typename E::wide_t s = block_distance<T, NORM, G, VEC, WRITE>(x, z, beg, len, lane);
            if (valid && lane == 0) {
                const typename E::score_t sc = weighted<E>(s, weight, b);
                if (kF) fs += (double)sc;
                else is += (u64)sc;
                ++nb;
                ne += len;
            }
        }
    }
    norm_epilogue<T>(fs, is, nb, ne, rs, out, NORM == kNormDefault);
}

// Lost shards as a per-block mask, for lost sets with more runs than LostSet holds.  Up to kShardsByValue shard
// flags travel inside the launch parameters (so the call reads no host memory after it returns and can be
// recorded by stream capture); longer masks are read from device memory.
constexpr int kShardsByValue = 1024;
struct ShardFlags {
    uint8_t lost[kShardsByValue];
};
static __global__ void __launch_bounds__(kThreads)
k_expand_shards(Geom g, ShardFlags by_value, const uint8_t *__restrict__ shard_mask, uint8_t *__restrict__ block_mask) {
    const uint64_t b = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    if (b >= g.n_blocks) return;
    const uint32_t s = g.shard_of((uint32_t)b);
    block_mask[b] = (shard_mask ? shard_mask[s] : by_value.lost[s]) != 0;
}

// ---- reduction of per-block partials as a kernel of its own -----------------------
// (layouts cut into segments: their per-block partials come from a combine kernel, see segments.cuh)

constexpr int kReduceTile = 1024;  // work items per CTA in the reduction
constexpr int kReducePer = kReduceTile / kThreads;

template <typename T>
__global__ void __launch_bounds__(kThreads)
k_reduce_partials(const typename Elem<T>::score_t *__restrict__ part, Geom g, LostSet S, NormScratch rs,
                  NormInfoDev *out, bool take_sqrt) {
    double fs = 0.0;
    unsigned long long is = 0, nb = 0, ne = 0;
    const uint64_t base = (uint64_t)blockIdx.x * kReduceTile;
#pragma unroll
    for (int j = 0; j < kReducePer; ++j) {
        uint32_t b;
        if (S.block_of(base + threadIdx.x + (uint64_t)j * kThreads, b)) {
            uint64_t beg, len;
            g.range(b, beg, len);
            ++nb;
            ne += len;
            if (std::is_same<T, float>::value) fs += (double)part[b];
            else is += (unsigned long long)part[b];
        }
    }
    norm_epilogue<T>(fs, is, nb, ne, rs, out, take_sqrt);
}

// ---- plain copy (z := x at init, checkpoint reload) -------------------------

static __global__ void __launch_bounds__(kThreads)
k_copy_elems(uint32_t *__restrict__ dst, const uint32_t *__restrict__ src, uint64_t n) {
    const uint64_t nvec = n >> 2;
    const uint64_t stride = (uint64_t)gridDim.x * kThreads;
    uint4 *d4 = reinterpret_cast<uint4 *>(dst);
    const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
    for (uint64_t v = (uint64_t)blockIdx.x * kThreads + threadIdx.x; v < nvec; v += stride)
        st_stream(d4 + v, ld_stream(s4 + v));
    if (blockIdx.x == 0 && threadIdx.x < (n & 3)) dst[(nvec << 2) + threadIdx.x] = src[(nvec << 2) + threadIdx.x];
}

}  // namespace scar
