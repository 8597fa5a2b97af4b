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

template <int G, typename W> __device__ __forceinline__ W group_sum(W v) {
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One batch = four units (16-byte vectors, or single elements on the
// element-wise path) per stream and lane, G units apart.  Units past the end of
// the block load as zero, which adds nothing to either distance.
template <typename U, int G>
__device__ __forceinline__ void load_batch(const U *__restrict__ xs, const U *__restrict__ zs, uint64_t u, uint64_t n,
                                           U (&xr)[4], U (&zr)[4]) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint64_t i = u + (uint64_t)j * G;
        if (i < n) {
            xr[j] = ld_stream(xs + i);
            zr[j] = ld_stream(zs + i);
        } else {
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
    if (!WRITE) {
        // Read-only pass: nothing can hold back the loads, so the plain loop is
        // the faster form (full batches unguarded, then one guarded batch).  A
        // batch counts as full only when it is full for every lane of the group,
        // so the lanes of a group never diverge between the two forms.
        for (; u - lane + step <= n; u += step) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                xc[j] = ld_stream(xs + u + (uint64_t)j * G);
                zc[j] = ld_stream(zs + u + (uint64_t)j * G);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) E::addu(a[j], xc[j], zc[j]);
            if (E::kFlush && (++it & kFlushMask) == 0) {
                total += ((wide_t)a[0] + (wide_t)a[1]) + ((wide_t)a[2] + (wide_t)a[3]);
                a[0] = a[1] = a[2] = a[3] = 0;
            }
        }
        if (u < n) {
            load_batch<U, G>(xs, zs, u, n, xc, zc);
#pragma unroll
            for (int j = 0; j < 4; ++j) E::addu(a[j], xc[j], zc[j]);
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

struct SelState;  // select.cuh

// Block total -> stored score, times the block's weight when the caller set
// weights (float data only; Appendix C: a positive combination of block norms
// is still a norm).
template <typename E>
__device__ __forceinline__ typename E::score_t weighted(typename E::wide_t s, const float *__restrict__ weight,
                                                        uint64_t b) {
    if (std::is_same<typename E::wide_t, double>::value && weight) s = (typename E::wide_t)((double)s * (double)weight[b]);
    return (typename E::score_t)s;
}

template <typename T, int NORM, int G, bool VEC>
__global__ void __launch_bounds__(kThreads)
k_block_scores(const T *__restrict__ x, const T *__restrict__ z, Geom g, const float *__restrict__ weight,
               typename Elem<T, NORM>::score_t *__restrict__ score, unsigned long long *key_or, unsigned *hist0,
               int hist0_len) {
    using E = Elem<T, NORM>;
    const int lane = threadIdx.x & (G - 1);
    const uint64_t grp = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    const bool valid = grp < g.n_blocks;
    uint64_t beg = 0, len = 0;
    if (valid) g.range((uint32_t)grp, beg, len);
    typename E::wide_t s = block_distance<T, NORM, G, VEC, false>(const_cast<T *>(x), z, beg, len, lane);
    if (valid && lane == 0) {
        typename E::score_t sc = weighted<E>(s, weight, grp);
        score[grp] = sc;
        if (sizeof(typename E::score_t) == 8) {
            // Remember which key bits occur at all, so that radix passes over
            // digits that are zero in every key can be skipped.
            unsigned long long bits = (unsigned long long)sc;
            unsigned long long seen = *reinterpret_cast<volatile unsigned long long *>(key_or);
            if (bits & ~seen) atomicOr(key_or, bits);
        }
    }
    // The first radix histogram is accumulated after this kernel; clear it here.
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i < hist0_len; i += kThreads) hist0[i] = 0;
}

// ---- a4 / a5: per-block perturbation over the lost set, optional restore ---

template <typename T, int NORM, int G, bool VEC, bool WRITE>
__global__ void __launch_bounds__(kThreads)
k_recover_blocks(T *__restrict__ x, const T *__restrict__ z, Geom g, LostSet S, const float *__restrict__ weight,
                 typename Elem<T, NORM>::score_t *__restrict__ part) {
    using E = Elem<T, NORM>;
    griddep_launch();  // the reduction that follows may be scheduled early; it waits for this grid before reading
    const int lane = threadIdx.x & (G - 1);
    if (G < 32 && S.mode == 2) {
        // Per-block mask with several blocks per warp: a warp takes 32 consecutive
        // blocks, ballots which are lost and hands only those to its groups, so that
        // a sparse mask does not leave most lanes idle.
        constexpr int kGroups = 32 / G;
        const int wl = threadIdx.x & 31, gi = wl / G;
        const uint64_t b0 = (((uint64_t)blockIdx.x * kThreads + threadIdx.x) >> 5) * 32;
        const bool lost = b0 + wl < g.n_blocks && S.mask[b0 + wl] != 0;
        const unsigned bal = __ballot_sync(0xffffffffu, lost);
        const int cnt = __popc(bal);
        for (int t0 = 0; t0 < cnt; t0 += kGroups) {  // same trip count for every lane of the warp
            const int t = t0 + gi;
            const bool valid = t < cnt;
            uint32_t b = 0;
            uint64_t beg = 0, len = 0;
            if (valid) {
                b = (uint32_t)(b0 + __fns(bal, 0, t + 1));
                g.range(b, beg, len);
            }
            typename E::wide_t s = block_distance<T, NORM, G, VEC, WRITE>(x, z, beg, len, lane);
            if (valid && lane == 0) part[b] = weighted<E>(s, weight, b);
        }
        return;
    }
    const uint64_t w = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    uint32_t b = 0;
    const bool valid = S.block_of(w, b);
    uint64_t beg = 0, len = 0;
    if (valid) g.range(b, beg, len);
    typename E::wide_t s = block_distance<T, NORM, G, VEC, WRITE>(x, z, beg, len, lane);
    if (valid && lane == 0) part[b] = weighted<E>(s, weight, b);
}

// Lost shards as a per-block mask, for lost sets with more runs than LostSet holds.
static __global__ void __launch_bounds__(kThreads)
k_expand_shards(Geom g, const uint8_t *__restrict__ shard_mask, uint8_t *__restrict__ block_mask) {
    const uint64_t b = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    if (b < g.n_blocks) block_mask[b] = shard_mask[g.shard_of((uint32_t)b)] != 0;
}

// ---- final reduction of the per-block partials in a fixed order -------------

struct NormInfoDev {
    double l2;
    unsigned long long l1;
    unsigned long long lost_blocks;
    unsigned long long lost_elems;
};

constexpr int kReduceTile = 1024;  // work items per CTA in the reduction
constexpr int kReducePer = kReduceTile / kThreads;

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

// Each CTA sums a fixed tile of per-block partials (fp64 for float data, exact
// 64-bit for integer data) together with the lost block/element counts; the
// CTA that finishes last adds the tile sums in tile order.  Which CTA is last
// does not affect the order of any addition.
template <typename T>
__global__ void __launch_bounds__(kThreads)
k_reduce_partials(const typename Elem<T>::score_t *__restrict__ part, Geom g, LostSet S, double *tile_sum,
                  unsigned long long *tile_l1, unsigned long long *tile_blocks, unsigned long long *tile_elems,
                  unsigned *ticket, NormInfoDev *out, bool take_sqrt) {
    __shared__ double shd[kThreads / 32];
    __shared__ unsigned long long shu[kThreads / 32];
    __shared__ bool is_last;
    griddep_wait();
    const uint64_t base = (uint64_t)blockIdx.x * kReduceTile;
    double fs = 0.0;
    unsigned long long is = 0, nb = 0, ne = 0;
    uint32_t bj[kReducePer];
    bool ok[kReducePer];
#pragma unroll
    for (int j = 0; j < kReducePer; ++j) ok[j] = S.block_of(base + threadIdx.x + (uint64_t)j * kThreads, bj[j]);
    typename Elem<T>::score_t pj[kReducePer];
#pragma unroll
    for (int j = 0; j < kReducePer; ++j) pj[j] = ok[j] ? part[bj[j]] : (typename Elem<T>::score_t)0;
#pragma unroll
    for (int j = 0; j < kReducePer; ++j)
        if (ok[j]) {
            uint64_t beg, len;
            g.range(bj[j], beg, len);
            ++nb;
            ne += len;
            if (std::is_same<T, float>::value) fs += (double)pj[j];
            else is += (unsigned long long)pj[j];
        }
    fs = cta_sum<double>(fs, shd);
    is = cta_sum<unsigned long long>(is, shu);
    nb = cta_sum<unsigned long long>(nb, shu);
    ne = cta_sum<unsigned long long>(ne, shu);
    if (threadIdx.x == 0) {
        tile_sum[blockIdx.x] = fs;
        tile_l1[blockIdx.x] = is;
        tile_blocks[blockIdx.x] = nb;
        tile_elems[blockIdx.x] = ne;
        __threadfence();
        is_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    fs = 0.0; is = 0; nb = 0; ne = 0;
    for (unsigned t = threadIdx.x; t < gridDim.x; t += kThreads) {
        fs += *reinterpret_cast<volatile double *>(tile_sum + t);
        is += *reinterpret_cast<volatile unsigned long long *>(tile_l1 + t);
        nb += *reinterpret_cast<volatile unsigned long long *>(tile_blocks + t);
        ne += *reinterpret_cast<volatile unsigned long long *>(tile_elems + t);
    }
    fs = cta_sum<double>(fs, shd);
    is = cta_sum<unsigned long long>(is, shu);
    nb = cta_sum<unsigned long long>(nb, shu);
    ne = cta_sum<unsigned long long>(ne, shu);
    if (threadIdx.x == 0) {
        out->l2 = take_sqrt ? sqrt(fs) : fs;  // l2 norms sum squares; l1 / weighted-l1 norms sum as they are
        out->l1 = is;
        out->lost_blocks = nb;
        out->lost_elems = ne;
        *ticket = 0;
    }
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
