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
// The whole selection is ONE kernel, launched cooperatively (every CTA is
// resident), so its phases are separated by grid-wide barriers instead of
// kernel boundaries: the score array is small (4-8 bytes per block), and five
// to eight dependent launches cost more than the work itself.  Each CTA owns a
// contiguous range of 2048-key tiles.
//
//   digit passes   most-significant digit first: shared-memory histogram of
//                  the keys that match the prefix so far, flushed with integer
//                  atomics; barrier; every CTA resolves the digit from the
//                  global histogram (the same small scan in every CTA).
//                  Digits that are zero in every uint64 key are skipped.
//   counts         with the threshold key tau and `need` (how many keys equal
//                  to tau are taken): per-CTA counts and summed lengths of the
//                  keys above / equal to tau; barrier; every CTA scans those
//                  into its own output bases
//   boundary       only when the tau-keys run out inside one CTA's range: that
//                  CTA sums the lengths of the ones it takes; barrier
//   emit           ordered compaction into sel[] / poff[]
//
// The barrier is a counter in global memory with a bounded spin: a CTA that
// gives up records an error and leaves, and the host reports SCAR_ERR_TIMEOUT.
#pragma once
#include "block_pass.cuh"

namespace scar {

constexpr int kMaxPasses = 6;
constexpr int kHistBins = 2048;
constexpr int kSelTile = 2048;  // keys per tile
constexpr int kPerThread = kSelTile / kThreads;
constexpr unsigned kBarrierSpinLimit = 1u << 21;  // each try is a global load and a short sleep: gives up after >= 0.1 s

struct SelState {
    unsigned long long key_or;  // OR of all uint64 keys seen since the last selection
    unsigned long long partial_len;  // summed length of the tau-blocks taken in the boundary CTA
    unsigned barrier;           // arrivals at the grid barrier during the running selection
    unsigned departed;          // CTAs that have passed their last barrier
    unsigned error;             // non-zero once a barrier wait gave up
    unsigned ticket_reduce;     // ticket of the perturbation-norm reduction (block_pass.cuh)
    unsigned hist[kMaxPasses][kHistBins];
};

struct SaveInfoDev {
    unsigned long long k;
    unsigned long long payload_elems;
    unsigned long long nonfinite_blocks;
    unsigned long long error;  // copy of SelState::error at the end of the selection
};

// One entry per CTA of the selection kernel.
struct CtaArrays {
    unsigned *gt;               // keys > tau
    unsigned *eq;               // keys == tau
    unsigned *nf;               // non-finite scores
    unsigned long long *len_gt; // summed block lengths of the above
    unsigned long long *len_eq;
};

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

// Exclusive prefix sum of one value per thread over the CTA; *total gets the sum.
template <typename W> __device__ __forceinline__ W cta_excl_scan(W v, W *sh /*kThreads/32 + 1*/, W *total) {
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
    for (int i = 0; i < kThreads / 32; ++i) {
        W t = sh[i];
        if (i < w) before += t;
        all += t;
    }
    if (total) *total = all;
    return before + inc - v;
}

// Sums N values per thread over the CTA with one pair of barriers (the selection kernel is a chain of
// short dependent phases, so barriers are what it pays for).  sh holds N * kThreads / 32 words.
template <int N>
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
    for (int i = 0; i < N; ++i) {
        unsigned long long t = 0;
#pragma unroll
        for (int j = 0; j < kThreads / 32; ++j) t += sh[j * N + i];
        v[i] = t;
    }
}

// Grid-wide barrier number `phase` (1, 2, ...) of a cooperative launch: every
// CTA of the grid must call it the same number of times.  Returns false when
// the wait was abandoned (it cannot happen while all CTAs are resident, which a
// cooperative launch guarantees; the bound is there so that nothing can hang).
__device__ __forceinline__ bool grid_barrier(SelState *st, unsigned phase) {
    __shared__ bool ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned target = phase * gridDim.x;
        bool good = true;
        if (atomicAdd(&st->barrier, 1u) + 1 < target) {  // the last CTA to arrive does not wait
            volatile unsigned *ctr = &st->barrier;
            volatile unsigned *err = &st->error;
            unsigned tries = 0;
            while (*ctr < target) {
                if (++tries > kBarrierSpinLimit || ((tries & 1023u) == 0 && *err != 0)) {
                    atomicExch(&st->error, 1u);
                    good = false;
                    break;
                }
                __nanosleep(32);
            }
        }
        __threadfence();
        ok = good;
    }
    __syncthreads();
    return ok;
}

// Resolves one digit: scanning bins from the highest down, finds the bin d with
//   count(bins > d) < remaining <= count(bins >= d)
// and returns it; remaining becomes the rank wanted inside bin d.
template <int WIDTH>
__device__ __forceinline__ unsigned resolve_digit_w(const unsigned *hist, unsigned long long &remaining,
                                                    unsigned long long *sh_scan, unsigned long long *sh_out) {
    constexpr int nb = 1 << WIDTH;
    constexpr int per = nb / kThreads;  // 8 or 4: a compile-time count, so all loads are in flight together
    unsigned local[per];
    unsigned long long sum = 0;
#pragma unroll
    for (int i = 0; i < per; ++i) local[i] = __ldcg(hist + (nb - 1 - (threadIdx.x * per + i)));
#pragma unroll
    for (int i = 0; i < per; ++i) sum += local[i];
    unsigned long long cum = cta_excl_scan<unsigned long long>(sum, sh_scan, nullptr);
#pragma unroll
    for (int i = 0; i < per; ++i) {
        unsigned long long h = local[i];
        if (cum < remaining && remaining <= cum + h) {
            sh_out[0] = (unsigned long long)(nb - 1 - (threadIdx.x * per + i));
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

// Flags of the kPerThread consecutive blocks a thread owns in tile t.
template <typename S>
__device__ __forceinline__ void tile_flags(const S *__restrict__ score, unsigned long long n_blocks, unsigned t, bool none,
                                           typename ScoreKey<S>::K tau, unsigned &gt_bits, unsigned &eq_bits,
                                           unsigned &nf_bits) {
    using SK = ScoreKey<S>;
    using K = typename SK::K;
    gt_bits = eq_bits = nf_bits = 0;
    const unsigned long long first = (unsigned long long)t * kSelTile + (unsigned long long)threadIdx.x * kPerThread;
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
        unsigned long long b = first + j;
        if (b < n_blocks) {
            K key = SK::key(score[b]);
            if (SK::nonfinite(key)) nf_bits |= 1u << j;
            if (!none) {
                if (key > tau) gt_bits |= 1u << j;
                else if (key == tau) eq_bits |= 1u << j;
            }
        }
    }
}

template <typename S>
__global__ void __launch_bounds__(kThreads)
k_select(const S *__restrict__ score, Geom g, unsigned long long k, SelState *st, CtaArrays ca, SaveInfoDev *info,
         uint32_t *__restrict__ sel, unsigned long long *__restrict__ poff, unsigned n_tiles, unsigned tiles_per_cta) {
    using SK = ScoreKey<S>;
    using K = typename SK::K;
    using KT = KeyTraits<K>;
    typedef unsigned long long u64;
    __shared__ unsigned sh_hist[kHistBins];
    __shared__ u64 sh_scan[kThreads / 32 + 1];
    __shared__ u64 sh_out[2];
    __shared__ u64 sh_red[6 * kThreads / 32];
    __shared__ long long sh_boundary;
    __shared__ u64 sh_boundary_take;
    __shared__ bool sh_last;

    griddep_launch();  // the pack kernel may be scheduled while this one runs; it waits before reading sel / poff
    const u64 B = g.n_blocks;
    const unsigned t_lo = blockIdx.x * tiles_per_cta;
    const unsigned t_hi = t_lo + tiles_per_cta < n_tiles ? t_lo + tiles_per_cta : n_tiles;
    const bool none = k == 0;
    const u64 key_or = KT::kSkippable ? st->key_or : ~0ull;  // reset only after the last barrier
    unsigned phase = 0;
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
            for (int i = threadIdx.x; i < kHistBins; i += kThreads) sh_hist[i] = 0;
            __syncthreads();
            for (unsigned t = t_lo; t < t_hi; ++t) {
                const u64 base = (u64)t * kSelTile;
#pragma unroll
                for (int j = 0; j < kPerThread; ++j) {
                    const u64 i = base + threadIdx.x + (u64)j * kThreads;
                    if (i < B) {
                        const K key = SK::key(score[i]);
                        const bool match = p == 0 || ((u64)key >> (shift + width)) == prefix;
                        if (match) atomicAdd(&sh_hist[(unsigned)(((u64)key >> shift) & mask)], 1u);
                    }
                }
            }
            __syncthreads();
            for (int i = threadIdx.x; i < (1 << width); i += kThreads) {
                const unsigned c = sh_hist[i];
                if (c) atomicAdd(&st->hist[p][i], c);
            }
            alive = grid_barrier(st, ++phase);
            if (alive) prefix = (prefix << width) | resolve_digit(st->hist[p], width, need, sh_scan, sh_out);
        }
    }
    const K tau = (K)prefix;

    // ---- counts over this CTA's tiles
    u64 c_gt = 0, c_eq = 0, c_nf = 0, lgt = 0, leq = 0;
    if (alive) {
        for (unsigned t = t_lo; t < t_hi; ++t) {
            unsigned gt_bits, eq_bits, nf_bits;
            tile_flags<S>(score, B, t, none, tau, gt_bits, eq_bits, nf_bits);
            const u64 first = (u64)t * kSelTile + (u64)threadIdx.x * kPerThread;
            for (int j = 0; j < kPerThread; ++j)
                if ((gt_bits | eq_bits) >> j & 1u) {
                    uint64_t beg, len;
                    g.range((uint32_t)(first + j), beg, len);
                    if (gt_bits >> j & 1u) lgt += len;
                    else leq += len;
                }
            c_gt += __popc(gt_bits);
            c_eq += __popc(eq_bits);
            c_nf += __popc(nf_bits);
        }
        u64 five[5] = {c_gt, c_eq, c_nf, lgt, leq};
        cta_sum_n<5>(five, sh_red);
        c_gt = five[0], c_eq = five[1], c_nf = five[2], lgt = five[3], leq = five[4];
        if (threadIdx.x == 0) {
            ca.gt[blockIdx.x] = (unsigned)c_gt;
            ca.eq[blockIdx.x] = (unsigned)c_eq;
            ca.nf[blockIdx.x] = (unsigned)c_nf;
            ca.len_gt[blockIdx.x] = lgt;
            ca.len_eq[blockIdx.x] = leq;
            sh_boundary = -1;
            sh_boundary_take = 0;
        }
        alive = grid_barrier(st, ++phase);
    }

    // ---- every CTA scans the per-CTA counts into its own bases (the same scan in every CTA)
    u64 my_eq_before = 0, my_sel_base = 0, my_len_base = 0, total_n = 0, total_l = 0, total_nf = 0;
    long long cb = -1;
    if (alive) {
        u64 carry = 0, a_eq = 0, a_n = 0, a_l = 0, t_n = 0, t_l = 0, t_nf = 0;
        for (unsigned c0 = 0; c0 < gridDim.x; c0 += kThreads) {
            const unsigned c = c0 + threadIdx.x;
            const bool in = c < gridDim.x;
            const u64 e = in ? __ldcg(ca.eq + c) : 0;
            u64 tot;
            const u64 ex = carry + cta_excl_scan<u64>(e, sh_scan, &tot);
            carry += tot;
            if (in) {
                u64 take = need > ex ? need - ex : 0;
                if (take > e) take = e;
                if (take != 0 && take != e) {  // the tau-keys run out inside this CTA's range
                    sh_boundary = c;
                    sh_boundary_take = take;
                }
                const u64 n = __ldcg(ca.gt + c) + take;
                const u64 l = __ldcg(ca.len_gt + c) + (take == e ? __ldcg(ca.len_eq + c) : 0);
                t_n += n;
                t_l += l;
                t_nf += __ldcg(ca.nf + c);
                if (c < blockIdx.x) {
                    a_eq += e;
                    a_n += n;
                    a_l += l;
                }
            }
        }
        u64 six[6] = {a_eq, a_n, a_l, t_n, t_l, t_nf};
        cta_sum_n<6>(six, sh_red);
        my_eq_before = six[0], my_sel_base = six[1], my_len_base = six[2];
        total_n = six[3], total_l = six[4], total_nf = six[5];
        cb = sh_boundary;  // written before the barriers inside cta_sum_n
    }

    // ---- boundary CTA: summed length of the tau-blocks it takes (lowest ids first)
    if (alive && cb >= 0) {  // the same decision in every CTA
        if ((long long)blockIdx.x == cb) {
            const u64 take = sh_boundary_take;
            u64 run = 0, pl = 0;
            for (unsigned t = t_lo; t < t_hi; ++t) {
                unsigned gt_bits, eq_bits, nf_bits;
                tile_flags<S>(score, B, t, false, tau, gt_bits, eq_bits, nf_bits);
                u64 tot;
                u64 rank = run + cta_excl_scan<u64>(__popc(eq_bits), sh_scan, &tot);
                run += tot;
                const u64 first = (u64)t * kSelTile + (u64)threadIdx.x * kPerThread;
                for (int j = 0; j < kPerThread; ++j)
                    if (eq_bits >> j & 1u) {
                        if (rank < take) {
                            uint64_t beg, len;
                            g.range((uint32_t)(first + j), beg, len);
                            pl += len;
                        }
                        ++rank;
                    }
            }
            pl = cta_sum<u64>(pl, sh_red);
            if (threadIdx.x == 0) st->partial_len = pl;
        }
        alive = grid_barrier(st, ++phase);
        if (alive) {
            const u64 pl = __ldcg(&st->partial_len);
            total_l += pl;
            if ((long long)blockIdx.x > cb) my_len_base += pl;
        }
    }

    // ---- emit: ordered compaction of this CTA's tiles
    if (alive && !none) {
        u64 run_eq = my_eq_before, pos_base = my_sel_base, off_base = my_len_base;
        for (unsigned t = t_lo; t < t_hi; ++t) {
            unsigned gt_bits, eq_bits, nf_bits;
            tile_flags<S>(score, B, t, false, tau, gt_bits, eq_bits, nf_bits);
            u64 tot_eq, tot_n, tot_l;
            u64 rank = run_eq + cta_excl_scan<u64>(__popc(eq_bits), sh_scan, &tot_eq);
            unsigned take_bits = gt_bits;
            for (int j = 0; j < kPerThread; ++j)
                if (eq_bits >> j & 1u) {
                    if (rank < need) take_bits |= 1u << j;
                    ++rank;
                }
            const u64 first = (u64)t * kSelTile + (u64)threadIdx.x * kPerThread;
            u64 lens[kPerThread];
            u64 lsum = 0;
#pragma unroll
            for (int j = 0; j < kPerThread; ++j) {
                lens[j] = 0;
                if (take_bits >> j & 1u) {
                    uint64_t beg, len;
                    g.range((uint32_t)(first + j), beg, len);
                    lens[j] = len;
                    lsum += len;
                }
            }
            // one scan for both outputs: block counts in the top 16 bits (at most 2048 per tile), summed
            // lengths below (a buffer has fewer than 2^48 elements: init rejects more)
            u64 tot_both;
            const u64 both = cta_excl_scan<u64>(((u64)__popc(take_bits) << 48) | lsum, sh_scan, &tot_both);
            u64 pos = pos_base + (both >> 48);
            u64 off = off_base + (both & ((1ull << 48) - 1));
            tot_n = tot_both >> 48;
            tot_l = tot_both & ((1ull << 48) - 1);
#pragma unroll
            for (int j = 0; j < kPerThread; ++j)
                if (take_bits >> j & 1u) {
                    sel[pos] = (uint32_t)(first + j);
                    poff[pos] = off;
                    ++pos;
                    off += lens[j];
                }
            run_eq += tot_eq;
            pos_base += tot_n;
            off_base += tot_l;
        }
    }
    if (alive && blockIdx.x == 0 && threadIdx.x == 0) {
        info->k = total_n;
        info->payload_elems = total_l;
        info->nonfinite_blocks = total_nf;
        poff[total_n] = total_l;
    }

    // ---- the CTA that leaves last puts the shared state back for the next selection
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        sh_last = atomicAdd(&st->departed, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    for (int p = 0; p < KT::kPasses; ++p)
        for (int i = threadIdx.x; i < kHistBins; i += kThreads) st->hist[p][i] = 0;
    if (threadIdx.x == 0) {
        const unsigned err = *reinterpret_cast<volatile unsigned *>(&st->error);
        info->error = err;
        if (err) {  // a barrier gave up: nothing was selected, and the pack kernel must copy nothing
            info->k = 0;
            info->payload_elems = 0;
        }
        st->key_or = 0;  // forget which uint64 key bits were seen
        st->barrier = 0;
        st->departed = 0;
        st->error = 0;
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
