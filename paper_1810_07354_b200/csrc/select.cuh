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
//   k_radix_pass x P   most-significant digit first; each CTA first resolves the
//                      previous digit from the previous pass's global histogram
//                      (every CTA repeats the same small scan), then histograms
//                      its tile of keys that match the prefix so far
//   k_select_count     resolves the last digit -> threshold key tau and `need`
//                      (how many keys equal to tau are taken); per-tile counts;
//                      the CTA that finishes last turns them into per-tile bases
//   k_select_emit      ordered compaction into sel[] / poff[]
//
// No kernel waits on another CTA: cross-CTA order comes from kernel boundaries
// and from a ticket counter whose last taker does the epilogue.
#pragma once
#include "block_pass.cuh"

namespace scar {

constexpr int kMaxPasses = 6;
constexpr int kHistBins = 2048;
constexpr int kSelTile = 2048;  // keys per CTA in every selection kernel
constexpr int kPerThread = kSelTile / kThreads;

struct SelState {
    unsigned long long key_or;  // OR of all uint64 keys seen since the last selection
    unsigned long long prefix[kMaxPasses];
    unsigned long long remaining[kMaxPasses];
    unsigned ticket_count;
    unsigned ticket_reduce;
    unsigned hist[kMaxPasses][kHistBins];
};

struct SaveInfoDev {
    unsigned long long k;
    unsigned long long payload_elems;
    unsigned long long nonfinite_blocks;
};

struct TileArrays {
    unsigned *gt;               // keys > tau per tile
    unsigned *eq;               // keys == tau per tile
    unsigned *nf;               // non-finite scores per tile
    unsigned long long *len_gt; // summed block lengths of the above
    unsigned long long *len_eq;
    unsigned *eq_base;          // exclusive scans written by the last CTA
    unsigned *sel_base;
    unsigned long long *len_base;
};

template <typename K> struct KeyTraits;
template <> struct KeyTraits<unsigned> {
    static constexpr int kPasses = 3;
    static constexpr bool kSkippable = false;
    __host__ __device__ static constexpr int shift(int p) { return p == 0 ? 21 : (p == 1 ? 10 : 0); }
    __host__ __device__ static constexpr int width(int p) { return p == 2 ? 10 : 11; }
    static __device__ __forceinline__ unsigned key(float s) {
        unsigned u = __float_as_uint(s) & 0x7fffffffu;
        return u > 0x7f800000u ? 0x7f800000u : u;
    }
    static __device__ __forceinline__ bool nonfinite(unsigned k) { return k == 0x7f800000u; }
};
template <> struct KeyTraits<unsigned long long> {
    static constexpr int kPasses = 6;
    static constexpr bool kSkippable = true;
    __host__ __device__ static constexpr int shift(int p) {
        return p == 0 ? 53 : p == 1 ? 42 : p == 2 ? 31 : p == 3 ? 20 : p == 4 ? 10 : 0;
    }
    __host__ __device__ static constexpr int width(int p) { return p >= 4 ? 10 : 11; }
    static __device__ __forceinline__ unsigned long long key(unsigned long long s) { return s; }
    static __device__ __forceinline__ bool nonfinite(unsigned long long) { return false; }
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

// Resolves one digit: scanning bins from the highest down, finds the bin d with
//   count(bins > d) < remaining <= count(bins >= d)
// and returns it; remaining becomes the rank wanted inside bin d.
__device__ __forceinline__ unsigned resolve_digit(const unsigned *hist, int width, unsigned long long &remaining,
                                                  unsigned long long *sh_scan, unsigned long long *sh_out) {
    const int nb = 1 << width;
    const int per = nb / kThreads;  // 8 or 4
    unsigned local[kHistBins / kThreads];
    unsigned long long sum = 0;
    for (int i = 0; i < per; ++i) {
        local[i] = hist[nb - 1 - (threadIdx.x * per + i)];
        sum += local[i];
    }
    unsigned long long cum = cta_excl_scan<unsigned long long>(sum, sh_scan, nullptr);
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

// State after resolving passes 0..p-1, identical in every CTA.  p == 0: empty
// prefix, remaining = k.  CTA 0 records the newly resolved digit for the next kernel.
template <typename K>
__device__ __forceinline__ void resolve_prefix(SelState *st, int p, unsigned long long k, unsigned long long key_or,
                                               unsigned long long &prefix, unsigned long long &remaining,
                                               unsigned long long *sh_scan, unsigned long long *sh_out) {
    using KT = KeyTraits<K>;
    prefix = 0;
    remaining = k;
    if (p == 0) return;
    if (p >= 2) {
        prefix = st->prefix[p - 2];
        remaining = st->remaining[p - 2];
    }
    const int q = p - 1;
    const unsigned long long mask = (1ull << KT::width(q)) - 1;
    unsigned d = 0;
    if (!KT::kSkippable || ((key_or >> KT::shift(q)) & mask) != 0)
        d = resolve_digit(st->hist[q], KT::width(q), remaining, sh_scan, sh_out);
    prefix = (prefix << KT::width(q)) | d;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        st->prefix[q] = prefix;
        st->remaining[q] = remaining;
    }
}

template <typename K, typename S>
__global__ void __launch_bounds__(kThreads)
k_radix_pass(const S *__restrict__ score, unsigned long long n_blocks, unsigned long long k, int p, SelState *st) {
    using KT = KeyTraits<K>;
    __shared__ unsigned sh_hist[kHistBins];
    __shared__ unsigned long long sh_scan[kThreads / 32 + 1];
    __shared__ unsigned long long sh_out[2];
    const unsigned long long key_or = KT::kSkippable ? st->key_or : ~0ull;
    unsigned long long prefix, remaining;
    resolve_prefix<K>(st, p, k, key_or, prefix, remaining, sh_scan, sh_out);
    if (blockIdx.x == 0 && p + 1 < KT::kPasses)
        for (int i = threadIdx.x; i < kHistBins; i += kThreads) st->hist[p + 1][i] = 0;
    const int shift = KT::shift(p), width = KT::width(p);
    const unsigned long long mask = (1ull << width) - 1;
    if (KT::kSkippable && ((key_or >> shift) & mask) == 0) return;  // this digit is 0 in every key
    for (int i = threadIdx.x; i < kHistBins; i += kThreads) sh_hist[i] = 0;
    __syncthreads();
    const unsigned long long base = (unsigned long long)blockIdx.x * kSelTile;
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
        unsigned long long i = base + threadIdx.x + (unsigned long long)j * kThreads;
        if (i < n_blocks) {
            K key = KT::key(score[i]);
            bool match = p == 0 || ((unsigned long long)key >> (shift + width)) == prefix;
            if (match) atomicAdd(&sh_hist[(unsigned)(((unsigned long long)key >> shift) & mask)], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < (1 << width); i += kThreads) {
        unsigned c = sh_hist[i];
        if (c) atomicAdd(&st->hist[p][i], c);
    }
}

// Flags of the kPerThread consecutive blocks a thread owns in its tile.
template <typename K, typename S>
__device__ __forceinline__ void tile_flags(const S *__restrict__ score, unsigned long long n_blocks, bool none, K tau,
                                           unsigned &gt_bits, unsigned &eq_bits, unsigned &nf_bits) {
    using KT = KeyTraits<K>;
    gt_bits = eq_bits = nf_bits = 0;
    const unsigned long long first = (unsigned long long)blockIdx.x * kSelTile + (unsigned long long)threadIdx.x * kPerThread;
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
        unsigned long long b = first + j;
        if (b < n_blocks) {
            K key = KT::key(score[b]);
            if (KT::nonfinite(key)) nf_bits |= 1u << j;
            if (!none) {
                if (key > tau) gt_bits |= 1u << j;
                else if (key == tau) eq_bits |= 1u << j;
            }
        }
    }
}

template <typename K, typename S>
__global__ void __launch_bounds__(kThreads)
k_select_count(const S *__restrict__ score, Geom g, unsigned long long k, SelState *st, TileArrays ta,
               SaveInfoDev *info, unsigned long long *poff) {
    using KT = KeyTraits<K>;
    __shared__ unsigned long long sh_scan[kThreads / 32 + 1];
    __shared__ unsigned long long sh_out[2];
    __shared__ unsigned long long sh_red[kThreads / 32];
    __shared__ bool is_last;
    __shared__ long long sh_boundary;
    const bool none = k == 0;
    unsigned long long prefix = 0, need = 0;
    if (!none) {
        const unsigned long long key_or = KT::kSkippable ? st->key_or : ~0ull;
        resolve_prefix<K>(st, KT::kPasses, k, key_or, prefix, need, sh_scan, sh_out);
    }
    const K tau = (K)prefix;
    unsigned gt_bits, eq_bits, nf_bits;
    tile_flags<K, S>(score, g.n_blocks, none, tau, gt_bits, eq_bits, nf_bits);
    unsigned long long lgt = 0, leq = 0;
    const unsigned long long first = (unsigned long long)blockIdx.x * kSelTile + (unsigned long long)threadIdx.x * kPerThread;
    for (int j = 0; j < kPerThread; ++j)
        if ((gt_bits | eq_bits) >> j & 1u) {
            uint64_t beg, len;
            g.range((uint32_t)(first + j), beg, len);
            if (gt_bits >> j & 1u) lgt += len; else leq += len;
        }
    unsigned long long c_gt = cta_sum<unsigned long long>(__popc(gt_bits), sh_red);
    unsigned long long c_eq = cta_sum<unsigned long long>(__popc(eq_bits), sh_red);
    unsigned long long c_nf = cta_sum<unsigned long long>(__popc(nf_bits), sh_red);
    lgt = cta_sum<unsigned long long>(lgt, sh_red);
    leq = cta_sum<unsigned long long>(leq, sh_red);
    if (threadIdx.x == 0) {
        ta.gt[blockIdx.x] = (unsigned)c_gt;
        ta.eq[blockIdx.x] = (unsigned)c_eq;
        ta.nf[blockIdx.x] = (unsigned)c_nf;
        ta.len_gt[blockIdx.x] = lgt;
        ta.len_eq[blockIdx.x] = leq;
        __threadfence();
        is_last = atomicAdd(&st->ticket_count, 1u) == gridDim.x - 1;
        sh_boundary = -1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    const unsigned nt = gridDim.x;
    volatile unsigned *v_gt = ta.gt, *v_eq = ta.eq, *v_nf = ta.nf;
    volatile unsigned long long *v_lgt = ta.len_gt, *v_leq = ta.len_eq;

    // A: ranks of the tau-keys before each tile; find the tile where `need` runs out mid-tile.
    unsigned long long carry = 0, nf_total = 0;
    for (unsigned c = 0; c < nt; c += kThreads) {
        unsigned t = c + threadIdx.x;
        unsigned long long e = t < nt ? v_eq[t] : 0, tot;
        unsigned long long ex = carry + cta_excl_scan<unsigned long long>(e, sh_scan, &tot);
        if (t < nt) {
            ta.eq_base[t] = (unsigned)ex;
            if (ex < need && need < ex + e) sh_boundary = t;
            nf_total += v_nf[t];
        }
        carry += tot;
        __syncthreads();
    }
    nf_total = cta_sum<unsigned long long>(nf_total, sh_red);
    __syncthreads();
    const long long tb = sh_boundary;

    // B: summed length of the tau-blocks actually taken inside the boundary tile.
    unsigned long long partial_len = 0;
    if (tb >= 0) {
        const unsigned long long tfirst = (unsigned long long)tb * kSelTile + (unsigned long long)threadIdx.x * kPerThread;
        unsigned eb = 0;
        for (int j = 0; j < kPerThread; ++j) {
            unsigned long long b = tfirst + j;
            if (b < g.n_blocks && KT::key(score[b]) == tau) eb |= 1u << j;
        }
        unsigned long long rank = ta.eq_base[tb] + cta_excl_scan<unsigned long long>(__popc(eb), sh_scan, nullptr);
        unsigned long long pl = 0;
        for (int j = 0; j < kPerThread; ++j)
            if (eb >> j & 1u) {
                if (rank < need) {
                    uint64_t beg, len;
                    g.range((uint32_t)(tfirst + j), beg, len);
                    pl += len;
                }
                ++rank;
            }
        partial_len = cta_sum<unsigned long long>(pl, sh_red);
        __syncthreads();
    }

    // C: per-tile output bases.
    unsigned long long carry_n = 0, carry_l = 0;
    for (unsigned c = 0; c < nt; c += kThreads) {
        unsigned t = c + threadIdx.x;
        unsigned long long n = 0, l = 0, tot_n, tot_l;
        if (t < nt) {
            unsigned long long e = v_eq[t], ex = ta.eq_base[t];
            unsigned long long take = need > ex ? need - ex : 0;
            if (take > e) take = e;
            n = v_gt[t] + take;
            l = v_lgt[t];
            if (take == e) l += v_leq[t];
            else if (take != 0) l += partial_len;
        }
        unsigned long long exn = carry_n + cta_excl_scan<unsigned long long>(n, sh_scan, &tot_n);
        unsigned long long exl = carry_l + cta_excl_scan<unsigned long long>(l, sh_scan, &tot_l);
        if (t < nt) {
            ta.sel_base[t] = (unsigned)exn;
            ta.len_base[t] = exl;
        }
        carry_n += tot_n;
        carry_l += tot_l;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        info->k = carry_n;
        info->payload_elems = carry_l;
        info->nonfinite_blocks = nf_total;
        poff[carry_n] = carry_l;
        st->ticket_count = 0;
    }
}

template <typename K, typename S>
__global__ void __launch_bounds__(kThreads)
k_select_emit(const S *__restrict__ score, Geom g, SelState *st, TileArrays ta, uint32_t *__restrict__ sel,
              unsigned long long *__restrict__ poff) {
    using KT = KeyTraits<K>;
    __shared__ unsigned long long sh_scan[kThreads / 32 + 1];
    const K tau = (K)st->prefix[KT::kPasses - 1];
    const unsigned long long need = st->remaining[KT::kPasses - 1];
    unsigned gt_bits, eq_bits, nf_bits;
    tile_flags<K, S>(score, g.n_blocks, false, tau, gt_bits, eq_bits, nf_bits);
    unsigned long long rank =
        ta.eq_base[blockIdx.x] + cta_excl_scan<unsigned long long>(__popc(eq_bits), sh_scan, nullptr);
    unsigned take_bits = gt_bits;
    for (int j = 0; j < kPerThread; ++j)
        if (eq_bits >> j & 1u) {
            if (rank < need) take_bits |= 1u << j;
            ++rank;
        }
    const unsigned long long first = (unsigned long long)blockIdx.x * kSelTile + (unsigned long long)threadIdx.x * kPerThread;
    unsigned long long lens[kPerThread];
    unsigned long long lsum = 0;
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
    unsigned long long pos =
        ta.sel_base[blockIdx.x] + cta_excl_scan<unsigned long long>(__popc(take_bits), sh_scan, nullptr);
    unsigned long long off = ta.len_base[blockIdx.x] + cta_excl_scan<unsigned long long>(lsum, sh_scan, nullptr);
#pragma unroll
    for (int j = 0; j < kPerThread; ++j)
        if (take_bits >> j & 1u) {
            sel[pos] = (uint32_t)(first + j);
            poff[pos] = off;
            ++pos;
            off += lens[j];
        }
    // Selection is over: forget which uint64 key bits were seen.
    if (blockIdx.x == 0 && threadIdx.x == 0) st->key_or = 0;
}

}  // namespace scar
