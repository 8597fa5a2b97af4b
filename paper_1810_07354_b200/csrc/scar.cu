// Host side of libscar: context, argument validation, launch sequencing and
// the extern "C" entry points declared in include/scar.h.  Every step of the
// checkpoint / recovery pass runs in the kernels of block_pass.cuh, select.cuh
// and pack.cuh; there is no CPU path.
#include <algorithm>
#include <cerrno>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <new>
#include <type_traits>
#include <vector>

#include <unistd.h>

#include "scar.h"

#include "block_pass.cuh"
#include "pack.cuh"
#include "segments.cuh"
#include "select.cuh"

using namespace scar;

namespace {

constexpr int kNumEvents = 6;

}  // namespace

// Device buffers one save writes: payload, id list, offsets, result record.
struct OutSet {
    void *payload = nullptr;
    uint32_t *sel = nullptr;
    unsigned long long *poff = nullptr;
    SaveInfoDev *info = nullptr;
};

// One of the two slots of the asynchronous drain (Section 4.3: the output to storage happens in the
// background while training resumes): a device output set plus its pinned host mirror.
struct DrainSlot {
    OutSet dev{};
    void *h_payload = nullptr;
    uint32_t *h_sel = nullptr;
    unsigned long long *h_poff = nullptr;
    SaveInfoDev *h_info = nullptr;
    cudaEvent_t saved = nullptr, drained = nullptr;
    uint64_t k = 0, ticket = 0;
    int state = 0;  // 0 free, 1 holds a save that was not handed to the drain, 2 draining, 3 host owns the buffers
};

struct scar_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    scar_dtype dt = SCAR_F32;
    Geom g{};
    int group_lanes = 32;

    void *x = nullptr;  // caller-owned
    void *z = nullptr;
    OutSet cur{};   // where the next save writes
    OutSet last{};  // what the most recent save wrote (views and result fetches read this)
    void *score = nullptr;  // float[B] or uint64[B]
    void *part = nullptr;   // per-block perturbation partials, same type as score (segment mode only)
    uint64_t *d_boff = nullptr;
    // segment mode (layouts with very long blocks)
    bool seg_mode = false;
    Segs segs{};
    void *seg_part = nullptr;      // double[n_segs] or uint64[n_segs]
    uint32_t *wide_blocks = nullptr;  // blocks with more than kWideSegs segments
    unsigned n_wide_blocks = 0;
    int norm = SCAR_NORM_DEFAULT;
    float *d_weight = nullptr;  // per-block weights of the norm, or nullptr
    float *d_weight_buf = nullptr;
    uint8_t *d_shard_mask = nullptr;  // only for shard masks too long to travel in launch parameters
    uint8_t *h_shard_mask = nullptr;  // pinned staging copy of such a mask
    uint8_t *d_block_mask = nullptr;  // only used when a shard mask has too many runs
    SelState *st = nullptr;
    // multi-GPU form of a save (scar_ckpt_priority_save_sharded): scratch for the selection over all ranks' scores
    OutSet glob{};                 // ids / offsets / record of the global selection (no payload)
    uint64_t glob_blocks = 0;      // capacity of glob in blocks
    uint32_t *member = nullptr;    // B flags: this rank's blocks that the global selection took
    unsigned long long *d_count = nullptr;  // how many
    unsigned long long *h_count = nullptr;  // pinned
    bool arm_never = false;  // self-test: the next selection's waits expect an arrival that never comes
    int n_sms = 1;
    NormScratch rs{};  // per-CTA / per-tile partials and tickets of the fused norm reduction
    unsigned long long *norm_scratch = nullptr;  // what rs points into
    size_t norm_scratch_bytes = 0;
    NormInfoDev *d_norm = nullptr;
    SaveInfoDev *h_save = nullptr;  // pinned
    NormInfoDev *h_norm = nullptr;  // pinned
    bool have_save = false, have_norm = false;

    // asynchronous drain (off until scar_ckpt_drain_init)
    bool drain = false;
    DrainSlot slot[2];
    int cur_slot = 0;
    cudaStream_t drain_stream = nullptr;
    uint64_t drain_cap_k = 0, drain_cap_elems = 0, next_ticket = 0;
    uint64_t max_block_len = 0;

    // persistent copy of the running checkpoint (scar_ckpt_store_* / scar_ckpt_load_stored)
    std::vector<uint64_t> h_boff;  // host copy of explicit block offsets (empty for implicit layouts)
    std::vector<uint64_t> longest_prefix;  // explicit layouts: [k] = elements of the k longest blocks
    char *io_stage = nullptr;      // pinned staging buffer for whole-checkpoint transfers

    // debug contexts (scar_ckpt_init_guarded): every device allocation sits between two bands of kGuardBytes
    // bytes of a known pattern
    bool guarded = false;
    struct Band {
        const uint8_t *user;  // the buffer the library uses
        size_t bytes;         // its size: the bands are [user - kGuardBytes, user) and [user + bytes, + kGuardBytes)
    };
    std::vector<Band> bands;
    unsigned long long *d_bad = nullptr;  // result of the guard check

    std::vector<void *> owned;  // device allocations to free
    std::vector<void *> owned_host;  // pinned host allocations to free
    uint64_t launches = 0;
    uint64_t round_cursor = 0;  // first block of the next round-robin save

    bool profile = false;
    cudaEvent_t ev[kNumEvents] = {};
    int last_call = 0;  // 1 = save, 2 = recover / norm, 3 = scores only
    bool ran_select = false, ran_pack = false;
};

namespace {

#define CU_TRY(expr)                                  \
    do {                                              \
        cudaError_t e_ = (expr);                      \
        if (e_ != cudaSuccess) return SCAR_ERR_CUDA;  \
    } while (0)

int check_device(const scar_ctx *c) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SCAR_ERR_CUDA;
    return dev == c->device ? SCAR_OK : SCAR_ERR_STATE;
}

constexpr size_t kGuardBytes = 256;  // keeps guarded buffers 256-byte aligned, like cudaMalloc's own
constexpr int kGuardPattern = 0xA5;

template <typename P> int dev_alloc(scar_ctx *c, P **p, size_t bytes) {
    void *q = nullptr;
    if (bytes == 0) bytes = 16;
    if (!c->guarded) {
        if (cudaMalloc(&q, bytes) != cudaSuccess) {
            cudaGetLastError();
            return SCAR_ERR_ALLOC;
        }
        c->owned.push_back(q);
        *p = static_cast<P *>(q);
        return SCAR_OK;
    }
    // the tail band starts at the first byte behind the buffer, so an overrun of a single element lands in it
    if (cudaMalloc(&q, bytes + 2 * kGuardBytes) != cudaSuccess) {
        cudaGetLastError();
        return SCAR_ERR_ALLOC;
    }
    c->owned.push_back(q);
    uint8_t *user = static_cast<uint8_t *>(q) + kGuardBytes;
    if (cudaMemsetAsync(q, kGuardPattern, kGuardBytes, c->stream) != cudaSuccess ||
        cudaMemsetAsync(user + bytes, kGuardPattern, kGuardBytes, c->stream) != cudaSuccess)
        return SCAR_ERR_CUDA;
    c->bands.push_back({user, bytes});
    *p = reinterpret_cast<P *>(user);
    return SCAR_OK;
}

// One CTA per buffer: counts the bytes of its two bands that no longer hold the pattern.
constexpr int kBandsPerLaunch = 48;
struct BandList {
    const uint8_t *user[kBandsPerLaunch];
    unsigned long long bytes[kBandsPerLaunch];
};
__global__ void __launch_bounds__(kThreads)
k_check_guards(BandList list, unsigned long long *bad) {
    const uint8_t *user = list.user[blockIdx.x];
    unsigned wrong = 0;
    for (unsigned i = threadIdx.x; i < 2 * kGuardBytes; i += kThreads) {
        const uint8_t v = i < kGuardBytes ? user[(long long)i - (long long)kGuardBytes]
                                          : user[list.bytes[blockIdx.x] + (i - kGuardBytes)];
        wrong += v != (uint8_t)kGuardPattern;
    }
    wrong = __reduce_add_sync(0xffffffffu, wrong);
    if ((threadIdx.x & 31) == 0 && wrong) atomicAdd(bad, (unsigned long long)wrong);
}

// Validates the caller's layout and fills the host-side fields of Geom
// (boff is set later, once the offsets are on the device).
int resolve_layout(const scar_layout *L, Geom &g) {
    if (L->n_shards < 1 || L->n_elems >= (1ull << 48)) return SCAR_ERR_LAYOUT;
    g = Geom{};
    g.n_elems = L->n_elems;
    g.n_shards = L->n_shards;
    if (L->block_offsets) {
        const uint64_t nb = L->n_blocks;
        if (nb > 0xffffffffull - 1) return SCAR_ERR_LAYOUT;
        const uint64_t *o = L->block_offsets;
        if (o[0] != 0 || o[nb] != L->n_elems) return SCAR_ERR_LAYOUT;
        bool vec = true;
        for (uint64_t b = 0; b < nb; ++b) {
            if (o[b + 1] < o[b]) return SCAR_ERR_LAYOUT;
            if (o[b] & 3) vec = false;
        }
        if (o[nb] & 3) vec = false;
        g.n_blocks = nb;
        g.row_len = L->n_elems;
        g.block_elems = 0;
        g.blocks_per_row = 0;
        g.vec_ok = vec;
        return SCAR_OK;
    }
    if (L->n_elems == 0) {
        g.n_blocks = 0;
        g.row_len = 0;
        g.block_elems = L->block_elems ? L->block_elems : 1;
        g.blocks_per_row = 1;
        g.vec_ok = 1;
        return SCAR_OK;
    }
    if (L->block_elems == 0) return SCAR_ERR_LAYOUT;
    const uint64_t row = L->row_elems ? L->row_elems : L->n_elems;
    if (row > L->n_elems || L->n_elems % row != 0) return SCAR_ERR_LAYOUT;
    const uint64_t per_row = (row + L->block_elems - 1) / L->block_elems;
    const uint64_t rows = L->n_elems / row;
    if (per_row > 0xfffffffeull || rows > 0xfffffffeull || per_row * rows > 0xfffffffeull) return SCAR_ERR_LAYOUT;
    g.row_len = row;
    g.block_elems = L->block_elems;
    g.blocks_per_row = (uint32_t)per_row;
    g.n_blocks = per_row * rows;
    g.vec_ok = (row % 4 == 0) && (L->block_elems % 4 == 0);
    return SCAR_OK;
}

// Lanes per block: about four 16-byte vectors (or four elements on the
// element-wise path) per lane and stream, between 4 lanes and a full warp.
int pick_group_lanes(const Geom &g) {
    if (g.n_blocks == 0) return 32;
    double units = (double)g.n_elems / (double)g.n_blocks;
    if (g.vec_ok) units /= 4.0;
    int G = 4;
    while (G < 32 && G * 4 < units) G <<= 1;
    return G;
}

template <typename F> void dispatch_group(int G, bool vec, F &&f) {
    auto go = [&](auto gl) {
        if (vec) f(gl, std::true_type{});
        else f(gl, std::false_type{});
    };
    switch (G) {
        case 4: go(std::integral_constant<int, 4>{}); break;
        case 8: go(std::integral_constant<int, 8>{}); break;
        case 16: go(std::integral_constant<int, 16>{}); break;
        default: go(std::integral_constant<int, 32>{}); break;
    }
}

unsigned grid_for_groups(uint64_t n_groups, int G) {
    const uint64_t per_cta = kThreads / G;
    return (unsigned)((n_groups + per_cta - 1) / per_cta);
}

// Launch that may overlap the tail of the kernel before it on the stream (the kernel calls griddep_wait()
// before it reads that kernel's output).  Off while per-phase timing is on: phases would blur.
template <typename... KArgs, typename... Args>
void launch_after(scar_ctx *c, void (*kern)(KArgs...), unsigned grid, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = c->stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = c->profile ? 0 : 1;
    cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

void record(scar_ctx *c, int i) {
    if (c->profile) cudaEventRecord(c->ev[i], c->stream);
}

// a1
// info: result record of the save this scoring pass belongs to (cleared by the kernel), or nullptr
template <typename T, int NORM> void launch_scores_as(scar_ctx *c, SaveInfoDev *info) {
    using S = typename Elem<T, NORM>::score_t;
    dispatch_group(c->group_lanes, c->g.vec_ok != 0, [&](auto gl, auto vec) {
        constexpr int G = decltype(gl)::value;
        constexpr bool VEC = decltype(vec)::value;
        k_block_scores<T, NORM, G, VEC><<<grid_for_groups(c->g.n_blocks, G), kThreads, 0, c->stream>>>(
            static_cast<const T *>(c->x), static_cast<const T *>(c->z), c->g, c->d_weight, static_cast<S *>(c->score),
            c->st, info);
    });
    ++c->launches;
}

unsigned grid_for_warps(uint64_t n_warps) { return (unsigned)((n_warps + kThreads / 32 - 1) / (kThreads / 32)); }

// Segment sums -> block totals: one warp per block, plus one CTA per block that has very many segments.
template <typename T, int NORM>
void launch_combine(scar_ctx *c, const typename Elem<T, NORM>::wide_t *sp, const uint8_t *mask,
                    typename Elem<T, NORM>::score_t *out, unsigned long long *key_or, SelState *sel_state,
                    SaveInfoDev *info) {
    k_combine_segments<T, NORM, false><<<grid_for_warps(c->g.n_blocks), kThreads, 0, c->stream>>>(
        c->segs, c->g.n_blocks, nullptr, sp, c->d_weight, mask, out, key_or, sel_state, info);
    ++c->launches;
    if (c->n_wide_blocks) {
        k_combine_segments<T, NORM, true><<<c->n_wide_blocks, kThreads, 0, c->stream>>>(
            c->segs, c->g.n_blocks, c->wide_blocks, sp, c->d_weight, mask, out, key_or, nullptr, nullptr);
        ++c->launches;
    }
}

template <typename T, int NORM> void launch_segment_scores(scar_ctx *c, SaveInfoDev *info) {
    using W = typename Elem<T, NORM>::wide_t;
    using S = typename Elem<T, NORM>::score_t;
    T *x = static_cast<T *>(c->x);
    const T *z = static_cast<const T *>(c->z);
    W *sp = static_cast<W *>(c->seg_part);
    if (c->g.vec_ok)
        k_segment_pass<T, NORM, true, false><<<grid_for_warps(c->segs.n), kThreads, 0, c->stream>>>(x, z, c->g, c->segs,
                                                                                                 nullptr, sp);
    else
        k_segment_pass<T, NORM, false, false><<<grid_for_warps(c->segs.n), kThreads, 0, c->stream>>>(x, z, c->g, c->segs,
                                                                                                  nullptr, sp);
    launch_combine<T, NORM>(c, sp, nullptr, static_cast<S *>(c->score), &c->st->key_or, c->st, info);
    ++c->launches;
}

void launch_scores(scar_ctx *c, SaveInfoDev *info) {
    if (c->g.n_blocks == 0) return;
    if (c->seg_mode) {
        if (c->dt == SCAR_I32) launch_segment_scores<int, kNormDefault>(c, info);
        else if (c->norm == SCAR_NORM_L1) launch_segment_scores<float, kNormL1>(c, info);
        else launch_segment_scores<float, kNormDefault>(c, info);
        return;
    }
    if (c->dt == SCAR_I32) launch_scores_as<int, kNormDefault>(c, info);
    else if (c->norm == SCAR_NORM_L1) launch_scores_as<float, kNormL1>(c, info);
    else launch_scores_as<float, kNormDefault>(c, info);
}

// a1 + a3 fused for k == B
template <typename T, int NORM> void launch_full_save(scar_ctx *c) {
    using S = typename Elem<T, NORM>::score_t;
    dispatch_group(c->group_lanes, c->g.vec_ok != 0, [&](auto gl, auto vec) {
        constexpr int G = decltype(gl)::value;
        constexpr bool VEC = decltype(vec)::value;
        k_full_save<T, NORM, G, VEC><<<grid_for_groups(c->g.n_blocks, G), kThreads, 0, c->stream>>>(
            static_cast<const T *>(c->x), static_cast<T *>(c->z), static_cast<T *>(c->cur.payload), c->g, c->d_weight,
            static_cast<S *>(c->score), c->cur.sel, c->cur.poff, c->cur.info);
    });
    ++c->launches;
}

// Launch shape of a selection over n_blocks keys: contiguous tile ranges over at most one CTA per SM (few enough
// that a meeting of all CTAs costs a couple of microseconds, always resident, and fewer than the exchange has
// threads).
struct SelectShape {
    unsigned n_tiles, tiles_per_cta, grid;
};
SelectShape select_shape(const scar_ctx *c, uint64_t n_blocks) {
    SelectShape sh;
    sh.n_tiles = (unsigned)((n_blocks + kSelTile - 1) / kSelTile);
    if (sh.n_tiles == 0) sh.n_tiles = 1;
    const unsigned cap = (unsigned)c->n_sms < (unsigned)kMaxSelCtas - 1 ? (unsigned)c->n_sms : (unsigned)kMaxSelCtas - 1;
    sh.tiles_per_cta = (sh.n_tiles + cap - 1) / cap;
    sh.grid = (sh.n_tiles + sh.tiles_per_cta - 1) / sh.tiles_per_cta;
    return sh;
}

// a2: one cooperative launch (all CTAs resident, so its waits cannot deadlock) over the keys `score` of the
// blocks of `g`, writing ids, offsets and the result record to `to`.  The selection state must be zero when the
// kernel starts: the scoring pass that precedes a prioritized save clears it (pre_cleared), any other caller
// gets a memset here.
template <typename S>
int launch_select(scar_ctx *c, const S *score, const Geom &g, uint64_t k, const OutSet &to, bool pre_cleared) {
    if (!pre_cleared) {
        CU_TRY(cudaMemsetAsync(reinterpret_cast<char *>(c->st) + kSelZeroFrom, 0, sizeof(SelState) - kSelZeroFrom,
                               c->stream));
        CU_TRY(cudaMemsetAsync(to.info, 0, sizeof(SaveInfoDev), c->stream));
    }
    const SelectShape sh = select_shape(c, g.n_blocks);
    Geom geom = g;
    OutSet out = to;
    unsigned long long kk = k;
    unsigned k32 = (unsigned)k, nt = sh.n_tiles, per = sh.tiles_per_cta, never = c->arm_never ? 1u : 0u;
    c->arm_never = false;
    if (per == 1 && sh.grid == 1) {
        // A single CTA has nobody to wait for: no co-residency to guarantee, a plain launch starts sooner, and its
        // histograms never leave shared memory.  (The timeout self-test needs a wait, so it runs the form that has one.)
        if (never)
            k_select_tile<S, false><<<1, kSelThreads, 0, c->stream>>>(score, geom, k32, c->st, out.info, out.sel, out.poff, never);
        else
            k_select_tile<S, true><<<1, kSelThreads, 0, c->stream>>>(score, geom, k32, c->st, out.info, out.sel, out.poff, never);
        CU_TRY(cudaGetLastError());
    } else if (per == 1) {  // the usual case: one tile per CTA
        void *args[] = {&score, &geom, &k32, &c->st, &out.info, &out.sel, &out.poff, &never};
        CU_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(&k_select_tile<S, false>), dim3(sh.grid),
                                           dim3(kSelThreads), args, 0, c->stream));
    } else {
        void *args[] = {&score, &geom, &kk, &c->st, &out.info, &out.sel, &out.poff, &nt, &per, &never};
        CU_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(&k_select<S>), dim3(sh.grid),
                                           dim3(kSelThreads), args, 0, c->stream));
    }
    ++c->launches;
    return SCAR_OK;
}

// Checks once that the selection kernels can be launched cooperatively and notes the SM count.
template <typename S> int select_occupancy(int &occ) {
    int o = 0;
    CU_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, k_select<S>, kSelThreads, 0));
    occ = o < occ ? o : occ;
    CU_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, k_select_tile<S, false>, kSelThreads, 0));
    occ = o < occ ? o : occ;
    return SCAR_OK;
}

int plan_select(scar_ctx *c) {
    int coop = 0, sms = 0, occ = 1 << 30, rc;
    CU_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device));
    CU_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device));
    if ((rc = select_occupancy<float>(occ)) != SCAR_OK || (rc = select_occupancy<unsigned long long>(occ)) != SCAR_OK ||
        (rc = select_occupancy<unsigned>(occ)) != SCAR_OK)
        return rc;
    if (!coop || sms < 1 || occ < 1) return SCAR_ERR_CUDA;
    c->n_sms = sms;
    return SCAR_OK;
}

// a1 + a3 fused for k == B on a segmented layout
template <typename T, int NORM> void launch_full_save_segments_as(scar_ctx *c) {
    using W = typename Elem<T, NORM>::wide_t;
    using S = typename Elem<T, NORM>::score_t;
    const T *x = static_cast<const T *>(c->x);
    T *z = static_cast<T *>(c->z), *pay = static_cast<T *>(c->cur.payload);
    W *sp = static_cast<W *>(c->seg_part);
    const unsigned grid = grid_for_warps(c->segs.n);
    if (c->g.vec_ok) k_segment_full_save<T, NORM, true><<<grid, kThreads, 0, c->stream>>>(x, z, pay, c->g, c->segs, sp);
    else k_segment_full_save<T, NORM, false><<<grid, kThreads, 0, c->stream>>>(x, z, pay, c->g, c->segs, sp);
    ++c->launches;
    launch_combine<T, NORM>(c, sp, nullptr, static_cast<S *>(c->score), nullptr, nullptr, nullptr);
    k_full_save_ids<S><<<(unsigned)((c->g.n_blocks + kThreads - 1) / kThreads), kThreads, 0, c->stream>>>(
        c->g, static_cast<const S *>(c->score), c->cur.sel, c->cur.poff, c->cur.info);
    ++c->launches;
}

void launch_full_save_segments(scar_ctx *c) {
    if (c->dt == SCAR_I32) launch_full_save_segments_as<int, kNormDefault>(c);
    else if (c->norm == SCAR_NORM_L1) launch_full_save_segments_as<float, kNormL1>(c);
    else launch_full_save_segments_as<float, kNormDefault>(c);
}

// a3
void launch_pack(scar_ctx *c, uint64_t k) {
    if (k == 0) return;
    if (c->seg_mode) {
        const uint32_t *x = static_cast<const uint32_t *>(c->x);
        uint32_t *z = static_cast<uint32_t *>(c->z), *pay = static_cast<uint32_t *>(c->cur.payload);
        const unsigned want = grid_for_warps(c->segs.n), cap = (unsigned)c->n_sms * 8u;
        const unsigned grid = want < cap ? want : cap;
        if (c->g.vec_ok)
            launch_after(c, k_pack_segments<true>, grid, x, z, pay, c->g, c->segs, (const uint32_t *)c->cur.sel,
                         (const unsigned long long *)c->cur.poff, (const SaveInfoDev *)c->cur.info);
        else
            launch_after(c, k_pack_segments<false>, grid, x, z, pay, c->g, c->segs, (const uint32_t *)c->cur.sel,
                         (const unsigned long long *)c->cur.poff, (const SaveInfoDev *)c->cur.info);
        ++c->launches;
        return;
    }
    dispatch_group(c->group_lanes, c->g.vec_ok != 0, [&](auto gl, auto vec) {
        constexpr int G = decltype(gl)::value;
        constexpr bool VEC = decltype(vec)::value;
        launch_after(c, k_pack_update<G, VEC>, grid_for_groups(k, G), static_cast<const uint32_t *>(c->x),
                     static_cast<uint32_t *>(c->z), static_cast<uint32_t *>(c->cur.payload), c->g, c->cur.sel,
                     c->cur.poff, (unsigned long long)k, c->cur.info);
    });
    ++c->launches;
}

// a4 / a5: one launch; the kernel's last CTA finishes the norm
template <typename T, int NORM> int launch_recover_as(scar_ctx *c, const LostSet &S, bool write) {
    using Sc = typename Elem<T, NORM>::score_t;
    if (S.n_work == 0) {  // nothing lost: zero perturbation, x untouched
        CU_TRY(cudaMemsetAsync(c->d_norm, 0, sizeof(NormInfoDev), c->stream));
        record(c, 4);
        record(c, 5);
        return SCAR_OK;
    }
    if (c->seg_mode) {
        // S is "all blocks" (mode 0) or a per-block mask (mode 2) here: enqueue_recover turns shard runs into a mask
        using W = typename Elem<T, NORM>::wide_t;
        T *x = static_cast<T *>(c->x);
        const T *z = static_cast<const T *>(c->z);
        W *sp = static_cast<W *>(c->seg_part);
        const uint8_t *mask = S.mode == 2 ? S.mask : nullptr;
        const unsigned grid = grid_for_warps(c->segs.n);
        if (c->g.vec_ok) {
            if (write) k_segment_pass<T, NORM, true, true><<<grid, kThreads, 0, c->stream>>>(x, z, c->g, c->segs, mask, sp);
            else k_segment_pass<T, NORM, true, false><<<grid, kThreads, 0, c->stream>>>(x, z, c->g, c->segs, mask, sp);
        } else {
            if (write) k_segment_pass<T, NORM, false, true><<<grid, kThreads, 0, c->stream>>>(x, z, c->g, c->segs, mask, sp);
            else k_segment_pass<T, NORM, false, false><<<grid, kThreads, 0, c->stream>>>(x, z, c->g, c->segs, mask, sp);
        }
        ++c->launches;
        launch_combine<T, NORM>(c, sp, mask, static_cast<Sc *>(c->part), nullptr, nullptr, nullptr);
        record(c, 4);
        const uint64_t tiles = (S.n_work + kReduceTile - 1) / kReduceTile;
        k_reduce_partials<T><<<(unsigned)tiles, kThreads, 0, c->stream>>>(static_cast<const Sc *>(c->part), c->g, S,
                                                                         c->rs, c->d_norm, NORM == kNormDefault);
        ++c->launches;
        record(c, 5);
        return SCAR_OK;
    }
    const RecoverShape sh = recover_shape(S.mode, S.n_work, c->group_lanes, write);
    dispatch_group(c->group_lanes, c->g.vec_ok != 0, [&](auto gl, auto vec) {
        constexpr int G = decltype(gl)::value;
        constexpr bool VEC = decltype(vec)::value;
        T *x = static_cast<T *>(c->x);
        const T *z = static_cast<const T *>(c->z);
        if (S.mode == 2) {
            if (write)
                k_recover_blocks<T, NORM, G, VEC, true, true><<<sh.grid, kThreads, 0, c->stream>>>(
                    x, z, c->g, S, sh.chunk, c->d_weight, c->rs, c->d_norm);
            else
                k_recover_blocks<T, NORM, G, VEC, false, true><<<sh.grid, kThreads, 0, c->stream>>>(
                    x, z, c->g, S, sh.chunk, c->d_weight, c->rs, c->d_norm);
        } else {
            if (write)
                k_recover_blocks<T, NORM, G, VEC, true, false><<<sh.grid, kThreads, 0, c->stream>>>(
                    x, z, c->g, S, sh.chunk, c->d_weight, c->rs, c->d_norm);
            else
                k_recover_blocks<T, NORM, G, VEC, false, false><<<sh.grid, kThreads, 0, c->stream>>>(
                    x, z, c->g, S, sh.chunk, c->d_weight, c->rs, c->d_norm);
        }
    });
    ++c->launches;
    record(c, 4);
    record(c, 5);
    return SCAR_OK;
}

int launch_recover(scar_ctx *c, const LostSet &S, bool write) {
    if (c->dt == SCAR_I32) return launch_recover_as<int, kNormDefault>(c, S, write);
    if (c->norm == SCAR_NORM_L1) return launch_recover_as<float, kNormL1>(c, S, write);
    return launch_recover_as<float, kNormDefault>(c, S, write);
}

int copy_elems(scar_ctx *c, void *dst, const void *src, uint64_t n) {
    if (n == 0) return SCAR_OK;
    const uint64_t want = ((n >> 2) + kThreads - 1) / kThreads, cap = (uint64_t)c->n_sms * 16u;
    unsigned grid = (unsigned)(want < 1 ? 1 : (want > cap ? cap : want));
    k_copy_elems<<<grid, kThreads, 0, c->stream>>>(static_cast<uint32_t *>(dst), static_cast<const uint32_t *>(src), n);
    ++c->launches;
    CU_TRY(cudaGetLastError());
    return SCAR_OK;
}

int fetch_save(scar_ctx *c, scar_save_info *out) {
    CU_TRY(cudaMemcpyAsync(c->h_save, c->last.info, sizeof(SaveInfoDev), cudaMemcpyDeviceToHost, c->stream));
    CU_TRY(cudaStreamSynchronize(c->stream));
    if (c->h_save->error) {
        // A grid barrier of the selection gave up; its outputs are not valid.  The kernel has
        // already put its barrier state back, so the context stays usable.
        CU_TRY(cudaMemsetAsync(&c->last.info->error, 0, sizeof(unsigned long long), c->stream));
        return SCAR_ERR_TIMEOUT;
    }
    out->k = c->h_save->k;
    out->payload_elems = c->h_save->payload_elems;
    out->nonfinite_blocks = c->h_save->nonfinite_blocks;
    return SCAR_OK;
}

int fetch_norm(scar_ctx *c, scar_norm_info *out) {
    CU_TRY(cudaMemcpyAsync(c->h_norm, c->d_norm, sizeof(NormInfoDev), cudaMemcpyDeviceToHost, c->stream));
    CU_TRY(cudaStreamSynchronize(c->stream));
    if (c->h_norm->lost_blocks == kSlotEmpty) {
        // A bounded wait of the reduction gave up (a slot never arrived).  Slots may be left in any state:
        // empty them all before the next pass.
        CU_TRY(cudaMemsetAsync(c->norm_scratch, 0xff, c->norm_scratch_bytes, c->stream));
        return SCAR_ERR_TIMEOUT;
    }
    out->l2 = c->h_norm->l2;
    out->l1 = c->h_norm->l1;
    out->lost_blocks = c->h_norm->lost_blocks;
    out->lost_elems = c->h_norm->lost_elems;
    return SCAR_OK;
}

int k_from_r(double r, uint64_t n_blocks, uint64_t *k) {
    if (!(r >= 0.0 && r <= 1.0)) return SCAR_ERR_INVALID_ARG;
    long long v = llround(r * (double)n_blocks);
    uint64_t kk = v < 0 ? 0 : (uint64_t)v;
    if (kk > n_blocks) kk = n_blocks;
    if (kk == 0 && r > 0.0 && n_blocks > 0) kk = 1;
    *k = kk;
    return SCAR_OK;
}

// Most elements any k blocks of the layout can hold (the k longest blocks).
uint64_t save_bound(const scar_ctx *c, uint64_t k) {
    if (!c->longest_prefix.empty()) return c->longest_prefix[k];
    if (c->g.n_blocks == 0) return 0;
    const uint64_t per_row = c->g.blocks_per_row, blk = c->g.row_len < c->g.block_elems ? c->g.row_len : c->g.block_elems;
    const uint64_t tail = c->g.row_len - (per_row - 1) * c->g.block_elems;  // last block of a row, <= blk
    const uint64_t n_full = tail < blk ? (c->g.n_blocks / per_row) * (per_row - 1) : c->g.n_blocks;
    return (k < n_full ? k : n_full) * blk + (k > n_full ? (k - n_full) * tail : 0);
}

// Before anything is enqueued: in drain mode the save must fit the slot it writes to.  Changes nothing.
int save_fits(const scar_ctx *c, uint64_t k) {
    if (!c->drain) return SCAR_OK;
    const DrainSlot &sl = c->slot[c->cur_slot];
    if (sl.state >= 2) return SCAR_ERR_STATE;  // both slots are still out: release the older ticket first
    if (k > c->drain_cap_k || save_bound(c, k) > c->drain_cap_elems) return SCAR_ERR_CAPACITY;
    return SCAR_OK;
}

// After every launch of a save went through: only now does the context point at the new save.
void commit_save(scar_ctx *c, uint64_t k) {
    if (c->drain) {
        DrainSlot &sl = c->slot[c->cur_slot];
        sl.k = k;
        sl.state = 1;
    }
    c->last = c->cur;
    c->have_save = true;
}

int enqueue_save(scar_ctx *c, uint64_t k) {
    const int rc_fit = save_fits(c, k);
    if (rc_fit != SCAR_OK) return rc_fit;
    c->last_call = 1;
    c->ran_select = c->ran_pack = false;
    record(c, 0);
    if (c->g.n_blocks == 0) {
        CU_TRY(cudaMemsetAsync(c->cur.info, 0, sizeof(SaveInfoDev), c->stream));
        CU_TRY(cudaMemsetAsync(c->cur.poff, 0, sizeof(unsigned long long), c->stream));
        commit_save(c, k);
        return SCAR_OK;
    }
    if (k == c->g.n_blocks) {
        // Full checkpoint: nothing to choose, so one fused pass scores, packs and refreshes z.
        CU_TRY(cudaMemsetAsync(c->cur.info, 0, sizeof(SaveInfoDev), c->stream));
        if (c->seg_mode) launch_full_save_segments(c);
        else if (c->dt == SCAR_I32) launch_full_save<int, kNormDefault>(c);
        else if (c->norm == SCAR_NORM_L1) launch_full_save<float, kNormL1>(c);
        else launch_full_save<float, kNormDefault>(c);
        record(c, 1);
        record(c, 2);
        record(c, 3);
        CU_TRY(cudaGetLastError());
        c->ran_select = c->ran_pack = true;
        commit_save(c, k);
        return SCAR_OK;
    }
    launch_scores(c, c->cur.info);
    record(c, 1);
    const int rc_sel =
        c->dt == SCAR_F32
            ? launch_select<float>(c, static_cast<const float *>(c->score), c->g, k, c->cur, true)
            : launch_select<unsigned long long>(c, static_cast<const unsigned long long *>(c->score), c->g, k, c->cur, true);
    if (rc_sel != SCAR_OK) {
        cudaGetLastError();
        return rc_sel;
    }
    record(c, 2);
    launch_pack(c, k);
    record(c, 3);
    CU_TRY(cudaGetLastError());
    c->ran_select = true;
    c->ran_pack = k > 0;
    commit_save(c, k);
    return SCAR_OK;
}

// Saves with a selector that does not look at distances (Section 5.4: `round`, `random`):
// no scoring pass; selection, then the same pack + cache refresh as a prioritized save.
int enqueue_baseline_save(scar_ctx *c, uint64_t k, const uint32_t *d_priorities) {
    const int rc_fit = save_fits(c, k);
    if (rc_fit != SCAR_OK) return rc_fit;
    c->last_call = 1;
    c->ran_select = c->ran_pack = false;
    record(c, 0);
    record(c, 1);
    if (c->g.n_blocks == 0) {
        CU_TRY(cudaMemsetAsync(c->cur.info, 0, sizeof(SaveInfoDev), c->stream));
        CU_TRY(cudaMemsetAsync(c->cur.poff, 0, sizeof(unsigned long long), c->stream));
        commit_save(c, k);
        return SCAR_OK;
    }
    if (d_priorities) {
        const int rc = launch_select<unsigned>(c, d_priorities, c->g, k, c->cur, false);
        if (rc != SCAR_OK) {
            cudaGetLastError();
            return rc;
        }
    } else {
        const unsigned grid = (unsigned)((k + kThreads - 1) / kThreads);
        k_select_round<<<grid ? grid : 1, kThreads, 0, c->stream>>>(c->g, c->round_cursor, k, c->cur.sel, c->cur.poff,
                                                                      c->cur.info);
        ++c->launches;
    }
    record(c, 2);
    launch_pack(c, k);
    record(c, 3);
    CU_TRY(cudaGetLastError());
    if (!d_priorities) c->round_cursor = (c->round_cursor + k) % c->g.n_blocks;  // only once the save is on its way
    c->ran_select = true;
    c->ran_pack = k > 0;
    commit_save(c, k);
    return SCAR_OK;
}

int enqueue_recover(scar_ctx *c, const LostSet &S, bool write) {
    c->last_call = 2;
    record(c, 0);
    if (c->g.n_blocks == 0) {
        CU_TRY(cudaMemsetAsync(c->d_norm, 0, sizeof(NormInfoDev), c->stream));
        c->have_norm = true;
        return SCAR_OK;
    }
    const int rc = launch_recover(c, S, write);
    if (rc != SCAR_OK) return rc;
    CU_TRY(cudaGetLastError());
    c->have_norm = true;
    return SCAR_OK;
}

// Element range of block b from the host copy of the layout.
void host_range(const scar_ctx *c, uint64_t b, uint64_t &beg, uint64_t &len) {
    if (!c->h_boff.empty()) {
        beg = c->h_boff[b];
        len = c->h_boff[b + 1] - beg;
        return;
    }
    const uint64_t row = b / c->g.blocks_per_row, j = b % c->g.blocks_per_row, o = j * c->g.block_elems;
    beg = row * c->g.row_len + o;
    len = c->g.row_len - o < c->g.block_elems ? c->g.row_len - o : c->g.block_elems;
}

LostSet all_lost(const scar_ctx *c) {
    LostSet S{};
    S.mode = 0;
    S.n_work = c->g.n_blocks;
    return S;
}

LostSet block_mask_set(const scar_ctx *c, const uint8_t *d_lost_blocks) {
    LostSet S{};
    S.mode = 2;
    S.mask = d_lost_blocks;
    S.n_work = c->g.n_blocks;
    return S;
}

// Lost shards -> runs of consecutive lost blocks (adjacent lost shards merge,
// shards that own no block vanish).  With more runs than LostSet can carry,
// the shard mask is expanded into a per-block mask on the device instead: up
// to kShardsByValue shard flags travel in the launch parameters, longer masks
// go through a pinned buffer of the context (so no copy ever reads the
// caller's array after this returns).
int shard_set(scar_ctx *c, const uint8_t *h_lost_shards, LostSet &S) {
    const uint64_t B = c->g.n_blocks, n_sh = c->g.n_shards;
    S = LostSet{};
    S.mode = 1;
    bool overflow = false;
    uint64_t work = 0;
    for (uint64_t s = 0; s < n_sh && B; ++s) {
        if (!h_lost_shards[s]) continue;
        const uint64_t lo = (uint64_t)(((unsigned __int128)s * B) / n_sh);
        const uint64_t hi = (uint64_t)(((unsigned __int128)(s + 1) * B) / n_sh);
        if (lo == hi) continue;
        if (S.n_runs > 0 && (uint64_t)S.run_first[S.n_runs - 1] + (work - S.run_start[S.n_runs - 1]) == lo) {
            work += hi - lo;  // extends the previous run
        } else {
            if (S.n_runs == kMaxRuns) {
                overflow = true;
                break;
            }
            S.run_first[S.n_runs] = (uint32_t)lo;
            S.run_start[S.n_runs] = (uint32_t)work;
            ++S.n_runs;
            work += hi - lo;
        }
        S.run_start[S.n_runs] = (uint32_t)work;
    }
    S.n_work = work;
    if (B == 0 || (!overflow && !c->seg_mode)) return SCAR_OK;  // segment mode walks segments: it always wants a block mask
    ShardFlags flags{};
    const uint8_t *d_mask = nullptr;
    if (n_sh <= (uint64_t)kShardsByValue) {
        memcpy(flags.lost, h_lost_shards, n_sh);
    } else {
        // the pinned buffer may still be the source of an earlier call's copy
        CU_TRY(cudaStreamSynchronize(c->stream));
        memcpy(c->h_shard_mask, h_lost_shards, n_sh);
        CU_TRY(cudaMemcpyAsync(c->d_shard_mask, c->h_shard_mask, n_sh, cudaMemcpyHostToDevice, c->stream));
        d_mask = c->d_shard_mask;
    }
    k_expand_shards<<<(unsigned)((B + kThreads - 1) / kThreads), kThreads, 0, c->stream>>>(c->g, flags, d_mask,
                                                                                          c->d_block_mask);
    ++c->launches;
    CU_TRY(cudaGetLastError());
    S = block_mask_set(c, c->d_block_mask);
    return SCAR_OK;
}

void destroy_impl(scar_ctx *c) {
    cudaStreamSynchronize(c->stream);
    if (c->drain_stream) cudaStreamSynchronize(c->drain_stream);
    for (void *p : c->owned) cudaFree(p);
    for (void *p : c->owned_host) cudaFreeHost(p);
    for (auto &sl : c->slot) {
        if (sl.saved) cudaEventDestroy(sl.saved);
        if (sl.drained) cudaEventDestroy(sl.drained);
    }
    if (c->drain_stream) cudaStreamDestroy(c->drain_stream);
    if (c->h_save) cudaFreeHost(c->h_save);
    if (c->h_norm) cudaFreeHost(c->h_norm);
    for (auto &e : c->ev)
        if (e) cudaEventDestroy(e);
    delete c;
}

}  // namespace

extern "C" {

static int init_impl(scar_ctx **out, void *d_x, scar_dtype dt, const scar_layout *layout, void *cuda_stream,
                     bool guarded) {
    if (!out) return SCAR_ERR_INVALID_ARG;
    *out = nullptr;
    if (!layout || (dt != SCAR_F32 && dt != SCAR_I32)) return SCAR_ERR_INVALID_ARG;
    if (layout->n_elems > 0 && !d_x) return SCAR_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_x) & 15) return SCAR_ERR_INVALID_ARG;
    Geom g;
    int rc = resolve_layout(layout, g);
    if (rc != SCAR_OK) return rc;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return SCAR_ERR_CUDA;
    }
    scar_ctx *c = new (std::nothrow) scar_ctx;
    if (!c) return SCAR_ERR_ALLOC;
    c->device = dev;
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    c->guarded = guarded;
    c->dt = dt;
    c->g = g;
    c->x = d_x;
    c->group_lanes = pick_group_lanes(g);
    if (layout->block_offsets) {
        c->h_boff.assign(layout->block_offsets, layout->block_offsets + g.n_blocks + 1);
        std::vector<uint64_t> lens(g.n_blocks);
        for (uint64_t b = 0; b < g.n_blocks; ++b) lens[b] = layout->block_offsets[b + 1] - layout->block_offsets[b];
        std::sort(lens.begin(), lens.end(), std::greater<uint64_t>());
        c->longest_prefix.assign(g.n_blocks + 1, 0);
        for (uint64_t b = 0; b < g.n_blocks; ++b) c->longest_prefix[b + 1] = c->longest_prefix[b] + lens[b];
        c->max_block_len = g.n_blocks ? lens[0] : 0;
    } else {
        c->max_block_len = g.row_len < g.block_elems ? g.row_len : g.block_elems;
    }

    const uint64_t N = g.n_elems, B = g.n_blocks;
    const size_t score_bytes = (dt == SCAR_F32 ? 4 : 8) * B;
    const bool long_blocks = c->max_block_len > 2 * kSegElems;

    rc = SCAR_OK;
    auto A = [&](auto **p, size_t bytes) {
        if (rc == SCAR_OK) rc = dev_alloc(c, p, bytes);
    };
    A(&c->z, N * 4);
    A(&c->cur.payload, N * 4);
    A(&c->score, score_bytes);
    if (long_blocks) A(&c->part, score_bytes);
    A(&c->cur.sel, B * 4);
    A(&c->cur.poff, (B + 1) * 8);
    if (g.n_shards > (uint32_t)kShardsByValue) {
        A(&c->d_shard_mask, g.n_shards);
        if (rc == SCAR_OK) {
            void *q = nullptr;
            if (cudaMallocHost(&q, g.n_shards) != cudaSuccess) {
                cudaGetLastError();
                rc = SCAR_ERR_ALLOC;
            } else {
                c->owned_host.push_back(q);
                c->h_shard_mask = static_cast<uint8_t *>(q);
            }
        }
    }
    A(&c->d_block_mask, B);
    A(&c->st, sizeof(SelState));
    if (rc == SCAR_OK) rc = plan_select(c);
    // CTAs of the largest recovery / norm launch (segmented layouts reduce kReduceTile blocks per CTA: fewer)
    const uint64_t max_ctas = recover_max_ctas(B, c->group_lanes);
    c->norm_scratch_bytes = norm_scratch_words(max_ctas) * 8;
    A(&c->norm_scratch, c->norm_scratch_bytes);
    if (rc == SCAR_OK) c->rs = norm_scratch_at(c->norm_scratch, max_ctas);
    A(&c->cur.info, sizeof(SaveInfoDev));
    A(&c->d_norm, sizeof(NormInfoDev));
    if (rc == SCAR_OK && layout->block_offsets) A(&c->d_boff, (B + 1) * 8);
    // Very long blocks: cut every block into segments (see segments.cuh).  The host tables live until the
    // stream synchronisation at the end of init.
    std::vector<uint32_t> seg_block, wide;
    std::vector<uint64_t> seg_beg, seg_first;
    if (rc == SCAR_OK && long_blocks) {
        seg_first.resize(B + 1);
        for (uint64_t b = 0; b < B; ++b) {
            uint64_t beg, len;
            if (layout->block_offsets) {
                beg = layout->block_offsets[b];
                len = layout->block_offsets[b + 1] - beg;
            } else {
                const uint64_t row = b / g.blocks_per_row, j = b % g.blocks_per_row, o = j * g.block_elems;
                beg = row * g.row_len + o;
                len = g.row_len - o < g.block_elems ? g.row_len - o : g.block_elems;
            }
            seg_first[b] = seg_block.size();
            for (uint64_t o = 0; o < len; o += kSegElems) {
                seg_block.push_back((uint32_t)b);
                seg_beg.push_back(beg + o);
            }
        }
        seg_first[B] = seg_block.size();
        for (uint64_t b = 0; b < B; ++b)
            if (seg_first[b + 1] - seg_first[b] > kWideSegs) wide.push_back((uint32_t)b);
        const uint64_t ns = seg_block.size();
        uint32_t *d_sb = nullptr;
        uint64_t *d_sbeg = nullptr, *d_sfirst = nullptr;
        A(&d_sb, ns * 4);
        A(&d_sbeg, ns * 8);
        A(&d_sfirst, (B + 1) * 8);
        A(&c->seg_part, ns * 8);
        A(&c->wide_blocks, wide.size() * 4);
        c->n_wide_blocks = (unsigned)wide.size();
        if (rc == SCAR_OK && !wide.empty() &&
            cudaMemcpyAsync(c->wide_blocks, wide.data(), wide.size() * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
            rc = SCAR_ERR_CUDA;
        if (rc == SCAR_OK &&
            (cudaMemcpyAsync(d_sb, seg_block.data(), ns * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
             cudaMemcpyAsync(d_sbeg, seg_beg.data(), ns * 8, cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
             cudaMemcpyAsync(d_sfirst, seg_first.data(), (B + 1) * 8, cudaMemcpyHostToDevice, c->stream) != cudaSuccess))
            rc = SCAR_ERR_CUDA;
        c->segs = Segs{d_sb, d_sbeg, d_sfirst, ns};
        c->seg_mode = rc == SCAR_OK;
    }
    if (rc == SCAR_OK && (cudaMallocHost(&c->h_save, sizeof(SaveInfoDev)) != cudaSuccess ||
                          cudaMallocHost(&c->h_norm, sizeof(NormInfoDev)) != cudaSuccess))
        rc = SCAR_ERR_ALLOC;
    if (rc == SCAR_OK) {
        bool ok = cudaMemsetAsync(c->st, 0, sizeof(SelState), c->stream) == cudaSuccess &&
                  cudaMemsetAsync(c->norm_scratch, 0xff, c->norm_scratch_bytes, c->stream) == cudaSuccess &&
                  cudaMemsetAsync(c->cur.info, 0, sizeof(SaveInfoDev), c->stream) == cudaSuccess &&
                  cudaMemsetAsync(c->d_norm, 0, sizeof(NormInfoDev), c->stream) == cudaSuccess &&
                  cudaMemsetAsync(c->score, 0, score_bytes ? score_bytes : 16, c->stream) == cudaSuccess &&
                  cudaMemsetAsync(c->cur.poff, 0, 8, c->stream) == cudaSuccess;
        if (ok && layout->block_offsets) {
            ok = cudaMemcpyAsync(c->d_boff, layout->block_offsets, (B + 1) * 8, cudaMemcpyHostToDevice, c->stream) ==
                 cudaSuccess;
            c->g.boff = c->d_boff;
        }
        if (!ok) rc = SCAR_ERR_CUDA;
    }
    // Section 4.2: the running checkpoint starts as the initial parameter values.
    if (rc == SCAR_OK) rc = copy_elems(c, c->z, c->x, N);
    if (rc == SCAR_OK && cudaStreamSynchronize(c->stream) != cudaSuccess) rc = SCAR_ERR_CUDA;
    if (rc != SCAR_OK) {
        cudaGetLastError();
        destroy_impl(c);
        return rc;
    }
    c->last = c->cur;
    *out = c;
    return SCAR_OK;
}

int scar_ckpt_init(scar_ctx **out, void *d_x, scar_dtype dt, const scar_layout *layout, void *cuda_stream) {
    return init_impl(out, d_x, dt, layout, cuda_stream, false);
}

int scar_ckpt_init_guarded(scar_ctx **out, void *d_x, scar_dtype dt, const scar_layout *layout, void *cuda_stream) {
    return init_impl(out, d_x, dt, layout, cuda_stream, true);
}

int scar_ckpt_debug_check_guards(scar_ctx *c, uint64_t *bad_bytes) {
    if (!c || !bad_bytes) return SCAR_ERR_INVALID_ARG;
    if (!c->guarded) return SCAR_ERR_STATE;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    if (!c->d_bad) {
        void *q = nullptr;  // not through dev_alloc: the list of bands must not change while it is walked
        if (cudaMalloc(&q, 8) != cudaSuccess) {
            cudaGetLastError();
            return SCAR_ERR_ALLOC;
        }
        c->owned.push_back(q);
        c->d_bad = static_cast<unsigned long long *>(q);
    }
    CU_TRY(cudaMemsetAsync(c->d_bad, 0, 8, c->stream));
    for (size_t i = 0; i < c->bands.size(); i += kBandsPerLaunch) {
        BandList list{};
        const size_t n = c->bands.size() - i < (size_t)kBandsPerLaunch ? c->bands.size() - i : (size_t)kBandsPerLaunch;
        for (size_t j = 0; j < n; ++j) {
            list.user[j] = c->bands[i + j].user;
            list.bytes[j] = c->bands[i + j].bytes;
        }
        k_check_guards<<<(unsigned)n, kThreads, 0, c->stream>>>(list, c->d_bad);
    }
    CU_TRY(cudaGetLastError());
    unsigned long long bad = 0;
    CU_TRY(cudaMemcpyAsync(&bad, c->d_bad, 8, cudaMemcpyDeviceToHost, c->stream));
    CU_TRY(cudaStreamSynchronize(c->stream));
    *bad_bytes = bad;
    return SCAR_OK;
}

int scar_ckpt_block_scores(scar_ctx *c) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    c->last_call = 3;
    record(c, 0);
    launch_scores(c, nullptr);
    record(c, 1);
    CU_TRY(cudaGetLastError());
    return SCAR_OK;
}

int scar_k_from_r(double r, uint64_t n_blocks, uint64_t *k) {
    if (!k) return SCAR_ERR_INVALID_ARG;
    return k_from_r(r, n_blocks, k);
}

int scar_ckpt_priority_save_k(scar_ctx *c, uint64_t k, scar_save_info *out) {
    if (!c || k > c->g.n_blocks) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    rc = enqueue_save(c, k);
    if (rc != SCAR_OK) return rc;
    return out ? fetch_save(c, out) : SCAR_OK;
}

int scar_ckpt_priority_save(scar_ctx *c, double r, scar_save_info *out) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    uint64_t k = 0;
    int rc = k_from_r(r, c->g.n_blocks, &k);
    if (rc != SCAR_OK) return rc;
    return scar_ckpt_priority_save_k(c, k, out);
}

int scar_ckpt_priority_save_sharded(scar_ctx *c, const void *d_global_scores, uint64_t n_global_blocks,
                                    uint64_t first_block, uint64_t k_global, scar_save_info *out) {
    if (!c || !out) return SCAR_ERR_INVALID_ARG;
    const uint64_t B = c->g.n_blocks;
    if (n_global_blocks > 0xfffffffeull || first_block > n_global_blocks || B > n_global_blocks - first_block ||
        k_global > n_global_blocks || (!d_global_scores && n_global_blocks))
        return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    if (n_global_blocks == 0 || B == 0) {  // nothing of this rank's to choose from: an empty save
        if ((rc = enqueue_baseline_save(c, 0, nullptr)) != SCAR_OK) return rc;
        return fetch_save(c, out);
    }
    // scratch for the selection over all ranks' scores, grown on demand
    if (c->glob_blocks < n_global_blocks) {
        CU_TRY(cudaStreamSynchronize(c->stream));
        if (c->glob.sel) {  // the smaller buffers stay owned (and are freed at destroy); layouts rarely change size
            c->glob = OutSet{};
            c->glob_blocks = 0;
        }
        if ((rc = dev_alloc(c, &c->glob.sel, n_global_blocks * 4)) != SCAR_OK ||
            (rc = dev_alloc(c, &c->glob.poff, (n_global_blocks + 1) * 8)) != SCAR_OK ||
            (!c->glob.info && (rc = dev_alloc(c, &c->glob.info, sizeof(SaveInfoDev))) != SCAR_OK))
            return rc;
        c->glob_blocks = n_global_blocks;
    }
    if (!c->member) {
        if ((rc = dev_alloc(c, &c->member, B * 4)) != SCAR_OK || (rc = dev_alloc(c, &c->d_count, 3 * 8)) != SCAR_OK)
            return rc;
        void *q = nullptr;
        if (cudaMallocHost(&q, 3 * 8) != cudaSuccess) {
            cudaGetLastError();
            return SCAR_ERR_ALLOC;
        }
        c->owned_host.push_back(q);
        c->h_count = static_cast<unsigned long long *>(q);
    }
    if ((rc = save_fits(c, B < k_global ? B : k_global)) != SCAR_OK) return rc;  // this rank saves at most min(B, k) blocks

    // checkpoint step 3 over the scores of all ranks: every rank runs the same deterministic selection.  Lengths
    // play no part here, so the global layout is taken as blocks of one element.
    Geom gg{};
    gg.n_elems = n_global_blocks;
    gg.row_len = 1;
    gg.n_blocks = n_global_blocks;
    gg.block_elems = 1;
    gg.blocks_per_row = 1;
    gg.n_shards = 1;
    gg.vec_ok = 0;
    rc = c->dt == SCAR_F32
             ? launch_select<float>(c, static_cast<const float *>(d_global_scores), gg, k_global, c->glob, false)
             : launch_select<unsigned long long>(c, static_cast<const unsigned long long *>(d_global_scores), gg,
                                                 k_global, c->glob, false);
    if (rc != SCAR_OK) {
        cudaGetLastError();
        return rc;
    }
    // which of the chosen blocks are this rank's, and how many
    CU_TRY(cudaMemsetAsync(c->member, 0, B * 4, c->stream));
    CU_TRY(cudaMemsetAsync(c->d_count, 0, 3 * 8, c->stream));
    if (k_global) {
        k_mark_members<<<(unsigned)((k_global + kThreads - 1) / kThreads), kThreads, 0, c->stream>>>(
            c->glob.sel, c->glob.info, first_block, B, c->member, c->d_count);
        ++c->launches;
    }
    CU_TRY(cudaMemcpyAsync(c->h_count, c->d_count, 3 * 8, cudaMemcpyDeviceToHost, c->stream));
    CU_TRY(cudaStreamSynchronize(c->stream));
    if (c->h_count[1]) {
        CU_TRY(cudaMemsetAsync(&c->glob.info->error, 0, sizeof(unsigned long long), c->stream));
        return SCAR_ERR_TIMEOUT;
    }
    const uint64_t k_local = c->h_count[0], nonfinite = c->h_count[2];
    // checkpoint step 4 on this rank's own blocks: the marks serve as priorities, so the k_local marked blocks are
    // exactly the k_local largest, and the usual selection + pack writes ids, offsets, payload and refreshes z
    rc = enqueue_baseline_save(c, k_local, c->member);
    if (rc != SCAR_OK) return rc;
    rc = fetch_save(c, out);
    if (rc == SCAR_OK) out->nonfinite_blocks = nonfinite;
    return rc;
}

int scar_ckpt_save_round(scar_ctx *c, uint64_t k, scar_save_info *out) {
    if (!c || k > c->g.n_blocks) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    rc = enqueue_baseline_save(c, k, nullptr);
    if (rc != SCAR_OK) return rc;
    return out ? fetch_save(c, out) : SCAR_OK;
}

int scar_ckpt_save_random(scar_ctx *c, uint64_t k, const uint32_t *d_priorities, scar_save_info *out) {
    if (!c || k > c->g.n_blocks || (!d_priorities && c->g.n_blocks)) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    rc = enqueue_baseline_save(c, k, d_priorities);
    if (rc != SCAR_OK) return rc;
    return out ? fetch_save(c, out) : SCAR_OK;
}

int scar_ckpt_round_cursor(scar_ctx *c, const uint64_t *set, uint64_t *get) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    if (set) {
        if (c->g.n_blocks ? *set >= c->g.n_blocks : *set != 0) return SCAR_ERR_INVALID_ARG;
        c->round_cursor = *set;
    }
    if (get) *get = c->round_cursor;
    return SCAR_OK;
}

int scar_recover_partial(scar_ctx *c, const uint8_t *h_lost_shards, scar_norm_info *out) {
    if (!c || !h_lost_shards) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    LostSet S{};
    rc = shard_set(c, h_lost_shards, S);
    if (rc == SCAR_OK) rc = enqueue_recover(c, S, true);
    if (rc != SCAR_OK) return rc;
    return out ? fetch_norm(c, out) : SCAR_OK;
}

int scar_recover_partial_blocks(scar_ctx *c, const uint8_t *d_lost_blocks, scar_norm_info *out) {
    if (!c || (!d_lost_blocks && c->g.n_blocks)) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    LostSet S = block_mask_set(c, d_lost_blocks);
    rc = enqueue_recover(c, S, true);
    if (rc != SCAR_OK) return rc;
    return out ? fetch_norm(c, out) : SCAR_OK;
}

int scar_perturbation_norm(scar_ctx *c, const uint8_t *h_lost_shards, scar_norm_info *out) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    LostSet S = all_lost(c);
    if (h_lost_shards) rc = shard_set(c, h_lost_shards, S);
    if (rc == SCAR_OK) rc = enqueue_recover(c, S, false);
    if (rc != SCAR_OK) return rc;
    return out ? fetch_norm(c, out) : SCAR_OK;
}

int scar_perturbation_norm_blocks(scar_ctx *c, const uint8_t *d_lost_blocks, scar_norm_info *out) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    LostSet S = d_lost_blocks ? block_mask_set(c, d_lost_blocks) : all_lost(c);
    rc = enqueue_recover(c, S, false);
    if (rc != SCAR_OK) return rc;
    return out ? fetch_norm(c, out) : SCAR_OK;
}

int scar_ckpt_priority_save_host(scar_ctx *c, const void *h_x, double r, void *h_payload, uint32_t *h_sel,
                                 uint64_t *h_poff, scar_save_info *out) {
    if (!c || !out || !h_poff) return SCAR_ERR_INVALID_ARG;
    const uint64_t N = c->g.n_elems;
    uint64_t k = 0;
    int rc = k_from_r(r, c->g.n_blocks, &k);
    if (rc != SCAR_OK) return rc;
    if (N && (!h_x || !h_payload)) return SCAR_ERR_INVALID_ARG;
    if (k && !h_sel) return SCAR_ERR_INVALID_ARG;
    rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    if (N) CU_TRY(cudaMemcpyAsync(c->x, h_x, N * 4, cudaMemcpyHostToDevice, c->stream));
    rc = enqueue_save(c, k);
    if (rc != SCAR_OK) return rc;
    // The id and offset lists have a size known up front; the payload length is data dependent.
    if (k) CU_TRY(cudaMemcpyAsync(h_sel, c->last.sel, k * 4, cudaMemcpyDeviceToHost, c->stream));
    CU_TRY(cudaMemcpyAsync(h_poff, c->last.poff, (k + 1) * 8, cudaMemcpyDeviceToHost, c->stream));
    rc = fetch_save(c, out);
    if (rc != SCAR_OK) return rc;
    if (out->payload_elems) {
        CU_TRY(cudaMemcpyAsync(h_payload, c->last.payload, out->payload_elems * 4, cudaMemcpyDeviceToHost, c->stream));
        CU_TRY(cudaStreamSynchronize(c->stream));
    }
    return SCAR_OK;
}

int scar_recover_partial_host(scar_ctx *c, void *h_x, const uint8_t *h_lost_shards, scar_norm_info *out) {
    if (!c || !h_lost_shards || !out) return SCAR_ERR_INVALID_ARG;
    if (c->g.n_elems && !h_x) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    // Element range of every lost shard, from the block offsets the library resolved.
    const uint64_t B = c->g.n_blocks, S = c->g.n_shards;
    std::vector<uint64_t> lo, hi;
    auto elem_of = [&](uint64_t b, uint64_t &e) -> int {
        if (b >= B) { e = c->g.n_elems; return SCAR_OK; }
        uint64_t len;
        host_range(c, b, e, len);
        return SCAR_OK;
    };
    for (uint64_t s = 0; s < S && B; ++s) {
        if (!h_lost_shards[s]) continue;
        uint64_t b0 = (uint64_t)(((unsigned __int128)s * B) / S), b1 = (uint64_t)(((unsigned __int128)(s + 1) * B) / S);
        if (b0 == b1) continue;
        uint64_t e0, e1;
        if ((rc = elem_of(b0, e0)) != SCAR_OK || (rc = elem_of(b1, e1)) != SCAR_OK) return rc;
        if (!lo.empty() && hi.back() == e0) hi.back() = e1;
        else { lo.push_back(e0); hi.push_back(e1); }
    }
    char *hx = static_cast<char *>(h_x), *dx = static_cast<char *>(c->x);
    for (size_t i = 0; i < lo.size(); ++i)
        CU_TRY(cudaMemcpyAsync(dx + lo[i] * 4, hx + lo[i] * 4, (hi[i] - lo[i]) * 4, cudaMemcpyHostToDevice, c->stream));
    LostSet Ls{};
    rc = shard_set(c, h_lost_shards, Ls);
    if (rc == SCAR_OK) rc = enqueue_recover(c, Ls, true);
    if (rc != SCAR_OK) return rc;
    for (size_t i = 0; i < lo.size(); ++i)
        CU_TRY(cudaMemcpyAsync(hx + lo[i] * 4, dx + lo[i] * 4, (hi[i] - lo[i]) * 4, cudaMemcpyDeviceToHost, c->stream));
    return fetch_norm(c, out);
}

int scar_ckpt_set_norm(scar_ctx *c, scar_norm norm, const float *h_block_weights) {
    if (!c || (norm != SCAR_NORM_DEFAULT && norm != SCAR_NORM_L1)) return SCAR_ERR_INVALID_ARG;
    if (c->dt == SCAR_I32 && h_block_weights) return SCAR_ERR_INVALID_ARG;  // integer scores stay exact integers
    const uint64_t B = c->g.n_blocks;
    if (h_block_weights)
        for (uint64_t b = 0; b < B; ++b)
            if (!(h_block_weights[b] >= 0.0f) || std::isinf(h_block_weights[b])) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    if (h_block_weights && B) {
        if (!c->d_weight_buf && (rc = dev_alloc(c, &c->d_weight_buf, B * 4)) != SCAR_OK) return rc;
        // pageable source: the copy has read h_block_weights by the time this returns
        CU_TRY(cudaMemcpyAsync(c->d_weight_buf, h_block_weights, B * 4, cudaMemcpyHostToDevice, c->stream));
        CU_TRY(cudaStreamSynchronize(c->stream));
        c->d_weight = c->d_weight_buf;
    } else {
        c->d_weight = nullptr;
    }
    c->norm = norm;
    return SCAR_OK;
}

int scar_ckpt_selftest_arm_timeout(scar_ctx *c) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    if (c->g.n_blocks == 0) return SCAR_ERR_STATE;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    // Host state only: the next selection is launched with waits that expect one arrival more than there are
    // CTAs, so every one of them runs out.
    c->arm_never = true;
    return SCAR_OK;
}

int scar_ckpt_drain_init(scar_ctx *c, uint64_t max_k, uint64_t max_payload_elems) {
    if (!c || c->drain) return c ? SCAR_ERR_STATE : SCAR_ERR_INVALID_ARG;
    if (max_k > c->g.n_blocks || max_payload_elems > c->g.n_elems) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    CU_TRY(cudaStreamSynchronize(c->stream));
    const size_t pay = max_payload_elems * 4, ids = max_k * 4, offs = (max_k + 1) * 8;
    DrainSlot &s0 = c->slot[0], &s1 = c->slot[1];
    s0.dev = c->cur;  // slot 0 reuses the context's own output set
    auto D = [&](auto **p, size_t bytes) {
        if (rc == SCAR_OK) rc = dev_alloc(c, p, bytes);
    };
    auto H = [&](auto **p, size_t bytes) {
        if (rc != SCAR_OK) return;
        void *q = nullptr;
        if (cudaMallocHost(&q, bytes ? bytes : 16) != cudaSuccess) {
            cudaGetLastError();
            rc = SCAR_ERR_ALLOC;
            return;
        }
        c->owned_host.push_back(q);
        *p = static_cast<std::remove_pointer_t<std::remove_reference_t<decltype(*p)>> *>(q);
    };
    D(&s1.dev.payload, pay);
    D(&s1.dev.sel, ids);
    D(&s1.dev.poff, offs);
    D(&s1.dev.info, sizeof(SaveInfoDev));
    for (auto &sl : c->slot) {
        H(&sl.h_payload, pay);
        H(&sl.h_sel, ids);
        H(&sl.h_poff, offs);
        H(&sl.h_info, sizeof(SaveInfoDev));
        if (rc == SCAR_OK && (cudaEventCreateWithFlags(&sl.saved, cudaEventDisableTiming) != cudaSuccess ||
                              cudaEventCreateWithFlags(&sl.drained, cudaEventDisableTiming) != cudaSuccess))
            rc = SCAR_ERR_CUDA;
    }
    if (rc == SCAR_OK && cudaStreamCreateWithFlags(&c->drain_stream, cudaStreamNonBlocking) != cudaSuccess)
        rc = SCAR_ERR_CUDA;
    if (rc == SCAR_OK && (cudaMemsetAsync(s1.dev.info, 0, sizeof(SaveInfoDev), c->stream) != cudaSuccess ||
                          cudaMemsetAsync(s1.dev.poff, 0, 8, c->stream) != cudaSuccess))
        rc = SCAR_ERR_CUDA;
    if (rc != SCAR_OK) {
        cudaGetLastError();
        return rc;  // what was allocated stays owned by the context and is freed by destroy
    }
    c->drain_cap_k = max_k;
    c->drain_cap_elems = max_payload_elems;
    c->cur_slot = 0;
    c->drain = true;
    return SCAR_OK;
}

int scar_ckpt_drain_enqueue(scar_ctx *c, uint64_t *ticket) {
    if (!c || !ticket) return SCAR_ERR_INVALID_ARG;
    if (!c->drain) return SCAR_ERR_STATE;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    DrainSlot &sl = c->slot[c->cur_slot];
    if (sl.state != 1) return SCAR_ERR_STATE;
    CU_TRY(cudaEventRecord(sl.saved, c->stream));
    CU_TRY(cudaStreamWaitEvent(c->drain_stream, sl.saved, 0));
    // The payload length is only known on the device; the k longest blocks bound it and are known here.
    uint64_t elems = save_bound(c, sl.k);
    if (elems > c->drain_cap_elems) elems = c->drain_cap_elems;
    CU_TRY(cudaMemcpyAsync(sl.h_info, sl.dev.info, sizeof(SaveInfoDev), cudaMemcpyDeviceToHost, c->drain_stream));
    if (sl.k) CU_TRY(cudaMemcpyAsync(sl.h_sel, sl.dev.sel, sl.k * 4, cudaMemcpyDeviceToHost, c->drain_stream));
    CU_TRY(cudaMemcpyAsync(sl.h_poff, sl.dev.poff, (sl.k + 1) * 8, cudaMemcpyDeviceToHost, c->drain_stream));
    if (elems) CU_TRY(cudaMemcpyAsync(sl.h_payload, sl.dev.payload, elems * 4, cudaMemcpyDeviceToHost, c->drain_stream));
    CU_TRY(cudaEventRecord(sl.drained, c->drain_stream));
    sl.state = 2;
    sl.ticket = ++c->next_ticket;
    *ticket = sl.ticket;
    c->cur_slot = 1 - c->cur_slot;
    c->cur = c->slot[c->cur_slot].dev;
    return SCAR_OK;
}

static DrainSlot *slot_of(scar_ctx *c, uint64_t ticket) {
    for (auto &sl : c->slot)
        if (sl.state >= 2 && sl.ticket == ticket) return &sl;
    return nullptr;
}

int scar_ckpt_drain_done(scar_ctx *c, uint64_t ticket) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    DrainSlot *sl = c->drain ? slot_of(c, ticket) : nullptr;
    if (!sl) return SCAR_ERR_STATE;
    if (sl->state == 3) return 1;
    cudaError_t e = cudaEventQuery(sl->drained);
    if (e == cudaSuccess) return 1;
    if (e == cudaErrorNotReady) return 0;
    cudaGetLastError();
    return SCAR_ERR_CUDA;
}

int scar_ckpt_drain_wait(scar_ctx *c, uint64_t ticket, scar_drain_view *out) {
    if (!c || !out) return SCAR_ERR_INVALID_ARG;
    DrainSlot *sl = c->drain ? slot_of(c, ticket) : nullptr;
    if (!sl) return SCAR_ERR_STATE;
    CU_TRY(cudaEventSynchronize(sl->drained));
    sl->state = 3;
    if (sl->h_info->error) return SCAR_ERR_TIMEOUT;
    out->info.k = sl->h_info->k;
    out->info.payload_elems = sl->h_info->payload_elems;
    out->info.nonfinite_blocks = sl->h_info->nonfinite_blocks;
    out->h_sel = sl->h_sel;
    out->h_poff = reinterpret_cast<const uint64_t *>(sl->h_poff);
    out->h_payload = sl->h_payload;
    return SCAR_OK;
}

int scar_ckpt_drain_release(scar_ctx *c, uint64_t ticket) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    DrainSlot *sl = c->drain ? slot_of(c, ticket) : nullptr;
    if (!sl) return SCAR_ERR_STATE;
    if (sl->state == 2) CU_TRY(cudaEventSynchronize(sl->drained));
    sl->state = 0;
    sl->ticket = 0;
    return SCAR_OK;
}

// ---- the running checkpoint in persistent storage (Sections 4.2, 4.3) ---------------------------

namespace {

constexpr size_t kIoStageBytes = 64u << 20;

int write_all(int fd, const char *p, size_t n, uint64_t off) {
    while (n) {
        const ssize_t w = pwrite(fd, p, n, (off_t)off);
        if (w < 0) {
            if (errno == EINTR) continue;
            return SCAR_ERR_IO;
        }
        if (w == 0) return SCAR_ERR_IO;
        p += w;
        n -= (size_t)w;
        off += (uint64_t)w;
    }
    return SCAR_OK;
}

int read_all(int fd, char *p, size_t n, uint64_t off) {
    while (n) {
        const ssize_t r = pread(fd, p, n, (off_t)off);
        if (r < 0) {
            if (errno == EINTR) continue;
            return SCAR_ERR_IO;
        }
        if (r == 0) return SCAR_ERR_IO;  // the file is shorter than the checkpoint
        p += r;
        n -= (size_t)r;
        off += (uint64_t)r;
    }
    return SCAR_OK;
}

int ensure_stage(scar_ctx *c) {
    if (c->io_stage) return SCAR_OK;
    void *q = nullptr;
    if (cudaMallocHost(&q, kIoStageBytes) != cudaSuccess) {
        cudaGetLastError();
        return SCAR_ERR_ALLOC;
    }
    c->owned_host.push_back(q);
    c->io_stage = static_cast<char *>(q);
    return SCAR_OK;
}

}  // namespace

int scar_ckpt_store_full(scar_ctx *c, int fd) {
    if (!c || fd < 0) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc == SCAR_OK) rc = ensure_stage(c);
    if (rc != SCAR_OK) return rc;
    const uint64_t bytes = c->g.n_elems * 4;
    const char *z = static_cast<const char *>(c->z);
    for (uint64_t off = 0; off < bytes; off += kIoStageBytes) {
        const size_t n = (size_t)(bytes - off < kIoStageBytes ? bytes - off : kIoStageBytes);
        CU_TRY(cudaMemcpyAsync(c->io_stage, z + off, n, cudaMemcpyDeviceToHost, c->stream));
        CU_TRY(cudaStreamSynchronize(c->stream));
        if ((rc = write_all(fd, c->io_stage, n, off)) != SCAR_OK) return rc;
    }
    return SCAR_OK;
}

int scar_ckpt_load_stored(scar_ctx *c, int fd) {
    if (!c || fd < 0) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc == SCAR_OK) rc = ensure_stage(c);
    if (rc != SCAR_OK) return rc;
    const uint64_t bytes = c->g.n_elems * 4;
    char *z = static_cast<char *>(c->z);
    for (uint64_t off = 0; off < bytes; off += kIoStageBytes) {
        const size_t n = (size_t)(bytes - off < kIoStageBytes ? bytes - off : kIoStageBytes);
        if ((rc = read_all(fd, c->io_stage, n, off)) != SCAR_OK) return rc;
        CU_TRY(cudaMemcpyAsync(z + off, c->io_stage, n, cudaMemcpyHostToDevice, c->stream));
        CU_TRY(cudaStreamSynchronize(c->stream));  // the staging buffer is reused by the next chunk
    }
    return SCAR_OK;
}

int scar_ckpt_store_drained(scar_ctx *c, uint64_t ticket, int fd) {
    if (!c || fd < 0) return SCAR_ERR_INVALID_ARG;
    DrainSlot *sl = c->drain ? slot_of(c, ticket) : nullptr;
    if (!sl) return SCAR_ERR_STATE;
    CU_TRY(cudaEventSynchronize(sl->drained));
    sl->state = 3;
    if (sl->h_info->error) return SCAR_ERR_TIMEOUT;
    const uint64_t k = sl->h_info->k;
    const char *payload = static_cast<const char *>(sl->h_payload);
    // Runs of consecutive block ids are contiguous both in the payload and in the file: one write per run.
    uint64_t j = 0;
    while (j < k) {
        uint64_t e = j;
        while (e + 1 < k && sl->h_sel[e + 1] == sl->h_sel[e] + 1) ++e;
        uint64_t beg, len;
        host_range(c, sl->h_sel[j], beg, len);
        const uint64_t n_elems = sl->h_poff[e + 1] - sl->h_poff[j];
        const int rc = write_all(fd, payload + sl->h_poff[j] * 4, (size_t)n_elems * 4, beg * 4);
        if (rc != SCAR_OK) return rc;
        j = e + 1;
    }
    return SCAR_OK;
}

int scar_ckpt_load(scar_ctx *c, const void *d_z_src) {
    if (!c || (!d_z_src && c->g.n_elems)) return SCAR_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_z_src) & 15) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    return copy_elems(c, c->z, d_z_src, c->g.n_elems);
}

int scar_ckpt_last_info(scar_ctx *c, scar_save_info *save, scar_norm_info *norm) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    if ((save && !c->have_save) || (norm && !c->have_norm)) return SCAR_ERR_STATE;
    if (save && (rc = fetch_save(c, save)) != SCAR_OK) return rc;
    if (norm && (rc = fetch_norm(c, norm)) != SCAR_OK) return rc;
    if (!save && !norm) CU_TRY(cudaStreamSynchronize(c->stream));
    return SCAR_OK;
}

int scar_ckpt_view(scar_ctx *c, const void **d_z, const void **d_scores, const uint32_t **d_sel,
                   const uint64_t **d_poff, const void **d_payload) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    if (d_z) *d_z = c->z;
    if (d_scores) *d_scores = c->score;
    if (d_sel) *d_sel = c->last.sel;
    if (d_poff) *d_poff = reinterpret_cast<const uint64_t *>(c->last.poff);
    if (d_payload) *d_payload = c->last.payload;
    return SCAR_OK;
}

uint64_t scar_ckpt_n_blocks(const scar_ctx *c) { return c ? c->g.n_blocks : 0; }

uint64_t scar_ckpt_launch_count(const scar_ctx *c) { return c ? c->launches : 0; }

int scar_ckpt_profile(scar_ctx *c, int enable) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    if (enable && !c->ev[0])
        for (auto &e : c->ev) CU_TRY(cudaEventCreate(&e));
    c->profile = enable != 0;
    c->last_call = 0;
    return SCAR_OK;
}

int scar_ckpt_profile_read(scar_ctx *c, float ms[5]) {
    if (!c || !ms) return SCAR_ERR_INVALID_ARG;
    if (!c->profile) return SCAR_ERR_STATE;
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    for (int i = 0; i < 5; ++i) ms[i] = 0.f;
    CU_TRY(cudaStreamSynchronize(c->stream));
    if (c->g.n_blocks == 0) return SCAR_OK;
    if (c->last_call == 1 || c->last_call == 3) {
        CU_TRY(cudaEventElapsedTime(&ms[0], c->ev[0], c->ev[1]));
        if (c->last_call == 1) {
            CU_TRY(cudaEventElapsedTime(&ms[1], c->ev[1], c->ev[2]));
            CU_TRY(cudaEventElapsedTime(&ms[2], c->ev[2], c->ev[3]));
        }
    } else if (c->last_call == 2) {
        CU_TRY(cudaEventElapsedTime(&ms[3], c->ev[0], c->ev[4]));
        CU_TRY(cudaEventElapsedTime(&ms[4], c->ev[4], c->ev[5]));
    }
    return SCAR_OK;
}

int scar_ckpt_debug_select_stamps(scar_ctx *c, int64_t stamps[32]) {
    if (!c || !stamps) return SCAR_ERR_INVALID_ARG;
#ifdef SCAR_SELECT_STAMPS
    static_assert(kSelStamps == 32, "size stated in scar.h");
    int rc = check_device(c);
    if (rc != SCAR_OK) return rc;
    CU_TRY(cudaStreamSynchronize(c->stream));
    CU_TRY(cudaMemcpy(stamps, c->st->stamp, sizeof(long long) * kSelStamps, cudaMemcpyDeviceToHost));
    return SCAR_OK;
#else
    return SCAR_ERR_STATE;
#endif
}

int scar_ckpt_destroy(scar_ctx *c) {
    if (!c) return SCAR_ERR_INVALID_ARG;
    destroy_impl(c);
    return SCAR_OK;
}

const char *scar_strerror(int code) {
    switch (code) {
        case SCAR_OK: return "ok";
        case SCAR_ERR_INVALID_ARG: return "invalid argument";
        case SCAR_ERR_LAYOUT: return "inconsistent block layout";
        case SCAR_ERR_ALLOC: return "allocation failed";
        case SCAR_ERR_CUDA: return "CUDA runtime error";
        case SCAR_ERR_STATE: return "call not valid in this state";
        case SCAR_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case SCAR_ERR_CAPACITY: return "problem exceeds a fixed-size internal buffer";
        case SCAR_ERR_IO: return "reading or writing the stored checkpoint failed";
        default: return "unknown error";
    }
}

}  // extern "C"
