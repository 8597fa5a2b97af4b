// scar_perturbation_norm_static: the read-only perturbation norm for callers
// that must not allocate.
//
// Who needs this: code that runs where device allocation is off limits or
// unaffordable - a failure handler that has to size up the damage while the
// process is already short of memory, a step of a latency-critical loop where a
// cudaMalloc (which synchronises the device) is not acceptable, or a host
// framework that hands a plug-in a fixed memory budget and forbids it to grow.
// Such callers cannot create a scar_ctx, because scar_ckpt_init allocates the
// checkpoint copy and its work arrays.
//
// The regular norm pass keeps one partial sum per CTA of its kernel, a few
// per-tile sums and ticket counters in memory that the context allocated.  Here
// that scratch is a fixed array in the library's device image instead, so every
// GPU that loads the library carries it (about 0.3 MiB) until the process
// exits, and the block count is capped at SCAR_STATIC_MAX_BLOCKS.
#include <cstdint>
#include <mutex>

#include "scar.h"

#include "block_pass.cuh"

using namespace scar;

namespace {

constexpr uint64_t kStaticMaxBlocks = SCAR_STATIC_MAX_BLOCKS;
// The pass launches at most one CTA per kThreads / 4 blocks (the narrowest group has 4 lanes).
constexpr uint64_t kStaticMaxCtas = kStaticMaxBlocks / (kThreads / 4) + 1;
// 8-byte words: two slots per CTA, three per watcher.
constexpr uint64_t kScratchWords = 2 * kStaticMaxCtas + 3 * kMaxWatchers;
// Behind them, a band of words that nothing may write: it is filled with a pattern when the address is looked up
// and scar_static_debug_check_guard counts the bytes that have changed since.
constexpr uint64_t kGuardWords = 32;
constexpr int kGuardPattern = 0xA5;

// In host code this name is only a handle for cudaGetSymbolAddress: it is not
// a device address and must never be passed to a kernel as one.
static __device__ __align__(256) unsigned long long g_static_scratch[kScratchWords + kGuardWords];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned long long *g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device, looked up once
// per device (with that device current) and remembered.
int scratch_on_current_device(unsigned long long **out, cudaStream_t stream) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SCAR_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return SCAR_ERR_STATE;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return SCAR_ERR_CUDA;
        }
        if (cudaMemsetAsync(static_cast<unsigned long long *>(p) + kScratchWords, kGuardPattern, kGuardWords * 8, stream) !=
            cudaSuccess)
            return SCAR_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<unsigned long long *>(p);
    }
    *out = g_scratch_addr[dev];
    return SCAR_OK;
}

static_assert(sizeof(NormInfoDev) == sizeof(scar_norm_info), "result layouts must agree");

template <typename T>
int run_static(const void *d_x, const void *d_z, const Geom &g, const LostSet &S, unsigned long long *scratch,
               scar_norm_info *d_out, cudaStream_t stream) {
    double units = (double)g.n_elems / (double)g.n_blocks;
    if (g.vec_ok) units /= 4.0;
    int G = 4;
    while (G < 32 && G * 4 < units) G <<= 1;
    const RecoverShape sh = recover_shape(S.mode, S.n_work, G, false);
    if (sh.grid > kStaticMaxCtas) return SCAR_ERR_CAPACITY;
    const NormScratch rs = norm_scratch_at(scratch, sh.grid);
    // Every call shares the array, and an earlier call may have laid it out for another grid size: the slots
    // this call uses have to start out empty (all bits set).
    if (cudaMemsetAsync(scratch, 0xff, norm_scratch_words(sh.grid) * 8, stream) != cudaSuccess) return SCAR_ERR_CUDA;
    T *x = static_cast<T *>(const_cast<void *>(d_x));  // the read-only instantiation never stores
    const T *z = static_cast<const T *>(d_z);
    NormInfoDev *out = reinterpret_cast<NormInfoDev *>(d_out);
#define SCAR_STATIC_LAUNCH(G_, VEC_)                                                                               \
    do {                                                                                                           \
        if (S.mode == 2)                                                                                           \
            k_recover_blocks<T, kNormDefault, G_, VEC_, false, true><<<sh.grid, kThreads, 0, stream>>>(           \
                x, z, g, S, sh.chunk, nullptr, rs, out);                                                           \
        else                                                                                                       \
            k_recover_blocks<T, kNormDefault, G_, VEC_, false, false><<<sh.grid, kThreads, 0, stream>>>(          \
                x, z, g, S, sh.chunk, nullptr, rs, out);                                                           \
    } while (0)
    if (g.vec_ok) {
        if (G == 4) SCAR_STATIC_LAUNCH(4, true);
        else if (G == 8) SCAR_STATIC_LAUNCH(8, true);
        else if (G == 16) SCAR_STATIC_LAUNCH(16, true);
        else SCAR_STATIC_LAUNCH(32, true);
    } else {
        if (G == 4) SCAR_STATIC_LAUNCH(4, false);
        else if (G == 8) SCAR_STATIC_LAUNCH(8, false);
        else if (G == 16) SCAR_STATIC_LAUNCH(16, false);
        else SCAR_STATIC_LAUNCH(32, false);
    }
#undef SCAR_STATIC_LAUNCH
    return cudaGetLastError() == cudaSuccess ? SCAR_OK : SCAR_ERR_CUDA;
}

}  // namespace

extern "C" int scar_perturbation_norm_static(const void *d_x, const void *d_z, scar_dtype dt, const scar_layout *layout,
                                             const uint8_t *d_lost_blocks, scar_norm_info *d_out, void *cuda_stream) {
    if (!layout || !d_out || (dt != SCAR_F32 && dt != SCAR_I32)) return SCAR_ERR_INVALID_ARG;
    if (layout->block_offsets) return SCAR_ERR_INVALID_ARG;  // explicit offsets would have to be copied to the device
    if (layout->n_elems > 0 && (!d_x || !d_z)) return SCAR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_x) | reinterpret_cast<uintptr_t>(d_z)) & 15) return SCAR_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // Looked up first, so that even a call on an empty layout is a complete warm-up of this device.
    unsigned long long *scratch = nullptr;
    int rc = scratch_on_current_device(&scratch, stream);
    if (rc != SCAR_OK) return rc;
    if (layout->n_elems == 0)
        return cudaMemsetAsync(d_out, 0, sizeof(scar_norm_info), stream) == cudaSuccess ? SCAR_OK : SCAR_ERR_CUDA;
    if (layout->block_elems == 0) return SCAR_ERR_LAYOUT;
    const uint64_t row = layout->row_elems ? layout->row_elems : layout->n_elems;
    if (row > layout->n_elems || layout->n_elems % row != 0) return SCAR_ERR_LAYOUT;
    const uint64_t per_row = (row + layout->block_elems - 1) / layout->block_elems;
    const uint64_t rows = layout->n_elems / row;
    if (per_row > kStaticMaxBlocks || rows > kStaticMaxBlocks || per_row * rows > kStaticMaxBlocks)
        return SCAR_ERR_CAPACITY;

    Geom g{};
    g.n_elems = layout->n_elems;
    g.row_len = row;
    g.n_blocks = per_row * rows;
    g.boff = nullptr;
    g.block_elems = layout->block_elems;
    g.blocks_per_row = (uint32_t)per_row;
    g.n_shards = 1;
    g.vec_ok = (row % 4 == 0) && (layout->block_elems % 4 == 0);
    LostSet S{};
    S.mode = d_lost_blocks ? 2 : 0;
    S.mask = d_lost_blocks;
    S.n_work = g.n_blocks;

    return dt == SCAR_F32 ? run_static<float>(d_x, d_z, g, S, scratch, d_out, stream)
                          : run_static<int>(d_x, d_z, g, S, scratch, d_out, stream);
}

extern "C" int scar_static_debug_check_guard(uint64_t *bad_bytes) {
    if (!bad_bytes) return SCAR_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SCAR_ERR_CUDA;
    unsigned long long *base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (dev < 0 || dev >= kMaxDevices || !g_scratch_addr[dev]) return SCAR_ERR_STATE;  // never used on this device
        base = g_scratch_addr[dev];
    }
    unsigned char tail[kGuardWords * 8];
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(tail, base + kScratchWords, sizeof tail, cudaMemcpyDeviceToHost) != cudaSuccess)
        return SCAR_ERR_CUDA;
    uint64_t bad = 0;
    for (unsigned char b : tail) bad += b != (unsigned char)kGuardPattern;
    *bad_bytes = bad;
    return SCAR_OK;
}
