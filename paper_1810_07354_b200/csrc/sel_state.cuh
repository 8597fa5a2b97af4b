// Device-side state of the block selection (select.cuh) and the result record of a save.  Kept apart from the
// selection kernel because the kernel that runs before it on the stream (the scoring pass) clears this state.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace scar {

struct SaveInfoDev {
    unsigned long long k;
    unsigned long long payload_elems;
    unsigned long long nonfinite_blocks;
    unsigned long long error;  // non-zero when a wait of the selection gave up: sel / poff are not valid
};

constexpr int kMaxPasses = 6;
constexpr int kHistBins = 2048;
constexpr int kSelThreads = 512;
constexpr int kSelPerThread = 8;
constexpr int kSelTile = kSelThreads * kSelPerThread;  // keys per tile
constexpr int kMaxSelCtas = kSelThreads;  // the exchange reads one record per thread; grids stay below this
// A wait polls at most this often, sleeping 256 ns between polls once it has polled 4096 times: it gives up after
// a quarter of a second at the earliest and about a second in practice.
constexpr unsigned kSpinLimit = 1u << 20;
constexpr unsigned kSelDirectKeys = 64;  // a digit pass over at most this many keys skips the shared histogram

// Diagnostic builds (-DSCAR_SELECT_STAMPS) record where the selection kernel's time goes: thread 0 of CTA 0
// writes its SM's cycle counter at up to kSelStamps marked points; scar_ckpt_debug_select_stamps reads them.
constexpr int kSelStamps = 32;
#ifdef SCAR_SELECT_STAMPS
#define SEL_STAMP(st, i)                                                      \
    do {                                                                      \
        if (blockIdx.x == 0 && threadIdx.x == 0) (st)->stamp[i] = clock64(); \
    } while (0)
#else
#define SEL_STAMP(st, i) \
    do {                 \
    } while (0)
#endif

// What one CTA tells the others once tau is known.  Every word holds its value PLUS ONE, and the state is zero
// when a selection starts: a word that reads non-zero has arrived (an aligned word is written whole), so the
// writer needs no fence and the reader no separate flag; it polls until all the words it needs are there.
struct SelRecord {
    unsigned c_gt;   // keys > tau
    unsigned c_eq;   // keys == tau
    unsigned c_nf;   // non-finite scores
    unsigned unused;
    unsigned long long len_gt;  // summed block lengths of the keys > tau
    unsigned long long len_eq;
};

struct SelState {
    unsigned long long key_or;  // OR of all uint64 keys seen since the last selection
    unsigned long long reserved;
    // ---- everything from here on is zero when a selection starts
    unsigned arrive[kMaxPasses];  // arrivals after each digit pass (k_select only; k_select_tile needs none)
    unsigned error;               // non-zero once a wait gave up
    unsigned reserved2;
    unsigned hist[kMaxPasses][kHistBins];
    SelRecord rec[kMaxSelCtas];
#ifdef SCAR_SELECT_STAMPS
    long long stamp[kSelStamps];  // SM cycle counter of CTA 0 at the points SEL_STAMP marks (diagnostic builds only)
#endif
};
constexpr size_t kSelZeroFrom = offsetof(SelState, arrive);
constexpr unsigned kSelZeroVecs = (unsigned)((sizeof(SelState) - kSelZeroFrom) / 16);
static_assert(kSelZeroFrom % 16 == 0 && (sizeof(SelState) - kSelZeroFrom) % 16 == 0, "cleared with 16-byte stores");
static_assert(offsetof(SelState, hist) % 16 == 0, "histogram rows are read as 16-byte vectors");


// Zeroes the part of SelState a selection expects to find zero, and the result record of the save about to
// run.  Called by every thread of the kernel that precedes the selection on the stream (the scoring pass): its
// first CTAs share the 64 KiB, which costs that kernel nothing measurable and keeps a memset off the critical
// path between scoring and selection.
constexpr unsigned kSelClearCtas = 16;
__device__ __forceinline__ void sel_state_clear(SelState *st, SaveInfoDev *info) {
    const unsigned nc = gridDim.x < kSelClearCtas ? gridDim.x : kSelClearCtas;
    if (blockIdx.x >= nc) return;
    uint4 *p = reinterpret_cast<uint4 *>(reinterpret_cast<char *>(st) + kSelZeroFrom);
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < kSelZeroVecs; i += nc * blockDim.x)
        p[i] = make_uint4(0u, 0u, 0u, 0u);
    if (info && blockIdx.x == 0 && threadIdx.x == 0) {
        info->k = 0;
        info->payload_elems = 0;
        info->nonfinite_blocks = 0;
        info->error = 0;
    }
}

}  // namespace scar
