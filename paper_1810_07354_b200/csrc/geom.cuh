// Block geometry shared by every kernel of the library (device side).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace scar {

// Resolved layout.  Implicit form: rows of row_len elements cut into blocks of
// block_elems (last block of a row shorter when row_len % block_elems != 0).
// Explicit form: boff holds B + 1 element offsets in device memory.
struct Geom {
    uint64_t n_elems;
    uint64_t row_len;
    uint64_t n_blocks;
    const uint64_t *boff;  // nullptr for the implicit form
    uint32_t block_elems;
    uint32_t blocks_per_row;
    uint32_t n_shards;
    uint32_t vec_ok;  // every block starts and ends on a 4-element (16-byte) boundary

    __device__ __forceinline__ void range(uint32_t b, uint64_t &beg, uint64_t &len) const {
        if (boff) {
            beg = boff[b];
            len = boff[b + 1] - beg;
        } else if (blocks_per_row == 1) {
            beg = (uint64_t)b * row_len;
            len = row_len;
        } else {
            uint32_t row = b / blocks_per_row;
            uint32_t j = b - row * blocks_per_row;
            uint64_t o = (uint64_t)j * block_elems;
            beg = (uint64_t)row * row_len + o;
            uint64_t rem = row_len - o;
            len = rem < block_elems ? rem : (uint64_t)block_elems;
        }
    }

    // Shard s owns blocks [floor(s*B/S), floor((s+1)*B/S)); the owner of b is
    // the largest s with floor(s*B/S) <= b, i.e. floor(((b+1)*S - 1) / B).
    __device__ __forceinline__ uint32_t shard_of(uint32_t b) const {
        return (uint32_t)((((uint64_t)b + 1) * n_shards - 1) / n_blocks);
    }
};

// Lengths of consecutive blocks, without a division per block: the row position of the first block is worked
// out once and then counted up.
struct BlockLens {
    const Geom &g;
    uint32_t b, j;  // current block and its position within its row (implicit layouts)
    __device__ __forceinline__ BlockLens(const Geom &geom, uint32_t first) : g(geom), b(first), j(0) {
        if (!g.boff && g.blocks_per_row > 1) j = first % g.blocks_per_row;
    }
    // length of the current block; moves on to the next one
    __device__ __forceinline__ uint64_t next() {
        uint64_t len;
        if (g.boff) {
            len = g.boff[b + 1] - g.boff[b];
        } else if (g.blocks_per_row == 1) {
            len = g.row_len;
        } else {
            const uint64_t rem = g.row_len - (uint64_t)j * g.block_elems;
            len = rem < g.block_elems ? rem : (uint64_t)g.block_elems;
            if (++j == g.blocks_per_row) j = 0;
        }
        ++b;
        return len;
    }
};

// The lost set S of a recovery (Section 4.1), as a list of work items that the
// recovery kernels map to blocks.
//   mode 0: every block is lost; work item w is block w.
//   mode 1: runs of consecutive lost blocks (lost shards, adjacent ones merged);
//           only lost blocks are work items, so no CTA is launched for the rest.
//   mode 2: per-block mask in device memory; work item w is block w, skipped
//           when mask[w] == 0.
constexpr int kMaxRuns = 32;
struct LostSet {
    const uint8_t *mask;
    uint64_t n_work;
    int mode;
    int n_runs;
    uint32_t run_first[kMaxRuns];      // first block of run r
    uint32_t run_start[kMaxRuns + 1];  // work items before run r

    __device__ __forceinline__ bool block_of(uint64_t w, uint32_t &b) const {
        if (w >= n_work) return false;
        if (mode == 1) {
            int r = 0;
            while (r + 1 < n_runs && w >= run_start[r + 1]) ++r;
            b = run_first[r] + (uint32_t)(w - run_start[r]);
            return true;
        }
        b = (uint32_t)w;
        return mode == 0 || mask[b] != 0;
    }
};

}  // namespace scar
