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

// How a kernel decides whether block b belongs to the lost set S.
struct LostSet {
    const uint8_t *mask;  // per shard (mode 1) or per block (mode 2); unused in mode 0
    int mode;             // 0: every block lost, 1: shard mask, 2: block mask
    __device__ __forceinline__ bool lost(const Geom &g, uint32_t b) const {
        if (mode == 0) return true;
        if (mode == 1) return mask[g.shard_of(b)] != 0;
        return mask[b] != 0;
    }
};

}  // namespace scar
