// Host-side construction (and per-context caching) of TMA tensor maps.
#pragma once
#include <cuda.h>
#include <stdint.h>

struct cascade_ctx;

// Tiled map over a row-major bf16 matrix [rows][cols] (cols contiguous) with a box of
// [box_rows][box_cols]; box_cols * 2 bytes must be <= 128 and is the 128-byte-swizzle span.
// Returns nullptr on failure.  The returned pointer stays valid at least until 4000 other maps have been
// looked up on the context (the cache evicts the map that has gone unused for longest).
const CUtensorMap* get_tmap_2d_bf16(cascade_ctx* ctx, const void* base, uint64_t rows, uint64_t cols,
                                    uint64_t row_stride_elems, uint32_t box_rows, uint32_t box_cols);

// 4-D map [d3][d2][d1][d0] bf16, d0 contiguous, strides in elements for d1..d3, box sizes per dim.
const CUtensorMap* get_tmap_4d_bf16(cascade_ctx* ctx, const void* base, const uint64_t dims[4],
                                    const uint64_t strides_elems[3], const uint32_t box[4]);
// General form: rank 2..4, dims[0] contiguous, strides in elements for dims 1..rank-1.
const CUtensorMap* get_tmap_bf16(cascade_ctx* ctx, const void* base, int rank, const uint64_t* dims,
                                 const uint64_t* strides_elems, const uint32_t* box);
void free_tmap_cache(cascade_ctx* ctx);
