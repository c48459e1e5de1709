// Internal helpers shared by the translation unit of libswaa: status word, tile arithmetic,
// small PTX wrappers.  Nothing here is part of the C ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "swaa.h"

namespace swaa {

// ---------------------------------------------------------------- status word
// One word per device (a __device__ variable has one instance per device that loads the module).
// 0 = ok; the first error wins.
__device__ int g_device_status = 0;

__device__ __forceinline__ void record_device_error(int code) { atomicCAS(&g_device_status, 0, code); }

inline std::atomic<uint64_t>& launch_counter() {
    static std::atomic<uint64_t> c{0};
    return c;
}

// ---------------------------------------------------------------- tile arithmetic (host + device)
// Key tiles visited by the query tile of rows [i0, i1] (positions inside one sequence), App. A: only
// the tiles holding a visible key are enumerated, which makes prefill work linear in L at fixed W.
struct TileRange {
    int n_sink_tiles;  // tiles 0 .. n_sink_tiles-1 hold sink keys that lie before the band
    int n_lo, n_hi;    // band (or, for full attention, whole causal prefix): tiles n_lo .. n_hi
    __host__ __device__ int count() const { return n_sink_tiles + (n_hi - n_lo + 1); }
    __host__ __device__ int tile(int t) const { return t < n_sink_tiles ? t : n_lo + (t - n_sink_tiles); }
};

__host__ __device__ inline TileRange tile_range(int i0, int i1, int BN, int W, int S, bool is_full) {
    TileRange r;
    r.n_hi = i1 / BN;
    if (is_full) {
        r.n_sink_tiles = 0;
        r.n_lo = 0;
        return r;
    }
    long long first = (long long)i0 - (long long)W + 1;  // first window key of the tile's first row
    r.n_lo = first <= 0 ? 0 : (int)(first / BN);
    long long sink_tiles = ((long long)S + BN - 1) / BN;  // tiles holding a key j < S
    r.n_sink_tiles = (int)(sink_tiles < r.n_lo ? sink_tiles : r.n_lo);
    return r;
}

// True when some (i, j) with i in [i0, i1], j in [j0, j1] is not visible, so the element predicate
// must be applied.  Conservative: may return true for a tile that happens to be fully visible.
__host__ __device__ inline bool tile_needs_mask(int i0, int i1, int j0, int j1, int W, int S, bool is_full) {
    if (j1 > i0) return true;                         // some key is after some query (or past the sequence)
    if (is_full) return false;
    if ((long long)j0 >= (long long)i1 - W + 1) return false;  // whole tile inside every row's window
    if (j1 < S) return false;                         // whole tile is sink keys
    return true;
}

// ---------------------------------------------------------------- small device helpers
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

}  // namespace swaa
