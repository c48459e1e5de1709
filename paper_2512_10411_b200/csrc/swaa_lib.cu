// libswaa: C-ABI entry points (see include/swaa.h).  Host-side validation, planning and launches.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <algorithm>
#include <cmath>
#include <mutex>
#include <random>
#include <vector>

#include "swaa.h"
#include "swaa_internal.cuh"
#include "swaa_decode.cuh"
#include "swaa_prefill.cuh"
#include "swaa_backward.cuh"
#include "swaa_backward_tc.cuh"

namespace swaa {

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceInfo {
    bool known = false;
    int sm_count = 0;
    int cc_major = 0;
};

// Properties of the current device, queried once per device.
static int current_device_info(DeviceInfo* out) {
    static std::mutex mu;
    static DeviceInfo table[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SWAA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!table[dev].known) {
        int sms = 0, major = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SWAA_ERR_CUDA;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
            return SWAA_ERR_CUDA;
        table[dev].sm_count = sms;
        table[dev].cc_major = major;
        table[dev].known = true;
    }
    *out = table[dev];
    return SWAA_OK;
}

// ------------------------------------------------------------------------------------------ decode
struct DecodePlan {
    int NH;      // 8-head blocks per chunk (1 or 2)
    int HG;      // chunks per kv head
    int blocks;  // persistent grid size
    bool too_large;
    size_t off_part, bytes;
};

// One block per SM, fewer when the whole problem has fewer tiles than that.  Depends only on the
// shape arguments and the SM count (sequence lengths are read on the device).
static DecodePlan plan_decode(int B, int Hq, int Hkv, int D, int Lmax, int window, int n_sink, int is_full,
                              int sm_count, bool paged = false, bool shard = false) {
    DecodePlan pl;
    const int G = Hq / Hkv;
    pl.NH = G > 8 ? 2 : 1;
    const int HC = 8 * pl.NH;
    pl.HG = (G + HC - 1) / HC;
    const SeqGeom longest = decode_seq_geom(Lmax, Lmax, window, n_sink, is_full, paged);
    // upper bound on the tiles of one item: a shorter sequence may have one more (ragged) sink tile; a shard of a
    // longer sequence at most its rows in tiles plus a ragged sink and a ragged window tile
    const long long per_item = shard ? ((long long)Lmax + kDecodeTileKeys - 1) / kDecodeTileKeys + 2 : (long long)longest.nt + 1;
    const long long tiles_ub = (long long)B * Hkv * pl.HG * per_item;
    long long blocks = (tiles_ub + kDecodeMinTilesPerBlock - 1) / kDecodeMinTilesPerBlock;
    const long long sms = sm_count > 0 ? sm_count : 148;
    if (blocks > sms) blocks = sms;
    if (blocks < 1) blocks = 1;
    // Cuts on item boundaries.  The cache rows of one sequence interleave its kv heads (a 64-key tile of one head is
    // 64 pieces of 2*D bytes, Hkv*2*D bytes apart), so HBM is used best when the heads of a sequence are streamed
    // at the same rows at the same time.  That is what happens when every block owns whole items, or every item is
    // cut into the same number of blocks: consecutive blocks then walk consecutive heads in step (equal lengths
    // assumed; ragged batches lose the alignment, not the correctness).  Measured on workload 4 with 128 items:
    // 128 blocks against 148: FA decode 597 us against 652 us, SWA decode 47 us against 54 us (there is also no
    // partial-result merge left); 120 or 132 blocks are no better than 148.  Below three quarters of the SMs the
    // loss of parallel streams outweighs the gain (111 blocks: 660 us).
    const long long items = (long long)B * Hkv * pl.HG;
    if (blocks == sms) {
        for (long long b = sms; b * 4 >= sms * 3; --b)
            if (items % b == 0 || b % items == 0) {
                blocks = b;
                break;
            }
    }
    pl.blocks = (int)blocks;
    pl.too_large = tiles_ub / blocks > 0x3fffffffLL;  // the kernel counts a block's tiles in an int
    pl.off_part = ((size_t)pl.blocks * sizeof(unsigned long long) + 255) / 256 * 256;
    pl.bytes = pl.off_part + (size_t)2 * pl.blocks * HC * (D + 2) * sizeof(float);
    return pl;
}

// 48-bit stamps, unique per call within the process and never 0.  They start at a random point so that
// what an earlier process or an unrelated buffer left in a workspace does not look like a live ticket.
static unsigned long long next_call_stamp() {
    static std::atomic<unsigned long long> counter{[] {
        std::random_device rd;
        const unsigned long long r = ((unsigned long long)rd() << 32) ^ (unsigned long long)rd();
        return (r & 0x3fffffffffffull) | 0x400000000000ull;  // in [2^46, 2^47)
    }()};
    return counter.fetch_add(1, std::memory_order_relaxed) & 0xffffffffffffull;
}

static int check_decode_shape(int B, int Hq, int Hkv, int D, int Lmax, int window, int n_sink, int is_full) {
    if (B < 0 || Lmax < 1 || Hq < 1 || Hkv < 1 || n_sink < 0) return SWAA_ERR_INVALID_ARG;
    if (!is_full && window < 1) return SWAA_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || (D != 64 && D != 128)) return SWAA_ERR_UNSUPPORTED;
    return SWAA_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, resolved through the runtime so that the library does not link
// against the driver directly.
static EncodeTiledFn encode_tiled_fn() {
    static std::mutex mu;
    static EncodeTiledFn fn = nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Encoded tensor maps are kept in a small host-side table keyed by everything that goes into them: a serving loop
// calls with the same buffers and shapes step after step, and four encodings per call are a measurable part of a
// 50 us decode step.  A tensor map holds no device state (address and geometry only), so an entry stays valid for
// as long as its key matches, whatever happens to the memory behind it.
struct MapKey {
    const void* base;
    int kind, a, b, c, d, e;
    bool operator==(const MapKey& o) const {
        return base == o.base && kind == o.kind && a == o.a && b == o.b && c == o.c && d == o.d && e == o.e;
    }
};
static bool cached_map(const MapKey& key, CUtensorMap* out, const CUtensorMap* store) {
    constexpr int kSlots = 64;
    struct Slot {
        bool used = false;
        MapKey key{};
        CUtensorMap map{};
    };
    static std::mutex mu;
    static Slot slots[kSlots];
    static unsigned next = 0;
    std::lock_guard<std::mutex> lock(mu);
    if (store == nullptr) {
        for (int i = 0; i < kSlots; ++i)
            if (slots[i].used && slots[i].key == key) {
                *out = slots[i].map;
                return true;
            }
        return false;
    }
    Slot& s = slots[next++ % kSlots];  // oldest entry goes
    s.used = true;
    s.key = key;
    s.map = *store;
    return true;
}

// Tensor map over a bf16 cache [B, Lmax, Hkv, D]: dimensions (D, Hkv, Lmax, B) innermost first; one box
// is [box_keys entries] x [1 head] x [64 channels] = rows of 128 bytes, written with the 128-byte swizzle.
// Rows past Lmax are filled with zeros.
static int make_cache_map_uncached(CUtensorMap* map, const void* base, int B, int Lmax, int Hkv, int D, int box_keys);
static int make_cache_map(CUtensorMap* map, const void* base, int B, int Lmax, int Hkv, int D, int box_keys) {
    const MapKey key{base, 1, B, Lmax, Hkv, D, box_keys};
    if (cached_map(key, map, nullptr)) return SWAA_OK;
    const int rc = make_cache_map_uncached(map, base, B, Lmax, Hkv, D, box_keys);
    if (rc == SWAA_OK) cached_map(key, nullptr, map);
    return rc;
}
static int make_cache_map_uncached(CUtensorMap* map, const void* base, int B, int Lmax, int Hkv, int D, int box_keys) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return SWAA_ERR_CUDA;
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Hkv, (cuuint64_t)Lmax, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)Hkv * D * 2, (cuuint64_t)Lmax * Hkv * D * 2};
    const cuuint32_t box[4] = {64, 1, (cuuint32_t)box_keys, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SWAA_OK : SWAA_ERR_CUDA;
}

// The dynamic shared-memory limit of a kernel instance is set once per device (it is a per-device function attribute).
template <typename Kernel>
static int ensure_dynamic_smem(Kernel kernel, int bytes, std::atomic<bool> (&done)[64]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SWAA_ERR_CUDA;
    if (done[dev].load(std::memory_order_acquire)) return SWAA_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return SWAA_ERR_CUDA;
    done[dev].store(true, std::memory_order_release);
    return SWAA_OK;
}

template <int D, int NH, bool kPaged, bool kShard = false>
static int launch_decode(const CUtensorMap (&tm)[4], const DecodeParams& p, int blocks, cudaStream_t st) {
    using L = DecodeSmem<D, NH>;
    static std::atomic<bool> attr_done[64];
    if (ensure_dynamic_smem(decode_kernel<D, NH, kPaged, kShard>, L::kDynamicBytes, attr_done) != SWAA_OK) return SWAA_ERR_CUDA;
    decode_kernel<D, NH, kPaged, kShard><<<(unsigned)blocks, kDecodeThreads, L::kDynamicBytes, st>>>(tm[0], tm[1], tm[2], tm[3], p);
    launch_counter().fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? SWAA_OK : SWAA_ERR_CUDA;
}

}  // namespace swaa

using namespace swaa;

extern "C" size_t swaa_decode_workspace_size(int B, int Hq, int Hkv, int D, int Lmax, int window, int n_sink,
                                             int is_full) {
    if (check_decode_shape(B, Hq, Hkv, D, Lmax, window, n_sink, is_full) != SWAA_OK || B == 0) return 256;
    DeviceInfo info;
    if (current_device_info(&info) != SWAA_OK) info.sm_count = 148;
    return plan_decode(B, Hq, Hkv, D, Lmax, window, n_sink, is_full, info.sm_count).bytes;
}

extern "C" int swaa_decode_num_blocks(int B, int Hq, int Hkv, int D, int Lmax, int window, int n_sink,
                                      int is_full) {
    if (check_decode_shape(B, Hq, Hkv, D, Lmax, window, n_sink, is_full) != SWAA_OK || B == 0) return 1;
    DeviceInfo info;
    if (current_device_info(&info) != SWAA_OK) info.sm_count = 148;
    return plan_decode(B, Hq, Hkv, D, Lmax, window, n_sink, is_full, info.sm_count).blocks;
}

namespace swaa {

// Shared body of swaa_decode (block_table == nullptr: dense cache [B, Lmax, Hkv, D]) and swaa_decode_paged
// (cache = pages [num_pages, page_size, Hkv, D]; Lmax = max_blocks * page_size).
static int decode_impl(const void* q, const void* kcache, const void* vcache, void* out, const int32_t* seqlens,
                       const int32_t* block_table, int max_blocks, int num_pages, int page_size, int B, int Lmax, int Hq,
                       int Hkv, int D, int window, int n_sink, int is_full, float scale, void* workspace,
                       size_t workspace_bytes, void* stream, float* part_out = nullptr, int pos0 = 0) {
    const bool paged = block_table != nullptr;
    const bool shard = part_out != nullptr;  // one shard of a cache cut along the context: `out` is not used
    int rc = check_decode_shape(B, Hq, Hkv, D, Lmax, window, n_sink, is_full);
    if (rc != SWAA_OK) return rc;
    if (B == 0) return SWAA_OK;
    if (!q || !kcache || !vcache || (!out && !shard) || !seqlens) return SWAA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(kcache) || !aligned16(vcache) || !aligned16(out)) return SWAA_ERR_INVALID_ARG;
    if (shard && (pos0 < 0 || (reinterpret_cast<uintptr_t>(part_out) & 3u) != 0)) return SWAA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(seqlens) & 3u) != 0 || (reinterpret_cast<uintptr_t>(block_table) & 3u) != 0)
        return SWAA_ERR_INVALID_ARG;
    DeviceInfo info;
    rc = current_device_info(&info);
    if (rc != SWAA_OK) return rc;
    if (info.cc_major != 10) return SWAA_ERR_UNSUPPORTED;
    const DecodePlan pl = plan_decode(B, Hq, Hkv, D, Lmax, window, n_sink, is_full, info.sm_count, paged, shard);
    if (pl.too_large) return SWAA_ERR_UNSUPPORTED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || workspace_bytes < pl.bytes)
        return SWAA_ERR_WORKSPACE;

    // K, V with the full box; K, V with the small box.  A paged cache is addressed as (page, row in page).
    CUtensorMap tm[4];
    const int outer = paged ? num_pages : B, rows = paged ? page_size : Lmax;
    if ((rc = make_cache_map(&tm[0], kcache, outer, rows, Hkv, D, kDecodeTileKeys)) != SWAA_OK) return rc;
    if ((rc = make_cache_map(&tm[1], vcache, outer, rows, Hkv, D, kDecodeTileKeys)) != SWAA_OK) return rc;
    if ((rc = make_cache_map(&tm[2], kcache, outer, rows, Hkv, D, kDecodeSmallBoxKeys)) != SWAA_OK) return rc;
    if ((rc = make_cache_map(&tm[3], vcache, outer, rows, Hkv, D, kDecodeSmallBoxKeys)) != SWAA_OK) return rc;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    DecodeParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.seqlens = seqlens;
    p.B = B;
    p.Lmax = Lmax;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.G = Hq / Hkv;
    p.HG = pl.HG;
    p.IPB = Hkv * pl.HG;
    p.window = window;
    p.n_sink = n_sink;
    p.is_full = is_full ? 1 : 0;
    const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)D);
    p.sl2 = sc * 1.4426950408889634f;
    char* ws = static_cast<char*>(workspace);
    p.tickets = reinterpret_cast<unsigned long long*>(ws);
    p.part = reinterpret_cast<float*>(ws + pl.off_part);
    p.stamp = next_call_stamp();
    p.block_table = block_table;
    p.max_blocks = max_blocks;
    p.page_tiles = paged ? page_size / kDecodeTileKeys : 1;
    p.num_pages = num_pages;
    p.pos0 = pos0;
    p.scale = sc;
    p.part_out = part_out;
    if (shard) {
        if (D == 128)
            return pl.NH == 1 ? launch_decode<128, 1, false, true>(tm, p, pl.blocks, st)
                              : launch_decode<128, 2, false, true>(tm, p, pl.blocks, st);
        return pl.NH == 1 ? launch_decode<64, 1, false, true>(tm, p, pl.blocks, st)
                          : launch_decode<64, 2, false, true>(tm, p, pl.blocks, st);
    }
    if (paged) {
        if (D == 128)
            return pl.NH == 1 ? launch_decode<128, 1, true>(tm, p, pl.blocks, st)
                              : launch_decode<128, 2, true>(tm, p, pl.blocks, st);
        return pl.NH == 1 ? launch_decode<64, 1, true>(tm, p, pl.blocks, st) : launch_decode<64, 2, true>(tm, p, pl.blocks, st);
    }
    if (D == 128)
        return pl.NH == 1 ? launch_decode<128, 1, false>(tm, p, pl.blocks, st)
                          : launch_decode<128, 2, false>(tm, p, pl.blocks, st);
    return pl.NH == 1 ? launch_decode<64, 1, false>(tm, p, pl.blocks, st) : launch_decode<64, 2, false>(tm, p, pl.blocks, st);
}

static int check_paged_shape(int max_blocks, int num_pages, int page_size) {
    if (max_blocks < 1 || num_pages < 1 || page_size < 1) return SWAA_ERR_INVALID_ARG;
    if (page_size % kDecodeTileKeys != 0) return SWAA_ERR_UNSUPPORTED;
    if ((long long)max_blocks * page_size > 2147483647LL) return SWAA_ERR_UNSUPPORTED;
    return SWAA_OK;
}

}  // namespace swaa

extern "C" int swaa_decode(const void* q, const void* kcache, const void* vcache, void* out, const int32_t* seqlens,
                           int B, int Lmax, int Hq, int Hkv, int D, int window, int n_sink, int is_full, float scale,
                           void* workspace, size_t workspace_bytes, void* stream) {
    return decode_impl(q, kcache, vcache, out, seqlens, nullptr, 0, 0, 0, B, Lmax, Hq, Hkv, D, window, n_sink, is_full,
                       scale, workspace, workspace_bytes, stream);
}

extern "C" size_t swaa_decode_paged_workspace_size(int B, int Hq, int Hkv, int D, int max_blocks, int page_size,
                                                   int window, int n_sink, int is_full) {
    if (check_paged_shape(max_blocks, 1, page_size) != SWAA_OK) return 256;
    const int Lmax = max_blocks * page_size;
    if (check_decode_shape(B, Hq, Hkv, D, Lmax, window, n_sink, is_full) != SWAA_OK || B == 0) return 256;
    DeviceInfo info;
    if (current_device_info(&info) != SWAA_OK) info.sm_count = 148;
    return plan_decode(B, Hq, Hkv, D, Lmax, window, n_sink, is_full, info.sm_count, true).bytes;
}

extern "C" int swaa_decode_paged(const void* q, const void* kpages, const void* vpages, void* out,
                                 const int32_t* block_table, const int32_t* seqlens, int B, int max_blocks,
                                 int num_pages, int page_size, int Hq, int Hkv, int D, int window, int n_sink,
                                 int is_full, float scale, void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = check_paged_shape(max_blocks, num_pages, page_size);
    if (rc != SWAA_OK) return rc;
    if (!block_table) return SWAA_ERR_INVALID_ARG;
    return decode_impl(q, kpages, vpages, out, seqlens, block_table, max_blocks, num_pages, page_size, B,
                       max_blocks * page_size, Hq, Hkv, D, window, n_sink, is_full, scale, workspace, workspace_bytes,
                       stream);
}

// ------------------------------------------------------- decode with the cache cut along the context
extern "C" size_t swaa_decode_partial_workspace_size(int B, int Hq, int Hkv, int D, int Lshard, int window, int n_sink,
                                                     int is_full) {
    if (check_decode_shape(B, Hq, Hkv, D, Lshard, window, n_sink, is_full) != SWAA_OK || B == 0) return 256;
    DeviceInfo info;
    if (current_device_info(&info) != SWAA_OK) info.sm_count = 148;
    return plan_decode(B, Hq, Hkv, D, Lshard, window, n_sink, is_full, info.sm_count, false, true).bytes;
}

extern "C" int swaa_decode_partial(const void* q, const void* kshard, const void* vshard, float* partial_out,
                                   const int32_t* seqlens, int B, int Lshard, int key_pos0, int Hq, int Hkv, int D,
                                   int window, int n_sink, int is_full, float scale, void* workspace,
                                   size_t workspace_bytes, void* stream) {
    if (!partial_out) return SWAA_ERR_INVALID_ARG;
    return decode_impl(q, kshard, vshard, nullptr, seqlens, nullptr, 0, 0, 0, B, Lshard, Hq, Hkv, D, window, n_sink,
                       is_full, scale, workspace, workspace_bytes, stream, partial_out, key_pos0);
}

extern "C" int swaa_decode_combine(const float* partials, int P, int B, int Hq, int D, void* out, void* stream) {
    if (P < 1 || B < 0 || Hq < 1) return SWAA_ERR_INVALID_ARG;
    if (D != 64 && D != 128) return SWAA_ERR_UNSUPPORTED;
    if (B == 0) return SWAA_OK;
    if (!partials || !out || (reinterpret_cast<uintptr_t>(partials) & 3u) != 0 || (reinterpret_cast<uintptr_t>(out) & 1u) != 0)
        return SWAA_ERR_INVALID_ARG;
    if ((long long)B * Hq > 0x3fffffffLL) return SWAA_ERR_UNSUPPORTED;
    const int rows = B * Hq;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const unsigned blocks = (unsigned)((rows + 3) / 4);  // four warps per block, one row each
    if (D == 128)
        decode_combine_kernel<128><<<blocks, 128, 0, st>>>(partials, P, rows, static_cast<__nv_bfloat16*>(out));
    else
        decode_combine_kernel<64><<<blocks, 128, 0, st>>>(partials, P, rows, static_cast<__nv_bfloat16*>(out));
    launch_counter().fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? SWAA_OK : SWAA_ERR_CUDA;
}

// ----------------------------------------------------------------------------------------- prefill
namespace swaa {

// Tensor map over a token-major bf16 tensor [T, H, D]: dimensions (D, H, T) innermost first; one box is
// [128 tokens] x [1 head] x [64 channels] = 128 rows of 128 bytes, written with the 128-byte swizzle.
static int make_token_major_map_uncached(CUtensorMap* map, const void* base, int T, int H, int D, int box_tokens);
static int make_token_major_map(CUtensorMap* map, const void* base, int T, int H, int D, int box_tokens = 128) {
    const MapKey key{base, 2, T, H, D, box_tokens, 0};
    if (cached_map(key, map, nullptr)) return SWAA_OK;
    const int rc = make_token_major_map_uncached(map, base, T, H, D, box_tokens);
    if (rc == SWAA_OK) cached_map(key, nullptr, map);
    return rc;
}
static int make_token_major_map_uncached(CUtensorMap* map, const void* base, int T, int H, int D, int box_tokens) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return SWAA_ERR_CUDA;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)T};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)H * D * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)box_tokens};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SWAA_OK : SWAA_ERR_CUDA;
}

// fp32 [T][H][D] accumulator, boxes of [rows][1 head][D] without swizzle (target of bulk reduce-add copies).
static int make_accum_map(CUtensorMap* map, const float* base, int T, int H, int D, int box_rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return SWAA_ERR_CUDA;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)T};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 4, (cuuint64_t)H * D * 4};
    const cuuint32_t box[3] = {(cuuint32_t)D, 1, (cuuint32_t)box_rows};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SWAA_OK : SWAA_ERR_CUDA;
}

template <int D, int kMode, bool kLseOnly = false>
static int launch_prefill(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                          const CUtensorMap& tsk, const CUtensorMap& tsv, const PrefillParams& p, int sm_count,
                          cudaStream_t st) {
    using L = PrefillSmem<D>;
    static std::atomic<bool> attr_done[64];
    if (ensure_dynamic_smem(prefill_kernel<D, kMode, kLseOnly>, L::kDynamicBytes, attr_done) != SWAA_OK) return SWAA_ERR_CUDA;
    // persistent blocks: one per SM (or fewer when there is less work), each walks its share of the items
    long long blocks = (long long)p.n_pairs * p.tiles_ub;
    if (blocks > sm_count) blocks = sm_count;
    prefill_kernel<D, kMode, kLseOnly><<<(unsigned)blocks, kPrefillThreads, L::kDynamicBytes, st>>>(tq, tk, tv, to, tsk, tsv, p);
    launch_counter().fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? SWAA_OK : SWAA_ERR_CUDA;
}

}  // namespace swaa

namespace swaa {

// Shared body of swaa_prefill (cu_seqlens_k == nullptr: keys are packed like the queries) and
// swaa_prefill_chunked.
struct PagedKV {  // keys and values in pages (null block_table: packed layout)
    const int32_t* block_table = nullptr;
    int max_blocks = 0, num_pages = 0, page_size = 0;
};

struct PrefillExtras {
    const uint8_t* is_full_seq = nullptr;  // mask policy per sequence (chunked / paged)
    // context-parallel prefill: local keys start at key_pos0[b]; sink rows in [B, sink_rows, Hkv, D] buffers
    bool context_parallel = false;
    bool lse_only = false;  // chunked layout only: write lse and nothing else (q, k needed; v and out are not touched)
    const int32_t* key_pos0 = nullptr;
    const void* sink_k = nullptr;
    const void* sink_v = nullptr;
    int sink_rows = 0;
};

static int prefill_impl(const void* q, const void* k, const void* v, void* out, const int32_t* cu_seqlens_q,
                        const int32_t* cu_seqlens_k, int B, int Tq, int Tk, int max_seqlen_q, int max_seqlen_k, int Hq,
                        int Hkv, int D, int window, int n_sink, int is_full, float scale, float* lse, void* stream,
                        const PagedKV& paged = PagedKV(), const PrefillExtras& ex = PrefillExtras()) {
    if (B < 0 || Tq < 0 || Tk < 0 || max_seqlen_q < 0 || max_seqlen_k < 0 || Hq < 1 || Hkv < 1 || n_sink < 0)
        return SWAA_ERR_INVALID_ARG;
    if ((!is_full || ex.is_full_seq != nullptr) && window < 1) return SWAA_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || (D != 64 && D != 128)) return SWAA_ERR_UNSUPPORTED;
    if (B == 0 || Tq == 0) return SWAA_OK;
    if (ex.lse_only) {  // v and out stand in with q's address: never dereferenced, only encoded into unused tensor maps
        if (!lse || !cu_seqlens_k || paged.block_table || ex.context_parallel) return SWAA_ERR_INVALID_ARG;
        v = k;
        out = const_cast<void*>(q);
    }
    if (!q || !k || !v || !out || !cu_seqlens_q) return SWAA_ERR_INVALID_ARG;
    if (ex.context_parallel) {
        if (!ex.key_pos0 || ex.sink_rows < 0 || (reinterpret_cast<uintptr_t>(ex.key_pos0) & 3u) != 0)
            return SWAA_ERR_INVALID_ARG;
        if (ex.sink_rows > 0 && (!ex.sink_k || !ex.sink_v || !aligned16(ex.sink_k) || !aligned16(ex.sink_v)))
            return SWAA_ERR_INVALID_ARG;
    }
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return SWAA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(cu_seqlens_q) & 3u) != 0 || (reinterpret_cast<uintptr_t>(cu_seqlens_k) & 3u) != 0 ||
        (reinterpret_cast<uintptr_t>(lse) & 3u) != 0)
        return SWAA_ERR_INVALID_ARG;
    const bool is_paged = paged.block_table != nullptr;
    if (!is_paged && Tk < Tq) return SWAA_ERR_INVALID_ARG;
    DeviceInfo info;
    int rc = current_device_info(&info);
    if (rc != SWAA_OK) return rc;
    if (info.cc_major != 10) return SWAA_ERR_UNSUPPORTED;

    CUtensorMap tq, tk, tv, to;
    if ((rc = make_token_major_map(&tq, q, Tq, Hq, D)) != SWAA_OK) return rc;
    if (is_paged) {  // (D, Hkv, page_size, num_pages), boxes of 128 rows of one page
        if ((rc = make_cache_map(&tk, k, paged.num_pages, paged.page_size, Hkv, D, kPrefillBN)) != SWAA_OK) return rc;
        if ((rc = make_cache_map(&tv, v, paged.num_pages, paged.page_size, Hkv, D, kPrefillBN)) != SWAA_OK) return rc;
    } else {
        if ((rc = make_token_major_map(&tk, k, Tk, Hkv, D)) != SWAA_OK) return rc;
        if ((rc = make_token_major_map(&tv, v, Tk, Hkv, D)) != SWAA_OK) return rc;
    }
    if ((rc = make_token_major_map(&to, out, Tq, Hq, D, 32)) != SWAA_OK) return rc;  // output rows, 32 at a time
    CUtensorMap tsk = tk, tsv = tv;  // only the context-parallel instance reads these
    if (ex.context_parallel && ex.sink_rows > 0) {  // (D, Hkv, sink_rows, B); rows past sink_rows read as zeros
        if ((rc = make_cache_map(&tsk, ex.sink_k, B, ex.sink_rows, Hkv, D, kPrefillBN)) != SWAA_OK) return rc;
        if ((rc = make_cache_map(&tsv, ex.sink_v, B, ex.sink_rows, Hkv, D, kPrefillBN)) != SWAA_OK) return rc;
    }

    PrefillParams p;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.cu_seqlens = cu_seqlens_q;
    p.cu_seqlens_k = cu_seqlens_k;
    p.B = B;
    p.T = Tq;
    p.Tk = Tk;
    p.max_seqlen = max_seqlen_q;
    p.max_seqlen_k = max_seqlen_k;
    p.block_table = paged.block_table;
    p.max_blocks = paged.max_blocks;
    p.page_size = paged.page_size;
    p.num_pages = paged.num_pages;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.G = Hq / Hkv;
    p.pairs_per_kv = (p.G + 1) / 2;
    p.n_pairs = Hkv * p.pairs_per_kv;
    const long long ub_a = (long long)Tq / kPrefillBM + B;
    const long long ub_b = (long long)B * ((max_seqlen_q + kPrefillBM - 1) / kPrefillBM);
    const long long ub = ub_a < ub_b ? ub_a : ub_b;
    if (ub > 2147483647LL / p.n_pairs) return SWAA_ERR_UNSUPPORTED;
    p.tiles_ub = (int)ub;
    if (p.tiles_ub == 0) return SWAA_OK;  // max_seqlen == 0: nothing can be valid
    // a window that covers the longest key sequence is full causal attention for every row; clamping keeps the
    // kernel's 32-bit column arithmetic (column - window) far from overflow
    // (context-parallel: positions are offset by key_pos0, so the bound there is a constant far above any length)
    if (ex.context_parallel) {
        if (window > (1 << 30)) window = 1 << 30;
    } else if (!is_full && max_seqlen_k >= 1 && window > max_seqlen_k) {
        window = max_seqlen_k;
    }
    p.window = window;
    p.n_sink = n_sink;
    p.is_full = is_full ? 1 : 0;
    p.is_full_seq = ex.is_full_seq;
    p.key_pos0 = ex.key_pos0;
    // with no sink rows supplied only a participant whose keys start at position 0 can have sink keys
    p.sink_rows = ex.sink_rows;
    p.scale = scale > 0.f ? scale : 1.0f / sqrtf((float)D);
    p.sl2 = p.scale * 1.4426950408889634f;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (ex.context_parallel)
        return D == 128 ? launch_prefill<128, 3>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st)
                        : launch_prefill<64, 3>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st);
    if (is_paged)
        return D == 128 ? launch_prefill<128, 2>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st)
                        : launch_prefill<64, 2>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st);
    if (ex.lse_only)
        return D == 128 ? launch_prefill<128, 1, true>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st)
                        : launch_prefill<64, 1, true>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st);
    if (cu_seqlens_k != nullptr)
        return D == 128 ? launch_prefill<128, 1>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st)
                        : launch_prefill<64, 1>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st);
    return D == 128 ? launch_prefill<128, 0>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st)
                    : launch_prefill<64, 0>(tq, tk, tv, to, tsk, tsv, p, info.sm_count, st);
}

}  // namespace swaa

extern "C" int swaa_prefill(const void* q, const void* k, const void* v, void* out, const int32_t* cu_seqlens, int B,
                            int T, int max_seqlen, int Hq, int Hkv, int D, int window, int n_sink, int is_full,
                            float scale, float* lse, void* stream) {
    return prefill_impl(q, k, v, out, cu_seqlens, nullptr, B, T, T, max_seqlen, max_seqlen, Hq, Hkv, D, window, n_sink,
                        is_full, scale, lse, stream);
}

extern "C" int swaa_prefill_chunked(const void* q, const void* k, const void* v, void* out,
                                    const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k, int B, int Tq, int Tk,
                                    int max_seqlen_q, int max_seqlen_k, int Hq, int Hkv, int D, int window, int n_sink,
                                    int is_full, float scale, float* lse, void* stream) {
    if (!cu_seqlens_k) return SWAA_ERR_INVALID_ARG;
    return prefill_impl(q, k, v, out, cu_seqlens_q, cu_seqlens_k, B, Tq, Tk, max_seqlen_q, max_seqlen_k, Hq, Hkv, D,
                        window, n_sink, is_full, scale, lse, stream);
}

extern "C" int swaa_prefill_paged(const void* q, const void* kpages, const void* vpages, void* out,
                                  const int32_t* cu_seqlens_q, const int32_t* seqlens_k, const int32_t* block_table, int B,
                                  int Tq, int max_seqlen_q, int max_blocks, int num_pages, int page_size, int Hq, int Hkv,
                                  int D, int window, int n_sink, int is_full, float scale, float* lse, void* stream) {
    if (!seqlens_k || !block_table) return SWAA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(block_table) & 3u) != 0) return SWAA_ERR_INVALID_ARG;
    if (max_blocks < 1 || num_pages < 1 || page_size < 1) return SWAA_ERR_INVALID_ARG;
    if (page_size % kPrefillBN != 0 || (long long)max_blocks * page_size > 2147483647LL) return SWAA_ERR_UNSUPPORTED;
    PagedKV pg;
    pg.block_table = block_table;
    pg.max_blocks = max_blocks;
    pg.num_pages = num_pages;
    pg.page_size = page_size;
    return prefill_impl(q, kpages, vpages, out, cu_seqlens_q, seqlens_k, B, Tq, 0, max_seqlen_q, max_blocks * page_size, Hq,
                        Hkv, D, window, n_sink, is_full, scale, lse, stream, pg);
}

extern "C" int swaa_prefill_chunked_mixed(const void* q, const void* k, const void* v, void* out,
                                          const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k,
                                          const uint8_t* is_full_seq, int B, int Tq, int Tk, int max_seqlen_q,
                                          int max_seqlen_k, int Hq, int Hkv, int D, int window, int n_sink, float scale,
                                          float* lse, void* stream) {
    if (!cu_seqlens_k || !is_full_seq) return SWAA_ERR_INVALID_ARG;
    PrefillExtras ex;
    ex.is_full_seq = is_full_seq;
    return prefill_impl(q, k, v, out, cu_seqlens_q, cu_seqlens_k, B, Tq, Tk, max_seqlen_q, max_seqlen_k, Hq, Hkv, D,
                        window, n_sink, 0, scale, lse, stream, PagedKV(), ex);
}

extern "C" int swaa_prefill_paged_mixed(const void* q, const void* kpages, const void* vpages, void* out,
                                        const int32_t* cu_seqlens_q, const int32_t* seqlens_k,
                                        const int32_t* block_table, const uint8_t* is_full_seq, int B, int Tq,
                                        int max_seqlen_q, int max_blocks, int num_pages, int page_size, int Hq, int Hkv,
                                        int D, int window, int n_sink, float scale, float* lse, void* stream) {
    if (!seqlens_k || !block_table || !is_full_seq) return SWAA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(block_table) & 3u) != 0) return SWAA_ERR_INVALID_ARG;
    if (max_blocks < 1 || num_pages < 1 || page_size < 1) return SWAA_ERR_INVALID_ARG;
    if (page_size % kPrefillBN != 0 || (long long)max_blocks * page_size > 2147483647LL) return SWAA_ERR_UNSUPPORTED;
    PagedKV pg;
    pg.block_table = block_table;
    pg.max_blocks = max_blocks;
    pg.num_pages = num_pages;
    pg.page_size = page_size;
    PrefillExtras ex;
    ex.is_full_seq = is_full_seq;
    return prefill_impl(q, kpages, vpages, out, cu_seqlens_q, seqlens_k, B, Tq, 0, max_seqlen_q, max_blocks * page_size, Hq,
                        Hkv, D, window, n_sink, 0, scale, lse, stream, pg, ex);
}

extern "C" int swaa_prefill_context_parallel(const void* q, const void* k_local, const void* v_local,
                                             const void* sink_k, const void* sink_v, void* out,
                                             const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k,
                                             const int32_t* key_pos0, int B, int Tq, int Tk, int max_seqlen_q,
                                             int max_seqlen_k, int sink_rows, int Hq, int Hkv, int D, int window,
                                             int n_sink, float scale, float* lse, void* stream) {
    if (!cu_seqlens_k || !key_pos0) return SWAA_ERR_INVALID_ARG;
    PrefillExtras ex;
    ex.context_parallel = true;
    ex.key_pos0 = key_pos0;
    ex.sink_k = sink_k;
    ex.sink_v = sink_v;
    ex.sink_rows = sink_rows;
    return prefill_impl(q, k_local, v_local, out, cu_seqlens_q, cu_seqlens_k, B, Tq, Tk, max_seqlen_q, max_seqlen_k, Hq,
                        Hkv, D, window, n_sink, 0, scale, lse, stream, PagedKV(), ex);
}

// -------------------------------------------------------------------------------------- backward
namespace swaa {

// Workspace: [dq accumulator | dk, dv accumulators of the split sink tiles] (zeroed by one memset) | delta | lse2.
struct BackwardWorkspace {
    size_t off_dkv, zero_bytes, off_delta, off_lse2, bytes;
    int sink_rows;
};

static BackwardWorkspace backward_workspace(int B, int T, int Hq, int Hkv, int D, int n_sink) {
    BackwardWorkspace w;
    // rows of the key tiles that hold sink keys, in whole tiles of the wider of the two kernels
    const long long t_rows = ((long long)T + kBwdTcKeys - 1) / kBwdTcKeys * kBwdTcKeys;
    const long long s_rows = ((long long)n_sink + kBwdTcKeys - 1) / kBwdTcKeys * kBwdTcKeys;
    w.sink_rows = (int)(s_rows < t_rows ? s_rows : t_rows);
    w.off_dkv = ((size_t)T * Hq * D * sizeof(float) + 255) / 256 * 256;
    w.zero_bytes = w.off_dkv + 2 * (size_t)B * w.sink_rows * Hkv * D * sizeof(float);
    w.off_delta = (w.zero_bytes + 255) / 256 * 256;
    w.off_lse2 = w.off_delta + ((size_t)Hq * T * sizeof(float) + 255) / 256 * 256;
    w.bytes = w.off_lse2 + (size_t)Hq * T * sizeof(float);
    return w;
}

// D = 128 runs on the tcgen05 kernel (128-key tiles), D = 64 on the warp-level kernel (64-key tiles).
template <int D>
static int launch_backward(const void* q, const void* k, const void* v, const void* out, const void* dout,
                           const BackwardParams& p, void* dq, int max_seqlen, size_t dkv_zero_bytes, cudaStream_t st) {
    constexpr bool kTc = D == 128;
    constexpr int kKeyTile = kTc ? kBwdTcKeys : kBwdTile;
    constexpr int kRowTile = kTc ? kBwdTcRows : kBwdTile;
    CUtensorMap tq, tk, tv, tdo;
    int rc;
    if ((rc = make_token_major_map(&tq, q, p.T, p.Hq, D, kRowTile)) != SWAA_OK) return rc;
    if ((rc = make_token_major_map(&tk, k, p.T, p.Hkv, D, kKeyTile)) != SWAA_OK) return rc;
    if ((rc = make_token_major_map(&tv, v, p.T, p.Hkv, D, kKeyTile)) != SWAA_OK) return rc;
    if ((rc = make_token_major_map(&tdo, dout, p.T, p.Hq, D, kRowTile)) != SWAA_OK) return rc;
    const size_t n_acc = (size_t)p.T * p.Hq * D;
    // the dq accumulator is cleared by the kernel that computes the row terms; the (small) dk, dv accumulators here
    if (dkv_zero_bytes > 0 && cudaMemsetAsync(p.dkv_accum, 0, dkv_zero_bytes, st) != cudaSuccess) return SWAA_ERR_CUDA;
    const int rows = p.T * p.Hq;
    backward_delta_kernel<D><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(out), static_cast<const __nv_bfloat16*>(dout), p.lse,
        const_cast<float*>(p.delta), const_cast<float*>(p.lse2), p.dq_accum, p.T, p.Hq);
    const int ntiles = (max_seqlen + kKeyTile - 1) / kKeyTile;
    const dim3 grid((unsigned)(p.sink_tiles * p.chunks + (ntiles - p.sink_tiles)), (unsigned)p.Hkv, (unsigned)p.B);
    if constexpr (kTc) {
        if (cudaFuncSetAttribute(backward_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 BackwardTcSmem::kDynamicBytes) != cudaSuccess)
            return SWAA_ERR_CUDA;
        CUtensorMap tacc;
        if ((rc = make_accum_map(&tacc, p.dq_accum, p.T, p.Hq, D, kBwdTcRows)) != SWAA_OK) return rc;
        backward_tc_kernel<<<grid, kBwdTcThreads, BackwardTcSmem::kDynamicBytes, st>>>(tq, tk, tv, tdo, tacc, p);
    } else {
        using L = BackwardSmem<D>;
        if (cudaFuncSetAttribute(backward_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) !=
            cudaSuccess)
            return SWAA_ERR_CUDA;
        backward_kernel<D><<<grid, kBwdThreads, L::kDynamicBytes, st>>>(tq, tk, tv, tdo, p);
    }
    backward_convert_dq_kernel<<<(unsigned)((n_acc / 4 + 255) / 256 + 1), 256, 0, st>>>(
        p.dq_accum, static_cast<__nv_bfloat16*>(dq), n_acc);
    int launches = 3;
    if (p.sink_tiles > 0) {
        const int sink_rows = p.sink_tiles * kKeyTile;
        const size_t plane = (size_t)p.B * sink_rows * p.Hkv * D;
        backward_convert_dkv_kernel<<<(unsigned)((plane / 4 + 255) / 256), 256, 0, st>>>(
            p.dkv_accum, p.dk, p.dv, p.cu_seqlens, p.B, p.T, p.max_seqlen, sink_rows, p.Hkv, D);
        ++launches;
    }
    launch_counter().fetch_add((uint64_t)launches, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? SWAA_OK : SWAA_ERR_CUDA;
}

}  // namespace swaa

extern "C" size_t swaa_prefill_backward_workspace_size(int B, int T, int Hq, int Hkv, int D, int n_sink) {
    if (B < 1 || T < 1 || Hq < 1 || Hkv < 1 || D < 1 || n_sink < 0) return 256;
    return backward_workspace(B, T, Hq, Hkv, D, n_sink).bytes;
}

extern "C" int swaa_prefill_backward(const void* q, const void* k, const void* v, const void* out, const void* dout,
                                     const float* lse, const int32_t* cu_seqlens, int B, int T, int max_seqlen, int Hq,
                                     int Hkv, int D, int window, int n_sink, int is_full, float scale, void* dq, void* dk,
                                     void* dv, void* workspace, size_t workspace_bytes, void* stream) {
    if (B < 0 || T < 0 || max_seqlen < 0 || Hq < 1 || Hkv < 1 || n_sink < 0) return SWAA_ERR_INVALID_ARG;
    if (!is_full && window < 1) return SWAA_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || (D != 64 && D != 128)) return SWAA_ERR_UNSUPPORTED;
    if (B > 65535 || Hkv > 65535) return SWAA_ERR_UNSUPPORTED;  // grid dimensions
    if (B == 0 || T == 0 || max_seqlen == 0) return SWAA_OK;
    if (!q || !k || !v || !out || !dout || !lse || !cu_seqlens || !dq || !dk || !dv) return SWAA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(dout) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return SWAA_ERR_INVALID_ARG;
    const BackwardWorkspace w = backward_workspace(B, T, Hq, Hkv, D, n_sink);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || workspace_bytes < w.bytes)
        return SWAA_ERR_WORKSPACE;
    DeviceInfo info;
    const int rc = current_device_info(&info);
    if (rc != SWAA_OK) return rc;
    if (info.cc_major != 10) return SWAA_ERR_UNSUPPORTED;
    char* ws = static_cast<char*>(workspace);
    BackwardParams p;
    p.lse = lse;
    p.dq_accum = reinterpret_cast<float*>(ws);
    p.dkv_accum = reinterpret_cast<float*>(ws + w.off_dkv);
    p.delta = reinterpret_cast<float*>(ws + w.off_delta);
    p.lse2 = reinterpret_cast<float*>(ws + w.off_lse2);
    p.dk = static_cast<__nv_bfloat16*>(dk);
    p.dv = static_cast<__nv_bfloat16*>(dv);
    p.cu_seqlens = cu_seqlens;
    p.B = B;
    p.T = T;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.G = Hq / Hkv;
    p.max_seqlen = max_seqlen;
    p.window = window;
    p.n_sink = n_sink;
    p.is_full = is_full ? 1 : 0;
    p.scale = scale > 0.f ? scale : 1.0f / sqrtf((float)D);
    // Key tiles that hold sink keys meet every later query tile: with long sequences their query range is cut
    // into chunks handled by separate blocks, which add dk, dv into the fp32 accumulators.
    const int key_tile = D == 128 ? kBwdTcKeys : kBwdTile;  // the two kernels' key tiles; both step over 64 query rows
    const int ntiles = (max_seqlen + key_tile - 1) / key_tile;
    p.chunks = ((max_seqlen + 63) / 64 + kBwdChunkTiles - 1) / kBwdChunkTiles;
    p.sink_tiles = 0;
    if (!is_full && p.chunks > 1) {
        const int st_need = (int)(((long long)n_sink + key_tile - 1) / key_tile);
        p.sink_tiles = st_need < ntiles ? st_need : ntiles;
        if (p.sink_tiles * key_tile > w.sink_rows) p.sink_tiles = w.sink_rows / key_tile;
    }
    if (p.sink_tiles == 0) p.chunks = 1;
    if ((long long)p.sink_tiles * p.chunks + (ntiles - p.sink_tiles) > 0x7fffffffLL) return SWAA_ERR_UNSUPPORTED;
    const size_t dkv_zero_bytes = 2 * (size_t)B * p.sink_tiles * key_tile * Hkv * D * sizeof(float);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    return D == 128 ? launch_backward<128>(q, k, v, out, dout, p, dq, max_seqlen, dkv_zero_bytes, st)
                    : launch_backward<64>(q, k, v, out, dout, p, dq, max_seqlen, dkv_zero_bytes, st);
}

// ------------------------------------------------------------------------------------ lazy ratio
namespace swaa {

// ratio[h] = mean over t of exp(lse_recent[h, t] - lse_full[h, t]); one block per head.
__global__ void lazy_ratio_reduce_kernel(const float* __restrict__ lse_recent, const float* __restrict__ lse_full,
                                         int Tq, float* __restrict__ ratio) {
    __shared__ float warp_sums[8];
    const int h = blockIdx.x;
    float acc = 0.f;
    for (int t = threadIdx.x; t < Tq; t += blockDim.x)
        acc += __expf(lse_recent[(size_t)h * Tq + t] - lse_full[(size_t)h * Tq + t]);
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float total = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) total += warp_sums[w];
        ratio[h] = total / (float)Tq;
    }
}

}  // namespace swaa

extern "C" int swaa_lazy_ratio(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_q,
                               const int32_t* cu_seqlens_k, int B, int Tq, int Tk, int max_seqlen_q, int max_seqlen_k,
                               int Hq, int Hkv, int D, int recent, int n_sink, float scale, float* ratio,
                               void* scratch_out, float* scratch_lse, void* stream) {
    (void)v;            // the probe needs no values: both passes run the kernel instance that only forms log-sum-exps
    (void)scratch_out;
    if (!ratio || !scratch_lse || !cu_seqlens_k) return SWAA_ERR_INVALID_ARG;
    if (recent < 1 || B < 1 || Tq < 1) return SWAA_ERR_INVALID_ARG;
    float* lse_recent = scratch_lse;
    float* lse_full = scratch_lse + (size_t)Hq * Tq;
    PrefillExtras ex;
    ex.lse_only = true;
    int rc = prefill_impl(q, k, nullptr, nullptr, cu_seqlens_q, cu_seqlens_k, B, Tq, Tk, max_seqlen_q, max_seqlen_k, Hq,
                          Hkv, D, recent, n_sink, 0, scale, lse_recent, stream, PagedKV(), ex);
    if (rc != SWAA_OK) return rc;
    rc = prefill_impl(q, k, nullptr, nullptr, cu_seqlens_q, cu_seqlens_k, B, Tq, Tk, max_seqlen_q, max_seqlen_k, Hq, Hkv, D,
                      1, 0, 1, scale, lse_full, stream, PagedKV(), ex);
    if (rc != SWAA_OK) return rc;
    lazy_ratio_reduce_kernel<<<(unsigned)Hq, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(lse_recent, lse_full, Tq,
                                                                                                ratio);
    launch_counter().fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? SWAA_OK : SWAA_ERR_CUDA;
}

// ------------------------------------------------------------------- decode without allocation
namespace swaa {

// Split-K scratch of swaa_decode_static.  One instance per device that loads this module; shared by
// every call on that device.  In host code this name is only a handle for cudaGetSymbolAddress: it
// is not a device address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_decode_static_scratch[SWAA_DECODE_STATIC_SCRATCH_BYTES];

// Device address of the scratch array on the current device, looked up once per device.
static int decode_static_scratch(void** out) {
    static std::mutex mu;
    static void* table[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SWAA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (table[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_decode_static_scratch) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return SWAA_ERR_CUDA;
        }
        table[dev] = ptr;
    }
    *out = table[dev];
    return SWAA_OK;
}

}  // namespace swaa

extern "C" int swaa_decode_static(const void* q, const void* kcache, const void* vcache, void* out,
                                  const int32_t* seqlens, int B, int Lmax, int Hq, int Hkv, int D, int window,
                                  int n_sink, int is_full, float scale, void* stream) {
    const int rc = check_decode_shape(B, Hq, Hkv, D, Lmax, window, n_sink, is_full);
    if (rc != SWAA_OK) return rc;
    if (B == 0) return SWAA_OK;
    // Reject what does not fit the fixed array before touching the device.
    if (swaa_decode_workspace_size(B, Hq, Hkv, D, Lmax, window, n_sink, is_full) > SWAA_DECODE_STATIC_SCRATCH_BYTES)
        return SWAA_ERR_WORKSPACE;
    void* scratch = nullptr;
    const int rs = decode_static_scratch(&scratch);
    if (rs != SWAA_OK) return rs;
    // Same kernel and same plan as swaa_decode.  Nothing in the scratch has to start at zero: tickets are
    // stamped per call, partial results are written before they are read.
    return swaa_decode(q, kcache, vcache, out, seqlens, B, Lmax, Hq, Hkv, D, window, n_sink, is_full, scale, scratch,
                       SWAA_DECODE_STATIC_SCRATCH_BYTES, stream);
}

// ---------------------------------------------------------------------------------------- schedule
extern "C" int swaa_schedule_is_full(const swaa_policy* policy, int layer, int phase) {
    if (!policy || policy->n_layers < 0 || layer < 0 || layer >= policy->n_layers) return SWAA_ERR_INVALID_ARG;
    if (phase != SWAA_PHASE_PREFILL && phase != SWAA_PHASE_DECODE) return SWAA_ERR_INVALID_ARG;
    if (policy->fa_start < 0 || policy->fa_step < 0) return SWAA_ERR_INVALID_ARG;
    if (phase == SWAA_PHASE_DECODE && policy->fa_decode) return 1;
    if (policy->fa_mask != nullptr) return policy->fa_mask[layer] != 0 ? 1 : 0;
    if (policy->fa_step > 0 && layer >= policy->fa_start && (layer - policy->fa_start) % policy->fa_step == 0) return 1;
    return 0;
}

extern "C" int swaa_schedule_fill(const swaa_policy* policy, int phase, uint8_t* is_full_out) {
    if (!policy || !is_full_out || policy->n_layers < 0) return SWAA_ERR_INVALID_ARG;
    for (int l = 0; l < policy->n_layers; ++l) {
        const int r = swaa_schedule_is_full(policy, l, phase);
        if (r < 0) return r;
        is_full_out[l] = (uint8_t)r;
    }
    return SWAA_OK;
}

extern "C" int swaa_schedule_select_fa_layers(const float* ratio, int n_layers, int n_heads, int n_lazy, int fa_on_lazy,
                                              uint8_t* fa_mask_out) {
    if (!ratio || !fa_mask_out || n_layers < 0 || n_heads < 1 || n_lazy < 0 || n_lazy > n_layers)
        return SWAA_ERR_INVALID_ARG;
    std::vector<double> mean((size_t)n_layers);
    std::vector<int> order((size_t)n_layers);
    for (int l = 0; l < n_layers; ++l) {
        double acc = 0.0;
        for (int h = 0; h < n_heads; ++h) acc += (double)ratio[(size_t)l * n_heads + h];
        if (!std::isfinite(acc)) return SWAA_ERR_INVALID_ARG;
        mean[(size_t)l] = acc / n_heads;
        order[(size_t)l] = l;
    }
    // laziest first; the stable sort keeps the lower index ahead among equal ratios
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return mean[(size_t)a] > mean[(size_t)b]; });
    for (int r = 0; r < n_layers; ++r) {
        const bool lazy = r < n_lazy;
        fa_mask_out[order[(size_t)r]] = (uint8_t)((fa_on_lazy != 0) == lazy ? 1 : 0);
    }
    return SWAA_OK;
}

// -------------------------------------------------------------------------------- trimmed cache
extern "C" long long swaa_trimmed_cache_slot(long long pos, int window, int n_sink) {
    if (window < 1 || n_sink < 0 || pos < 0) return -1;
    return pos < n_sink ? pos : (long long)n_sink + (pos - n_sink) % window;
}

extern "C" long long swaa_trimmed_cache_len(long long len, int window, int n_sink) {
    if (window < 1 || n_sink < 0 || len < 0) return -1;
    const long long cap = (long long)n_sink + window;
    return len < cap ? len : cap;
}

// ------------------------------------------------------------------------------- tile enumeration
extern "C" int swaa_prefill_block_m(void) { return kPrefillBM; }
extern "C" int swaa_prefill_block_n(void) { return kPrefillBN; }

extern "C" int swaa_prefill_tile_range(int L, int m, int BM, int BN, int window, int n_sink, int is_full,
                                       int* n_sink_tiles, int* n_lo, int* n_hi) {
    if (L < 1 || BM < 1 || BN < 1 || m < 0 || (long long)m * BM >= L || n_sink < 0 || (!is_full && window < 1))
        return SWAA_ERR_INVALID_ARG;
    if (!n_sink_tiles || !n_lo || !n_hi) return SWAA_ERR_INVALID_ARG;
    const int i0 = m * BM;
    const int i1 = (L < i0 + BM ? L : i0 + BM) - 1;
    const TileRange r = tile_range(i0, i1, BN, window, n_sink, is_full != 0);
    *n_sink_tiles = r.n_sink_tiles;
    *n_lo = r.n_lo;
    *n_hi = r.n_hi;
    return SWAA_OK;
}

extern "C" int swaa_prefill_tile_needs_mask(int L, int m, int n, int BM, int BN, int window, int n_sink,
                                            int is_full) {
    if (L < 1 || BM < 1 || BN < 1 || m < 0 || n < 0 || (long long)m * BM >= L || n_sink < 0 ||
        (!is_full && window < 1))
        return SWAA_ERR_INVALID_ARG;
    const int i0 = m * BM;
    const int i1 = (L < i0 + BM ? L : i0 + BM) - 1;
    return tile_needs_mask(i0, i1, n * BN, n * BN + BN - 1, window, n_sink, is_full != 0) ? 1 : 0;
}

// ------------------------------------------------------------------------------------------ status
extern "C" const char* swaa_status_str(int status) {
    switch (status) {
        case SWAA_OK: return "SWAA_OK";
        case SWAA_ERR_INVALID_ARG: return "SWAA_ERR_INVALID_ARG";
        case SWAA_ERR_UNSUPPORTED: return "SWAA_ERR_UNSUPPORTED";
        case SWAA_ERR_CUDA: return "SWAA_ERR_CUDA";
        case SWAA_ERR_WORKSPACE: return "SWAA_ERR_WORKSPACE";
        case SWAA_ERR_BAD_SEQLENS: return "SWAA_ERR_BAD_SEQLENS";
        case SWAA_ERR_TIMEOUT: return "SWAA_ERR_TIMEOUT";
        default: return "SWAA_ERR_UNKNOWN";
    }
}

extern "C" int swaa_last_device_status(void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return SWAA_ERR_CUDA;
    int value = 0;
    if (cudaMemcpyFromSymbol(&value, g_device_status, sizeof(int)) != cudaSuccess) return SWAA_ERR_CUDA;
    if (value != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return SWAA_ERR_CUDA;
    }
    return value;
}

extern "C" uint64_t swaa_kernel_launch_count(void) { return launch_counter().load(std::memory_order_relaxed); }
