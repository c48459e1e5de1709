// Decode attention (one query token per sequence) -- HBM-bound streaming kernel.
//
// Sec. 3.1.1 ("FA Decode"): the generated token attends to every earlier token, so the kernel
// streams the whole KV cache of its sequence; an SWA decode step reads the first n_sink entries plus
// the last `window` entries only.  App. A: the full-context cache is retained for decoding.
//
// Work decomposition.  An item is one (sequence, key/value head, chunk of up to 8*NH query heads of
// that head's group); all query heads of a chunk are processed together so each K/V byte is fetched
// once.  The visible cache entries of an item are cut into tiles of 64 keys (sink tiles, then window
// tiles starting at the first window key).  All tiles of all items form one list in (sequence, item,
// tile) order, and block c of a persistent grid (at most one block per SM; the host prefers a block count that puts
// the cuts on item boundaries, see plan_decode) owns the contiguous run
// [c * tpc, (c+1) * tpc) of it, so every SM streams the same number of bytes whatever the batch
// shape.  A block therefore holds at most two incomplete items (the first and the last of its run);
// it writes complete items straight to `out` and incomplete ones as (max, sum, unnormalised O)
// partials, which the last block to finish an item merges (atomic ticket, same launch).  A ticket
// carries a per-call stamp, so stale workspace contents are recognised and nothing has to be cleared.
//
// Data path.  One producer thread keeps a ring of shared-memory stages full with TMA tile copies
// (K and V boxes of [64 keys][64 channels], 128-byte swizzle; a 16-key box for tiles with at most 16
// visible keys, e.g. the sinks), so that the bytes in flight per SM do not depend on registers or
// occupancy.  Four consumer warps each take 16 keys of every tile and run
// both contractions on warp-level tensor-core MMAs with fp32 accumulation in the transposed form
//     S^T[16 keys x 8 heads] = K[16 keys x D] * Q^T[D x 8 heads]
//     O^T[16 ch  x 8 heads] += V^T[16 ch x 16 keys] * P^T[16 keys x 8 heads]
// so that the small head count sits in the MMA's N = 8 dimension.  K fragments come from ldmatrix, V^T
// fragments from ldmatrix.trans, and P^T reaches the second product's B fragment through movmatrix.
//
// Every mbarrier wait is bounded; a wait that runs out records SWAA_ERR_TIMEOUT, the consumers finish
// their loops without computing or storing, and the producer waits (bounded) for its copies in flight.
#pragma once

#include "swaa_internal.cuh"
#include "swaa_ptx.cuh"

namespace swaa {

struct DecodeParams {
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    const int32_t* seqlens;
    int B, Lmax, Hq, Hkv, G;
    int HG;        // head chunks per kv head (each chunk holds up to 8*NH query heads)
    int IPB;       // items per sequence = Hkv * HG
    int window, n_sink, is_full;
    float sl2;     // softmax scale * log2(e)
    unsigned long long* tickets;  // [gridDim.x]; (call stamp << 16 | arrivals), needs no initialisation
    unsigned long long stamp;     // 48-bit number unique to this call (never 0)
    float* part;   // [2 * gridDim.x][8*NH][D + 2]: per head (max in score units, sum, unnormalised O)
    // paged cache only: entry j of sequence b lives in page block_table[b * max_blocks + j / page_size]
    const int32_t* block_table;
    int max_blocks, page_tiles /* page_size / 64 */, num_pages;
    // one shard of a cache cut along the context (kShard): the buffers hold positions pos0 .. pos0 + Lmax - 1 of every
    // sequence, seqlens are total lengths, and every row's result leaves as a partial (max, sum, unnormalised O)
    int pos0;
    float scale;      // softmax scale (natural-log units of the exported maximum)
    float* part_out;  // [B, Hq, D + 2]
};

constexpr int kDecodeTileKeys = 64;
constexpr int kDecodeSmallBoxKeys = 16;  // second TMA box for tiles with few visible keys
constexpr int kDecodeConsumerWarps = 4;
constexpr int kDecodeConsumerThreads = kDecodeConsumerWarps * 32;
constexpr int kDecodeThreads = kDecodeConsumerThreads + 32;  // + the producer warp
constexpr int kDecodeMinTilesPerBlock = 4;                   // do not cut the list finer than 256 keys
constexpr int kDecodeWarpScanMaxB = 1024;                    // batches up to this size: warp-local scan

template <int D, int NH>
struct DecodeSmem {
    static constexpr int kPanels = D / 64;
    static constexpr int kPanelBytes = kDecodeTileKeys * 128;       // [64 keys][64 ch] bf16
    static constexpr int kTileBytes = kPanels * kPanelBytes;        // one K or V tile
    static constexpr int kStageBytes = 2 * kTileBytes;              // K then V
    static constexpr int kHC = 8 * NH;
    static constexpr int kMergeBytes = kDecodeConsumerWarps * kHC * (D + 1 + 2) * 4;  // O, max, sum per warp
    static constexpr int kStages = (220 * 1024 - kMergeBytes) / kStageBytes < 12 ? (220 * 1024 - kMergeBytes) / kStageBytes : 12;
    static constexpr int kOffMerge = kStages * kStageBytes;
    static constexpr int kOffBar = kOffMerge + ((kMergeBytes + 15) / 16) * 16;
    static constexpr int kOffMisc = kOffBar + 3 * kStages * 8;
    static constexpr int kBytes = kOffMisc + 64;
    static constexpr int kDynamicBytes = kBytes + 1024;  // room to align the base to 1024 B
};

// Visible part of one sequence's cache, in tiles, as row ranges of the buffer the kernel reads.
struct SeqGeom {
    int len;  // valid entries (0 when seqlens[b] is out of range)
    int sb;   // first sink row (0 unless the buffer is a shard that starts inside the sinks)
    int se;   // end of the sink rows that lie before the window
    int nst;  // sink tiles
    int nt;   // tiles per item
    int wb;   // first window row
    int we;   // end of the window rows (the sequence's last valid entry + 1)
    int w0;   // first row of the first window tile: wb (dense cache), or wb rounded down to a tile (paged cache)
};

// With `aligned` the window tiles start on multiples of the tile size, so that no tile straddles a page of
// a paged cache; the keys before the window in the first window tile are then masked like those past the end.
__host__ __device__ inline SeqGeom decode_seq_geom(int len, int Lmax, int window, int n_sink, int is_full,
                                                   bool aligned = false) {
    SeqGeom s;
    if (len < 1 || len > Lmax) {
        s.len = s.sb = s.se = s.nst = s.nt = s.wb = s.we = s.w0 = 0;
        return s;
    }
    s.len = len;
    s.wb = is_full ? 0 : (len > window ? len - window : 0);
    s.we = len;
    s.sb = 0;
    s.se = is_full ? 0 : (n_sink < s.wb ? n_sink : s.wb);
    s.nst = (s.se + kDecodeTileKeys - 1) / kDecodeTileKeys;
    s.w0 = aligned ? s.wb / kDecodeTileKeys * kDecodeTileKeys : s.wb;
    s.nt = s.nst + (len - s.w0 + kDecodeTileKeys - 1) / kDecodeTileKeys;
    return s;
}

// The same for a shard that holds positions [pos0, pos0 + rows) of a sequence of `len` tokens in total: the visible
// positions (sinks before the window, then the window ending at the query at len - 1) cut to what the shard holds
// and moved to its row numbers.  A shard may hold no visible key at all (nt == 0 with len >= 1).
__host__ __device__ inline SeqGeom decode_shard_geom(int len, int rows, int pos0, int window, int n_sink, int is_full) {
    SeqGeom s;
    s.len = s.sb = s.se = s.nst = s.nt = s.wb = s.we = s.w0 = 0;
    if (len < 1) return s;
    s.len = len;
    const long long end = (long long)pos0 + rows;  // first position past the shard
    const int lo = is_full ? 0 : (len > window ? len - window : 0);
    const int ns = is_full ? 0 : (n_sink < lo ? n_sink : lo);
    const long long sb = pos0 < ns ? pos0 : ns, se = end < ns ? end : ns;          // sinks in [pos0, end)
    const long long wb = lo > pos0 ? lo : pos0, we = end < len ? end : len;        // window in [pos0, end)
    if (se > sb) {
        s.sb = (int)(sb - pos0);
        s.se = (int)(se - pos0);
    }
    if (we > wb) {
        s.wb = (int)(wb - pos0);
        s.we = (int)(we - pos0);
    }
    s.w0 = s.wb;
    s.nst = (s.se - s.sb + kDecodeTileKeys - 1) / kDecodeTileKeys;
    s.nt = s.nst + (s.we - s.w0 + kDecodeTileKeys - 1) / kDecodeTileKeys;
    return s;
}

// Position in the global tile list; every role of a block walks the same positions.
template <bool kPaged, bool kShard>
struct DecodeWalker {
    int b, hv, ti;
    SeqGeom s;
    static __device__ __forceinline__ SeqGeom geom(const DecodeParams& p, int b) {
        if (kShard) return decode_shard_geom(__ldg(p.seqlens + b), p.Lmax, p.pos0, p.window, p.n_sink, p.is_full);
        return decode_seq_geom(__ldg(p.seqlens + b), p.Lmax, p.window, p.n_sink, p.is_full, kPaged);
    }
    __device__ __forceinline__ void seek(const DecodeParams& p, int b0, long long off) {
        b = b0;
        s = geom(p, b);
        hv = (int)(off / s.nt);
        ti = (int)(off - (long long)hv * s.nt);
    }
    __device__ __forceinline__ void next(const DecodeParams& p) {
        if (++ti < s.nt) return;
        ti = 0;
        if (++hv < p.IPB) return;
        hv = 0;
        while (++b < p.B) {
            s = geom(p, b);
            if (s.nt > 0) return;
        }
        s.nt = 0;  // past the last sequence
    }
    __device__ __forceinline__ int key0() const {
        return ti < s.nst ? s.sb + ti * kDecodeTileKeys : s.w0 + (ti - s.nst) * kDecodeTileKeys;
    }
    // rows [vbegin, vend) of this tile hold visible keys; vbegin > 0 only in the first window tile of a paged cache
    __device__ __forceinline__ int vend() const {
        const int left = (ti < s.nst ? s.se : s.we) - key0();
        return left < kDecodeTileKeys ? left : kDecodeTileKeys;
    }
    __device__ __forceinline__ int vbegin() const { return (kPaged && ti == s.nst) ? s.wb - s.w0 : 0; }
};

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

__device__ __forceinline__ void consumer_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(kDecodeConsumerThreads) : "memory");
}

template <int D, int NH, bool kPaged, bool kShard = false>
__global__ void __launch_bounds__(kDecodeThreads, 1)
decode_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
              const __grid_constant__ CUtensorMap tm_k16, const __grid_constant__ CUtensorMap tm_v16, const DecodeParams p) {
    static_assert(D == 64 || D == 128, "head size");
    using L = DecodeSmem<D, NH>;
    constexpr int ST = L::kStages;
    constexpr int NKK = D / 16;  // 16-channel steps of the first product = 16-channel row blocks of O^T
    constexpr int HC = L::kHC;   // query heads per chunk

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    float* sm_o = reinterpret_cast<float*>(smem_gen + L::kOffMerge);   // [warps][HC][D + 1]
    float* sm_m = sm_o + kDecodeConsumerWarps * HC * (D + 1);          // [warps][HC]
    float* sm_l = sm_m + kDecodeConsumerWarps * HC;                    // [warps][HC]
    const uint32_t bars = smem_base + L::kOffBar;
    auto bar_kf = [&](int s) -> uint32_t { return bars + 8u * (uint32_t)s; };
    auto bar_vf = [&](int s) -> uint32_t { return bars + 8u * (uint32_t)(ST + s); };
    auto bar_e = [&](int s) -> uint32_t { return bars + 8u * (uint32_t)(2 * ST + s); };
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + L::kOffMisc);
    volatile int* sm_last = abort_flag + 1;

    __shared__ long long sc_scan[kDecodeThreads];
    __shared__ long long sc_off;
    __shared__ int sc_b0;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ncta = (int)gridDim.x, cta = (int)blockIdx.x;

    if (tid == 0) {
        *abort_flag = 0;
        *sm_last = 0;
        for (int s = 0; s < ST; ++s) {
            mbar_init(bar_kf(s), 1u);
            mbar_init(bar_vf(s), 1u);
            mbar_init(bar_e(s), (uint32_t)kDecodeConsumerWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid == kDecodeConsumerThreads) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_v)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k16)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_v16)) : "memory");
    }

    // ---- where does this block's run of the global tile list start?  (scan of tiles per sequence)
    auto tiles_of = [&](int b) -> long long { return (long long)DecodeWalker<kPaged, kShard>::geom(p, b).nt * p.IPB; };
    // A sequence without tiles.  Dense / paged cache: its length is out of range; report it and zero its output
    // rows.  Shard: also what a shard that holds none of the sequence's visible keys looks like; its rows get the
    // empty partial (-inf, 0, 0...), and only a length < 1 is an error.  One block does the stores.
    auto zero_fill_bad = [&](int b) {
        if (!kShard || __ldg(p.seqlens + b) < 1) record_device_error(SWAA_ERR_BAD_SEQLENS);
        if (b % ncta == cta) {
            if (kShard) {
                float* o = p.part_out + (size_t)b * p.Hq * (D + 2);
                for (int i = 0; i < p.Hq * (D + 2); ++i) o[i] = (i % (D + 2) == 0) ? -INFINITY : 0.f;
            } else {
                uint4* o = reinterpret_cast<uint4*>(p.out + (size_t)b * p.Hq * D);
                for (int i = 0; i < p.Hq * D / 8; ++i) o[i] = make_uint4(0, 0, 0, 0);
            }
        }
    };
    long long total, tpc, t0, t1, off0 = 0;
    int b0 = 0;
    if (p.B <= kDecodeWarpScanMaxB) {
        // small batch: every warp scans all sequences by itself with shuffles, no block-level exchange
        total = 0;
        for (int base = 0; base < p.B; base += 32) {
            const int b = base + lane;
            long long nb = 0;
            if (b < p.B) {
                nb = tiles_of(b);
                if (nb == 0 && warp == 0) zero_fill_bad(b);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) nb += __shfl_xor_sync(0xffffffffu, nb, o);
            total += nb;
        }
        tpc = (total + ncta - 1) / ncta;
        if (tpc < kDecodeMinTilesPerBlock) tpc = kDecodeMinTilesPerBlock;
        t0 = (long long)cta * tpc;
        t1 = total < t0 + tpc ? total : t0 + tpc;
        if (t0 < t1) {
            long long run = 0;
            for (int base = 0; base < p.B; base += 32) {
                const int b = base + lane;
                const long long nb = b < p.B ? tiles_of(b) : 0;
                long long incl = nb;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const long long v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                const bool here = run + incl - nb <= t0 && t0 < run + incl;
                const unsigned hit = __ballot_sync(0xffffffffu, here);
                if (hit) {
                    const int src = __ffs(hit) - 1;
                    b0 = base + src;
                    off0 = t0 - (run + __shfl_sync(0xffffffffu, incl - nb, src));
                    break;
                }
                run += __shfl_sync(0xffffffffu, incl, 31);
            }
        }
        __syncthreads();  // barrier initialisation
    } else {
        const int chunk = (p.B + kDecodeThreads - 1) / kDecodeThreads;
        const int bb = min(p.B, tid * chunk), be = min(p.B, bb + chunk);
        long long mine = 0;
        for (int b = bb; b < be; ++b) {
            const long long nb = tiles_of(b);
            if (nb == 0) zero_fill_bad(b);
            mine += nb;
        }
        sc_scan[tid] = mine;
        __syncthreads();
        for (int off = 1; off < kDecodeThreads; off <<= 1) {
            const long long v = tid >= off ? sc_scan[tid - off] : 0;
            __syncthreads();
            sc_scan[tid] += v;
            __syncthreads();
        }
        total = sc_scan[kDecodeThreads - 1];
        tpc = (total + ncta - 1) / ncta;
        if (tpc < kDecodeMinTilesPerBlock) tpc = kDecodeMinTilesPerBlock;
        t0 = (long long)cta * tpc;
        t1 = total < t0 + tpc ? total : t0 + tpc;
        if (t0 < t1 && sc_scan[tid] - mine <= t0 && t0 < sc_scan[tid]) {
            long long acc = sc_scan[tid] - mine;
            for (int b = bb; b < be; ++b) {
                const long long nb = tiles_of(b);
                if (t0 < acc + nb) {
                    sc_b0 = b;
                    sc_off = t0 - acc;
                    break;
                }
                acc += nb;
            }
        }
        __syncthreads();
        b0 = sc_b0;
        off0 = sc_off;
    }
    if (t0 >= t1) return;  // nothing for this block (uniform; nobody waits on a barrier)
    const int cnt = (int)(t1 - t0);  // tpc <= tiles of the whole problem / blocks, far below 2^31 in practice

    if (warp == kDecodeConsumerWarps) {
        // =========================================================================== TMA producer
        if (lane == 0) {
            DecodeWalker<kPaged, kShard> w;
            w.seek(p, b0, off0);
            bool ok = true;
            int n = 0, s = 0;
            uint32_t ph = 0;
            for (; n < cnt; ++n, w.next(p)) {
                ok = mbar_wait(bar_e(s), ph ^ 1u, abort_flag);
                if (!ok) break;
                const int key0 = w.key0(), hk = w.hv / p.HG;
                int c2 = key0, c3 = w.b;  // TMA coordinates: (entry, sequence) or (row in page, page)
                if (kPaged) {
                    const int tile = key0 / kDecodeTileKeys;
                    c3 = __ldg(p.block_table + (size_t)w.b * p.max_blocks + tile / p.page_tiles);
                    c2 = (tile % p.page_tiles) * kDecodeTileKeys;
                    if (c3 < 0 || c3 >= p.num_pages) {
                        record_device_error(SWAA_ERR_BAD_SEQLENS);
                        c3 = p.num_pages;  // out of range: the copy delivers zeros
                    }
                }
                const uint32_t dst = smem_base + (uint32_t)s * L::kStageBytes;
                // a tile with at most 16 visible keys (typically the sinks) is fetched with the 16-row box
                const bool small = w.vend() <= kDecodeSmallBoxKeys;
                const CUtensorMap* mk = small ? &tm_k16 : &tm_k;
                const CUtensorMap* mv = small ? &tm_v16 : &tm_v;
                const uint32_t bytes = small ? (uint32_t)(L::kPanels * kDecodeSmallBoxKeys * 128) : (uint32_t)L::kTileBytes;
                mbar_arrive_expect_tx(bar_kf(s), bytes);
#pragma unroll
                for (int pn = 0; pn < L::kPanels; ++pn)
                    tma_load_4d(dst + pn * L::kPanelBytes, mk, pn * 64, hk, c2, c3, bar_kf(s));
                mbar_arrive_expect_tx(bar_vf(s), bytes);
#pragma unroll
                for (int pn = 0; pn < L::kPanels; ++pn)
                    tma_load_4d(dst + L::kTileBytes + pn * L::kPanelBytes, mv, pn * 64, hk, c2, c3, bar_vf(s));
                if (++s == ST) {
                    s = 0;
                    ph ^= 1u;
                }
            }
            if (!ok) {
                // give the copies in flight a bounded chance to land before the block's memory is released
                const uint64_t tw = global_timer_ns();
                bool landed = false;
                while (!landed && global_timer_ns() - tw < kWaitLimitNs) {
                    landed = true;
                    for (int m = max(0, n - ST); m < n; ++m) {
                        landed = landed && mbar_try_wait(bar_kf(m % ST), (uint32_t)(m / ST) & 1u);
                        landed = landed && mbar_try_wait(bar_vf(m % ST), (uint32_t)(m / ST) & 1u);
                    }
                }
            }
        }
        return;
    }

    // ============================================================================== consumers
    const int g = lane >> 2, c = lane & 3;
    // ldmatrix row addresses inside a tile (byte offset of the row, and the row's swizzle key)
    const int krow = 16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1);  // K: matrices (keys lo/hi) x (channels lo/hi)
    const int kchk = lane >> 4;
    const int vrow = 16 * warp + (lane & 7) + 8 * (lane >> 4);        // V: matrices (channels lo/hi) x (keys lo/hi)
    const int vchk = (lane >> 3) & 1;

    DecodeWalker<kPaged, kShard> w;
    w.seek(p, b0, off0);
    bool ok = true;
    bool first_seg = true;
    int n = 0, s = 0;
    uint32_t ph = 0;
    while (n < cnt) {
        // ---- one segment: the tiles of the current item that belong to this block
        const int b = w.b, hv = w.hv, ti_begin = w.ti, nt = w.s.nt;
        const int seg_tiles = min(cnt - n, nt - ti_begin);
        const long long seg_t0 = t0 + n;
        const int hk = hv / p.HG, ch = hv - hk * p.HG;
        const int h0 = hk * p.G + ch * HC;      // first query head of this chunk
        const int gc = min(HC, p.G - ch * HC);  // heads in this chunk

        // Q^T fragments (B operand): lane (g, c) holds channels 16kk + 2c, +1 and 16kk + 2c + 8, +9 of head g
        uint32_t qf[NH][NKK][2];
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
            const int hh = nh * 8 + g;
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(p.q + ((size_t)b * p.Hq + h0 + (hh < gc ? hh : 0)) * D);
#pragma unroll
            for (int kk = 0; kk < NKK; ++kk) {
                qf[nh][kk][0] = hh < gc ? __ldg(qrow + kk * 8 + c) : 0u;
                qf[nh][kk][1] = hh < gc ? __ldg(qrow + kk * 8 + c + 4) : 0u;
            }
        }
        float m_run[NH][2], l_run[NH][2], oacc[NH][NKK][4];
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
            m_run[nh][0] = m_run[nh][1] = -INFINITY;
            l_run[nh][0] = l_run[nh][1] = 0.f;
#pragma unroll
            for (int qb = 0; qb < NKK; ++qb)
#pragma unroll
                for (int r = 0; r < 4; ++r) oacc[nh][qb][r] = 0.f;
        }

        for (int j = 0; j < seg_tiles; ++j, ++n, w.next(p)) {
            const int vw = w.vend() - 16 * warp;            // this warp's keys [vb, vw) of its 16 are visible
            const int vb = kPaged ? max(w.vbegin() - 16 * warp, 0) : 0;
            const uint32_t stage = smem_base + (uint32_t)s * L::kStageBytes;
            // warp-wide decisions after a bounded wait: ldmatrix, mma.sync and the shuffles need all 32 lanes
            ok = __all_sync(0xffffffffu, ok && mbar_wait(bar_kf(s), ph, abort_flag));
            if (ok && min(vw, 16) > vb) {  // some of this warp's 16 keys are visible
                // ---- S^T = K Q^T : rows = keys (g, g+8), cols = heads (2c, 2c+1)
                float sacc[NH][4];
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) sacc[nh][0] = sacc[nh][1] = sacc[nh][2] = sacc[nh][3] = 0.f;
#pragma unroll
                for (int kk = 0; kk < NKK; ++kk) {
                    const int chunk16 = 2 * kk + kchk;
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4(stage + (uint32_t)((chunk16 >> 3) * L::kPanelBytes + krow * 128 +
                                                   (((chunk16 & 7) ^ (krow & 7)) << 4)),
                                a0, a1, a2, a3);
#pragma unroll
                    for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(sacc[nh], a0, a1, a2, a3, qf[nh][kk][0], qf[nh][kk][1]);
                }

                // ---- online softmax over this warp's 16 keys
                const bool ok0 = g < vw && g >= vb, ok1 = g + 8 < vw && g + 8 >= vb;
                uint32_t pb[NH][2];
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) {
                    float alpha[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float s0 = ok0 ? sacc[nh][e] : -INFINITY;
                        const float s1 = ok1 ? sacc[nh][2 + e] : -INFINITY;
                        float bm = fmaxf(s0, s1);
                        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 4));
                        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 8));
                        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));
                        const float m_new = fmaxf(m_run[nh][e], bm);  // finite: one of the warp's keys is visible
                        alpha[e] = ex2f((m_run[nh][e] - m_new) * p.sl2);
                        m_run[nh][e] = m_new;
                        const float off = m_new * p.sl2;
                        const float p0 = ex2f(fmaf(s0, p.sl2, -off));
                        const float p1 = ex2f(fmaf(s1, p.sl2, -off));
                        l_run[nh][e] = l_run[nh][e] * alpha[e] + p0 + p1;
                        sacc[nh][e] = p0;
                        sacc[nh][2 + e] = p1;
                    }
                    if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
                        for (int qb = 0; qb < NKK; ++qb) {
                            oacc[nh][qb][0] *= alpha[0];
                            oacc[nh][qb][1] *= alpha[1];
                            oacc[nh][qb][2] *= alpha[0];
                            oacc[nh][qb][3] *= alpha[1];
                        }
                    }
                    // P^T as the B fragment: (keys 2c, 2c+1 | 2c+8, 2c+9 ; head g)
                    pb[nh][0] = movmatrix_trans(pack_bf16x2(sacc[nh][0], sacc[nh][1]));
                    pb[nh][1] = movmatrix_trans(pack_bf16x2(sacc[nh][2], sacc[nh][3]));
                }

                // ---- O^T += V^T P^T : rows = channels (16qb + g, 16qb + g + 8), cols = heads (2c, 2c+1)
                ok = __all_sync(0xffffffffu, mbar_wait(bar_vf(s), ph, abort_flag));
                if (ok) {
                    // rows of the tile past the last visible key may hold anything (also NaN): clear them
                    auto vis = [&](int key) { return key < vw && key >= vb; };
                    const uint32_t mlo = (vis(2 * c) ? 0x0000ffffu : 0u) | (vis(2 * c + 1) ? 0xffff0000u : 0u);
                    const uint32_t mhi = (vis(2 * c + 8) ? 0x0000ffffu : 0u) | (vis(2 * c + 9) ? 0xffff0000u : 0u);
#pragma unroll
                    for (int qb = 0; qb < NKK; ++qb) {
                        const int chunk16 = 2 * qb + vchk;
                        uint32_t a0, a1, a2, a3;
                        ldmatrix_x4_trans(stage + (uint32_t)(L::kTileBytes + (chunk16 >> 3) * L::kPanelBytes + vrow * 128 +
                                                             (((chunk16 & 7) ^ (vrow & 7)) << 4)),
                                          a0, a1, a2, a3);
                        if (vw < 16 || vb > 0) {
                            a0 &= mlo;
                            a1 &= mlo;
                            a2 &= mhi;
                            a3 &= mhi;
                        }
#pragma unroll
                        for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(oacc[nh][qb], a0, a1, a2, a3, pb[nh][0], pb[nh][1]);
                    }
                }
            } else {
                ok = __all_sync(0xffffffffu, ok && mbar_wait(bar_vf(s), ph, abort_flag));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_e(s));
            if (++s == ST) {
                s = 0;
                ph ^= 1u;
            }
        }

        // ---- merge the four warps of the block through shared memory
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float l = l_run[nh][e];
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                l += __shfl_xor_sync(0xffffffffu, l, 8);
                l += __shfl_xor_sync(0xffffffffu, l, 16);
                const int hh = nh * 8 + 2 * c + e;
                if (g == 0) {
                    sm_m[warp * HC + hh] = m_run[nh][e];
                    sm_l[warp * HC + hh] = l;
                }
                float* orow = sm_o + (size_t)(warp * HC + hh) * (D + 1);
#pragma unroll
                for (int qb = 0; qb < NKK; ++qb) {
                    orow[16 * qb + g] = oacc[nh][qb][e];
                    orow[16 * qb + g + 8] = oacc[nh][qb][2 + e];
                }
            }
        }
        consumer_sync();

        const bool complete = ti_begin == 0 && seg_tiles == nt;
        const int slot = 2 * cta + (first_seg ? 0 : 1);
        float* my_part = p.part + (size_t)slot * HC * (D + 2);
        for (int idx = tid; idx < gc * D; idx += kDecodeConsumerThreads) {
            const int hh = idx / D, d = idx - hh * D;
            float M = -INFINITY;
#pragma unroll
            for (int wi = 0; wi < kDecodeConsumerWarps; ++wi) M = fmaxf(M, sm_m[wi * HC + hh]);
            float den = 0.f, num = 0.f;
#pragma unroll
            for (int wi = 0; wi < kDecodeConsumerWarps; ++wi) {
                const float mw = sm_m[wi * HC + hh];
                const float wgt = mw == -INFINITY ? 0.f : ex2f((mw - M) * p.sl2);
                den += wgt * sm_l[wi * HC + hh];
                num += wgt * sm_o[(size_t)(wi * HC + hh) * (D + 1) + d];
            }
            if (!ok) continue;
            if (complete) {
                if (kShard) {  // the row's result leaves as a partial: (max in natural-log units, sum, unnormalised O)
                    float* po = p.part_out + ((size_t)b * p.Hq + h0 + hh) * (D + 2);
                    po[2 + d] = num;
                    if (d == 0) {
                        po[0] = M * p.scale;
                        po[1] = den;
                    }
                } else {
                    p.out[((size_t)b * p.Hq + h0 + hh) * D + d] = __float2bfloat16_rn(den > 0.f ? num / den : 0.f);
                }
            } else {
                my_part[hh * (D + 2) + 2 + d] = num;
                if (d == 0) {
                    my_part[hh * (D + 2) + 0] = M;
                    my_part[hh * (D + 2) + 1] = den;
                }
            }
        }
        if (!complete) {
            // ---- the last block of this item to arrive merges the item's partials
            const long long T0 = seg_t0 - ti_begin, T1 = T0 + nt;
            const int c_first = (int)(T0 / tpc), c_last = (int)((T1 - 1) / tpc);
            const int n_parts = c_last - c_first + 1;
            __threadfence();  // this block's partial is visible before its ticket
            consumer_sync();
            if (tid == 0) {
                // A ticket whose stamp is not this call's is left over from an earlier call (or was never
                // written): the first block to arrive restarts it, so the workspace needs no clearing.
                unsigned long long* t = p.tickets + c_first;
                if (n_parts == 2) {
                    // two blocks share the item (the common case): one exchange tells who came second
                    const unsigned long long mine = (p.stamp << 16) | 1ull;
                    *sm_last = atomicExch(t, mine) == mine ? 1 : 0;
                } else {
                    unsigned long long seen = *reinterpret_cast<volatile unsigned long long*>(t), want;
                    for (;;) {
                        want = (seen >> 16) == p.stamp ? seen + 1ull : ((p.stamp << 16) | 1ull);
                        const unsigned long long prev = atomicCAS(t, seen, want);
                        if (prev == seen) break;
                        seen = prev;
                    }
                    *sm_last = ((int)(want & 0xffffull) == n_parts) ? 1 : 0;
                }
            }
            consumer_sync();
            if (*sm_last && ok) {
                __threadfence();
                const bool first_is_slot1 = (long long)c_first * tpc != T0;
                auto slot_of = [&](int cc) { return 2 * cc + ((cc == c_first && first_is_slot1) ? 1 : 0); };
                for (int idx = tid; idx < gc * D; idx += kDecodeConsumerThreads) {
                    const int hh = idx / D, d = idx - hh * D;
                    float M = -INFINITY, den = 0.f, num = 0.f;
                    if (n_parts <= 4) {
                        // few parts: every load is issued before the first is needed (one round trip to L2)
                        float ms[4], ls[4], os[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            ms[i] = -INFINITY;
                            ls[i] = os[i] = 0.f;
                            if (i < n_parts) {
                                const float* pp = p.part + ((size_t)slot_of(c_first + i) * HC + hh) * (D + 2);
                                ms[i] = __ldcg(pp);
                                ls[i] = __ldcg(pp + 1);
                                os[i] = __ldcg(pp + 2 + d);
                            }
                        }
                        M = fmaxf(fmaxf(ms[0], ms[1]), fmaxf(ms[2], ms[3]));
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float wgt = ms[i] == -INFINITY ? 0.f : ex2f((ms[i] - M) * p.sl2);
                            den += wgt * ls[i];
                            num += wgt * os[i];
                        }
                    } else {
                        // many parts (a long item of a small batch): eight partials per round trip to L2, merged
                        // into a running (max, sum, O) -- loads one by one would cost a round trip each
                        for (int c0 = c_first; c0 <= c_last; c0 += 8) {
                            float ms[8], ls[8], os[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                ms[i] = -INFINITY;
                                ls[i] = os[i] = 0.f;
                                if (c0 + i <= c_last) {
                                    const float* pp = p.part + ((size_t)slot_of(c0 + i) * HC + hh) * (D + 2);
                                    ms[i] = __ldcg(pp);
                                    ls[i] = __ldcg(pp + 1);
                                    os[i] = __ldcg(pp + 2 + d);
                                }
                            }
                            float Mn = M;
#pragma unroll
                            for (int i = 0; i < 8; ++i) Mn = fmaxf(Mn, ms[i]);
                            const float keep = M == -INFINITY ? 0.f : ex2f((M - Mn) * p.sl2);
                            den *= keep;
                            num *= keep;
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const float wgt = ms[i] == -INFINITY ? 0.f : ex2f((ms[i] - Mn) * p.sl2);
                                den += wgt * ls[i];
                                num += wgt * os[i];
                            }
                            M = Mn;
                        }
                    }
                    if (kShard) {
                        float* po = p.part_out + ((size_t)b * p.Hq + h0 + hh) * (D + 2);
                        po[2 + d] = num;
                        if (d == 0) {
                            po[0] = M * p.scale;
                            po[1] = den;
                        }
                    } else {
                        p.out[((size_t)b * p.Hq + h0 + hh) * D + d] = __float2bfloat16_rn(den > 0.f ? num / den : 0.f);
                    }
                }
            }
        }
        consumer_sync();  // the merge buffers are free for the next segment
        first_seg = false;
    }
}

// Log-sum-exp combine of P partial results per (sequence, head) row: one warp per row, lanes over the channels.
// part [P][rows][D + 2] = (max in natural-log units, sum, unnormalised O); empty partials (sum == 0) are skipped; a
// row without any non-empty partial gives zeros.
template <int D>
__global__ void decode_combine_kernel(const float* __restrict__ part, int P, int rows, __nv_bfloat16* __restrict__ out) {
    const int row = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (row >= rows) return;
    float M = -INFINITY;
    for (int s = 0; s < P; ++s) {
        const float* pr = part + ((size_t)s * rows + row) * (D + 2);
        if (pr[1] > 0.f) M = fmaxf(M, pr[0]);
    }
    float den = 0.f, acc[D / 32];
#pragma unroll
    for (int c = 0; c < D / 32; ++c) acc[c] = 0.f;
    for (int s = 0; s < P; ++s) {
        const float* pr = part + ((size_t)s * rows + row) * (D + 2);
        if (!(pr[1] > 0.f)) continue;
        const float w = __expf(pr[0] - M);
        den += w * pr[1];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) acc[c] += w * pr[2 + c * 32 + lane];
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) out[(size_t)row * D + c * 32 + lane] = __float2bfloat16_rn(acc[c] * inv);
}

}  // namespace swaa
