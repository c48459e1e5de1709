// Prefill attention for sm_100a: tcgen05 MMAs accumulating in tensor memory, TMA-staged operands,
// online softmax with one thread per query row.
//
// Mask policy (Sec. 1, 3.1.2, 3.2.1; App. A): a query at position i of its sequence sees key j iff
//     j <= i  and  ( is_full  or  j > i - window  or  j < n_sink ).
// Only the key tiles that hold a visible key are visited (the sink tiles and the diagonal band), so
// the work is O(L * window) as App. A states; the element predicate is evaluated only on tiles that
// are not entirely visible.
//
// One thread block processes one 128-row query tile for TWO query heads of the same GQA group
// ("sides" A and B).  Both sides need exactly the same K/V tiles and the same masks, so each K/V tile
// is staged in shared memory once and feeds four MMAs.  Roles:
//   warps 0-3   softmax of side A   (thread = query row; lane quadrant = TMEM lane quadrant)
//   warps 4-7   softmax of side B
//   warp  8     TMA producer (one elected lane): Q tiles once, then the K and V tile rings
//   warp  9     MMA issuer (one elected lane) and TMEM allocation
// Tensor memory (512 columns x 128 lanes of 32 bit): S_A | S_B | O_A | O_B.  The bf16 probabilities
// P overwrite the first 64 columns of their own S and are consumed from TMEM as the A operand of
// O += P V.  V tiles are used as the MN-major B operand exactly as TMA lands them.
// Per key tile n the issuer runs  PV_A(n) QK_A(n+1) PV_B(n) QK_B(n+1), so the softmax of one side
// overlaps the MMAs of the other; P arrives in two parts (keys 0..95, then 96..127) and the first six of the
// eight P V instructions are issued on the first.  The running maximum is only raised (and O rescaled) when it grows
// by more than 2^8; the final division by the row sum makes the result independent of that choice.
//
// Every wait is bounded: a wait that runs out records SWAA_ERR_TIMEOUT, all roles leave their loops,
// the block waits (bounded) for its outstanding copies, frees its tensor memory and returns.
#pragma once

#include <cuda.h>

#include "swaa_internal.cuh"
#include "swaa_ptx.cuh"

namespace swaa {

constexpr int kPrefillBM = 128;
constexpr int kPrefillBN = 128;
constexpr int kPrefillThreads = 384;  // 8 softmax warps + 4 auxiliary warps (producer, issuer, 2 idle)
constexpr float kRescaleThreshold = 8.0f;                   // log2 units

struct PrefillParams {
    __nv_bfloat16* out;
    float* lse;             // nullable, [Hq, T]
    const int32_t* cu_seqlens;    // queries (and keys, when cu_seqlens_k is null)
    const int32_t* cu_seqlens_k;  // nullable: keys of a chunked prefill, len_k >= len_q per sequence
    int B, T, max_seqlen, Hq, Hkv, G;
    int Tk, max_seqlen_k;         // packed key tokens and longest key sequence (chunked prefill only)
    // paged keys/values (kMode 2): cu_seqlens_k holds the key LENGTHS [B]; entry j of sequence b lives in page
    // block_table[b * max_blocks + j / page_size] at row j % page_size
    const int32_t* block_table;
    int max_blocks, page_size, num_pages;
    int pairs_per_kv;       // ceil(G / 2)
    int n_pairs;            // Hkv * pairs_per_kv
    int tiles_ub;           // upper bound on the number of query tiles over all sequences
    int window, n_sink, is_full;
    const uint8_t* is_full_seq;   // nullable (chunked / paged): mask policy per sequence, replaces is_full
    // context-parallel prefill (kMode 3): the local keys of sequence b start at position key_pos0[b]; the keys at
    // positions 0 .. sink_rows-1 of every sequence come from a separate buffer [B, sink_rows, Hkv, D]
    const int32_t* key_pos0;
    int sink_rows;
    float sl2;              // softmax scale * log2(e)
    float scale;
};

// ------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The same with the shared-memory descriptors given as (low word, shared high word): the low word holds
// the start address and the leading-dimension offset, so stepping through a tile is one 32-bit add per operand.
__device__ __forceinline__ void mma_ss_lh(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_ts_lh(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Packed pairs of fp32 in one 64-bit register (two lanes per FMA/ADD instruction on sm_100).
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// 2^x for a pair of arguments on the FMA and integer pipes instead of the special-function unit:
// x = n + f with n = round(x), f in [-1/2, 1/2]; 2^f by a cubic with constant term exactly 1 (minimax fit of
// the other three coefficients: relative error 1.0e-4, far below the bf16 rounding of P), so that 2^0 = 1
// exactly as on the special-function unit and a row of equal scores sums to its key count; n is added into
// the exponent field.  The argument is first raised to -127, where the result is exactly 0 (f = 0, the cubic gives
// 1.0 and the exponent field cancels), so masked scores (-inf) and anything below 2^-127 give exact zeros as
// ex2.approx.ftz does, at the price of one max per element instead of a compare and a select.
__device__ __forceinline__ void exp2_poly_x2(float x0, float x1, float& r0, float& r1) {
    const float kMagic = 12582912.f;  // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
    x0 = fmaxf(x0, -127.f);
    x1 = fmaxf(x1, -127.f);
    const uint64_t xx = pack_f32x2(x0, x1);
    uint64_t t, fl, f, q;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(t) : "l"(xx), "l"(pack_f32x2(kMagic, kMagic)));
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(fl) : "l"(t), "l"(pack_f32x2(kMagic, kMagic)));
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(f) : "l"(xx), "l"(fl));
    q = fma_f32x2(f, pack_f32x2(0.055009059607982635f, 0.055009059607982635f),
                  pack_f32x2(0.2422109693288803f, 0.2422109693288803f));
    q = fma_f32x2(q, f, pack_f32x2(0.6932829022407532f, 0.6932829022407532f));
    q = fma_f32x2(q, f, pack_f32x2(1.0f, 1.0f));
    float t0, t1, q0, q1;
    unpack_f32x2(t, t0, t1);
    unpack_f32x2(q, q0, q1);
    r0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
    r1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}

// Bit c (0..15) set: column pair c of every 32-column chunk of a score tile takes the polynomial path: a quarter
// of the exponentials (measured best among 1/8, 3/16, 1/4, 5/16, 1/2, 3/4 and several placements).
constexpr uint32_t kPolyPairMask = 0x8888u;

#define SWAA_R8(r, o) "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), "=r"(r[o + 7])
#define SWAA_I8(r, o) "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]), "r"(r[o + 7])

// 32 lanes x 32 consecutive columns: thread `lane` of the warp receives columns c .. c+31 of TMEM
// lane (quadrant base + lane).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
        "%29,%30,%31}, [%32];"
        : SWAA_R8(r, 0), SWAA_R8(r, 8), SWAA_R8(r, 16), SWAA_R8(r, 24)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
        "%29,%30,%31};" ::SWAA_I8(r, 0),
        SWAA_I8(r, 8), SWAA_I8(r, 16), SWAA_I8(r, 24), "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};" ::
            SWAA_I8(r, 0),
        SWAA_I8(r, 8), "r"(taddr)
        : "memory");
}

// Shared-memory matrix descriptors for tiles stored as 128-byte rows with the 128-byte swizzle (what
// TMA writes for a [rows][64 bf16] box).  14-bit fields hold byte values >> 4.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of this architecture
    d |= (uint64_t)2 << 61;  // 128-byte swizzle
    return d;
}

// kind::f16 instruction descriptor: bf16 x bf16 -> f32, M x N, A K-major, B K- or MN-major.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

template <int D>
struct PrefillSmem {
    static constexpr int kTileBytes = 128 * D * 2;  // one 128-row tile of Q, K or V
    static constexpr int kPanelBytes = 128 * 128;   // one [128 rows][64 ch] panel
    static constexpr int kPanels = D / 64;
    static constexpr int kStages = D == 128 ? 2 : 4;
    static constexpr int kOffQ = 0;                              // two tiles (sides A, B)
    static constexpr int kOffK = 2 * kTileBytes;                 // kStages tiles
    static constexpr int kOffV = kOffK + kStages * kTileBytes;   // kStages tiles
    static constexpr int kOffStage = kOffV + kStages * kTileBytes;  // 8 x 4 KiB: per-warp output staging
    static constexpr int kOffBar = kOffStage + 8 * 4096;
    // barriers: Q full/empty, K full/empty, V full/empty per stage, per side S-full / P-ready / O-done /
    // O-free, work-descriptor full/empty per slot, final, V-tile-cleared per stage (paged keys only)
    static constexpr int kNumBars = 2 + 4 * kStages + 8 + 4 + 1 + kStages + 2;
    static constexpr int kOffMisc = kOffBar + kNumBars * 8;      // tmem slot, abort flag, work descriptors
    static constexpr int kBytes = kOffMisc + 128;
    static constexpr int kDynamicBytes = kBytes + 1024;          // room to align the base to 1024 B
};

// One unit of work: a 128-row query tile of one sequence for one pair of query heads.
struct WorkItem {
    int valid, seq_start, seq_len, m_tile, pair;
    int k_start;  // first packed key token of the sequence (= seq_start for self attention; sequence index when paged)
    int k_off;    // index of the sequence's first query among its (local) keys: len_k - len_q (0 for self attention)
    int full;     // this item runs full causal attention (per sequence in a mixed batch)
    int n_sink;   // sink keys among the local keys (context-parallel: n_sink - key_pos0, clamped; else n_sink)
    int s_rem;    // context-parallel: sink keys that come from the separate sink buffer, min(n_sink, key_pos0)
    int b;        // context-parallel: sequence index (row of the sink buffer)
};

// kMode 0: self attention.  1: chunked prefill, the queries are the last len_q tokens of a longer key sequence
// (separate packing of the keys).  2: the same with keys and values in pages addressed through a block table.
// 3: context-parallel prefill, mode 1 with the local keys starting at position key_pos0[b] of their sequence and the
// sink keys before that position read from a separate buffer (tm_sk, tm_sv) as leading key tiles of the item.
// The self-attention instance compiles the offsets away.
// kLseOnly: only the log-sum-exp of every row is wanted (the lazy-ratio probe): no V tiles are fetched, no P V product
// is issued, P is not formed and nothing is written to `out`; the barrier protocol stays the same, with "P ready"
// meaning "S has been read" and the V-tile barriers completed by a plain arrival.
template <int D, int kMode, bool kLseOnly = false>
__global__ void __launch_bounds__(kPrefillThreads, 1)
prefill_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
               const __grid_constant__ CUtensorMap tm_sk, const __grid_constant__ CUtensorMap tm_sv,
               const PrefillParams p) {
    using L = PrefillSmem<D>;
    constexpr bool kChunked = kMode >= 1, kPaged = kMode == 2, kCp = kMode == 3;
    constexpr int BM = kPrefillBM, BN = kPrefillBN;
    constexpr int ST = L::kStages;
    constexpr uint32_t kIdescQK = make_idesc(BM, BN, 0);
    constexpr uint32_t kIdescPV = make_idesc(BM, D, 1);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base + L::kOffQ, sK = smem_base + L::kOffK, sV = smem_base + L::kOffV;
    const uint32_t sStage = smem_base + L::kOffStage;
    const uint32_t bars = smem_base + L::kOffBar;
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
    // barrier indices
    constexpr int BAR_QF = 0, BAR_QE = 1, BAR_KF = 2, BAR_KE = BAR_KF + ST, BAR_VF = BAR_KE + ST, BAR_VE = BAR_VF + ST;
    constexpr int BAR_SF = BAR_VE + ST, BAR_PR = BAR_SF + 2, BAR_OD = BAR_PR + 2, BAR_OF = BAR_OD + 2;
    constexpr int BAR_WF = BAR_OF + 2, BAR_WE = BAR_WF + 2, BAR_FIN = BAR_WE + 2;
    // paged only, one per ring stage: the rows of the V tile in that stage past the last key have been cleared.
    // Completed once per cleared tile; producer and issuer each keep the stage's phase bit.  The producer cannot
    // clear a stage twice before the issuer has waited for the first clear: reusing the stage needs the
    // issuer's V-empty commit, which follows that wait.
    constexpr int BAR_VC = BAR_FIN + 1;
    // per side: the last quarter of P (keys 96..127) has been written; BAR_PR then stands for the first three quarters
    constexpr int BAR_PQ = BAR_VC + ST;
    static_assert(BAR_PQ + 2 == L::kNumBars, "barrier count");
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + L::kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* work_ring = reinterpret_cast<volatile int*>(tmem_slot + 4);  // 2 slots x 12 ints

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool full_all = p.is_full != 0;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int i = 0; i < L::kNumBars; ++i) {
            uint32_t count = 1u;
            if (i == BAR_PR || i == BAR_PR + 1 || i == BAR_OF || i == BAR_OF + 1) count = 128u;  // softmax threads
            if (i == BAR_PQ || i == BAR_PQ + 1) count = 128u;
            if (i == BAR_WE || i == BAR_WE + 1) count = 10u;  // producer, issuer, one lane per softmax warp
            mbar_init(bar(i), count);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {  // TMEM: all 512 columns (S_A, S_B, O_A, O_B)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Consumers of the work ring: wait for descriptor `it`, copy it, release the slot.
    auto fetch_work = [&](int it, WorkItem& w, bool release) -> bool {
        const int slot = it & 1;
        if (!mbar_wait(bar(BAR_WF + slot), (uint32_t)(it >> 1) & 1u, abort_flag)) return false;
        volatile int* d = work_ring + slot * 12;
        w.valid = d[0];
        w.seq_start = d[1];
        w.seq_len = d[2];
        w.m_tile = d[3];
        w.pair = d[4];
        w.k_start = kChunked ? d[5] : w.seq_start;
        w.k_off = kChunked ? d[6] : 0;
        w.full = kChunked ? d[7] : (full_all ? 1 : 0);
        w.n_sink = kCp ? d[8] : p.n_sink;
        w.s_rem = kCp ? d[9] : 0;
        w.b = kCp ? d[10] : 0;
        if (release) mbar_arrive(bar(BAR_WE + slot));
        return true;
    };

    // Register budget per scheduler partition: two softmax warps at 216 + one auxiliary warp at 72.
    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
      if (warp == 10) {
        // ====================================================================== work scheduler
        // Walks this block's work items w = blockIdx.x, blockIdx.x + gridDim.x, ... and publishes their
        // descriptors.  Items are ordered heavy-first: last sequence first, last tile of a sequence first.
        if (lane == 0) {
            if (p.cu_seqlens[0] != 0 || p.cu_seqlens[p.B] != p.T) record_device_error(SWAA_ERR_BAD_SEQLENS);
            int b = p.B, acc = 0, cur_nt = 0, cur_s = 0, cur_len = 0, cur_ks = 0, cur_off = 0;
            int cur_full = full_all ? 1 : 0, cur_sink = p.n_sink, cur_srem = 0;
            auto next_seq = [&]() {
                acc += cur_nt;
                --b;
                cur_nt = 0;
                if (b >= 0) {
                    const int s0 = p.cu_seqlens[b], e0 = p.cu_seqlens[b + 1];
                    int len = e0 - s0;
                    if (len < 0 || len > p.max_seqlen || s0 < 0 || e0 > p.T) {
                        record_device_error(SWAA_ERR_BAD_SEQLENS);
                        len = 0;
                    }
                    cur_ks = s0;
                    cur_off = 0;
                    if (kPaged) {  // keys in pages: cu_seqlens_k holds the key lengths
                        const int lk = p.cu_seqlens_k[b];
                        if (lk < len || lk > p.max_seqlen_k) {
                            record_device_error(SWAA_ERR_BAD_SEQLENS);
                            len = 0;
                        }
                        cur_ks = b;
                        cur_off = lk - len;
                    } else if (kChunked) {  // chunked prefill: the queries are the last `len` tokens
                        const int ks = p.cu_seqlens_k[b], ke = p.cu_seqlens_k[b + 1];
                        if (ke - ks < len || ke - ks > p.max_seqlen_k || ks < 0 || ke > p.Tk) {
                            record_device_error(SWAA_ERR_BAD_SEQLENS);
                            len = 0;
                        }
                        cur_ks = ks;
                        cur_off = ke - ks - len;
                        if (kCp) {
                            // the local keys start at position p0: the sink keys before it come from the sink buffer,
                            // and the window of the first query must not reach below p0 (halo of window - 1 keys)
                            const int p0 = p.key_pos0[b];
                            if (p0 < 0 || (p0 > 0 && cur_off < p.window - 1) || (p0 > 0 && p.n_sink > p.sink_rows)) {
                                record_device_error(SWAA_ERR_BAD_SEQLENS);
                                len = 0;
                            }
                            cur_srem = p0 < p.n_sink ? max(p0, 0) : p.n_sink;
                            cur_sink = p.n_sink - cur_srem;
                        }
                    }
                    if (kChunked && p.is_full_seq != nullptr) cur_full = p.is_full_seq[b] != 0 ? 1 : 0;
                    cur_s = s0;
                    cur_len = len;
                    cur_nt = (len + BM - 1) / BM;
                }
            };
            next_seq();
            for (int it = 0;; ++it) {
                const long long w = (long long)blockIdx.x + (long long)it * gridDim.x;
                const long long tile_id = w / p.n_pairs;
                const int pair = (int)(w - tile_id * p.n_pairs);
                while (b >= 0 && tile_id >= (long long)acc + cur_nt) next_seq();
                const int slot = it & 1;
                if (!mbar_wait(bar(BAR_WE + slot), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag)) break;
                volatile int* d = work_ring + slot * 12;
                d[0] = b >= 0 ? 1 : 0;
                d[1] = cur_s;
                d[2] = cur_len;
                d[3] = b >= 0 ? cur_nt - 1 - (int)(tile_id - acc) : 0;
                d[4] = pair;
                if (kChunked) {
                    d[5] = cur_ks;
                    d[6] = cur_off;
                    d[7] = cur_full;
                }
                if (kCp) {
                    d[8] = cur_sink;
                    d[9] = cur_srem;
                    d[10] = b;
                }
                mbar_arrive(bar(BAR_WF + slot));
                if (b < 0) break;
            }
        }
        __syncwarp();
      } else if (warp == 8) {
        // =========================================================================== TMA producer
        if (lane == 0) {
            int g = 0;           // K/V tiles issued so far (ring position)
            bool ok = true, q_in_flight = false;
            int items = 0;
            for (int it = 0; ok; ++it) {
                WorkItem w;
                ok = fetch_work(it, w, true);
                if (!ok || !w.valid) break;
                const int hk = w.pair / p.pairs_per_kv;
                const int hA = hk * p.G + 2 * (w.pair - hk * p.pairs_per_kv);
                const bool hasB = (hA + 1) < (hk + 1) * p.G;
                const int i0 = w.m_tile * BM, i1 = min(w.seq_len, i0 + BM) - 1;
                const TileRange tr = tile_range(i0 + w.k_off, i1 + w.k_off, BN, p.window, w.n_sink, w.full != 0);
                const int n_rem = kCp ? (w.s_rem + BN - 1) / BN : 0;  // leading tiles from the sink buffer
                const int nt = n_rem + tr.count();
                // Q tiles of both sides (the previous item's last QK must have retired)
                ok = mbar_wait(bar(BAR_QE), ((uint32_t)items & 1u) ^ 1u, abort_flag);
                if (!ok) break;
                const int tq = w.seq_start + i0;
                mbar_arrive_expect_tx(bar(BAR_QF), (hasB ? 2u : 1u) * (uint32_t)L::kTileBytes);
#pragma unroll
                for (int pn = 0; pn < L::kPanels; ++pn) {
                    tma_load_3d(sQ + pn * L::kPanelBytes, &tm_q, pn * 64, hA, tq, bar(BAR_QF));
                    if (hasB)
                        tma_load_3d(sQ + L::kTileBytes + pn * L::kPanelBytes, &tm_q, pn * 64, hA + 1, tq, bar(BAR_QF));
                }
                q_in_flight = true;
                ++items;
                for (int n = 0; n < nt; ++n, ++g) {
                    const int s = g % ST;
                    const uint32_t ph = (uint32_t)(g / ST) & 1u;
                    const bool remote = kCp && n < n_rem;
                    const int kt = remote ? n * BN : tr.tile(n - n_rem) * BN;  // first key of the tile, counted inside the (local) keys
                    int tk = w.k_start + kt, page = 0;  // packed token index, or (row in page, page) when paged
                    if (kPaged) {
                        page = __ldg(p.block_table + (size_t)w.k_start * p.max_blocks + kt / p.page_size);
                        tk = kt % p.page_size;
                        if (page < 0 || page >= p.num_pages) {
                            record_device_error(SWAA_ERR_BAD_SEQLENS);
                            page = p.num_pages;  // out of range: the copy delivers zeros
                        }
                    }
                    ok = mbar_wait(bar(BAR_KE + s), ph ^ 1u, abort_flag);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar(BAR_KF + s), (uint32_t)L::kTileBytes);
#pragma unroll
                    for (int pn = 0; pn < L::kPanels; ++pn) {
                        if (kPaged) tma_load_4d(sK + s * L::kTileBytes + pn * L::kPanelBytes, &tm_k, pn * 64, hk, tk, page, bar(BAR_KF + s));
                        else if (remote) tma_load_4d(sK + s * L::kTileBytes + pn * L::kPanelBytes, &tm_sk, pn * 64, hk, kt, w.b, bar(BAR_KF + s));
                        else tma_load_3d(sK + s * L::kTileBytes + pn * L::kPanelBytes, &tm_k, pn * 64, hk, tk, bar(BAR_KF + s));
                    }
                    ok = mbar_wait(bar(BAR_VE + s), ph ^ 1u, abort_flag);
                    if (!ok) {
                        mbar_wait(bar(BAR_KF + s), ph, abort_flag);  // the K copy just issued
                        break;
                    }
                    if (kLseOnly) {
                        mbar_arrive(bar(BAR_VF + s));  // no V tile: complete the stage's barrier by hand
                        continue;
                    }
                    mbar_arrive_expect_tx(bar(BAR_VF + s), (uint32_t)L::kTileBytes);
#pragma unroll
                    for (int pn = 0; pn < L::kPanels; ++pn) {
                        if (kPaged) tma_load_4d(sV + s * L::kTileBytes + pn * L::kPanelBytes, &tm_v, pn * 64, hk, tk, page, bar(BAR_VF + s));
                        else if (remote) tma_load_4d(sV + s * L::kTileBytes + pn * L::kPanelBytes, &tm_sv, pn * 64, hk, kt, w.b, bar(BAR_VF + s));
                        else tma_load_3d(sV + s * L::kTileBytes + pn * L::kPanelBytes, &tm_v, pn * 64, hk, tk, bar(BAR_VF + s));
                    }
                    if (kPaged) {
                        // The rows of a page past the sequence's last key may hold anything (also NaN, and 0 * NaN is
                        // NaN in the PV product): clear them in the V tile before the issuer may use it.  Only the last
                        // key tile of a sequence that does not end on a tile boundary is concerned.
                        const int first_bad = w.k_off + w.seq_len - kt;  // rows [first_bad, BN) lie past the last key
                        if (first_bad < BN) {
                            ok = mbar_wait(bar(BAR_VF + s), ph, abort_flag);
                            if (!ok) break;
                            for (int r = max(first_bad, 0); r < BN; ++r)
#pragma unroll
                                for (int pn = 0; pn < L::kPanels; ++pn)
#pragma unroll
                                    for (int j = 0; j < 8; ++j)
                                        st_shared_v4(sV + s * L::kTileBytes + pn * L::kPanelBytes + r * 128 + j * 16, 0u, 0u, 0u, 0u);
                            fence_proxy_async_smem();
                            mbar_arrive(bar(BAR_VC + s));
                        }
                    }
                }
            }
            if (!ok) {
                // give outstanding copies a bounded chance to land before the block's memory is released
                const uint64_t t0 = global_timer_ns();
                bool landed = false;
                while (!landed && global_timer_ns() - t0 < kWaitLimitNs) {
                    landed = !q_in_flight || mbar_try_wait(bar(BAR_QF), (uint32_t)(items - 1) & 1u);
                    for (int n = max(0, g - ST); n < g; ++n) {
                        landed = landed && mbar_try_wait(bar(BAR_KF + n % ST), (uint32_t)(n / ST) & 1u);
                        landed = landed && mbar_try_wait(bar(BAR_VF + n % ST), (uint32_t)(n / ST) & 1u);
                    }
                }
            }
        }
        __syncwarp();
      } else if (warp == 9) {
        // ============================================================================ MMA issuer
        if (lane == 0) {
            const uint32_t tS[2] = {tmem_base, tmem_base + 128u};
            const uint32_t tO[2] = {tmem_base + 256u, tmem_base + 256u + (uint32_t)D};
            // Descriptor words are built once: per operand tile a low word (address, leading-dimension offset)
            // and one shared high word (stride 1024 B, descriptor version, 128-byte swizzle).  The issue latency
            // of this thread is part of every tile's critical path, so the per-MMA work is one add per operand.
            const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0, 0, 1024) >> 32);
            uint32_t q_lo[2], k_lo[ST], v_lo[ST];
#pragma unroll
            for (int sd = 0; sd < 2; ++sd) q_lo[sd] = (uint32_t)smem_desc_sw128(sQ + sd * L::kTileBytes, 16, 1024);
#pragma unroll
            for (int st = 0; st < ST; ++st) {
                k_lo[st] = (uint32_t)smem_desc_sw128(sK + st * L::kTileBytes, 16, 1024);
                v_lo[st] = (uint32_t)smem_desc_sw128(sV + st * L::kTileBytes, L::kPanelBytes, 1024);
            }
            auto pick = [&](const uint32_t (&arr)[ST], int stage) -> uint32_t {  // register array, static indices only
                uint32_t r = arr[0];
#pragma unroll
                for (int st = 1; st < ST; ++st) r = stage == st ? arr[st] : r;
                return r;
            };
            auto issue_qk = [&](int side, int stage) {
                const uint32_t qa = side ? q_lo[1] : q_lo[0], kb = pick(k_lo, stage), d = tS[side];
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = ((uint32_t)(kk >> 2) * L::kPanelBytes + (uint32_t)(kk & 3) * 32u) >> 4;
                    mma_ss_lh(d, qa + off, kb + off, desc_hi, kIdescQK, kk > 0 ? 1u : 0u);
                }
            };
            auto issue_pv = [&](int side, int stage, bool acc, int kk0, int kk1) {
                const uint32_t vb = pick(v_lo, stage), d = tO[side], a = tS[side];
#pragma unroll
                for (int kk = kk0; kk < kk1; ++kk) {
                    // P: 16 keys = 8 TMEM columns of packed bf16 pairs.  V: 16 key rows of 128 bytes.
                    mma_ts_lh(d, a + (uint32_t)kk * 8u, vb + (((uint32_t)kk * 2048u) >> 4), desc_hi, kIdescPV,
                              (acc || kk > 0) ? 1u : 0u);
                }
            };
            int g = 0;                 // K/V ring position
            int gs[2] = {0, 0};        // tiles processed per side (phase of S-full / P-ready / O-done)
            int items_side[2] = {0, 0};
            int items = 0;
            uint32_t vc_phase = 0;  // paged only: bit s = phase of the stage's V-tile-cleared barrier
            bool ok = true;
            for (int it = 0; ok; ++it) {
                WorkItem w;
                ok = fetch_work(it, w, true);
                if (!ok || !w.valid) break;
                const int hk = w.pair / p.pairs_per_kv;
                const int hA = hk * p.G + 2 * (w.pair - hk * p.pairs_per_kv);
                const bool hasB = (hA + 1) < (hk + 1) * p.G;
                const int i0 = w.m_tile * BM, i1 = min(w.seq_len, i0 + BM) - 1;
                const TileRange trng = tile_range(i0 + w.k_off, i1 + w.k_off, BN, p.window, w.n_sink, w.full != 0);
                const int nt = (kCp ? (w.s_rem + BN - 1) / BN : 0) + trng.count();
                ok = mbar_wait(bar(BAR_QF), (uint32_t)items & 1u, abort_flag) &&
                     mbar_wait(bar(BAR_KF + g % ST), (uint32_t)(g / ST) & 1u, abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_qk(0, g % ST);
                tc_commit(bar(BAR_SF + 0));
                if (hasB) {
                    issue_qk(1, g % ST);
                    tc_commit(bar(BAR_SF + 1));
                }
                tc_commit(bar(BAR_KE + g % ST));
                if (nt == 1) tc_commit(bar(BAR_QE));  // Q is no longer needed by this item
                for (int n = 0; n < nt; ++n, ++g) {
                    const int sv = g % ST;
                    const uint32_t pv = (uint32_t)(g / ST) & 1u;
                    const bool has_next = n + 1 < nt;
                    const int sk = (g + 1) % ST;
                    const uint32_t pk = (uint32_t)((g + 1) / ST) & 1u;
                    // The tiles first (they landed long ago as a rule), then the side's P: a look at a barrier costs
                    // this thread some 80 cycles even when it has completed, and what follows the P barrier is on
                    // the side's critical path softmax -> PV -> QK -> softmax.
                    ok = mbar_wait(bar(BAR_VF + sv), pv, abort_flag) &&
                         (!has_next || mbar_wait(bar(BAR_KF + sk), pk, abort_flag)) &&
                         mbar_wait(bar(BAR_PR + 0), (uint32_t)gs[0] & 1u, abort_flag);
                    if (kPaged && ok && w.k_off + w.seq_len - trng.tile(n) * BN < BN) {
                        // last key tile of a sequence that ends inside it: the producer clears the rows past the end
                        ok = mbar_wait(bar(BAR_VC + sv), (vc_phase >> sv) & 1u, abort_flag);
                        vc_phase ^= 1u << sv;
                    }
                    // the first PV of an item overwrites O: the previous item's epilogue must have read it
                    if (ok && n == 0) ok = mbar_wait(bar(BAR_OF + 0), ((uint32_t)items_side[0] & 1u) ^ 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    // the first three quarters of P are there: their products run while the softmax warps finish
                    // the last quarter
                    if (!kLseOnly) issue_pv(0, sv, n > 0, 0, 6);
                    ok = mbar_wait(bar(BAR_PQ + 0), (uint32_t)gs[0] & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    if (!kLseOnly) issue_pv(0, sv, n > 0, 6, 8);
                    // O-done is only waited for by the item's epilogue: between tiles the S-full barrier of tile n + 1
                    // already implies PV(n) (a commit covers every product issued before it), and every commit costs
                    // this thread some 40 cycles
                    if (!has_next) tc_commit(bar(BAR_OD + 0));
                    ++gs[0];
                    if (has_next) {
                        issue_qk(0, sk);
                        tc_commit(bar(BAR_SF + 0));
                    }
                    if (hasB) {
                        ok = mbar_wait(bar(BAR_PR + 1), (uint32_t)gs[1] & 1u, abort_flag);
                        if (ok && n == 0)
                            ok = mbar_wait(bar(BAR_OF + 1), ((uint32_t)items_side[1] & 1u) ^ 1u, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        if (!kLseOnly) issue_pv(1, sv, n > 0, 0, 6);
                        ok = mbar_wait(bar(BAR_PQ + 1), (uint32_t)gs[1] & 1u, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        if (!kLseOnly) issue_pv(1, sv, n > 0, 6, 8);
                        if (!has_next) tc_commit(bar(BAR_OD + 1));
                        ++gs[1];
                        if (has_next) {
                            issue_qk(1, sk);
                            tc_commit(bar(BAR_SF + 1));
                        }
                    }
                    tc_commit(bar(BAR_VE + sv));
                    if (has_next) {
                        tc_commit(bar(BAR_KE + sk));
                        if (n + 2 == nt) tc_commit(bar(BAR_QE));  // that was the item's last QK
                    }
                }
                ++items;
                ++items_side[0];
                if (hasB) ++items_side[1];
            }
            // all MMAs issued by this thread must have retired before the tensor memory is freed
            tc_commit(bar(BAR_FIN));
            mbar_wait(bar(BAR_FIN), 0, abort_flag);
        }
        __syncwarp();
      }
    } else {
        // ==================================================================== softmax + epilogue
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        const int side = warp >> 2;
        const int wq = warp & 3;
        const int row = wq * 32 + lane;
        const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
        const uint32_t tS = tmem_base + lane_base + (uint32_t)side * 128u;
        const uint32_t tO = tmem_base + lane_base + 256u + (uint32_t)side * (uint32_t)D;
        int gs = 0;          // tiles processed by this side so far
        int items_done = 0;  // items finished by this side (phase of O-done)
        bool ok = true;
        for (int it = 0; ok; ++it) {
            WorkItem w;
            // every decision taken after a bounded wait is made for the whole warp: the warp-wide tensor-memory
            // instructions and votes below need all 32 lanes
            ok = __all_sync(0xffffffffu, fetch_work(it, w, false));
            if (!ok) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_WE + (it & 1)));
            if (!w.valid) break;
            const int hk = w.pair / p.pairs_per_kv;
            const int hA = hk * p.G + 2 * (w.pair - hk * p.pairs_per_kv);
            const bool hasB = (hA + 1) < (hk + 1) * p.G;
            if (side == 1 && !hasB) continue;
            const int seq_start = w.seq_start, seq_len = w.seq_len;
            const int q0 = w.m_tile * BM;    // first query of the tile, counted inside the sequence's queries
            const int iq = q0 + row;         // this thread's query, same counting
            const int i0 = q0 + w.k_off, i1 = min(seq_len, q0 + BM) - 1 + w.k_off;  // positions inside the sequence
            const bool full = w.full != 0;
            const TileRange tr = tile_range(i0, i1, BN, p.window, w.n_sink, full);
            const int n_rem = kCp ? (w.s_rem + BN - 1) / BN : 0;  // leading tiles from the sink buffer
            const int nt = n_rem + tr.count();
            const int i = iq + w.k_off;      // index of this thread's query among the (local) keys of its sequence
            const int h = hA + side;
            float m_used = -INFINITY, l_sum = 0.f;
            for (int n = 0; n < nt; ++n, ++gs) {
                // a tile from the sink buffer holds positions before every local key: all rows see exactly its keys
                // below s_rem; no window or causal edge runs through it
                const bool remote = kCp && n < n_rem;
                const int j0 = remote ? n * BN : tr.tile(n - n_rem) * BN;
                const bool need_mask = remote ? (w.s_rem - j0 < BN)
                                              : tile_needs_mask(i0, i1, j0, j0 + BN - 1, p.window, w.n_sink, full);
                ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SF + side), (uint32_t)gs & 1u, abort_flag));
                if (!ok) break;
                tc_fence_after();
                uint32_t sr[128];
                tmem_ld32(tS + 0, sr + 0);
                tmem_ld32(tS + 32, sr + 32);
                tmem_ld32(tS + 64, sr + 64);
                tmem_ld32(tS + 96, sr + 96);
                tc_wait_ld();
                if (kLseOnly) {  // S is in registers: the next Q K^T of this side may overwrite it
                    tc_fence_before();
                    mbar_arrive(bar(BAR_PR + side));
                    mbar_arrive(bar(BAR_PQ + side));
                }
                uint32_t vis[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
                if (need_mask) {
                    // Bit b of vis[cc] <=> column c = 32*cc + b of this tile is visible to this row:
                    //   c <= dc  and  ( c > wl  or  c < sk ).
                    const int dc = remote ? (1 << 20) : i - j0;
                    const int wl = remote ? (1 << 20) : (full ? -1 : dc - p.window);
                    const int sk = remote ? w.s_rem - j0 : (full ? 0 : w.n_sink - j0);
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        const int d = dc - 32 * cc, wd = wl - 32 * cc, sn = sk - 32 * cc;
                        const uint32_t causal = d >= 31 ? 0xffffffffu : (d < 0 ? 0u : ((2u << d) - 1u));
                        const uint32_t win = wd < 0 ? 0xffffffffu : (wd >= 31 ? 0u : ~((2u << wd) - 1u));
                        const uint32_t snk = sn <= 0 ? 0u : (sn >= 32 ? 0xffffffffu : ((1u << sn) - 1u));
                        vis[cc] = causal & (win | snk);
#pragma unroll
                        for (int b = 0; b < 32; ++b)
                            sr[cc * 32 + b] = ((vis[cc] >> b) & 1u) ? sr[cc * 32 + b] : 0xff800000u;  // -inf
                    }
                }
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 128; c += 8) {
                    mx0 = fmax3(mx0, __uint_as_float(sr[c + 0]), __uint_as_float(sr[c + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3]));
                    mx2 = fmax3(mx2, __uint_as_float(sr[c + 4]), __uint_as_float(sr[c + 5]));
                    mx3 = fmax3(mx3, __uint_as_float(sr[c + 6]), __uint_as_float(sr[c + 7]));
                }
                const float rmax = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                const float m_new = fmaxf(m_used, rmax);
                const bool need = (m_used != -INFINITY) && ((m_new - m_used) * p.sl2 > kRescaleThreshold);
                if (__any_sync(0xffffffffu, need)) {
                    // raise the reference maximum of every row of this warp and rescale O accordingly; PV of the
                    // previous tile has completed: it was issued before the QK whose S-full barrier this warp passed
                    const float alpha = (m_used == -INFINITY) ? 1.f : ex2f((m_used - m_new) * p.sl2);
#pragma unroll
                    for (int cc = 0; cc < (kLseOnly ? 0 : D / 32); ++cc) {
                        uint32_t orr[32];
                        tmem_ld32(tO + cc * 32, orr);
                        tc_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * alpha);
                        tmem_st32(tO + cc * 32, orr);
                    }
                    if (!kLseOnly) tc_wait_st();
                    l_sum *= alpha;
                    m_used = m_new;
                } else if (m_used == -INFINITY) {
                    m_used = m_new;  // nothing accumulated yet for this row
                }
                const float off = (m_used == -INFINITY) ? 0.f : m_used * p.sl2;
                const uint64_t sl2x2 = pack_f32x2(p.sl2, p.sl2), noffx2 = pack_f32x2(-off, -off);
                uint64_t psum_a = pack_f32x2(0.f, 0.f), psum_b = pack_f32x2(0.f, 0.f);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t pk[16];
                    if (need_mask && __all_sync(0xffffffffu, vis[cc] == 0u)) {
                        // no row of this warp sees any of these 32 keys: P = 0 without touching the MUFU
#pragma unroll
                        for (int c = 0; c < 16; ++c) pk[c] = 0u;
                        if (!kLseOnly) {
                            tmem_st16(tS + cc * 16, pk);
                            if (cc == 2) {  // three quarters of P written: hand them to the issuer
                                tc_wait_st();
                                tc_fence_before();
                                mbar_arrive(bar(BAR_PR + side));
                            }
                        }
                        continue;
                    }
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const uint64_t x = fma_f32x2(
                            pack_f32x2(__uint_as_float(sr[cc * 32 + 2 * c]), __uint_as_float(sr[cc * 32 + 2 * c + 1])),
                            sl2x2, noffx2);
                        float x0, x1;
                        unpack_f32x2(x, x0, x1);
                        float p0, p1;
                        if ((kPolyPairMask >> c) & 1u) {
                            exp2_poly_x2(x0, x1, p0, p1);  // FMA pipe: takes load off the special-function unit
                        } else {
                            p0 = ex2f(x0);
                            p1 = ex2f(x1);
                        }
                        if (c & 1) psum_b = add_f32x2(psum_b, pack_f32x2(p0, p1));
                        else psum_a = add_f32x2(psum_a, pack_f32x2(p0, p1));
                        if (!kLseOnly) pk[c] = pack_bf16x2(p0, p1);
                    }
                    if (!kLseOnly) {
                        tmem_st16(tS + cc * 16, pk);
                        if (cc == 2) {  // three quarters of P written: hand them to the issuer
                            tc_wait_st();
                            tc_fence_before();
                            mbar_arrive(bar(BAR_PR + side));
                        }
                    }
                }
                {
                    float a0, a1;
                    unpack_f32x2(add_f32x2(psum_a, psum_b), a0, a1);
                    l_sum += a0 + a1;
                }
                if (!kLseOnly) {
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(bar(BAR_PQ + side));
                }
            }
            if (!ok) break;
            // ---- epilogue of this item: O / l -> bf16 -> global
            ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_OD + side), (uint32_t)items_done & 1u, abort_flag));
            if (!ok) break;
            ++items_done;
            tc_fence_after();
            uint32_t orr[D];
            if (!kLseOnly) {
#pragma unroll
                for (int cc = 0; cc < D / 32; ++cc) tmem_ld32(tO + cc * 32, orr + cc * 32);
                tc_wait_ld();
            }
            tc_fence_before();
            mbar_arrive(bar(BAR_OF + side));  // O may be overwritten by the next item's first PV
            const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
            if (kLseOnly) {
                // nothing to store but the log-sum-exp below
            } else if (q0 + wq * 32 + 31 < seq_len) {
                // all 32 rows of this warp are valid: stage [32 rows][64 ch] panels in shared memory in the
                // 128-byte-swizzled layout and let TMA write them (fully coalesced, off the LSU path)
                const uint32_t stage = sStage + (uint32_t)warp * 4096u;
#pragma unroll
                for (int pn = 0; pn < D / 64; ++pn) {
                    if (lane == 0) tma_store_wait_read();  // the previous store has finished reading the stage
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t* o8 = orr + pn * 64 + j * 8;
                        st_shared_v4(stage + (uint32_t)lane * 128u + (uint32_t)((j ^ (lane & 7)) * 16),
                                     pack_bf16x2(__uint_as_float(o8[0]) * inv, __uint_as_float(o8[1]) * inv),
                                     pack_bf16x2(__uint_as_float(o8[2]) * inv, __uint_as_float(o8[3]) * inv),
                                     pack_bf16x2(__uint_as_float(o8[4]) * inv, __uint_as_float(o8[5]) * inv),
                                     pack_bf16x2(__uint_as_float(o8[6]) * inv, __uint_as_float(o8[7]) * inv));
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_3d(&tm_o, stage, pn * 64, h, seq_start + q0 + wq * 32);
                        tma_store_commit();
                    }
                }
            } else if (iq < seq_len) {
                // ragged tail of a sequence: plain predicated row stores
                __nv_bfloat16* orow = p.out + ((size_t)(seq_start + iq) * p.Hq + h) * D;
#pragma unroll
                for (int v = 0; v < D / 8; ++v) {
                    uint4 o4;
                    o4.x = pack_bf16x2(__uint_as_float(orr[v * 8 + 0]) * inv, __uint_as_float(orr[v * 8 + 1]) * inv);
                    o4.y = pack_bf16x2(__uint_as_float(orr[v * 8 + 2]) * inv, __uint_as_float(orr[v * 8 + 3]) * inv);
                    o4.z = pack_bf16x2(__uint_as_float(orr[v * 8 + 4]) * inv, __uint_as_float(orr[v * 8 + 5]) * inv);
                    o4.w = pack_bf16x2(__uint_as_float(orr[v * 8 + 6]) * inv, __uint_as_float(orr[v * 8 + 7]) * inv);
                    *reinterpret_cast<uint4*>(orow + v * 8) = o4;
                }
            }
            if (iq < seq_len && p.lse != nullptr) {
                const float lse2 = (m_used == -INFINITY) ? -INFINITY : m_used * p.sl2 + log2f(l_sum);
                p.lse[(size_t)h * p.T + seq_start + iq] = lse2 * 0.6931471805599453f;
            }
        }
        if (lane == 0) tma_store_wait_all();  // outstanding output stores of this warp
    }

    // ---- teardown: every thread arrives here (also after a failed wait); free the tensor memory
    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace swaa
