// Backward pass of the prefill attention on the tcgen05 tensor cores (head dimension 128), Sec. 3.2.2.
//
// One block owns a tile of 128 keys of one (sequence, kv head) and walks the 64-row query tiles that can
// see it, for every query head of the GQA group.  All five products of a step run as tcgen05.mma with the
// accumulators in tensor memory:
//
//   S^T  = K  Q^T    [128 keys x 64 rows]   A = K tile, B = Q tile        (both K-major, shared memory)
//   dP^T = V  dO^T   [128 keys x 64 rows]   A = V tile, B = dO tile
//   dV  += P^T  dO   [128 keys x D]         A = P^T in tensor memory (bf16), B = dO tile read MN-major
//   dK  += dS^T Q    [128 keys x D]         A = dS^T in tensor memory,        B = Q tile read MN-major
//   dQ^T = K^T dS^T  [D x 64 rows]          A = K tile read MN-major, B = dS^T in shared memory (MN-major)
//
// with P^T = exp2(S^T * scale * log2e - lse2[row]) and dS^T = P^T * (scale * dP^T - scale * delta[row]) computed by
// the thread that owns the key (one tensor-memory lane per key).  dV and dK stay in tensor memory for the
// whole block; dQ^T goes through shared memory (transposed to [rows][D], in the ring stage of the step's Q and dO
// tiles, which are dead by then) and is added to an fp32 accumulator in global memory by one bulk reduce-add copy (per-lane atomics saturate the L2 atomic units and stall the block's
// other shared-memory traffic behind them).  Two groups of four warps take alternate steps, each with its own S^T/dP^T columns, so the
// element-wise work of one step overlaps the products of the other.
//
// Tensor memory (512 columns): dV [0,128) | dK [128,256) | X_0 [256,384) | X_1 [384,512); X_g holds
// S^T [0,64) and dP^T [64,128) of the group's step, then P^T (bf16 pairs, [0,32)) and dS^T ([64,96)),
// then dQ^T [0,64).  The tensor core runs the products of one issuing thread in order, which is what
// makes these overlays safe.
//
// Warps 0-7: the two element-wise groups; warp 8: TMA producer (K, V once; Q, dO and the row terms per
// step through a ring of four stages); warp 9: MMA issuer.  Every wait is bounded.
#pragma once

#include <type_traits>

#include "swaa_backward.cuh"
#include "swaa_prefill.cuh"  // tcgen05 wrappers, descriptors

namespace swaa {

constexpr int kBwdTcKeys = 128;    // keys per block
constexpr int kBwdTcRows = 64;     // query rows per step
constexpr int kBwdTcThreads = 320;
constexpr int kBwdTcStages = 4;    // ring of (Q, dO, row terms); a stage also stages the step's dQ on its way out

struct BackwardTcSmem {
    static constexpr int D = 128;
    static constexpr int kKVTileBytes = kBwdTcKeys * D * 2;    // 32 KiB: two panels of [128][64 ch]
    static constexpr int kKVPanelBytes = kBwdTcKeys * 128;
    static constexpr int kQTileBytes = kBwdTcRows * D * 2;     // 16 KiB: two panels of [64][64 ch]
    static constexpr int kQPanelBytes = kBwdTcRows * 128;
    static constexpr int kStageBytes = 2 * kQTileBytes;        // Q then dO
    static constexpr int kDSBytes = kBwdTcKeys * 128;          // dS^T [128 keys][64 rows] bf16
    static constexpr int kOffK = 0, kOffV = kKVTileBytes;
    static constexpr int kOffRing = 2 * kKVTileBytes;
    static constexpr int kOffDS = kOffRing + kBwdTcStages * kStageBytes;  // two buffers (one per group)
    static constexpr int kOffRows = kOffDS + 2 * kDSBytes;     // per stage: lse2[64], delta[64] (fp32)
    static constexpr int kOffBar = kOffRows + kBwdTcStages * 128 * 4;
    static constexpr int kNumBars = 1 + 2 * kBwdTcStages + 4 * 2 + 1;
    static constexpr int kOffMisc = kOffBar + kNumBars * 8;
    static constexpr int kBytes = kOffMisc + 32;
    static constexpr int kDynamicBytes = kBytes;  // the kernel declares the array 1024-byte aligned and checks it
    static_assert(kDynamicBytes <= 232448, "shared memory per block");
};

// kind::f16 instruction descriptor with both operands read MN-major from shared memory.
__host__ __device__ constexpr uint32_t make_idesc_mn_mn(int M, int N) { return make_idesc(M, N, 1) | (1u << 15); }

// Vote of the 128 threads of one element-wise group (named barrier `id`): true when `pred` holds for all of them.
// A bounded wait can give up in one thread and succeed in its neighbour; the vote makes the group leave together,
// which the plain group barriers further down rely on.
__device__ __forceinline__ bool group_all(bool pred, int id) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\tbar.red.and.pred q, %2, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(id)
        : "memory");
    return r != 0;
}

__global__ void __launch_bounds__(kBwdTcThreads, 1)
backward_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                   const __grid_constant__ CUtensorMap tm_dq, const BackwardParams p) {
    using L = BackwardTcSmem;
    constexpr int D = 128, BK = kBwdTcKeys, BR = kBwdTcRows, NQ = kBwdTcStages;
    constexpr uint32_t kIdS = make_idesc(BK, BR, 0);      // S^T, dP^T
    constexpr uint32_t kIdKV = make_idesc(BK, D, 1);      // dV, dK (A from tensor memory)
    constexpr uint32_t kIdDQ = make_idesc_mn_mn(D, BR);   // dQ^T

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t smem_base = smem_u32(smem_raw);
    uint8_t* smem_gen = smem_raw;
    if ((smem_base & 1023u) != 0u) {  // the swizzled tiles need it; uniform, before any barrier or allocation
        if (threadIdx.x == 0) record_device_error(SWAA_ERR_CUDA);
        return;
    }
    const uint32_t sK = smem_base + L::kOffK, sV = smem_base + L::kOffV, sRing = smem_base + L::kOffRing;
    const uint32_t sDS = smem_base + L::kOffDS;
    float* s_rows = reinterpret_cast<float*>(smem_gen + L::kOffRows);
    const uint32_t bars = smem_base + L::kOffBar;
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
    constexpr int BAR_KV = 0, BAR_QF = 1, BAR_QE = BAR_QF + NQ, BAR_SF = BAR_QE + NQ, BAR_PR = BAR_SF + 2;
    constexpr int BAR_DQ = BAR_PR + 2, BAR_DR = BAR_DQ + 2, BAR_FIN = BAR_DR + 2;
    static_assert(BAR_FIN + 1 == L::kNumBars, "barrier count");
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + L::kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hk = blockIdx.y, b = blockIdx.z;
    // blockIdx.x -> (key tile, chunk of its query range); see backward_kernel
    int n_tile, chunk = -1;
    if ((int)blockIdx.x < p.sink_tiles * p.chunks) {
        n_tile = (int)blockIdx.x / p.chunks;
        chunk = (int)blockIdx.x - n_tile * p.chunks;
    } else {
        n_tile = p.sink_tiles + ((int)blockIdx.x - p.sink_tiles * p.chunks);
    }
    const int seq_start = p.cu_seqlens[b], Lseq = p.cu_seqlens[b + 1] - seq_start;
    const int j0 = n_tile * BK;
    if (Lseq <= 0 || Lseq > p.max_seqlen || j0 >= Lseq || seq_start < 0 ||
        seq_start + Lseq > p.T) {  // uniform: before any barrier or allocation
        if (threadIdx.x == 0 && (Lseq < 0 || Lseq > p.max_seqlen || seq_start < 0 || seq_start + Lseq > p.T))
            record_device_error(SWAA_ERR_BAD_SEQLENS);
        return;
    }
    const bool full = p.is_full != 0;
    const int j1 = j0 + BK - 1;  // keys past the end of the sequence are masked like future keys
    int m_lo = j0 / BR;
    int m_hi = (full || j0 < p.n_sink) ? (Lseq - 1) / BR
                                       : (int)(min((long long)Lseq - 1, (long long)j1 + p.window - 1) / BR);
    const bool split = chunk >= 0;
    if (split) {
        m_lo += chunk * kBwdChunkTiles;
        m_hi = min(m_hi, m_lo + kBwdChunkTiles - 1);
        if (m_lo > m_hi) return;
    }
    const int nm = m_hi - m_lo + 1, n_steps = nm * p.G;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int i = 0; i < L::kNumBars; ++i) {
            uint32_t count = 1u;
            if (i >= BAR_QF && i < BAR_QF + NQ) count = 33u;  // the TMA transaction + the 32 lanes that write the row terms
            if ((i >= BAR_PR && i < BAR_PR + 2) || (i >= BAR_DR && i < BAR_DR + 2)) count = 128u;
            mbar_init(bar(i), count);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tDV = tmem_base, tDK = tmem_base + 128u;
    const float sl2 = p.scale * 1.4426950408889634f;

    if (warp == 8) {
        // ================================================================================= producer
        bool ok = true;
        if (lane == 0) {
            mbar_arrive_expect_tx(bar(BAR_KV), 2u * (uint32_t)L::kKVTileBytes);
#pragma unroll
            for (int pn = 0; pn < 2; ++pn) {
                tma_load_3d(sK + pn * L::kKVPanelBytes, &tm_k, pn * 64, hk, seq_start + j0, bar(BAR_KV));
                tma_load_3d(sV + pn * L::kKVPanelBytes, &tm_v, pn * 64, hk, seq_start + j0, bar(BAR_KV));
            }
        }
        int issued = 0;
        for (int s = 0; s < n_steps; ++s) {
            const int st = s % NQ;
            if (s >= NQ) ok = mbar_wait(bar(BAR_QE + st), (uint32_t)(s / NQ - 1) & 1u, abort_flag);
            if (!ok) break;
            const int h = hk * p.G + s / nm, i0 = (m_lo + s % nm) * BR;
            if (lane == 0) {
                const uint32_t dst = sRing + (uint32_t)st * L::kStageBytes;
                mbar_arrive_expect_tx(bar(BAR_QF + st), (uint32_t)L::kStageBytes);
#pragma unroll
                for (int pn = 0; pn < 2; ++pn) {
                    tma_load_3d(dst + pn * L::kQPanelBytes, &tm_q, pn * 64, h, seq_start + i0, bar(BAR_QF + st));
                    tma_load_3d(dst + L::kQTileBytes + pn * L::kQPanelBytes, &tm_do, pn * 64, h, seq_start + i0,
                                bar(BAR_QF + st));
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {  // 64 x lse2, 64 x delta (negated, delta scaled); zeros past the end of the sequence
                const int idx = lane + 32 * q, r = idx & 63, i = i0 + r;
                const float* src = (idx < 64 ? p.lse2 : p.delta) + (size_t)h * p.T + seq_start;
                // stored ready for one fused multiply-add each: -lse2 and -delta * scale
                s_rows[st * 128 + idx] = i < Lseq ? -src[i] * (idx < 64 ? 1.f : p.scale) : 0.f;
            }
            mbar_arrive(bar(BAR_QF + st));
            issued = s + 1;
        }
        if (!ok) {  // give outstanding copies a bounded chance to land before the block's memory is released
            const uint64_t t0 = global_timer_ns();
            bool landed = false;
            while (!landed && global_timer_ns() - t0 < kWaitLimitNs) {
                landed = mbar_try_wait(bar(BAR_KV), 0u);
                for (int s = max(0, issued - NQ); s < issued; ++s)
                    landed = landed && mbar_try_wait(bar(BAR_QF + s % NQ), (uint32_t)(s / NQ) & 1u);
            }
        }
        __syncwarp();
    } else if (warp == 9) {
        // =================================================================================== issuer
        if (lane == 0) {
            const uint32_t hi = (uint32_t)(smem_desc_sw128(0, 0, 1024) >> 32);
            const uint32_t k_a = (uint32_t)smem_desc_sw128(sK, 16, 1024);                    // K tile, K-major (A)
            const uint32_t v_a = (uint32_t)smem_desc_sw128(sV, 16, 1024);                    // V tile, K-major (A)
            const uint32_t k_t = (uint32_t)smem_desc_sw128(sK, L::kKVPanelBytes, 1024);      // K tile, MN-major (A)
            const uint32_t q_b0 = (uint32_t)smem_desc_sw128(sRing, 16, 1024);                // Q tile of stage 0, K-major (B)
            const uint32_t q_t0 = (uint32_t)smem_desc_sw128(sRing, L::kQPanelBytes, 1024);   // Q tile of stage 0, MN-major (B)
            const uint32_t ds_t0 = (uint32_t)smem_desc_sw128(sDS, 16, 1024);                 // dS^T of group 0, MN-major (B)
            constexpr uint32_t kStageStep = (uint32_t)L::kStageBytes >> 4, kDoStep = (uint32_t)L::kQTileBytes >> 4;
            constexpr uint32_t kDsStep = (uint32_t)L::kDSBytes >> 4;
            // S^T = K Q^T (columns [0,64) of X_{s & 1}) and dP^T = V dO^T (columns [64,128)) of step s
            auto issue_st = [&](int s) {
                const uint32_t qb = q_b0 + (uint32_t)(s % NQ) * kStageStep, tX = tmem_base + 256u + 128u * (uint32_t)(s & 1);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t oa = ((uint32_t)(kk >> 2) * L::kKVPanelBytes + (uint32_t)(kk & 3) * 32u) >> 4;
                    const uint32_t ob = ((uint32_t)(kk >> 2) * L::kQPanelBytes + (uint32_t)(kk & 3) * 32u) >> 4;
                    mma_ss_lh(tX, k_a + oa, qb + ob, hi, kIdS, kk > 0 ? 1u : 0u);
                }
            };
            auto issue_dp = [&](int s) {
                const uint32_t qb = q_b0 + (uint32_t)(s % NQ) * kStageStep, tX = tmem_base + 256u + 128u * (uint32_t)(s & 1);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t oa = ((uint32_t)(kk >> 2) * L::kKVPanelBytes + (uint32_t)(kk & 3) * 32u) >> 4;
                    const uint32_t ob = ((uint32_t)(kk >> 2) * L::kQPanelBytes + (uint32_t)(kk & 3) * 32u) >> 4;
                    mma_ss_lh(tX + 64u, v_a + oa, qb + kDoStep + ob, hi, kIdS, kk > 0 ? 1u : 0u);
                }
            };
            // dV += P^T dO, dK += dS^T Q, dQ^T = K^T dS^T of step s
            auto issue_g = [&](int s) {
                const uint32_t qt = q_t0 + (uint32_t)(s % NQ) * kStageStep, tX = tmem_base + 256u + 128u * (uint32_t)(s & 1);
                const uint32_t ds = ds_t0 + (uint32_t)(s & 1) * kDsStep;
#pragma unroll
                for (int kk = 0; kk < BR / 16; ++kk) {  // 16 rows: 8 columns of bf16 pairs, 16 rows of 128 bytes
                    const uint32_t ob = ((uint32_t)kk * 2048u) >> 4;
                    mma_ts_lh(tDV, tX + (uint32_t)kk * 8u, qt + kDoStep + ob, hi, kIdKV, (s > 0 || kk > 0) ? 1u : 0u);
                    mma_ts_lh(tDK, tX + 64u + (uint32_t)kk * 8u, qt + ob, hi, kIdKV, (s > 0 || kk > 0) ? 1u : 0u);
                }
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk) {  // 16 keys: 16 rows of 128 bytes in both operands
                    const uint32_t o = ((uint32_t)kk * 2048u) >> 4;
                    mma_ss_lh(tX, k_t + o, ds + o, hi, kIdDQ, kk > 0 ? 1u : 0u);
                }
            };
            bool ok = mbar_wait(bar(BAR_KV), 0u, abort_flag);
            for (int s = 0; s < 2 && s < n_steps && ok; ++s) {
                ok = mbar_wait(bar(BAR_QF + s % NQ), 0u, abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_dp(s);
                issue_st(s);
                tc_commit(bar(BAR_SF + s));
            }
            // Steady state: G(s) as soon as the group has written P^T, dS^T of step s; then the products that feed
            // the same group's step s + 2.  dP^T(s+2) only needs columns [64,128), free once G(s) has run (products
            // run in issue order), and fills the time until the group has taken dQ^T(s) out of the columns that
            // S^T(s+2) overwrites.  (Every look at a barrier costs this thread about 80 cycles during which no
            // product is issued; folding the tile barrier into the group's arrival was slower all the same, because
            // dP^T then waits for the read-out too.)
            for (int s = 0; s < n_steps && ok; ++s) {
                const int g = s & 1;
                const uint32_t ph = (uint32_t)(s >> 1) & 1u;
                ok = mbar_wait(bar(BAR_PR + g), ph, abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_g(s);
                tc_commit(bar(BAR_DQ + g));
                if (s + 2 < n_steps) {
                    // (this look falls under the tail of G(s); ahead of the wait for the group it was slower)
                    ok = mbar_wait(bar(BAR_QF + (s + 2) % NQ), (uint32_t)((s + 2) / NQ) & 1u, abort_flag);
                    if (!ok) break;
                    issue_dp(s + 2);
                    ok = mbar_wait(bar(BAR_DR + g), ph, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_st(s + 2);
                    tc_commit(bar(BAR_SF + g));
                }
            }
            // all products issued by this thread must have retired before the tensor memory is read or freed
            tc_commit(bar(BAR_FIN));
            mbar_wait(bar(BAR_FIN), 0u, abort_flag);
        }
        __syncwarp();
    } else {
        // ===================================================================== element-wise groups
        const int grp = warp >> 2, quad = warp & 3;
        const int kl = 32 * quad + lane;  // tensor-memory lane: the key (S^T, dP^T, dV, dK) or the channel (dQ^T)
        const int j = j0 + kl;
        const uint32_t lane_bits = (uint32_t)(32 * quad) << 16;
        const uint32_t tX = tmem_base + lane_bits + 256u + 128u * (uint32_t)grp;
        const uint32_t sDSg = sDS + (uint32_t)grp * L::kDSBytes + (uint32_t)kl * 128u;
        // rows of the step that this key sees: i in [max(j, .), hi) with hi = end of the window (or of the sequence)
        const int vis_hi = (full || j < p.n_sink) ? Lseq : (int)min((long long)Lseq, (long long)j + p.window);
        bool ok = true;
        int pending_stage = -1;  // thread kl == 0: ring stage that holds the previous step's dQ staging
        // One half (32 rows) of the element-wise step; kMask: the tile has pairs outside the mask.
        const uint64_t sl2x2 = pack_f32x2(sl2, sl2), scx2 = pack_f32x2(p.scale, p.scale);
        auto half_step = [&](auto mask_tag, int half, const float* rows, int i0) {
            constexpr bool kMask = decltype(mask_tag)::value;
            uint32_t sv[32], dv[32], pk[16], dk[16];
            tmem_ld32(tX + 32u * (uint32_t)half, sv);
            tmem_ld32(tX + 64u + 32u * (uint32_t)half, dv);
            tc_wait_ld();
            // visible rows of this half, as offsets: r in [r_lo, r_hi)
            const int r_lo = j - i0 - 32 * half, r_hi = vis_hi - i0 - 32 * half;
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
                const int r = 32 * half + e;
                const float4 l4 = *reinterpret_cast<const float4*>(rows + r);       // -lse2 of four rows
                const float4 d4 = *reinterpret_cast<const float4*>(rows + 64 + r);  // -delta * scale
                float pv[4], dsv[4];
#pragma unroll
                for (int u = 0; u < 4; u += 2) {  // two rows per packed fp32 instruction
                    const uint64_t x = fma_f32x2(pack_f32x2(__uint_as_float(sv[e + u]), __uint_as_float(sv[e + u + 1])), sl2x2,
                                                 u ? pack_f32x2(l4.z, l4.w) : pack_f32x2(l4.x, l4.y));
                    const uint64_t t = fma_f32x2(pack_f32x2(__uint_as_float(dv[e + u]), __uint_as_float(dv[e + u + 1])), scx2,
                                                 u ? pack_f32x2(d4.z, d4.w) : pack_f32x2(d4.x, d4.y));
                    float x0, x1;
                    unpack_f32x2(x, x0, x1);
                    pv[u] = ex2f(x0);
                    pv[u + 1] = ex2f(x1);
                    uint64_t d2;
                    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d2) : "l"(pack_f32x2(pv[u], pv[u + 1])), "l"(t));
                    unpack_f32x2(d2, dsv[u], dsv[u + 1]);
                }
                if (kMask) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const bool vis = e + u >= r_lo && e + u < r_hi;
                        pv[u] = vis ? pv[u] : 0.f;
                        dsv[u] = vis ? dsv[u] : 0.f;
                    }
                }
                pk[e >> 1] = pack_bf16x2(pv[0], pv[1]);
                pk[(e >> 1) + 1] = pack_bf16x2(pv[2], pv[3]);
                dk[e >> 1] = pack_bf16x2(dsv[0], dsv[1]);
                dk[(e >> 1) + 1] = pack_bf16x2(dsv[2], dsv[3]);
            }
            // P^T and dS^T as bf16 pairs over columns that this thread has already read
            tmem_st16(tX + 16u * (uint32_t)half, pk);
            tmem_st16(tX + 64u + 16u * (uint32_t)half, dk);
#pragma unroll
            for (int q = 0; q < 4; ++q) {  // dS^T row of this key: 16-byte chunk 4*half + q, 128-byte swizzle
                const int ch = 4 * half + q;
                st_shared_v4(sDSg + (uint32_t)((ch ^ (kl & 7)) << 4), dk[4 * q], dk[4 * q + 1], dk[4 * q + 2],
                             dk[4 * q + 3]);
            }
        };
        for (int s = grp; s < n_steps && ok; s += 2) {
            const int st = s % NQ;
            const uint32_t ph = (uint32_t)(s >> 1) & 1u;
            const int h = hk * p.G + s / nm, i0 = (m_lo + s % nm) * BR;
            const int i1 = min(i0 + BR, Lseq) - 1;
            ok = group_all(mbar_wait(bar(BAR_QF + st), (uint32_t)(s / NQ) & 1u, abort_flag) &&
                               mbar_wait(bar(BAR_SF + grp), ph, abort_flag),
                           1 + grp);
            if (!ok) break;
            tc_fence_after();
            if (kl == 0 && pending_stage >= 0) {
                // the reduce-add of this group's previous step has read its staging (issued two steps ago): hand
                // the ring stage back to the producer
                tma_store_wait_read();
                mbar_arrive(bar(BAR_QE + pending_stage));
                pending_stage = -1;
            }
            const float* rows = s_rows + st * 128;
            const bool need_mask = i0 + BR > Lseq || tile_needs_mask(i0, i1, j0, j1, p.window, p.n_sink, full);
            if (need_mask) {
                half_step(std::true_type{}, 0, rows, i0);
                half_step(std::true_type{}, 1, rows, i0);
            } else {
                half_step(std::false_type{}, 0, rows, i0);
                half_step(std::false_type{}, 1, rows, i0);
            }
            tc_wait_st();
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar(BAR_PR + grp));

            // ---- dQ^T of this step (lane = channel, column = row) -> [64 rows][128 channels] fp32 in the step's
            // ring stage (Q and dO are no longer needed once dQ^T is complete) -> one bulk reduce-add of the box
            // into the fp32 accumulator.  Rows of the box past the end of the sequence receive exact zeros (their
            // dS^T columns are zero); rows past T are clipped by the copy.
            ok = group_all(mbar_wait(bar(BAR_DQ + grp), ph, abort_flag), 1 + grp);
            if (!ok) break;
            tc_fence_after();
            const uint32_t stg = sRing + (uint32_t)st * L::kStageBytes + (uint32_t)kl * 4u;
            {
                uint32_t v0[32], v1[32];
                tmem_ld32(tX, v0);
                tmem_ld32(tX + 32u, v1);
                tc_wait_ld();
                // the group's columns may take the next S^T as soon as dQ^T is in registers
                tc_fence_before();
                mbar_arrive(bar(BAR_DR + grp));
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(stg + (uint32_t)(e * 512)), "r"(v0[e]) : "memory");
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(stg + (uint32_t)((32 + e) * 512)), "r"(v1[e]) : "memory");
                }
            }
            fence_proxy_async_smem();
            asm volatile("bar.sync %0, 128;" ::"r"(1 + grp) : "memory");
            if (kl == 0) {
                tma_reduce_add_3d(&tm_dq, sRing + (uint32_t)st * L::kStageBytes, 0, h, seq_start + i0);
                tma_store_commit();
                pending_stage = st;
            }
        }
        if (kl == 0) tma_store_wait_all();  // this group's reductions into dq have been performed
        // ---- dV (group 0) and dK (group 1) rows of this thread's key
        if (ok) ok = mbar_wait(bar(BAR_FIN), 0u, abort_flag);
        if (ok) {
            tc_fence_after();
            const uint32_t tAcc = tmem_base + lane_bits + 128u * (uint32_t)grp;
            if (split) {
                const int sink_rows = p.sink_tiles * BK;
                const size_t plane = (size_t)p.B * sink_rows * p.Hkv * D;
                float* dst = p.dkv_accum + (size_t)(1 - grp) * plane +  // plane 0: dk, plane 1: dv
                             (((size_t)b * sink_rows + j) * p.Hkv + hk) * D;
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint32_t v[32];
                    tmem_ld32(tAcc + 32u * (uint32_t)c4, v);
                    tc_wait_ld();
                    if (j < Lseq) {
#pragma unroll
                        for (int e = 0; e < 32; e += 2)
                            atomicAdd(reinterpret_cast<float2*>(dst + 32 * c4 + e),
                                      make_float2(__uint_as_float(v[e]), __uint_as_float(v[e + 1])));
                    }
                }
            } else {
                __nv_bfloat16* dst = (grp == 0 ? p.dv : p.dk) + ((size_t)(seq_start + j) * p.Hkv + hk) * D;
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint32_t v[32];
                    tmem_ld32(tAcc + 32u * (uint32_t)c4, v);
                    tc_wait_ld();
                    if (j < Lseq) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint4 o;
                            o.x = pack_bf16x2(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
                            o.y = pack_bf16x2(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
                            o.z = pack_bf16x2(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5]));
                            o.w = pack_bf16x2(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7]));
                            *reinterpret_cast<uint4*>(dst + 32 * c4 + e) = o;
                        }
                    }
                }
            }
        }
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
