// Backward pass of the prefill attention under the same mask policy (for SWA-aware fine-tuning, Sec. 3.2.2:
// the adapted model is trained with the mask it will be served with).
//
// Given q, k, v, out, dout and the log-sum-exp rows of the forward pass:
//     P_ij   = exp(scale * q_i.k_j - lse_i)            for visible (i, j), else 0
//     dV_j   = sum_i P_ij dO_i
//     dP_ij  = dO_i . v_j,   delta_i = dO_i . out_i
//     dS_ij  = P_ij (dP_ij - delta_i)
//     dQ_i   = scale * sum_j dS_ij k_j,   dK_j = scale * sum_i dS_ij q_i
// with dK, dV summed over the query heads of a GQA group.
//
// This file holds the parts shared by the two kernels (parameters, the row-term and conversion kernels) and
// the warp-level kernel used for head dimension 64; head dimension 128 runs on the tcgen05 kernel of
// swaa_backward_tc.cuh.
//
// Warp-level kernel: one thread block owns one 64-key tile of one (sequence, key/value head) and keeps its dK and dV in
// registers; it walks the query heads of the group and, per head, only the 64-row query tiles that can
// see the key tile (the band above it, plus every later tile when the key tile holds sink keys), so the
// work is O(L * window) like the forward pass (App. A).  Each of the four warps owns 16 keys: it forms
// S^T = K Q^T, P^T, dP^T = V dO^T and dS^T for its keys against the 64 query rows with warp-level
// tensor-core MMAs (fp32 accumulation), feeds P^T and dS^T straight back as A operands for
// dV += P^T dO and dK += dS^T Q, and leaves dS^T in shared memory, from where every warp takes the 16
// query rows it owns to form dQ += dS K; dQ is accumulated across key tiles in an fp32 buffer with
// atomic adds and converted to bf16 by a second kernel.  Tiles are staged by TMA (128-byte swizzle).  The key
// tiles that hold sink keys meet every later query tile: with long sequences their query range is cut into
// chunks handled by separate blocks, which add dK and dV into fp32 accumulators (converted by a third kernel).
#pragma once

#include "swaa_internal.cuh"
#include "swaa_ptx.cuh"
#include "swaa_decode.cuh"  // mma_bf16_16816

namespace swaa {

struct BackwardParams {
    const float* lse;        // [Hq, T] natural log (forward output)
    const float* lse2;       // [Hq, T] the same times log2(e), written with delta
    const float* delta;      // [Hq, T]
    float* dkv_accum;        // [2][B][sink_rows][Hkv][D] fp32, zeroed: dk, dv of the sink tiles, which are split over blocks
    int sink_tiles;          // key tiles that hold sink keys (their query range is cut into chunks), 0 for full attention
    int chunks;              // blocks per sink tile
    float* dq_accum;         // [T, Hq, D] fp32, zeroed before the launch
    __nv_bfloat16* dk;       // [T, Hkv, D]
    __nv_bfloat16* dv;
    const int32_t* cu_seqlens;
    int B, T, Hq, Hkv, G;
    int max_seqlen;          // the launch covers sequences up to this length; a longer one is reported and skipped
    int window, n_sink, is_full;
    float scale;
};

constexpr int kBwdTile = 64;      // keys per block and query rows per step
constexpr int kBwdThreads = 128;  // four warps, 16 keys each
constexpr int kBwdChunkTiles = 32; // query tiles per block of a sink key tile

template <int D>
struct BackwardSmem {
    static constexpr int kPanels = D / 64;
    static constexpr int kPanelBytes = kBwdTile * 128;
    static constexpr int kTileBytes = kPanels * kPanelBytes;  // one [64][D] bf16 tile
    static constexpr int kOffK = 0, kOffV = kTileBytes;
    static constexpr int kOffQ = 2 * kTileBytes;              // two buffers of (Q tile, dO tile)
    static constexpr int kOffDS = 6 * kTileBytes;             // dS^T [64 keys][64 rows] bf16, 128-byte rows, swizzled
    static constexpr int kOffRow = kOffDS + kBwdTile * 128;   // two buffers of (lse * log2e, delta) of the 64 rows (fp32)
    static constexpr int kOffBar = kOffRow + 4 * kBwdTile * 4;
    static constexpr int kBytes = kOffBar + 3 * 8 + 16;
    static constexpr int kDynamicBytes = kBytes + 1024;
};

// delta[h, t] = sum_d out[t, h, d] * dout[t, h, d] and lse2 = lse * log2(e); one warp per (t, h), which also clears
// its row of the fp32 dq accumulator.
template <int D>
__global__ void backward_delta_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                                      const float* __restrict__ lse, float* __restrict__ delta,
                                      float* __restrict__ lse2, float* __restrict__ dq_accum, int T, int Hq) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= T * Hq) return;
    const int t = row / Hq, h = row - t * Hq;
    const __nv_bfloat16* o = out + (size_t)row * D;
    const __nv_bfloat16* g = dout + (size_t)row * D;
    float acc = 0.f;
    for (int d = lane * 2; d < D; d += 64) {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(o + d));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(g + d));
        acc += a.x * b.x + a.y * b.y;
    }
    for (int d = lane * 4; d < D; d += 128)
        *reinterpret_cast<float4*>(dq_accum + (size_t)row * D + d) = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) {
        delta[(size_t)h * T + t] = acc;
        lse2[(size_t)h * T + t] = lse[(size_t)h * T + t] * 1.4426950408889634f;
    }
}

// dq = bf16(dq_accum)
__global__ void backward_convert_dq_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, size_t n) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i + 3 < n) {
        const float4 v = *reinterpret_cast<const float4*>(acc + i);
        *reinterpret_cast<uint2*>(dq + i) = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
    } else {
        for (size_t j = i; j < n; ++j) dq[j] = __float2bfloat16_rn(acc[j]);
    }
}

// dk, dv rows of the split key tiles = bf16(dkv_accum); one thread per four channels of one (b, row, kv head).
__global__ void backward_convert_dkv_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dk,
                                            __nv_bfloat16* __restrict__ dv, const int32_t* __restrict__ cu_seqlens, int B,
                                            int T, int max_seqlen, int sink_rows, int Hkv, int D) {
    const size_t plane = (size_t)B * sink_rows * Hkv * D;
    const size_t e = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (e >= plane) return;
    const size_t row = e / ((size_t)Hkv * D);  // b * sink_rows + j
    const int b = (int)(row / sink_rows), j = (int)(row - (size_t)b * sink_rows);
    const int seq_start = cu_seqlens[b], Lseq = cu_seqlens[b + 1] - seq_start;
    if (j >= Lseq || Lseq > max_seqlen || seq_start < 0 || seq_start + Lseq > T) return;
    const size_t dst = (size_t)(seq_start + j) * Hkv * D + (e - row * (size_t)Hkv * D);
    const float4 a = *reinterpret_cast<const float4*>(acc + e);
    const float4 c = *reinterpret_cast<const float4*>(acc + plane + e);
    *reinterpret_cast<uint2*>(dk + dst) = make_uint2(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w));
    *reinterpret_cast<uint2*>(dv + dst) = make_uint2(pack_bf16x2(c.x, c.y), pack_bf16x2(c.z, c.w));
}

// Address of the 16-byte chunk `chunk` (0..D/8-1) of row `row` of a [64][D] tile stored as 64-channel
// panels of 128-byte rows with the 128-byte swizzle.
__device__ __forceinline__ uint32_t bwd_tile_addr(uint32_t base, int row, int chunk) {
    return base + (uint32_t)((chunk >> 3) * (kBwdTile * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
backward_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                const BackwardParams p) {
    using L = BackwardSmem<D>;
    constexpr int BT = kBwdTile;
    constexpr int NKK = D / 16;  // 16-channel steps
    constexpr int ND = D / 8;    // 8-channel output tiles

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sK = smem_base + L::kOffK, sV = smem_base + L::kOffV, sDS = smem_base + L::kOffDS;
    const uint32_t sQD = smem_base + L::kOffQ;  // buffer u: Q at sQD + u * 2 * tile, dO one tile further
    float* s_rows = reinterpret_cast<float*>(smem_gen + L::kOffRow);  // buffer u: lse2 at [u*128 .. +63], delta at [+64 ..]
    const uint32_t bar_kv = smem_base + L::kOffBar, bar_q0 = bar_kv + 8;  // bar_q0 + 8 * u
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + L::kOffBar + 24);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
    const int hk = blockIdx.y, b = blockIdx.z;
    // blockIdx.x -> (key tile, chunk of its query range): the tiles that hold sink keys meet every later query
    // tile, so their range is cut into chunks of kBwdChunkTiles query tiles handled by separate blocks
    int n_tile, chunk = -1;
    if ((int)blockIdx.x < p.sink_tiles * p.chunks) {
        n_tile = (int)blockIdx.x / p.chunks;
        chunk = (int)blockIdx.x - n_tile * p.chunks;
    } else {
        n_tile = p.sink_tiles + ((int)blockIdx.x - p.sink_tiles * p.chunks);
    }
    const int seq_start = p.cu_seqlens[b], Lseq = p.cu_seqlens[b + 1] - seq_start;
    const int j0 = n_tile * BT;
    if (Lseq <= 0 || Lseq > p.max_seqlen || j0 >= Lseq || seq_start < 0 || seq_start + Lseq > p.T) {
        if (tid == 0 && (Lseq < 0 || Lseq > p.max_seqlen || seq_start < 0 || seq_start + Lseq > p.T))
            record_device_error(SWAA_ERR_BAD_SEQLENS);
        return;
    }
    const bool full = p.is_full != 0;
    const int j1 = min(j0 + BT, Lseq) - 1;
    // query tiles that can see this key tile: the band above it; all later ones if it holds sink keys
    int m_lo = j0 / BT;
    int m_hi = (full || j0 < p.n_sink) ? (Lseq - 1) / BT
                                       : (int)(min((long long)Lseq - 1, (long long)j1 + p.window - 1) / BT);
    const bool split = chunk >= 0;  // dK, dV of this tile come from several blocks: accumulate in fp32
    if (split) {
        m_lo += chunk * kBwdChunkTiles;
        m_hi = min(m_hi, m_lo + kBwdChunkTiles - 1);
        if (m_lo > m_hi) return;
    }
    const int nm = m_hi - m_lo + 1, n_steps = nm * p.G;

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar_kv, 1u);
        mbar_init(bar_q0, 1u);
        mbar_init(bar_q0 + 8, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Loads of step s (query head hq = s / nm, query tile m = m_lo + s % nm) into buffer s & 1: Q and dO tiles by
    // TMA, the 64 row terms by 4-byte asynchronous copies (zero-filled past the end of the sequence).
    auto issue_step = [&](int s_) {
        const int u = s_ & 1, h_ = hk * p.G + s_ / nm, i0_ = (m_lo + s_ % nm) * BT;
        if (tid == 0) {
            const uint32_t dst = sQD + (uint32_t)u * 2u * L::kTileBytes, bq = bar_q0 + 8u * (uint32_t)u;
            mbar_arrive_expect_tx(bq, 2u * (uint32_t)L::kTileBytes);
#pragma unroll
            for (int pn = 0; pn < L::kPanels; ++pn) {
                tma_load_3d(dst + pn * L::kPanelBytes, &tm_q, pn * 64, h_, seq_start + i0_, bq);
                tma_load_3d(dst + L::kTileBytes + pn * L::kPanelBytes, &tm_do, pn * 64, h_, seq_start + i0_, bq);
            }
        }
        {
            const int r = tid & 63, i = i0_ + r;
            const float* src = (tid < 64 ? p.lse2 : p.delta) + (size_t)h_ * p.T + seq_start + (i < Lseq ? i : 0);
            const uint32_t dsts = smem_u32(s_rows + u * 128 + tid);
            const int nbytes = i < Lseq ? 4 : 0;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dsts), "l"(src), "r"(nbytes) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
    };
    if (tid == 0) {
        mbar_arrive_expect_tx(bar_kv, 2u * (uint32_t)L::kTileBytes);
#pragma unroll
        for (int pn = 0; pn < L::kPanels; ++pn) {
            tma_load_3d(sK + pn * L::kPanelBytes, &tm_k, pn * 64, hk, seq_start + j0, bar_kv);
            tma_load_3d(sV + pn * L::kPanelBytes, &tm_v, pn * 64, hk, seq_start + j0, bar_kv);
        }
    }
    issue_step(0);
    bool ok = __syncthreads_and(mbar_wait(bar_kv, 0u, abort_flag)) != 0;  // one decision for the whole block

    float dk_acc[ND][4], dv_acc[ND][4];
#pragma unroll
    for (int nd = 0; nd < ND; ++nd)
#pragma unroll
        for (int r = 0; r < 4; ++r) dk_acc[nd][r] = dv_acc[nd][r] = 0.f;

    const float sl2 = p.scale * 1.4426950408889634f;
    const int krow = 16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1);  // A fragments of K_w / V_w (non-transposed)
    const int kchk = lane >> 4;
    for (int step = 0; step < n_steps && ok; ++step) {
        {
            const int u = step & 1;
            const int h = hk * p.G + step / nm, i0 = (m_lo + step % nm) * BT;
            const uint32_t sQ = sQD + (uint32_t)u * 2u * L::kTileBytes, sDO = sQ + L::kTileBytes;
            const float* s_lse = s_rows + u * 128;
            const float* s_delta = s_lse + 64;
            // this step's tiles and row terms have landed; every warp is done with the previous step, whose
            // buffers (and dS^T) may now be refilled
            asm volatile("cp.async.wait_all;" ::: "memory");
            ok = __syncthreads_and(mbar_wait(bar_q0 + 8u * (uint32_t)u, (uint32_t)(step >> 1) & 1u, abort_flag)) != 0;
            if (!ok) break;
            if (step + 1 < n_steps) issue_step(step + 1);

            // ---- S^T = K_w Q^T and dP^T = V_w dO^T : [16 keys] x [64 rows]
            float st[8][4], dpt[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int r = 0; r < 4; ++r) st[nt][r] = dpt[nt][r] = 0.f;
#pragma unroll
            for (int kk = 0; kk < NKK; ++kk) {
                uint32_t ka0, ka1, ka2, ka3, va0, va1, va2, va3;
                ldmatrix_x4(bwd_tile_addr(sK, krow, 2 * kk + kchk), ka0, ka1, ka2, ka3);
                ldmatrix_x4(bwd_tile_addr(sV, krow, 2 * kk + kchk), va0, va1, va2, va3);
#pragma unroll
                for (int jp = 0; jp < 4; ++jp) {  // pairs of 8-row tiles of the query rows
                    const int row = 16 * jp + (lane & 7) + 8 * (lane >> 4), chk = 2 * kk + ((lane >> 3) & 1);
                    uint32_t q0, q1, q2, q3, o0, o1, o2, o3;
                    ldmatrix_x4(bwd_tile_addr(sQ, row, chk), q0, q1, q2, q3);
                    ldmatrix_x4(bwd_tile_addr(sDO, row, chk), o0, o1, o2, o3);
                    mma_bf16_16816(st[2 * jp], ka0, ka1, ka2, ka3, q0, q1);
                    mma_bf16_16816(st[2 * jp + 1], ka0, ka1, ka2, ka3, q2, q3);
                    mma_bf16_16816(dpt[2 * jp], va0, va1, va2, va3, o0, o1);
                    mma_bf16_16816(dpt[2 * jp + 1], va0, va1, va2, va3, o2, o3);
                }
            }
            // ---- P^T and dS^T (scaled) in the accumulator layout: keys (g, g+8) x rows (8nt + 2c, +1)
            uint32_t pT[8][2], dsT[8][2];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
                for (int kh = 0; kh < 2; ++kh) {
                    const int j = j0 + 16 * warp + g + 8 * kh;
                    float pv[2], dv2[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int r = 8 * nt + 2 * c + e, i = i0 + r;
                        const bool vis = i < Lseq && j <= i && (full || j > i - p.window || j < p.n_sink);
                        const float pr = vis ? ex2f(fmaf(st[nt][2 * kh + e], sl2, -s_lse[r])) : 0.f;
                        pv[e] = pr;
                        dv2[e] = pr * (dpt[nt][2 * kh + e] - s_delta[r]) * p.scale;
                    }
                    pT[nt][kh] = pack_bf16x2(pv[0], pv[1]);
                    dsT[nt][kh] = pack_bf16x2(dv2[0], dv2[1]);
                    // dS^T to shared memory for the dQ product: row = key, 16-byte chunk = nt, swizzled
                    const int key = 16 * warp + g + 8 * kh;
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(sDS + (uint32_t)(key * 128 + ((nt ^ (key & 7)) << 4) + 4 * c)),
                                 "r"(dsT[nt][kh])
                                 : "memory");
                }
            }
            // ---- dV_w += P^T dO,  dK_w += dS^T Q : [16 keys] x [D], contraction over the 64 rows
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const int row = 16 * ks + (lane & 7) + 8 * ((lane >> 3) & 1);
#pragma unroll
                for (int nd = 0; nd < ND; nd += 2) {
                    uint32_t o0, o1, o2, o3, q0, q1, q2, q3;
                    ldmatrix_x4_trans(bwd_tile_addr(sDO, row, nd + (lane >> 4)), o0, o1, o2, o3);
                    ldmatrix_x4_trans(bwd_tile_addr(sQ, row, nd + (lane >> 4)), q0, q1, q2, q3);
                    mma_bf16_16816(dv_acc[nd], pT[2 * ks][0], pT[2 * ks][1], pT[2 * ks + 1][0], pT[2 * ks + 1][1], o0, o1);
                    mma_bf16_16816(dv_acc[nd + 1], pT[2 * ks][0], pT[2 * ks][1], pT[2 * ks + 1][0], pT[2 * ks + 1][1], o2, o3);
                    mma_bf16_16816(dk_acc[nd], dsT[2 * ks][0], dsT[2 * ks][1], dsT[2 * ks + 1][0], dsT[2 * ks + 1][1], q0, q1);
                    mma_bf16_16816(dk_acc[nd + 1], dsT[2 * ks][0], dsT[2 * ks][1], dsT[2 * ks + 1][0], dsT[2 * ks + 1][1], q2, q3);
                }
            }
            __syncthreads();  // dS^T of all four warps is in shared memory
            // ---- dQ (rows 16w .. 16w+15) += dS K : contraction over the 64 keys; two halves of D to bound registers
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float dq_acc[ND / 2][4];
#pragma unroll
                for (int nd = 0; nd < ND / 2; ++nd)
#pragma unroll
                    for (int r = 0; r < 4; ++r) dq_acc[nd][r] = 0.f;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    uint32_t a0, a1, a2, a3;
                    {
                        const int key = 16 * ks + (lane & 7) + 8 * (lane >> 4), chk = 2 * warp + ((lane >> 3) & 1);
                        ldmatrix_x4_trans(sDS + (uint32_t)(key * 128 + ((chk ^ (key & 7)) << 4)), a0, a1, a2, a3);
                    }
                    const int krw = 16 * ks + (lane & 7) + 8 * ((lane >> 3) & 1);
#pragma unroll
                    for (int nd = 0; nd < ND / 2; nd += 2) {
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4_trans(bwd_tile_addr(sK, krw, half * (ND / 2) + nd + (lane >> 4)), b0, b1, b2, b3);
                        mma_bf16_16816(dq_acc[nd], a0, a1, a2, a3, b0, b1);
                        mma_bf16_16816(dq_acc[nd + 1], a0, a1, a2, a3, b2, b3);
                    }
                }
#pragma unroll
                for (int rh = 0; rh < 2; ++rh) {
                    const int i = i0 + 16 * warp + g + 8 * rh;
                    if (i < Lseq) {
                        float* dst = p.dq_accum + ((size_t)(seq_start + i) * p.Hq + h) * D + half * (D / 2) + 2 * c;
#pragma unroll
                        for (int nd = 0; nd < ND / 2; ++nd)
                            atomicAdd(reinterpret_cast<float2*>(dst + 8 * nd),
                                      make_float2(dq_acc[nd][2 * rh], dq_acc[nd][2 * rh + 1]));
                    }
                }
            }
        }
    }
    if (!ok) return;
    // ---- dK, dV rows of this warp's keys
    if (split) {
        const int sink_rows = p.sink_tiles * BT;
        const size_t plane = (size_t)p.B * sink_rows * p.Hkv * D;
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) {
            const int j = j0 + 16 * warp + g + 8 * kh;
            if (j < Lseq) {
                float* dkr = p.dkv_accum + (((size_t)b * sink_rows + j) * p.Hkv + hk) * D + 2 * c;
#pragma unroll
                for (int nd = 0; nd < ND; ++nd) {
                    atomicAdd(reinterpret_cast<float2*>(dkr + 8 * nd), make_float2(dk_acc[nd][2 * kh], dk_acc[nd][2 * kh + 1]));
                    atomicAdd(reinterpret_cast<float2*>(dkr + plane + 8 * nd),
                              make_float2(dv_acc[nd][2 * kh], dv_acc[nd][2 * kh + 1]));
                }
            }
        }
        return;
    }
#pragma unroll
    for (int kh = 0; kh < 2; ++kh) {
        const int j = j0 + 16 * warp + g + 8 * kh;
        if (j < Lseq) {
            __nv_bfloat16* dkr = p.dk + ((size_t)(seq_start + j) * p.Hkv + hk) * D + 2 * c;
            __nv_bfloat16* dvr = p.dv + ((size_t)(seq_start + j) * p.Hkv + hk) * D + 2 * c;
#pragma unroll
            for (int nd = 0; nd < ND; ++nd) {
                *reinterpret_cast<uint32_t*>(dkr + 8 * nd) = pack_bf16x2(dk_acc[nd][2 * kh], dk_acc[nd][2 * kh + 1]);
                *reinterpret_cast<uint32_t*>(dvr + 8 * nd) = pack_bf16x2(dv_acc[nd][2 * kh], dv_acc[nd][2 * kh + 1]);
            }
        }
    }
}

}  // namespace swaa
