// Backward pass of the prefill attention under the same mask policy (for SWA-aware fine-tuning, Sec. 3.3:
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
// One thread block owns one 64-key tile of one (sequence, key/value head) and keeps its dK and dV in
// registers; it walks the query heads of the group and, per head, only the 64-row query tiles that can
// see the key tile (the band above it, plus every later tile when the key tile holds sink keys), so the
// work is O(L * window) like the forward pass (App. A).  Each of the four warps owns 16 keys: it forms
// S^T = K Q^T, P^T, dP^T = V dO^T and dS^T for its keys against the 64 query rows with warp-level
// tensor-core MMAs (fp32 accumulation), feeds P^T and dS^T straight back as A operands for
// dV += P^T dO and dK += dS^T Q, and leaves dS^T in shared memory, from where every warp takes the 16
// query rows it owns to form dQ += dS K; dQ is accumulated across key tiles in an fp32 buffer with
// atomic adds and converted to bf16 by a second kernel.  Tiles are staged by TMA (128-byte swizzle).
#pragma once

#include "swaa_internal.cuh"
#include "swaa_ptx.cuh"
#include "swaa_decode.cuh"  // mma_bf16_16816

namespace swaa {

struct BackwardParams {
    const float* lse;        // [Hq, T] natural log
    const float* delta;      // [Hq, T]
    float* dq_accum;         // [T, Hq, D] fp32, zeroed before the launch
    __nv_bfloat16* dk;       // [T, Hkv, D]
    __nv_bfloat16* dv;
    const int32_t* cu_seqlens;
    int B, T, Hq, Hkv, G;
    int window, n_sink, is_full;
    float scale;
};

constexpr int kBwdTile = 64;      // keys per block and query rows per step
constexpr int kBwdThreads = 128;  // four warps, 16 keys each

template <int D>
struct BackwardSmem {
    static constexpr int kPanels = D / 64;
    static constexpr int kPanelBytes = kBwdTile * 128;
    static constexpr int kTileBytes = kPanels * kPanelBytes;  // one [64][D] bf16 tile
    static constexpr int kOffK = 0, kOffV = kTileBytes, kOffQ = 2 * kTileBytes, kOffDO = 3 * kTileBytes;
    static constexpr int kOffDS = 4 * kTileBytes;             // dS^T [64 keys][64 rows] bf16, 128-byte rows, swizzled
    static constexpr int kOffRow = kOffDS + kBwdTile * 128;   // lse, delta of the 64 rows (fp32)
    static constexpr int kOffBar = kOffRow + 2 * kBwdTile * 4;
    static constexpr int kBytes = kOffBar + 2 * 8 + 16;
    static constexpr int kDynamicBytes = kBytes + 1024;
};

// delta[h, t] = sum_d out[t, h, d] * dout[t, h, d]; one warp per (t, h).
template <int D>
__global__ void backward_delta_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                                      float* __restrict__ delta, int T, int Hq) {
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
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) delta[(size_t)h * T + t] = acc;
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
    const uint32_t sK = smem_base + L::kOffK, sV = smem_base + L::kOffV, sQ = smem_base + L::kOffQ;
    const uint32_t sDO = smem_base + L::kOffDO, sDS = smem_base + L::kOffDS;
    float* s_lse = reinterpret_cast<float*>(smem_gen + L::kOffRow);
    float* s_delta = s_lse + BT;
    const uint32_t bar_kv = smem_base + L::kOffBar, bar_q = bar_kv + 8;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + L::kOffBar + 16);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
    const int n_tile = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int seq_start = p.cu_seqlens[b], Lseq = p.cu_seqlens[b + 1] - seq_start;
    const int j0 = n_tile * BT;
    if (Lseq <= 0 || j0 >= Lseq || seq_start < 0 || seq_start + Lseq > p.T) {
        if (tid == 0 && (Lseq < 0 || seq_start < 0 || seq_start + Lseq > p.T)) record_device_error(SWAA_ERR_BAD_SEQLENS);
        return;
    }
    const bool full = p.is_full != 0;
    const int j1 = min(j0 + BT, Lseq) - 1;
    // query tiles that can see this key tile: the band above it; all later ones if it holds sink keys
    const int m_lo = j0 / BT;
    const int m_hi = (full || j0 < p.n_sink) ? (Lseq - 1) / BT
                                             : (int)(min((long long)Lseq - 1, (long long)j1 + p.window - 1) / BT);

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar_kv, 1u);
        mbar_init(bar_q, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        mbar_arrive_expect_tx(bar_kv, 2u * (uint32_t)L::kTileBytes);
#pragma unroll
        for (int pn = 0; pn < L::kPanels; ++pn) {
            tma_load_3d(sK + pn * L::kPanelBytes, &tm_k, pn * 64, hk, seq_start + j0, bar_kv);
            tma_load_3d(sV + pn * L::kPanelBytes, &tm_v, pn * 64, hk, seq_start + j0, bar_kv);
        }
    }
    bool ok = __syncthreads_and(mbar_wait(bar_kv, 0u, abort_flag)) != 0;  // one decision for the whole block

    float dk_acc[ND][4], dv_acc[ND][4];
#pragma unroll
    for (int nd = 0; nd < ND; ++nd)
#pragma unroll
        for (int r = 0; r < 4; ++r) dk_acc[nd][r] = dv_acc[nd][r] = 0.f;

    const float sl2 = p.scale * 1.4426950408889634f;
    const int krow = 16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1);  // A fragments of K_w / V_w (non-transposed)
    const int kchk = lane >> 4;
    uint32_t step = 0;
    for (int hq = 0; hq < p.G && ok; ++hq) {
        const int h = hk * p.G + hq;
        for (int m = m_lo; m <= m_hi && ok; ++m, ++step) {
            const int i0 = m * BT;
            __syncthreads();  // everybody is done with the previous Q, dO, dS^T and row data
            if (tid == 0) {
                mbar_arrive_expect_tx(bar_q, 2u * (uint32_t)L::kTileBytes);
#pragma unroll
                for (int pn = 0; pn < L::kPanels; ++pn) {
                    tma_load_3d(sQ + pn * L::kPanelBytes, &tm_q, pn * 64, h, seq_start + i0, bar_q);
                    tma_load_3d(sDO + pn * L::kPanelBytes, &tm_do, pn * 64, h, seq_start + i0, bar_q);
                }
            }
            if (tid < BT) {
                const int i = i0 + tid;
                s_lse[tid] = i < Lseq ? p.lse[(size_t)h * p.T + seq_start + i] * 1.4426950408889634f : 0.f;
                s_delta[tid] = i < Lseq ? p.delta[(size_t)h * p.T + seq_start + i] : 0.f;
            }
            ok = __syncthreads_and(mbar_wait(bar_q, step & 1u, abort_flag)) != 0;  // also publishes the row data
            if (!ok) break;

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
