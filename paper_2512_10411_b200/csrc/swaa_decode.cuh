// Split-K decode attention (one query token per sequence) -- HBM-bound.
//
// Sec. 3.1.1 ("FA Decode"): the generated token attends to every earlier token, so the kernel
// streams the whole KV cache of its sequence; an SWA decode step reads the first n_sink entries plus
// the last `window` entries only.  App. A: the full-context cache is retained for decoding.
//
// Work decomposition: one thread block per (key/value head, key split, sequence).  All G = Hq/Hkv
// query heads of the group are processed together so every K/V byte is read from HBM exactly once.
// The visible cache entries form one virtual index space [0, n_vis) = sinks ++ window, cut into blocks
// of 16 keys; a split owns a contiguous run of blocks and its four warps take them round-robin.
//
// Data path: each lane reads 16-byte pieces of K/V rows straight into registers (a warp covers whole
// 256-byte rows, so the loads are fully coalesced), and both contractions run on warp-level tensor
// core MMAs with fp32 accumulation in the transposed form
//     S^T[16 keys x 8 heads] = K[16 keys x D] * Q^T[D x 8 heads]
//     O^T[16 ch  x 8 heads] += V^T[16 ch x 16 keys] * P^T[16 keys x 8 heads]
// so that the small head count sits in the MMA's N = 8 dimension and no accumulator rows are wasted.
// The contraction index of the first product is a fixed permutation of the channels, chosen so that
// an A/B fragment register is exactly one 32-bit word of a 16-byte load (a dot product does not care
// about the order of its terms).  P^T reaches the second product's B fragment through movmatrix.
// Partial (max, sum, O) triples of the splits are merged by the last block to finish (atomic ticket).
#pragma once

#include "swaa_internal.cuh"

namespace swaa {

struct DecodeParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* kc;
    const __nv_bfloat16* vc;
    __nv_bfloat16* out;
    const int32_t* seqlens;
    int B, Lmax, Hq, Hkv, G;
    int HG;        // head chunks per kv head (each chunk holds up to 8*NH query heads)
    int window, n_sink, is_full;
    float sl2;     // softmax scale * log2(e)
    int nsplit;
    int* counters;     // [B * Hkv * HG] tickets, zeroed before the launch
    float* part_ml;    // [B, Hq, nsplit, 2]  (running max in score units, sum)
    float* part_o;     // [B, Hq, nsplit, D]  unnormalised
};

constexpr int kDecodeWarps = 4;
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kDecodeBlockKeys = 16;

__device__ __forceinline__ uint4 ld_stream16(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }

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

__device__ __forceinline__ uint32_t u4_word(const uint4& v, int i) {
    return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w));
}

// 16-bit element e (0..7) of two 16-byte pieces packed as (lo = a[e], hi = b[e]).
__device__ __forceinline__ uint32_t pair_elem(const uint4& a, const uint4& b, int e) {
    const uint32_t wa = u4_word(a, e >> 1), wb = u4_word(b, e >> 1);
    return (e & 1) ? __byte_perm(wa, wb, 0x7632) : __byte_perm(wa, wb, 0x5410);
}

template <int D, int NH>
__global__ void __launch_bounds__(kDecodeThreads, 2) decode_kernel(const DecodeParams p) {
    static_assert(D == 64 || D == 128, "head size");
    constexpr int NKI = D / 32;   // 16-byte pieces of one K row per lane
    constexpr int NCH = D / 64;   // 16-byte pieces of one V row per lane
    constexpr int NQ = D / 16;    // 16-channel M-blocks of O^T
    constexpr int HC = 8 * NH;    // query heads per chunk

    const int hv = blockIdx.x, split = blockIdx.y, b = blockIdx.z;
    const int hk = hv / p.HG, ch = hv - hk * p.HG;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
    const int h0 = hk * p.G + ch * HC;                 // first query head of this chunk
    const int gc = min(HC, p.G - ch * HC);             // heads in this chunk

    int len = p.seqlens[b];
    if (len < 1 || len > p.Lmax) {
        if (tid == 0) record_device_error(SWAA_ERR_BAD_SEQLENS);
        len = 0;
    }
    const int lo = p.is_full ? 0 : max(0, len - p.window);
    const int ns = p.is_full ? 0 : min(p.n_sink, lo);
    const int n_vis = ns + (len - lo);
    const int nblk = (n_vis + kDecodeBlockKeys - 1) / kDecodeBlockKeys;
    const int bps = (nblk + p.nsplit - 1) / p.nsplit;
    const int blk_begin = split * bps;
    const int blk_end = min(nblk, blk_begin + bps);

    const size_t row_stride = (size_t)p.Hkv * D;  // elements between consecutive cache entries
    const __nv_bfloat16* kbase = p.kc + ((size_t)b * p.Lmax * p.Hkv + hk) * D;
    const __nv_bfloat16* vbase = p.vc + ((size_t)b * p.Lmax * p.Hkv + hk) * D;
    auto key_of = [&](int v) -> size_t {  // virtual index -> cache entry (clamped to stay in bounds)
        v = min(v, n_vis - 1);
        return (size_t)(v < ns ? v : lo + (v - ns));
    };

    // Q^T fragments: lane (g, c) holds, for head g of each 8-head block, pieces 4i+c of the row.
    uint4 qf[NH][NKI];
#pragma unroll
    for (int nh = 0; nh < NH; ++nh) {
        const int hh = nh * 8 + g;
#pragma unroll
        for (int i = 0; i < NKI; ++i) {
            if (hh < gc)
                qf[nh][i] = *reinterpret_cast<const uint4*>(p.q + ((size_t)b * p.Hq + h0 + hh) * D + (4 * i + c) * 8);
            else
                qf[nh][i] = make_uint4(0, 0, 0, 0);
        }
    }

    float m_run[NH][2], l_run[NH][2], oacc[NH][NQ][4];
#pragma unroll
    for (int nh = 0; nh < NH; ++nh) {
        m_run[nh][0] = m_run[nh][1] = -INFINITY;
        l_run[nh][0] = l_run[nh][1] = 0.f;
#pragma unroll
        for (int qb = 0; qb < NQ; ++qb)
#pragma unroll
            for (int r = 0; r < 4; ++r) oacc[nh][qb][r] = 0.f;
    }

    uint4 kcur[2][NKI], vcur[4][NCH], knext[2][NKI], vnext[4][NCH];
    auto load_k = [&](int blk, uint4 (&kr)[2][NKI]) {
        const int v0 = blk * kDecodeBlockKeys;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const __nv_bfloat16* row = kbase + key_of(v0 + g + 8 * r) * row_stride;
#pragma unroll
            for (int i = 0; i < NKI; ++i) kr[r][i] = ld_stream16(row + (4 * i + c) * 8);
        }
    };
    auto load_v = [&](int blk, uint4 (&vr)[4][NCH]) {
        const int v0 = blk * kDecodeBlockKeys;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int slot = 2 * c + (r & 1) + 8 * (r >> 1);  // keys 2c, 2c+1, 2c+8, 2c+9
            const __nv_bfloat16* row = vbase + key_of(v0 + slot) * row_stride;
#pragma unroll
            for (int j = 0; j < NCH; ++j) vr[r][j] = ld_stream16(row + (g + 8 * j) * 8);
        }
    };

    int blk = blk_begin + warp;
    if (blk < blk_end) {
        load_k(blk, kcur);
        load_v(blk, vcur);
    }
    for (; blk < blk_end; blk += kDecodeWarps) {
        const int nxt = blk + kDecodeWarps;
        const bool has_next = nxt < blk_end;
        if (has_next) load_k(nxt, knext);

        // ---- S^T = K Q^T : rows = keys (g, g+8), cols = heads (2c, 2c+1)
        float sacc[NH][4];
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
            sacc[nh][0] = sacc[nh][1] = sacc[nh][2] = sacc[nh][3] = 0.f;
#pragma unroll
            for (int i = 0; i < NKI; ++i) {
                mma_bf16_16816(sacc[nh], kcur[0][i].x, kcur[1][i].x, kcur[0][i].y, kcur[1][i].y, qf[nh][i].x,
                               qf[nh][i].y);
                mma_bf16_16816(sacc[nh], kcur[0][i].z, kcur[1][i].z, kcur[0][i].w, kcur[1][i].w, qf[nh][i].z,
                               qf[nh][i].w);
            }
        }
        if (has_next) load_v(nxt, vnext);

        // ---- online softmax over the 16 keys of this block
        const int v0 = blk * kDecodeBlockKeys;
        const bool ok0 = v0 + g < n_vis, ok1 = v0 + g + 8 < n_vis;
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
                const float m_new = fmaxf(m_run[nh][e], bm);  // finite: key v0 is always valid
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
                for (int qb = 0; qb < NQ; ++qb) {
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

        // ---- O^T += V^T P^T : rows = channels, cols = heads
#pragma unroll
        for (int qb = 0; qb < NQ; ++qb) {
            uint32_t a0, a1, a2, a3;
            if (D == 128) {  // rows g -> channel 8g+qb (piece g), rows g+8 -> channel 8(g+8)+qb (piece g+8)
                a0 = pair_elem(vcur[0][0], vcur[1][0], qb);
                a1 = pair_elem(vcur[0][NCH - 1], vcur[1][NCH - 1], qb);
                a2 = pair_elem(vcur[2][0], vcur[3][0], qb);
                a3 = pair_elem(vcur[2][NCH - 1], vcur[3][NCH - 1], qb);
            } else {         // one piece per row: rows g -> channel 8g+qb, rows g+8 -> channel 8g+4+qb
                a0 = pair_elem(vcur[0][0], vcur[1][0], qb);
                a1 = pair_elem(vcur[0][0], vcur[1][0], qb + 4);
                a2 = pair_elem(vcur[2][0], vcur[3][0], qb);
                a3 = pair_elem(vcur[2][0], vcur[3][0], qb + 4);
            }
#pragma unroll
            for (int nh = 0; nh < NH; ++nh) mma_bf16_16816(oacc[nh][qb], a0, a1, a2, a3, pb[nh][0], pb[nh][1]);
        }

        if (has_next) {
#pragma unroll
            for (int r = 0; r < 2; ++r)
#pragma unroll
                for (int i = 0; i < NKI; ++i) kcur[r][i] = knext[r][i];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int j = 0; j < NCH; ++j) vcur[r][j] = vnext[r][j];
        }
    }

    // ---- merge the four warps of the block through shared memory
    __shared__ float sm_m[kDecodeWarps][HC], sm_l[kDecodeWarps][HC];
    __shared__ float sm_o[kDecodeWarps][HC][D + 1];
    __shared__ int sm_last;
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
                sm_m[warp][hh] = m_run[nh][e];
                sm_l[warp][hh] = l;
            }
#pragma unroll
            for (int qb = 0; qb < NQ; ++qb) {
                const int dA = (D == 128) ? 8 * g + qb : 8 * g + qb;
                const int dB = (D == 128) ? 8 * (g + 8) + qb : 8 * g + 4 + qb;
                sm_o[warp][hh][dA] = oacc[nh][qb][e];
                sm_o[warp][hh][dB] = oacc[nh][qb][2 + e];
            }
        }
    }
    __syncthreads();

    const bool direct = p.nsplit == 1;
    for (int idx = tid; idx < gc * D; idx += kDecodeThreads) {
        const int hh = idx / D, d = idx - hh * D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) M = fmaxf(M, sm_m[w][hh]);
        float den = 0.f, num = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            const float wgt = sm_m[w][hh] == -INFINITY ? 0.f : ex2f((sm_m[w][hh] - M) * p.sl2);
            den += wgt * sm_l[w][hh];
            num += wgt * sm_o[w][hh][d];
        }
        const size_t row = (size_t)b * p.Hq + h0 + hh;
        if (direct) {
            p.out[row * D + d] = __float2bfloat16_rn(den > 0.f ? num / den : 0.f);
        } else {
            p.part_o[(row * p.nsplit + split) * D + d] = num;
            if (d == 0) {
                p.part_ml[(row * p.nsplit + split) * 2 + 0] = M;
                p.part_ml[(row * p.nsplit + split) * 2 + 1] = den;
            }
        }
    }
    if (direct) return;

    // ---- the last block of this (sequence, head chunk) to arrive merges the splits
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(&p.counters[b * gridDim.x + hv], 1);
        sm_last = (ticket == p.nsplit - 1);
    }
    __syncthreads();
    if (!sm_last) return;
    __threadfence();
    for (int idx = tid; idx < gc * D; idx += kDecodeThreads) {
        const int hh = idx / D, d = idx - hh * D;
        const size_t row = (size_t)b * p.Hq + h0 + hh;
        const float* ml = p.part_ml + row * p.nsplit * 2;
        float M = -INFINITY;
        for (int s = 0; s < p.nsplit; ++s) M = fmaxf(M, __ldcg(ml + 2 * s));
        float den = 0.f, num = 0.f;
        for (int s = 0; s < p.nsplit; ++s) {
            const float ms = __ldcg(ml + 2 * s);
            const float wgt = ms == -INFINITY ? 0.f : ex2f((ms - M) * p.sl2);
            den += wgt * __ldcg(ml + 2 * s + 1);
            num += wgt * __ldcg(p.part_o + (row * p.nsplit + s) * D + d);
        }
        p.out[row * D + d] = __float2bfloat16_rn(den > 0.f ? num / den : 0.f);
    }
}

}  // namespace swaa
