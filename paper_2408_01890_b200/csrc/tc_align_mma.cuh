// Warp-level pieces of the head-axis aligner (Sec. 5.1) on mma.sync: one link of the FFN applied to 16 (query, key)
// positions held as register fragments, and the weight-fragment images it reads.  Shared by the stand-alone aligner
// kernel (tc_align.cu) and the fused score kernel (tc_scores.cu).  Hq = 32 heads, hidden width 64, two-layer FFNs.
#pragma once
#include "common.cuh"
#include "tc_common.cuh"

namespace lisa {
namespace alignmma {

using namespace tc;

constexpr int HQ = 32, MH = 64;
constexpr int W1F_BYTES = 2 * 8 * 32 * 8;     // B fragments of W1: [k-step][n-tile][lane] x (b0, b1)
constexpr int W2F_BYTES = 4 * 4 * 32 * 8;     // B fragments of W2
constexpr int LINK_BYTES = W1F_BYTES + W2F_BYTES + (MH + HQ) * 4;   // + b1 as 32 packed fp16 pairs (padded to 64 words), b2[32] fp32
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ldw(const void* p, int idx, int dtype) { return p ? ld_elem(p, idx, dtype) : 0.f; }

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t* r, uint32_t saddr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr) : "memory");
}
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t saddr, const uint32_t* r) {
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1,%2,%3,%4};"
                 ::"r"(saddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
// d += a (16x16, row) . b (16x8, col), fp16 in, fp32 accumulate
__device__ __forceinline__ void mma_f16(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// d = a (16x16, row) . b (16x8, col) + c with fp16 accumulators: the two result registers hold rows g and g+8 as
// packed pairs of columns (2t, 2t+1), which is exactly the A-fragment arrangement of a following MMA.
__device__ __forceinline__ void mma_f16acc(uint32_t* d, const uint32_t* a, uint32_t b0, uint32_t b1, uint32_t c0, uint32_t c1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f16.f16.f16.f16 {%0,%1}, {%2,%3,%4,%5}, {%6,%7}, {%8,%9};"
                 : "=r"(d[0]), "=r"(d[1])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(c0), "r"(c1));
}
// d = a . b + c, fp32 accumulators, c given separately (a bias pair repeated for both rows)
__device__ __forceinline__ void mma_f16_bias(float* d, const uint32_t* a, uint32_t b0, uint32_t b1, float c0, float c1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%10,%11};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c0), "f"(c1));
}

// Activation of two hidden units held as a packed fp16 pair; the result is again a packed pair (an A-fragment
// register of the second layer's MMA).
template <int ACT>
__device__ __forceinline__ uint32_t act_h2(uint32_t x) {
    if constexpr (ACT == LISA_ACT_RELU) {
        uint32_t r;
        asm("max.f16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(0u));
        return r;
    }
    if constexpr (ACT == LISA_ACT_SILU) {
        // x * sigmoid(x) = (x/2) tanh(x/2) + x/2: one packed multiply, one packed tanh, one packed fused multiply-add
        uint32_t hx, th, r;
        asm("mul.f16x2 %0, %1, %2;" : "=r"(hx) : "r"(x), "r"(0x38003800u));   // 0.5, 0.5
        asm("tanh.approx.f16x2 %0, %1;" : "=r"(th) : "r"(hx));
        asm("fma.rn.f16x2 %0, %1, %2, %1;" : "=r"(r) : "r"(hx), "r"(th));
        return r;
    }
    return x;
}

// One link on a warp's 16 positions: afr = A fragments (2 k-steps of 16 heads) -> y = W2^T act(W1^T a + b1) + b2
// as four accumulator tiles of 8 heads.  The first layer accumulates in fp16 (32 products per hidden unit, the
// result is rounded to fp16 for the second layer's operand in any case): its accumulator registers ARE the second
// layer's A fragments, so the activation is one to three packed instructions per register and nothing is converted
// or repacked.  The second layer accumulates in fp32.  b1h holds b1 as packed fp16 pairs, b2 is fp32.
// The fragments of W1 and W2 come either from shared memory (w1f/w2f, one 8-byte load per MMA) or, when REGW, from
// the register copies w1r/w2r that a warp keeps for its whole life (single-link calls).
// `side` is called once, after the first layer's MMAs have been issued: unrelated instructions placed there (the copies
// of neighbouring pieces) issue while this warp's MMAs wait for their turn on the tensor pipe.
// BIAS = false: b1 and b2 are known to be absent (zero accumulator start, nothing loaded).
template <int ACT, bool REGW, bool BIAS = true, typename Side>
__device__ __forceinline__ void ffn_link(const uint32_t (*afr)[4], const uint2* w1f, const uint2* w2f, const uint2* w1r, const uint2* w2r,
                                         const uint32_t* b1h, const float* b2, int lane, float (*y)[4], Side side) {
    const int t = lane & 3;
    uint32_t h[8][2];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t bb = BIAS ? b1h[j * 4 + t] : 0u;
        const uint2 w = REGW ? w1r[j] : w1f[j * 32 + lane];
        mma_f16acc(h[j], afr[0], w.x, w.y, bb, bb);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint2 w = REGW ? w1r[8 + j] : w1f[(8 + j) * 32 + lane];
        mma_f16acc(h[j], afr[1], w.x, w.y, h[j][0], h[j][1]);
    }
    side();
    uint32_t hfr[4][4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        hfr[s][0] = act_h2<ACT>(h[2 * s][0]);
        hfr[s][1] = act_h2<ACT>(h[2 * s][1]);
        hfr[s][2] = act_h2<ACT>(h[2 * s + 1][0]);
        hfr[s][3] = act_h2<ACT>(h[2 * s + 1][1]);
    }
#pragma unroll
    for (int j2 = 0; j2 < 4; ++j2) {
        const float2 bb = BIAS ? *reinterpret_cast<const float2*>(b2 + j2 * 8 + 2 * t) : make_float2(0.f, 0.f);
        const uint2 w = REGW ? w2r[j2] : w2f[j2 * 32 + lane];
        mma_f16_bias(y[j2], hfr[0], w.x, w.y, bb.x, bb.y);
    }
#pragma unroll
    for (int s = 1; s < 4; ++s)
#pragma unroll
        for (int j2 = 0; j2 < 4; ++j2) {
            const uint2 w = REGW ? w2r[s * 4 + j2] : w2f[(s * 4 + j2) * 32 + lane];
            mma_f16(y[j2], hfr[s], w.x, w.y);
        }
}


// The same link on NSTR strips of 16 positions at once, weights from shared memory: each 8-byte weight fragment is
// loaded once and feeds NSTR MMAs.  With one strip the shared-memory pipe moves 256 bytes per MMA, which at the MMA
// rate of the SM is about all it can deliver; two strips halve that.
template <int ACT, bool BIAS, int NSTR>
__device__ __forceinline__ void ffn_link_strips(const uint32_t (*afr)[2][4], const uint2* w1f, const uint2* w2f, const uint32_t* b1h,
                                                const float* b2, int lane, float (*y)[4][4]) {
    const int t = lane & 3;
    uint32_t h[NSTR][8][2];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t bb = BIAS ? b1h[j * 4 + t] : 0u;
        const uint2 w = w1f[j * 32 + lane];
#pragma unroll
        for (int s = 0; s < NSTR; ++s) mma_f16acc(h[s][j], afr[s][0], w.x, w.y, bb, bb);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint2 w = w1f[(8 + j) * 32 + lane];
#pragma unroll
        for (int s = 0; s < NSTR; ++s) mma_f16acc(h[s][j], afr[s][1], w.x, w.y, h[s][j][0], h[s][j][1]);
    }
#pragma unroll
    for (int s = 0; s < NSTR; ++s)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            h[s][j][0] = act_h2<ACT>(h[s][j][0]);
            h[s][j][1] = act_h2<ACT>(h[s][j][1]);
        }
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
#pragma unroll
        for (int j2 = 0; j2 < 4; ++j2) {
            const uint2 w = w2f[(ks * 4 + j2) * 32 + lane];
#pragma unroll
            for (int s = 0; s < NSTR; ++s) {
                const uint32_t hfr[4] = {h[s][2 * ks][0], h[s][2 * ks][1], h[s][2 * ks + 1][0], h[s][2 * ks + 1][1]};
                if (ks == 0) {
                    const float2 bb = BIAS ? *reinterpret_cast<const float2*>(b2 + j2 * 8 + 2 * t) : make_float2(0.f, 0.f);
                    mma_f16_bias(y[s][j2], hfr, w.x, w.y, bb.x, bb.y);
                } else {
                    mma_f16(y[s][j2], hfr, w.x, w.y);
                }
            }
        }
}


// What a link's FFN is, as far as this 32 -> 64 -> 32 two-layer engine is concerned.  The variants without a hidden
// layer run on the same engine with an identity first layer (exact: every hidden unit is one fp16 input times one):
//   KIND_FFN     y = W2^T act(W1^T a + b1) + b2                       (Sec. 5.1, two-layer FFN, m = 64)
//   KIND_SINGLE  y = W1^T a + b1, W1 [32, 32]                         (one linear layer, no activation)
//   KIND_PLUS    y = a                                                 (no FFN: A_n = A_{n-1} + A_Delta)
constexpr int KIND_FFN = 0, KIND_SINGLE = 1, KIND_PLUS = 2;

__host__ __device__ inline int link_kind(int integrate, int ffn_layers) {
    return integrate == LISA_INTEGRATE_PLUS ? KIND_PLUS : (ffn_layers == 1 ? KIND_SINGLE : KIND_FFN);
}

// All nthreads threads of a CTA: one link's weights as ready-made B fragments in shared memory at `dst` (LINK_BYTES):
// W1 fragments, W2 fragments (times out_scale), b1 as packed fp16 pairs, b2 (times out_scale) as fp32.
__device__ __forceinline__ void stage_link_fragments(uint8_t* dst, const void* w1, const void* b1, const void* w2, const void* b2, int wd,
                                                     int kind, float out_scale, int tid, int nthreads) {
    uint2* w1f = reinterpret_cast<uint2*>(dst);
    uint2* w2f = reinterpret_cast<uint2*>(dst + W1F_BYTES);
    float* bias = reinterpret_cast<float*>(dst + W1F_BYTES + W2F_BYTES);
    // first layer [32 heads][64 hidden] and second layer [64 hidden][32 heads] as this link's kind defines them
    auto first = [&](int k, int n) -> float { return kind == KIND_FFN ? ld_elem(w1, k * MH + n, wd) : (k == n ? 1.f : 0.f); };
    auto second = [&](int k, int n) -> float {
        if (kind == KIND_FFN) return ld_elem(w2, k * HQ + n, wd);
        if (kind == KIND_SINGLE) return k < HQ ? ld_elem(w1, k * HQ + n, wd) : 0.f;
        return k == n ? 1.f : 0.f;
    };
    for (int e = tid; e < 2 * 8 * 32; e += nthreads) {   // k = head, n = hidden
        const int ln = e & 31, j = (e >> 5) & 7, ks = e >> 8, g = ln >> 2, t = ln & 3;
        const int k0 = ks * 16 + 2 * t, n = j * 8 + g;
        uint2 w;
        w.x = pack_f16(first(k0, n), first(k0 + 1, n));
        w.y = pack_f16(first(k0 + 8, n), first(k0 + 9, n));
        w1f[e] = w;
    }
    for (int e = tid; e < 4 * 4 * 32; e += nthreads) {   // k = hidden, n = head
        const int ln = e & 31, j2 = (e >> 5) & 3, s2 = e >> 7, g = ln >> 2, t = ln & 3;
        const int k0 = s2 * 16 + 2 * t, n = j2 * 8 + g;
        uint2 w;
        w.x = pack_f16(second(k0, n) * out_scale, second(k0 + 1, n) * out_scale);
        w.y = pack_f16(second(k0 + 8, n) * out_scale, second(k0 + 9, n) * out_scale);
        w2f[e] = w;
    }
    for (int e = tid; e < MH / 2; e += nthreads)   // b1 as packed fp16 pairs (the first layer's accumulator format)
        reinterpret_cast<uint32_t*>(bias)[e] = kind == KIND_FFN ? pack_f16(ldw(b1, 2 * e, wd), ldw(b1, 2 * e + 1, wd)) : 0u;
    for (int e = tid; e < HQ; e += nthreads)
        bias[MH + e] = (kind == KIND_FFN ? ldw(b2, e, wd) : (kind == KIND_SINGLE ? ldw(b1, e, wd) : 0.f)) * out_scale;
}

// Byte offset of 16-byte chunk `chunk` (0..7) of head `head` inside a [32 heads][64 positions] fp16 piece (one 128-byte line
// per head, chunk index XOR-ed with the head so that the eight rows of an 8x8 matrix fall into distinct banks).
__device__ __forceinline__ uint32_t piece_off64(int head, int chunk) { return (uint32_t)(head * 128 + ((chunk ^ (head & 7)) << 4)); }

}  // namespace alignmma
}  // namespace lisa
