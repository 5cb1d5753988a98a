// Decode step of a shared layer (Sec. 5.2, decoding stage) and of a standard layer (Eq. 1-2, last row).
//
// Both are streaming scans over a cache, bound by HBM bandwidth.  Work is split over (sequence b,
// chunk of 128 cached positions); a CTA handles ALL heads of its chunk because the aligner mixes heads:
//   phase A  scores of the chunk for every head
//            shared:   A[:,j] = W2^T act(W1^T prev[:,j] + b1) + b2 + q'.K'_j/sqrt(r)     (Eq. 3-4)
//            standard: A[h,j] = q_h.K_j/sqrt(d)                                           (Eq. 2)
//            and, if asked, the fp32 row handed to the next shared layer
//   phase B  chunk-local softmax statistics (max, sum) per head and the partial product with V
// A second kernel merges the per-chunk partials (m, l, o) into the output (split-K softmax).
// K' is cached transposed ([r][L_cap], position contiguous) so that r = 21 needs no padding and every
// load is a full 16-byte vector along the position axis; V rows are 256 contiguous bytes.
#include "common.cuh"

namespace lisa {
namespace {

constexpr int kChunk = 128;
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct DecodeParams {
    int B, Hq, Hkv, d, L_cap, L_uniform, n_chunks;
    const int32_t* seq_lens;
    // shared layer
    const void* prev;       // fp32, or bf16 when row_bf16
    int64_t prev_sb, prev_sh;
    TView qp;
    const void* kpT;
    int r, m, act, integrate, ffn_layers, w_dtype;
    const void *w1, *b1, *w2, *b2;
    // standard layer
    TView q;
    const void* kcache;
    // common
    const void* vcache;
    int cache_dtype;
    void* out_scores;       // fp32, or bf16 when row_bf16
    int64_t sc_sb, sc_sh;
    int row_bf16;           // the score rows handed between layers are bf16 (Sec. 5.2 counts them at 2 bytes) instead of fp32
    float *ws_m, *ws_l, *ws_o;
    TView o;
};

// Score-row access: RB = rows are bf16.
template <bool RB>
__device__ __forceinline__ float ld_row(const void* p, int64_t i) {
    if constexpr (RB) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i]);
    else return reinterpret_cast<const float*>(p)[i];
}
template <bool RB>
__device__ __forceinline__ void st_row(void* p, int64_t i, float v) {
    if constexpr (RB) reinterpret_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(p)[i] = v;
}

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
}

__device__ __forceinline__ float ldw(const void* p, int idx, int dtype) { return p ? ld_elem(p, idx, dtype) : 0.f; }

__device__ __forceinline__ uint32_t f32_to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
// d += a (16x8, row) . b (8x8, col), tf32 in, fp32 accumulate
__device__ __forceinline__ void mma_tf32(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Partial P.V of a FULL chunk (all kChunk rows valid), bf16 cache, LPR = d/8 lanes per V row.  A warp streams the
// V rows of its heads as one software-pipelined sequence: two register sets of eight 16-byte loads per lane
// alternate, and the last batch of a head already prefetches the first batch of the warp's next head, so loads
// stay in flight across batches and across heads.  All offsets are compile-time constants off one pointer.
template <int LPR>
__device__ __forceinline__ void pv_full_chunk(const DecodeParams& p, const float* s_s, int b, size_t part, int j0) {
    constexpr int RSTEP = 32 / LPR;            // rows fetched by one warp-wide load
    constexpr int NB = kChunk / RSTEP / 8;     // batches of 8 loads per head (even)
    constexpr int D = LPR * 8;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane % LPR, rsel = lane / LPR;
    const int Hq = p.Hq, G = p.Hq / p.Hkv;
    auto head_ptr = [&](int h) {
        return reinterpret_cast<const uint4*>(p.vcache) + (((size_t)b * p.Hkv + h / G) * p.L_cap + j0 + rsel) * LPR + sub;
    };
    if (warp >= Hq) return;
    const uint4* hp = head_ptr(warp);
    uint4 ra[8], rb[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) ra[u] = ld_stream16(hp + u * RSTEP * LPR);
    for (int h = warp; h < Hq; h += kWarps) {
        const bool has_next = h + kWarps < Hq;
        const uint4* np = has_next ? head_ptr(h + kWarps) : hp;
        const float* ps = s_s + h * kChunk + rsel;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int bi = 0; bi < NB; bi += 2) {
#pragma unroll
            for (int u = 0; u < 8; ++u) rb[u] = ld_stream16(hp + ((bi + 1) * 8 + u) * RSTEP * LPR);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                float f[8];
                bf16x8_to_f32(ra[u], f);
                const float pj = ps[(bi * 8 + u) * RSTEP];
#pragma unroll
                for (int t = 0; t < 8; ++t) acc[t] = fmaf(pj, f[t], acc[t]);
            }
            if (bi + 2 < NB) {
#pragma unroll
                for (int u = 0; u < 8; ++u) ra[u] = ld_stream16(hp + ((bi + 2) * 8 + u) * RSTEP * LPR);
            } else if (has_next) {
#pragma unroll
                for (int u = 0; u < 8; ++u) ra[u] = ld_stream16(np + u * RSTEP * LPR);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                float f[8];
                bf16x8_to_f32(rb[u], f);
                const float pj = ps[((bi + 1) * 8 + u) * RSTEP];
#pragma unroll
                for (int t = 0; t < 8; ++t) acc[t] = fmaf(pj, f[t], acc[t]);
            }
        }
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
            for (int t = 0; t < 8; ++t) acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], off);
        if (rsel == 0) {
            float4* dst = reinterpret_cast<float4*>(p.ws_o + (part + h) * D + sub * 8);
            dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
            dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
        }
        hp = np;
    }
}

// ---------------------------------------------------------------------------------------------
// Phase B: s_s[h][kChunk] holds the chunk's scores (-inf beyond the sequence end). Produces the
// chunk's (max, sum, unnormalised P.V) per head into the workspace.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void softmax_pv_chunk(const DecodeParams& p, float* s_s, int b, int chunk, int nrows) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Hq = p.Hq, d = p.d, G = p.Hq / p.Hkv;
    const size_t part = ((size_t)b * p.n_chunks + chunk) * Hq;
    for (int h = warp; h < Hq; h += kWarps) {
        float v[kChunk / 32];
        float cmax = -INFINITY;
#pragma unroll
        for (int t = 0; t < kChunk / 32; ++t) {
            v[t] = s_s[h * kChunk + lane + 32 * t];
            cmax = fmaxf(cmax, v[t]);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, off));
        float sum = 0.f;
#pragma unroll
        for (int t = 0; t < kChunk / 32; ++t) {
            const float e = __expf(v[t] - cmax);
            s_s[h * kChunk + lane + 32 * t] = e;
            sum += e;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (lane == 0) {
            p.ws_m[part + h] = cmax;
            p.ws_l[part + h] = sum;
        }
    }
    __syncthreads();
    const int j0 = chunk * kChunk;
    if (p.cache_dtype == LISA_BF16) {
        if (nrows == kChunk) {
            if (d == 128) pv_full_chunk<16>(p, s_s, b, part, j0);
            else if (d == 64) pv_full_chunk<8>(p, s_s, b, part, j0);
            else pv_full_chunk<4>(p, s_s, b, part, j0);
        } else {
            // ragged last chunk of a sequence: plain loop
            const int lpr = d / 8, rstep = 32 / lpr, sub = lane % lpr, rsel = lane / lpr;
            for (int h = warp; h < Hq; h += kWarps) {
                const uint4* vbase = reinterpret_cast<const uint4*>(p.vcache) +
                                     (((size_t)b * p.Hkv + h / G) * p.L_cap + j0) * lpr + sub;
                const float* ps = s_s + h * kChunk;
                float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                for (int jj = rsel; jj < nrows; jj += rstep) {
                    float f[8];
                    bf16x8_to_f32(ld_stream16(vbase + (size_t)jj * lpr), f);
                    const float pj = ps[jj];
#pragma unroll
                    for (int t = 0; t < 8; ++t) acc[t] = fmaf(pj, f[t], acc[t]);
                }
                for (int off = lpr; off < 32; off <<= 1)
#pragma unroll
                    for (int t = 0; t < 8; ++t) acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], off);
                if (rsel == 0) {
                    float4* dst = reinterpret_cast<float4*>(p.ws_o + (part + h) * d + sub * 8);
                    dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
                    dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
                }
            }
        }
    } else {
        // fp32 cache: thread per output column
        for (int e = tid; e < Hq * d; e += kThreads) {
            const int h = e / d, x = e % d;
            const float* vb = reinterpret_cast<const float*>(p.vcache) + (((size_t)b * p.Hkv + h / G) * p.L_cap + j0) * d + x;
            float acc = 0.f;
            for (int jj = 0; jj < nrows; ++jj) acc = fmaf(s_s[h * kChunk + jj], vb[(size_t)jj * d], acc);
            p.ws_o[(part + h) * d + x] = acc;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Shared layer.  HQ_C/M_C > 0: compile-time sizes, aligner on the tensor cores (ADD, two layers, bf16 cache,
// M_C % 8 == 0, HQ_C % 8 == 0).  HQ_C == 0: any supported mode and size, per-thread scratch arrays.
// ---------------------------------------------------------------------------------------------
// CTAS: CTAs per SM the kernel is compiled for.  Three hide the FFN phase (no loads in flight from the CTA that is in it)
// better than two, at 80 instead of 128 registers; which one a launch takes depends on how its grid fills the waves.
template <int HQ_C, int M_C, bool RB, int CTAS = 2>
__global__ void __launch_bounds__(kThreads, HQ_C ? CTAS : 1) shared_decode_chunk_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(16) float smem[];
    const int b = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x;
    chain_release();
    const int j0 = chunk * kChunk;
    const int Hq = HQ_C ? HQ_C : p.Hq;
    const int m = M_C ? M_C : (p.integrate == LISA_INTEGRATE_PLUS ? 0 : p.m);
    const int r = p.r, G = Hq / p.Hkv;
    const int h_in = p.integrate == LISA_INTEGRATE_CONCAT ? 2 * Hq : Hq;

    float* s_s = smem;                      // [Hq][kChunk]  delta, then scores, then exp
    float* qp_s = s_s + Hq * kChunk;        // [Hq][kMaxRank]
    // weight rows are padded in the tensor-core path (strides m + 8 and Hq + 4) so that the fragment loads of a
    // warp spread over all shared-memory banks
    const int w1_ld = HQ_C ? m + 8 : m, w2_ld = HQ_C ? Hq + 4 : Hq;
    float* w1_s = qp_s + Hq * kMaxRank;     // [h_in][w1_ld]
    float* w2_s = w1_s + h_in * w1_ld;      // [m][w2_ld]
    float* b1_s = w2_s + m * w2_ld;         // [m]
    float* b2_s = b1_s + m;                 // [Hq]

    // the aligner's weights are constants of the model: staged while the kernel before this one may still be running
    if (p.integrate != LISA_INTEGRATE_PLUS) {
        for (int e = tid; e < h_in * m; e += kThreads) w1_s[(e / m) * w1_ld + e % m] = ld_elem(p.w1, e, p.w_dtype);
        for (int e = tid; e < m; e += kThreads) b1_s[e] = ldw(p.b1, e, p.w_dtype);
        if (p.ffn_layers == 2) {
            for (int e = tid; e < m * Hq; e += kThreads) w2_s[(e / Hq) * w2_ld + e % Hq] = ld_elem(p.w2, e, p.w_dtype);
            for (int e = tid; e < Hq; e += kThreads) b2_s[e] = ldw(p.b2, e, p.w_dtype);
        }
    }
    chain_wait();   // from here on: lengths, Q', the caches and the score row, which earlier kernels of the stream produce
    const int L = p.seq_lens ? min(p.seq_lens[b], p.L_uniform) : p.L_uniform;   // never beyond the chunks the launch covers
    if (j0 >= L) return;
    const int nrows = min(kChunk, L - j0);
    for (int e = tid; e < Hq * r; e += kThreads) {
        const int h = e / r, x = e % r;
        qp_s[h * kMaxRank + x] = ld_elem(p.qp.ptr, b * p.qp.sb + h * p.qp.sh + x, p.qp.dtype);
    }
    __syncthreads();

    // A_Delta for the chunk (Eq. 3): unit = (head, 8 consecutive positions)
    const float inv_sqrt_r = rsqrtf((float)r);
    if (p.cache_dtype == LISA_BF16) {
        for (int u = tid; u < Hq * (kChunk / 8); u += kThreads) {
            const int h = u / (kChunk / 8), j8 = u % (kChunk / 8);
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (j0 + j8 * 8 < p.L_cap) {
                const __nv_bfloat16* base = reinterpret_cast<const __nv_bfloat16*>(p.kpT) +
                                            ((size_t)b * p.Hkv + h / G) * r * p.L_cap + j0 + j8 * 8;
                for (int x0 = 0; x0 < r; x0 += 8) {   // eight independent 16-byte loads in flight per lane
                    uint4 raw[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        raw[e] = x0 + e < r ? ld_stream16(base + (size_t)(x0 + e) * p.L_cap) : make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        float f[8];
                        bf16x8_to_f32(raw[e], f);
                        const float qx = x0 + e < r ? qp_s[h * kMaxRank + x0 + e] : 0.f;
#pragma unroll
                        for (int t = 0; t < 8; ++t) acc[t] = fmaf(qx, f[t], acc[t]);
                    }
                }
            }
            float4* dst = reinterpret_cast<float4*>(s_s + h * kChunk + j8 * 8);
            dst[0] = make_float4(acc[0] * inv_sqrt_r, acc[1] * inv_sqrt_r, acc[2] * inv_sqrt_r, acc[3] * inv_sqrt_r);
            dst[1] = make_float4(acc[4] * inv_sqrt_r, acc[5] * inv_sqrt_r, acc[6] * inv_sqrt_r, acc[7] * inv_sqrt_r);
        }
    } else {
        for (int u = tid; u < Hq * kChunk; u += kThreads) {
            const int h = u / kChunk, jj = u % kChunk;
            float acc = 0.f;
            if (jj < nrows) {
                const float* base = reinterpret_cast<const float*>(p.kpT) + ((size_t)b * p.Hkv + h / G) * r * p.L_cap + j0 + jj;
                for (int x = 0; x < r; ++x) acc = fmaf(qp_s[h * kMaxRank + x], base[(size_t)x * p.L_cap], acc);
            }
            s_s[u] = acc * inv_sqrt_r;
        }
    }
    __syncthreads();

    const int pos = tid & (kChunk - 1), half = tid / kChunk;
    const bool valid = pos < nrows;
    const int64_t prev_i = b * p.prev_sb + j0 + pos;     // this thread's position in the previous layer's row of head 0
    const int64_t out_i = b * p.sc_sb + j0 + pos;

    if constexpr (HQ_C > 0) {
        // ADD, two-layer FFN on the tensor cores (mma.sync m16n8k8, tf32 operands, fp32 accumulation): a warp owns
        // 16 positions of the chunk as the M dimension.  Layer 1: [16 x HQ] . [HQ x M]; its accumulator fragments,
        // after bias and activation, ARE the A fragments of layer 2 when hidden unit 8j + 2t / 8j + 2t + 1 is taken
        // as k-index t / t + 4 of k-step j (the order of the hidden units inside the sum is free), so nothing moves
        // between lanes.  bf16 weights are exact in tf32; the fp32 score row is rounded to tf32 (2^-11 relative).
        constexpr int KS1 = HQ_C / 8, NT1 = M_C / 8, NT2 = HQ_C / 8;   // the second layer has NT1 k-steps
        const int lane = tid & 31, warp = tid >> 5;
        const int g = lane >> 2, t = lane & 3;
        const int p0 = warp * 16 + g, p1 = p0 + 8;              // this lane's two position rows
        const bool ok0 = p0 < nrows, ok1 = p1 < nrows;
        const int64_t prow = b * p.prev_sb + j0;
        uint32_t afr[KS1][4];
#pragma unroll
        for (int ks = 0; ks < KS1; ++ks) {
            const int64_t r0 = prow + (int64_t)(ks * 8 + t) * p.prev_sh;
            const int64_t r1 = prow + (int64_t)(ks * 8 + t + 4) * p.prev_sh;
            afr[ks][0] = f32_to_tf32(ok0 ? ld_row<RB>(p.prev, r0 + p0) : 0.f);
            afr[ks][1] = f32_to_tf32(ok1 ? ld_row<RB>(p.prev, r0 + p1) : 0.f);
            afr[ks][2] = f32_to_tf32(ok0 ? ld_row<RB>(p.prev, r1 + p0) : 0.f);
            afr[ks][3] = f32_to_tf32(ok1 ? ld_row<RB>(p.prev, r1 + p1) : 0.f);
        }
        float yacc[NT2][4];
#pragma unroll
        for (int j2 = 0; j2 < NT2; ++j2) {
            const float bb0 = b2_s[j2 * 8 + 2 * t], bb1 = b2_s[j2 * 8 + 2 * t + 1];
            yacc[j2][0] = bb0; yacc[j2][1] = bb1; yacc[j2][2] = bb0; yacc[j2][3] = bb1;
        }
#pragma unroll
        for (int j = 0; j < NT1; ++j) {
            // one 8-wide slice of hidden units: layer 1, activation, then straight into layer 2 as k-step j
            float hacc[4];
            hacc[0] = hacc[2] = b1_s[j * 8 + 2 * t];
            hacc[1] = hacc[3] = b1_s[j * 8 + 2 * t + 1];
#pragma unroll
            for (int ks = 0; ks < KS1; ++ks) {
                const uint32_t w0 = __float_as_uint(w1_s[(ks * 8 + t) * w1_ld + j * 8 + g]);
                const uint32_t w1v = __float_as_uint(w1_s[(ks * 8 + t + 4) * w1_ld + j * 8 + g]);
                mma_tf32(hacc, afr[ks], w0, w1v);
            }
            uint32_t hfr[4];
            hfr[0] = f32_to_tf32(act_apply(hacc[0], p.act));   // (row g,   k = t)     <- column 2t
            hfr[1] = f32_to_tf32(act_apply(hacc[2], p.act));   // (row g+8, k = t)
            hfr[2] = f32_to_tf32(act_apply(hacc[1], p.act));   // (row g,   k = t + 4) <- column 2t + 1
            hfr[3] = f32_to_tf32(act_apply(hacc[3], p.act));   // (row g+8, k = t + 4)
#pragma unroll
            for (int j2 = 0; j2 < NT2; ++j2) {
                const uint32_t w0 = __float_as_uint(w2_s[(j * 8 + 2 * t) * w2_ld + j2 * 8 + g]);
                const uint32_t w1v = __float_as_uint(w2_s[(j * 8 + 2 * t + 1) * w2_ld + j2 * 8 + g]);
                mma_tf32(yacc[j2], hfr, w0, w1v);
            }
        }
        // scores = FFN + A_Delta; yacc[j2]: [0] (p0, head 8 j2 + 2t), [1] (p0, +1), [2] (p1, 2t), [3] (p1, +1)
        const int64_t out0 = b * p.sc_sb + j0;
#pragma unroll
        for (int j2 = 0; j2 < NT2; ++j2) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int hh = j2 * 8 + 2 * t + (e & 1);
                const int pp = (e & 2) ? p1 : p0;
                const bool okp = (e & 2) ? ok1 : ok0;
                const float sc = yacc[j2][e] + s_s[hh * kChunk + pp];
                s_s[hh * kChunk + pp] = okp ? sc : -INFINITY;
                if (okp && p.out_scores) st_row<RB>(p.out_scores, out0 + (int64_t)hh * p.sc_sh + pp, sc);
            }
        }
    } else {
        if (half == 0) {
            float a[kMaxHeads], dl[kMaxHeads], hid[kMaxHidden];
            for (int h = 0; h < Hq; ++h) {
                a[h] = valid ? ld_row<RB>(p.prev, prev_i + h * p.prev_sh) : 0.f;
                dl[h] = s_s[h * kChunk + pos];
            }
            if (p.integrate == LISA_INTEGRATE_PLUS) {
                for (int g = 0; g < Hq; ++g) a[g] += dl[g];
            } else {
                for (int u = 0; u < m; ++u) {
                    float s = b1_s[u];
                    for (int x = 0; x < Hq; ++x) s = fmaf(a[x], w1_s[x * m + u], s);
                    if (p.integrate == LISA_INTEGRATE_CONCAT)
                        for (int x = 0; x < Hq; ++x) s = fmaf(dl[x], w1_s[(Hq + x) * m + u], s);
                    hid[u] = s;
                }
                if (p.ffn_layers == 1) {
                    for (int g = 0; g < Hq; ++g) a[g] = hid[g];
                } else {
                    for (int u = 0; u < m; ++u) hid[u] = act_apply(hid[u], p.act);
                    for (int g = 0; g < Hq; ++g) {
                        float s = b2_s[g];
                        for (int u = 0; u < m; ++u) s = fmaf(hid[u], w2_s[u * Hq + g], s);
                        a[g] = s;
                    }
                }
                if (p.integrate == LISA_INTEGRATE_ADD)
                    for (int g = 0; g < Hq; ++g) a[g] += dl[g];
            }
            for (int g = 0; g < Hq; ++g) {
                s_s[g * kChunk + pos] = valid ? a[g] : -INFINITY;
                if (valid && p.out_scores) st_row<RB>(p.out_scores, out_i + g * p.sc_sh, a[g]);
            }
        }
    }
    __syncthreads();
    softmax_pv_chunk(p, s_s, b, chunk, nrows);
}

// Scores of a FULL chunk for a standard layer, d = 128, bf16 cache: s_s[h][j] = q_h . K_j / sqrt(d).  Same streaming
// scheme as pv_full_chunk (two register sets of eight 16-byte loads per lane, prefetch across heads).  A lane holds
// the partial dot products of eight rows over its 8 of the 128 dimensions; the sum over the 16 lanes of a row is a
// butterfly that halves the number of live values at every step (8 shuffles per batch instead of 32).
__device__ __forceinline__ void anchor_qk_full_chunk(const DecodeParams& p, float* s_s, const float* q_s, int b, int j0,
                                                     float inv_sqrt_d) {
    constexpr int LPR = 16, RSTEP = 2, NB = kChunk / RSTEP / 8;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane & 15, rsel = lane >> 4;
    const int Hq = p.Hq, G = p.Hq / p.Hkv;
    auto head_ptr = [&](int h) {
        return reinterpret_cast<const uint4*>(p.kcache) + (((size_t)b * p.Hkv + h / G) * p.L_cap + j0 + rsel) * LPR + sub;
    };
    if (warp >= Hq) return;
    const uint4* hp = head_ptr(warp);
    uint4 ra[8], rb[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) ra[u] = ld_stream16(hp + u * RSTEP * LPR);
    const int urow = ((sub & 8) ? 4 : 0) + ((sub & 4) ? 2 : 0) + ((sub & 2) ? 1 : 0);  // row of the batch this lane ends up with
    auto reduce_store = [&](const uint4* regs, const float* qv, float* srow, int bi) {
        float dot[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            float f[8];
            bf16x8_to_f32(regs[u], f);
            float acc = 0.f;
#pragma unroll
            for (int t = 0; t < 8; ++t) acc = fmaf(qv[t], f[t], acc);
            dot[u] = acc;
        }
        float v4[4], v2[2];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float send = (sub & 8) ? dot[i] : dot[i + 4];
            const float keep = (sub & 8) ? dot[i + 4] : dot[i];
            v4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float send = (sub & 4) ? v4[i] : v4[i + 2];
            const float keep = (sub & 4) ? v4[i + 2] : v4[i];
            v2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
        }
        const float send = (sub & 2) ? v2[0] : v2[1];
        const float keep = (sub & 2) ? v2[1] : v2[0];
        float v1 = keep + __shfl_xor_sync(0xffffffffu, send, 2);
        v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
        if ((sub & 1) == 0) srow[(bi * 8 + urow) * RSTEP + rsel] = v1 * inv_sqrt_d;
    };
    for (int h = warp; h < Hq; h += kWarps) {
        const bool has_next = h + kWarps < Hq;
        const uint4* np = has_next ? head_ptr(h + kWarps) : hp;
        float qv[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) qv[t] = q_s[h * 128 + sub * 8 + t];
        float* srow = s_s + h * kChunk;
#pragma unroll
        for (int bi = 0; bi < NB; bi += 2) {
#pragma unroll
            for (int u = 0; u < 8; ++u) rb[u] = ld_stream16(hp + ((bi + 1) * 8 + u) * RSTEP * LPR);
            reduce_store(ra, qv, srow, bi);
            if (bi + 2 < NB) {
#pragma unroll
                for (int u = 0; u < 8; ++u) ra[u] = ld_stream16(hp + ((bi + 2) * 8 + u) * RSTEP * LPR);
            } else if (has_next) {
#pragma unroll
                for (int u = 0; u < 8; ++u) ra[u] = ld_stream16(np + u * RSTEP * LPR);
            }
            reduce_store(rb, qv, srow, bi + 1);
        }
        hp = np;
    }
}

// ---------------------------------------------------------------------------------------------
// Standard layer: scores from the K cache.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 2) anchor_decode_chunk_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(16) float smem[];
    const int b = blockIdx.y, chunk = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    chain_release();
    chain_wait();
    const int L = p.seq_lens ? min(p.seq_lens[b], p.L_uniform) : p.L_uniform;   // never beyond the chunks the launch covers
    const int j0 = chunk * kChunk;
    if (j0 >= L) return;
    const int nrows = min(kChunk, L - j0);
    const int Hq = p.Hq, d = p.d, G = Hq / p.Hkv;
    float* s_s = smem;               // [Hq][kChunk]
    float* q_s = s_s + Hq * kChunk;  // [Hq][d]
    for (int e = tid; e < Hq * d; e += kThreads) {
        const int h = e / d, x = e % d;
        q_s[e] = ld_elem(p.q.ptr, b * p.q.sb + h * p.q.sh + x, p.q.dtype);
    }
    __syncthreads();
    const float inv_sqrt_d = rsqrtf((float)d);
    if (p.cache_dtype == LISA_BF16 && d == 128 && nrows == kChunk) {
        anchor_qk_full_chunk(p, s_s, q_s, b, j0, inv_sqrt_d);
    } else if (p.cache_dtype == LISA_BF16) {
        const int lpr = d / 8, rstep = 32 / lpr, sub = lane % lpr, rsel = lane / lpr;
        for (int h = warp; h < Hq; h += kWarps) {
            float qv[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) qv[t] = q_s[h * d + sub * 8 + t];
            const uint4* kbase = reinterpret_cast<const uint4*>(p.kcache) +
                                 (((size_t)b * p.Hkv + h / G) * p.L_cap + j0) * lpr + sub;
            for (int jb = 0; jb < kChunk; jb += 4 * rstep) {
                float dot[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int jj = jb + u * rstep + rsel;
                    dot[u] = 0.f;
                    if (jj < nrows) {
                        float f[8];
                        bf16x8_to_f32(ld_stream16(kbase + (size_t)jj * lpr), f);
#pragma unroll
                        for (int t = 0; t < 8; ++t) dot[u] = fmaf(qv[t], f[t], dot[u]);
                    }
                }
                for (int off = lpr >> 1; off > 0; off >>= 1)
#pragma unroll
                    for (int u = 0; u < 4; ++u) dot[u] += __shfl_xor_sync(0xffffffffu, dot[u], off);
                if (sub == 0) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int jj = jb + u * rstep + rsel;
                        if (jj < kChunk) s_s[h * kChunk + jj] = jj < nrows ? dot[u] * inv_sqrt_d : -INFINITY;
                    }
                }
            }
        }
    } else {
        for (int u = tid; u < Hq * kChunk; u += kThreads) {
            const int h = u / kChunk, jj = u % kChunk;
            float acc = -INFINITY;
            if (jj < nrows) {
                const float* kr = reinterpret_cast<const float*>(p.kcache) + (((size_t)b * p.Hkv + h / G) * p.L_cap + j0 + jj) * d;
                acc = 0.f;
                for (int x = 0; x < d; ++x) acc = fmaf(q_s[h * d + x], kr[x], acc);
                acc *= inv_sqrt_d;
            }
            s_s[u] = acc;
        }
    }
    __syncthreads();
    if (p.out_scores) {
        for (int u = tid; u < Hq * kChunk; u += kThreads) {
            const int h = u / kChunk, jj = u % kChunk;
            if (jj < nrows) {
                if (p.row_bf16) st_row<true>(p.out_scores, b * p.sc_sb + h * p.sc_sh + j0 + jj, s_s[u]);
                else st_row<false>(p.out_scores, b * p.sc_sb + h * p.sc_sh + j0 + jj, s_s[u]);
            }
        }
    }
    softmax_pv_chunk(p, s_s, b, chunk, nrows);
}

// Merge the per-chunk (m, l, o) partials of one (b, h): o = sum_c e^{m_c - M} o_c / sum_c e^{m_c - M} l_c.
__global__ void decode_merge_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ float s_w[];   // per chunk: exp(m_c - M) / sum, the weight of the chunk's partial output
    const int h = blockIdx.x, b = blockIdx.y, x = threadIdx.x;
    chain_release();
    chain_wait();
    const int L = p.seq_lens ? min(p.seq_lens[b], p.L_uniform) : p.L_uniform;   // never beyond the chunks the launch covers
    const int nc = (L + kChunk - 1) / kChunk;
    const size_t base = (size_t)b * p.n_chunks * p.Hq + h;
    if (x < 32) {
        // the first warp turns the chunks' (m, l) into weights: one chunk per lane and step, reductions by shuffle
        float M = -INFINITY;
        for (int c = x; c < nc; c += 32) M = fmaxf(M, p.ws_m[base + (size_t)c * p.Hq]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        float den = 0.f;
        for (int c = x; c < nc; c += 32) {
            const float w = __expf(p.ws_m[base + (size_t)c * p.Hq] - M);
            s_w[c] = w;
            den = fmaf(w, p.ws_l[base + (size_t)c * p.Hq], den);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
        const float inv = 1.f / den;
        for (int c = x; c < nc; c += 32) s_w[c] *= inv;
    }
    __syncthreads();
    // every thread one output column: independent loads, four accumulators
    const float* po = p.ws_o + base * p.d + x;
    const size_t step = (size_t)p.Hq * p.d;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int c = 0;
    for (; c + 4 <= nc; c += 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[j] = fmaf(s_w[c + j], po[(size_t)(c + j) * step], acc[j]);
    }
    for (; c < nc; ++c) acc[0] = fmaf(s_w[c], po[(size_t)c * step], acc[0]);
    st_elem(const_cast<void*>(p.o.ptr), b * p.o.sb + h * p.o.sh + x, p.o.dtype, (acc[0] + acc[1]) + (acc[2] + acc[3]));
}

void carve_workspace(DecodeParams& p, void* ws) {
    const size_t n = (size_t)p.B * p.n_chunks * p.Hq;
    const size_t npad = (n + 3) & ~(size_t)3;  // keeps the o partials 16-byte aligned
    p.ws_m = reinterpret_cast<float*>(ws);
    p.ws_l = p.ws_m + npad;
    p.ws_o = p.ws_l + npad;
}

template <typename K>
cudaError_t set_smem(K kernel, size_t smem) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

}  // namespace

// Dynamic shared memory of the shared-layer chunk kernel: scores [Hq][kChunk], q' [Hq][kMaxRank], W1 and W2 (rows padded
// by 8 and 4 floats on the tensor-core path; the same bound is used for every path), b1, b2.
size_t shared_decode_smem(int Hq, int m_link, int integrate) {
    const int h_in = integrate == LISA_INTEGRATE_CONCAT ? 2 * Hq : Hq;
    const int m = integrate == LISA_INTEGRATE_PLUS ? 0 : m_link;
    return sizeof(float) * ((size_t)Hq * kChunk + (size_t)Hq * kMaxRank + (size_t)h_in * (m + 8) + (size_t)m * (Hq + 4) + m + Hq + 8);
}

size_t decode_workspace(int B, int Hq, int d, int L) {
    const size_t nc = (size_t)(L + kChunk - 1) / kChunk;
    const size_t n = (size_t)B * nc * Hq;
    const size_t npad = (n + 3) & ~(size_t)3;
    size_t bytes = (2 * npad + n * d) * sizeof(float);
    return (bytes + 255) & ~(size_t)255;
}

cudaError_t launch_shared_decode(const lisa_shared_decode_args& a, void* ws, cudaStream_t s) {
    const lisa_kvcache_layer& c = *a.cache;
    DecodeParams p{};
    p.B = a.B; p.Hq = a.Hq; p.Hkv = c.Hkv; p.d = c.d; p.L_cap = c.L_cap; p.L_uniform = a.L;
    p.n_chunks = (a.L + kChunk - 1) / kChunk;
    p.seq_lens = a.seq_lens;
    p.prev = a.prev_scores; p.prev_sb = a.prev_stride_b; p.prev_sh = a.prev_stride_h;
    p.qp = make_view(a.link.qp);
    p.kpT = c.k; p.vcache = c.v; p.cache_dtype = c.dtype;
    p.r = c.r; p.m = a.link.m; p.act = a.link.act; p.integrate = a.link.integrate; p.ffn_layers = a.link.ffn_layers;
    p.w_dtype = a.link.w_dtype;
    p.w1 = a.link.w1; p.b1 = a.link.b1; p.w2 = a.link.w2; p.b2 = a.link.b2;
    p.out_scores = a.out_scores; p.sc_sb = a.scores_stride_b; p.sc_sh = a.scores_stride_h;
    p.row_bf16 = a.scores_dtype == LISA_BF16;
    p.o = make_view(a.o);
    carve_workspace(p, ws);
    const size_t smem = shared_decode_smem(p.Hq, p.m, p.integrate);
    dim3 grid(p.n_chunks, p.B);
    const bool fast = p.integrate == LISA_INTEGRATE_ADD && p.ffn_layers == 2 && c.dtype == LISA_BF16;
    cudaError_t e;
#define LISA_LAUNCH_CHUNK(HQ_, M_, CTAS_)                                                                          \
    do {                                                                                                           \
        if (p.row_bf16) {                                                                                          \
            if ((e = set_smem(shared_decode_chunk_kernel<HQ_, M_, true, CTAS_>, smem)) != cudaSuccess) return e;   \
            e = launch_chained(shared_decode_chunk_kernel<HQ_, M_, true, CTAS_>, grid, dim3(kThreads), smem, s, p); \
        } else {                                                                                                   \
            if ((e = set_smem(shared_decode_chunk_kernel<HQ_, M_, false, CTAS_>, smem)) != cudaSuccess) return e;  \
            e = launch_chained(shared_decode_chunk_kernel<HQ_, M_, false, CTAS_>, grid, dim3(kThreads), smem, s, p); \
        }                                                                                                          \
    } while (0)
    // Two or three CTAs per SM: a CTA of the three-per-SM build takes about 1.3 times as long as one of the two-per-SM
    // build runs beside one neighbour (measured at B 64, L 4096, 40 heads: 0.534 against 0.566 ms for the whole grid), and the
    // grid runs in whole waves of CTAs: take the build whose waves cost less.
    const int64_t n_ctas = (int64_t)p.n_chunks * p.B, sms = sm_count();
    const bool three = 1.3 * (double)((n_ctas + 3 * sms - 1) / (3 * sms)) < (double)((n_ctas + 2 * sms - 1) / (2 * sms));
    if (fast && p.Hq == 40 && p.m == 80) { if (three) LISA_LAUNCH_CHUNK(40, 80, 3); else LISA_LAUNCH_CHUNK(40, 80, 2); }
    else if (fast && p.Hq == 32 && p.m == 64) { if (three) LISA_LAUNCH_CHUNK(32, 64, 3); else LISA_LAUNCH_CHUNK(32, 64, 2); }
    else LISA_LAUNCH_CHUNK(0, 0, 2);
#undef LISA_LAUNCH_CHUNK
    if (e != cudaSuccess) return e;
    e = launch_chained(decode_merge_kernel, dim3(p.Hq, p.B), dim3(p.d), (size_t)p.n_chunks * sizeof(float), s, p);
    count_launches(2);
    return e;
}

cudaError_t launch_anchor_decode(const lisa_anchor_args& a, void* ws, cudaStream_t s) {
    const lisa_kvcache_layer& c = *a.cache;
    DecodeParams p{};
    p.B = a.B; p.Hq = a.Hq; p.Hkv = c.Hkv; p.d = c.d; p.L_cap = c.L_cap; p.L_uniform = a.L;
    p.n_chunks = (a.L + kChunk - 1) / kChunk;
    p.seq_lens = a.seq_lens;
    p.q = make_view(a.q);
    p.kcache = c.k; p.vcache = c.v; p.cache_dtype = c.dtype;
    p.out_scores = a.out_scores; p.sc_sb = a.scores_stride_b; p.sc_sh = a.scores_stride_h;
    p.row_bf16 = a.scores_dtype == LISA_BF16;
    p.o = make_view(a.o);
    carve_workspace(p, ws);
    const size_t smem = sizeof(float) * ((size_t)p.Hq * kChunk + (size_t)p.Hq * p.d);
    cudaError_t e;
    if ((e = set_smem(anchor_decode_chunk_kernel, smem)) != cudaSuccess) return e;
    if ((e = launch_chained(anchor_decode_chunk_kernel, dim3(p.n_chunks, p.B), dim3(kThreads), smem, s, p)) != cudaSuccess) return e;
    e = launch_chained(decode_merge_kernel, dim3(p.Hq, p.B), dim3(p.d), (size_t)p.n_chunks * sizeof(float), s, p);
    count_launches(2);
    return e;
}

}  // namespace lisa
