// Head-axis aligner (Sec. 5.1), one link per launch, on warp-level tensor-core MMAs, for the shapes and Integrate modes
// the chain kernel of tc_align.cu does not take:
//   CONCAT  (32 heads)        A_k = W2^T act(W1^T [A_{k-1}; D_k] + b1) + b2    W1 [64, m], W2 [m, 32], m <= 256: the paper's
//                             complete model (Sec. 5.1, "An overview of LiSA": 64 x 256 and 256 x 32), and its one-layer
//                             form A_k = W1^T [A_{k-1}; D_k] + b1 with W1 [64, 32]
//   ADD     (32 or 40 heads)  A_k = FFN_k(A_{k-1}) + D_k with a two-layer FFN of hidden width m <= 256 (40 -> 80 -> 40 is the
//                             LLaMA2-13B shape), one linear layer, or no FFN at all (PLUS)
// Forms without a hidden layer run with an identity first layer (exact: every hidden unit is one fp16 input times one).
//
// Planes (fp16, blocked [row block of 128][column block of 64][row][B*heads + head][64 columns]):
//   plane_x  the link's input scores (A_0 = Q0.K0^T/sqrt(d) for the first link)
//   plane_d  D_k = Q'_k.K'_k^T/sqrt(r), already scaled (Eq. 3); ADD: may be absent (the top link's difference is added by
//            the attention kernel)
// Outputs go over the inputs, which are dead once the launch has read them: the scores for the next link (unscaled) and
// log2(e) times the FFN output for the attention kernel (which works in the exp2 domain), each over plane_x or plane_d
// as the caller says.
// A warp owns pieces of 32 key positions of one query row; per 16-position strip the A fragments come from ldmatrix.trans,
// the hidden layer is computed CHUNK units at a time with fp16 accumulators whose registers are the A fragments of the
// second layer (see tc_align_mma.cuh), the output accumulates in fp32 over the chunks.
#include <algorithm>

#include "tc_align_mma.cuh"

namespace lisa {
namespace {

using namespace tc;
using alignmma::act_h2;
using alignmma::KIND_FFN;
using alignmma::KIND_PLUS;
using alignmma::KIND_SINGLE;
using alignmma::kLog2e;
using alignmma::ldmatrix_x4_trans;
using alignmma::ldw;
using alignmma::mma_f16;
using alignmma::mma_f16acc;
using alignmma::stmatrix_x4_trans;

constexpr int UNIT = 128, PP = 32;
constexpr int kStages = 2;

struct LinkParams {
    int B, N, row0, qt_begin, qt_count, units_per_batch;
    int64_t plane_cols;
    int d_row0;                         // geometry of plane_d where it differs from plane_x's
    int64_t d_plane_cols;
    __half *plane_x, *plane_d;          // plane_d == nullptr: no difference plane (ADD, top link)
    int dst_next, dst_scaled;           // where the next link's input / the attention kernel's plane go: -1 nowhere, 0 plane_x, 1 plane_d
    const void *w1, *b1, *w2, *b2;
    int w_dtype, m, kind;               // kind: KIND_FFN (hidden width m) / KIND_SINGLE / KIND_PLUS
};

// NH heads; CONCAT: the difference plane is the second half of the FFN's input; the hidden layer is CHUNK * NCHUNK wide
template <int NH, bool CONCAT, int CHUNK, int NCHUNK>
struct Shape {
    static constexpr int HB = (NH + 15) / 16;                 // 16-head blocks of a plane (the last one zero-padded)
    static constexpr int KS_IN = CONCAT ? 2 * HB : HB;        // k-steps of the first layer
    static constexpr int H_IN = CONCAT ? 2 * NH : NH;
    static constexpr int MHID = CHUNK * NCHUNK;
    static constexpr int NT_OUT = NH / 8;                     // 8-head n-tiles of the output
    static constexpr int PLANE_SCR = HB * 16 * PP * 2;        // [heads, padded][32 positions] fp16
    static constexpr int W1F = KS_IN * (MHID / 8) * 32 * 8;
    static constexpr int W2F = (MHID / 16) * NT_OUT * 32 * 8;
    static constexpr int WEIGHTS = W1F + W2F + (MHID / 2 + HB * 16) * 4;
    static_assert(NH % 8 == 0 && CHUNK % 16 == 0 && (!CONCAT || NH % 16 == 0), "fragment shapes");
};

template <int NH, bool CONCAT, int CHUNK, int NCHUNK, int ACT, int NTHREADS>
__global__ void __launch_bounds__(NTHREADS, 1) tc_align_link_kernel(const __grid_constant__ LinkParams p) {
    using S = Shape<NH, CONCAT, CHUNK, NCHUNK>;
    constexpr int HB = S::HB, KS_IN = S::KS_IN, MHID = S::MHID, NT_OUT = S::NT_OUT, PLANE_SCR = S::PLANE_SCR;
    extern __shared__ __align__(16) uint8_t smem[];
    uint2* w1f = reinterpret_cast<uint2*>(smem);                               // [k-step KS_IN][n-tile MHID/8][lane]
    uint2* w2f = reinterpret_cast<uint2*>(smem + S::W1F);                      // [k-step MHID/16][n-tile NT_OUT][lane]
    uint32_t* b1h = reinterpret_cast<uint32_t*>(smem + S::W1F + S::W2F);       // [MHID/2] packed fp16 pairs
    float* b2 = reinterpret_cast<float*>(b1h + MHID / 2);                      // [HB * 16]
    uint8_t* sScr = smem + S::WEIGHTS;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m = p.m, wd = p.w_dtype, kind = p.kind;

    // ---- weights as ready-made B fragments; inputs beyond the heads and hidden units beyond m are zero rows / columns ----
    auto first = [&](int k, int n) -> float {      // [inputs][hidden]
        if (k >= S::H_IN) return 0.f;
        if (kind != KIND_FFN) return k == n ? 1.f : 0.f;
        return n < m ? ld_elem(p.w1, k * m + n, wd) : 0.f;
    };
    auto second = [&](int k, int n) -> float {     // [hidden][heads]
        if (kind == KIND_FFN) return k < m ? ld_elem(p.w2, k * NH + n, wd) : 0.f;
        if (kind == KIND_SINGLE) return k < S::H_IN ? ld_elem(p.w1, k * NH + n, wd) : 0.f;
        return k == n ? 1.f : 0.f;
    };
    // input index of row kk of the first layer's K dimension: with CONCAT the difference plane's heads follow the padded block of the scores
    auto in_index = [&](int kk) -> int {
        if (!CONCAT) return kk < NH ? kk : 1 << 20;
        const int half = kk / (HB * 16), h = kk % (HB * 16);
        return h < NH ? half * NH + h : 1 << 20;
    };
    for (int e = tid; e < KS_IN * (MHID / 8) * 32; e += NTHREADS) {
        const int ln = e & 31, j = (e >> 5) % (MHID / 8), ks = (e >> 5) / (MHID / 8), g = ln >> 2, t = ln & 3;
        const int k0 = ks * 16 + 2 * t, n = j * 8 + g;
        w1f[e] = make_uint2(pack_f16(first(in_index(k0), n), first(in_index(k0 + 1), n)), pack_f16(first(in_index(k0 + 8), n), first(in_index(k0 + 9), n)));
    }
    for (int e = tid; e < (MHID / 16) * NT_OUT * 32; e += NTHREADS) {
        const int ln = e & 31, j2 = (e >> 5) % NT_OUT, s2 = (e >> 5) / NT_OUT, g = ln >> 2, t = ln & 3;
        const int k0 = s2 * 16 + 2 * t, n = j2 * 8 + g;
        w2f[e] = make_uint2(pack_f16(second(k0, n), second(k0 + 1, n)), pack_f16(second(k0 + 8, n), second(k0 + 9, n)));
    }
    for (int e = tid; e < MHID / 2; e += NTHREADS)
        b1h[e] = (kind != KIND_FFN || 2 * e >= m) ? 0u : pack_f16(ldw(p.b1, 2 * e, wd), 2 * e + 1 < m ? ldw(p.b1, 2 * e + 1, wd) : 0.f);
    for (int e = tid; e < HB * 16; e += NTHREADS)
        b2[e] = e >= NH ? 0.f : (kind == KIND_FFN ? ldw(p.b2, e, wd) : (kind == KIND_SINGLE ? ldw(p.b1, e, wd) : 0.f));
    // the scratch rows of the padding heads stay zero for the whole launch (copies only touch real heads)
    for (int e = tid; e < (NTHREADS / 32) * kStages * 2 * PLANE_SCR / 16; e += NTHREADS) reinterpret_cast<uint4*>(sScr)[e] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();

    // ---- this warp's contiguous range of pieces: (batch, query tile, row, 64-key block, half) ----
    const int pB = p.B, pN = p.N, p_row0 = p.row0, p_qt0 = p.qt_begin, p_qt1 = p.qt_begin + p.qt_count;
    const int p_ncb = (int)(p.plane_cols >> 6);
    const int p_row0_d = p.d_row0, p_ncb_d = (int)(p.d_plane_cols >> 6);
    constexpr int PPU = UNIT / PP;
    const long long n_pieces = (long long)p.units_per_batch * pB * PPU;
    const long long n_warps = (long long)gridDim.x * (NTHREADS / 32);
    const long long per_warp = (n_pieces + n_warps - 1) / n_warps;
    const long long s_begin = min(n_pieces, ((long long)blockIdx.x * (NTHREADS / 32) + warp) * per_warp);
    const long long s_end = min(n_pieces, s_begin + per_warp);
    if (s_begin >= s_end) return;
    struct Cursor { int b, t, row, jb, sub; };
    Cursor cu;
    {
        const long long u = s_begin / PPU;
        cu.sub = (int)(s_begin % PPU);
        cu.b = (int)(u / p.units_per_batch);
        int rem = (int)(u - (long long)cu.b * p.units_per_batch);
        cu.t = p_qt0;
        for (;; ++cu.t) {
            const int n_t = min(UNIT, pN - cu.t * UNIT) * (cu.t + 1);
            if (rem < n_t || cu.t + 1 >= p_qt1) break;
            rem -= n_t;
        }
        cu.row = rem / (cu.t + 1);
        cu.jb = rem - cu.row * (cu.t + 1);
    }
    auto advance = [&](Cursor& x) {
        if (++x.sub < PPU) return;
        x.sub = 0;
        if (++x.jb <= x.t) return;
        x.jb = 0;
        if (++x.row < min(UNIT, pN - x.t * UNIT)) return;
        x.row = 0;
        if (++x.t < p_qt1) return;
        x.t = p_qt0;
        ++x.b;
    };
    // four lanes cover the 64 bytes [head][32 positions] of one head: a warp-wide access moves 8 heads
    constexpr int CPR = PP / 8, HPA = 32 / CPR, NACC = NH / HPA;
    const int l_head = lane / CPR, l_chunk = lane % CPR;
    auto piece_off = [&](const Cursor& x, int which) {   // which: 0 = plane_x's geometry, 1 = plane_d's
        const int r = x.t * UNIT + x.row - (which ? p_row0_d : p_row0);
        const int col = x.sub * PP;
        const int64_t blk = (int64_t)(r >> 7) * (which ? p_ncb_d : p_ncb) + (x.jb * 2 + (col >> 6));
        return ((blk * 128 + (r & 127)) * (pB * NH) + (x.b * NH + l_head)) * 64 + (col & 63) + l_chunk * 8;
    };
    auto scr_off = [&](int head, int chunk) { return (uint32_t)(head * (PP * 2) + ((chunk ^ ((head >> 1) & 3)) << 4)); };
    uint8_t* scr = sScr + warp * (kStages * 2 * PLANE_SCR);   // [stage][plane x, plane d][heads][64 B]
    __half* const gx = p.plane_x;
    __half* const gd = p.plane_d;
    const bool has_d = gd != nullptr;
    auto fetch = [&](const Cursor& x, int buf) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            if (k == 1 && !has_d) break;
            const int64_t off = piece_off(x, k);
            const __half* src = k == 0 ? gx : gd;
#pragma unroll
            for (int i = 0; i < NACC; ++i) {
                const uint32_t dst = smem_u32(scr + (buf * 2 + k) * PLANE_SCR) + scr_off(l_head + HPA * i, l_chunk);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src + off + i * (HPA * 64)) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    const int mi = lane >> 3, lr = lane & 7, t4 = lane & 3;
    auto frag_off = [&](int s2, int x) { return scr_off(x * 16 + 8 * (mi >> 1) + lr, 2 * s2 + (mi & 1)); };
    const int dst_next = p.dst_next, dst_scaled = p.dst_scaled;

    fetch(cu, 0);
    Cursor ahead = cu;
    advance(ahead);
    int buf = 0;
    for (long long sidx = s_begin; sidx < s_end; ++sidx) {
        const Cursor here = cu;
        advance(cu);
        if (sidx + 1 < s_end) { fetch(ahead, buf ^ 1); advance(ahead); }
        else asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        __syncwarp();
        const uint32_t base_x = smem_u32(scr + (buf * 2) * PLANE_SCR), base_d = base_x + PLANE_SCR;
        // both 16-position strips of the piece go through the FFN together: every weight fragment read from shared memory
        // feeds two MMAs (with one, the shared-memory pipe moves 256 bytes per MMA, about all it delivers at the MMA rate)
        constexpr int NS = PP / 16;
        {
            uint32_t afr[NS][KS_IN][4];      // CONCAT: the first HB k-steps are the heads of the scores, the others the heads of D_k
#pragma unroll
            for (int s2 = 0; s2 < NS; ++s2)
#pragma unroll
                for (int x = 0; x < HB; ++x) {
                    ldmatrix_x4_trans(afr[s2][x], base_x + frag_off(s2, x));
                    if constexpr (CONCAT) ldmatrix_x4_trans(afr[s2][HB + x], base_d + frag_off(s2, x));
                }
            float y[NS][2 * HB][4];
#pragma unroll
            for (int j2 = 0; j2 < 2 * HB; ++j2) {
                const float2 bb = *reinterpret_cast<const float2*>(b2 + j2 * 8 + 2 * t4);
#pragma unroll
                for (int s2 = 0; s2 < NS; ++s2) { y[s2][j2][0] = bb.x; y[s2][j2][1] = bb.y; y[s2][j2][2] = bb.x; y[s2][j2][3] = bb.y; }
            }
#pragma unroll 1
            for (int q = 0; q < NCHUNK; ++q) {
                uint32_t h[NS][CHUNK / 8][2];
#pragma unroll
                for (int j = 0; j < CHUNK / 8; ++j) {
                    const uint32_t bb = b1h[(q * (CHUNK / 8) + j) * 4 + t4];
                    const uint2 w = w1f[(q * (CHUNK / 8) + j) * 32 + lane];
#pragma unroll
                    for (int s2 = 0; s2 < NS; ++s2) mma_f16acc(h[s2][j], afr[s2][0], w.x, w.y, bb, bb);
                }
#pragma unroll
                for (int ks = 1; ks < KS_IN; ++ks)
#pragma unroll
                    for (int j = 0; j < CHUNK / 8; ++j) {
                        const uint2 w = w1f[(ks * (MHID / 8) + q * (CHUNK / 8) + j) * 32 + lane];
#pragma unroll
                        for (int s2 = 0; s2 < NS; ++s2) mma_f16acc(h[s2][j], afr[s2][ks], w.x, w.y, h[s2][j][0], h[s2][j][1]);
                    }
#pragma unroll
                for (int s2 = 0; s2 < NS; ++s2)
#pragma unroll
                    for (int j = 0; j < CHUNK / 8; ++j) {
                        h[s2][j][0] = act_h2<ACT>(h[s2][j][0]);
                        h[s2][j][1] = act_h2<ACT>(h[s2][j][1]);
                    }
#pragma unroll
                for (int s = 0; s < CHUNK / 16; ++s)
#pragma unroll
                    for (int j2 = 0; j2 < NT_OUT; ++j2) {
                        const uint2 w = w2f[((q * (CHUNK / 16) + s) * NT_OUT + j2) * 32 + lane];
#pragma unroll
                        for (int s2 = 0; s2 < NS; ++s2) {
                            const uint32_t hfr[4] = {h[s2][2 * s][0], h[s2][2 * s][1], h[s2][2 * s + 1][0], h[s2][2 * s + 1][1]};
                            mma_f16(y[s2][j2], hfr, w.x, w.y);
                        }
                    }
            }
            // every lane has read its fragments of the scores (the MMAs that consumed them have completed): results go back transposed
            __syncwarp();
            if (dst_scaled >= 0) {
                const uint32_t base = dst_scaled == 0 ? base_x : base_d;
#pragma unroll
                for (int s2 = 0; s2 < NS; ++s2)
#pragma unroll
                    for (int x = 0; x < HB; ++x) {
                        uint32_t r[4];
                        r[0] = pack_f16(y[s2][2 * x][0] * kLog2e, y[s2][2 * x][1] * kLog2e);
                        r[1] = pack_f16(y[s2][2 * x][2] * kLog2e, y[s2][2 * x][3] * kLog2e);
                        r[2] = pack_f16(y[s2][2 * x + 1][0] * kLog2e, y[s2][2 * x + 1][1] * kLog2e);
                        r[3] = pack_f16(y[s2][2 * x + 1][2] * kLog2e, y[s2][2 * x + 1][3] * kLog2e);
                        stmatrix_x4_trans(base + frag_off(s2, x), r);
                    }
            }
            if (dst_next >= 0) {
                if constexpr (!CONCAT) {
                    if (has_d) {   // A_k = FFN(A_{k-1}) + D_k: the difference in the fragment arrangement the scores came in
#pragma unroll
                        for (int s2 = 0; s2 < NS; ++s2)
#pragma unroll
                            for (int x = 0; x < HB; ++x) {
                                uint32_t dfr[4];
                                ldmatrix_x4_trans(dfr, base_d + frag_off(s2, x));
#pragma unroll
                                for (int qq = 0; qq < 4; ++qq) {
                                    const float2 dv = unpack_f16(dfr[qq]);
                                    y[s2][2 * x + (qq >> 1)][2 * (qq & 1)] += dv.x;
                                    y[s2][2 * x + (qq >> 1)][2 * (qq & 1) + 1] += dv.y;
                                }
                            }
                        __syncwarp();   // all lanes hold their part of D_k before it is overwritten
                    }
                }
                const uint32_t base = dst_next == 0 ? base_x : base_d;
#pragma unroll
                for (int s2 = 0; s2 < NS; ++s2)
#pragma unroll
                    for (int x = 0; x < HB; ++x) {
                        uint32_t r[4];
                        r[0] = pack_f16(y[s2][2 * x][0], y[s2][2 * x][1]);
                        r[1] = pack_f16(y[s2][2 * x][2], y[s2][2 * x][3]);
                        r[2] = pack_f16(y[s2][2 * x + 1][0], y[s2][2 * x + 1][1]);
                        r[3] = pack_f16(y[s2][2 * x + 1][2], y[s2][2 * x + 1][3]);
                        stmatrix_x4_trans(base + frag_off(s2, x), r);
                    }
            }
        }
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            if (dst_next != k && dst_scaled != k) continue;
            const int64_t here_off = piece_off(here, k);
            __half* dst = k == 0 ? gx : gd;
#pragma unroll
            for (int i = 0; i < NACC; ++i)
                *reinterpret_cast<uint4*>(dst + here_off + i * (HPA * 64)) =
                    *reinterpret_cast<const uint4*>(scr + (buf * 2 + k) * PLANE_SCR + scr_off(l_head + HPA * i, l_chunk));
        }
        __syncwarp();   // the next iteration's fetch refills the other buffer; this one is refilled an iteration later
        buf ^= 1;
    }
}

template <int NH, bool CONCAT, int CHUNK, int NCHUNK, int NTHREADS>
cudaError_t launch_shape(const LinkParams& p, int act, unsigned grid, cudaStream_t stream) {
    using S = Shape<NH, CONCAT, CHUNK, NCHUNK>;
    const size_t smem = (size_t)S::WEIGHTS + (size_t)(NTHREADS / 32) * kStages * 2 * S::PLANE_SCR;
    static_assert(S::WEIGHTS + (NTHREADS / 32) * kStages * 2 * S::PLANE_SCR <= 232448, "one CTA's shared memory");
    auto kernel = act == LISA_ACT_RELU   ? tc_align_link_kernel<NH, CONCAT, CHUNK, NCHUNK, LISA_ACT_RELU, NTHREADS>
                  : act == LISA_ACT_SILU ? tc_align_link_kernel<NH, CONCAT, CHUNK, NCHUNK, LISA_ACT_SILU, NTHREADS>
                                         : tc_align_link_kernel<NH, CONCAT, CHUNK, NCHUNK, LISA_ACT_NONE, NTHREADS>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, NTHREADS, smem, stream>>>(p);
    return cudaGetLastError();
}

bool link_ok(int Hq, const lisa_link& l) {
    if (l.integrate == LISA_INTEGRATE_PLUS) return Hq == 32 || Hq == 40;
    if (l.integrate == LISA_INTEGRATE_CONCAT) {
        if (Hq != 32) return false;
        return l.ffn_layers == 2 ? (l.m >= 1 && l.m <= 256) : l.m == Hq;
    }
    if (Hq != 32 && Hq != 40) return false;
    return l.ffn_layers == 2 ? (l.m >= 1 && l.m <= 256) : l.m == Hq;
}

}  // namespace

bool tc_align_concat_supported(int Hq, const lisa_link* links, int chain) {
    if (chain < 1) return false;
    for (int k = 0; k < chain; ++k)
        if (links[k].integrate != LISA_INTEGRATE_CONCAT || !link_ok(Hq, links[k])) return false;
    return true;
}

// Chains of adding (or FFN-free) links, one launch per link: 32 or 40 heads, hidden width up to 256.
bool tc_align_link_supported(int Hq, const lisa_link* links, int chain) {
    if (chain < 1) return false;
    for (int k = 0; k < chain; ++k)
        if (links[k].integrate == LISA_INTEGRATE_CONCAT || !link_ok(Hq, links[k])) return false;
    return true;
}

cudaError_t launch_tc_align_link(const TcAlignLinkArgs& a, cudaStream_t stream) {
    if (a.plane_cols % 64 != 0 || a.plane_rows % 128 != 0) return cudaErrorInvalidValue;
    const lisa_link& l = *a.link;
    if (!link_ok(a.Hq, l)) return cudaErrorInvalidValue;
    const bool concat = l.integrate == LISA_INTEGRATE_CONCAT;
    if (concat && !a.plane_d) return cudaErrorInvalidValue;
    LinkParams p{};
    p.B = a.B; p.N = a.N; p.row0 = a.row0 >= 0 ? a.row0 : a.qt_begin * UNIT; p.qt_begin = a.qt_begin; p.qt_count = a.qt_count;
    if (p.row0 % UNIT != 0 || p.row0 > a.qt_begin * UNIT) return cudaErrorInvalidValue;
    p.plane_cols = a.plane_cols;
    p.d_plane_cols = a.d_plane_cols > 0 ? a.d_plane_cols : a.plane_cols;
    p.d_row0 = a.d_plane_cols > 0 ? (a.d_row0 >= 0 ? a.d_row0 : a.qt_begin * UNIT) : p.row0;
    if (p.d_plane_cols % 64 != 0 || p.d_row0 % UNIT != 0 || p.d_row0 > a.qt_begin * UNIT || (a.d_plane_cols > 0 && a.d_plane_rows % 128 != 0))
        return cudaErrorInvalidValue;
    for (int t = a.qt_begin; t < a.qt_begin + a.qt_count; ++t) p.units_per_batch += std::min(UNIT, a.N - t * UNIT) * (t + 1);
    p.plane_x = reinterpret_cast<__half*>(a.plane_x); p.plane_d = reinterpret_cast<__half*>(a.plane_d);
    p.dst_next = a.dst_next; p.dst_scaled = a.dst_scaled;
    p.w1 = l.w1; p.b1 = l.b1; p.w2 = l.w2; p.b2 = l.b2; p.w_dtype = l.w_dtype;
    p.kind = alignmma::link_kind(l.integrate, l.ffn_layers);
    p.m = l.m;
    const int act = p.kind == KIND_FFN ? l.act : LISA_ACT_NONE;
    const int64_t total_units = (int64_t)p.units_per_batch * a.B;
    if (total_units <= 0 || total_units > 0x7fffffff) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)std::min<int64_t>((total_units + 3) / 4, sm_count());
    const bool narrow = p.kind != KIND_FFN || l.m <= 64;   // hidden layer (or identity) within 64 units
    cudaError_t e;
    if (concat) e = narrow ? launch_shape<32, true, 64, 1, 512>(p, act, grid, stream) : launch_shape<32, true, 64, 4, 512>(p, act, grid, stream);
    else if (a.Hq == 32) e = narrow ? launch_shape<32, false, 64, 1, 512>(p, act, grid, stream) : launch_shape<32, false, 64, 4, 512>(p, act, grid, stream);
    else if (narrow) e = launch_shape<40, false, 64, 1, 384>(p, act, grid, stream);
    else if (l.m <= 80) e = launch_shape<40, false, 80, 1, 384>(p, act, grid, stream);
    else e = launch_shape<40, false, 64, 4, 384>(p, act, grid, stream);
    count_launches(1);
    return e;
}

}  // namespace lisa
