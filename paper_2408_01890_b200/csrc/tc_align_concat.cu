// Head-axis aligner for the concatenating Integrate (Sec. 5.1, "An overview of LiSA": the FFN fuses [A_{n-1}; A_Delta],
// the paper's complete model, 64 x 256 and 256 x 32 for 32 heads), one link per launch, on warp-level tensor-core MMAs.
//
// Planes (fp16, blocked [row block of 128][column block of 64][row][B*32 + head][64 columns]):
//   in_a  = A_{k-1}  (A_0 = Q0.K0^T/sqrt(d) for the first link, the previous launch's output otherwise)
//   in_d  = D_k = Q'_k.K'_k^T/sqrt(r), already scaled (Eq. 3)
//   A_k[:, i, j] = W2^T act(W1^T [A_{k-1}[:, i, j]; D_k[:, i, j]] + b1) + b2        W1 [64, m], W2 [m, 32]
// and the one-layer form A_k = W1^T [A_{k-1}; D_k] + b1 with W1 [64, 32] (run as m = 64 with an identity first layer:
// exact, every hidden unit is one fp16 input times one).
// Output: A_k over in_a (for the next link) and/or log2(e) * A_k over in_d (for the attention kernel, which works in
// the exp2 domain): D_k is dead once this launch has read it.
// A warp owns pieces of 32 key positions of one query row; per 16-position strip the A fragments of both planes come
// from ldmatrix.trans, the hidden layer is computed 64 units at a time with fp16 accumulators whose registers are the
// A fragments of the second layer (see tc_align_mma.cuh), the output accumulates in fp32 over the hidden chunks.
#include <algorithm>

#include "tc_align_mma.cuh"

namespace lisa {
namespace {

using namespace tc;
using namespace alignmma;

constexpr int UNIT = 128, PP = 32, KIN = 64;
constexpr int kThreads = 512, kStages = 2;
constexpr int PLANE_SCR = HQ * PP * 2;      // [32 heads][32 positions] fp16

struct ConcatParams {
    int B, N, row0, qt_begin, qt_count, units_per_batch;
    int64_t plane_cols;
    __half *in_a, *in_d;
    int write_next, write_scaled;       // A_k over in_a; log2(e) * A_k over in_d
    const void *w1, *b1, *w2, *b2;
    int w_dtype, m, act, single;        // single: one linear layer W1 [64, 32]
};

template <int MHID>
struct Sizes {
    static constexpr int W1F = (KIN / 16) * (MHID / 8) * 32 * 8;
    static constexpr int W2F = (MHID / 16) * 4 * 32 * 8;
    static constexpr int WEIGHTS = W1F + W2F + (MHID / 2 + HQ) * 4;
};

template <int MHID, int ACT>
__global__ void __launch_bounds__(kThreads, 1) tc_align_concat_kernel(const __grid_constant__ ConcatParams p) {
    extern __shared__ __align__(16) uint8_t smem[];
    uint2* w1f = reinterpret_cast<uint2*>(smem);                                   // [k-step 4][n-tile MHID/8][lane]
    uint2* w2f = reinterpret_cast<uint2*>(smem + Sizes<MHID>::W1F);               // [k-step MHID/16][n-tile 4][lane]
    uint32_t* b1h = reinterpret_cast<uint32_t*>(smem + Sizes<MHID>::W1F + Sizes<MHID>::W2F);   // [MHID/2] packed fp16 pairs
    float* b2 = reinterpret_cast<float*>(b1h + MHID / 2);                          // [32]
    uint8_t* sScr = smem + Sizes<MHID>::WEIGHTS;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m = p.m, wd = p.w_dtype;

    // ---- weights as ready-made B fragments; hidden units beyond m are zero columns / rows (they contribute act(0).0 = 0) ----
    auto first = [&](int k, int n) -> float {      // [64 inputs][MHID hidden]
        if (p.single) return k == n ? 1.f : 0.f;
        return n < m ? ld_elem(p.w1, k * m + n, wd) : 0.f;
    };
    auto second = [&](int k, int n) -> float {     // [MHID hidden][32 heads]
        if (p.single) return k < KIN ? ld_elem(p.w1, k * HQ + n, wd) : 0.f;
        return k < m ? ld_elem(p.w2, k * HQ + n, wd) : 0.f;
    };
    for (int e = tid; e < (KIN / 16) * (MHID / 8) * 32; e += kThreads) {
        const int ln = e & 31, j = (e >> 5) % (MHID / 8), ks = (e >> 5) / (MHID / 8), g = ln >> 2, t = ln & 3;
        const int k0 = ks * 16 + 2 * t, n = j * 8 + g;
        w1f[e] = make_uint2(pack_f16(first(k0, n), first(k0 + 1, n)), pack_f16(first(k0 + 8, n), first(k0 + 9, n)));
    }
    for (int e = tid; e < (MHID / 16) * 4 * 32; e += kThreads) {
        const int ln = e & 31, j2 = (e >> 5) & 3, s2 = e >> 7, g = ln >> 2, t = ln & 3;
        const int k0 = s2 * 16 + 2 * t, n = j2 * 8 + g;
        w2f[e] = make_uint2(pack_f16(second(k0, n), second(k0 + 1, n)), pack_f16(second(k0 + 8, n), second(k0 + 9, n)));
    }
    for (int e = tid; e < MHID / 2; e += kThreads)
        b1h[e] = (p.single || 2 * e >= m) ? 0u : pack_f16(ldw(p.b1, 2 * e, wd), 2 * e + 1 < m ? ldw(p.b1, 2 * e + 1, wd) : 0.f);
    for (int e = tid; e < HQ; e += kThreads) b2[e] = p.single ? ldw(p.b1, e, wd) : ldw(p.b2, e, wd);
    __syncthreads();

    // ---- this warp's contiguous range of pieces: (batch, query tile, row, 64-key block, half) ----
    const int pB = p.B, pN = p.N, p_row0 = p.row0, p_qt0 = p.qt_begin, p_qt1 = p.qt_begin + p.qt_count;
    const int p_ncb = (int)(p.plane_cols >> 6);
    constexpr int PPU = UNIT / PP;
    const long long n_pieces = (long long)p.units_per_batch * pB * PPU;
    const long long n_warps = (long long)gridDim.x * (kThreads / 32);
    const long long per_warp = (n_pieces + n_warps - 1) / n_warps;
    const long long s_begin = min(n_pieces, ((long long)blockIdx.x * (kThreads / 32) + warp) * per_warp);
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
    // four lanes cover the 64 bytes [head][32 positions] of one head: a warp-wide access moves 8 heads, four accesses a plane
    constexpr int CPR = PP / 8, HPA = 32 / CPR, NACC = HQ / HPA;
    const int l_head = lane / CPR, l_chunk = lane % CPR;
    auto piece_off = [&](const Cursor& x) {
        const int r = x.t * UNIT + x.row - p_row0;
        const int col = x.sub * PP;
        const int64_t blk = (int64_t)(r >> 7) * p_ncb + (x.jb * 2 + (col >> 6));
        return ((blk * 128 + (r & 127)) * (pB * HQ) + (x.b * HQ + l_head)) * 64 + (col & 63) + l_chunk * 8;
    };
    auto scr_off = [&](int head, int chunk) { return (uint32_t)(head * (PP * 2) + ((chunk ^ ((head >> 1) & 3)) << 4)); };
    uint8_t* scr = sScr + warp * (kStages * 2 * PLANE_SCR);   // [stage][plane a, plane d][32 heads][64 B]
    __half* const in_a = p.in_a;
    __half* const in_d = p.in_d;
    auto fetch = [&](const Cursor& x, int buf) {
        const int64_t off = piece_off(x);
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const __half* src = k == 0 ? in_a : in_d;
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
    const bool write_next = p.write_next != 0, write_scaled = p.write_scaled != 0;

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
        const uint32_t base_a = smem_u32(scr + (buf * 2) * PLANE_SCR), base_d = base_a + PLANE_SCR;
#pragma unroll
        for (int s2 = 0; s2 < PP / 16; ++s2) {
            const uint32_t off0 = frag_off(s2, 0), off1 = frag_off(s2, 1);
            uint32_t afr[KIN / 16][4];      // k-steps 0, 1: heads of A_{k-1}; 2, 3: heads of D_k
            ldmatrix_x4_trans(afr[0], base_a + off0);
            ldmatrix_x4_trans(afr[1], base_a + off1);
            ldmatrix_x4_trans(afr[2], base_d + off0);
            ldmatrix_x4_trans(afr[3], base_d + off1);
            float y[4][4];
#pragma unroll
            for (int j2 = 0; j2 < 4; ++j2) {
                const float2 bb = *reinterpret_cast<const float2*>(b2 + j2 * 8 + 2 * t4);
                y[j2][0] = bb.x; y[j2][1] = bb.y; y[j2][2] = bb.x; y[j2][3] = bb.y;
            }
#pragma unroll 1
            for (int q = 0; q < MHID / 64; ++q) {
                uint32_t h[8][2];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t bb = b1h[(q * 8 + j) * 4 + t4];
                    const uint2 w = w1f[(0 * (MHID / 8) + q * 8 + j) * 32 + lane];
                    mma_f16acc(h[j], afr[0], w.x, w.y, bb, bb);
                }
#pragma unroll
                for (int ks = 1; ks < KIN / 16; ++ks)
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint2 w = w1f[(ks * (MHID / 8) + q * 8 + j) * 32 + lane];
                        mma_f16acc(h[j], afr[ks], w.x, w.y, h[j][0], h[j][1]);
                    }
                uint32_t hfr[4][4];
#pragma unroll
                for (int s = 0; s < 4; ++s) {
                    hfr[s][0] = act_h2<ACT>(h[2 * s][0]);
                    hfr[s][1] = act_h2<ACT>(h[2 * s][1]);
                    hfr[s][2] = act_h2<ACT>(h[2 * s + 1][0]);
                    hfr[s][3] = act_h2<ACT>(h[2 * s + 1][1]);
                }
#pragma unroll
                for (int s = 0; s < 4; ++s)
#pragma unroll
                    for (int j2 = 0; j2 < 4; ++j2) {
                        const uint2 w = w2f[((q * 4 + s) * 4 + j2) * 32 + lane];
                        mma_f16(y[j2], hfr[s], w.x, w.y);
                    }
            }
            // every lane has read its fragments of both planes (the MMAs that consumed them have completed): write the
            // result back transposed, unscaled over A and/or scaled over D
            __syncwarp();
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                uint32_t r[4];
                if (write_next) {
                    r[0] = pack_f16(y[2 * x][0], y[2 * x][1]);
                    r[1] = pack_f16(y[2 * x][2], y[2 * x][3]);
                    r[2] = pack_f16(y[2 * x + 1][0], y[2 * x + 1][1]);
                    r[3] = pack_f16(y[2 * x + 1][2], y[2 * x + 1][3]);
                    stmatrix_x4_trans(base_a + (x ? off1 : off0), r);
                }
                if (write_scaled) {
                    r[0] = pack_f16(y[2 * x][0] * kLog2e, y[2 * x][1] * kLog2e);
                    r[1] = pack_f16(y[2 * x][2] * kLog2e, y[2 * x][3] * kLog2e);
                    r[2] = pack_f16(y[2 * x + 1][0] * kLog2e, y[2 * x + 1][1] * kLog2e);
                    r[3] = pack_f16(y[2 * x + 1][2] * kLog2e, y[2 * x + 1][3] * kLog2e);
                    stmatrix_x4_trans(base_d + (x ? off1 : off0), r);
                }
            }
        }
        __syncwarp();
        const int64_t here_off = piece_off(here);
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            if (k == 0 ? !write_next : !write_scaled) continue;
            __half* dst = k == 0 ? in_a : in_d;
#pragma unroll
            for (int i = 0; i < NACC; ++i)
                *reinterpret_cast<uint4*>(dst + here_off + i * (HPA * 64)) =
                    *reinterpret_cast<const uint4*>(scr + (buf * 2 + k) * PLANE_SCR + scr_off(l_head + HPA * i, l_chunk));
        }
        __syncwarp();   // the next iteration's fetch refills the other buffer; this one is refilled an iteration later
        buf ^= 1;
    }
}

template <int MHID>
cudaError_t launch_for_width(const ConcatParams& p, int act, unsigned grid, cudaStream_t stream) {
    const size_t smem = (size_t)Sizes<MHID>::WEIGHTS + (size_t)(kThreads / 32) * kStages * 2 * PLANE_SCR;
    auto kernel = act == LISA_ACT_RELU ? tc_align_concat_kernel<MHID, LISA_ACT_RELU>
                : act == LISA_ACT_SILU ? tc_align_concat_kernel<MHID, LISA_ACT_SILU> : tc_align_concat_kernel<MHID, LISA_ACT_NONE>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, kThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

bool tc_align_concat_supported(int Hq, const lisa_link* links, int chain) {
    if (Hq != HQ || chain < 1) return false;
    for (int k = 0; k < chain; ++k) {
        const lisa_link& l = links[k];
        if (l.integrate != LISA_INTEGRATE_CONCAT) return false;
        if (l.ffn_layers == 2 ? (l.m < 1 || l.m > 256) : l.m != HQ) return false;
    }
    return true;
}

cudaError_t launch_tc_align_concat(const TcAlignConcatArgs& a, cudaStream_t stream) {
    if (a.plane_cols % 64 != 0 || a.plane_rows % 128 != 0) return cudaErrorInvalidValue;
    const lisa_link& l = *a.link;
    ConcatParams p{};
    p.B = a.B; p.N = a.N; p.row0 = a.qt_begin * UNIT; p.qt_begin = a.qt_begin; p.qt_count = a.qt_count;
    p.plane_cols = a.plane_cols;
    for (int t = a.qt_begin; t < a.qt_begin + a.qt_count; ++t) p.units_per_batch += std::min(UNIT, a.N - t * UNIT) * (t + 1);
    p.in_a = reinterpret_cast<__half*>(a.plane_a); p.in_d = reinterpret_cast<__half*>(a.plane_d);
    p.write_next = a.write_next ? 1 : 0; p.write_scaled = a.write_scaled ? 1 : 0;
    p.w1 = l.w1; p.b1 = l.b1; p.w2 = l.w2; p.b2 = l.b2; p.w_dtype = l.w_dtype;
    p.single = l.ffn_layers == 1 ? 1 : 0;
    p.m = p.single ? 64 : l.m;
    p.act = p.single ? LISA_ACT_NONE : l.act;
    const int64_t total_units = (int64_t)p.units_per_batch * a.B;
    if (total_units <= 0 || total_units > 0x7fffffff) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)std::min<int64_t>((total_units + 3) / 4, sm_count());
    cudaError_t e = p.m <= 64 ? launch_for_width<64>(p, p.act, grid, stream) : launch_for_width<256>(p, p.act, grid, stream);
    count_launches(1);
    return e;
}

}  // namespace lisa
