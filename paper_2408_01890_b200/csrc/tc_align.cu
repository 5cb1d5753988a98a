// Head-axis aligner on tensor cores (Sec. 5.1): the FFN chain of a shared layer applied to score planes.
//
// Input: fp16 planes, blocked [row block of 128][column block of 64][row][B*Hq][64 columns], (fp16, not bf16: three more mantissa bits keep a chain of several links
// inside the accuracy bar; scores are O(10), far from fp16's range limit, and conversions saturate) holding
// A_0 = Q0.K0^T/sqrt(d) (Eq. 2) and, for chain depth c > 1, the already scaled differences
// D_k = Q'_k.K'_k^T/sqrt(r) (Eq. 3) of the links k < c.  Output, in place of the A_0 plane:
// Y = log2(e) * FFN_c(A_{c-1}) where A_k = FFN_k(A_{k-1}) + D_k (Eq. 4, ADD) -- the final link's D_c is added by
// the attention kernel that consumes Y.  Hq = 32 heads, hidden width 64, two-layer FFNs.
//
// A warp owns pieces of 32 key positions of one query row and, within a piece, strips of 16 positions as the M
// dimension of warp-level MMAs (mma.sync m16n8k16), keeping the whole chain in registers:
//   global -> scratch      cp.async, 16 bytes per lane, four lanes per head, several pieces ahead
//   H = A [16 x 32] . W1   A fragments by ldmatrix.trans from the warp's [head][position] scratch, so the
//                          [head][position] -> [position][head] transposition costs nothing; fp16 accumulators
//   Y = act(H + b1) . W2   the accumulator registers of H ARE the A fragments of this MMA (packed activation, no
//                          conversion); fp32 accumulators
//   A_k = Y + b2 + D_k     D_k read with the same ldmatrix.trans; packed again it feeds the next link
// and the last Y goes back through the scratch with stmatrix.trans and out with 16-byte stores.
// Why not tcgen05 here: the contractions are tiny (K = 32/64, N = 64/32) and an elementwise step sits between any
// two of them, so with tensor-memory accumulators every step pays a round trip through TMEM, shared memory and an
// mbarrier hand-off between the issuing thread and the threads that apply the activation; measured on B200 that
// version spent ~13 clocks per position and link (tensor pipe 5% busy).  mma.sync runs at a quarter of the tcgen05
// rate (measured 555 TFLOP/s) but nothing leaves the registers.  Every warp is independent: no block-wide barrier
// after set-up, no mbarrier, no wait that could hang.  The kernel is bound by the planes it moves (4 bytes per
// position and head for one link), not by its arithmetic.
#include <algorithm>

#include "tc_align_mma.cuh"

namespace lisa {
namespace {

using namespace tc;
using namespace alignmma;

constexpr int UNIT = 128;
constexpr int kWorkers = 512, kStages = 2;                        // weights read from shared memory: one 16-warp CTA per SM
constexpr int kRegwThreads = 128, kRegwCtas = 3, kRegwStages = 3, kRegwPiece = 64; // weights held in registers (single link)
// the last link's output leaves multiplied by log2(e): the attention kernel that adds it to its logits works in the exp2 domain
constexpr int kMaxTcChain = 3;

struct AlignParams {
    int B, N, chain;               // chain = number of links applied here (c)
    int row0, qt_begin, qt_count;  // planes hold query rows row0.. ; this launch covers tiles [qt_begin, qt_begin + qt_count)
    int units_per_batch;           // sum over the covered tiles of valid rows x key blocks
    int64_t plane_rows, plane_cols;
    __half* planes[kMaxTcChain];   // [0] = A_0 in / Y out; [k] = D_k for k = 1..c-1; blocked, see tc_flash.cu
    const void *w1[kMaxTcChain], *b1[kMaxTcChain], *w2[kMaxTcChain], *b2[kMaxTcChain];
    int w_dtype[kMaxTcChain], act[kMaxTcChain], kind[kMaxTcChain];   // kind: KIND_FFN / KIND_SINGLE / KIND_PLUS
    int store_all;                 // 1: the output of EVERY link k leaves (times log2 e) in plane k, for a chain of layers
    int* status;
};

// Each warp works alone on pieces of 32 key positions of one query row: no block-wide barrier, no producer warp.
//   global -> scratch    cp.async, 16 bytes per lane, four lanes per head (64 contiguous bytes), one piece ahead
//   scratch -> fragments ldmatrix.trans per 16-position strip
//   chain in registers   (ffn_link)
//   result               stmatrix.trans back into the scratch, then 16 bytes per lane to the plane
// ACT0: the activation of every link as a compile-time constant, or -1 = look at the parameters link by link.
// ACT0 >= 8: additionally, the link has no biases.
template <bool REGW, int NT, int MIN_CTAS, int STAGES, int PP, int ACT0>
__global__ void __launch_bounds__(NT, MIN_CTAS)
tc_align_kernel(const __grid_constant__ AlignParams p) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int c = p.chain;
    uint8_t* sW = smem;                               // per link: W1 fragments, W2 fragments, b1[64], b2[32]
    uint8_t* sScr = sW + c * LINK_BYTES;              // per warp: STAGES buffers of c planes x [32 heads][64 B]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- one-time set-up: weights as ready-made B fragments (fp16, the last link's W2/b2 times log2 e) ----
    for (int k = 0; k < c; ++k) {
        // the last link's log2(e) is folded into its W2 and b2, except where every link's output leaves (store_all with
        // more than one link): there the stored values are scaled instead and the chain continues unscaled
        const float out_scale = (k == c - 1 && (!p.store_all || c == 1)) ? kLog2e : 1.f;
        stage_link_fragments(sW + k * LINK_BYTES, p.w1[k], p.b1[k], p.w2[k], p.b2[k], p.w_dtype[k], p.kind[k], out_scale, tid, NT);
    }
    __syncthreads();

    // Parameter fields of the main loop, read once into registers: behind the asm statements (memory clobbers) the
    // compiler would re-read them from the parameter bank every time, the per-link ones through a run-time index.
    const int pB = p.B, pN = p.N, p_row0 = p.row0, p_qt0 = p.qt_begin, p_qt1 = p.qt_begin + p.qt_count;
    const int p_ncb = (int)(p.plane_cols >> 6);
    const bool store_all = p.store_all != 0;
    __half* const plane0 = p.planes[0];
    __half* const plane1 = p.planes[1];
    __half* const plane2 = p.planes[2];
    auto plane_ptr = [&](int k) { return k == 0 ? plane0 : (k == 1 ? plane1 : plane2); };
    const int act0 = p.act[0], act1 = p.act[1], act2 = p.act[2];
    // ---- this warp's contiguous range of pieces; a piece is PP (32 or 64) positions of a 128-position unit ----
    constexpr int PPU = UNIT / PP;                 // pieces per unit
    constexpr int PLANE_SCR = HQ * PP * 2;         // scratch bytes of one plane of a piece: [32 heads][PP positions]
    constexpr int CPR = PP / 8;                    // 16-byte chunks per head row
    const long long n_pieces = (long long)p.units_per_batch * pB * PPU;
    const long long n_warps = (long long)gridDim.x * (NT / 32);
    const long long per_warp = (n_pieces + n_warps - 1) / n_warps;
    const long long s_begin = min(n_pieces, ((long long)blockIdx.x * (NT / 32) + warp) * per_warp);
    const long long s_end = min(n_pieces, s_begin + per_warp);
    if (s_begin >= s_end) return;
    struct Cursor { int b, t, row, jb, sub; };   // batch, query tile, row in the tile, key block, piece in the block
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
    // Global <-> scratch: CPR lanes cover the PP * 2 bytes [head][PP positions] of one head, so one warp-wide access
    // touches 32 / CPR heads; 128 / CPR... PP * 4 / 32 accesses move a piece of one plane (with PP = 64 a piece is one
    // contiguous 4 KB run of the blocked plane).  Scratch rows are one head; the 16-byte chunk index is XOR-ed with
    // the head index (over as many bits as there are chunks) so that the 8 rows of an 8x8 matrix fall into distinct banks.
    constexpr int HPA = 32 / CPR;                  // heads per warp-wide access
    constexpr int NACC = HQ / HPA;                 // accesses per plane and piece
    const int l_head = lane / CPR, l_chunk = lane % CPR;
    // element offset of [this lane's first head][this piece] + this lane's chunk; the lane's other heads follow every
    // HPA * 64 elements (blocked plane: [row block of 128][column block of 64][row in block][b*HQ + head][64 columns])
    auto piece_off = [&](const Cursor& x) {
        const int r = x.t * UNIT + x.row - p_row0;
        const int col = x.sub * PP;                // within the 128-column key block
        const int64_t blk = (int64_t)(r >> 7) * p_ncb + (x.jb * 2 + (col >> 6));
        return ((blk * 128 + (r & 127)) * (pB * HQ) + (x.b * HQ + l_head)) * 64 + (col & 63) + l_chunk * 8;
    };
    auto scr_off = [&](int head, int chunk) {
        return (uint32_t)(head * (PP * 2) + ((chunk ^ (PP == 64 ? (head & 7) : ((head >> 1) & 3))) << 4));
    };
    uint8_t* scr = sScr + warp * (STAGES * c * PLANE_SCR);   // [STAGES buffers][c planes][32 heads][PP * 2 B]
    auto fetch = [&](const Cursor& x, int buf) {          // asynchronous global -> scratch copy of a piece, all planes
        const int64_t off = piece_off(x);
#pragma unroll
        for (int k = 0; k < kMaxTcChain; ++k)
            if (k < c) {
#pragma unroll
                for (int i = 0; i < NACC; ++i) {
                    const int head = l_head + HPA * i;
                    const uint32_t dst = smem_u32(scr + (buf * c + k) * PLANE_SCR) + scr_off(head, l_chunk);
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(plane_ptr(k) + off + i * (HPA * 64)) : "memory");
                }
            }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    const int mi = lane >> 3, lr = lane & 7;               // ldmatrix/stmatrix: matrix index and row supplied by this lane
    // strip s2 (16 positions) of the piece, 16-head block x: head block half (mi >> 1), position half (mi & 1)
    auto frag_off = [&](int s2, int x) { return scr_off(x * 16 + 8 * (mi >> 1) + lr, 2 * s2 + (mi & 1)); };

    uint2 w1r[16], w2r[16];
    if constexpr (REGW) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            w1r[i] = reinterpret_cast<const uint2*>(sW)[i * 32 + lane];
            w2r[i] = reinterpret_cast<const uint2*>(sW + W1F_BYTES)[i * 32 + lane];
        }
    }
    if constexpr (REGW) {
        // One link, weights in registers.  Three scratch buffers rotate: the piece being worked on, the next one (copied
        // in meanwhile) and the previous one (copied out meanwhile).  Both copies are cut into one part per strip and
        // issued in the middle of the strip's FFN, between its two groups of MMAs, where the warp would otherwise only
        // wait for its turn on the tensor pipe; done as blocks of their own before and after a piece, they cost the
        // warp about a quarter of its time with nothing of its own on the pipe.
        static_assert(!REGW || STAGES == 3, "previous, current and next piece");
        constexpr int NS = PP / 16, APS = NACC / NS;   // strips per piece, accesses of each copy per strip
        static_assert(!REGW || NACC % NS == 0, "the copies divide evenly over the strips");
        const uint2* w1f = reinterpret_cast<const uint2*>(sW);
        const uint2* w2f = reinterpret_cast<const uint2*>(sW + W1F_BYTES);
        const float* b1 = reinterpret_cast<const float*>(sW + W1F_BYTES + W2F_BYTES);
        const uint32_t* b1h = reinterpret_cast<const uint32_t*>(b1);
        fetch(cu, 0);
        Cursor here = cu, nxt = cu, prev = cu;
        advance(nxt);
        bool has_prev = false;
        int b_cur = 0, b_next = 1, b_prev = 2;
        for (long long sidx = s_begin; sidx < s_end; ++sidx) {
            const bool has_next = sidx + 1 < s_end;
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();
            __half* const g_next = plane0 + (has_next ? piece_off(nxt) : 0);
            __half* const g_prev = plane0 + (has_prev ? piece_off(prev) : 0);
            const uint32_t base = smem_u32(scr + b_cur * PLANE_SCR), s_next = smem_u32(scr + b_next * PLANE_SCR);
            const uint8_t* s_prev = scr + b_prev * PLANE_SCR;
#pragma unroll
            for (int s2 = 0; s2 < NS; ++s2) {
                const uint32_t off0 = frag_off(s2, 0), off1 = frag_off(s2, 1);
                uint32_t afr[2][4];
                ldmatrix_x4_trans(afr[0], base + off0);
                ldmatrix_x4_trans(afr[1], base + off1);
                float y[4][4];
                auto side = [&] {
#pragma unroll
                    for (int j = 0; j < APS; ++j) {
                        const int i = s2 * APS + j, head = l_head + HPA * i;
                        const uint32_t so = scr_off(head, l_chunk);
                        if (has_next) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s_next + so), "l"(g_next + i * (HPA * 64)) : "memory");
                        if (has_prev) *reinterpret_cast<uint4*>(g_prev + i * (HPA * 64)) = *reinterpret_cast<const uint4*>(s_prev + so);
                    }
                };
                ffn_link<(ACT0 < 0 ? LISA_ACT_NONE : (ACT0 & 7)), true, (ACT0 < 8)>(afr, w1f, w2f, w1r, w2r, b1h, b1 + MH, lane, y, side);
                __syncwarp();
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    uint32_t r[4];
                    r[0] = pack_f16(y[2 * x][0], y[2 * x][1]);
                    r[1] = pack_f16(y[2 * x][2], y[2 * x][3]);
                    r[2] = pack_f16(y[2 * x + 1][0], y[2 * x + 1][1]);
                    r[3] = pack_f16(y[2 * x + 1][2], y[2 * x + 1][3]);
                    stmatrix_x4_trans(base + (x ? off1 : off0), r);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            __syncwarp();
            prev = here; has_prev = true;
            here = nxt;
            if (has_next) advance(nxt);
            const int b_old = b_prev;
            b_prev = b_cur; b_cur = b_next; b_next = b_old;
        }
        // the last piece leaves on its own
        {
            const int64_t off = piece_off(prev);
#pragma unroll
            for (int i = 0; i < NACC; ++i) {
                const int head = l_head + HPA * i;
                *reinterpret_cast<uint4*>(plane0 + off + i * (HPA * 64)) = *reinterpret_cast<const uint4*>(scr + b_prev * PLANE_SCR + scr_off(head, l_chunk));
            }
        }
        return;
    }
    // STAGES - 1 pieces are in flight ahead of the one being worked on; one commit group per piece (an empty group
    // past the end keeps the count uniform), so waiting for all but the newest STAGES - 1 groups completes this one.
    Cursor ahead = cu;
    long long fidx = s_begin;
#pragma unroll
    for (int i = 0; i < STAGES - 1; ++i, ++fidx) {
        if (fidx < s_end) { fetch(ahead, i); advance(ahead); }
        else asm volatile("cp.async.commit_group;" ::: "memory");
    }
    int buf = 0, fbuf = STAGES - 1;
    for (long long sidx = s_begin; sidx < s_end; ++sidx, ++fidx) {
        const Cursor here = cu;
        advance(cu);
        if (fidx < s_end) { fetch(ahead, fbuf); advance(ahead); }
        else asm volatile("cp.async.commit_group;" ::: "memory");
        fbuf = fbuf + 1 == STAGES ? 0 : fbuf + 1;
        asm volatile("cp.async.wait_group %0;" ::"n"(STAGES - 1) : "memory");
        __syncwarp();
        const uint32_t base = smem_u32(scr + buf * c * PLANE_SCR);
        // both 16-position strips of the piece go through the chain together: every weight fragment read from shared
        // memory feeds two MMAs
        constexpr int NS = PP / 16;
        static_assert(REGW || NS == 2, "the chain path works on two strips at a time");
        {
            uint32_t afr[NS][2][4];
#pragma unroll
            for (int s2 = 0; s2 < NS; ++s2) {
                ldmatrix_x4_trans(afr[s2][0], base + frag_off(s2, 0));
                ldmatrix_x4_trans(afr[s2][1], base + frag_off(s2, 1));
            }
            float y[NS][4][4];
            for (int k = 0; k < c; ++k) {
                const uint2* w1f = reinterpret_cast<const uint2*>(sW + k * LINK_BYTES);
                const uint2* w2f = reinterpret_cast<const uint2*>(sW + k * LINK_BYTES + W1F_BYTES);
                const float* b1 = reinterpret_cast<const float*>(sW + k * LINK_BYTES + W1F_BYTES + W2F_BYTES);
                const uint32_t* b1h = reinterpret_cast<const uint32_t*>(b1);
                const int act = k == 0 ? act0 : (k == 1 ? act1 : act2);
                if constexpr (ACT0 >= 0) {   // every link has this activation (and, from 8 up, no biases)
                    ffn_link_strips<(ACT0 & 7), (ACT0 < 8), NS>(afr, w1f, w2f, b1h, b1 + MH, lane, y);
                } else {
                    if (act == LISA_ACT_RELU) ffn_link_strips<LISA_ACT_RELU, true, NS>(afr, w1f, w2f, b1h, b1 + MH, lane, y);
                    else if (act == LISA_ACT_SILU) ffn_link_strips<LISA_ACT_SILU, true, NS>(afr, w1f, w2f, b1h, b1 + MH, lane, y);
                    else ffn_link_strips<LISA_ACT_NONE, true, NS>(afr, w1f, w2f, b1h, b1 + MH, lane, y);
                }
                if (store_all && k + 1 < c) {
                    // a chain of layers: link k's own output leaves too, over plane k's place in the scratch (plane 0 = A_0
                    // and plane k = D_k have been consumed by every lane before this link's MMAs could complete)
                    __syncwarp();
#pragma unroll
                    for (int s2 = 0; s2 < NS; ++s2)
#pragma unroll
                        for (int x = 0; x < 2; ++x) {
                            uint32_t r[4];
                            r[0] = pack_f16(y[s2][2 * x][0] * kLog2e, y[s2][2 * x][1] * kLog2e);
                            r[1] = pack_f16(y[s2][2 * x][2] * kLog2e, y[s2][2 * x][3] * kLog2e);
                            r[2] = pack_f16(y[s2][2 * x + 1][0] * kLog2e, y[s2][2 * x + 1][1] * kLog2e);
                            r[3] = pack_f16(y[s2][2 * x + 1][2] * kLog2e, y[s2][2 * x + 1][3] * kLog2e);
                            stmatrix_x4_trans(base + k * PLANE_SCR + frag_off(s2, x), r);
                        }
                }
                if (k + 1 < c) {
                    // A_{k+1} = y + D_{k+1}; the difference comes in the same fragment arrangement as A did
#pragma unroll
                    for (int s2 = 0; s2 < NS; ++s2)
#pragma unroll
                        for (int x = 0; x < 2; ++x) {
                            uint32_t dfr[4];
                            ldmatrix_x4_trans(dfr, base + (k + 1) * PLANE_SCR + frag_off(s2, x));
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float2 dv = unpack_f16(dfr[q]);
                                float* yy = y[s2][2 * x + (q >> 1)] + 2 * (q & 1);
                                afr[s2][x][q] = pack_f16(yy[0] + dv.x, yy[1] + dv.y);
                            }
                        }
                }
            }
            // the last link's result over its place in the scratch (plane 0, or plane c-1 in a chain of layers; every
            // lane's ldmatrix of it is done), transposed back
            const float last_scale = (store_all && c > 1) ? kLog2e : 1.f;
            const uint32_t last_plane = store_all ? (uint32_t)(c - 1) * PLANE_SCR : 0u;
            __syncwarp();
#pragma unroll
            for (int s2 = 0; s2 < NS; ++s2)
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    uint32_t r[4];
                    r[0] = pack_f16(y[s2][2 * x][0] * last_scale, y[s2][2 * x][1] * last_scale);
                    r[1] = pack_f16(y[s2][2 * x][2] * last_scale, y[s2][2 * x][3] * last_scale);
                    r[2] = pack_f16(y[s2][2 * x + 1][0] * last_scale, y[s2][2 * x + 1][1] * last_scale);
                    r[3] = pack_f16(y[s2][2 * x + 1][2] * last_scale, y[s2][2 * x + 1][3] * last_scale);
                    stmatrix_x4_trans(base + last_plane + frag_off(s2, x), r);
                }
        }
        __syncwarp();
        const int64_t here_off = piece_off(here);
#pragma unroll
        for (int k = 0; k < kMaxTcChain; ++k)
            if (k == 0 || (store_all && k < c)) {
#pragma unroll
                for (int i = 0; i < NACC; ++i) {
                    const int head = l_head + HPA * i;
                    *reinterpret_cast<uint4*>(plane_ptr(k) + here_off + i * (HPA * 64)) =
                        *reinterpret_cast<const uint4*>(scr + (buf * c + k) * PLANE_SCR + scr_off(head, l_chunk));
                }
            }
        __syncwarp();   // the next iteration's fetch refills the buffer that was stored one iteration ago, not this one
        buf = buf + 1 == STAGES ? 0 : buf + 1;
    }
}

size_t align_smem_bytes(int c, int threads, int stages, int piece) {
    return (size_t)c * (W1F_BYTES + W2F_BYTES + (MH + HQ) * 4) + (size_t)(threads / 32) * stages * c * (HQ * piece * 2) + 16;
}

}  // namespace

bool tc_align_supported(int Hq, const lisa_link* links, int chain) {
    if (Hq != HQ || chain < 1 || chain > kMaxTcChain) return false;
    for (int k = 0; k < chain; ++k) {
        const lisa_link& l = links[k];
        // ADD with the two-layer 32 -> 64 -> 32 FFN or with one linear 32 x 32 layer; PLUS (no FFN).  CONCAT runs on the general kernel.
        const bool ffn2 = l.integrate == LISA_INTEGRATE_ADD && l.ffn_layers == 2 && l.m == MH;
        const bool single = l.integrate == LISA_INTEGRATE_ADD && l.ffn_layers == 1 && l.m == HQ;
        if (!ffn2 && !single && l.integrate != LISA_INTEGRATE_PLUS) return false;
    }
    return true;
}

cudaError_t launch_tc_align(const TcAlignArgs& a, cudaStream_t stream) {
    AlignParams p{};
    p.B = a.B; p.N = a.N; p.chain = a.chain;
    p.row0 = a.row0 >= 0 ? a.row0 : a.qt_begin * UNIT; p.qt_begin = a.qt_begin; p.qt_count = a.qt_count;
    if (p.row0 % UNIT != 0 || p.row0 > a.qt_begin * UNIT) return cudaErrorInvalidValue;
    p.plane_rows = a.plane_rows; p.plane_cols = a.plane_cols;
    p.units_per_batch = 0;
    for (int t = a.qt_begin; t < a.qt_begin + a.qt_count; ++t) p.units_per_batch += std::min(UNIT, a.N - t * UNIT) * (t + 1);
    for (int k = 0; k < a.chain; ++k) {
        p.planes[k] = reinterpret_cast<__half*>(a.planes[k]);
        const lisa_link& l = a.links[k];
        p.w1[k] = l.w1; p.b1[k] = l.b1; p.w2[k] = l.w2; p.b2[k] = l.b2;
        p.kind[k] = link_kind(l.integrate, l.ffn_layers);
        p.w_dtype[k] = l.w_dtype; p.act[k] = p.kind[k] == KIND_FFN ? l.act : LISA_ACT_NONE;   // only a hidden layer has an activation
    }
    p.store_all = a.store_all ? 1 : 0;
    p.status = status_words();
    if (!p.status) return cudaErrorUnknown;
    if (a.plane_cols % 64 != 0 || a.plane_rows % 128 != 0) return cudaErrorInvalidValue;   // whole blocks
    // One link: its weight fragments live in registers, 4-warp CTAs, three per SM, three pieces in flight per warp.
    // Longer chains: weights in shared memory, one 16-warp CTA per SM, one piece in flight per warp.
    const bool regw = a.chain == 1;
    const int threads = regw ? kRegwThreads : kWorkers;
    const int ctas_per_sm = regw ? kRegwCtas : 1;
    const size_t smem = align_smem_bytes(a.chain, threads, regw ? kRegwStages : kStages, regw ? kRegwPiece : 32);
    auto kernel = tc_align_kernel<false, kWorkers, 1, kStages, 32, -1>;
    const int act = p.act[0];
    bool bias = false, same_act = true;
    for (int k = 0; k < a.chain; ++k) {
        bias = bias || (p.kind[k] != KIND_PLUS && (a.links[k].b1 || (p.kind[k] == KIND_FFN && a.links[k].b2)));
        same_act = same_act && p.act[k] == act;
    }
    if (!regw && same_act) {
#define LISA_ALIGN_CHAIN(A_) (bias ? tc_align_kernel<false, kWorkers, 1, kStages, 32, (A_)> : tc_align_kernel<false, kWorkers, 1, kStages, 32, (A_) + 8>)
        kernel = act == LISA_ACT_RELU ? LISA_ALIGN_CHAIN(LISA_ACT_RELU) : act == LISA_ACT_SILU ? LISA_ALIGN_CHAIN(LISA_ACT_SILU) : LISA_ALIGN_CHAIN(LISA_ACT_NONE);
#undef LISA_ALIGN_CHAIN
    }
    if (regw) {
#define LISA_ALIGN_REGW(A_) (bias ? tc_align_kernel<true, kRegwThreads, kRegwCtas, kRegwStages, kRegwPiece, (A_)> \
                                  : tc_align_kernel<true, kRegwThreads, kRegwCtas, kRegwStages, kRegwPiece, (A_) + 8>)
        kernel = act == LISA_ACT_RELU ? LISA_ALIGN_REGW(LISA_ACT_RELU) : act == LISA_ACT_SILU ? LISA_ALIGN_REGW(LISA_ACT_SILU) : LISA_ALIGN_REGW(LISA_ACT_NONE);
#undef LISA_ALIGN_REGW
    }
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t total_units = (int64_t)p.units_per_batch * a.B;
    if (total_units <= 0 || total_units > 0x7fffffff) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int max_ctas = a.ctas > 0 ? a.ctas : sms * ctas_per_sm;
    dim3 grid((unsigned)std::min<int64_t>((total_units + 3) / 4, max_ctas));  // at least a unit per warp
    kernel<<<grid, threads, smem, stream>>>(p);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace lisa
