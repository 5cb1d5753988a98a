// Head-axis aligner (Sec. 5.1) on tcgen05 tensor cores: the FFN chain of up to three links applied to fp16 score
// tiles, as a set of warp roles that a kernel instantiates (the stand-alone aligner kernel and the fused prefill
// kernel both do).
//
// A tile is 128 (query, key) positions -- two consecutive query rows x one block of 64 key columns -- with all HQ
// heads: in memory [row][head][64 columns] fp16 (one 128-byte line per head and row), which read as a
// tensor-core operand is "M = position contiguous, K = head": the transposition [head][position] ->
// [position][head] that the FFN needs is done by the MMA's operand addressing, not by any thread.
// Per tile t and link k (Eq. 3-4, ADD):
//   MMA1   H[128 x MH]  = X_k[128 x HQ] . W1_k              X_0 = A_0 tile; fp32 accumulator in tensor memory
//   E1     G = act(H + b1) as fp16, one 128-byte row per position (thread = position)
//   MMA2   Y[128 x HQ]  = G . W2_k
//   E2     y = Y + b2;  k + 1 < c: X_{k+1} = y + D_{k+1} written over the D_{k+1} tile (the next link's operand)
//          last link (or every link when all outputs are kept): y goes out, over a tile buffer whose content is dead
// Every (tile, link) has one 8 KB input box (A_0 for k = 0, D_k otherwise) that streams through a ring of NB
// buffers; two tiles are in flight per CTA so that one tile's elementwise stage covers the other's MMAs.
// Warps: 0-3 elementwise stages E1/E2 (thread = position = TMEM lane), 4 TMA loads and stores, 5 MMA issue.
#pragma once
#include "common.cuh"
#include "tc_common.cuh"

namespace lisa {
namespace alignrole {

using namespace tc;

constexpr int HQ = 32, MH = 64;
constexpr int kMaxLinks = 3;
constexpr int BOX_BYTES = 2 * HQ * 128;          // [2 rows][HQ heads][64 cols] fp16
constexpr int G_BYTES = 128 * MH * 2;            // act(H): [128 positions][MH] fp16
constexpr int W1_BYTES = HQ * MH * 2, W2_BYTES = MH * HQ * 2;
constexpr float kLog2e = 1.4426950408889634f;

// Instruction descriptor, kind::f16 with fp16 operands -> fp32 (A/B format fields 0 = f16).
__host__ __device__ constexpr uint32_t umma_idesc_f16(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

struct Weights {   // host pointers' device copies, by link
    const void *w1[kMaxLinks], *b1[kMaxLinks], *w2[kMaxLinks], *b2[kMaxLinks];
    int w_dtype[kMaxLinks], act[kMaxLinks];
};

// Shared-memory plan of the role set; everything 1024-byte aligned where an operand starts.
// NB_ ring buffers, room for the weights of CM links.
template <int NB_, int CM>
struct Smem {
    static constexpr int NB = NB_;
    static constexpr int OFF_W1 = 0;                                  // [CM] images of W1 (MN-major B operand)
    static constexpr int OFF_W2 = OFF_W1 + CM * W1_BYTES;             // [CM] images of W2^T (K-major B operand)
    static constexpr int OFF_BOX = OFF_W2 + CM * W2_BYTES;            // ring
    static constexpr int OFF_G = OFF_BOX + NB * BOX_BYTES;            // [2]
    static constexpr int OFF_BIAS = OFF_G + 2 * G_BYTES;              // [CM] b1[MH] fp32, b2[HQ] fp32
    static constexpr int OFF_BAR = OFF_BIAS + CM * (MH + HQ) * 4;
    static constexpr int N_BARS = 3 * NB + 12;
    static constexpr int TOTAL = OFF_BAR + N_BARS * 8 + 16;
    static constexpr uint32_t TMEM_COLS = 256;                        // H[2]: [0,128), Y[2]: [128,192)
};

struct TileCoord { int c1, c2, c3, c4; };   // TMA coordinates (head offset, row, column block, row block)

__device__ __forceinline__ uint32_t pack_f16_relu(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t silu_h2(uint32_t x) {   // x * sigmoid(x) = (x/2) tanh(x/2) + x/2 on a packed pair
    uint32_t hx, th, r;
    asm("mul.f16x2 %0, %1, %2;" : "=r"(hx) : "r"(x), "r"(0x38003800u));
    asm("tanh.approx.f16x2 %0, %1;" : "=r"(th) : "r"(hx));
    asm("fma.rn.f16x2 %0, %1, %2, %1;" : "=r"(r) : "r"(hx), "r"(th));
    return r;
}

struct Bars {
    uint64_t *a_full, *box_free, *out_ready;   // [NB]
    uint64_t *h_full, *h_free, *h_ready, *y_full, *y_free, *x_ready;   // [2]
};
template <class L>
__device__ __forceinline__ Bars bars_of(uint8_t* smem) {
    constexpr int NB = L::NB;
    uint64_t* b = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    return Bars{b, b + NB, b + 2 * NB, b + 3 * NB, b + 3 * NB + 2, b + 3 * NB + 4, b + 3 * NB + 6, b + 3 * NB + 8, b + 3 * NB + 10};
}

// One thread: barrier initialisation.
template <class L>
__device__ __forceinline__ void init_bars(uint8_t* smem) {
    constexpr int NB = L::NB;
    Bars B = bars_of<L>(smem);
    for (int i = 0; i < NB; ++i) { mbar_init(B.a_full + i, 1); mbar_init(B.box_free + i, 1); mbar_init(B.out_ready + i, 128); }
    for (int i = 0; i < 2; ++i) {
        mbar_init(B.h_full + i, 1); mbar_init(B.h_free + i, 128); mbar_init(B.h_ready + i, 128);
        mbar_init(B.y_full + i, 1); mbar_init(B.y_free + i, 128); mbar_init(B.x_ready + i, 128);
    }
}

// All threads of the CTA (nthreads of them): weights as ready-made operand images.  `fold_log2e`: the last link's
// W2 and b2 carry log2(e) (its output is consumed in the exp2 domain).
template <class L>
__device__ __forceinline__ void stage_weights(uint8_t* smem, const Weights& w, int c, bool fold_log2e, int tid, int nthreads) {
    for (int k = 0; k < c; ++k) {
        uint8_t* w1i = smem + L::OFF_W1 + k * W1_BYTES;
        uint8_t* w2i = smem + L::OFF_W2 + k * W2_BYTES;
        float* bias = reinterpret_cast<float*>(smem + L::OFF_BIAS) + k * (MH + HQ);
        const float out_scale = (k == c - 1 && fold_log2e) ? kLog2e : 1.f;
        const int wd = w.w_dtype[k];
        for (int e = tid; e < HQ * MH; e += nthreads) {   // W1 [head][hidden]: row = K index (head), 64 hidden = one 128-byte line
            const int kk = e / MH, n = e % MH;
            *reinterpret_cast<__half*>(w1i + kk * 128 + ((((n >> 3) ^ (kk & 7))) << 4) + (n & 7) * 2) = __float2half_rn(ld_elem(w.w1[k], e, wd));
        }
        for (int e = tid; e < MH * HQ; e += nthreads) {   // W2 [hidden][head] -> image [head out][hidden]: row = N index
            const int kk = e / HQ, n = e % HQ;
            *reinterpret_cast<__half*>(w2i + n * 128 + ((((kk >> 3) ^ (n & 7))) << 4) + (kk & 7) * 2) =
                __float2half_rn(ld_elem(w.w2[k], e, wd) * out_scale);
        }
        for (int e = tid; e < MH; e += nthreads) bias[e] = w.b1[k] ? ld_elem(w.b1[k], e, wd) : 0.f;
        for (int e = tid; e < HQ; e += nthreads) bias[MH + e] = (w.b2[k] ? ld_elem(w.b2[k], e, wd) : 0.f) * out_scale;
    }
}

// Box order shared by all roles: groups of two tiles; within a group link by link, within a link tile by tile.
__device__ __forceinline__ int box_index(int g, int k, int u, int n_in_group, int c) { return g * 2 * c + k * n_in_group + u; }

// ---- warp 5: MMA issue (all lanes run the loop, lane 0 issues) ------------------------------------------
template <class L>
__device__ __forceinline__ void mma_warp(uint8_t* smem, uint32_t tmem_base, int n_tiles, int c, int lane, volatile int* abort_flag) {
    constexpr int NB = L::NB;
    Bars B = bars_of<L>(smem);
    const uint32_t issue = lane == 0;
    constexpr uint32_t IDESC1 = umma_idesc_f16(128, MH, 1, 1);   // X: positions contiguous; W1: hidden contiguous
    constexpr uint32_t IDESC2 = umma_idesc_f16(128, HQ, 0, 0);   // G, W2^T: K contiguous
    auto desc_off = [](uint64_t d, uint32_t bytes) -> uint64_t { return (d & 0xffffffff00000000ull) | (uint32_t)((uint32_t)d + (bytes >> 4)); };
    const uint64_t dbox0 = umma_desc_sw128(smem_u32(smem + L::OFF_BOX), HQ * 128, 1024);
    const uint64_t dw1 = umma_desc_sw128(smem_u32(smem + L::OFF_W1), HQ * 128, 1024);
    const uint64_t dw2 = umma_desc_sw128(smem_u32(smem + L::OFF_W2), 16, 1024);
    const uint64_t dg0 = umma_desc_sw128(smem_u32(smem + L::OFF_G), 16, 1024);
    uint32_t ph_hfree = 0, ph_xready = 0, ph_hready = 0, ph_yfree = 0;   // bit u: parity of the next phase to wait for
    const int n_groups = (n_tiles + 1) >> 1;
    bool ok = true;
    for (int g = 0; ok && g < n_groups; ++g) {
        const int ng = min(2, n_tiles - 2 * g);
        for (int k = 0; ok && k < c; ++k) {
            for (int u = 0; u < ng; ++u) {
                const int i = box_index(g, k, u, ng, c), slot = i % NB;
                if (k == 0) ok = mbar_wait(B.a_full + slot, (uint32_t)(i / NB) & 1u, abort_flag);
                else { ok = mbar_wait(B.x_ready + u, (ph_xready >> u) & 1u, abort_flag); ph_xready ^= 1u << u; }
                ok = ok && mbar_wait(B.h_free + u, ((ph_hfree >> u) & 1u) ^ 1u, abort_flag);
                ph_hfree ^= 1u << u;
                if (!(ok = __all_sync(0xffffffffu, ok))) break;
                tc_fence_after();
                const uint64_t dx = desc_off(dbox0, slot * BOX_BYTES), dw = desc_off(dw1, k * W1_BYTES);
#pragma unroll
                for (int ks = 0; ks < HQ / 16; ++ks)
                    umma_ss_if(issue, tmem_base + u * MH, desc_off(dx, ks * 2048), desc_off(dw, ks * 2048), IDESC1, ks > 0);
                umma_commit_if(issue, B.h_full + u);
                // a box that nothing is written back into is free again once this MMA has read it
                umma_commit_if(issue, B.box_free + slot);
            }
            if (!ok) break;
            for (int u = 0; u < ng; ++u) {
                ok = mbar_wait(B.h_ready + u, (ph_hready >> u) & 1u, abort_flag) && mbar_wait(B.y_free + u, ((ph_yfree >> u) & 1u) ^ 1u, abort_flag);
                ph_hready ^= 1u << u; ph_yfree ^= 1u << u;
                if (!(ok = __all_sync(0xffffffffu, ok))) break;
                tc_fence_after();
                const uint64_t dg = desc_off(dg0, u * G_BYTES), dw = desc_off(dw2, k * W2_BYTES);
#pragma unroll
                for (int ks = 0; ks < MH / 16; ++ks)
                    umma_ss_if(issue, tmem_base + 128 + u * HQ, desc_off(dg, ks * 32), desc_off(dw, ks * 32), IDESC2, ks > 0);
                umma_commit_if(issue, B.y_full + u);
            }
        }
    }
}

// ---- warps 0-3: elementwise stages (thread = position) ----------------------------------------------------
// store_all: every link's output leaves (times log2 e, applied here); otherwise only the last link's (log2 e folded
// into its weights).
template <class L>
__device__ __forceinline__ void elementwise_warps(uint8_t* smem, uint32_t tmem_base, int n_tiles, int c, bool store_all, const int* acts,
                                                  const bool* has_bias, int tid, volatile int* abort_flag) {
    constexpr int NB = L::NB;
    Bars B = bars_of<L>(smem);
    const int row = tid, warp = tid >> 5;
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
    const int rsel = row >> 6, col = row & 63;
    // this position's 2 bytes inside a box: line of head h = rsel * HQ*128 + h * 128, 16-byte chunk (col / 8) ^ (h % 8)
    const uint32_t pos_off = (uint32_t)(rsel * HQ * 128 + (col & 7) * 2), pos_chunk = (uint32_t)(col >> 3);
    uint32_t ph_hfull = 0, ph_yfull = 0;
    const int n_groups = (n_tiles + 1) >> 1;
    bool ok = true;
    for (int g = 0; ok && g < n_groups; ++g) {
        const int ng = min(2, n_tiles - 2 * g);
        for (int k = 0; ok && k < c; ++k) {
            const float* bias = reinterpret_cast<const float*>(smem + L::OFF_BIAS) + k * (MH + HQ);
            const int act = acts[k];
            const bool biased = has_bias[k];
            // ---- E1: hidden activations ----
            for (int u = 0; u < ng; ++u) {
                if (!(ok = mbar_wait(B.h_full + u, (ph_hfull >> u) & 1u, abort_flag))) break;
                ph_hfull ^= 1u << u;
                tc_fence_after();
                uint32_t hr[MH];
#pragma unroll
                for (int q = 0; q < MH / 32; ++q) tmem_ld32(tmem_base + u * MH + lane_sel + q * 32, hr + q * 32);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(B.h_free + u);
                float* hf = reinterpret_cast<float*>(hr);
                if (biased) {
#pragma unroll
                    for (int j = 0; j < MH; ++j) hf[j] += bias[j];
                }
                uint8_t* gb = smem + L::OFF_G + u * G_BYTES;
#pragma unroll
                for (int q = 0; q < MH / 8; ++q) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float lo = hf[q * 8 + 2 * e], hi = hf[q * 8 + 2 * e + 1];
                        if (act == LISA_ACT_RELU) w[e] = pack_f16_relu(lo, hi);
                        else if (act == LISA_ACT_SILU) w[e] = silu_h2(pack_f16(lo, hi));
                        else w[e] = pack_f16(lo, hi);
                    }
                    *reinterpret_cast<uint4*>(gb + sw128_offset(row, q)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
                fence_async_smem();
                mbar_arrive(B.h_ready + u);
            }
            if (!ok) break;
            // ---- E2: link output ----
            for (int u = 0; u < ng; ++u) {
                if (!(ok = mbar_wait(B.y_full + u, (ph_yfull >> u) & 1u, abort_flag))) break;
                ph_yfull ^= 1u << u;
                tc_fence_after();
                uint32_t yr[HQ];
                tmem_ld32(tmem_base + 128 + u * HQ + lane_sel, yr);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(B.y_free + u);
                float* yf = reinterpret_cast<float*>(yr);
                if (biased) {
#pragma unroll
                    for (int h = 0; h < HQ; ++h) yf[h] += bias[MH + h];
                }
                const int i = box_index(g, k, u, ng, c), slot = i % NB;
                const bool stores = store_all || k == c - 1;
                if (stores) {
                    // over this link's own box: its operand has been consumed (MMA1 of this link completed before E1)
                    uint8_t* ob = smem + L::OFF_BOX + slot * BOX_BYTES + pos_off;
                    const float s = (store_all) ? kLog2e : 1.f;
#pragma unroll
                    for (int h = 0; h < HQ; ++h)
                        *reinterpret_cast<__half*>(ob + h * 128 + ((pos_chunk ^ (uint32_t)(h & 7)) << 4)) = __float2half_rn(yf[h] * s);
                    fence_async_smem();
                    mbar_arrive(B.out_ready + slot);
                }
                if (k + 1 < c) {
                    // X_{k+1} = y + D_{k+1}, in place over the D_{k+1} tile (its box must have landed)
                    const int i2 = box_index(g, k + 1, u, ng, c), slot2 = i2 % NB;
                    if (!(ok = mbar_wait(B.a_full + slot2, (uint32_t)(i2 / NB) & 1u, abort_flag))) break;
                    uint8_t* xb = smem + L::OFF_BOX + slot2 * BOX_BYTES + pos_off;
#pragma unroll
                    for (int h = 0; h < HQ; ++h) {
                        __half* px = reinterpret_cast<__half*>(xb + h * 128 + ((pos_chunk ^ (uint32_t)(h & 7)) << 4));
                        *px = __float2half_rn(yf[h] + __half2float(*px));
                    }
                    fence_async_smem();
                    mbar_arrive(B.x_ready + u);
                }
            }
        }
    }
}

// ---- warp 4: TMA loads and stores ---------------------------------------------------------------------------
// Feed: bool next(TileCoord&) walks this CTA's tiles in order; before_load()/after_store() are hooks that the fused
// kernel uses to wait for and announce whole chunks (they return false to give up).  Two copies of the feed walk
// the same sequence: one ahead for the loads, one for the stores.
template <class L, class Feed>
__device__ __forceinline__ void tma_warp(uint8_t* smem, Feed feed_load, Feed feed_store, int n_tiles, int c, bool store_all,
                                         const CUtensorMap* tm0, const CUtensorMap* tm1, const CUtensorMap* tm2, int lane,
                                         volatile int* abort_flag) {
    constexpr int NB = L::NB;
    Bars B = bars_of<L>(smem);
    if (lane != 0) return;
    tma_prefetch_desc(tm0);
    if (c > 1) tma_prefetch_desc(tm1);
    if (c > 2) tma_prefetch_desc(tm2);
    constexpr int LA = NB - 2;   // boxes loaded ahead of the one being retired
    const int n_groups = (n_tiles + 1) >> 1;
    // loader state
    int lg = 0, lk = 0, lu = 0, li = 0;
    TileCoord lt[2] = {}, st[2] = {};
    int l_ng = min(2, n_tiles), l_have = 0;   // tiles of the loader's current group already fetched from the feed
    auto issue_load = [&]() -> bool {          // loads box (lg, lk, lu); false when there is none left or a hook gave up
        if (lg >= n_groups) return true;
        if (lk == 0 && lu >= l_have) {          // first visit of this tile
            if (!feed_load.next(lt[lu])) return false;
            ++l_have;
        }
        const int slot = li % NB;
        tma_store_wait_read<2>();              // the store that read this buffer was committed at least two stores back: it has finished reading
        mbar_expect_tx(B.a_full + slot, BOX_BYTES);
        void* dst = smem + L::OFF_BOX + slot * BOX_BYTES;
        const TileCoord& t = lt[lu];
        if (lk == 0) tma_load_5d(dst, tm0, B.a_full + slot, 0, t.c1, t.c2, t.c3, t.c4);
        else if (lk == 1) tma_load_5d(dst, tm1, B.a_full + slot, 0, t.c1, t.c2, t.c3, t.c4);
        else tma_load_5d(dst, tm2, B.a_full + slot, 0, t.c1, t.c2, t.c3, t.c4);
        ++li;
        if (++lu == l_ng) {
            lu = 0;
            if (++lk == c) { lk = 0; ++lg; l_ng = min(2, n_tiles - 2 * lg); l_have = 0; }
        }
        return true;
    };
    bool ok = true;
    for (int j = 0; j < LA && ok; ++j) ok = issue_load();
    uint32_t ph_free = 0, ph_out = 0;
    int i = 0;
    for (int g = 0; ok && g < n_groups; ++g) {
        const int ng = min(2, n_tiles - 2 * g);
        for (int u = 0; u < ng; ++u) ok = ok && feed_store.next(st[u]);
        for (int k = 0; ok && k < c; ++k)
            for (int u = 0; ok && u < ng; ++u, ++i) {
                const int slot = i % NB;
                const bool stores = store_all || k == c - 1;
                // every box passes through box_free (its MMA1 has read it); a box that is written back also through out_ready
                ok = mbar_wait(B.box_free + slot, (ph_free >> slot) & 1u, abort_flag);
                ph_free ^= 1u << slot;
                if (ok && stores) {
                    ok = mbar_wait(B.out_ready + slot, (ph_out >> slot) & 1u, abort_flag);
                    ph_out ^= 1u << slot;
                    if (ok) {
                        const void* src = smem + L::OFF_BOX + slot * BOX_BYTES;
                        const TileCoord& t = st[u];
                        const int plane = store_all ? k : 0;
                        if (plane == 0) tma_store_5d(tm0, src, 0, t.c1, t.c2, t.c3, t.c4);
                        else if (plane == 1) tma_store_5d(tm1, src, 0, t.c1, t.c2, t.c3, t.c4);
                        else tma_store_5d(tm2, src, 0, t.c1, t.c2, t.c3, t.c4);
                        tma_store_commit();
                        if (k == c - 1) ok = feed_store.after_store();
                    }
                }
                if (ok) ok = issue_load();
            }
    }
    tma_store_wait_all<0>();
    if (!ok) *abort_flag = 1;
}

}  // namespace alignrole
}  // namespace lisa
