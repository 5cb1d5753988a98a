// Head-axis aligner on tensor cores (Sec. 5.1): the FFN chain of a shared layer applied to score planes.
//
// Input: fp16 planes [B*Hq][rows][cols] (fp16, not bf16: three more mantissa bits keep a chain of several links
// inside the accuracy bar; scores are O(10), far from fp16's range limit, and conversions saturate) holding A_0 = Q0.K0^T/sqrt(d) (Eq. 2) and, for chain depth c > 1, the
// already scaled differences D_k = Q'_k.K'_k^T/sqrt(r) (Eq. 3) of the links k < c.  Output, in place of the A_0
// plane: Y = log2(e) * FFN_c(A_{c-1}) where A_k = FFN_k(A_{k-1}) + D_k (Eq. 4, ADD) -- the final link's D_c is added by the
// attention kernel that consumes Y.  Hq = 32 heads, hidden width 64, two-layer FFNs.
//
// A work unit is 128 consecutive key positions of one query row; positions are the M dimension of the MMAs:
//   H  [128 x 64] = A [128 x 32] . W1 [32 x 64]     A read MN-major straight from the [head][position] planes
//   Y  [128 x 32] = act(H + b1) [128 x 64] . W2 [64 x 32]  (+ D_k [128 x 32] . I [32 x 32] for k < c)
// so the tensor core does the [head][position] -> [position][head] transposition.  One thread per position
// applies bias and activation between the two MMAs and writes the result planes.  Weights are converted to fp16.
#include <algorithm>

#include "common.cuh"
#include "tc_common.cuh"

namespace lisa {
namespace {

using namespace tc;

constexpr int HQ = 32, MH = 64, UNIT = 128;
constexpr int kThreads = 128;
constexpr int SLAB_BYTES = 2 * HQ * 128;   // [2 halves of 64 positions][32 heads][128 B]
constexpr int W1_BYTES = MH * 128;         // B operand, K-major: row = hidden unit, 64 k-slots (32 heads + zero pad)
constexpr int W2_BYTES = HQ * 128;         // row = output head, k = 64 hidden units
constexpr int AT_BYTES = UNIT * 128;       // A operand, K-major: row = position, 64 k-slots
constexpr uint32_t TMEM_COLS = 256;        // D1[2]: [0,128), D2[2]: [128,192)
constexpr float kLog2e = 1.4426950408889634f;  // the last link's output leaves multiplied by log2(e): the attention
                                               // kernel that adds it to its logits works in the exp2 domain
constexpr int kMaxTcChain = 3;  // shared memory holds the slabs and weights of at most three links

struct AlignParams {
    int B, N, chain;         // chain = number of links applied here (c)
    int row0, qt_begin, qt_count;  // planes hold query rows row0.. ; this launch covers tiles [qt_begin, qt_begin + qt_count)
    int stages;              // depth of the slab ring (2..4)
    int units_per_batch;     // sum over the covered tiles of valid rows x key blocks
    int64_t plane_rows, plane_cols;
    __half* planes[kMaxTcChain];  // [0] = A_0 in / Y out; [k] = D_k for k = 1..c-1
    const void *w1[kMaxTcChain], *b1[kMaxTcChain], *w2[kMaxTcChain], *b2[kMaxTcChain];
    int w_dtype[kMaxTcChain], act[kMaxTcChain];
    int* status;
};

__device__ __forceinline__ float ldw(const void* p, int idx, int dtype) { return p ? ld_elem(p, idx, dtype) : 0.f; }

// Activation of two hidden units, result packed fp16 (it feeds an fp16 MMA operand).
template <int ACT>
__device__ __forceinline__ uint32_t act_pair(float x0, float x1) {
    if constexpr (ACT == LISA_ACT_RELU) return pack_f16(fmaxf(x0, 0.f), fmaxf(x1, 0.f));
    if constexpr (ACT == LISA_ACT_SILU) {
        // x * sigmoid(x) with one ex2 and one rcp per unit (both full-rate MUFU ops; packed tanh is quarter rate)
        float e0, e1, r0, r1;
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(x0 * -1.4426950408889634f));
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(x1 * -1.4426950408889634f));
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(1.f + e0));
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(1.f + e1));
        return pack_f16(x0 * r0, x1 * r1);
    }
    return pack_f16(x0, x1);
}

// One position's 64 hidden pre-activations (32 at a time from tensor memory) -> bias, activation, fp16 -> its row
// of the K-major H tile.
template <int ACT, bool BIAS>
__device__ __forceinline__ void hidden_row(uint32_t taddr, const float* b1, uint8_t* hrow, int row) {
    uint32_t hr[64];
    tmem_ld32(taddr, hr);
    tmem_ld32(taddr + 32, hr + 32);
    tmem_wait_ld();
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        float x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = __uint_as_float(hr[q * 8 + e]) + (BIAS ? b1[q * 8 + e] : 0.f);
        uint4 v;
        v.x = act_pair<ACT>(x[0], x[1]); v.y = act_pair<ACT>(x[2], x[3]);
        v.z = act_pair<ACT>(x[4], x[5]); v.w = act_pair<ACT>(x[6], x[7]);
        *reinterpret_cast<uint4*>(hrow + sw128_offset(row, q)) = v;
    }
}

template <bool BIAS>
__device__ __forceinline__ void hidden_row_dispatch(int act, uint32_t taddr, const float* b1, uint8_t* hrow, int row) {
    if (act == LISA_ACT_RELU) hidden_row<LISA_ACT_RELU, BIAS>(taddr, b1, hrow, row);
    else if (act == LISA_ACT_SILU) hidden_row<LISA_ACT_SILU, BIAS>(taddr, b1, hrow, row);
    else hidden_row<LISA_ACT_NONE, BIAS>(taddr, b1, hrow, row);
}

struct TensorMaps {
    CUtensorMap m[kMaxTcChain];
};

__global__ void __launch_bounds__(kThreads + 64, 2)
tc_align_kernel(const __grid_constant__ AlignParams p, const __grid_constant__ TensorMaps maps) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int c = p.chain;
    // Units are processed in pairs; everything a unit touches exists twice (index j = 0,1 inside the pair).
    // layout: [2 stages][2 units][c slabs] | H[2] | A[2] (c > 1) | out[2] | identity | W1,W2 per link | biases | barriers
    uint8_t* sSlab = smem;
    uint8_t* sH = sSlab + 4 * c * SLAB_BYTES;
    uint8_t* sA = sH + 2 * AT_BYTES;
    uint8_t* sOut = sA + (c > 1 ? 2 * AT_BYTES : 0);
    uint8_t* sI = sOut + 2 * SLAB_BYTES;
    uint8_t* sW = sI + W2_BYTES;
    float* sBias = reinterpret_cast<float*>(sW + c * (W1_BYTES + W2_BYTES));  // per link: b1[64], b2[32]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sBias + c * (MH + HQ));
    uint64_t* full = bars;            // [2] stage filled by TMA
    uint64_t* slabs_done = bars + 2;  // [2] every MMA reading the stage's slabs has completed
    uint64_t* d1_full = bars + 4;     // [2] first-layer accumulator of unit j ready
    uint64_t* d2_full = bars + 6;     // [2] second-layer accumulator of unit j ready
    uint64_t* h_ready = bars + 8;     // [2] workers wrote H[j]
    uint64_t* a_ready = bars + 10;    // [2] workers wrote A[j] for the next link
    uint64_t* out_ready = bars + 12;  // [2] workers filled staging buffer i
    uint64_t* out_free = bars + 14;   // [2] the store of staging buffer i has read it
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 17);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int n_units = p.units_per_batch * p.B;
    // Every CTA owns a contiguous range of units [u_begin, u_end); units are numbered batch by batch, tile by
    // tile, row by row, key block by key block, so a cursor steps through them without any division.
    const int per_cta = (n_units + (int)gridDim.x - 1) / (int)gridDim.x;
    const int u_begin = min(n_units, (int)blockIdx.x * per_cta), u_end = min(n_units, u_begin + per_cta);
    const int n_mine = u_end - u_begin;
    const int n_pairs = (n_mine + 1) / 2;
    struct Cursor { int b, t, row, jb; };   // batch, query tile, row inside the tile, key block
    auto cursor_at = [&](int u) {
        Cursor cu;
        cu.b = u / p.units_per_batch;
        int rem = u - cu.b * p.units_per_batch;
        cu.t = p.qt_begin;
        for (;; ++cu.t) {
            const int n_t = min(UNIT, p.N - cu.t * UNIT) * (cu.t + 1);
            if (rem < n_t || cu.t + 1 >= p.qt_begin + p.qt_count) break;
            rem -= n_t;
        }
        cu.row = rem / (cu.t + 1);
        cu.jb = rem - cu.row * (cu.t + 1);
        return cu;
    };
    auto advance = [&](Cursor& cu) {
        if (++cu.jb <= cu.t) return;
        cu.jb = 0;
        if (++cu.row < min(UNIT, p.N - cu.t * UNIT)) return;
        cu.row = 0;
        if (++cu.t < p.qt_begin + p.qt_count) return;
        cu.t = p.qt_begin;
        ++cu.b;
    };

    // ---- one-time set-up: barriers, TMEM, weights as swizzled fp16 MMA operands ----
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(full + i, 1); mbar_init(slabs_done + i, 1);
            mbar_init(d1_full + i, 1); mbar_init(d2_full + i, 1);
            mbar_init(h_ready + i, kThreads); mbar_init(a_ready + i, kThreads);
            mbar_init(out_ready + i, kThreads); mbar_init(out_free + i, 1);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 4) tmem_alloc(tmem_slot, TMEM_COLS);
    for (int e = tid; e < (W2_BYTES + c * (W1_BYTES + W2_BYTES)) / 16; e += blockDim.x) reinterpret_cast<uint4*>(sI)[e] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int e = tid; e < HQ; e += blockDim.x)  // identity: row g, k-slot g
        *reinterpret_cast<__half*>(sI + sw128_offset(e, e >> 3) + (e & 7) * 2) = __float2half_rn(1.f);
    for (int k = 0; k < c; ++k) {
        uint8_t* w1t = sW + k * (W1_BYTES + W2_BYTES);
        uint8_t* w2t = w1t + W1_BYTES;
        for (int e = tid; e < HQ * MH; e += blockDim.x) {
            const int hh = e / MH, u = e % MH;  // W1[hh][u] -> row u, k-slot hh
            *reinterpret_cast<__half*>(w1t + sw128_offset(u, hh >> 3) + (hh & 7) * 2) = __float2half_rn(ld_elem(p.w1[k], e, p.w_dtype[k]));
            const int u2 = e / HQ, gg = e % HQ;  // W2[u2][gg] -> row gg, k-slot u2
            *reinterpret_cast<__half*>(w2t + sw128_offset(gg, u2 >> 3) + (u2 & 7) * 2) =
                __float2half_rn(ld_elem(p.w2[k], e, p.w_dtype[k]) * (k == c - 1 ? kLog2e : 1.f));
        }
        for (int e = tid; e < MH; e += blockDim.x) sBias[k * (MH + HQ) + e] = ldw(p.b1[k], e, p.w_dtype[k]);
        for (int e = tid; e < HQ; e += blockDim.x)
            sBias[k * (MH + HQ) + MH + e] = ldw(p.b2[k], e, p.w_dtype[k]) * (k == c - 1 ? kLog2e : 1.f);
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // D1[j] at columns j*64, D2[j] at 128 + j*32

    constexpr uint32_t IDESC_1_MN = umma_idesc_f16(UNIT, MH, 1, 0);
    constexpr uint32_t IDESC_1_K = umma_idesc_f16(UNIT, MH, 0, 0);
    constexpr uint32_t IDESC_2 = umma_idesc_f16(UNIT, HQ, 0, 0);
    constexpr uint32_t IDESC_ID = umma_idesc_f16(UNIT, HQ, 1, 0);

    if (warp == 4) {
        // =========================== producer + MMA issuer (one thread) ===========================
        if (tid == kThreads) {
            for (int k = 0; k < c; ++k) tma_prefetch_desc(&maps.m[k]);
            Cursor cu = cursor_at(u_begin);
            // loads the next pair of this CTA's range (in order) into the given stage: one 4-D TMA per unit and plane
            auto issue_loads = [&](int pair_idx, int stage) {
                const int nvalid = min(2, n_mine - 2 * pair_idx);
                mbar_expect_tx(full + stage, nvalid * c * SLAB_BYTES);
                for (int j = 0; j < nvalid; ++j) {
                    for (int k = 0; k < c; ++k)
                        tma_load_4d(sSlab + ((stage * 2 + j) * c + k) * SLAB_BYTES, &maps.m[k], full + stage, 0, cu.b * HQ, cu.jb * 2,
                                    cu.t * UNIT + cu.row - p.row0);
                    advance(cu);
                }
            };
            uint32_t ph_h[2] = {0, 0}, ph_a[2] = {0, 0};
            bool ok = true;
            int it = 0;
            if (n_pairs > 0) issue_loads(0, 0);
            for (int pr = 0; ok && pr < n_pairs; ++pr, ++it) {
                const int stage = it & 1;
                const int nu = min(2, n_mine - 2 * pr);
                const int prn = pr + 1;
                if (prn < n_pairs) {
                    // the other stage was read by the MMAs of the previous pair
                    if (it > 0 && !(ok = mbar_wait(slabs_done + (stage ^ 1), ((it - 1) >> 1) & 1, abort_flag))) break;
                    issue_loads(prn, stage ^ 1);
                }
                if (!(ok = mbar_wait(full + stage, (it >> 1) & 1, abort_flag))) break;
                for (int k = 0; ok && k < c; ++k) {
                    const uint32_t w1a = smem_u32(sW + k * (W1_BYTES + W2_BYTES)), w2a = w1a + W1_BYTES;
                    for (int j = 0; j < nu; ++j) {
                        if (k > 0 && !(ok = mbar_wait(a_ready + j, ph_a[j], abort_flag))) break;
                        if (k > 0) ph_a[j] ^= 1;
                        tc_fence_after();
                        const uint32_t slab = smem_u32(sSlab + (stage * 2 + j) * c * SLAB_BYTES);
#pragma unroll
                        for (int ks = 0; ks < HQ / 16; ++ks) {
                            const uint64_t bdesc = umma_desc_sw128(w1a + ks * 32, 16, 1024);
                            if (k == 0)  // A_0 slabs: MN-major, 64 positions per 128-byte row, one row per head
                                umma_ss(tmem_base + j * 64, umma_desc_sw128(slab + ks * 2048, HQ * 128, 1024), bdesc, IDESC_1_MN, ks > 0);
                            else         // A_k written by the workers, K-major
                                umma_ss(tmem_base + j * 64, umma_desc_sw128(smem_u32(sA + j * AT_BYTES) + ks * 32, 16, 1024), bdesc,
                                        IDESC_1_K, ks > 0);
                        }
                        umma_commit(d1_full + j);
                    }
                    if (!ok) break;
                    for (int j = 0; j < nu; ++j) {
                        if (!(ok = mbar_wait(h_ready + j, ph_h[j], abort_flag))) break;
                        ph_h[j] ^= 1;
                        tc_fence_after();
                        const uint32_t ha = smem_u32(sH + j * AT_BYTES);
#pragma unroll
                        for (int ks = 0; ks < MH / 16; ++ks)
                            umma_ss(tmem_base + 128 + j * 32, umma_desc_sw128(ha + ks * 32, 16, 1024), umma_desc_sw128(w2a + ks * 32, 16, 1024),
                                    IDESC_2, ks > 0);
                        if (k + 1 < c) {  // + D_{k+1} through an identity: planes are [head][position], i.e. MN-major A
                            const uint32_t dslab = smem_u32(sSlab + ((stage * 2 + j) * c + k + 1) * SLAB_BYTES);
#pragma unroll
                            for (int ks = 0; ks < HQ / 16; ++ks)
                                umma_ss(tmem_base + 128 + j * 32, umma_desc_sw128(dslab + ks * 2048, HQ * 128, 1024),
                                        umma_desc_sw128(smem_u32(sI) + ks * 32, 16, 1024), IDESC_ID, 1);
                        }
                        umma_commit(d2_full + j);
                        // last reader of this stage's slabs: MMA1 when c == 1, the identity MMA of link c-2 otherwise
                        if (j == nu - 1 && k == (c > 1 ? c - 2 : 0)) umma_commit(slabs_done + stage);
                    }
                }
            }
        }
    } else if (warp == 5) {
        // =========================== result stores (one thread) ===========================
        // Takes each filled staging buffer and writes its two 64-position halves to the [head][position] planes
        // with TMA (full 128-byte lines), so that no worker spends cycles issuing or waiting for stores.
        if (tid == kThreads + 32) {
            bool ok = true;
            int n_store = 0;
            Cursor cu = cursor_at(u_begin);
            for (int u = 0; ok && u < n_mine; ++u, ++n_store) {
                const int buf = n_store & 1;
                if (!(ok = mbar_wait(out_ready + buf, (n_store >> 1) & 1, abort_flag))) break;
                tma_store_4d(&maps.m[0], sOut + buf * SLAB_BYTES, 0, cu.b * HQ, cu.jb * 2, cu.t * UNIT + cu.row - p.row0);
                tma_store_commit();
                tma_store_wait_read<0>();
                mbar_arrive(out_free + buf);
                advance(cu);
            }
            tma_store_wait_all<0>();
        }
    } else {
        // =========================== workers: one thread per position ===========================
        const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
        uint32_t ph_d1[2] = {0, 0}, ph_d2[2] = {0, 0};
        bool ok = true;
        int it = 0, n_store = 0;
        for (int pr = 0; ok && pr < n_pairs; ++pr, ++it) {
            const int nu = min(2, n_mine - 2 * pr);
            for (int k = 0; ok && k < c; ++k) {
                const float* b1 = sBias + k * (MH + HQ);
                const float* b2 = b1 + MH;
                const int act = p.act[k];              // hoisted: kernel parameters indexed by k are slow to re-read
                const bool has_b1 = p.b1[k] != nullptr;
                // ---- hidden layer of both units: bias, activation, fp16, into the K-major H tiles ----
                for (int j = 0; j < nu; ++j) {
                    if (!(ok = mbar_wait(d1_full + j, ph_d1[j], abort_flag))) break;
                    ph_d1[j] ^= 1;
                    tc_fence_after();
                    if (has_b1) hidden_row_dispatch<true>(act, tmem_base + lane_sel + j * 64, b1, sH + j * AT_BYTES, tid);
                    else hidden_row_dispatch<false>(act, tmem_base + lane_sel + j * 64, b1, sH + j * AT_BYTES, tid);
                    fence_async_smem();
                    tc_fence_before();
                    mbar_arrive(h_ready + j);
                }
                if (!ok) break;
                // ---- second-layer results ----
                for (int j = 0; j < nu; ++j) {
                    if (!(ok = mbar_wait(d2_full + j, ph_d2[j], abort_flag))) break;
                    ph_d2[j] ^= 1;
                    tc_fence_after();
                    uint32_t yr[32];
                    tmem_ld32(tmem_base + lane_sel + 128 + j * 32, yr);
                    tmem_wait_ld();
                    if (k + 1 < c) {
                        // A_{k+1} for the next link, K-major: row = position, k-slots 0..31 = heads
                        uint8_t* arow = sA + j * AT_BYTES;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint4 v;
                            v.x = pack_f16(__uint_as_float(yr[q * 8 + 0]) + b2[q * 8 + 0], __uint_as_float(yr[q * 8 + 1]) + b2[q * 8 + 1]);
                            v.y = pack_f16(__uint_as_float(yr[q * 8 + 2]) + b2[q * 8 + 2], __uint_as_float(yr[q * 8 + 3]) + b2[q * 8 + 3]);
                            v.z = pack_f16(__uint_as_float(yr[q * 8 + 4]) + b2[q * 8 + 4], __uint_as_float(yr[q * 8 + 5]) + b2[q * 8 + 5]);
                            v.w = pack_f16(__uint_as_float(yr[q * 8 + 6]) + b2[q * 8 + 6], __uint_as_float(yr[q * 8 + 7]) + b2[q * 8 + 7]);
                            *reinterpret_cast<uint4*>(arow + sw128_offset(tid, q)) = v;
                        }
                        fence_async_smem();
                        tc_fence_before();
                        mbar_arrive(a_ready + j);
                    } else {
                        // Y back to the [head][position] plane: lane pairs swap so that each lane holds two adjacent
                        // positions of 16 heads and writes them as packed fp16 into a slab-shaped staging buffer;
                        // the store warp sends it off.
                        const int buf = n_store & 1;
                        if (n_store >= 2 && !(ok = mbar_wait(out_free + buf, ((n_store >> 1) - 1) & 1, abort_flag))) break;
                        ++n_store;
                        const int odd = tid & 1;
                        const int posl = (tid & 63) & ~1;        // even position of the pair inside its 64-position half
                        uint8_t* half_base = sOut + buf * SLAB_BYTES + (tid >> 6) * (HQ * 128);
#pragma unroll
                        for (int g = 0; g < HQ; g += 2) {
                            const float mine0 = __uint_as_float(yr[g]) + b2[g], mine1 = __uint_as_float(yr[g + 1]) + b2[g + 1];
                            // even lane keeps head g and receives the odd lane's head g; odd lane keeps head g+1
                            const float send = odd ? mine0 : mine1;
                            const float got = __shfl_xor_sync(0xffffffffu, send, 1);
                            const int hh = g + odd;
                            const uint32_t w = odd ? pack_f16(got, mine1) : pack_f16(mine0, got);
                            *reinterpret_cast<uint32_t*>(half_base + hh * 128 + (((posl >> 3) ^ (hh & 7)) << 4) + (posl & 7) * 2) = w;
                        }
                        fence_async_smem();
                        mbar_arrive(out_ready + buf);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (tid == 0) atomicAdd(p.status + 1, 1);
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 4) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

size_t align_smem_bytes(int c, int stages) {
    (void)stages;
    return (size_t)4 * c * SLAB_BYTES + (c > 1 ? 4 : 2) * AT_BYTES + 2 * SLAB_BYTES + W2_BYTES + (size_t)c * (W1_BYTES + W2_BYTES) + (size_t)c * (MH + HQ) * 4 + 256 + 1024;
}

}  // namespace


bool tc_align_supported(int Hq, const lisa_link* links, int chain) {
    if (Hq != HQ || chain < 1 || chain > kMaxTcChain) return false;
    for (int k = 0; k < chain; ++k) {
        const lisa_link& l = links[k];
        if (l.integrate != LISA_INTEGRATE_ADD || l.ffn_layers != 2 || l.m != MH) return false;
    }
    return true;
}

cudaError_t launch_tc_align(const TcAlignArgs& a, cudaStream_t stream) {
    AlignParams p{};
    TensorMaps maps;
    p.B = a.B; p.N = a.N; p.chain = a.chain;
    p.row0 = a.qt_begin * UNIT; p.qt_begin = a.qt_begin; p.qt_count = a.qt_count;
    p.stages = a.chain == 1 ? 3 : 2;
    p.units_per_batch = 0;
    for (int t = a.qt_begin; t < a.qt_begin + a.qt_count; ++t) p.units_per_batch += std::min(UNIT, a.N - t * UNIT) * (t + 1);
    p.plane_rows = a.plane_rows; p.plane_cols = a.plane_cols;
    for (int k = 0; k < a.chain; ++k) {
        p.planes[k] = reinterpret_cast<__half*>(a.planes[k]);
        const lisa_link& l = a.links[k];
        p.w1[k] = l.w1; p.b1[k] = l.b1; p.w2[k] = l.w2; p.b2[k] = l.b2;
        p.w_dtype[k] = l.w_dtype; p.act[k] = l.act;
        // 4-D view of the [B*Hq][rows][cols] planes: (column inside a 64-block, plane, 64-block, row).  A box of
        // 64 x 32 x 2 x 1 lands in shared memory as [half][head][64 positions]: one unit's slab in one copy.
        const uint64_t dims[4] = {64, (uint64_t)a.B * HQ, (uint64_t)a.plane_cols / 64, (uint64_t)a.plane_rows};
        const uint64_t str[3] = {(uint64_t)a.plane_cols * a.plane_rows * 2, 128, (uint64_t)a.plane_cols * 2};
        const uint32_t box[4] = {64, HQ, 2, 1};
        if (!make_tensor_map_bf16(&maps.m[k], a.planes[k], 4, dims, str, box, true)) return cudaErrorInvalidValue;
    }
    for (int k = a.chain; k < kMaxTcChain; ++k) maps.m[k] = maps.m[0];
    p.status = status_words();
    if (!p.status) return cudaErrorUnknown;
    const size_t smem = align_smem_bytes(a.chain, p.stages);
    cudaError_t e = cudaFuncSetAttribute(tc_align_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t total_units = (int64_t)p.units_per_batch * a.B;
    if (total_units <= 0 || total_units > 0x7fffffff) return cudaErrorInvalidValue;
    const int max_ctas = a.ctas > 0 ? a.ctas : 148 * 2;
    dim3 grid((unsigned)std::min<int64_t>((total_units + 7) / 8, max_ctas));  // at least eight units per CTA
    tc_align_kernel<<<grid, kThreads + 64, smem, stream>>>(p, maps);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace lisa
