// Head-axis aligner on tensor cores (Sec. 5.1): the FFN chain of a shared layer applied to score planes.
//
// Input: fp16 planes [B*Hq][rows][cols] (fp16, not bf16: three more mantissa bits keep a chain of several links
// inside the accuracy bar; scores are O(10), far from fp16's range limit, and conversions saturate) holding A_0 = Q0.K0^T/sqrt(d) (Eq. 2) and, for chain depth c > 1, the
// already scaled differences D_k = Q'_k.K'_k^T/sqrt(r) (Eq. 3) of the links k < c.  Output, in place of the A_0
// plane: Y = FFN_c(A_{c-1}) where A_k = FFN_k(A_{k-1}) + D_k (Eq. 4, ADD) -- the final link's D_c is added by the
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
constexpr uint32_t TMEM_COLS = 128;        // D1: [0,64), D2: [64,96)
constexpr int kMaxTcChain = 4;

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

__device__ __forceinline__ float act_fast(float x, int act) {
    if (act == LISA_ACT_RELU) return fmaxf(x, 0.f);
    if (act == LISA_ACT_SILU) return __fdividef(x, 1.f + __expf(-x));
    return x;
}

struct TensorMaps {
    CUtensorMap m[kMaxTcChain];
};

__global__ void __launch_bounds__(kThreads, 3)
tc_align_kernel(const __grid_constant__ AlignParams p, const __grid_constant__ TensorMaps maps) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int c = p.chain;
    const int S = p.stages;
    // layout: [S stages of c slabs] [H tile] [A tile] [identity] [W1,W2 per link] [biases] [barriers]
    uint8_t* sSlab = smem;
    uint8_t* sH = sSlab + S * c * SLAB_BYTES;
    uint8_t* sA = sH + AT_BYTES;
    uint8_t* sI = sA + AT_BYTES;
    uint8_t* sW = sI + W2_BYTES;
    float* sBias = reinterpret_cast<float*>(sW + c * (W1_BYTES + W2_BYTES));  // per link: b1[64], b2[32]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sBias + c * (MH + HQ));
    uint64_t* full = bars;      // [4]
    uint64_t* mma_bar = bars + 4;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 6);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int n_units = p.units_per_batch * p.B;
    // unit index -> (batch, query row, first key column): units are numbered tile by tile, row by row
    auto decode = [&](int u, int& b, int& row_g, int& col0) {
        b = u / p.units_per_batch;
        int rem = u - b * p.units_per_batch;
        int t = p.qt_begin;
        for (;; ++t) {
            const int n_t = min(UNIT, p.N - t * UNIT) * (t + 1);
            if (rem < n_t || t + 1 >= p.qt_begin + p.qt_count) break;
            rem -= n_t;
        }
        row_g = t * UNIT + rem / (t + 1);
        col0 = (rem % (t + 1)) * UNIT;
    };

    // ---- one-time set-up: barriers, TMEM, weights as swizzled MMA operands ----
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(full + i, 1);
        mbar_init(mma_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
        for (int k = 0; k < c; ++k) tma_prefetch_desc(&maps.m[k]);
    }
    if (warp == 0) tmem_alloc(tmem_slot, TMEM_COLS);
    for (int e = tid; e < (W2_BYTES + c * (W1_BYTES + W2_BYTES)) / 16; e += kThreads) reinterpret_cast<uint4*>(sI)[e] = make_uint4(0, 0, 0, 0);
    for (int e = tid; e < AT_BYTES / 16; e += kThreads) reinterpret_cast<uint4*>(sA)[e] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int e = tid; e < HQ; e += kThreads)  // identity: row g, k-slot g
        *reinterpret_cast<__half*>(sI + sw128_offset(e, e >> 3) + (e & 7) * 2) = __float2half_rn(1.f);
    for (int k = 0; k < c; ++k) {
        uint8_t* w1t = sW + k * (W1_BYTES + W2_BYTES);
        uint8_t* w2t = w1t + W1_BYTES;
        for (int e = tid; e < HQ * MH; e += kThreads) {
            const int hh = e / MH, u = e % MH;  // W1[hh][u] -> row u, k-slot hh
            *reinterpret_cast<__half*>(w1t + sw128_offset(u, hh >> 3) + (hh & 7) * 2) = __float2half_rn(ld_elem(p.w1[k], e, p.w_dtype[k]));
            const int u2 = e / HQ, gg = e % HQ;  // W2[u2][gg] -> row gg, k-slot u2
            *reinterpret_cast<__half*>(w2t + sw128_offset(gg, u2 >> 3) + (u2 & 7) * 2) = __float2half_rn(ld_elem(p.w2[k], e, p.w_dtype[k]));
        }
        for (int e = tid; e < MH; e += kThreads) sBias[k * (MH + HQ) + e] = ldw(p.b1[k], e, p.w_dtype[k]);
        for (int e = tid; e < HQ; e += kThreads) sBias[k * (MH + HQ) + MH + e] = ldw(p.b2[k], e, p.w_dtype[k]);
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_D1 = tmem_base, tmem_D2 = tmem_base + 64;
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;

    constexpr uint32_t IDESC_1_MN = umma_idesc_f16(UNIT, MH, 1, 0);
    constexpr uint32_t IDESC_1_K = umma_idesc_f16(UNIT, MH, 0, 0);
    constexpr uint32_t IDESC_2 = umma_idesc_f16(UNIT, HQ, 0, 0);
    constexpr uint32_t IDESC_ID = umma_idesc_f16(UNIT, HQ, 1, 0);

    auto issue_loads = [&](int u, int stage) {  // thread 0 only
        int b, row_g, col0;
        decode(u, b, row_g, col0);
        mbar_expect_tx(full + stage, c * SLAB_BYTES);
        for (int k = 0; k < c; ++k)
            for (int half = 0; half < 2; ++half)
                tma_load_3d(sSlab + (stage * c + k) * SLAB_BYTES + half * (HQ * 128), &maps.m[k], full + stage, col0 + half * 64,
                            row_g - p.row0, b * HQ);
    };

    uint32_t mma_phase = 0;
    bool ok = true;
    int it = 0;
    if (tid == 0)
        for (int i = 0; i < S - 1; ++i)
            if ((int)blockIdx.x + i * (int)gridDim.x < n_units) issue_loads(blockIdx.x + i * gridDim.x, i);
    for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x, ++it) {
        const int stage = it % S;
        const int un = u + (S - 1) * gridDim.x;
        // the stage refilled here held unit it-1, whose slabs and results every thread is done with (loop-end barrier)
        if (tid == 0 && un < n_units) issue_loads(un, (it + S - 1) % S);
        if (!(ok = mbar_wait(full + stage, (it / S) & 1, abort_flag))) break;
        int b, row_g, col0;
        decode(u, b, row_g, col0);
        const uint8_t* slabs = sSlab + stage * c * SLAB_BYTES;
        for (int k = 0; k < c; ++k) {
            const uint8_t* w1t = sW + k * (W1_BYTES + W2_BYTES);
            const uint8_t* w2t = w1t + W1_BYTES;
            const float* b1 = sBias + k * (MH + HQ);
            const float* b2 = b1 + MH;
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < HQ / 16; ++ks) {
                    const uint64_t bdesc = umma_desc_sw128(smem_u32(w1t) + ks * 32, 16, 1024);
                    if (k == 0)  // A_0 slabs: MN-major, 64 positions per 128-byte row, one row per head
                        umma_ss(tmem_D1, umma_desc_sw128(smem_u32(slabs) + ks * 2048, HQ * 128, 1024), bdesc, IDESC_1_MN, ks > 0);
                    else         // A_{k}: written by the threads, K-major
                        umma_ss(tmem_D1, umma_desc_sw128(smem_u32(sA) + ks * 32, 16, 1024), bdesc, IDESC_1_K, ks > 0);
                }
                umma_commit(mma_bar);
            }
            if (!(ok = mbar_wait(mma_bar, mma_phase, abort_flag))) break;
            mma_phase ^= 1;
            tc_fence_after();
            // hidden layer: bias, activation, fp16, into the K-major H tile (row = this thread's position)
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
                uint32_t hr[32];
                tmem_ld32(tmem_D1 + lane_sel + cc * 32, hr);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float e[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) e[j] = act_fast(__uint_as_float(hr[q * 8 + j]) + b1[cc * 32 + q * 8 + j], p.act[k]);
                    uint4 v;
                    v.x = pack_f16(e[0], e[1]); v.y = pack_f16(e[2], e[3]); v.z = pack_f16(e[4], e[5]); v.w = pack_f16(e[6], e[7]);
                    *reinterpret_cast<uint4*>(sH + sw128_offset(tid, cc * 4 + q)) = v;
                }
            }
            fence_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < MH / 16; ++ks)
                    umma_ss(tmem_D2, umma_desc_sw128(smem_u32(sH) + ks * 32, 16, 1024), umma_desc_sw128(smem_u32(w2t) + ks * 32, 16, 1024),
                            IDESC_2, ks > 0);
                if (k + 1 < c) {  // + D_{k+1} through an identity: planes are [head][position], i.e. MN-major A
                    const uint8_t* dslab = slabs + (k + 1) * SLAB_BYTES;
#pragma unroll
                    for (int ks = 0; ks < HQ / 16; ++ks)
                        umma_ss(tmem_D2, umma_desc_sw128(smem_u32(dslab) + ks * 2048, HQ * 128, 1024),
                                umma_desc_sw128(smem_u32(sI) + ks * 32, 16, 1024), IDESC_ID, 1);
                }
                umma_commit(mma_bar);
            }
            if (!(ok = mbar_wait(mma_bar, mma_phase, abort_flag))) break;
            mma_phase ^= 1;
            tc_fence_after();
            uint32_t yr[32];
            tmem_ld32(tmem_D2 + lane_sel, yr);
            tmem_wait_ld();
            if (k + 1 < c) {
                // A_{k+1} for the next link, K-major: row = position, k-slots 0..31 = heads
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 v;
                    v.x = pack_f16(__uint_as_float(yr[q * 8 + 0]) + b2[q * 8 + 0], __uint_as_float(yr[q * 8 + 1]) + b2[q * 8 + 1]);
                    v.y = pack_f16(__uint_as_float(yr[q * 8 + 2]) + b2[q * 8 + 2], __uint_as_float(yr[q * 8 + 3]) + b2[q * 8 + 3]);
                    v.z = pack_f16(__uint_as_float(yr[q * 8 + 4]) + b2[q * 8 + 4], __uint_as_float(yr[q * 8 + 5]) + b2[q * 8 + 5]);
                    v.w = pack_f16(__uint_as_float(yr[q * 8 + 6]) + b2[q * 8 + 6], __uint_as_float(yr[q * 8 + 7]) + b2[q * 8 + 7]);
                    *reinterpret_cast<uint4*>(sA + sw128_offset(tid, q)) = v;
                }
                fence_async_smem();
                tc_fence_before();
                __syncthreads();
            } else {
                __half* dst = p.planes[0] + ((int64_t)(b * HQ) * p.plane_rows + (row_g - p.row0)) * p.plane_cols + col0 + tid;
                const int64_t hstride = p.plane_rows * p.plane_cols;
#pragma unroll
                for (int g = 0; g < HQ; ++g) dst[g * hstride] = __float2half_rn(__uint_as_float(yr[g]) + b2[g]);
            }
        }
        // all reads of this stage's slabs (by the MMAs, now complete) and of D1/D2 are done before the
        // next iteration lets thread 0 refill the other stage / reissue MMAs
        tc_fence_before();
        __syncthreads();
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (tid == 0) atomicAdd(p.status + 1, 1);
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 0) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

size_t align_smem_bytes(int c, int stages) {
    return (size_t)stages * c * SLAB_BYTES + 2 * AT_BYTES + W2_BYTES + (size_t)c * (W1_BYTES + W2_BYTES) + (size_t)c * (MH + HQ) * 4 + 64 + 1024;
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
        const uint64_t dims[3] = {(uint64_t)a.plane_cols, (uint64_t)a.plane_rows, (uint64_t)a.B * HQ};
        const uint64_t str[2] = {(uint64_t)a.plane_cols * 2, (uint64_t)a.plane_cols * a.plane_rows * 2};
        const uint32_t box[3] = {64, 1, HQ};
        if (!make_tensor_map_bf16(&maps.m[k], a.planes[k], 3, dims, str, box, true)) return cudaErrorInvalidValue;
    }
    for (int k = a.chain; k < kMaxTcChain; ++k) maps.m[k] = maps.m[0];
    p.status = status_words();
    if (!p.status) return cudaErrorUnknown;
    const size_t smem = align_smem_bytes(a.chain, p.stages);
    cudaError_t e = cudaFuncSetAttribute(tc_align_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t total_units = (int64_t)p.units_per_batch * a.B;
    if (total_units <= 0 || total_units > 0x7fffffff) return cudaErrorInvalidValue;
    const int max_ctas = a.ctas > 0 ? a.ctas : 148 * 3;
    dim3 grid((unsigned)std::min<int64_t>(total_units, max_ctas));
    tc_align_kernel<<<grid, kThreads, smem, stream>>>(p, maps);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace lisa
