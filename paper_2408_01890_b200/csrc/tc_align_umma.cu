// Stand-alone head-axis aligner kernel (Sec. 5.1) on tcgen05 tensor cores: applies the FFN chain of a call's links
// to blocked fp16 score planes [row block of 128][column block of 64][row][B*Hq][64 columns], in place.
//
// planes[0] holds A_0 = Q0.K0^T/sqrt(d) (Eq. 2) and receives the output; planes[k], k = 1..c-1, hold the already
// scaled differences D_k = Q'_k.K'_k^T/sqrt(r) (Eq. 3) of the links below the top one.  Output:
// Y = log2(e) * FFN_c(A_{c-1}) with A_k = FFN_k(A_{k-1}) + D_k (Eq. 4, ADD); the top link's own D_c is added by the
// attention kernel that consumes Y.  With store_all, link k's output (times log2 e) is stored over plane k for every
// k: the layers of a whole chain are served by one pass.
// The warp roles are those of tc_align_role.cuh; this file adds the flat tile order and the launch.
#include <algorithm>

#include "tc_align_role.cuh"

namespace lisa {
namespace {

using namespace tc;
using namespace alignrole;

constexpr int kThreads = 192;   // warps 0-3 elementwise, 4 TMA, 5 MMA issue and tensor-memory owner

struct UmmaAlignParams {
    int B, N, chain, store_all;
    int qt_begin, qt_count;
    long long tiles_per_batch, tiles_total;
    Weights w;
    int* status;
};

__host__ __device__ inline int col_blocks(int qt, int N) { return min(2 * qt + 2, (N + 63) / 64); }
__host__ __device__ inline int row_pairs(int qt, int N) { return (min(128, N - qt * 128) + 1) / 2; }

// This CTA's contiguous range of the flat order (batch, query tile, column block, row pair).
struct FlatFeed {
    int N, qt0, qt1;
    int b, qt, cb, rp;
    long long left;
    __device__ void seek(long long begin, long long count, long long tiles_per_batch, int N_, int qt0_, int qt1_) {
        N = N_; qt0 = qt0_; qt1 = qt1_; left = count;
        b = (int)(begin / tiles_per_batch);
        long long rem = begin - (long long)b * tiles_per_batch;
        for (qt = qt0; qt + 1 < qt1; ++qt) {
            const long long n = (long long)col_blocks(qt, N) * row_pairs(qt, N);
            if (rem < n) break;
            rem -= n;
        }
        const int nrp = row_pairs(qt, N);
        cb = (int)(rem / nrp);
        rp = (int)(rem - (long long)cb * nrp);
    }
    __device__ bool next(TileCoord& t) {
        if (left <= 0) return false;
        --left;
        t.c1 = b * HQ; t.c2 = 2 * rp; t.c3 = cb; t.c4 = qt - qt0;
        if (++rp < row_pairs(qt, N)) return true;
        rp = 0;
        if (++cb < col_blocks(qt, N)) return true;
        cb = 0;
        if (++qt < qt1) return true;
        qt = qt0;
        ++b;
        return true;
    }
    __device__ bool after_store() { return true; }
};

// L: Smem<8, 1> for a single link, Smem<6, 3> for chains of two or three (both let two CTAs share an SM)
template <class L>
__global__ void __launch_bounds__(kThreads, 2)
tc_align_umma_kernel(const __grid_constant__ UmmaAlignParams p, const __grid_constant__ CUtensorMap tm0,
                     const __grid_constant__ CUtensorMap tm1, const __grid_constant__ CUtensorMap tm2) {
    extern __shared__ __align__(1024) uint8_t smem[];
    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicAdd(p.status + 1, 1);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint64_t* tail = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR) + L::N_BARS;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail) + 1;

    const long long per_cta = (p.tiles_total + gridDim.x - 1) / gridDim.x;
    const long long begin = min(p.tiles_total, (long long)blockIdx.x * per_cta);
    const int n_tiles = (int)(min(p.tiles_total, begin + per_cta) - begin);
    if (n_tiles <= 0) return;

    if (tid == 0) {
        init_bars<L>(smem);
        *abort_flag = 0;
        fence_barrier_init();
    }
    stage_weights<L>(smem, p.w, p.chain, !p.store_all, tid, kThreads);
    if (warp == 5) tmem_alloc(tmem_slot, L::TMEM_COLS);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 4) {
        FlatFeed feed;
        feed.seek(begin, n_tiles, p.tiles_per_batch, p.N, p.qt_begin, p.qt_begin + p.qt_count);
        tma_warp<L>(smem, feed, feed, n_tiles, p.chain, p.store_all != 0, &tm0, &tm1, &tm2, lane, abort_flag);
    } else if (warp == 5) {
        mma_warp<L>(smem, tmem_base, n_tiles, p.chain, lane, abort_flag);
    } else {
        int acts[kMaxLinks];
        bool biased[kMaxLinks];
        for (int k = 0; k < kMaxLinks; ++k) { acts[k] = p.w.act[k]; biased[k] = p.w.b1[k] != nullptr || p.w.b2[k] != nullptr; }
        elementwise_warps<L>(smem, tmem_base, n_tiles, p.chain, p.store_all != 0, acts, biased, tid, abort_flag);
    }
    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (tid == 0) atomicAdd(p.status + 1, 1);
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 5) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }
}

}  // namespace

bool tc_align_supported(int Hq, const lisa_link* links, int chain) {
    if (Hq != HQ || chain < 1 || chain > kMaxLinks) return false;
    for (int k = 0; k < chain; ++k) {
        const lisa_link& l = links[k];
        if (l.integrate != LISA_INTEGRATE_ADD || l.ffn_layers != 2 || l.m != MH) return false;
    }
    return true;
}

cudaError_t launch_tc_align(const TcAlignArgs& a, cudaStream_t stream) {
    if (a.plane_cols % 64 != 0 || a.plane_rows % 128 != 0) return cudaErrorInvalidValue;   // whole blocks
    UmmaAlignParams p{};
    p.B = a.B; p.N = a.N; p.chain = a.chain; p.store_all = a.store_all ? 1 : 0;
    p.qt_begin = a.qt_begin; p.qt_count = a.qt_count;
    for (int t = a.qt_begin; t < a.qt_begin + a.qt_count; ++t) p.tiles_per_batch += (long long)col_blocks(t, a.N) * row_pairs(t, a.N);
    p.tiles_total = p.tiles_per_batch * a.B;
    if (p.tiles_total <= 0) return cudaErrorInvalidValue;
    for (int k = 0; k < a.chain; ++k) {
        const lisa_link& l = a.links[k];
        p.w.w1[k] = l.w1; p.w.b1[k] = l.b1; p.w.w2[k] = l.w2; p.w.b2[k] = l.b2;
        p.w.w_dtype[k] = l.w_dtype; p.w.act[k] = l.act;
    }
    p.status = status_words();
    if (!p.status) return cudaErrorUnknown;
    // one box = two rows x all heads of one batch element x 64 columns
    CUtensorMap tm[kMaxLinks];
    const uint64_t bh = (uint64_t)a.B * HQ, ncb = (uint64_t)a.plane_cols / 64, nrb = (uint64_t)a.plane_rows / 128;
    const uint64_t dims[5] = {64, bh, 128, ncb, nrb};
    const uint64_t str[4] = {128, bh * 128, 128 * bh * 128, ncb * 128 * bh * 128};
    const uint32_t box[5] = {64, (uint32_t)HQ, 2, 1, 1};
    for (int k = 0; k < kMaxLinks; ++k) {
        const int src = k < a.chain ? k : 0;
        if (!make_tensor_map_bf16(&tm[k], a.planes[src], 5, dims, str, box, true)) return cudaErrorInvalidValue;
    }
    int dev = 0, sms = 0;
    cudaError_t e;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int max_ctas = a.ctas > 0 ? a.ctas : 2 * sms;
    const unsigned grid = (unsigned)std::min<long long>((p.tiles_total + 3) / 4, max_ctas);
    if (a.chain == 1) {
        using L = Smem<8, 1>;
        static_assert(L::TOTAL <= 115712, "two CTAs per SM");
        if ((e = cudaFuncSetAttribute(tc_align_umma_kernel<L>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL)) != cudaSuccess) return e;
        tc_align_umma_kernel<L><<<grid, kThreads, L::TOTAL, stream>>>(p, tm[0], tm[1], tm[2]);
    } else {
        using L = Smem<6, 3>;
        static_assert(L::TOTAL <= 115712, "two CTAs per SM");
        if ((e = cudaFuncSetAttribute(tc_align_umma_kernel<L>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL)) != cudaSuccess) return e;
        tc_align_umma_kernel<L><<<grid, kThreads, L::TOTAL, stream>>>(p, tm[0], tm[1], tm[2]);
    }
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace lisa
