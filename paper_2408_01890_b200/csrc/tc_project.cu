// Projection GEMM on tcgen05 tensor cores: C[B*N, n_out] = X[B*N, K] . W[K, n_out], bf16 in, fp32 accumulation in tensor
// memory, bf16 out, the columns of C scattered straight into up to four [B, N, H, x] tensors (Eq. 1: H W^V_i and the
// product with W^O; Eq. 3: H W^Q_LR, H W^K_LR).
//
// One persistent CTA per SM walks 128 x 256 output tiles.  Warp 0 streams 64-deep K slices of X (K-major rows) and W
// (rows of n_out, i.e. the N dimension contiguous: an MN-major B operand, so W is used as stored, no transposed copy)
// through a four-stage TMA ring; warp 1 issues the MMAs (M 128, N 256, K 16) into one of two 256-column accumulators;
// warps 4-7 drain the other one (thread = output row), round to bf16 and store.  Every wait is bounded.
#include <algorithm>

#include "common.cuh"
#include "tc_common.cuh"

namespace lisa {
namespace {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BK * BN * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int kThreads = 256;
constexpr int kMaxOut = 4;

struct ProjOut {
    void* ptr;
    int64_t sb, sn, sh;
    int32_t x, col0, cols;   // head width; first column of C and number of columns (H * x) that belong to this tensor
    int32_t row_dense;       // sh == x: a row's columns are contiguous from ptr + b*sb + n*sn
};

struct ProjParams {
    int B, N, K, n_out, n_outputs;
    int m_tiles_per_batch, n_tiles;
    long long tiles_total;
    ProjOut out[kMaxOut];
    int* status;
};

constexpr int OFF_BAR = STAGES * STAGE_BYTES;
constexpr int SMEM_TOTAL = OFF_BAR + 256;

__global__ void __launch_bounds__(kThreads, 1)
tc_project_kernel(const __grid_constant__ ProjParams p, const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW) {
    extern __shared__ __align__(1024) uint8_t smem[];
    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicAdd(p.status + 1, 1);
        return;
    }
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint64_t* full = bars;                 // [STAGES]
    uint64_t* empty = bars + STAGES;       // [STAGES]
    uint64_t* acc_full = bars + 2 * STAGES;    // [2]
    uint64_t* acc_empty = bars + 2 * STAGES + 2;   // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES + 5);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(acc_full + i, 1); mbar_init(acc_empty + i, 128); }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int k_slices = (p.K + BK - 1) / BK;
    // tile index -> (batch, row tile, column tile); column tiles vary fastest so that concurrent CTAs share their X rows in L2
    auto tile_coord = [&](long long tile, int& b, int& mt, int& nt) {
        nt = (int)(tile % p.n_tiles);
        const long long r = tile / p.n_tiles;
        mt = (int)(r % p.m_tiles_per_batch);
        b = (int)(r / p.m_tiles_per_batch);
    };

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) { tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmW); }
        long long it = 0;   // running slice count over all tiles of this CTA
        bool ok = true;
        for (long long tile = blockIdx.x; ok && tile < p.tiles_total; tile += gridDim.x) {
            int b, mt, nt;
            tile_coord(tile, b, mt, nt);
            for (int ks = 0; ks < k_slices; ++ks, ++it) {
                const int s = (int)(it % STAGES);
                if (lane == 0) {
                    ok = mbar_wait(empty + s, (uint32_t)((it / STAGES) & 1) ^ 1u, abort_flag);
                    if (ok) mbar_expect_tx(full + s, STAGE_BYTES);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                uint8_t* sa = smem + s * STAGE_BYTES;
                uint8_t* sb = sa + A_BYTES;
                // X slice: [128 rows][64 k]; W slice: four [64 k][64 n] quarters
                if (lane == 0) {
                    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                                 ::"r"(smem_u32(sa)), "l"(&tmX), "r"(smem_u32(full + s)), "r"(ks * BK), "r"(mt * BM), "r"(b) : "memory");
                }
                __syncwarp();
                if (lane < BN / 64) {
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                                 ::"r"(smem_u32(sb + lane * (BK * 128))), "l"(&tmW), "r"(smem_u32(full + s)), "r"(nt * BN + lane * 64), "r"(ks * BK) : "memory");
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer (warp-uniform control flow, lane 0 issues) ------------------------------
        const uint32_t issue = lane == 0;
        constexpr uint32_t IDESC = umma_idesc_bf16(BM, BN, 0, 1);   // X: K contiguous; W: N contiguous
        auto desc_off = [](uint64_t d, uint32_t bytes) -> uint64_t { return (d & 0xffffffff00000000ull) | (uint32_t)((uint32_t)d + (bytes >> 4)); };
        const uint64_t da0 = umma_desc_sw128(smem_u32(smem), 16, 1024);
        const uint64_t db0 = umma_desc_sw128(smem_u32(smem + A_BYTES), BK * 128, 1024);
        long long it = 0;
        int n_acc = 0;
        bool ok = true;
        for (long long tile = blockIdx.x; ok && tile < p.tiles_total; tile += gridDim.x, ++n_acc) {
            const int a = n_acc & 1;
            ok = mbar_wait(acc_empty + a, (uint32_t)((n_acc >> 1) & 1) ^ 1u, abort_flag);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;
            tc_fence_after();
            const uint32_t dst = tmem_base + a * BN;
            for (int ks = 0; ks < k_slices; ++ks, ++it) {
                const int s = (int)(it % STAGES);
                ok = mbar_wait(full + s, (uint32_t)((it / STAGES) & 1), abort_flag);
                if (!(ok = __all_sync(0xffffffffu, ok))) break;
                tc_fence_after();
                const uint64_t da = desc_off(da0, s * STAGE_BYTES), db = desc_off(db0, s * STAGE_BYTES);
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk)
                    umma_ss_if(issue, dst, desc_off(da, kk * 32), desc_off(db, kk * 2048), IDESC, (ks > 0) || (kk > 0));
                umma_commit_if(issue, empty + s);
            }
            if (!ok) break;
            umma_commit_if(issue, acc_full + a);
        }
    } else if (warp >= 4) {
        // ------------------------------ epilogue (thread = output row) ------------------------------
        const int row = tid - 128;
        const uint32_t lane_sel = (uint32_t)((warp - 4) * 32) << 16;
        int n_acc = 0;
        bool ok = true;
        for (long long tile = blockIdx.x; ok && tile < p.tiles_total; tile += gridDim.x, ++n_acc) {
            int b, mt, nt;
            tile_coord(tile, b, mt, nt);
            const int a = n_acc & 1;
            if (!(ok = mbar_wait(acc_full + a, (uint32_t)((n_acc >> 1) & 1), abort_flag))) break;
            tc_fence_after();
            const int n = mt * BM + row;
            const bool row_ok = n < p.N;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_base + a * BN + lane_sel + c * 32, r);
                tmem_wait_ld();
                if (c == BN / 32 - 1) {   // the accumulator is in registers: hand it back before the stores
                    tc_fence_before();
                    mbar_arrive(acc_empty + a);
                }
                const int col_base = nt * BN + c * 32;
                if (!row_ok || col_base >= p.n_out) continue;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int col = col_base + g * 8;
                    if (col >= p.n_out) break;
                    uint4 v;
                    v.x = pack_bf16(__uint_as_float(r[g * 8 + 0]), __uint_as_float(r[g * 8 + 1]));
                    v.y = pack_bf16(__uint_as_float(r[g * 8 + 2]), __uint_as_float(r[g * 8 + 3]));
                    v.z = pack_bf16(__uint_as_float(r[g * 8 + 4]), __uint_as_float(r[g * 8 + 5]));
                    v.w = pack_bf16(__uint_as_float(r[g * 8 + 6]), __uint_as_float(r[g * 8 + 7]));
                    // which output tensor holds column `col`
                    int o = 0;
                    while (o + 1 < p.n_outputs && col >= p.out[o].col0 + p.out[o].cols) ++o;
                    const ProjOut& t = p.out[o];
                    const int rel = col - t.col0;
                    __nv_bfloat16* base = reinterpret_cast<__nv_bfloat16*>(t.ptr) + b * t.sb + (int64_t)n * t.sn;
                    if (t.row_dense && rel + 8 <= t.cols && ((reinterpret_cast<uintptr_t>(base + rel) & 15u) == 0)) {
                        *reinterpret_cast<uint4*>(base + rel) = v;
                    } else {
                        const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
                        int oo = o;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int cj = col + j;
                            if (cj >= p.n_out) break;
                            while (oo + 1 < p.n_outputs && cj >= p.out[oo].col0 + p.out[oo].cols) ++oo;
                            const ProjOut& tt = p.out[oo];
                            const int rj = cj - tt.col0;
                            reinterpret_cast<__nv_bfloat16*>(tt.ptr)[b * tt.sb + (int64_t)n * tt.sn + (int64_t)(rj / tt.x) * tt.sh + rj % tt.x] = e[j];
                        }
                    }
                }
            }
        }
    }
    // ------------------------------ teardown ------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (tid == 0) atomicAdd(p.status + 1, 1);
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// General path: one thread per output element, fp32 accumulation in the order of k; any dtype and stride.
struct GenOut { void* ptr; int64_t sb, sn, sh; int32_t dtype, x, col0, cols; };
struct GenParams {
    int B, N, K, n_out, n_outputs;
    TView x;
    const void* w;
    int w_dtype;
    GenOut out[kMaxOut];
};
__global__ void generic_project_kernel(const __grid_constant__ GenParams p) {
    const int64_t total = (int64_t)p.B * p.N * p.n_out;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int col = (int)(e % p.n_out);
        const int64_t r = e / p.n_out;
        const int n = (int)(r % p.N), b = (int)(r / p.N);
        float acc = 0.f;
        for (int k = 0; k < p.K; ++k)
            acc = fmaf(ld_elem(p.x.ptr, b * p.x.sb + (int64_t)n * p.x.sn + k, p.x.dtype), ld_elem(p.w, (int64_t)k * p.n_out + col, p.w_dtype), acc);
        int o = 0;
        while (o + 1 < p.n_outputs && col >= p.out[o].col0 + p.out[o].cols) ++o;
        const GenOut& t = p.out[o];
        const int rel = col - t.col0;
        st_elem(t.ptr, b * t.sb + (int64_t)n * t.sn + (int64_t)(rel / t.x) * t.sh + rel % t.x, t.dtype, acc);
    }
}

}  // namespace

cudaError_t launch_generic_project(const lisa_project_args& a, cudaStream_t stream) {
    GenParams p{};
    p.B = a.B; p.N = a.N; p.K = a.d_in; p.n_outputs = a.n_outputs;
    p.x = make_view(a.x); p.w = a.w; p.w_dtype = a.w_dtype;
    int col = 0;
    for (int o = 0; o < a.n_outputs; ++o) {
        const lisa_project_output& src = a.outputs[o];
        p.out[o] = GenOut{src.t.ptr, src.t.stride_b, src.t.stride_n, src.t.stride_h, src.t.dtype, src.x, col, src.H * src.x};
        col += src.H * src.x;
    }
    p.n_out = col;
    const int64_t total = (int64_t)a.B * a.N * col;
    const int blocks = (int)std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, (int64_t)sm_count() * 32));
    generic_project_kernel<<<blocks, 256, 0, stream>>>(p);
    count_launches(1);
    return cudaGetLastError();
}

bool tc_project_supported(const lisa_project_args& a) {
    if (a.x.dtype != LISA_BF16 || a.w_dtype != LISA_BF16) return false;
    if ((reinterpret_cast<uintptr_t>(a.x.ptr) & 15u) || (reinterpret_cast<uintptr_t>(a.w) & 15u)) return false;
    if (a.d_in % 8 != 0 || a.x.stride_n % 8 != 0 || a.x.stride_b % 8 != 0 || a.x.stride_n < a.d_in) return false;
    int n_out = 0;
    for (int o = 0; o < a.n_outputs; ++o) {
        if (a.outputs[o].t.dtype != LISA_BF16) return false;
        n_out += a.outputs[o].H * a.outputs[o].x;
    }
    return n_out % 8 == 0;   // rows of W must be whole 16-byte units for the tensor map
}

cudaError_t launch_tc_project(const lisa_project_args& a, cudaStream_t stream) {
    ProjParams p{};
    p.B = a.B; p.N = a.N; p.K = a.d_in; p.n_outputs = a.n_outputs;
    int col = 0;
    for (int o = 0; o < a.n_outputs; ++o) {
        const lisa_project_output& src = a.outputs[o];
        ProjOut& t = p.out[o];
        t.ptr = src.t.ptr; t.sb = src.t.stride_b; t.sn = src.t.stride_n; t.sh = src.t.stride_h;
        t.x = src.x; t.col0 = col; t.cols = src.H * src.x;
        t.row_dense = (src.t.stride_h == src.x || src.H == 1) ? 1 : 0;
        col += t.cols;
    }
    p.n_out = col;
    p.m_tiles_per_batch = (a.N + BM - 1) / BM;
    p.n_tiles = (p.n_out + BN - 1) / BN;
    p.tiles_total = (long long)a.B * p.m_tiles_per_batch * p.n_tiles;
    p.status = status_words();
    if (!p.status) return cudaErrorUnknown;
    CUtensorMap tmX, tmW;
    {
        const uint64_t dims[3] = {(uint64_t)a.d_in, (uint64_t)a.N, (uint64_t)a.B};
        const uint64_t str[2] = {(uint64_t)a.x.stride_n * 2, (uint64_t)a.x.stride_b * 2};
        const uint32_t box[3] = {(uint32_t)BK, (uint32_t)BM, 1};
        if (!make_tensor_map_bf16(&tmX, a.x.ptr, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        const uint64_t dims[2] = {(uint64_t)p.n_out, (uint64_t)a.d_in};
        const uint64_t str[1] = {(uint64_t)p.n_out * 2};
        const uint32_t box[2] = {64, (uint32_t)BK};
        if (!make_tensor_map_bf16(&tmW, a.w, 2, dims, str, box)) return cudaErrorInvalidValue;
    }
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(tc_project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_TOTAL)) != cudaSuccess) return e;
    const unsigned grid = (unsigned)std::min<long long>(p.tiles_total, sm_count());
    tc_project_kernel<<<grid, kThreads, SMEM_TOTAL, stream>>>(p, tmX, tmW);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace lisa
