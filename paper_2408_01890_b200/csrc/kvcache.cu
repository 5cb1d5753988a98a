// Cache append (Sec. 2.2 "KV cache"; Sec. 5.2: a shared layer stores K_LR in place of K).
// STANDARD layers keep K as [B][Hkv][L_cap][d]; SHARED layers keep K' transposed, [B][Hkv][r][L_cap],
// so that the decode kernel reads full 16-byte vectors along the position axis whatever r is.
#include <algorithm>

#include "common.cuh"

namespace lisa {
namespace {

struct AppendParams {
    int B, Hkv, L_cap, d, r, n_new, kind, dtype;
    TView k, v;
    void* kc;
    void* vc;
    const int32_t* lens_before;
    int* status;
};

// rows of d elements (V, or K of a STANDARD layer): one thread per 16 bytes
template <typename Vec, int kElems>
__device__ __forceinline__ void append_rows(const AppendParams& p, const TView& src, void* dst_base, bool count_drops) {
    const int vec_per_row = p.d / kElems;
    const int64_t total = (int64_t)p.B * p.n_new * p.Hkv * vec_per_row;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int vi = (int)(e % vec_per_row);
        int64_t rest = e / vec_per_row;
        const int g = (int)(rest % p.Hkv); rest /= p.Hkv;
        const int t = (int)(rest % p.n_new);
        const int b = (int)(rest / p.n_new);
        const int pos = (p.lens_before ? p.lens_before[b] : 0) + t;
        if (pos >= p.L_cap || pos < 0) {
            if (count_drops && vi == 0 && g == 0) atomicAdd(p.status, 1);
            continue;
        }
        const char* sp = reinterpret_cast<const char*>(src.ptr) +
                         (b * src.sb + t * src.sn + g * src.sh) * (int64_t)(sizeof(Vec) / kElems) + (int64_t)vi * sizeof(Vec);
        Vec val = *reinterpret_cast<const Vec*>(sp);
        Vec* dp = reinterpret_cast<Vec*>(dst_base) + (((int64_t)b * p.Hkv + g) * p.L_cap + pos) * vec_per_row + vi;
        *dp = val;
    }
}

// K' of a SHARED layer: thread per (b, g, t); consecutive threads write consecutive positions
template <typename T>
__device__ __forceinline__ void append_kp_transposed(const AppendParams& p) {
    const int64_t total = (int64_t)p.B * p.Hkv * p.n_new;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int t = (int)(e % p.n_new);
        int64_t rest = e / p.n_new;
        const int g = (int)(rest % p.Hkv);
        const int b = (int)(rest / p.Hkv);
        const int pos = (p.lens_before ? p.lens_before[b] : 0) + t;
        if (pos >= p.L_cap || pos < 0) continue;  // counted by the V kernel
        const T* sp = reinterpret_cast<const T*>(p.k.ptr) + b * p.k.sb + t * p.k.sn + g * p.k.sh;
        T* dp = reinterpret_cast<T*>(p.kc) + ((int64_t)b * p.Hkv + g) * p.r * p.L_cap + pos;
        for (int x = 0; x < p.r; ++x) dp[(int64_t)x * p.L_cap] = sp[x];
    }
}

// One launch appends both halves of a layer's cache: blockIdx.y = 0 the V rows, 1 the K rows (STANDARD) or the
// transposed K_LR columns (SHARED).
template <typename Vec, int kElems, typename T>
__global__ void append_kernel(const __grid_constant__ AppendParams p) {
    chain_release();
    chain_wait();
    if (blockIdx.y == 0) append_rows<Vec, kElems>(p, p.v, p.vc, true);
    else if (p.kind == LISA_CACHE_STANDARD) append_rows<Vec, kElems>(p, p.k, p.kc, false);
    else append_kp_transposed<T>(p);
}

}  // namespace

cudaError_t launch_kvcache_append(const lisa_kvcache_layer& c, const lisa_tensor& k, const lisa_tensor& v,
                                  const int32_t* lens_before, int n_new, cudaStream_t s) {
    AppendParams p{c.B, c.Hkv, c.L_cap, c.d, c.r, n_new, c.kind, c.dtype, make_view(k), make_view(v), c.k, c.v,
                   lens_before, status_words()};
    if (!p.status) return cudaErrorUnknown;
    const int threads = 256;
    const int64_t rows = (int64_t)c.B * n_new * c.Hkv;
    auto blocks_for = [&](int64_t n) { return (int)std::max<int64_t>(1, std::min<int64_t>((n + threads - 1) / threads, sm_count() * 16)); };
    cudaError_t e;
    if (c.dtype == LISA_BF16) e = launch_chained(append_kernel<uint4, 8, __nv_bfloat16>, dim3(blocks_for(rows * (c.d / 8)), 2), dim3(threads), 0, s, p);
    else e = launch_chained(append_kernel<float4, 4, float>, dim3(blocks_for(rows * (c.d / 4)), 2), dim3(threads), 0, s, p);
    count_launches(1);
    return e;
}

}  // namespace lisa
