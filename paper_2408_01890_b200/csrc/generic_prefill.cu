// General SIMT prefill of a LiSA shared layer (and, with chain_len == 0, of a standard layer).
//
// One CTA per query row (b, i).  Keys are visited in chunks of 128; thread t of a chunk owns key
// j and rebuilds the whole score chain for that position in fp32: the anchor score q0.k0/sqrt(d) for
// every head (Eq. 2), then per link the low-rank difference q'.k'/sqrt(r) (Eq. 3), the head-axis FFN
// and the integration (Sec. 5.1, Eq. 4).  The chunk's final scores go to shared memory, get the causal
// mask (keys j > i are never visited), an online softmax per head, and the product with V (Eq. 1).
// The N x N x Hq scores are never stored.  Every integrate mode, activation, FFN depth, dtype and
// shape in the supported range runs here; the tensor-core kernels cover the fast cases.
#include "common.cuh"

namespace lisa {
namespace {

constexpr int kChunk = 128;
constexpr int kThreads = 128;

struct PrefillParams {
    int B, N, Hq, Hkv, d, c;
    TView q0, k0, v, o;
    LinkDev links[kMaxChain];
};

__device__ __forceinline__ float ldw(const void* p, int idx, int dtype) { return p ? ld_elem(p, idx, dtype) : 0.f; }

// Sec. 5.1 at one position: a <- Integrate(Align(a), dl).  hid is scratch of kMaxHidden floats.
__device__ void align_integrate(float* a, const float* dl, int Hq, const LinkDev& lk, float* hid) {
    if (lk.integrate == LISA_INTEGRATE_PLUS) {
        for (int g = 0; g < Hq; ++g) a[g] += dl[g];
        return;
    }
    const int m = lk.m;
    for (int u = 0; u < m; ++u) {
        float s = ldw(lk.b1, u, lk.w_dtype);
        for (int x = 0; x < Hq; ++x) s = fmaf(a[x], ld_elem(lk.w1, (int64_t)x * m + u, lk.w_dtype), s);
        if (lk.integrate == LISA_INTEGRATE_CONCAT)
            for (int x = 0; x < Hq; ++x) s = fmaf(dl[x], ld_elem(lk.w1, (int64_t)(Hq + x) * m + u, lk.w_dtype), s);
        hid[u] = s;
    }
    if (lk.ffn_layers == 1) {
        for (int g = 0; g < Hq; ++g) a[g] = hid[g];
    } else {
        for (int u = 0; u < m; ++u) hid[u] = act_apply(hid[u], lk.act);
        for (int g = 0; g < Hq; ++g) {
            float s = ldw(lk.b2, g, lk.w_dtype);
            for (int u = 0; u < m; ++u) s = fmaf(hid[u], ld_elem(lk.w2, (int64_t)u * Hq + g, lk.w_dtype), s);
            a[g] = s;
        }
    }
    if (lk.integrate == LISA_INTEGRATE_ADD)
        for (int g = 0; g < Hq; ++g) a[g] += dl[g];
}

__global__ void __launch_bounds__(kThreads) generic_prefill_kernel(const __grid_constant__ PrefillParams p) {
    extern __shared__ float smem[];
    const int b = blockIdx.y, i = blockIdx.x, tid = threadIdx.x;
    const int Hq = p.Hq, d = p.d, G = p.Hq / p.Hkv;
    float* q0_s = smem;                       // [Hq*d]
    float* o_s = q0_s + Hq * d;               // [Hq*d]
    float* s_s = o_s + Hq * d;                // [Hq*kChunk]
    float* m_s = s_s + Hq * kChunk;           // [Hq]
    float* l_s = m_s + Hq;                    // [Hq]
    float* sc_s = l_s + Hq;                   // [Hq]
    float* qp_s = sc_s + Hq;                  // [c][Hq*kMaxRank]

    for (int e = tid; e < Hq * d; e += kThreads) {
        const int h = e / d, x = e % d;
        q0_s[e] = ld_elem(p.q0.ptr, b * p.q0.sb + i * p.q0.sn + h * p.q0.sh + x, p.q0.dtype);
        o_s[e] = 0.f;
    }
    for (int k = 0; k < p.c; ++k) {
        const LinkDev& lk = p.links[k];
        for (int e = tid; e < Hq * lk.r; e += kThreads) {
            const int h = e / lk.r, x = e % lk.r;
            qp_s[k * Hq * kMaxRank + h * kMaxRank + x] =
                ld_elem(lk.qp.ptr, b * lk.qp.sb + i * lk.qp.sn + h * lk.qp.sh + x, lk.qp.dtype);
        }
    }
    for (int h = tid; h < Hq; h += kThreads) {
        m_s[h] = -INFINITY;
        l_s[h] = 0.f;
    }
    __syncthreads();

    float a[kMaxHeads], dl[kMaxHeads], hid[kMaxHidden];
    const float inv_sqrt_d = rsqrtf((float)d);
    const int warp = tid >> 5, lane = tid & 31;

    for (int j0 = 0; j0 <= i; j0 += kChunk) {
        const int j = j0 + tid;
        if (j <= i) {
            for (int h = 0; h < Hq; ++h) {
                const int64_t kb = b * p.k0.sb + (int64_t)j * p.k0.sn + (h / G) * p.k0.sh;
                float s = 0.f;
                for (int x = 0; x < d; ++x) s = fmaf(q0_s[h * d + x], ld_elem(p.k0.ptr, kb + x, p.k0.dtype), s);
                a[h] = s * inv_sqrt_d;
            }
            for (int k = 0; k < p.c; ++k) {
                const LinkDev& lk = p.links[k];
                const float inv_sqrt_r = rsqrtf((float)lk.r);
                for (int h = 0; h < Hq; ++h) {
                    const int64_t kb = b * lk.kp.sb + (int64_t)j * lk.kp.sn + (h / G) * lk.kp.sh;
                    const float* qrow = qp_s + k * Hq * kMaxRank + h * kMaxRank;
                    float s = 0.f;
                    for (int x = 0; x < lk.r; ++x) s = fmaf(qrow[x], ld_elem(lk.kp.ptr, kb + x, lk.kp.dtype), s);
                    dl[h] = s * inv_sqrt_r;
                }
                align_integrate(a, dl, Hq, lk, hid);
            }
            for (int h = 0; h < Hq; ++h) s_s[h * kChunk + tid] = a[h];
        } else {
            for (int h = 0; h < Hq; ++h) s_s[h * kChunk + tid] = -INFINITY;  // causal mask, after the chain
        }
        __syncthreads();
        for (int h = warp; h < Hq; h += kThreads / 32) {
            float v[kChunk / 32];
            float cmax = -INFINITY;
#pragma unroll
            for (int t = 0; t < kChunk / 32; ++t) {
                v[t] = s_s[h * kChunk + lane + 32 * t];
                cmax = fmaxf(cmax, v[t]);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, off));
            const float m_old = m_s[h];
            const float m_new = fmaxf(m_old, cmax);
            float sum = 0.f;
#pragma unroll
            for (int t = 0; t < kChunk / 32; ++t) {
                const float e = __expf(v[t] - m_new);
                s_s[h * kChunk + lane + 32 * t] = e;
                sum += e;
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            if (lane == 0) {
                const float sc = __expf(m_old - m_new);
                sc_s[h] = sc;
                l_s[h] = l_s[h] * sc + sum;
                m_s[h] = m_new;
            }
        }
        __syncthreads();
        if (tid < d) {
            const int nk = min(kChunk, i + 1 - j0);
            for (int h = 0; h < Hq; ++h) {
                float acc = o_s[h * d + tid] * sc_s[h];
                const int64_t vb = b * p.v.sb + (int64_t)j0 * p.v.sn + (h / G) * p.v.sh + tid;
                for (int jj = 0; jj < nk; ++jj)
                    acc = fmaf(s_s[h * kChunk + jj], ld_elem(p.v.ptr, vb + (int64_t)jj * p.v.sn, p.v.dtype), acc);
                o_s[h * d + tid] = acc;
            }
        }
        __syncthreads();
    }
    if (tid < d)
        for (int h = 0; h < Hq; ++h)
            st_elem(const_cast<void*>(p.o.ptr), b * p.o.sb + i * p.o.sn + h * p.o.sh + tid, p.o.dtype,
                    o_s[h * d + tid] / l_s[h]);
}

size_t smem_bytes(int Hq, int d, int c) {
    return sizeof(float) * ((size_t)2 * Hq * d + (size_t)Hq * kChunk + 3 * (size_t)Hq + (size_t)c * Hq * kMaxRank);
}

}  // namespace

cudaError_t launch_generic_prefill(const lisa_shared_prefill_args& a, cudaStream_t s) {
    PrefillParams p;
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.d = a.d; p.c = a.chain_len;
    p.q0 = make_view(a.q0); p.k0 = make_view(a.k0); p.v = make_view(a.v); p.o = make_view(a.o);
    for (int k = 0; k < a.chain_len; ++k) p.links[k] = make_link(a.links[k]);
    const size_t smem = smem_bytes(a.Hq, a.d, a.chain_len);
    cudaError_t e = cudaFuncSetAttribute(generic_prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid(a.N, a.B);
    generic_prefill_kernel<<<grid, kThreads, smem, s>>>(p);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace lisa
