// C-ABI entry points: host-side validation and dispatch.  No arithmetic of the method lives here.
#include <atomic>
#include <cmath>
#include <cstring>

#include "common.cuh"

namespace lisa {

static __device__ int g_status[4];
static thread_local int t_last_cuda_error = 0;

static std::atomic<int> g_force_general{0};
static std::atomic<uint64_t> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int* status_words() {
    static int* cached[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status) != cudaSuccess) return nullptr;
        cached[dev] = reinterpret_cast<int*>(p);
    }
    return cached[dev];
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 1;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {

lisa_status_t cuda_fail(cudaError_t e) {
    t_last_cuda_error = (int)e;
    (void)cudaGetLastError();  // do not let a non-sticky error leak into the next call's launch check
    return LISA_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool dtype_ok(int dt) { return dt == LISA_F32 || dt == LISA_BF16; }
size_t esize(int dt) { return dt == LISA_BF16 ? 2 : 4; }

lisa_status_t check_tensor(const lisa_tensor& t) {
    if (!t.ptr || !dtype_ok(t.dtype) || !aligned16(t.ptr)) return LISA_ERR_INVALID_ARG;
    return LISA_OK;
}

lisa_status_t check_dims(int B, int N, int Hq, int Hkv, int d) {
    if (B < 1 || N < 1 || Hq < 1 || Hkv < 1 || d < 1) return LISA_ERR_INVALID_ARG;
    if (Hq % Hkv != 0) return LISA_ERR_INVALID_ARG;
    if (Hq > kMaxHeads) return LISA_ERR_UNSUPPORTED;
    if (d != 32 && d != 64 && d != 128) return LISA_ERR_UNSUPPORTED;
    return LISA_OK;
}

lisa_status_t check_link(const lisa_link& l, int Hq, bool prefill) {
    if (l.r < 1) return LISA_ERR_INVALID_ARG;
    if (l.r > kMaxRank) return LISA_ERR_UNSUPPORTED;
    if (l.integrate < LISA_INTEGRATE_ADD || l.integrate > LISA_INTEGRATE_PLUS) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = check_tensor(l.qp);
    if (st != LISA_OK) return st;
    if (prefill && (st = check_tensor(l.kp)) != LISA_OK) return st;
    if (l.integrate == LISA_INTEGRATE_PLUS) return LISA_OK;
    if (l.act < LISA_ACT_NONE || l.act > LISA_ACT_SILU) return LISA_ERR_INVALID_ARG;
    if (l.ffn_layers != 1 && l.ffn_layers != 2) return LISA_ERR_INVALID_ARG;
    if (!dtype_ok(l.w_dtype) || !l.w1 || l.m < 1) return LISA_ERR_INVALID_ARG;
    if (l.m > kMaxHidden) return LISA_ERR_UNSUPPORTED;
    if (l.ffn_layers == 2 && !l.w2) return LISA_ERR_INVALID_ARG;
    if (l.ffn_layers == 1 && l.m != Hq) return LISA_ERR_INVALID_ARG;
    return LISA_OK;
}

lisa_status_t check_cache(const lisa_kvcache_layer* c, int kind, bool need_ptrs) {
    if (!c || c->kind != kind || !dtype_ok(c->dtype)) return LISA_ERR_INVALID_ARG;
    if (c->B < 1 || c->Hkv < 1 || c->L_cap < 8 || c->L_cap % 8 != 0) return LISA_ERR_INVALID_ARG;
    if (c->d != 32 && c->d != 64 && c->d != 128) return LISA_ERR_UNSUPPORTED;
    if (kind == LISA_CACHE_SHARED) {
        if (c->r < 1) return LISA_ERR_INVALID_ARG;
        if (c->r > kMaxRank) return LISA_ERR_UNSUPPORTED;
    }
    if (need_ptrs && (!c->k || !c->v || !aligned16(c->k) || !aligned16(c->v))) return LISA_ERR_INVALID_ARG;
    return LISA_OK;
}

// Largest dynamic shared memory a CTA may opt into on the current device (B200: 227 KB, also the answer when the
// query fails, e.g. with no device present).
size_t max_optin_smem() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess || v <= 0) {
        (void)cudaGetLastError();
        return 232448;
    }
    return (size_t)v;
}

lisa_status_t check_workspace(const void* ws, size_t have, size_t need) {
    if (need == 0) return LISA_OK;
    if (!ws || have < need || !aligned16(ws)) return LISA_ERR_WORKSPACE;
    return LISA_OK;
}

lisa_status_t validate_prefill(const lisa_shared_prefill_args* a) {
    if (!a || a->struct_size != sizeof(lisa_shared_prefill_args)) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = check_dims(a->B, a->N, a->Hq, a->Hkv, a->d);
    if (st != LISA_OK) return st;
    if (a->chain_len < 0) return LISA_ERR_INVALID_ARG;
    if (a->chain_len > kMaxChain) return LISA_ERR_UNSUPPORTED;
    if (a->chain_len > 0 && !a->links) return LISA_ERR_INVALID_ARG;
    const lisa_tensor* ts[4] = {&a->q0, &a->k0, &a->v, &a->o};
    for (const lisa_tensor* t : ts)
        if ((st = check_tensor(*t)) != LISA_OK) return st;
    for (int k = 0; k < a->chain_len; ++k)
        if ((st = check_link(a->links[k], a->Hq, true)) != LISA_OK) return st;
    return LISA_OK;
}

lisa_status_t validate_anchor_decode(const lisa_anchor_args* a) {
    lisa_status_t st = check_cache(a->cache, LISA_CACHE_STANDARD, true);
    if (st != LISA_OK) return st;
    const lisa_kvcache_layer& c = *a->cache;
    if (a->Nq != 1 || a->B > c.B || a->Hkv != c.Hkv || a->d != c.d) return LISA_ERR_INVALID_ARG;
    if (a->L < 1 || a->L > c.L_cap) return LISA_ERR_INVALID_ARG;
    if ((st = check_tensor(a->q)) != LISA_OK || (st = check_tensor(a->o)) != LISA_OK) return st;
    if (a->scores_dtype != LISA_F32 && a->scores_dtype != LISA_BF16) return LISA_ERR_INVALID_ARG;
    if (a->out_scores && (reinterpret_cast<uintptr_t>(a->out_scores) & (a->scores_dtype == LISA_BF16 ? 1u : 3u))) return LISA_ERR_INVALID_ARG;
    return LISA_OK;
}

lisa_status_t validate_shared_decode(const lisa_shared_decode_args* a) {
    if (!a || a->struct_size != sizeof(lisa_shared_decode_args)) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = check_cache(a->cache, LISA_CACHE_SHARED, true);
    if (st != LISA_OK) return st;
    const lisa_kvcache_layer& c = *a->cache;
    if ((st = check_dims(a->B, 1, a->Hq, c.Hkv, c.d)) != LISA_OK) return st;
    if (a->B > c.B || a->L < 1 || a->L > c.L_cap) return LISA_ERR_INVALID_ARG;
    if (a->link.r != c.r) return LISA_ERR_INVALID_ARG;
    if ((st = check_link(a->link, a->Hq, false)) != LISA_OK) return st;
    if (a->scores_dtype != LISA_F32 && a->scores_dtype != LISA_BF16) return LISA_ERR_INVALID_ARG;
    const uintptr_t row_align = a->scores_dtype == LISA_BF16 ? 1u : 3u;
    if (!a->prev_scores || (reinterpret_cast<uintptr_t>(a->prev_scores) & row_align)) return LISA_ERR_INVALID_ARG;
    if (a->out_scores && (reinterpret_cast<uintptr_t>(a->out_scores) & row_align)) return LISA_ERR_INVALID_ARG;
    if (a->out_scores && a->out_scores == a->prev_scores) return LISA_ERR_INVALID_ARG;
    if ((st = check_tensor(a->o)) != LISA_OK) return st;
    // a head count and FFN width whose weights do not fit one CTA's shared memory are outside the kernel's range
    if (shared_decode_smem(a->Hq, a->link.m, a->link.integrate) > max_optin_smem()) return LISA_ERR_UNSUPPORTED;
    return LISA_OK;
}

}  // namespace
}  // namespace lisa

using namespace lisa;

extern "C" {

int lisa_version(void) { return 1000; }
void lisa_force_general_kernels(int on) { g_force_general.store(on ? 1 : 0); }
uint64_t lisa_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }
int lisa_last_cuda_error(void) { return t_last_cuda_error; }

const char* lisa_status_string(int status) {
    switch (status) {
        case LISA_OK: return "ok";
        case LISA_ERR_INVALID_ARG: return "invalid argument";
        case LISA_ERR_UNSUPPORTED: return "unsupported shape or type";
        case LISA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case LISA_ERR_CUDA: return "CUDA error";
        case LISA_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

lisa_status_t lisa_kvcache_bytes(const lisa_kvcache_layer* layer, size_t* k_bytes, size_t* v_bytes) {
    if (!layer || !k_bytes || !v_bytes) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = check_cache(layer, layer->kind, false);
    if (st != LISA_OK) return st;
    if (layer->kind != LISA_CACHE_STANDARD && layer->kind != LISA_CACHE_SHARED) return LISA_ERR_INVALID_ARG;
    const size_t rows = (size_t)layer->B * layer->Hkv * layer->L_cap;
    const size_t kw = layer->kind == LISA_CACHE_SHARED ? (size_t)layer->r : (size_t)layer->d;
    *k_bytes = rows * kw * esize(layer->dtype);
    *v_bytes = rows * (size_t)layer->d * esize(layer->dtype);
    return LISA_OK;
}

namespace {
// The single-layer call that computes layer k (0-based) of a chain.
lisa_shared_prefill_args chain_layer(const lisa_shared_prefill_chain_args& a, int k) {
    lisa_shared_prefill_args p;
    std::memset(&p, 0, sizeof(p));
    p.struct_size = sizeof(p);
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.d = a.d; p.chain_len = k + 1;
    p.q0 = a.q0; p.k0 = a.k0; p.v = a.v[k]; p.o = a.o[k];
    p.links = a.links;
    p.workspace = a.workspace; p.workspace_bytes = a.workspace_bytes;
    return p;
}

// The one-link layer a carried call runs, validated; where the anchor's q0, k0 are not read (every layer but the first
// of a chain) descriptors of the right shape stand in for them so that the common checks apply unchanged.
lisa_status_t carried_layer(const lisa_shared_prefill_carry_args& a, lisa_shared_prefill_args* out) {
    lisa_shared_prefill_args p = a.layer;
    if (p.struct_size != sizeof(lisa_shared_prefill_args) || p.chain_len != 1 || !p.links) return LISA_ERR_INVALID_ARG;
    if (!a.first) { p.q0 = p.o; p.k0 = p.v; }
    lisa_status_t st = validate_prefill(&p);
    if (st != LISA_OK) return st;
    if (!tc_shared_prefill_supported(p)) return LISA_ERR_UNSUPPORTED;
    *out = p;
    return LISA_OK;
}
}  // namespace

size_t lisa_prefill_scores_bytes(int32_t B, int32_t N, int32_t Hq) {
    return (B < 1 || N < 1 || Hq < 1) ? 0 : tc_carry_bytes(B, N, Hq);
}

static lisa_status_t shared_prefill_carry_impl(const lisa_shared_prefill_carry_args* a, lisa_stream_t stream, TcHostIO* ho);
lisa_status_t lisa_attn_shared_prefill_carry(const lisa_shared_prefill_carry_args* a, lisa_stream_t stream) {
    return shared_prefill_carry_impl(a, stream, nullptr);
}
// ho: the layer's output is also wanted in host memory (the host-memory entry points)
static lisa_status_t shared_prefill_carry_impl(const lisa_shared_prefill_carry_args* a, lisa_stream_t stream, TcHostIO* ho) {
    if (!a || a->struct_size != sizeof(lisa_shared_prefill_carry_args)) return LISA_ERR_INVALID_ARG;
    lisa_shared_prefill_args p;
    lisa_status_t st = carried_layer(*a, &p);
    if (st != LISA_OK) return st;
    if (!a->scores || (reinterpret_cast<uintptr_t>(a->scores) & 255u) || a->scores_bytes < tc_carry_bytes(p.B, p.N, p.Hq)) return LISA_ERR_INVALID_ARG;
    if ((st = check_workspace(p.workspace, p.workspace_bytes, tc_shared_prefill_carry_workspace(p))) != LISA_OK) return st;
    const TcCarry cy{a->scores, a->first != 0, a->keep != 0};
    cudaError_t e = launch_tc_shared_prefill_chain(p, nullptr, nullptr, p.workspace, static_cast<cudaStream_t>(stream), &cy, ho);
    return e == cudaSuccess ? LISA_OK : cuda_fail(e);
}

lisa_status_t lisa_workspace_bytes(int32_t op, const void* args, size_t* bytes) {
    if (!args || !bytes) return LISA_ERR_INVALID_ARG;
    if (op == LISA_OP_ANCHOR) {
        const lisa_anchor_args* a = static_cast<const lisa_anchor_args*>(args);
        if (a->struct_size != sizeof(lisa_anchor_args)) return LISA_ERR_INVALID_ARG;
        *bytes = a->cache ? decode_workspace(a->B, a->Hq, a->d, a->L) : 0;
        return LISA_OK;
    }
    if (op == LISA_OP_SHARED_PREFILL) {
        const lisa_shared_prefill_args* a = static_cast<const lisa_shared_prefill_args*>(args);
        if (a->struct_size != sizeof(lisa_shared_prefill_args)) return LISA_ERR_INVALID_ARG;
        *bytes = 0;
        if (!g_force_general.load() && a->chain_len > 0 && a->links && a->Hq > 0 && a->Hkv > 0 && a->Hq % a->Hkv == 0 &&
            tc_shared_prefill_supported(*a))
            *bytes = tc_shared_prefill_workspace(*a);
        return LISA_OK;
    }
    if (op == LISA_OP_SHARED_PREFILL_CHAIN) {
        const lisa_shared_prefill_chain_args* a = static_cast<const lisa_shared_prefill_chain_args*>(args);
        if (a->struct_size != sizeof(lisa_shared_prefill_chain_args) || a->chain_len < 1 || !a->v || !a->o) return LISA_ERR_INVALID_ARG;
        size_t need = 0;   // the deepest layer needs the most, on either path
        for (int k = 0; k < a->chain_len; ++k) {
            const lisa_shared_prefill_args p = chain_layer(*a, k);
            size_t n = 0;
            lisa_status_t st = lisa_workspace_bytes(LISA_OP_SHARED_PREFILL, &p, &n);
            if (st != LISA_OK) return st;
            need = n > need ? n : need;
        }
        *bytes = need;
        return LISA_OK;
    }
    if (op == LISA_OP_SHARED_PREFILL_CARRY) {
        const lisa_shared_prefill_carry_args* a = static_cast<const lisa_shared_prefill_carry_args*>(args);
        if (a->struct_size != sizeof(lisa_shared_prefill_carry_args)) return LISA_ERR_INVALID_ARG;
        lisa_shared_prefill_args p;
        lisa_status_t st = carried_layer(*a, &p);
        if (st != LISA_OK) return st;
        *bytes = tc_shared_prefill_carry_workspace(p);
        return LISA_OK;
    }
    if (op == LISA_OP_SHARED_DECODE) {
        const lisa_shared_decode_args* a = static_cast<const lisa_shared_decode_args*>(args);
        if (a->struct_size != sizeof(lisa_shared_decode_args) || !a->cache) return LISA_ERR_INVALID_ARG;
        *bytes = decode_workspace(a->B, a->Hq, a->cache->d, a->L);
        return LISA_OK;
    }
    return LISA_ERR_INVALID_ARG;
}

static lisa_status_t shared_prefill_impl(const lisa_shared_prefill_args* a, lisa_stream_t stream, TcHostIO* ho);
lisa_status_t lisa_attn_shared_prefill(const lisa_shared_prefill_args* a, lisa_stream_t stream) {
    return shared_prefill_impl(a, stream, nullptr);
}
// Whole-tensor copies of the inputs a host-memory call left to the launching side (paths that do not stream them).
static cudaError_t host_inputs_whole(const lisa_shared_prefill_args& a, const TcHostIO& io, cudaStream_t s) {
    const size_t rows = (size_t)a.B * a.N;
    cudaError_t e = cudaSuccess;
    if (io.host_q0) e = cudaMemcpyAsync(a.q0.ptr, io.host_q0, rows * a.Hq * a.d * esize(a.q0.dtype), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && io.host_k0) e = cudaMemcpyAsync(a.k0.ptr, io.host_k0, rows * a.Hkv * a.d * esize(a.k0.dtype), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && io.host_v) e = cudaMemcpyAsync(a.v.ptr, io.host_v, rows * a.Hkv * a.d * esize(a.v.dtype), cudaMemcpyHostToDevice, s);
    return e;
}
static lisa_status_t shared_prefill_impl(const lisa_shared_prefill_args* a, lisa_stream_t stream, TcHostIO* ho) {
    lisa_status_t st = validate_prefill(a);
    if (st != LISA_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool orchestrated = !g_force_general.load() && a->chain_len > 0 && tc_shared_prefill_supported(*a);
    if (ho && !orchestrated) {   // the tensor-core orchestration brings the inputs in itself, wave by wave
        cudaError_t e = host_inputs_whole(*a, *ho, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (!g_force_general.load() && a->d == 128 && a->chain_len == 0) {
        TcFlashArgs f{a->B, a->N, a->Hq, a->Hkv, 128, a->q0, a->k0, a->v, a->o, 1.0f / sqrtf((float)a->d), nullptr, 0, 0,
                      0, (a->N + 127) / 128};
        if (tc_flash_supported(f)) {
            cudaError_t e = launch_tc_flash(f, s);
            return e == cudaSuccess ? LISA_OK : cuda_fail(e);
        }
    }
    if (orchestrated) {
        const size_t need = tc_shared_prefill_workspace(*a);
        if ((st = check_workspace(a->workspace, a->workspace_bytes, need)) != LISA_OK) return st;
        cudaError_t e = launch_tc_shared_prefill_chain(*a, nullptr, nullptr, a->workspace, s, nullptr, ho);
        return e == cudaSuccess ? LISA_OK : cuda_fail(e);
    }
    cudaError_t e = launch_generic_prefill(*a, s);
    return e == cudaSuccess ? LISA_OK : cuda_fail(e);
}

lisa_status_t lisa_attn_shared_prefill_chain(const lisa_shared_prefill_chain_args* a, lisa_stream_t stream) {
    if (!a || a->struct_size != sizeof(lisa_shared_prefill_chain_args) || a->chain_len < 1 || !a->v || !a->o || !a->links)
        return LISA_ERR_INVALID_ARG;
    // every layer is validated before anything is launched
    bool tensor_cores = !g_force_general.load();
    for (int k = 0; k < a->chain_len; ++k) {
        const lisa_shared_prefill_args p = chain_layer(*a, k);
        lisa_status_t st = validate_prefill(&p);
        if (st != LISA_OK) return st;
        tensor_cores = tensor_cores && tc_shared_prefill_supported(p);
    }
    size_t need = 0;
    lisa_status_t st = lisa_workspace_bytes(LISA_OP_SHARED_PREFILL_CHAIN, a, &need);
    if (st != LISA_OK) return st;
    if ((st = check_workspace(a->workspace, a->workspace_bytes, need)) != LISA_OK) return st;
    if (tensor_cores) {
        const lisa_shared_prefill_args deepest = chain_layer(*a, a->chain_len - 1);
        cudaError_t e = launch_tc_shared_prefill_chain(deepest, a->v, a->o, a->workspace, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? LISA_OK : cuda_fail(e);
    }
    for (int k = 0; k < a->chain_len; ++k) {
        const lisa_shared_prefill_args p = chain_layer(*a, k);
        if ((st = lisa_attn_shared_prefill(&p, stream)) != LISA_OK) return st;
    }
    return LISA_OK;
}

lisa_status_t lisa_attn_anchor(const lisa_anchor_args* a, lisa_stream_t stream) {
    if (!a || a->struct_size != sizeof(lisa_anchor_args)) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = check_dims(a->B, a->Nq, a->Hq, a->Hkv, a->d);
    if (st != LISA_OK) return st;
    if (a->cache) {
        if ((st = validate_anchor_decode(a)) != LISA_OK) return st;
        const size_t need = decode_workspace(a->B, a->Hq, a->d, a->L);
        if ((st = check_workspace(a->workspace, a->workspace_bytes, need)) != LISA_OK) return st;
        cudaError_t e = launch_anchor_decode(*a, a->workspace, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? LISA_OK : cuda_fail(e);
    }
    lisa_shared_prefill_args p;
    std::memset(&p, 0, sizeof(p));
    p.struct_size = sizeof(p);
    p.B = a->B; p.N = a->Nq; p.Hq = a->Hq; p.Hkv = a->Hkv; p.d = a->d; p.chain_len = 0;
    p.q0 = a->q; p.k0 = a->k; p.v = a->v; p.o = a->o;
    p.workspace = a->workspace; p.workspace_bytes = a->workspace_bytes;
    return lisa_attn_shared_prefill(&p, stream);
}

lisa_status_t lisa_attn_shared_decode(const lisa_shared_decode_args* a, lisa_stream_t stream) {
    lisa_status_t st = validate_shared_decode(a);
    if (st != LISA_OK) return st;
    const size_t need = decode_workspace(a->B, a->Hq, a->cache->d, a->L);
    if ((st = check_workspace(a->workspace, a->workspace_bytes, need)) != LISA_OK) return st;
    cudaError_t e = launch_shared_decode(*a, a->workspace, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? LISA_OK : cuda_fail(e);
}

// ---- decode with the scratch held inside the library image -----------------------------------------
// For callers that cannot allocate device memory when they decode (see lisa.h).  The array's name is only
// a host-side handle: kernels get the device address that cudaGetSymbolAddress returns for the current device.
static __device__ __align__(256) unsigned char g_static_scratch[LISA_STATIC_SCRATCH_BYTES];

// Device address of the array on the current device (looked up once per device); on failure *err holds the CUDA code.
static void* static_scratch_address(cudaError_t* err) {
    static void* cached[64] = {nullptr};
    int dev = 0;
    if ((*err = cudaGetDevice(&dev)) != cudaSuccess) return nullptr;
    if (dev < 0 || dev >= 64) { *err = cudaErrorInvalidDevice; return nullptr; }
    if (!cached[dev]) {
        void* p = nullptr;
        if ((*err = cudaGetSymbolAddress(&p, g_static_scratch)) != cudaSuccess) return nullptr;
        cached[dev] = p;
    }
    return cached[dev];
}

lisa_status_t lisa_attn_shared_decode_static(const lisa_shared_decode_args* a, lisa_stream_t stream) {
    lisa_status_t st = validate_shared_decode(a);
    if (st != LISA_OK) return st;
    const size_t need = decode_workspace(a->B, a->Hq, a->cache->d, a->L);
    if (need > (size_t)LISA_STATIC_SCRATCH_BYTES) return LISA_ERR_WORKSPACE;
    cudaError_t lookup = cudaSuccess;
    void* scratch = static_scratch_address(&lookup);
    if (!scratch) return cuda_fail(lookup);
    cudaError_t e = launch_shared_decode(*a, scratch, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? LISA_OK : cuda_fail(e);
}

lisa_status_t lisa_project(const lisa_project_args* a, lisa_stream_t stream) {
    if (!a || a->struct_size != sizeof(lisa_project_args)) return LISA_ERR_INVALID_ARG;
    if (a->B < 1 || a->N < 1 || a->d_in < 1 || a->n_outputs < 1 || a->n_outputs > 4) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = check_tensor(a->x);
    if (st != LISA_OK) return st;
    if (!a->w || !aligned16(a->w) || !dtype_ok(a->w_dtype) || a->w_dtype != a->x.dtype) return LISA_ERR_INVALID_ARG;
    for (int o = 0; o < a->n_outputs; ++o) {
        if ((st = check_tensor(a->outputs[o].t)) != LISA_OK) return st;
        if (a->outputs[o].H < 1 || a->outputs[o].x < 1) return LISA_ERR_INVALID_ARG;
    }
    cudaError_t e = (!g_force_general.load() && tc_project_supported(*a)) ? launch_tc_project(*a, static_cast<cudaStream_t>(stream))
                                                                          : launch_generic_project(*a, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? LISA_OK : cuda_fail(e);
}

lisa_status_t lisa_kvcache_append(const lisa_kvcache_layer* layer, const lisa_tensor* k_or_kp, const lisa_tensor* v,
                                  const int32_t* seq_lens_before, int32_t n_new, lisa_stream_t stream) {
    if (!layer || !k_or_kp || !v || n_new < 1) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = check_cache(layer, layer->kind, true);
    if (st != LISA_OK) return st;
    if ((st = check_tensor(*k_or_kp)) != LISA_OK || (st = check_tensor(*v)) != LISA_OK) return st;
    if (k_or_kp->dtype != layer->dtype || v->dtype != layer->dtype) return LISA_ERR_INVALID_ARG;
    const int64_t vec = 16 / (int64_t)esize(layer->dtype);  // rows of d elements move as 16-byte vectors
    auto rows_ok = [&](const lisa_tensor& t) { return t.stride_b % vec == 0 && t.stride_n % vec == 0 && t.stride_h % vec == 0; };
    if (!rows_ok(*v)) return LISA_ERR_INVALID_ARG;
    if (layer->kind == LISA_CACHE_STANDARD && !rows_ok(*k_or_kp)) return LISA_ERR_INVALID_ARG;
    cudaError_t e = launch_kvcache_append(*layer, *k_or_kp, *v, seq_lens_before, n_new, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? LISA_OK : cuda_fail(e);
}

namespace {
// Walks the layers of a multi-layer cache: per-layer descriptor and 256-byte aligned offsets of k and v.
lisa_status_t walk_cache(const lisa_kvcache_desc* d, char* base, lisa_kvcache* out, size_t* total) {
    if (!d || d->struct_size != sizeof(lisa_kvcache_desc) || !d->kinds) return LISA_ERR_INVALID_ARG;
    if (d->n_layers < 1 || d->n_layers > LISA_MAX_LAYERS) return LISA_ERR_INVALID_ARG;
    size_t off = 0;
    for (int l = 0; l < d->n_layers; ++l) {
        lisa_kvcache_layer layer{d->kinds[l], d->dtype, d->B, d->Hkv, d->L_cap, d->d, d->kinds[l] == LISA_CACHE_SHARED ? d->r : 0, 0, nullptr, nullptr};
        if (layer.kind != LISA_CACHE_STANDARD && layer.kind != LISA_CACHE_SHARED) return LISA_ERR_INVALID_ARG;
        size_t kb = 0, vb = 0;
        lisa_status_t st = lisa_kvcache_bytes(&layer, &kb, &vb);
        if (st != LISA_OK) return st;
        if (base) { layer.k = base + off; }
        off += (kb + 255) & ~(size_t)255;
        if (base) { layer.v = base + off; }
        off += (vb + 255) & ~(size_t)255;
        if (out) out->layers[l] = layer;
    }
    if (out) { out->n_layers = d->n_layers; out->reserved = 0; }
    if (total) *total = off;
    return LISA_OK;
}
}  // namespace

lisa_status_t lisa_kvcache_total_bytes(const lisa_kvcache_desc* desc, size_t* bytes) {
    if (!bytes) return LISA_ERR_INVALID_ARG;
    return walk_cache(desc, nullptr, nullptr, bytes);
}

lisa_status_t lisa_kvcache_init(const lisa_kvcache_desc* desc, void* base, size_t base_bytes, lisa_kvcache* cache) {
    if (!cache || !base || (reinterpret_cast<uintptr_t>(base) & 255u)) return LISA_ERR_INVALID_ARG;
    size_t need = 0;
    lisa_status_t st = walk_cache(desc, nullptr, nullptr, &need);
    if (st != LISA_OK) return st;
    if (base_bytes < need) return LISA_ERR_WORKSPACE;
    return walk_cache(desc, static_cast<char*>(base), cache, nullptr);
}

lisa_status_t lisa_kvcache_append_layer(const lisa_kvcache* cache, int32_t layer, const lisa_tensor* k_or_kp, const lisa_tensor* v,
                                        const int32_t* seq_lens_before, int32_t n_new, lisa_stream_t stream) {
    if (!cache || layer < 0 || layer >= cache->n_layers || cache->n_layers > LISA_MAX_LAYERS) return LISA_ERR_INVALID_ARG;
    return lisa_kvcache_append(&cache->layers[layer], k_or_kp, v, seq_lens_before, n_new, stream);
}

lisa_status_t lisa_prefill_phase_timing(int enable) {
    cudaError_t e = prefill_phase_timing(enable != 0);
    return e == cudaSuccess ? LISA_OK : cuda_fail(e);
}

lisa_status_t lisa_prefill_phase_times(float* ms4) {
    if (!ms4) return LISA_ERR_INVALID_ARG;
    cudaError_t e = prefill_phase_times(ms4);
    return e == cudaSuccess ? LISA_OK : cuda_fail(e);
}

lisa_status_t lisa_check(lisa_stream_t stream) {
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    int* dev = status_words();
    if (!dev) return cuda_fail(cudaErrorUnknown);
    int host[4] = {0, 0, 0, 0};
    if ((e = cudaMemcpy(host, dev, sizeof(host), cudaMemcpyDeviceToHost)) != cudaSuccess) return cuda_fail(e);
    if (host[0] || host[1]) {
        if ((e = cudaMemset(dev, 0, sizeof(host))) != cudaSuccess) return cuda_fail(e);
    }
    if (host[1]) return LISA_ERR_TIMEOUT;
    if (host[0]) return LISA_ERR_INVALID_ARG;
    return LISA_OK;
}

// ---- host-memory variant: stage in, run, copy out -------------------------------------------------
namespace {
struct Arena {
    char* base;
    size_t off;
    void* take(size_t bytes) {
        void* p = base ? base + off : nullptr;
        off += (bytes + 255) & ~(size_t)255;
        return p;
    }
};

// Lays the call's tensors out in the arena. With arena.base == nullptr only the size is computed.
// dev receives device-side copies of the descriptors; h2d lists (dst, src, bytes) to copy.
struct Copy { void* dst; const void* src; size_t bytes; int streamed; };   // streamed: q0 (1), k0 (2), v (3) -- left to the launching side

// anchor == false: q0 and k0 are not read by the call (a carried layer past the first): nothing is staged for them.
size_t plan_host_call(const lisa_shared_prefill_args& h, char* base, lisa_shared_prefill_args* dev, lisa_link* dlinks,
                      Copy* copies, int* n_copies, size_t* o_bytes, bool anchor = true) {
    Arena ar{base, 0};
    int nc = 0;
    auto dense = [&](const lisa_tensor& src, int H, int x, lisa_tensor* dst, bool copy_in, int streamed = 0) {
        const size_t bytes = (size_t)h.B * h.N * H * x * esize(src.dtype);
        void* p = ar.take(bytes);
        if (dst) {
            *dst = lisa_tensor{p, src.dtype, 0, (int64_t)h.N * H * x, (int64_t)H * x, (int64_t)x};
            if (copy_in) copies[nc++] = Copy{p, src.ptr, bytes, streamed};
        }
        return bytes;
    };
    if (anchor) {
        dense(h.q0, h.Hq, h.d, dev ? &dev->q0 : nullptr, true, 1);
        dense(h.k0, h.Hkv, h.d, dev ? &dev->k0 : nullptr, true, 2);
    }
    dense(h.v, h.Hkv, h.d, dev ? &dev->v : nullptr, true, 3);
    const size_t ob = dense(h.o, h.Hq, h.d, dev ? &dev->o : nullptr, false);
    if (o_bytes) *o_bytes = ob;
    for (int k = 0; k < h.chain_len; ++k) {
        const lisa_link& l = h.links[k];
        lisa_link* dl = dlinks ? &dlinks[k] : nullptr;
        if (dl) *dl = l;
        dense(l.qp, h.Hq, l.r, dl ? &dl->qp : nullptr, true);
        dense(l.kp, h.Hkv, l.r, dl ? &dl->kp : nullptr, true);
        if (l.integrate == LISA_INTEGRATE_PLUS) continue;
        const int h_in = l.integrate == LISA_INTEGRATE_CONCAT ? 2 * h.Hq : h.Hq;
        const size_t ws = esize(l.w_dtype);
        auto weight = [&](const void* src, size_t n, const void** dst) {
            if (!src) return;
            void* p = ar.take(n * ws);
            if (dst) { *dst = p; copies[nc++] = Copy{p, src, n * ws, 0}; }
        };
        weight(l.w1, (size_t)h_in * l.m, dl ? &dl->w1 : nullptr);
        weight(l.b1, (size_t)l.m, dl ? &dl->b1 : nullptr);
        if (l.ffn_layers == 2) {
            weight(l.w2, (size_t)l.m * h.Hq, dl ? &dl->w2 : nullptr);
            weight(l.b2, (size_t)h.Hq, dl ? &dl->b2 : nullptr);
        }
    }
    if (n_copies) *n_copies = nc;
    return ar.off;
}

lisa_status_t validate_host_args(const lisa_shared_prefill_args* a) {
    if (!a || a->struct_size != sizeof(lisa_shared_prefill_args)) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = check_dims(a->B, a->N, a->Hq, a->Hkv, a->d);
    if (st != LISA_OK) return st;
    if (a->chain_len < 0 || (a->chain_len > 0 && !a->links)) return LISA_ERR_INVALID_ARG;
    if (a->chain_len > kMaxChain) return LISA_ERR_UNSUPPORTED;
    if (!a->q0.ptr || !a->k0.ptr || !a->v.ptr || !a->o.ptr) return LISA_ERR_INVALID_ARG;
    if (!dtype_ok(a->q0.dtype) || !dtype_ok(a->k0.dtype) || !dtype_ok(a->v.dtype) || !dtype_ok(a->o.dtype))
        return LISA_ERR_INVALID_ARG;
    for (int k = 0; k < a->chain_len; ++k) {
        const lisa_link& l = a->links[k];
        if (!l.qp.ptr || !l.kp.ptr || !dtype_ok(l.qp.dtype) || !dtype_ok(l.kp.dtype)) return LISA_ERR_INVALID_ARG;
        if (l.r < 1 || l.m < 0 || !dtype_ok(l.w_dtype)) return LISA_ERR_INVALID_ARG;
        if (l.r > kMaxRank || l.m > kMaxHidden) return LISA_ERR_UNSUPPORTED;
    }
    return LISA_OK;
}
}  // namespace

namespace {
// Scratch bytes of the staged call.  The host descriptors' strides are ignored by contract, so the question is put
// to the dense device-side descriptors the call will actually run with (laid out from a 256-byte aligned dummy base:
// only strides and alignment matter to the answer, the pointers are not read).
lisa_status_t staged_workspace_bytes(const lisa_shared_prefill_args& h, size_t* ws) {
    lisa_shared_prefill_args dev = h;
    lisa_link dlinks[kMaxChain];
    Copy copies[3 + 6 * kMaxChain];
    int nc = 0;
    plan_host_call(h, reinterpret_cast<char*>(uintptr_t(1) << 20), &dev, dlinks, copies, &nc, nullptr);
    dev.links = dlinks;
    return lisa_workspace_bytes(LISA_OP_SHARED_PREFILL, &dev, ws);
}
}  // namespace

lisa_status_t lisa_host_arena_bytes(const lisa_shared_prefill_args* host_args, size_t* bytes) {
    if (!bytes) return LISA_ERR_INVALID_ARG;
    lisa_status_t st = validate_host_args(host_args);
    if (st != LISA_OK) return st;
    size_t ws = 0;
    if ((st = staged_workspace_bytes(*host_args, &ws)) != LISA_OK) return st;
    *bytes = plan_host_call(*host_args, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr) + ((ws + 255) & ~(size_t)255);
    return LISA_OK;
}

lisa_status_t lisa_attn_shared_prefill_host(const lisa_shared_prefill_args* host_args, void* device_arena,
                                            size_t arena_bytes, lisa_stream_t stream) {
    size_t need = 0;
    lisa_status_t st = lisa_host_arena_bytes(host_args, &need);
    if (st != LISA_OK) return st;
    if (!device_arena || arena_bytes < need || (reinterpret_cast<uintptr_t>(device_arena) & 255u)) return LISA_ERR_WORKSPACE;
    lisa_shared_prefill_args dev = *host_args;
    lisa_link dlinks[kMaxChain];
    Copy copies[3 + 6 * kMaxChain];
    int nc = 0;
    size_t o_bytes = 0;
    const size_t used = plan_host_call(*host_args, static_cast<char*>(device_arena), &dev, dlinks, copies, &nc, &o_bytes);
    dev.links = dlinks;
    size_t ws = 0;
    if ((st = lisa_workspace_bytes(LISA_OP_SHARED_PREFILL, &dev, &ws)) != LISA_OK) return st;
    dev.workspace = ws ? static_cast<char*>(device_arena) + used : nullptr;
    dev.workspace_bytes = ws;
    // everything that can refuse the call is checked before the first copy is enqueued
    if ((st = validate_prefill(&dev)) != LISA_OK) return st;
    if (used + ((ws + 255) & ~(size_t)255) > arena_bytes) return LISA_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    // q0, k0, v come in and o goes back wave by wave while other waves compute, where the path supports it
    TcHostIO ho{host_args->o.ptr, nullptr, nullptr, nullptr, false};
    for (int i = 0; i < nc; ++i) {
        if (copies[i].streamed == 1) ho.host_q0 = copies[i].src;
        else if (copies[i].streamed == 2) ho.host_k0 = copies[i].src;
        else if (copies[i].streamed == 3) ho.host_v = copies[i].src;
        else if ((e = cudaMemcpyAsync(copies[i].dst, copies[i].src, copies[i].bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess)
            return cuda_fail(e);
    }
    if ((st = shared_prefill_impl(&dev, stream, &ho)) != LISA_OK) return st;
    if (!ho.out_done && (e = cudaMemcpyAsync(host_args->o.ptr, dev.o.ptr, o_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(e);
    return LISA_OK;
}


// ---- carried scores, tensors in host memory ----
namespace {
// The device-side form of a carried host call laid out in the arena (base == nullptr: sizes only), validated, with its workspace.
lisa_status_t plan_carry_host(const lisa_shared_prefill_carry_args& h, char* base, lisa_shared_prefill_carry_args* dev, lisa_link* dlink,
                              Copy* copies, int* nc, size_t* o_bytes, size_t* total) {
    if (h.struct_size != sizeof(lisa_shared_prefill_carry_args)) return LISA_ERR_INVALID_ARG;
    lisa_shared_prefill_args hl = h.layer;
    if (hl.struct_size != sizeof(lisa_shared_prefill_args) || hl.chain_len != 1 || !hl.links) return LISA_ERR_INVALID_ARG;
    if (!h.first) { hl.q0 = hl.o; hl.k0 = hl.v; }   // not read: descriptors of the right shape for the common checks
    lisa_status_t st = validate_host_args(&hl);
    if (st != LISA_OK) return st;
    *dev = h;
    char* lay = base ? base : reinterpret_cast<char*>(uintptr_t(1) << 20);   // strides and alignment are all the size query needs
    const size_t used = plan_host_call(hl, lay, &dev->layer, dlink, copies, nc, o_bytes, h.first != 0);
    dev->layer.links = dlink;
    if (!h.first) { dev->layer.q0 = lisa_tensor{}; dev->layer.k0 = lisa_tensor{}; }
    size_t ws = 0;
    if ((st = lisa_workspace_bytes(LISA_OP_SHARED_PREFILL_CARRY, dev, &ws)) != LISA_OK) return st;
    dev->layer.workspace = ws ? lay + used : nullptr;
    dev->layer.workspace_bytes = ws;
    *total = used + ((ws + 255) & ~(size_t)255);
    return LISA_OK;
}
}  // namespace

lisa_status_t lisa_carry_host_arena_bytes(const lisa_shared_prefill_carry_args* host_args, size_t* bytes) {
    if (!host_args || !bytes) return LISA_ERR_INVALID_ARG;
    lisa_shared_prefill_carry_args dev;
    lisa_link dlink[1];
    Copy copies[3 + 6];
    int nc = 0;
    size_t ob = 0;
    return plan_carry_host(*host_args, nullptr, &dev, dlink, copies, &nc, &ob, bytes);
}

lisa_status_t lisa_attn_shared_prefill_carry_host(const lisa_shared_prefill_carry_args* host_args, void* device_arena, size_t arena_bytes,
                                                  lisa_stream_t stream) {
    if (!host_args) return LISA_ERR_INVALID_ARG;
    if (!device_arena || (reinterpret_cast<uintptr_t>(device_arena) & 255u)) return LISA_ERR_WORKSPACE;
    lisa_shared_prefill_carry_args dev;
    lisa_link dlink[1];
    Copy copies[3 + 6];
    int nc = 0;
    size_t o_bytes = 0, need = 0;
    lisa_status_t st = plan_carry_host(*host_args, static_cast<char*>(device_arena), &dev, dlink, copies, &nc, &o_bytes, &need);
    if (st != LISA_OK) return st;
    if (arena_bytes < need) return LISA_ERR_WORKSPACE;
    // everything that can refuse the call is checked before the first copy is enqueued
    lisa_shared_prefill_args checked;
    if ((st = carried_layer(dev, &checked)) != LISA_OK) return st;
    if (!dev.scores || (reinterpret_cast<uintptr_t>(dev.scores) & 255u) || dev.scores_bytes < tc_carry_bytes(checked.B, checked.N, checked.Hq))
        return LISA_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    TcHostIO ho{host_args->layer.o.ptr, nullptr, nullptr, nullptr, false};
    for (int i = 0; i < nc; ++i) {
        if (copies[i].streamed == 1) ho.host_q0 = copies[i].src;
        else if (copies[i].streamed == 2) ho.host_k0 = copies[i].src;
        else if (copies[i].streamed == 3) ho.host_v = copies[i].src;
        else if ((e = cudaMemcpyAsync(copies[i].dst, copies[i].src, copies[i].bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess)
            return cuda_fail(e);
    }
    if ((st = shared_prefill_carry_impl(&dev, stream, &ho)) != LISA_OK) return st;
    if (!ho.out_done && (e = cudaMemcpyAsync(host_args->layer.o.ptr, dev.layer.o.ptr, o_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(e);
    return LISA_OK;
}

}  // extern "C"
