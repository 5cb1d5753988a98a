// Shared device/host helpers of the LiSA CUDA library: tensor views, element loads, status word.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lisa.h"
#include "lisa_debug.h"

namespace lisa {

constexpr int kMaxHeads = 64;
constexpr int kMaxHidden = 256;
constexpr int kMaxChain = 8;
constexpr int kMaxRank = 32;

// Strided view of [B, N, H, x] passed by value to kernels.
struct TView {
    const void* ptr;
    int64_t sb, sn, sh;
    int32_t dtype;
};

inline TView make_view(const lisa_tensor& t) { return TView{t.ptr, t.stride_b, t.stride_n, t.stride_h, t.dtype}; }

// Aligner FFN of one link, by value.
struct LinkDev {
    TView qp, kp;
    const void *w1, *b1, *w2, *b2;
    int32_t w_dtype, r, m, act, integrate, ffn_layers;
};

inline LinkDev make_link(const lisa_link& l) {
    return LinkDev{make_view(l.qp), make_view(l.kp), l.w1, l.b1, l.w2, l.b2, l.w_dtype, l.r, l.m, l.act, l.integrate,
                   l.ffn_layers};
}

__device__ __forceinline__ float ld_elem(const void* p, int64_t idx, int dtype) {
    if (dtype == LISA_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[idx]);
    return reinterpret_cast<const float*>(p)[idx];
}

__device__ __forceinline__ void st_elem(void* p, int64_t idx, int dtype, float v) {
    if (dtype == LISA_BF16)
        reinterpret_cast<__nv_bfloat16*>(p)[idx] = __float2bfloat16_rn(v);
    else
        reinterpret_cast<float*>(p)[idx] = v;
}

__device__ __forceinline__ float act_apply(float x, int act) {
    if (act == LISA_ACT_RELU) return fmaxf(x, 0.f);
    if (act == LISA_ACT_SILU) return x / (1.f + __expf(-x));
    return x;
}

// Device status words (this device's copy): [0] cache appends dropped, [1] bounded waits that ran out.
// Host function; returns the device address to hand to kernels, or nullptr if the lookup failed.
int* status_words();

// Streaming multiprocessors of the current device (cached per device; 1 if the query fails).
int sm_count();

// Adds n to the process-wide count of kernels enqueued by the library.
void count_launches(int n);

// Host-side launchers implemented in the .cu files. Each returns the cudaError_t of its launches.
cudaError_t launch_generic_prefill(const lisa_shared_prefill_args& a, cudaStream_t s);

cudaError_t launch_shared_decode(const lisa_shared_decode_args& a, void* ws, cudaStream_t s);
cudaError_t launch_anchor_decode(const lisa_anchor_args& a, void* ws, cudaStream_t s);
size_t decode_workspace(int B, int Hq, int d, int L);
size_t shared_decode_smem(int Hq, int m, int integrate);   // dynamic shared memory the shared-layer decode kernel asks for

// Tensor-core flash kernel (head width 128, bf16): O = softmax_causal(QA.KA^T * scale [+ plane]) . V for query tiles
// [qt_begin, qt_begin + qt_count).  qa [B,N,Hq,kd], ka [B,N,Hkv,kd] with kd in {64,128}; plane (optional) holds
// bf16 blocked [rows/128][cols/64][128][B*Hq][64] pre-computed scores for query rows qt_begin*128 onwards.
struct TcFlashArgs {
    int B, N, Hq, Hkv, kd;
    lisa_tensor qa, ka, v, o;
    float scale;
    const void* plane;
    int64_t plane_rows, plane_cols;
    int qt_begin, qt_count;
    // emit_plane != nullptr: no attention; the scaled scores of the covered tiles are written there as bf16
    // (blocked [rows/128][cols/64][128][B*Hq][64], rows relative to qt_begin*128); v, o and plane are then ignored.
    void* emit_plane = nullptr;
    int ksteps = 0;  // 16-wide k-steps to issue (0 = kd/16); the columns beyond are zero padding
    // carry != nullptr (with plane): the finished pre-softmax logits (scores * scale + plane, unmasked, fp16) of the covered
    // tiles are written there, same blocked layout and geometry as plane; may be the plane itself (each tile is stored
    // after it was read).
    void* carry = nullptr;
    int plane_row0 = -1;  // first query row the plane / emit_plane / carry buffers hold (-1: qt_begin * 128)
};
bool tc_flash_supported(const TcFlashArgs& a);
cudaError_t launch_tc_flash(const TcFlashArgs& a, cudaStream_t s);

// Tensor-core aligner: applies the FFN chain of links[0..chain) to the score planes in place (see tc_align.cu).
// planes[0] = A_0 in / Y out, planes[k] = D_k (already scaled) for k = 1..chain-1; all blocked [rows/128][cols/64][128][B*32][64].
struct TcAlignArgs {
    int B, N, chain, qt_begin, qt_count;
    int64_t plane_rows, plane_cols;
    void* planes[4];
    const lisa_link* links;
    int ctas = 0;  // grid size (0 = three per SM)
    int row0 = -1;  // first query row the planes hold (-1: qt_begin * 128)
    bool store_all = false;  // every link's output is stored (times log2 e): link k (0-based) into planes[k]
};
bool tc_align_supported(int Hq, const lisa_link* links, int chain);
cudaError_t launch_tc_align(const TcAlignArgs& a, cudaStream_t s);

// Tensor-core aligner, one link per launch (tc_align_link.cu): the concatenating Integrate at 32 heads, and the adding forms
// at 32 or 40 heads with a hidden layer of up to 256 units.  Reads plane_x = the link's input scores and plane_d = D_k
// (adding forms: may be null, then nothing is added); writes the next link's input (unscaled; the adding forms include
// D_k) and/or log2(e) times the FFN's output, each over plane_x (0) or plane_d (1), or nowhere (-1).
struct TcAlignLinkArgs {
    int B, N, Hq, qt_begin, qt_count;
    int64_t plane_rows, plane_cols;
    void *plane_x, *plane_d;
    const lisa_link* link;
    int dst_next, dst_scaled;
    int row0 = -1;  // first query row the planes hold (-1: qt_begin * 128)
    // plane_d with a geometry of its own (0 / -1: the same as plane_x): carried scores as plane_x, a wave's plane as plane_d
    int64_t d_plane_rows = 0, d_plane_cols = 0;
    int d_row0 = -1;
};
bool tc_align_concat_supported(int Hq, const lisa_link* links, int chain);
bool tc_align_link_supported(int Hq, const lisa_link* links, int chain);
cudaError_t launch_tc_align_link(const TcAlignLinkArgs& a, cudaStream_t s);

// Programmatic dependent launch for chains of short kernels (the decode step: append, chunk, merge, layer after layer):
// a kernel launched with launch_chained may start while its predecessor in the stream is still running; it must call
// chain_wait() before it touches anything an earlier kernel wrote or still reads (what it does before -- staging constant
// weights -- overlaps the predecessor's tail), and calls chain_release() early so that its own successor can be set up.
// chain_wait() returns once the predecessor has completed and its writes are visible; as every kernel of such a chain
// waits before it finishes, completion is transitive.  In a kernel launched the ordinary way both are no-ops.
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename Params>
cudaError_t launch_chained(void (*kernel)(Params), dim3 grid, dim3 block, size_t smem, cudaStream_t s, const Params& p) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

// Packs Q' or K' ([B,N,H,r], any strides) into zero-padded bf16 [B][H][N][64] rows for the tensor-core kernels.
cudaError_t launch_pack_lowrank(const lisa_tensor& src, int B, int N, int H, int r, void* dst, cudaStream_t s);

// Tensor-core prefill of a shared layer (tc_prefill.cu): emit planes -> align -> attention, wave by wave.
bool tc_shared_prefill_supported(const lisa_shared_prefill_args& a);
size_t tc_shared_prefill_workspace(const lisa_shared_prefill_args& a);
// Carried scores (lisa_attn_shared_prefill_carry): the chain's running scores A_n of the whole prompt live in a caller's
// buffer, blocked like the planes with N rounded up to 128 in both directions.  With `carry` set, a one-link call works
// in place on that buffer: `first` emits A_0 there, the aligner runs over it, and the attention kernel writes A_n back
// when `keep`.
struct TcCarry {
    void* scores;
    bool first, keep;
};
// Host-memory entry points: q0, k0, v (each may be null: nothing to bring in) and o live in host memory, dense [B,N,H,d]
// like their device copies in the arena.  The tensor-core path streams them: before a wave starts, its rows of q0, k0
// and v are copied in on a stream of the library's own (a wave needs the keys and values up to its last row, and the
// waves run from row 0 up); after the wave's attention kernel its rows of o are copied out on another; both are joined
// into the caller's stream at the end.  out_done is set when the output copies were enqueued; otherwise the caller
// copies o itself.  Whoever launches the layer's kernels brings the inputs in first (whole tensors where not streamed).
struct TcHostIO {
    void* host_o;
    const void *host_q0, *host_k0, *host_v;
    bool out_done;
};
size_t tc_carry_bytes(int B, int N, int Hq);
size_t tc_shared_prefill_carry_workspace(const lisa_shared_prefill_args& a);
cudaError_t launch_tc_shared_prefill(const lisa_shared_prefill_args& a, void* ws, cudaStream_t s);
// vs/os: per-layer V and O of a chain of a.chain_len layers (nullptr: only the deepest layer, a.v / a.o)
cudaError_t launch_tc_shared_prefill_chain(const lisa_shared_prefill_args& a, const lisa_tensor* vs, const lisa_tensor* os, void* ws,
                                           cudaStream_t s, const TcCarry* carry = nullptr, TcHostIO* host_io = nullptr);
cudaError_t prefill_phase_timing(bool enable);
cudaError_t prefill_phase_times(float* ms4);

// Projection GEMM (tc_project.cu): tensor-core kernel for aligned bf16, general kernel otherwise.
bool tc_project_supported(const lisa_project_args& a);
cudaError_t launch_tc_project(const lisa_project_args& a, cudaStream_t s);
cudaError_t launch_generic_project(const lisa_project_args& a, cudaStream_t s);

cudaError_t launch_kvcache_append(const lisa_kvcache_layer& c, const lisa_tensor& k, const lisa_tensor& v,
                                  const int32_t* lens_before, int n_new, cudaStream_t s);

}  // namespace lisa
