// Tensor-core prefill of a shared layer (Sec. 5.1, Eq. 3-4, then Eq. 1): host-side orchestration.
//
// The aligner mixes all heads at one (query, key) position while softmax.V needs one running output per
// head, so the layer runs as three tensor-core kernels that exchange fp16 score planes [row][head][col]
// through a workspace sized to stay in L2, one wave of query tiles at a time:
//   1. tc_flash (emit)   A_0 = Q0.K0^T/sqrt(d) per head, and D_k = Q'_k.K'_k^T/sqrt(r) for the links k < c
//   2. tc_align          per position: the FFN chain over the head axis, Y written over A_0
//   3. tc_flash (plane)  per head: logits = Y + Q'_c.K'_c^T/sqrt(r), causal softmax, .V
// The recomputing calls store only the wave's strip of rows of the N x N x Hq scores; the carried call keeps the whole
// prompt's scores in the caller's buffer and works in place on it (see launch_tc_shared_prefill_chain).
#include <algorithm>
#include <cmath>
#include <mutex>

#include "common.cuh"

namespace lisa {
namespace {

constexpr int kTile = 128;
constexpr int kPadRank = 64;
constexpr int kMaxPackLinks = 4;   // links whose Q', K' one call packs (the aligner takes chains of up to three)
// A wave takes query tiles until its head-partitioned kernels have at least kWaveCtasPerSm CTAs per SM (with
// fewer, the grids do not fill the GPU and launch and tail costs dominate) and then further tiles while the causal
// part of its score planes stays within kWaveBytes.  Measured on B200: grid fill matters far more than keeping
// the planes inside the 126 MB L2.
constexpr size_t kWaveBytes = (size_t)256 << 20;
constexpr int kWaveCtasPerSm = 4;

// Every Q' and K' of a call is packed by one launch: blockIdx.y selects the tensor.
struct PackJobs {
    TView src[2 * kMaxPackLinks];
    __nv_bfloat16* dst[2 * kMaxPackLinks];
    int H[2 * kMaxPackLinks], r[2 * kMaxPackLinks];
};

__global__ void pack_lowrank_kernel(const __grid_constant__ PackJobs jobs, int B, int N) {
    const TView src = jobs.src[blockIdx.y];
    const int H = jobs.H[blockIdx.y], r = jobs.r[blockIdx.y];
    __nv_bfloat16* dst = jobs.dst[blockIdx.y];
    const int64_t total = (int64_t)B * H * N * (kPadRank / 8);
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int chunk = (int)(e % (kPadRank / 8));
        int64_t rest = e / (kPadRank / 8);
        const int n = (int)(rest % N); rest /= N;
        const int h = (int)(rest % H);
        const int b = (int)(rest / H);
        const __nv_bfloat16* sp = reinterpret_cast<const __nv_bfloat16*>(src.ptr) + b * src.sb + (int64_t)n * src.sn + h * src.sh;
        __align__(16) __nv_bfloat16 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int x = chunk * 8 + j;
            v[j] = x < r ? sp[x] : __float2bfloat16_rn(0.f);
        }
        *reinterpret_cast<uint4*>(dst + e * 8) = *reinterpret_cast<const uint4*>(v);
    }
}

// Optional per-phase timing of the tensor-core prefill (lisa_prefill_phase_timing): CUDA events recorded on the
// caller's stream around each internal kernel, summed per phase when read.  Off by default.
constexpr int kPhases = 4;       // 0 pack, 1 emit score planes, 2 aligner, 3 attention
constexpr int kMaxMarks = 2048;
struct PhaseTimer {
    bool on = false;
    int n = 0;
    cudaEvent_t ev[2 * kMaxMarks];
    int phase[kMaxMarks];
} g_pt;

struct PhaseMark {
    cudaStream_t s;
    int idx;
    PhaseMark(int phase, cudaStream_t stream) : s(stream), idx(-1) {
        if (g_pt.on && g_pt.n < kMaxMarks) {
            idx = g_pt.n++;
            g_pt.phase[idx] = phase;
            cudaEventRecord(g_pt.ev[2 * idx], s);
        }
    }
    ~PhaseMark() {
        if (idx >= 0) cudaEventRecord(g_pt.ev[2 * idx + 1], s);
    }
};

struct Wave { int begin, count; };

// carried: the scores live in the caller's buffer, a wave has no planes of its own and its size is free
int plan_waves(int B, int N, int Hq, int c, Wave* waves, int max_waves, bool carried = false) {
    const int min_ctas = kWaveCtasPerSm * sm_count();
    const int n_qt = (N + kTile - 1) / kTile;
    const size_t per_col_tile = (size_t)B * Hq * kTile * kTile * 2 * c;
    int n = 0, qt = 0;
    while (qt < n_qt) {
        size_t bytes = 0;
        int cnt = 0;
        while (qt + cnt < n_qt && (B * Hq * cnt < min_ctas || bytes + per_col_tile * (qt + cnt + 1) <= kWaveBytes)) {
            bytes += per_col_tile * (qt + cnt + 1);
            ++cnt;
        }
        // The head-partitioned kernels run one CTA per (batch, head, query tile), two per SM at a time, and the CTAs of a wave
        // weigh about the same: a wave of 2.2 rounds of CTAs takes as long as one of 3.  Tiles are added (while the planes,
        // where the wave has any, stay within four times the budget) until the last round is at least nine tenths full, or the best fill found is taken.
        {
            const int64_t slots = 2 * (int64_t)sm_count();
            auto fill = [&](int k) { const int64_t n = (int64_t)B * Hq * k; return (double)n / (double)(((n + slots - 1) / slots) * slots); };
            int best = cnt;
            size_t grow = bytes;
            for (int k = cnt; qt + k <= n_qt && k <= cnt + 16; ++k) {
                if (k > cnt) { grow += per_col_tile * (qt + k); if (!carried && grow > 4 * kWaveBytes) break; }
                if (fill(k) > fill(best) + 1e-9) best = k;
                if (fill(k) >= 0.9) { best = k; break; }
            }
            cnt = best;
        }
        if (waves && n < max_waves) waves[n] = Wave{qt, cnt};
        ++n;
        qt += cnt;
    }
    return n;
}

// The concatenating Integrate feeds every link's difference to its FFN as a plane of its own, the top link's included:
// one plane more than the adding forms, where the attention kernel adds the top link's difference itself.
bool concat_chain(const lisa_shared_prefill_args& a) { return a.chain_len > 0 && a.links[0].integrate == LISA_INTEGRATE_CONCAT; }
int plane_count(const lisa_shared_prefill_args& a) { return a.chain_len + (concat_chain(a) ? 1 : 0); }

// Waves are independent of one another, and the three kernels of a wave stress different things (the emit kernel only
// writes HBM, the attention kernel mostly reads it, the aligner is bound by its MMA rate), so up to kWaveSets waves are
// in flight at a time, each on a stream and a set of planes of its own: wave w uses set w % sets, and set reuse is
// ordered by the stream the set belongs to.
constexpr int kWaveSets = 3;

struct Layout {
    size_t qp_off[kMaxChain], kp_off[kMaxChain], plane_off[kWaveSets][kMaxChain + 1];
    int64_t plane_rows, plane_cols;
    int sets;
    size_t total;
};

// carried: the scores live in the caller's buffer; the workspace holds the packed Q', K' and, for the concatenating
// Integrate, the wave's plane of the link's difference
Layout plan_layout(const lisa_shared_prefill_args& a, bool carried = false) {
    Layout l{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 1023) & ~(size_t)1023; return o; };
    for (int k = 0; k < a.chain_len; ++k) {
        l.qp_off[k] = take((size_t)a.B * a.Hq * a.N * kPadRank * 2);
        l.kp_off[k] = take((size_t)a.B * a.Hkv * a.N * kPadRank * 2);
    }
    const int n_qt = (a.N + kTile - 1) / kTile;
    Wave waves[1024];
    const int nw = plan_waves(a.B, a.N, a.Hq, carried ? 1 : plane_count(a), waves, 1024, carried && !concat_chain(a));
    int max_cnt = 1;
    for (int i = 0; i < std::min(nw, 1024); ++i) max_cnt = std::max(max_cnt, waves[i].count);
    l.plane_rows = (int64_t)max_cnt * kTile;
    l.plane_cols = (int64_t)n_qt * kTile;
    l.sets = std::max(1, std::min(kWaveSets, nw));
    for (int set = 0; set < l.sets; ++set)
        for (int k = 0; k < plane_count(a); ++k)
            if (!carried || (concat_chain(a) && k == 1)) l.plane_off[set][k] = take((size_t)a.B * a.Hq * l.plane_rows * l.plane_cols * 2);
    l.total = off;
    return l;
}

lisa_tensor packed_view(void* ptr, int H, int N) {
    return lisa_tensor{ptr, LISA_BF16, 0, (int64_t)H * N * kPadRank, (int64_t)kPadRank, (int64_t)N * kPadRank};
}

}  // namespace

cudaError_t launch_pack_lowrank(const lisa_tensor& src, int B, int N, int H, int r, void* dst, cudaStream_t s) {
    PackJobs jobs{};
    jobs.src[0] = make_view(src); jobs.dst[0] = reinterpret_cast<__nv_bfloat16*>(dst); jobs.H[0] = H; jobs.r[0] = r;
    const int64_t total = (int64_t)B * H * N * (kPadRank / 8);
    const int blocks = (int)std::min<int64_t>((total + 255) / 256, sm_count() * 32);
    pack_lowrank_kernel<<<dim3(blocks, 1), 256, 0, s>>>(jobs, B, N);
    count_launches(1);
    return cudaGetLastError();
}

bool tc_shared_prefill_supported(const lisa_shared_prefill_args& a) {
    if (a.d != 128 || a.chain_len < 1 || a.N > kTile * 1024) return false;
    if (!tc_align_supported(a.Hq, a.links, a.chain_len) && !tc_align_concat_supported(a.Hq, a.links, a.chain_len) &&
        !tc_align_link_supported(a.Hq, a.links, a.chain_len))
        return false;
    for (int k = 0; k < a.chain_len; ++k)
        if (a.links[k].qp.dtype != LISA_BF16 || a.links[k].kp.dtype != LISA_BF16 || a.links[k].r > 32) return false;
    TcFlashArgs f{a.B, a.N, a.Hq, a.Hkv, 128, a.q0, a.k0, a.v, a.o, 1.f, nullptr, 0, 0, 0, 1};
    return tc_flash_supported(f);
}

// + 1024: the launch aligns the caller's pointer up to the 1024 bytes the swizzled tiles need
size_t tc_shared_prefill_workspace(const lisa_shared_prefill_args& a) { return plan_layout(a).total + 1024; }
size_t tc_shared_prefill_carry_workspace(const lisa_shared_prefill_args& a) { return plan_layout(a, true).total + 1024; }
size_t tc_carry_bytes(int B, int N, int Hq) {
    const size_t n = (size_t)(N + kTile - 1) / kTile * kTile;
    return (size_t)B * Hq * n * n * 2;
}

namespace {
// The packing of Q'/K' feeds only the kernels that come after the first emit (the attention kernel; the emits of the
// differences of deeper chains), so it runs beside that emit on a stream of the library's own: forked from the
// caller's stream with one event and joined with another before its first consumer.  One stream and one event pair
// per device, created on first use; the fork and the join are each enqueued under a lock, so calls from several host
// threads cannot pair one call's wait with another call's record.
struct SideStream {
    cudaStream_t stream = nullptr;                 // packing of Q'/K'
    cudaEvent_t fork = nullptr, join = nullptr;
    cudaStream_t wave[kWaveSets - 1] = {};         // waves beside the caller's stream
    cudaEvent_t wave_done[kWaveSets - 1] = {};
    cudaStream_t copy_out = nullptr, copy_in = nullptr;   // host-memory entry points: finished rows out, the next wave's rows in
    cudaEvent_t rows_done = nullptr, copy_done = nullptr, rows_in = nullptr;
    bool ok = false;
};
SideStream g_side[64];
std::mutex g_side_mutex;

SideStream* side_stream() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    SideStream& ss = g_side[dev];
    if (!ss.ok) {
        if (cudaStreamCreateWithFlags(&ss.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&ss.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&ss.join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        for (int i = 0; i < kWaveSets - 1; ++i) {
            if (cudaStreamCreateWithFlags(&ss.wave[i], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
            if (cudaEventCreateWithFlags(&ss.wave_done[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        }
        if (cudaStreamCreateWithFlags(&ss.copy_out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&ss.rows_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&ss.copy_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithFlags(&ss.copy_in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&ss.rows_in, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        ss.ok = true;
    }
    return &ss;
}

// The host-memory entry points hand q0, k0, v (host, each may be null) and o (host) to the orchestration (TcHostIO).
// Where the side streams exist and the device copies are dense, the tensors are streamed: before a wave starts, its rows of
// q0, k0 and v are copied in on the copy-in stream (the waves run from row 0 up, and a wave needs keys and values up to
// its last row: exactly what has been copied by then) and the wave's stream waits for them; after the wave's attention
// kernel its rows of o go out on the copy-out stream.  Otherwise the inputs are copied whole on the caller's stream
// before anything reads them, and the caller copies o afterwards (out_done stays false).
struct HostIo {
    const lisa_shared_prefill_args& a;
    TcHostIO* ho;
    SideStream* side;
    cudaStream_t s;
    bool stream_out = false, stream_in = false;

    HostIo(const lisa_shared_prefill_args& args, TcHostIO* io, SideStream* ss, cudaStream_t caller, bool one_layer)
        : a(args), ho(io), side(ss), s(caller) {
        auto dense = [&](const lisa_tensor& t, int H) {
            return t.stride_h == a.d && t.stride_n == (int64_t)H * a.d && t.stride_b == (int64_t)a.N * H * a.d;
        };
        stream_out = ho && ho->host_o && side && one_layer && dense(a.o, a.Hq);
        stream_in = has_in() && stream_out && dense(a.q0, a.Hq) && dense(a.k0, a.Hkv) && dense(a.v, a.Hkv);
    }
    bool has_in() const { return ho && (ho->host_q0 || ho->host_k0 || ho->host_v); }
    // rows [r0, r1) of a dense [B,N,H,d] bf16 tensor, one copy per sequence
    cudaError_t copy_rows(void* dst, const void* src, int H, int64_t r0, int64_t r1, cudaMemcpyKind kind, cudaStream_t cs) const {
        for (int b = 0; b < a.B; ++b) {
            const int64_t off = ((int64_t)b * a.N + r0) * H * a.d * 2;
            cudaError_t e = cudaMemcpyAsync(static_cast<char*>(dst) + off, static_cast<const char*>(src) + off,
                                            (size_t)(r1 - r0) * H * a.d * 2, kind, cs);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    }
    cudaError_t inputs(int64_t r0, int64_t r1, cudaStream_t cs) const {
        cudaError_t e;
        if (ho->host_q0 && (e = copy_rows(a.q0.ptr, ho->host_q0, a.Hq, r0, r1, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return e;
        if (ho->host_k0 && (e = copy_rows(a.k0.ptr, ho->host_k0, a.Hkv, r0, r1, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return e;
        if (ho->host_v && (e = copy_rows(a.v.ptr, ho->host_v, a.Hkv, r0, r1, cudaMemcpyHostToDevice, cs)) != cudaSuccess) return e;
        return cudaSuccess;
    }
    // before the first kernel: whole inputs where they are not streamed; the copy-in stream ordered behind everything
    // enqueued before the call (earlier users of the arena) where they are
    cudaError_t begin() const {
        if (has_in() && !stream_in) return inputs(0, a.N, s);
        if (!stream_in) return cudaSuccess;
        std::lock_guard<std::mutex> lock(g_side_mutex);
        cudaError_t e = cudaEventRecord(side->fork, s);
        return e != cudaSuccess ? e : cudaStreamWaitEvent(side->copy_in, side->fork, 0);
    }
    static void rows_of(const Wave& wv, int N, int64_t* r0, int64_t* r1) {
        *r0 = (int64_t)wv.begin * kTile;
        *r1 = std::min<int64_t>(N, (int64_t)(wv.begin + wv.count) * kTile);
    }
    cudaError_t rows_in(const Wave& wv, cudaStream_t st) const {
        int64_t r0, r1;
        rows_of(wv, a.N, &r0, &r1);
        cudaError_t e = inputs(r0, r1, side->copy_in);
        if (e != cudaSuccess) return e;
        if ((e = cudaEventRecord(side->rows_in, side->copy_in)) != cudaSuccess) return e;
        return cudaStreamWaitEvent(st, side->rows_in, 0);   // everything copied so far: the wave's rows and all rows before them
    }
    cudaError_t rows_out(const Wave& wv, cudaStream_t st) const {
        int64_t r0, r1;
        rows_of(wv, a.N, &r0, &r1);
        cudaError_t e = cudaEventRecord(side->rows_done, st);
        if (e != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(side->copy_out, side->rows_done, 0)) != cudaSuccess) return e;
        return copy_rows(ho->host_o, a.o.ptr, a.Hq, r0, r1, cudaMemcpyDeviceToHost, side->copy_out);
    }
};
}  // namespace

cudaError_t launch_tc_shared_prefill(const lisa_shared_prefill_args& a, void* ws, cudaStream_t s) {
    return launch_tc_shared_prefill_chain(a, nullptr, nullptr, ws, s);
}

// With vs/os == nullptr: the layer at chain depth c (a.v, a.o).  With vs/os[c]: all c layers of the chain in one
// pass -- the anchor scores and the differences are emitted once, the aligner stores every link's output (link k
// over plane k), and one attention kernel per layer consumes its plane with its own Q', K' and V.
// With cy: one link, in place on the caller's carried scores (rows from 0, N rounded up to whole tiles both ways): no A_0
// unless this is the first layer of its chain, no wave planes, and the attention kernel leaves A_n behind when asked.
cudaError_t launch_tc_shared_prefill_chain(const lisa_shared_prefill_args& a, const lisa_tensor* vs, const lisa_tensor* os, void* ws,
                                           cudaStream_t s, const TcCarry* cy, TcHostIO* ho) {
    const bool all_layers = vs != nullptr;
    if (ho) ho->out_done = false;
    if (cy && (all_layers || a.chain_len != 1 || !cy->scores)) return cudaErrorInvalidValue;
    const Layout l = plan_layout(a, cy != nullptr);
    // geometry of the plane that holds the running scores: the caller's buffer (whole prompt, rows from 0) or a wave's plane
    const int64_t x_rows = cy ? (int64_t)(a.N + kTile - 1) / kTile * kTile : l.plane_rows, x_cols = cy ? x_rows : l.plane_cols;
    char* const plane_base = cy ? reinterpret_cast<char*>(cy->scores) : nullptr;
    const int row0 = cy ? 0 : -1;
    char* base = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(ws) + 1023) & ~(uintptr_t)1023);
    const int c = a.chain_len;
    cudaError_t e;
    SideStream* side = nullptr;
    {
        PhaseMark mark(0, s);
        PackJobs jobs{};
        for (int k = 0; k < c; ++k) {
            jobs.src[2 * k] = make_view(a.links[k].qp); jobs.dst[2 * k] = reinterpret_cast<__nv_bfloat16*>(base + l.qp_off[k]);
            jobs.H[2 * k] = a.Hq; jobs.r[2 * k] = a.links[k].r;
            jobs.src[2 * k + 1] = make_view(a.links[k].kp); jobs.dst[2 * k + 1] = reinterpret_cast<__nv_bfloat16*>(base + l.kp_off[k]);
            jobs.H[2 * k + 1] = a.Hkv; jobs.r[2 * k + 1] = a.links[k].r;
        }
        const int64_t total = (int64_t)a.B * a.Hq * a.N * (kPadRank / 8);
        const int blocks = (int)std::min<int64_t>((total + 255) / 256, sm_count() * 16);
        // beside the first emit, unless the per-kernel timing is on (then every kernel is timed on the caller's stream)
        if (!g_pt.on) {
            std::lock_guard<std::mutex> lock(g_side_mutex);
            side = side_stream();
            if (side) {
                if ((e = cudaEventRecord(side->fork, s)) != cudaSuccess) return e;
                if ((e = cudaStreamWaitEvent(side->stream, side->fork, 0)) != cudaSuccess) return e;
                pack_lowrank_kernel<<<dim3(blocks, 2 * c), 256, 0, side->stream>>>(jobs, a.B, a.N);
                if ((e = cudaGetLastError()) != cudaSuccess) return e;
                if ((e = cudaEventRecord(side->join, side->stream)) != cudaSuccess) return e;
            }
        }
        if (!side) pack_lowrank_kernel<<<dim3(blocks, 2 * c), 256, 0, s>>>(jobs, a.B, a.N);
        count_launches(1);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    bool joined = side == nullptr;
    auto join_pack = [&]() -> cudaError_t {   // before the first kernel that reads the packed Q'/K'
        if (joined) return cudaSuccess;
        joined = true;
        std::lock_guard<std::mutex> lock(g_side_mutex);
        return cudaStreamWaitEvent(s, side->join, 0);
    };
    const bool concat = concat_chain(a);
    Wave waves[1024];
    int nw = plan_waves(a.B, a.N, a.Hq, cy ? 1 : plane_count(a), waves, 1024, cy != nullptr && !concat);
    // A host-memory call whose prompt fits fewer than four waves is cut into four strips of query tiles all the same (they
    // run one after the other in the planes laid out for the larger waves): its time is the copies', and strips let the
    // copies in, the compute and the copies out overlap.
    if (ho && side && !all_layers && nw < 4) {
        const int n_qt = (a.N + kTile - 1) / kTile, per = (n_qt + 3) / 4;
        if (n_qt >= 4) {
            nw = 0;
            for (int qt = 0; qt < n_qt; qt += per) waves[nw++] = Wave{qt, std::min(per, n_qt - qt)};
        }
    }
    // Several waves in flight (see kWaveSets): wave w runs on stream w % sets (0 = the caller's) with plane set w % sets.
    // All of it is forked from and joined back into the caller's stream inside this call, under the lock that keeps
    // another host thread's call from interleaving its event records with these waits.
    const int sets = (side && nw >= 2) ? std::min(l.sets, nw) : 1;
    // host-memory calls: inputs in and output out wave by wave beside the compute (see HostIo), where the path allows it
    HostIo io{a, ho, side, s, !all_layers};
    const bool stream_out = io.stream_out, stream_in = io.stream_in;
    if ((e = io.begin()) != cudaSuccess) return e;
    auto copy_in = [&](const Wave& wv, cudaStream_t st) { return io.rows_in(wv, st); };
    auto copy_out = [&](const Wave& wv, cudaStream_t st) { return io.rows_out(wv, st); };
    std::unique_lock<std::mutex> wave_lock(g_side_mutex, std::defer_lock);
    if (sets > 1 || stream_out) {
        wave_lock.lock();
        if ((e = cudaStreamWaitEvent(s, side->join, 0)) != cudaSuccess) return e;   // every wave stream starts with the packed Q'/K' ready
        joined = true;
        if ((e = cudaEventRecord(side->fork, s)) != cudaSuccess) return e;
        for (int i = 0; i + 1 < sets; ++i)
            if ((e = cudaStreamWaitEvent(side->wave[i], side->fork, 0)) != cudaSuccess) return e;
    }
    for (int w = 0; w < nw; ++w) {
        const Wave wv = waves[w];
        const int set = w % sets;
        cudaStream_t st = set == 0 ? s : side->wave[set - 1];
        const size_t* po = l.plane_off[set];
        if (stream_in && (e = copy_in(wv, st)) != cudaSuccess) return e;
        // 1. anchor scores and the differences of the links below the top one
        const TcFlashArgs fw{a.B, a.N, a.Hq, a.Hkv, 128, a.q0, a.k0, a.v, a.o, 1.f / sqrtf((float)a.d), nullptr, l.plane_rows, l.plane_cols,
                             wv.begin, wv.count};                 // the wave's own planes
        TcFlashArgs f = fw;                                       // the plane of the running scores
        f.plane_rows = x_rows; f.plane_cols = x_cols; f.plane_row0 = row0;
        char* const x_plane = cy ? plane_base : base + po[0];
        f.emit_plane = x_plane;
        if (!cy || cy->first) {
            PhaseMark mark(1, st);
            if ((e = launch_tc_flash(f, st)) != cudaSuccess) return e;
        }
        for (int k = 0; k + (concat ? 0 : 1) < c; ++k) {   // the concatenating form also needs the top link's difference as a plane
            if ((e = join_pack()) != cudaSuccess) return e;
            PhaseMark mark(1, st);
            TcFlashArgs fd = fw;
            fd.kd = kPadRank;
            fd.qa = packed_view(base + l.qp_off[k], a.Hq, a.N);
            fd.ka = packed_view(base + l.kp_off[k], a.Hkv, a.N);
            fd.scale = 1.f / sqrtf((float)a.links[k].r);
            fd.ksteps = (a.links[k].r + 15) / 16;
            fd.emit_plane = base + po[k + 1];
            if ((e = launch_tc_flash(fd, st)) != cudaSuccess) return e;
        }
        if (concat) {
            // 2c. link by link: A_k = FFN_k([A_{k-1}; D_k]) over plane 0; log2(e) * A_k over D_k's plane where a layer's
            // attention consumes it (the top link's; every link's when all layers of the chain are computed)
            for (int k = 0; k < c; ++k) {
                // carried: the one link reads A_{n-1} from the caller's buffer and leaves A_n there when asked
                TcAlignLinkArgs ac{a.B, a.N, a.Hq, wv.begin, wv.count, x_rows, x_cols, x_plane, base + po[k + 1],
                                   &a.links[k], (k + 1 < c || (cy && cy->keep)) ? 0 : -1, (all_layers || k == c - 1) ? 1 : -1, row0,
                                   l.plane_rows, l.plane_cols, -1};
                PhaseMark mark(2, st);
                if ((e = launch_tc_align_link(ac, st)) != cudaSuccess) return e;
            }
            // 3c. softmax and .V on the finished scores: the attention kernel's own difference is switched off (scale 0)
            for (int k = all_layers ? 0 : c - 1; k < c; ++k) {
                TcFlashArgs fv = fw;
                fv.kd = kPadRank;
                fv.qa = packed_view(base + l.qp_off[k], a.Hq, a.N);
                fv.ka = packed_view(base + l.kp_off[k], a.Hkv, a.N);
                fv.scale = 0.f;
                fv.ksteps = 1;
                fv.plane = base + po[k + 1];
                if (all_layers) { fv.v = vs[k]; fv.o = os[k]; }
                PhaseMark mark(3, st);
                if ((e = launch_tc_flash(fv, st)) != cudaSuccess) return e;
            }
            if (stream_out && (e = copy_out(wv, st)) != cudaSuccess) return e;
            continue;
        }
        const bool per_link = !tc_align_supported(a.Hq, a.links, c);
        if (per_link) {
            // 2l. shapes the chain kernel does not take (40 heads, wider hidden layers): one launch per link.  Link k reads
            // plane k, writes A_k = FFN_k(A_{k-1}) + D_k over plane k + 1 (which held D_k) and, where a layer's attention
            // consumes it, log2(e) * FFN_k(A_{k-1}) over plane k.
            for (int k = 0; k < c; ++k) {
                TcAlignLinkArgs al{a.B, a.N, a.Hq, wv.begin, wv.count, x_rows, x_cols, cy ? plane_base : base + po[k],
                                   k + 1 < c ? base + po[k + 1] : nullptr, &a.links[k], k + 1 < c ? 1 : -1,
                                   (all_layers || k == c - 1) ? 0 : -1, row0};
                PhaseMark mark(2, st);
                if ((e = launch_tc_align_link(al, st)) != cudaSuccess) return e;
            }
        }
        // 2. the FFN chain over the head axis, in place
        TcAlignArgs al{};
        al.B = a.B; al.N = a.N; al.chain = c; al.qt_begin = wv.begin; al.qt_count = wv.count;
        al.plane_rows = x_rows; al.plane_cols = x_cols;
        for (int k = 0; k < c; ++k) al.planes[k] = cy ? plane_base : base + po[k];
        al.links = a.links;
        al.row0 = row0;
        al.store_all = all_layers;
        if (!per_link) {
            PhaseMark mark(2, st);
            if ((e = launch_tc_align(al, st)) != cudaSuccess) return e;
        }
        // 3. each layer's own difference, softmax and .V
        if ((e = join_pack()) != cudaSuccess) return e;
        for (int k = all_layers ? 0 : c - 1; k < c; ++k) {
            TcFlashArgs fv = f;
            fv.emit_plane = nullptr;
            fv.kd = kPadRank;
            fv.qa = packed_view(base + l.qp_off[k], a.Hq, a.N);
            fv.ka = packed_view(base + l.kp_off[k], a.Hkv, a.N);
            fv.scale = 1.f / sqrtf((float)a.links[k].r);
            fv.ksteps = (a.links[k].r + 15) / 16;
            fv.plane = cy ? plane_base : base + po[all_layers ? k : (per_link ? c - 1 : 0)];
            if (cy && cy->keep) fv.carry = plane_base;
            if (all_layers) { fv.v = vs[k]; fv.o = os[k]; }
            PhaseMark mark(3, st);
            if ((e = launch_tc_flash(fv, st)) != cudaSuccess) return e;
        }
        if (stream_out && (e = copy_out(wv, st)) != cudaSuccess) return e;
    }
    if (stream_out) {
        if ((e = cudaEventRecord(side->copy_done, side->copy_out)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(s, side->copy_done, 0)) != cudaSuccess) return e;
        ho->out_done = true;
    }
    for (int i = 0; i + 1 < sets; ++i) {
        if ((e = cudaEventRecord(side->wave_done[i], side->wave[i])) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(s, side->wave_done[i], 0)) != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t prefill_phase_timing(bool enable) {
    if (enable == g_pt.on) { g_pt.n = 0; return cudaSuccess; }
    if (enable) {
        for (int i = 0; i < 2 * kMaxMarks; ++i) {
            cudaError_t e = cudaEventCreate(&g_pt.ev[i]);
            if (e != cudaSuccess) return e;
        }
    } else {
        for (int i = 0; i < 2 * kMaxMarks; ++i) cudaEventDestroy(g_pt.ev[i]);
    }
    g_pt.on = enable;
    g_pt.n = 0;
    return cudaSuccess;
}

cudaError_t prefill_phase_times(float* ms) {
    for (int i = 0; i < kPhases; ++i) ms[i] = 0.f;
    if (!g_pt.on) return cudaSuccess;
    for (int i = 0; i < g_pt.n; ++i) {
        cudaError_t e = cudaEventSynchronize(g_pt.ev[2 * i + 1]);
        if (e != cudaSuccess) return e;
        float t = 0.f;
        if ((e = cudaEventElapsedTime(&t, g_pt.ev[2 * i], g_pt.ev[2 * i + 1])) != cudaSuccess) return e;
        ms[g_pt.phase[i]] += t;
    }
    g_pt.n = 0;
    return cudaSuccess;
}

}  // namespace lisa
