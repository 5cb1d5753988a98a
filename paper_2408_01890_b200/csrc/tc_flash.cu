// Tensor-core flash kernel (tcgen05 + TMEM + TMA) for head width 128, bf16.
//
// One CTA per (batch b, query head h, 128-row query tile).  For every 64-key tile j up to the diagonal:
//   scores  S = QA . KA^T            tcgen05.mma (M 128, N 64), fp32 accumulator in tensor memory (two buffers, so
//                                    S(t+1) is computed while the softmax of tile t runs)
//   logits  A = S * scale (+ Y)      Y: optional fp16 tile of pre-computed scores (the aligned part of a
//                                    shared layer, Eq. 4; then QA/KA are the layer's low-rank Q'/K', Eq. 3)
//   causal mask (tiles that reach past the first query row), online softmax in registers (one thread per query
//   row), P as bf16
//   O += P . V                       tcgen05.mma (M 128, N 128, K 64), V read MN-major straight from its [key][d] tile
// With QA/KA = Q/K and no Y this is standard attention (Eq. 1-2).  In MODE_EMIT there is no softmax: the scaled
// scores leave as fp16 tiles (staged in shared memory, stored with TMA) for the aligner kernel.  In MODE_ATTN_CARRY the
// attention also writes its finished pre-softmax logits A = S * scale + Y (unmasked, Eq. 4's A_n) back as fp16 tiles: the
// next shared layer of a chain aligns those instead of recomputing the chain from the anchor's scores.
//
// Warp roles: warps 0-3 softmax/epilogue (thread = query row = TMEM lane), warp 4 TMA producer,
// warp 5 issuer of the score MMAs and TMEM owner, warp 6 issuer of the P.V MMAs (warp 7 only completes the warpgroup).  K and V(/Y) have their own rings: a K stage is free again as soon as its
// score MMA has run, a V stage after its P.V MMA.
// Sizing: the softmax warps are the slow stage (one exp2 per score on the 16-lane transcendental unit) and every
// hand-off between the roles costs a few hundred cycles of latency, so TWO CTAs share an SM and fill each other's
// gaps, prologues and epilogues: 64-key tiles keep a CTA at 112 KB of shared memory and 256 tensor-memory columns.
// Every wait is bounded; on expiry the CTA records it in the status word, drains and exits.
#include "common.cuh"
#include "tc_common.cuh"

namespace lisa {
namespace {

using namespace tc;

constexpr int BM = 128, BN = 64, D = 128;

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

constexpr int kPrefetchAhead = 2;   // tiles (0: no L2 prefetch)
constexpr int kThreads = 256;   // warpgroup 0: softmax/epilogue; warpgroup 1: producer, two MMA issuers, one idle warp

struct FlashParams {
    int B, N, Hq, Hkv;
    float scale_log2;  // score scale * log2(e)
    __nv_bfloat16* o;
    int64_t o_sb, o_sn, o_sh;
    int* status;
    int plane_row0;  // first query row held by the plane workspace (rows are stored relative to it)
    int qt_begin;    // this launch covers query tiles [qt_begin, qt_begin + gridDim.y)
    int head_major;  // grid is (query tiles, batch x heads) instead of (batch x heads, query tiles)
    int ksteps;      // 16-wide k-steps of the score MMA actually issued (<= KD/16; the rest is zero padding)
    float scale;     // MODE_EMIT: scores are multiplied by this before rounding to fp16
};

// MODE_ATTN: softmax(QA.KA^T).V;  MODE_ATTN_PLANE: the same with the pre-computed tile Y added to the logits
// (Y arrives already multiplied by log2(e));  MODE_EMIT: no softmax, the scaled scores go to the plane workspace;
// MODE_ATTN_CARRY: MODE_ATTN_PLANE that also stores the logits (divided by log2(e) again) through the fifth tensor map.
constexpr int MODE_ATTN = 0, MODE_ATTN_PLANE = 1, MODE_EMIT = 2, MODE_ATTN_CARRY = 3;

template <int KD, int MODE>
struct Smem {
    static constexpr bool PLANE = MODE == MODE_ATTN_PLANE || MODE == MODE_ATTN_CARRY;
    static constexpr bool EMIT = MODE == MODE_EMIT;
    static constexpr bool CARRY = MODE == MODE_ATTN_CARRY;
    // P (the bf16 probabilities, A operand of P.V) is double-buffered so that the softmax of tile t+1 never waits
    // for the P.V of tile t.  To stay inside half an SM's shared memory it borrows a buffer whose content is dead
    // by then: with a plane, the Y tile of the same stage (each thread has read its own row of Y and overwrites just
    // that row); with 128-wide keys, the K tile of the same stage (its score MMA has completed before the softmax
    // starts), which is then released by the P.V MMA instead of the score MMA -- hence three K stages.  64-wide
    // keys without a plane leave room for two buffers of their own.
    static constexpr bool P_IN_Y = PLANE;
    static constexpr bool P_IN_K = !EMIT && !PLANE && KD == 128;
    static constexpr bool P_OWN = !EMIT && !P_IN_Y && !P_IN_K;
    static constexpr int KST = (EMIT || P_IN_K) ? 3 : 2;  // K ring depth (V/Y: two stages)
    static constexpr int Q_BYTES = BM * KD * 2;
    static constexpr int K_BYTES = BN * KD * 2;
    static constexpr int V_BYTES = EMIT ? 0 : BN * D * 2;
    static constexpr int P_BYTES = BM * BN * 2;
    static constexpr int P_OWN_BYTES = P_OWN ? 2 * P_BYTES : 0;
    static constexpr int Y_BYTES = PLANE ? BM * BN * 2 : 0;
    // per epilogue warp: two buffers of [32 rows][128 B] (emit), one (carry)
    static constexpr int STG_BYTES = EMIT ? 4 * 2 * 4096 : (CARRY ? 4 * 4096 : 0);
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + Q_BYTES;
    static constexpr int OFF_V = OFF_K + KST * K_BYTES;
    static constexpr int OFF_P = OFF_V + 2 * V_BYTES;
    static constexpr int OFF_Y = OFF_P + P_OWN_BYTES;
    static constexpr int OFF_STG = OFF_Y + 2 * Y_BYTES;
    static constexpr int OFF_BAR = OFF_STG + STG_BYTES;
    static constexpr int TOTAL = OFF_BAR + 256;
    static constexpr uint32_t TMEM_COLS = EMIT ? 128 : 256;   // S[2]: [0,128), O: [128,256)
    static_assert(TOTAL <= 115712, "two CTAs must fit one SM's shared memory");
    static_assert(!P_IN_K || K_BYTES >= P_BYTES, "P must fit the K stage it borrows");
};

template <int KD, int MODE>
__global__ void __launch_bounds__(kThreads, 2)
tc_flash_kernel(const __grid_constant__ FlashParams p, const __grid_constant__ CUtensorMap tmQ,
                const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmC) {
    using L = Smem<KD, MODE>;
    constexpr bool PLANE = L::PLANE, EMIT = L::EMIT, CARRY = L::CARRY;
    constexpr int KST = L::KST;
    extern __shared__ __align__(1024) uint8_t smem[];
    // 128-byte-swizzled tiles need 1024-byte aligned bases; the dynamic window starts on such a boundary (there is no
    // static shared memory in this kernel).  Should that ever not hold, refuse loudly instead of computing garbage.
    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicAdd(p.status + 1, 1);
        return;
    }
    uint8_t* sQ = smem + L::OFF_Q;
    uint8_t* sK = smem + L::OFF_K;
    uint8_t* sV = smem + L::OFF_V;
    uint8_t* sP = smem + L::OFF_P;
    uint8_t* sY = smem + L::OFF_Y;
    uint8_t* sStg = smem + L::OFF_STG;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    uint64_t* q_full = bars + 0;
    uint64_t* k_full = bars + 1;    // [KST <= 3]
    uint64_t* k_empty = bars + 4;   // [KST <= 3]
    uint64_t* v_full = bars + 7;    // [2] V and Y of a stage
    uint64_t* v_empty = bars + 9;   // [2]
    uint64_t* s_full = bars + 11;   // [2] score buffer written by the MMA
    uint64_t* s_free = bars + 13;   // [2] score buffer copied to registers by all 128 rows
    uint64_t* p_full = bars + 15;   // [2]
    uint64_t* pv_done = bars + 17;  // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 19);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 20);
    // P of tile t
    auto p_buf = [&](int t) -> uint8_t* {
        if constexpr (L::P_IN_Y) return sY + (t & 1) * L::Y_BYTES;
        else if constexpr (L::P_IN_K) return sK + (t % KST) * L::K_BYTES;
        else return sP + (t & 1) * L::P_BYTES;
    };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // blockIdx.x (the fastest-dispatched index) runs over (batch, head), blockIdx.y over query tiles from the last one
    // down: every CTA of the heaviest tile is handed out before any lighter one, so the SMs finish close together
    // With keys and values too large for L2 to hold for all heads at once, the order is turned round: blockIdx.x runs over the
    // query tiles of one (batch, head), heaviest first, blockIdx.y over (batch, head), so that the CTAs resident at any time
    // share the K and V tiles of a few heads instead of re-reading every head's for each query tile.
    const int qt = p.qt_begin + (p.head_major ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)gridDim.y - 1 - (int)blockIdx.y);
    const int bh = p.head_major ? (int)blockIdx.y : (int)blockIdx.x;
    const int h = bh % p.Hq, b = bh / p.Hq;
    const int g = h / (p.Hq / p.Hkv);
    const int q0 = qt * BM;
    const int nt = min((q0 + BM) / BN, (p.N + BN - 1) / BN);  // key tiles 0..nt-1 reach the last query row / the last key

    if (tid == 0) {
        mbar_init(q_full, 1);
        for (int i = 0; i < KST; ++i) { mbar_init(k_full + i, 1); mbar_init(k_empty + i, 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(v_full + i, 1); mbar_init(v_empty + i, 1);
            mbar_init(s_full + i, 1); mbar_init(s_free + i, 128);
            mbar_init(p_full + i, 128); mbar_init(pv_done + i, 1);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 5) tmem_alloc(tmem_slot, L::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_O = tmem_base + 128;

    // The kernel is compiled for 128 registers per thread (two CTAs of 256 threads per SM).  The three single-thread
    // roles need few, the softmax threads (64 scores, their exponentials and a row of the accumulator in flight) more:
    // warpgroup 1 hands registers back and warpgroup 0 takes them (2 x (128 x 72 + 128 x 184) = 64 K).
    if (warp >= 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 4) {
        // ------------------------------ TMA producer ------------------------------
        // The two single-thread roles (this one and the MMA issuer) share their scheduler with busy softmax warps and
        // get an instruction slot every several cycles, so their loops are kept to a few dozen instructions per tile:
        // running stage counters instead of divisions, one wait/arm section by lane 0 per tile, then every copy of
        // the tile issued by different lanes (one 64-column box each).
        // V(t) (with Y(t)) travels together with K(t+1): both wait for the P.V of tile t-2 at the latest.
        constexpr int NQ = KD / 64, NK = KD / 64, NV = EMIT ? 0 : D / 64;
        if (lane == 0) {
            tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK);
            if (!EMIT) tma_prefetch_desc(&tmV);
            if (PLANE) tma_prefetch_desc(&tmY);
            mbar_expect_tx(q_full, L::Q_BYTES);
            mbar_expect_tx(k_full, L::K_BYTES);
        }
        __syncwarp();
        // One call site per tensor map, each reached with the map and the barrier uniform over the warp and only the
        // lane-dependent box differing, and a reconvergence point between sites.
        if (lane < NQ) tma_load_4d(sQ + lane * (BM * 128), &tmQ, q_full, lane * 64, h, q0, b);
        __syncwarp();
        if (lane < NK) tma_load_4d(sK + lane * (BN * 128), &tmK, k_full, lane * 64, g, 0, b);
        __syncwarp();
        int ks_next = 1 % KST;              // K stage of tile t+1
        uint32_t kpar_next = 1;             // parity to wait for on its "empty" barrier (first pass: passes at once)
        for (int t = 0; t < nt; ++t) {
            const int sv = t & 1;
            const bool more_k = t + 1 < nt;
            bool okp = true;
            if (lane == 0) {
                if constexpr (!EMIT) {
                    okp = mbar_wait(v_empty + sv, ((t >> 1) & 1) ^ 1, abort_flag);
                    if (okp) mbar_expect_tx(v_full + sv, L::V_BYTES + L::Y_BYTES);
                }
                if (okp && more_k) {
                    okp = mbar_wait(k_empty + ks_next, kpar_next, abort_flag);
                    if (okp) mbar_expect_tx(k_full + ks_next, L::K_BYTES);
                }
            }
            okp = __shfl_sync(0xffffffffu, okp, 0);
            if (!okp) break;
            if constexpr (!EMIT) {
                if (lane < NV) tma_load_4d(sV + sv * L::V_BYTES + lane * (BN * 128), &tmV, v_full + sv, lane * 64, g, t * BN, b);
                __syncwarp();
            }
            if constexpr (PLANE) {
                if (lane == 0) tma_load_5d(sY + sv * L::Y_BYTES, &tmY, v_full + sv, 0, b * p.Hq + h, 0, t, (q0 - p.plane_row0) / BM);
                __syncwarp();
            }
            if (more_k) {
                if (lane < NK) tma_load_4d(sK + ks_next * L::K_BYTES + lane * (BN * 128), &tmK, k_full + ks_next, lane * 64, g, (t + 1) * BN, b);
                __syncwarp();
            }
            // The V and Y stages of a tile cannot be refilled before the P.V of the tile two before it has run, one softmax pass
            // before they are needed -- less than a trip to HBM under load.  Their tiles are therefore asked into L2 earlier,
            // kPrefetchAhead tiles ahead of the one just issued.
            if constexpr (kPrefetchAhead > 0 && !EMIT) {
                if (t + kPrefetchAhead < nt) {
                    if (lane < NV) tma_prefetch_l2_4d(&tmV, lane * 64, g, (t + kPrefetchAhead) * BN, b);
                    __syncwarp();
                    if constexpr (PLANE) {
                        if (lane == 0) tma_prefetch_l2_5d(&tmY, 0, b * p.Hq + h, 0, t + kPrefetchAhead, (q0 - p.plane_row0) / BM);
                        __syncwarp();
                    }
                }
            }
            if (++ks_next == KST) { ks_next = 0; kpar_next ^= 1; }
        }
    } else if (warp == 5) {
        // ------------------------------ MMA issuer: scores ------------------------------
        // Issuing a tcgen05.mma holds the issuing thread for about as long as the MMAs queued before it take to run, so
        // the score MMAs and the P.V MMAs are issued by two different warps: each waits for its own operands and the
        // two hold-ups overlap instead of adding up.  Every lane of an issuing warp runs the loop (waits, stage
        // counters, descriptor arithmetic: all warp-uniform); only the MMA and commit instructions themselves are
        // predicated on lane 0.
        const uint32_t issue = lane == 0;
        constexpr uint32_t IDESC_QK = umma_idesc_bf16(BM, BN, 0, 0);
        const int ksteps = p.ksteps;
        // Descriptors are built once; per MMA only the start-address field (bits 0-13 of the low word, in
        // 16-byte units) moves, by a compile-time constant or a stage offset: no carry can leave the field.
        auto desc_off = [](uint64_t d, uint32_t bytes) -> uint64_t {
            return (d & 0xffffffff00000000ull) | (uint32_t)((uint32_t)d + (bytes >> 4));
        };
        const uint64_t dq0 = umma_desc_sw128(smem_u32(sQ), 16, 1024);
        const uint64_t dk0 = umma_desc_sw128(smem_u32(sK), 16, 1024);
        // scores of tile t into buffer t&1; needs K(t) loaded and (t >= 2) the buffer read by the softmax of t-2
        int sk = 0;
        uint32_t kpar = 0;
        bool ok = __all_sync(0xffffffffu, mbar_wait(q_full, 0, abort_flag));
        for (int t = 0; ok && t < nt; ++t) {
            const int s = t & 1;
            ok = mbar_wait(k_full + sk, kpar, abort_flag) && mbar_wait(s_free + s, ((t >> 1) & 1) ^ 1, abort_flag);
            if (!(ok = __all_sync(0xffffffffu, ok))) break;   // one verdict for the whole warp
            tc_fence_after();
            const uint64_t dk = desc_off(dk0, sk * L::K_BYTES);
            const uint32_t dst = tmem_base + s * BN;
#pragma unroll
            for (int ks = 0; ks < KD / 16; ++ks) {
                if (ks < ksteps) {
                    umma_ss_if(issue, dst, desc_off(dq0, (ks >> 2) * (BM * 128) + (ks & 3) * 32), desc_off(dk, (ks >> 2) * (BN * 128) + (ks & 3) * 32),
                               IDESC_QK, ks > 0);
                }
            }
            umma_commit_if(issue, s_full + s);
            if (!L::P_IN_K && t + KST < nt) umma_commit_if(issue, k_empty + sk);  // nobody waits for the last ones: do not arm them
            if (++sk == KST) { sk = 0; kpar ^= 1; }
        }
    } else if (warp == 6) {
        // ------------------------------ MMA issuer: P.V ------------------------------
        if constexpr (!EMIT) {
            const uint32_t issue = lane == 0;
            constexpr uint32_t IDESC_PV = umma_idesc_bf16(BM, D, 0, 1);
            auto desc_off = [](uint64_t d, uint32_t bytes) -> uint64_t {
                return (d & 0xffffffff00000000ull) | (uint32_t)((uint32_t)d + (bytes >> 4));
            };
            const uint64_t dv0 = umma_desc_sw128(smem_u32(sV), BN * 128, 1024);
            const uint64_t dp0 = umma_desc_sw128(smem_u32(p_buf(0)), 16, 1024);
            constexpr uint32_t P_STRIDE = L::P_IN_Y ? L::Y_BYTES : (L::P_IN_K ? L::K_BYTES : L::P_BYTES);
            int pk = 0;   // P_IN_K: K stage that holds P(t)
            bool ok = true;
            for (int t = 0; ok && t < nt; ++t) {
                const int s = t & 1;
                ok = mbar_wait(v_full + s, (t >> 1) & 1, abort_flag) && mbar_wait(p_full + s, (t >> 1) & 1, abort_flag);
                if (!(ok = __all_sync(0xffffffffu, ok))) break;
                tc_fence_after();
                const uint64_t dp = desc_off(dp0, (L::P_IN_K ? pk : s) * P_STRIDE);
                const uint64_t dv = desc_off(dv0, s * L::V_BYTES);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks) {
                    // P: K-major, 64 keys per 128-byte row; V: 16 keys = two 8-row groups, the next 64 d-columns
                    // BN * 128 bytes further on
                    umma_ss_if(issue, tmem_O, desc_off(dp, ks * 32), desc_off(dv, ks * 2048), IDESC_PV, (t > 0) || (ks > 0));
                }
                umma_commit_if(issue, pv_done + s);
                if (t + 2 < nt) umma_commit_if(issue, v_empty + s);
                if (L::P_IN_K && t + KST < nt) umma_commit_if(issue, k_empty + pk);
                if (++pk == KST) pk = 0;
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 184;");
        // ------------------------------ softmax / epilogue (thread = query row) ------------------------------
        const int row = tid;                       // 0..127, TMEM lane
        const int qi = q0 + row;                   // global query index
        const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
        const float scale_log2 = p.scale_log2, emit_scale = p.scale;
        float m_ref = -INFINITY, l_sum = 0.f;
        bool ok = true;
        for (int t = 0; t < nt; ++t) {
            const int s = t & 1;
            if (!(ok = mbar_wait(s_full + s, (t >> 1) & 1, abort_flag))) break;
            tc_fence_after();
            uint32_t sr[BN];
#pragma unroll
            for (int c = 0; c < BN / 32; ++c) tmem_ld32(tmem_base + s * BN + lane_sel + c * 32, sr + c * 32);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(s_free + s);
            float* sf = reinterpret_cast<float*>(sr);
            if constexpr (EMIT) {
                // this warp's 32 rows x 64 columns as fp16 into its staging buffer (swizzled like any other tile),
                // then lane 0 stores it with TMA
                uint8_t* stg = sStg + (warp * 2 + s) * 4096;
                if (t >= 2 && lane == 0) tma_store_wait_read<1>();  // the store of tile t-2 has read this buffer
                __syncwarp();
#pragma unroll
                for (int c = 0; c < BN / 8; ++c) {
                    uint4 v;
                    { const float2 t2 = __fmul2_rn(reinterpret_cast<const float2*>(sf)[c * 4 + 0], make_float2(emit_scale, emit_scale)); v.x = pack_f16(t2.x, t2.y); }
                    { const float2 t2 = __fmul2_rn(reinterpret_cast<const float2*>(sf)[c * 4 + 1], make_float2(emit_scale, emit_scale)); v.y = pack_f16(t2.x, t2.y); }
                    { const float2 t2 = __fmul2_rn(reinterpret_cast<const float2*>(sf)[c * 4 + 2], make_float2(emit_scale, emit_scale)); v.z = pack_f16(t2.x, t2.y); }
                    { const float2 t2 = __fmul2_rn(reinterpret_cast<const float2*>(sf)[c * 4 + 3], make_float2(emit_scale, emit_scale)); v.w = pack_f16(t2.x, t2.y); }
                    *reinterpret_cast<uint4*>(stg + sw128_offset(lane, c)) = v;
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_5d(&tmY, stg, 0, b * p.Hq + h, warp * 32, t, (q0 - p.plane_row0) / BM);
                    tma_store_commit();
                }
                continue;
            }
            if constexpr (PLANE) {
                if (!(ok = mbar_wait(v_full + s, (t >> 1) & 1, abort_flag))) break;  // Y of this stage has landed
                const uint8_t* yb = sY + s * L::Y_BYTES;
#pragma unroll
                for (int c = 0; c < BN / 8; ++c) {
                    const uint4 y = *reinterpret_cast<const uint4*>(yb + sw128_offset(row, c));
                    const uint32_t w[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float2* s2 = reinterpret_cast<float2*>(sf) + c * 4 + e;
                        *s2 = __ffma2_rn(*s2, make_float2(scale_log2, scale_log2), unpack_f16(w[e]));
                    }
                }
            }
            if constexpr (CARRY) {
                // the finished logits of this warp's 32 rows x 64 columns leave as fp16 (back in the natural-log domain,
                // before the mask: the next layer's aligner sees finite values everywhere) through the warp's staging buffer
                uint8_t* stg = sStg + warp * 4096;
                if (t >= 1 && lane == 0) tma_store_wait_read<0>();  // the store of the previous tile has read the buffer
                __syncwarp();
                constexpr float kLn2 = 0.6931471805599453f;
#pragma unroll
                for (int c = 0; c < BN / 8; ++c) {
                    uint4 v;
                    { const float2 t2 = __fmul2_rn(reinterpret_cast<const float2*>(sf)[c * 4 + 0], make_float2(kLn2, kLn2)); v.x = pack_f16(t2.x, t2.y); }
                    { const float2 t2 = __fmul2_rn(reinterpret_cast<const float2*>(sf)[c * 4 + 1], make_float2(kLn2, kLn2)); v.y = pack_f16(t2.x, t2.y); }
                    { const float2 t2 = __fmul2_rn(reinterpret_cast<const float2*>(sf)[c * 4 + 2], make_float2(kLn2, kLn2)); v.z = pack_f16(t2.x, t2.y); }
                    { const float2 t2 = __fmul2_rn(reinterpret_cast<const float2*>(sf)[c * 4 + 3], make_float2(kLn2, kLn2)); v.w = pack_f16(t2.x, t2.y); }
                    *reinterpret_cast<uint4*>(stg + sw128_offset(lane, c)) = v;
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_5d(&tmC, stg, 0, b * p.Hq + h, warp * 32, t, (q0 - p.plane_row0) / BM);
                    tma_store_commit();
                }
            }
            // from here on: PLANE -> sf holds log2-domain logits; otherwise raw scores, scaled inside the exp
            if (t * BN + BN - 1 > q0) {   // the tile reaches past the CTA's first query row: mask keys after each row
#pragma unroll
                for (int j = 0; j < BN; ++j)
                    if (t * BN + j > qi) sf[j] = -INFINITY;
            }
            float mx[4] = {sf[0], sf[1], sf[2], sf[3]};   // four independent chains instead of one of 64 dependent steps
#pragma unroll
            for (int j = 4; j + 8 <= BN; j += 8) {   // two new values per step and chain: a three-input maximum where there is one
                mx[0] = fmaxf(fmaxf(mx[0], sf[j]), sf[j + 4]); mx[1] = fmaxf(fmaxf(mx[1], sf[j + 1]), sf[j + 5]);
                mx[2] = fmaxf(fmaxf(mx[2], sf[j + 2]), sf[j + 6]); mx[3] = fmaxf(fmaxf(mx[3], sf[j + 3]), sf[j + 7]);
            }
            mx[0] = fmaxf(mx[0], sf[BN - 4]); mx[1] = fmaxf(mx[1], sf[BN - 3]);
            mx[2] = fmaxf(mx[2], sf[BN - 2]); mx[3] = fmaxf(mx[3], sf[BN - 1]);
            float m_t = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            if constexpr (!PLANE) m_t *= scale_log2;
            // lazy rescale: move the reference maximum only when some row of the warp outgrew it by 2^8
            // (a row with every key of this tile masked has m_t = -inf and never asks for it)
            const bool grow = m_t > m_ref + 8.f;
            const bool rescale = __any_sync(0xffffffffu, grow) || t == 0;
            float factor = 1.f;
            if (rescale) {
                const float m_new = fmaxf(m_ref, m_t);
                factor = fast_exp2(m_ref - m_new);
                m_ref = m_new;
            }
            if (t > 0 && rescale) {   // the accumulator is touched only after every P.V issued so far has landed in it
                if (!(ok = mbar_wait(pv_done + ((t - 1) & 1), ((t - 1) >> 1) & 1, abort_flag))) break;
                {
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t orr[32];
                        tmem_ld32(tmem_O + lane_sel + c * 32, orr);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            float2* o2 = reinterpret_cast<float2*>(orr) + j;
                            *o2 = __fmul2_rn(*o2, make_float2(factor, factor));
                        }
                        tmem_st32(tmem_O + lane_sel + c * 32, orr);
                    }
                    tmem_wait_st();
                }
            }
            // P(t) is announced on p_full[t & 1], a barrier whose phases the P.V warp tells apart by parity alone.  Since the
            // score MMAs no longer wait for the P.V MMAs, the softmax could finish tile t while P.V(t-2) has not even been
            // picked up: the barrier would then run two phases ahead and the waiting warp would never see its phase end.
            // So tile t's announcement waits until P.V(t-2) has completed (which also frees a P buffer of its own,
            // where the layout has one); two tiles back, this has nearly always happened already.
            if (t >= 2 && !(ok = mbar_wait(pv_done + s, ((t - 2) >> 1) & 1, abort_flag))) break;
            uint8_t* pb = p_buf(t);
            // The softmax warps are bound by the length of their own instruction chain, so the fp32 arithmetic around
            // the exponentials runs two values per instruction (packed fp32 pairs; the scores of a thread sit in
            // consecutive registers).
            float2 sum2 = make_float2(0.f, 0.f);
            const float2 neg_m2 = make_float2(-m_ref, -m_ref), scale2 = make_float2(scale_log2, scale_log2);
            const float2* sf2 = reinterpret_cast<const float2*>(sf);
#pragma unroll
            for (int c = 0; c < BN / 8; ++c) {
                float e[8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 x = PLANE ? __fadd2_rn(sf2[c * 4 + j], neg_m2) : __ffma2_rn(sf2[c * 4 + j], scale2, neg_m2);
                    e[2 * j] = fast_exp2(x.x);
                    e[2 * j + 1] = fast_exp2(x.y);
                    sum2 = __fadd2_rn(sum2, make_float2(e[2 * j], e[2 * j + 1]));
                }
                uint4 v;
                v.x = pack_bf16(e[0], e[1]); v.y = pack_bf16(e[2], e[3]); v.z = pack_bf16(e[4], e[5]); v.w = pack_bf16(e[6], e[7]);
                *reinterpret_cast<uint4*>(pb + sw128_offset(row, c)) = v;
            }
            l_sum = l_sum * factor + (sum2.x + sum2.y);
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(p_full + s);
        }
        if constexpr (EMIT || CARRY) {
            if (lane == 0) tma_store_wait_all<0>();
        }
        if constexpr (EMIT) {
        } else if (ok && mbar_wait(pv_done + ((nt - 1) & 1), ((nt - 1) >> 1) & 1, abort_flag)) {
            tc_fence_after();
            const float inv_l = 1.f / l_sum;
            __nv_bfloat16* orow = p.o + b * p.o_sb + (int64_t)qi * p.o_sn + h * p.o_sh;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t orr[32];
                tmem_ld32(tmem_O + lane_sel + c * 32, orr);
                tmem_wait_ld();
                if (qi < p.N) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint4 v;
                        v.x = pack_bf16(__uint_as_float(orr[q * 8 + 0]) * inv_l, __uint_as_float(orr[q * 8 + 1]) * inv_l);
                        v.y = pack_bf16(__uint_as_float(orr[q * 8 + 2]) * inv_l, __uint_as_float(orr[q * 8 + 3]) * inv_l);
                        v.z = pack_bf16(__uint_as_float(orr[q * 8 + 4]) * inv_l, __uint_as_float(orr[q * 8 + 5]) * inv_l);
                        v.w = pack_bf16(__uint_as_float(orr[q * 8 + 6]) * inv_l, __uint_as_float(orr[q * 8 + 7]) * inv_l);
                        *reinterpret_cast<uint4*>(orow + c * 32 + q * 8) = v;
                    }
                }
            }
        }
    }
    // ------------------------------ teardown ------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait ran out: give copies and MMAs still in flight time to land before the memory is released
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

bool make_tensor_map_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                          const uint32_t* box, bool fp16) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
            qres != cudaDriverEntryPointSuccess)
            return false;
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    cuuint64_t gdims[5], gstr[4];
    cuuint32_t gbox[5], estr[5];
    for (int i = 0; i < rank; ++i) { gdims[i] = dims[i]; gbox[i] = box[i]; estr[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
    return encode(map, fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdims, gstr, gbox, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {
bool tma_ok(const lisa_tensor& t) {
    return t.dtype == LISA_BF16 && (reinterpret_cast<uintptr_t>(t.ptr) & 15u) == 0 && t.stride_b % 8 == 0 && t.stride_n % 8 == 0 &&
           t.stride_h % 8 == 0 && t.stride_b > 0 && t.stride_n > 0 && t.stride_h > 0;
}
bool map_bnhx(CUtensorMap* m, const lisa_tensor& t, int B, int N, int H, int X, int rows) {
    const uint64_t dims[4] = {(uint64_t)X, (uint64_t)H, (uint64_t)N, (uint64_t)B};
    const uint64_t str[3] = {(uint64_t)t.stride_h * 2, (uint64_t)t.stride_n * 2, (uint64_t)t.stride_b * 2};
    const uint32_t box[4] = {64, 1, (uint32_t)rows, 1};
    return make_tensor_map_bf16(m, t.ptr, 4, dims, str, box);
}
}  // namespace

bool tc_flash_supported(const TcFlashArgs& a) {
    if (!((a.kd == 128 || a.kd == 64) && tma_ok(a.qa) && tma_ok(a.ka) && a.Hq % a.Hkv == 0)) return false;
    return a.emit_plane ? true : (tma_ok(a.v) && tma_ok(a.o));
}

cudaError_t launch_tc_flash(const TcFlashArgs& a, cudaStream_t stream) {
    CUtensorMap tmQ, tmK, tmV, tmY;
    if (!map_bnhx(&tmQ, a.qa, a.B, a.N, a.Hq, a.kd, BM) || !map_bnhx(&tmK, a.ka, a.B, a.N, a.Hkv, a.kd, BN)) return cudaErrorInvalidValue;
    tmV = tmQ;
    if (!a.emit_plane && !map_bnhx(&tmV, a.v, a.B, a.N, a.Hkv, D, BN)) return cudaErrorInvalidValue;
    tmY = tmQ;
    CUtensorMap tmC = tmQ;
    // Score planes are blocked [row block of 128][column block of 64][row in block][b*Hq + h][64 columns]: the 32
    // heads of a position lie 128 bytes apart (the aligner gathers them), and a head's 128 x 64 tile is 128 rows of 128
    // bytes spread over one 128 * B*Hq * 128-byte block, which the CTAs of all heads fill or drain at about the same time.
    if (a.emit_plane || a.plane) {
        if (a.plane_rows % BM != 0 || a.plane_cols % BN != 0) return cudaErrorInvalidValue;
        const uint64_t bh = (uint64_t)a.B * a.Hq, ncb = (uint64_t)a.plane_cols / BN, nrb = (uint64_t)a.plane_rows / BM;
        const uint64_t dims[5] = {(uint64_t)BN, bh, (uint64_t)BM, ncb, nrb};
        const uint64_t str[4] = {(uint64_t)BN * 2, bh * BN * 2, (uint64_t)BM * bh * BN * 2, ncb * BM * bh * BN * 2};
        // emit: one epilogue warp's 32 rows x 64 columns per copy; attention: the CTA's 128 rows x 64 columns
        const uint32_t box[5] = {(uint32_t)BN, 1, a.emit_plane ? 32u : (uint32_t)BM, 1, 1};
        if (!make_tensor_map_bf16(&tmY, a.emit_plane ? a.emit_plane : a.plane, 5, dims, str, box, true)) return cudaErrorInvalidValue;
        if (a.carry) {   // the logits leave one epilogue warp's 32 rows at a time
            if (a.emit_plane || !a.plane) return cudaErrorInvalidValue;
            const uint32_t cbox[5] = {(uint32_t)BN, 1, 32u, 1, 1};
            if (!make_tensor_map_bf16(&tmC, a.carry, 5, dims, str, cbox, true)) return cudaErrorInvalidValue;
        }
    }
    FlashParams p;
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    p.o = reinterpret_cast<__nv_bfloat16*>(a.o.ptr);
    p.o_sb = a.o.stride_b; p.o_sn = a.o.stride_n; p.o_sh = a.o.stride_h;
    p.status = status_words();
    if (!p.status) return cudaErrorUnknown;
    p.plane_row0 = a.plane_row0 >= 0 ? a.plane_row0 : a.qt_begin * BM;
    if (p.plane_row0 % BM != 0 || p.plane_row0 > a.qt_begin * BM) return cudaErrorInvalidValue;
    p.qt_begin = a.qt_begin;
    p.ksteps = a.ksteps > 0 ? a.ksteps : a.kd / 16;
    p.scale = a.scale;

    if (a.qt_count < 1 || a.qt_count > 65535) return cudaErrorInvalidValue;
    // K and V of all (batch, KV head) pairs against half of a 126 MB L2 (the other half for everything else that streams)
    const int64_t kv_bytes = (int64_t)a.B * a.Hkv * a.N * (a.kd + (a.emit_plane ? 0 : D)) * 2;
    p.head_major = kv_bytes > ((int64_t)63 << 20) && (int64_t)a.Hq * a.B <= 65535 && a.qt_count > 1;
    dim3 grid(a.Hq * a.B, a.qt_count);
    if (p.head_major) grid = dim3(a.qt_count, a.Hq * a.B);
    cudaError_t e;
#define LISA_LAUNCH_FLASH(KD_, PL_)                                                                                       \
    do {                                                                                                                   \
        auto kern = tc_flash_kernel<KD_, PL_>;                                                                             \
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<KD_, PL_>::TOTAL)) != cudaSuccess) \
            return e;                                                                                                      \
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess) \
            return e;                                                                                                      \
        kern<<<grid, kThreads, Smem<KD_, PL_>::TOTAL, stream>>>(p, tmQ, tmK, tmV, tmY, tmC);                                    \
    } while (0)
    if (a.emit_plane) {
        if (a.kd == 128) LISA_LAUNCH_FLASH(128, MODE_EMIT);
        else LISA_LAUNCH_FLASH(64, MODE_EMIT);
    } else if (a.kd == 128 && !a.plane) LISA_LAUNCH_FLASH(128, MODE_ATTN);
    else if (a.kd == 64 && a.plane && a.carry) LISA_LAUNCH_FLASH(64, MODE_ATTN_CARRY);
    else if (a.kd == 64 && a.plane) LISA_LAUNCH_FLASH(64, MODE_ATTN_PLANE);
    else if (a.kd == 64 && !a.plane) LISA_LAUNCH_FLASH(64, MODE_ATTN);
    else return cudaErrorInvalidValue;  // 128-wide scores plus a plane do not fit shared memory
#undef LISA_LAUNCH_FLASH
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace lisa
