// Warp-specialised HiFA4 attention forward for Bc = 64 (Algorithm 1 lines 4-13), d = 64, 128 or 256.
//
// One CTA = 128 query rows of one (batch, query head), 10 warps:
//   warps 0-7  softmax / quantize: warp w owns rows 32*(w%4).. of the tile and keys 32*(w/4).. of
//              every 64-key tile, i.e. half of the tile's single HIF4 group per thread; for the row
//              maximum each thread also reads the other half of its row from tensor memory (cheaper
//              than an exchange between the two threads: a poll of an mbarrier costs > 100 clk)
//   warp 8     TMA producer: Q once, then K and V^T tiles through two-stage rings
//   warp 9     tcgen05 issuer
// S has a single buffer that is released early: the softmax warps pull S(j) into registers and
// signal it free, and S(j+1) = Q K^T runs on the tensor pipe while they work on tile j; the BF16
// image of P-hat has its own tensor-memory columns and is the A operand of the PV MMA.
//   d = 256: 512 tensor-memory columns: [O | l] 0..271 (an N = 256 MMA for the channels, an N = 16
//            MMA on the same A operand for the ones block), Q-hat image 272..399 (A operand of
//            Q K^T from tensor memory), S 400..463, P-hat 464..495.  One CTA per SM.
//   d = 64:  as d = 128 with [O | l] 0..79 (one N = 80 MMA); 53 KB of shared memory.
//   d = 128: 256 tensor-memory columns: [O | l] 0..143 (one N = 144 MMA), S 144..207, P-hat
//            208..239; Q-hat stays in shared memory (SS-form Q K^T).  101 KB of shared memory and
//            <= 102 registers, so two CTAs share an SM and fill each other's synchronisation gaps.
// Polls for S(j+1) and PV(j-1) are issued early with test_wait (try_wait blocks while the phase is
// incomplete); the blocking wait is the fall-back.  Epilogue: O / l by reciprocal plus one correction
// step, FP32 output through a per-warp 32 x 32 shared-memory transpose (the K stages are idle by then).
// The grid is launched with programmatic stream serialization: everything before griddepcontrol.wait
// (barrier set-up, tensor-memory allocation) may overlap the tail of the preceding kernel.
// Template flags: P-hat dump, FP32-P variant, Q-Mean (key sums staged in shared memory by the producer).
// Every wait is bounded (see hifa4_attention_ws.cu for the failure protocol).
#include "hifa4_attention.cuh"

namespace hifa4 {

#ifndef HIFA4_WS64_KS128
#define HIFA4_WS64_KS128 2
#endif
#ifndef HIFA4_WS64_KS256
#define HIFA4_WS64_KS256 2
#endif
template <int D_>
struct WS64 {
    static constexpr int D = D_, BC = 64, STAGES = 2, KS = (D_ == 128) ? HIFA4_WS64_KS128 : (D_ == 256 ? HIFA4_WS64_KS256 : 2);
    static constexpr int NSW = 4 * KS, THREADS = (NSW + 2) * 32, W_TMA = NSW, W_MMA = NSW + 1;
    static constexpr int KPT = BC / KS, NU = KPT / 8;       // 32 keys = 4 level-2 units per thread and tile
    static constexpr int QSUB = D / 64;                     // 64-channel sub-tiles of Q and K
    static constexpr int Q_BYTES = QSUB * 16384;
    static constexpr int K_SUB = BC * 128;                  // 64 keys x 64 channels
    static constexpr int K_STAGE = QSUB * K_SUB;
    static constexpr int V_STAGE = (D + 16) * 128;          // D rows of V^T + 16 rows of ones, 64 keys wide
    static constexpr int Q_OFF = 0;
    static constexpr int K_OFF = Q_OFF + Q_BYTES;
    static constexpr int V_OFF = K_OFF + STAGES * K_STAGE;
    static constexpr int MISC_OFF = V_OFF + STAGES * V_STAGE;
    static constexpr int KSUM_OFF = MISC_OFF + 256;         // Q-Mean: channel sums of the tile's 64 keys, two stages
    static constexpr int SMEM_BYTES = KSUM_OFF + STAGES * 256 + 1024;
    static constexpr int O_COLS = D + 16;
    static constexpr bool Q_IN_TMEM = (D == 256);
    static constexpr int QT_COL = 272;                      // d = 256 only
    static constexpr int S_COL = (D == 256) ? 400 : 144;
    static constexpr int P_COL = S_COL + 64;
    static constexpr int TMEM_COLS = (D == 256) ? 512 : 256;
    static constexpr int CTAS_PER_SM = (D == 256) ? 1 : 2;
};
namespace ws64 {
enum { BAR_Q = 0, BAR_KF = 1, BAR_KE = 3, BAR_VF = 5, BAR_VE = 7, BAR_SF = 9, BAR_SFREE = 10, BAR_PF = 11,
       BAR_PV = 12, BAR_KSF = 13, BAR_QT = 17, N_BARS = 18 };
constexpr uint32_t WAIT_POLLS = 1u << 20;
}  // namespace ws64

static __device__ __forceinline__ bool wait64(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (uint32_t i = 0; i < ws64::WAIT_POLLS / 64; ++i) {
#pragma unroll 1
        for (int j = 0; j < 64; ++j)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    return false;
}

template <int DH, bool DBG, bool PF32, bool QM>
__global__ void __launch_bounds__(WS64<DH>::THREADS, WS64<DH>::CTAS_PER_SM)
attention_fwd_ws64_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                           const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ AttnArgs args)
{
    using namespace ws64;
    using C = WS64<DH>;
    constexpr int D = C::D, BC = C::BC, STAGES = C::STAGES, KS = C::KS, NSW = C::NSW, THREADS = C::THREADS;
    constexpr int W_TMA = C::W_TMA, W_MMA = C::W_MMA, KPT = C::KPT, NU = C::NU, QSUB = C::QSUB;
    constexpr int Q_BYTES = C::Q_BYTES, K_SUB = C::K_SUB, K_STAGE = C::K_STAGE, V_STAGE = C::V_STAGE;
    constexpr int O_COLS = C::O_COLS, QT_COL = C::QT_COL, S_COL = C::S_COL, P_COL = C::P_COL, TMEM_COLS = C::TMEM_COLS;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_s = smem_base + C::Q_OFF, k_s = smem_base + C::K_OFF, v_s = smem_base + C::V_OFF,
                   bars = smem_base + C::MISC_OFF;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + C::MISC_OFF + 8 * N_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + C::MISC_OFF + 8 * N_BARS + 8);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = args.N;
    const int n_qt = (N + 127) / 128;
    // 1-D grid, query block outermost and descending: the heaviest causal CTAs are scheduled first
    const int n_bh = args.B * args.Hq;
    // Long sequences, whose K/V images do not fit in L2 together: head outermost instead, so that the
    // CTAs in flight share the K/V of one or two heads; still heaviest first inside a head.
    const int qt = n_qt - 1 - (int)(args.head_major ? blockIdx.x % n_qt : blockIdx.x / n_bh);
    const int bh = (int)(args.head_major ? blockIdx.x / n_qt : blockIdx.x % n_bh);
    const int h = bh % args.Hq, b = bh / args.Hq;
    const int g = args.map.kv_of[h];
    const int q0 = qt * 128;
    const int bh_q = b * args.Hq + h, bh_kv = b * args.Hkv + g;
    const int last_key = args.causal ? min(q0 + 127, N - 1) : N - 1;
    const int n_tiles = last_key / BC + 1;

    if (tid == 0) {
        // A CTA that starts after another one reported a failure does nothing.  One thread reads the status
        // word (the load is in flight during the set-up below) and publishes the verdict through shared
        // memory, so that all roles of the CTA agree on it.
        const int status_now = args.d_status ? *reinterpret_cast<volatile int*>(args.d_status) : 0;
        mbar_init(bar(BAR_Q), 1);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(BAR_KF + s), 1); mbar_init(bar(BAR_KE + s), 1);
            mbar_init(bar(BAR_VF + s), 1); mbar_init(bar(BAR_VE + s), 1);
        }
        mbar_init(bar(BAR_SF), 1); mbar_init(bar(BAR_SFREE), NSW);
        mbar_init(bar(BAR_PF), NSW); mbar_init(bar(BAR_PV), 1); mbar_init(bar(BAR_QT), NSW);
        mbar_init(bar(BAR_KSF), 1); mbar_init(bar(BAR_KSF + 1), 1);
        fence_barrier_init();
        *abort_flag = status_now != 0 ? 2 : 0;
    }
    if (warp == W_MMA) { tmem_alloc(smem_u32((const void*)tmem_slot), TMEM_COLS); tmem_relinquish(); }
    if (warp == W_TMA && lane == 0) { tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_k); tma_prefetch_desc(&tmap_v); }
    for (int i = tid; i < STAGES * 128; i += THREADS) {           // ones rows under every V^T stage
        const int st = i / 128, off = (i % 128) * 16;
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};"
                     ::"r"(v_s + st * V_STAGE + D * 128 + off), "r"(0x3F803F80u) : "memory");
    }
    fence_proxy_async_smem();
    tc_fence_before();
    // The launch lets this grid start while its predecessor in the stream is still running (its CTAs
    // become resident and set themselves up as SMs drain); nothing the predecessor wrote is touched
    // before this point.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // The status word was read before the wait; a non-zero value may be one that the preceding work in the
    // stream has cleared since, so only that (rare) verdict is confirmed by a second read.
    if (tid == 0 && *abort_flag) *abort_flag = *reinterpret_cast<volatile int*>(args.d_status) != 0 ? 2 : 0;
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const bool dead = *abort_flag != 0;

    auto fail = [&](int site) {
        *abort_flag = 1;
        if (args.d_status) atomicCAS(args.d_status, 0, HIFA4_ERR_TIMEOUT + 16 * site);
    };

    if (dead) {
        // fall through to the common exit
    } else if (warp == W_TMA) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(bar(BAR_Q), Q_BYTES);
#pragma unroll
            for (int s = 0; s < QSUB; ++s) tma_load_3d(q_s + s * 16384, &tmap_q, bar(BAR_Q), 64 * s, q0, bh_q);
            for (int jt = 0; jt < n_tiles; ++jt) {
                const int st = jt & 1;
                const uint32_t ph = (uint32_t)(jt >> 1) & 1u;
                const int j0 = jt * BC;
                if (!wait64(bar(BAR_KE + st), ph ^ 1u, abort_flag)) { fail(1); break; }
                mbar_expect_tx(bar(BAR_KF + st), K_STAGE);
#pragma unroll
                for (int s = 0; s < QSUB; ++s)
                    tma_load_3d(k_s + st * K_STAGE + s * K_SUB, &tmap_k, bar(BAR_KF + st), 64 * s, j0, bh_kv);
                if (!wait64(bar(BAR_VE + st), ph ^ 1u, abort_flag)) { fail(2); break; }
                mbar_expect_tx(bar(BAR_VF + st), D * 128);
                tma_load_3d(v_s + st * V_STAGE, &tmap_v, bar(BAR_VF + st), j0, 0, bh_kv);
                if (QM) {
                    // Q-Mean: the 64 channel sums of this tile's keys; their stage is free with the V stage
                    // (PV(jt-2) complete means every softmax warp is past tile jt-2)
                    mbar_expect_tx(bar(BAR_KSF + st), 256);
                    bulk_load(smem_base + C::KSUM_OFF + st * 256, args.k_sum + (size_t)bh_kv * N + j0, 256, bar(BAR_KSF + st));
                }
            }
        }
    } else if (warp == W_MMA) {
        // ------------------------------------------------------------------ tcgen05 issuer
        constexpr uint32_t idesc_s = umma_idesc_bf16(128, BC);
        constexpr uint32_t idesc_o = umma_idesc_bf16(128, D == 256 ? 256 : O_COLS);
        constexpr uint32_t idesc_l = umma_idesc_bf16(128, 16);
        const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
        const uint32_t q_lo = umma_desc_lo(q_s), k_lo = umma_desc_lo(k_s), v_lo = umma_desc_lo(v_s);
        const bool leader = elect_one();
        bool ok = true;
        auto issue_qk = [&](int jt) {                     // S(jt) from K stage jt % 2 (D / 16 steps of 16 channels)
            const uint32_t b0 = k_lo + (jt & 1) * (K_STAGE >> 4);
            if (leader) {
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t kb = b0 + (kk >> 2) * (K_SUB >> 4) + (kk & 3) * 2;
                    if constexpr (C::Q_IN_TMEM) umma_bf16_ts_lo(tm + S_COL, tm + QT_COL + kk * 8, kb, idesc_s, kk ? 1u : 0u);
                    else umma_bf16_ss_lo(tm + S_COL, q_lo + (kk >> 2) * (16384 >> 4) + (kk & 3) * 2, kb, idesc_s, kk ? 1u : 0u);
                }
                umma_commit(bar(BAR_SF));
                umma_commit(bar(BAR_KE + (jt & 1)));
            }
            __syncwarp();
        };
        ok = wait64(bar(C::Q_IN_TMEM ? BAR_QT : BAR_Q), 0, abort_flag) && wait64(bar(BAR_KF), 0, abort_flag);
        if (ok) { tc_fence_after(); issue_qk(0); } else if (leader) fail(3);
        for (int jt = 0; ok && jt < n_tiles; ++jt) {
            const int st = jt & 1;
            const uint32_t ph = (uint32_t)(jt >> 1) & 1u, par = (uint32_t)jt & 1u;
            if (jt + 1 < n_tiles) {                       // S(jt+1) as soon as S(jt) sits in registers
                if (!wait64(bar(BAR_KF + (st ^ 1)), (uint32_t)((jt + 1) >> 1) & 1u, abort_flag)) { if (leader) fail(4); break; }
                if (!wait64(bar(BAR_SFREE), par, abort_flag)) { if (leader) fail(5); break; }
                tc_fence_after();
                issue_qk(jt + 1);
            }
            if (!wait64(bar(BAR_VF + st), ph, abort_flag)) { if (leader) fail(6); break; }
            if (!wait64(bar(BAR_PF), par, abort_flag)) { if (leader) fail(7); break; }
            tc_fence_after();
            const uint32_t b0 = v_lo + st * (V_STAGE >> 4);
            const uint32_t acc0 = jt > 0 ? 1u : 0u;
            if (leader) {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {            // 16 keys per step; channels (+ ones block)
                    umma_bf16_ts_lo(tm, tm + P_COL + kk * 8, b0 + kk * 2, idesc_o, kk ? 1u : acc0);
                    if constexpr (D == 256)                  // N = 272 does not exist: the ones block separately
                        umma_bf16_ts_lo(tm + 256, tm + P_COL + kk * 8, b0 + ((D * 128) >> 4) + kk * 2, idesc_l, kk ? 1u : acc0);
                }
                umma_commit(bar(BAR_PV));
                umma_commit(bar(BAR_VE + st));
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ softmax / quantize
        const int kq = warp >> 2, quarter = warp & 3;             // key half, row quarter
        const int r_loc = quarter * 32 + lane;                    // row inside the tile = TMEM lane
        const int row = q0 + r_loc;
        const uint32_t t_lane = tmem + ((uint32_t)(quarter * 32) << 16);
        const float LOG2E = 1.4426950408889634f;
        const int key_lim = args.causal ? min(row, N - 1) : N - 1;
        int dbg_slot = -1;
        if (DBG)
            for (int i = 0; i < args.dbg.n_blocks; ++i)
                if (args.dbg.blocks[3 * i] == b && args.dbg.blocks[3 * i + 1] == h && args.dbg.blocks[3 * i + 2] == qt)
                    dbg_slot = i;
        const float mu_row = (QM && row < N) ? args.q_mu[(size_t)bh_q * N + row] : 0.f;
        float m_run = -INFINITY;
        bool ok = true;

        // d = 256: Q-hat image, shared memory (swizzled TMA tiles) -> tensor memory; this thread moves 128
        // channels of its row = 64 columns of packed BF16 pairs.  (d = 128: the issuer waits for the
        // Q load itself.)
        if constexpr (C::Q_IN_TMEM) {
            static_assert(!C::Q_IN_TMEM || KS == 2 || KS == 4, "the Q copy splits a row over two or four threads");
            if (wait64(bar(BAR_Q), 0, abort_flag)) {
                const int sw = r_loc & 7;
                constexpr int PARTS = 4 / KS;                          // pieces of 64 channels (8 chunks, 32 columns)
#pragma unroll
                for (int half = 0; half < PARTS; ++half) {
                    uint32_t qw[32];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int chunk = (kq * PARTS + half) * 8 + c; // 16-byte chunk of the 512-byte row
                        const uint32_t a = q_s + (chunk >> 3) * 16384 + (r_loc >> 3) * 1024 + sw * 128 + (((chunk & 7) ^ sw) << 4);
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(qw[4 * c]), "=r"(qw[4 * c + 1]), "=r"(qw[4 * c + 2]), "=r"(qw[4 * c + 3]) : "r"(a));
                    }
                    tmem_st32(t_lane + QT_COL + (kq * PARTS + half) * 32, qw);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_QT));
            } else { fail(13); ok = false; }
        }

        bool sf_ready = false;
        for (int jt = 0; ok && jt < n_tiles; ++jt) {
            const int j0 = jt * BC;
            const uint32_t par = (uint32_t)jt & 1u;
            const int kbase = j0 + kq * KPT;
            // the poll for S(jt) was issued before the tail of the previous tile (a poll takes > 100 clk)
            if (!sf_ready && !wait64(bar(BAR_SF), par, abort_flag)) { fail(8); ok = false; break; }
            tc_fence_after();
            // The thread pulls its own KPT scores and, for the row maximum (line 7), the rest of the row
            // as well: the tile is one 64-key group, so row maximum = group maximum, and reading the other
            // columns again costs less than an exchange with the other threads of the row.
            float p[KPT], po[BC - KPT + 1];
            {
                uint32_t r[KPT], ro[BC - KPT + 1];
                if constexpr (KS == 1) {
                    uint32_t r1[32];
                    tmem_ld32(t_lane + S_COL, reinterpret_cast<uint32_t(&)[32]>(r[0]));
                    tmem_ld32(t_lane + S_COL + 32, r1);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[32 + i] = r1[i];
                } else if constexpr (KS == 2) {
                    tmem_ld32(t_lane + S_COL + kq * KPT, reinterpret_cast<uint32_t(&)[32]>(r[0]));
                    tmem_ld32(t_lane + S_COL + (kq ^ 1) * KPT, reinterpret_cast<uint32_t(&)[32]>(ro[0]));
                    tmem_wait_ld();
                } else {
                    static_assert(KS == 4, "key split of one, two or four threads per row");
                    tmem_ld16(t_lane + S_COL + kq * KPT, reinterpret_cast<uint32_t(&)[16]>(r[0]));
#pragma unroll
                    for (int o = 1; o < KS; ++o)               // part kq ^ o of the row goes to ro[(o - 1) * KPT ..]
                        tmem_ld16(t_lane + S_COL + (kq ^ o) * KPT, reinterpret_cast<uint32_t(&)[16]>(ro[(o - 1) * KPT]));
                    tmem_wait_ld();
                }
#pragma unroll
                for (int i = 0; i < KPT; ++i) p[i] = __uint_as_float(r[i]);
#pragma unroll
                for (int i = 0; i < BC - KPT; ++i) po[i] = __uint_as_float(ro[i]);
            }
            tc_fence_before();                                 // S(jt) is in registers: S(jt+1) may overwrite it
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_SFREE));

            auto obase = [&](int o) { return j0 + (kq ^ o) * KPT; };   // first key of the o-th other part of the row
            if (QM) {                                          // Q-Mean correction (line 6): + mu_i * sum_c k~_jc
                if (!wait64(bar(BAR_KSF + (jt & 1)), (uint32_t)(jt >> 1) & 1u, abort_flag)) { fail(15); ok = false; break; }
                const uint32_t ks_s = smem_base + C::KSUM_OFF + (jt & 1) * 256;
                auto add_part = [&](float* dst, int part) {     // keys part * KPT .. of the tile
#pragma unroll
                    for (int i = 0; i < KPT / 4; ++i) {
                        float4 ks;
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(ks.x), "=f"(ks.y), "=f"(ks.z), "=f"(ks.w) : "r"(ks_s + (part * KPT + 4 * i) * 4));
                        dst[4 * i] = fmaf(mu_row, ks.x, dst[4 * i]);
                        dst[4 * i + 1] = fmaf(mu_row, ks.y, dst[4 * i + 1]);
                        dst[4 * i + 2] = fmaf(mu_row, ks.z, dst[4 * i + 2]);
                        dst[4 * i + 3] = fmaf(mu_row, ks.w, dst[4 * i + 3]);
                    }
                };
                add_part(p, kq);
#pragma unroll
                for (int o = 1; o < KS; ++o) add_part(po + (o - 1) * KPT, kq ^ o);
            }
            const bool need_mask = (args.causal && (j0 + BC - 1 > q0)) || (j0 + BC > N);
            if (need_mask) {                                   // masked scores become -inf: exp gives exact zeros
#pragma unroll
                for (int i = 0; i < KPT; ++i) p[i] = (kbase + i > key_lim) ? -INFINITY : p[i];
#pragma unroll
                for (int o = 1; o < KS; ++o)
#pragma unroll
                    for (int i = 0; i < KPT; ++i)
                        po[(o - 1) * KPT + i] = (obase(o) + i > key_lim) ? -INFINITY : po[(o - 1) * KPT + i];
            }
            float mx;
            {
                float t4[KPT / 4];
#pragma unroll
                for (int i = 0; i < KPT / 4; ++i) t4[i] = fmaxf(max3(p[4 * i], p[4 * i + 1], p[4 * i + 2]), p[4 * i + 3]);
                if constexpr (KS > 1) {
#pragma unroll
                    for (int i = 0; i < (BC - KPT) / 4; ++i) {
                        float& t = t4[i % (KPT / 4)];
                        t = fmaxf(max3(t, po[4 * i], po[4 * i + 1]), fmaxf(po[4 * i + 2], po[4 * i + 3]));
                    }
                }
#pragma unroll
                for (int w = KPT / 8; w >= 1; w >>= 1)
#pragma unroll
                    for (int i = 0; i < w; ++i) t4[i] = fmaxf(t4[i], t4[i + w]);
                mx = t4[0];
            }

            const float m_new = fmaxf(m_run, f16_round(mx * args.c0));
            float rsc = 1.f;
            if (jt > 0 && m_new != m_run) rsc = f16_round(ex2_approx((m_run - m_new) * LOG2E));
            m_run = m_new;
            const float mL = m_run * LOG2E;
            const float A = p_of_score<PF32>(mx, args.c1, mL); // = max of P over the group (monotone map)

            // P = exp(S - m) in FP16 (line 9), P-hat = HIF4(P) (line 10)
            uint8_t* dc = nullptr;
            float* ds = nullptr;
            if (DBG && dbg_slot >= 0 && row < N && kbase < N) {
                const size_t r_idx = (size_t)dbg_slot * 128 + r_loc;
                if (args.dbg.p_codes) dc = args.dbg.p_codes + r_idx * N + kbase;
                if (args.dbg.p_step) ds = args.dbg.p_step + r_idx * (N / 4) + kbase / 4;
            }
            // poll for PV(jt-1) now, look at the answer after the exponentials
            const bool pv_ready = jt > 0 ? mbar_test_wait(bar(BAR_PV), par ^ 1u) : true;
            uint32_t w[NU * 4];
            const PQuantConst qc = p_quant_const(args.c1, mL, A);
            exp_quantize_units<NU, 0, NU, DBG, PF32>(p, qc, A == 0.f, w, dc, ds);
            // the P-hat columns and [O | l] are free once PV(jt-1) has completed (every warp observes
            // every phase of that barrier, in order)
            if (jt > 0) {
                if (!pv_ready && !wait64(bar(BAR_PV), par ^ 1u, abort_flag)) { fail(10); ok = false; break; }
                tc_fence_after();
            }
            sf_ready = mbar_test_wait(bar(BAR_SF), par ^ 1u);   // S(jt+1): answer used at the top of the next tile
            if constexpr (NU == 8) tmem_st32(t_lane + P_COL, w);
            else if constexpr (NU == 4) tmem_st16(t_lane + P_COL + kq * (KPT / 2), w);
            else tmem_st8(t_lane + P_COL + kq * (KPT / 2), w);
            // rescale history (line 8): each half of the row's threads owns half of the d + 16 columns
            if constexpr (D == 128 && KS == 2) {            // all of the thread's 72 columns in one round trip
                if (__any_sync(0xffffffffu, rsc != 1.f)) {
                    const uint32_t t_o = t_lane + kq * 72;
                    const uint64_t rr = pack2(rsc, rsc);
                    uint32_t r0[32], r1[32], r2[4], r3[4];
                    tmem_ld32(t_o, r0);
                    tmem_ld32(t_o + 32, r1);
                    tmem_ld4(t_o + 64, r2);
                    tmem_ld4(t_o + 68, r3);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float x0, x1;
                        unpack2(mul2(pack2(__uint_as_float(r0[i]), __uint_as_float(r0[i + 1])), rr), x0, x1);
                        r0[i] = __float_as_uint(x0);
                        r0[i + 1] = __float_as_uint(x1);
                    }
                    tmem_st32(t_o, r0);
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float x0, x1;
                        unpack2(mul2(pack2(__uint_as_float(r1[i]), __uint_as_float(r1[i + 1])), rr), x0, x1);
                        r1[i] = __float_as_uint(x0);
                        r1[i + 1] = __float_as_uint(x1);
                    }
                    tmem_st32(t_o + 32, r1);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        r2[i] = __float_as_uint(__uint_as_float(r2[i]) * rsc);
                        r3[i] = __float_as_uint(__uint_as_float(r3[i]) * rsc);
                    }
                    tmem_st4(t_o + 64, r2);
                    tmem_st4(t_o + 68, r3);
                }
            } else
            if (__any_sync(0xffffffffu, rsc != 1.f)) {
                constexpr int CW = O_COLS / KS;                // 136 or 72
                const uint32_t t_o = t_lane + kq * CW;
                const uint64_t rr = pack2(rsc, rsc);
#pragma unroll
                for (int cc = 0; cc < CW / 32; ++cc) {
                    uint32_t r[32];
                    tmem_ld32(t_o + cc * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float x0, x1;
                        unpack2(mul2(pack2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), rr), x0, x1);
                        r[i] = __float_as_uint(x0);
                        r[i + 1] = __float_as_uint(x1);
                    }
                    tmem_st32(t_o + cc * 32, r);
                }
#pragma unroll
                if constexpr (CW % 32 == 16) {                 // 144 = 4 x 32 + 16: only the l column of the tail matters
                    uint32_t r[4];
                    tmem_ld4(t_o + (CW / 32) * 32, r);
                    tmem_wait_ld();
                    r[0] = __float_as_uint(__uint_as_float(r[0]) * rsc);
                    tmem_st4(t_o + (CW / 32) * 32, r);
                } else {
#pragma unroll
                    for (int cc = 0; cc < (CW % 32) / 4; ++cc) {
                        uint32_t r[4];
                        tmem_ld4(t_o + (CW / 32) * 32 + cc * 4, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 4; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * rsc);
                        tmem_st4(t_o + (CW / 32) * 32 + cc * 4, r);
                    }
                }
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_PF));
        }

        // finalize: out = O / l with l rounded to FP16 (line 13); half kq writes channels (d/2)*kq..
        if (ok && wait64(bar(BAR_PV), (uint32_t)(n_tiles - 1) & 1u, abort_flag)) {
            tc_fence_after();
            uint32_t lr[4];
            tmem_ld4(t_lane + D, lr);
            tmem_wait_ld();
            const float ell = __uint_as_float(lr[0]);
            const float l16 = f16_round(ell);
            // O / l as the correctly rounded quotient from the correctly rounded reciprocal: q0 = O * y,
            // q = fma(fma(-q0, l, O), y, q0) (Markstein's correction step; no value here is near the ends of
            // the FP32 range: l >= 2^-24 is an FP16 value and |O| <= l * max|V|)
            const float rl = __frcp_rn(l16);
            if (DBG && dbg_slot >= 0 && row < N && kq == 0) {
                if (args.dbg.l_out) args.dbg.l_out[dbg_slot * 128 + r_loc] = ell;
                if (args.dbg.m_out) args.dbg.m_out[dbg_slot * 128 + r_loc] = m_run;
            }
            const size_t orow = ((size_t)bh_q * N + row) * D + kq * (D / KS);
            // FP32 output goes through a 32 x 32 transpose in shared memory (the K stages are idle by now:
            // every load has landed and every MMA has completed), so that a warp stores four whole
            // 128-byte lines per instruction instead of 32 pieces of 16 bytes.
            const uint32_t stage = k_s + (uint32_t)warp * 4096u;
#pragma unroll
            for (int cc = 0; cc < D / KS / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(t_lane + kq * (D / KS) + cc * 32, r);
                tmem_wait_ld();
                float o[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float a = __uint_as_float(r[i]);
                    const float q0 = a * rl;
                    o[i] = fmaf(fmaf(-q0, l16, a), rl, q0);
                }
                if (args.out_dtype == HIFA4_F32) {
#pragma unroll
                    for (int c4 = 0; c4 < 8; ++c4)
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};"
                                     ::"r"(stage + lane * 128 + ((c4 ^ (lane & 7)) << 4)), "f"(o[4 * c4]), "f"(o[4 * c4 + 1]),
                                       "f"(o[4 * c4 + 2]), "f"(o[4 * c4 + 3]) : "memory");
                    __syncwarp();
                    const int c4 = lane & 7;
                    float* obase = reinterpret_cast<float*>(args.out) + ((size_t)bh_q * N + q0 + quarter * 32) * D +
                                   kq * (D / KS) + cc * 32 + c4 * 4;
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int rr = it * 4 + (lane >> 3);
                        float4 v;
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                                     : "r"(stage + rr * 128 + ((c4 ^ (rr & 7)) << 4)));
                        if (q0 + quarter * 32 + rr < N) *reinterpret_cast<float4*>(obase + (size_t)rr * D) = v;
                    }
                    __syncwarp();
                } else if (row < N) {
                    uint32_t w[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        if (args.out_dtype == HIFA4_F16) {
                            __half2 t = __floats2half2_rn(o[2 * i], o[2 * i + 1]);
                            w[i] = *reinterpret_cast<uint32_t*>(&t);
                        } else {
                            __nv_bfloat162 t = __floats2bfloat162_rn(o[2 * i], o[2 * i + 1]);
                            w[i] = *reinterpret_cast<uint32_t*>(&t);
                        }
                    }
                    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(args.out) + orow + cc * 32);
#pragma unroll
                    for (int i = 0; i < 4; ++i) dst[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
                }
            }
        } else if (ok) {
            fail(11);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == W_MMA) { __syncwarp(); tmem_dealloc(tmem, TMEM_COLS); }
}

template <int DH, bool DBG, bool PF32, bool QM>
static int launch_ws64(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    using C = WS64<DH>;
    CUtensorMap mq, mk, mv;
    if (!make_bf16_map(&mq, qkv.q_mma, (uint64_t)sh.B * sh.Hq, sh.N, DH, 128)) return HIFA4_ERR_CUDA;
    if (!make_bf16_map(&mk, qkv.k_mma, (uint64_t)sh.B * sh.Hkv, sh.N, DH, C::BC)) return HIFA4_ERR_CUDA;
    if (!make_bf16_map(&mv, qkv.v_mma, (uint64_t)sh.B * sh.Hkv, DH, sh.N, DH)) return HIFA4_ERR_CUDA;
    auto kern = attention_fwd_ws64_kernel<DH, DBG, PF32, QM>;
    static SmemOptIn opt_in;
    if (!opt_in.ensure(kern, C::SMEM_BYTES)) return HIFA4_ERR_CUDA;
    dim3 grid((unsigned)(((sh.N + 127) / 128) * sh.Hq * sh.B));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(C::THREADS);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol.wait in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, mq, mk, mv, args);
    count_launch();
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? HIFA4_OK : HIFA4_ERR_CUDA;
}

template <int DH>
static int launch_ws64_d(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    const bool dbg = args.dbg.n_blocks > 0;
    if (args.p_f32) {                                      // variant: no Q-Mean, d = 128 or 256
        if constexpr (DH == 64) return HIFA4_ERR_UNSUPPORTED;
        else {
            if (args.qmean) return HIFA4_ERR_UNSUPPORTED;
            return dbg ? launch_ws64<DH, true, true, false>(sh, qkv, args, st) : launch_ws64<DH, false, true, false>(sh, qkv, args, st);
        }
    }
    if (args.qmean)
        return dbg ? launch_ws64<DH, true, false, true>(sh, qkv, args, st) : launch_ws64<DH, false, false, true>(sh, qkv, args, st);
    return dbg ? launch_ws64<DH, true, false, false>(sh, qkv, args, st) : launch_ws64<DH, false, false, false>(sh, qkv, args, st);
}

int launch_attention_ws64(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    if (sh.d == 256) return launch_ws64_d<256>(sh, qkv, args, st);
    if (sh.d == 128) return launch_ws64_d<128>(sh, qkv, args, st);
    if (sh.d == 64) return launch_ws64_d<64>(sh, qkv, args, st);
    return HIFA4_ERR_UNSUPPORTED;
}

}  // namespace hifa4
