// Warp-specialised HiFA4 attention forward for Bc = 64 (Algorithm 1 lines 4-13), d = 64, 128 or 256.
//
// One CTA = 128 query rows of one (batch, query head), 10 warps:
//   warps 0-7  softmax / quantize, one thread per query row and key tile: warps 0-3 own the even key
//              tiles, warps 4-7 the odd ones (warp w: rows 32*(w%4).., its tensor-memory lane quarter).
//              The two groups run half a period apart, so that on every scheduler one warp is in its
//              issue-bound phase (exponentials, quantizer) while the other one sits in a latency-bound
//              phase (tensor-memory loads and stores, barrier hand-offs); the running maximum of a row
//              passes from the owner of tile j to the owner of tile j+1 through shared memory, early in
//              tile j (it is known as soon as the row maximum of S(j) is)
//   warp 8     one thread: TMA loads of Q and of the K tiles (two-stage ring), tcgen05 issuer of S = Q K^T
//   warp 9     one thread: TMA loads of the V^T tiles (two-stage ring), issuer of [O | l] += P-hat [V | 1]
// Each of the two issues its MMA, waits for it to complete (which frees the tile's stage) and refills the
// stage two tiles ahead; the next MMA of the same kind cannot start earlier anyway (the next S needs the
// softmax warps to have pulled this S, the next P V needs the P-hat that follows this P V).
// Each MMA waits on ONE barrier: the barrier that releases S of a tile collects the bytes of the K tile
// (TMA transaction count) and the four "S is in registers" arrivals of the group that owns the previous tile,
// the one that releases P V collects the bytes of the V^T tile and the four "P-hat stored, history rescaled"
// arrivals of the tile's owners.  The two issuers run independently: a late P V never delays the next S (device timestamps
// of a single in-order issuer showed S(j+1) issued 1500 clk after it could have been).
// S has a single buffer that is released early: the softmax warps pull S(j) into registers and
// signal it free, and S(j+1) runs on the tensor pipe while they work on tile j; the BF16 image of P-hat
// has its own tensor-memory columns and is the A operand of the P V MMA.
// One tile is one 64-key HIF4 group of P per row, held by one thread: no row statistic is computed twice.
//   d = 256: 512 tensor-memory columns: [O | l] 0..271 (an N = 256 MMA for the channels, an N = 16
//            MMA on the same A operand for the ones block), Q-hat image 272..399 (A operand of
//            Q K^T from tensor memory), S 400..463, P-hat 464..495.  One CTA per SM.
//   d = 64:  as d = 128 with [O | l] 0..79 (one N = 80 MMA); 53 KB of shared memory.
//   d = 128: 256 tensor-memory columns: [O | l] 0..143 (one N = 144 MMA), S 144..207, P-hat
//            208..239; Q-hat stays in shared memory (SS-form Q K^T).  101 KB of shared memory, so two
//            CTAs share an SM and fill each other's synchronisation gaps.
// Every wait polls with test_wait (a thread suspended in try_wait was seen to notice a completed phase about
// 1000 clk late).  Epilogue: O / l by reciprocal plus one correction
// step, FP32 output through a per-warp 32 x 32 shared-memory transpose (the K stages are idle by then).
// The grid is launched with programmatic stream serialization: everything before griddepcontrol.wait
// (barrier set-up, tensor-memory allocation) may overlap the tail of the preceding kernel.
// Template flags: P-hat dump, FP32-P variant, Q-Mean (the K thread stages each tile's key sums in shared memory,
// two tiles ahead), self-test (one wait made to run out), raw Q (Q smoothed and quantized in shared memory by
// the softmax threads before the first S).
// Every wait is bounded (see hifa4_attention_ws.cu for the failure protocol).
#include "hifa4_attention.cuh"

namespace hifa4 {

// F8: the kind::f8f6f4 experiment (d = 128): Q and K tiles are one byte per element, S has one accumulator per
// 64-channel group, 304 tensor-memory columns, hence one CTA per SM.
template <int D_, bool F8 = false>
struct WS64 {
    static constexpr int D = D_, BC = 64, STAGES = 2;
    static constexpr int NSW = 8, THREADS = (NSW + 2) * 32, W_QK = NSW, W_PV = NSW + 1;   // two groups of 4 softmax warps
    static constexpr int NU = BC / 8;                       // 8 level-2 units (64 keys) per thread and tile
    static constexpr int QSUB = D / 64;                     // 64-channel sub-tiles of Q and K
    static constexpr int Q_BYTES = F8 ? 128 * D : QSUB * 16384;
    static constexpr int K_SUB = BC * 128;                  // 64 keys x 64 channels
    static constexpr int K_STAGE = F8 ? BC * D : QSUB * K_SUB;
    static constexpr int V_STAGE = (D + 16) * 128;          // D rows of V^T + 16 rows of ones, 64 keys wide
    static constexpr int Q_OFF = 0;
    static constexpr int K_OFF = Q_OFF + Q_BYTES;
    static constexpr int V_OFF = K_OFF + STAGES * K_STAGE;
    static constexpr int MISC_OFF = V_OFF + STAGES * V_STAGE;
    static constexpr int KSUM_SLOTS = 8;                    // Q-Mean: channel sums of a tile's 64 keys; slot = tile % 8
    static constexpr int KSUM_BYTES = F8 ? 512 : 256;       // (F8: the two group scales of each of the tile's keys instead)
    static constexpr int KSUM_OFF = MISC_OFF + 256;
    static constexpr int MX_OFF = KSUM_OFF + KSUM_SLOTS * KSUM_BYTES;  // running maxima handed from tile j to tile j+1: [2][128] floats
    static constexpr int SMEM_USED = MX_OFF + 2 * 512 + 1024;
    // F8 allocates all 512 tensor-memory columns: it asks for more than half of the SM's shared memory as well, so
    // that a second CTA never becomes resident only to block in the tensor-memory allocator
    static constexpr int SMEM_BYTES = (F8 && SMEM_USED < 120 * 1024) ? 120 * 1024 : SMEM_USED;
    static constexpr int O_COLS = D + 16;
    static constexpr bool Q_IN_TMEM = (D == 256);
    static constexpr int QT_COL = 272;                      // d = 256 only
    static constexpr int S_COL = (D == 256) ? 400 : 144;
    static constexpr int P_COL = S_COL + (F8 ? 128 : 64);
    static constexpr int TMEM_COLS = (D == 256 || F8) ? 512 : 256;
    static constexpr int CTAS_PER_SM = (D == 256 || F8) ? 1 : 2;
};
namespace ws64 {
// Index s = tile % 2 everywhere.  QKGO[s]: K stage s has landed and S is free (4 arrivals + 1 + bytes); PVGO[s]:
// V^T stage s has landed, the image of P-hat is stored and [O | l] rescaled (4 arrivals + 1 + bytes); KE / VE:
// stage free (MMA commit); SF[s]: S complete; PV[s]: P V complete; MR[s]: running maxima after the tile
// published (4 arrivals); KSF[tile % 8]: Q-Mean key sums landed (a barrier per slot); QT: Q-hat image copied to tensor memory.
// Two barriers per kind because each group of softmax warps sees every second tile only: a parity wait
// must observe every phase of its barrier.
enum { BAR_Q = 0, BAR_QKGO = 1, BAR_KE = 3, BAR_PVGO = 5, BAR_VE = 7, BAR_SF = 9, BAR_PV = 11, BAR_KSF = 13,
       BAR_MR = 21, BAR_QT = 23, N_BARS = 24 };
constexpr uint32_t WAIT_POLLS = 1u << 20;
}  // namespace ws64

// Bounded wait with non-blocking polls (softmax warps and issuers: a late wake-up sits on the critical path,
// and a thread suspended in try_wait was seen to notice a completed phase about 1000 clk late).
static __device__ __forceinline__ bool wait64(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                              uint32_t polls = ws64::WAIT_POLLS)
{
#pragma unroll 1
    for (uint32_t i = 0; i < polls; ++i) {
        if (mbar_test_wait(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    return false;
}
// One arrival from lane 0 of a converged warp, without a branch.
static __device__ __forceinline__ void arrive_lane0(uint32_t bar, int lane)
{
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.eq.s32 p, %1, 0;\n\t"
                 "@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}"
                 ::"r"(bar), "r"(lane) : "memory");
}

// SELFTEST: the instantiation behind hifa4_selftest_wait_timeout.  Its softmax warps withhold the arrival that
// releases P V and the issuer's wait for it gives up after 2^12 polls instead of 2^20; by then every TMA load
// has landed and no MMA is in flight, so the CTA leaves through the ordinary failure exit.
// QRAW: the Q tensor map is over the raw 16-bit Q; the softmax threads smooth and HIF4-quantize their CTA's 128 rows
// in shared memory (Algorithm 1 line 1) before the first S = Q K^T, so Q-hat never travels through HBM.
// F8QK: the kind::f8f6f4 experiment.  Q-hat and K-hat arrive as E4M3 images of element x micro-exponent (integers up
// to 28, exact) with one FP32 scale S/4 per (row, 64-channel group); S = Q K^T runs as two accumulators, one per
// channel group, and the softmax threads bind them: acc = (qs0 ks0_j) S0 + (qs1 ks1_j) S1, every product exact and
// the sum rounded once.  Measured against the BF16-image form, not a default path.
template <int DH, bool DBG, bool PF32, bool QM, bool SELFTEST = false, bool QRAW = false, bool F8QK = false>
__global__ void __launch_bounds__(WS64<DH, F8QK>::THREADS, WS64<DH, F8QK>::CTAS_PER_SM)
attention_fwd_ws64_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                           const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ AttnArgs args)
{
    using namespace ws64;
    using C = WS64<DH, F8QK>;
    static_assert(!QRAW || (DH == 128 && !QM && !DBG), "raw-Q launch: d = 128, no Q-Mean, no dump");
    static_assert(!F8QK || (DH == 128 && !QM && !DBG && !QRAW && !SELFTEST), "f8f6f4 experiment: d = 128, plain path");
    constexpr int D = C::D, BC = C::BC, STAGES = C::STAGES, NSW = C::NSW, THREADS = C::THREADS;
    constexpr int W_QK = C::W_QK, W_PV = C::W_PV, NU = C::NU, QSUB = C::QSUB;
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
    // 1-D grid.  The (batch, query head) pairs are taken in groups whose K/V images fit in L2 together (one group
    // when everything fits); inside a group the query block is outermost and descending, so that the heaviest
    // causal CTAs are scheduled first and the CTAs in flight share the K/V of the group's heads.
    const int gh = args.group_heads;                          // divides n_bh
    const int grp_i = (int)blockIdx.x / (n_qt * gh), in_grp = (int)blockIdx.x % (n_qt * gh);
    const int qt = n_qt - 1 - in_grp / gh;
    const int bh = grp_i * gh + in_grp % gh;
    const int h = bh % args.Hq, b = bh / args.Hq;
    const int g = args.map.kv_of[h];
    const int q0 = qt * 128;
    const int bh_q = b * args.Hq + h, bh_kv = b * args.Hkv + g;
    const int last_key = args.causal ? min(q0 + 127, N - 1) : N - 1;
    const int n_tiles = last_key / BC + 1;

    // TMA loads; the bytes of a K tile count on the barrier that releases its S = Q K^T, those of a V^T tile
    // on the barrier that releases its P V (one thread of warp W_QK resp. W_PV calls these)
    auto load_k = [&](int jt) {                               // K tile jt into stage jt % 2
        const int st = jt & 1;
        mbar_expect_tx(bar(BAR_QKGO + st), K_STAGE);
        if constexpr (F8QK) {
            tma_load_3d(k_s + st * K_STAGE, &tmap_k, bar(BAR_QKGO + st), 0, jt * BC, bh_kv);
            // the tile's 64 x 2 key group scales: eight slots with a barrier each, as the Q-Mean key sums below
            mbar_expect_tx(bar(BAR_KSF + (jt & 7)), 512);
            bulk_load(smem_base + C::KSUM_OFF + (jt & 7) * 512, args.k_gs + ((size_t)bh_kv * N + jt * BC) * 2, 512, bar(BAR_KSF + (jt & 7)));
        } else {
#pragma unroll
            for (int s = 0; s < QSUB; ++s)
                tma_load_3d(k_s + st * K_STAGE + s * K_SUB, &tmap_k, bar(BAR_QKGO + st), 64 * s, jt * BC, bh_kv);
        }
        if (QM) {
            // Q-Mean: the 64 channel sums of this tile's keys travel with the K tile, two tiles ahead of their use
            // right after S is pulled (with the V^T tile they arrived ~2000 clk after the softmax warps wanted
            // them).  Eight slots with a barrier each: slot jt % 8 held the sums of tile jt-8, and this load follows
            // S(jt-2), which was released by the group that owns tile jt-3 after it had pulled S(jt-3), which was
            // released by the owners of tile jt-4 - the group that read the slot during tile jt-8 and has finished
            // three tiles since.  (Two barriers by tile parity would not do: the sums of tile jt+2 can land before a
            // late reader has looked for those of tile jt, and a parity wait that is two phases behind never returns.)
            mbar_expect_tx(bar(BAR_KSF + (jt & 7)), 256);
            bulk_load(smem_base + C::KSUM_OFF + (jt & 7) * 256, args.k_sum + (size_t)bh_kv * N + jt * BC, 256, bar(BAR_KSF + (jt & 7)));
        }
    };
    auto load_v = [&](int jt) {                               // V^T tile jt into stage jt % 2
        const int st = jt & 1;
        mbar_expect_tx(bar(BAR_PVGO + st), D * 128);
        tma_load_3d(v_s + st * V_STAGE, &tmap_v, bar(BAR_PVGO + st), jt * BC, 0, bh_kv);
    };

    if (warp == W_QK && lane == 0) {
        // A CTA that starts after another one reported a failure does nothing.  One thread reads the status
        // word and publishes the verdict through shared memory, so that all roles of the CTA agree on it.
        // The same thread sets the barriers up and starts the first loads at once (Q and two K tiles), so that
        // they are in flight while the rest of the CTA sets itself up.
        int status_now = args.d_status ? *reinterpret_cast<volatile int*>(args.d_status) : 0;
        tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_k); tma_prefetch_desc(&tmap_v);
        mbar_init(bar(BAR_Q), 1);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(BAR_QKGO + s), 5); mbar_init(bar(BAR_KE + s), 1);
            mbar_init(bar(BAR_PVGO + s), 5); mbar_init(bar(BAR_VE + s), 1);
            mbar_init(bar(BAR_SF + s), 1); mbar_init(bar(BAR_PV + s), 1);
            for (int t = 0; t < 4; ++t) mbar_init(bar(BAR_KSF + 2 * t + s), 1);
            mbar_init(bar(BAR_MR + s), 4);
        }
        mbar_init(bar(BAR_QT), NSW);
        fence_barrier_init();
        // The launch lets this grid start while its predecessor in the stream is still running; nothing the
        // predecessor wrote is touched before this point.  A non-zero status word read before it may be one
        // that the preceding work in the stream has cleared since: that (rare) verdict is read again.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (status_now != 0) status_now = *reinterpret_cast<volatile int*>(args.d_status);
        *abort_flag = status_now != 0 ? 2 : 0;
        if (status_now == 0) {
            mbar_expect_tx(bar(BAR_Q), Q_BYTES);
            if constexpr (F8QK) {
                tma_load_3d(q_s, &tmap_q, bar(BAR_Q), 0, q0, bh_q);
            } else {
#pragma unroll
                for (int s = 0; s < QSUB; ++s) tma_load_3d(q_s + s * 16384, &tmap_q, bar(BAR_Q), 64 * s, q0, bh_q);
            }
            load_k(0);
            if (n_tiles > 1) load_k(1);
        }
    }
    if (warp == W_QK) { __syncwarp(); tmem_alloc(smem_u32((const void*)tmem_slot), TMEM_COLS); tmem_relinquish(); }
    for (int i = tid; i < STAGES * 128; i += THREADS) {           // ones rows under every V^T stage
        const int st = i / 128, off = (i % 128) * 16;
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};"
                     ::"r"(v_s + st * V_STAGE + D * 128 + off), "r"(0x3F803F80u) : "memory");
    }
    fence_proxy_async_smem();
    tc_fence_before();
    asm volatile("griddepcontrol.wait;" ::: "memory");
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
    } else if (warp == W_QK) {
        // ------------------------------------------------------------------ Q and K loads, issuer of S = Q K^T
        if (lane == 0) {
            constexpr uint32_t idesc_s = umma_idesc_bf16(128, BC);
            const uint32_t q_lo = umma_desc_lo(q_s), k_lo = umma_desc_lo(k_s);
            bool ok = wait64(bar(C::Q_IN_TMEM || QRAW ? BAR_QT : BAR_Q), 0, abort_flag);
            if (!ok) fail(3);
            for (int jt = 0; ok && jt < n_tiles; ++jt) {      // S(jt): K tile landed, S(jt-1) in registers
                const int st = jt & 1;
                const uint32_t ph = (uint32_t)(jt >> 1) & 1u;
                if (!wait64(bar(BAR_QKGO + st), ph, abort_flag)) { fail(4); break; }
                tc_fence_after();
                const uint32_t b0 = k_lo + st * (K_STAGE >> 4);
                if constexpr (F8QK) {
                    constexpr uint32_t idesc_f8 = umma_idesc_e4m3(128, BC);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)             // 32 channels per step; steps 0, 1 -> S0, steps 2, 3 -> S1
                        umma_f8_ss_lo(tmem + S_COL + (kk >> 1) * 64, q_lo + kk * 2, b0 + kk * 2, idesc_f8, kk & 1);
                } else {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {      // D / 16 steps of 16 channels
                        const uint32_t kb = b0 + (kk >> 2) * (K_SUB >> 4) + (kk & 3) * 2;
                        if constexpr (C::Q_IN_TMEM) umma_bf16_ts_lo(tmem + S_COL, tmem + QT_COL + kk * 8, kb, idesc_s, kk ? 1u : 0u);
                        else umma_bf16_ss_lo(tmem + S_COL, q_lo + (kk >> 2) * (16384 >> 4) + (kk & 3) * 2, kb, idesc_s, kk ? 1u : 0u);
                    }
                }
                umma_commit(bar(BAR_SF + st));
                umma_commit(bar(BAR_KE + st));
                if (jt + 2 < n_tiles) {                        // refill the stage once this MMA has read it
                    if (!wait64(bar(BAR_KE + st), ph, abort_flag)) { fail(1); break; }
                    load_k(jt + 2);
                }
            }
        }
    } else if (warp == W_PV) {
        // ------------------------------------------------------------------ V^T loads, issuer of [O | l] += P-hat [V | 1]
        if (lane == 0) {
            constexpr uint32_t idesc_o = umma_idesc_bf16(128, D == 256 ? 256 : O_COLS);
            constexpr uint32_t idesc_l = umma_idesc_bf16(128, 16);
            const uint32_t v_lo = umma_desc_lo(v_s);
            load_v(0);
            if (n_tiles > 1) load_v(1);
            for (int jt = 0; jt < n_tiles; ++jt) {            // V^T tile landed, P-hat(jt) stored, history rescaled
                const int st = jt & 1;
                const uint32_t ph = (uint32_t)(jt >> 1) & 1u;
                if (!wait64(bar(BAR_PVGO + st), ph, abort_flag, SELFTEST ? (1u << 12) : WAIT_POLLS)) { fail(7); break; }
                tc_fence_after();
                const uint32_t b0 = v_lo + st * (V_STAGE >> 4);
                const uint32_t acc0 = jt > 0 ? 1u : 0u;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {                // 16 keys per step; channels (+ ones block)
                    umma_bf16_ts_lo(tmem, tmem + P_COL + kk * 8, b0 + kk * 2, idesc_o, kk ? 1u : acc0);
                    if constexpr (D == 256)                      // N = 272 does not exist: the ones block separately
                        umma_bf16_ts_lo(tmem + 256, tmem + P_COL + kk * 8, b0 + ((D * 128) >> 4) + kk * 2, idesc_l, kk ? 1u : acc0);
                }
                umma_commit(bar(BAR_PV + st));
                umma_commit(bar(BAR_VE + st));
                if (jt + 2 < n_tiles) {                        // refill the stage once this MMA has read it
                    if (!wait64(bar(BAR_VE + st), ph, abort_flag)) { fail(2); break; }
                    load_v(jt + 2);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax / quantize
        const int grp = warp >> 2, quarter = warp & 3;            // tile parity owned, row quarter
        const int kq = grp;                                       // channel half in the Q-hat copy and in the epilogue
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
        float qs0 = 0.f, qs1 = 0.f;                                 // f8f6f4 experiment: the row's two group scales
        if (F8QK && row < N) {
            qs0 = args.q_gs[((size_t)bh_q * N + row) * 2];
            qs1 = args.q_gs[((size_t)bh_q * N + row) * 2 + 1];
        }
        float* mx_s = reinterpret_cast<float*>(smem_gen + C::MX_OFF);   // [2][128]
        float m_run = -INFINITY;
        bool ok = true;

        // d = 256: Q-hat image, shared memory (swizzled TMA tiles) -> tensor memory; this thread moves 128
        // channels of its row = 64 columns of packed BF16 pairs.  (d = 128: the issuer waits for the
        // Q load itself.)
        if constexpr (C::Q_IN_TMEM) {
            if (wait64(bar(BAR_Q), 0, abort_flag)) {
                const int sw = r_loc & 7;
#pragma unroll
                for (int half = 0; half < 2; ++half) {             // pieces of 64 channels (8 chunks, 32 columns)
                    uint32_t qw[32];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int chunk = (kq * 2 + half) * 8 + c;     // 16-byte chunk of the 512-byte row
                        const uint32_t a = q_s + (chunk >> 3) * 16384 + (r_loc >> 3) * 1024 + sw * 128 + (((chunk & 7) ^ sw) << 4);
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(qw[4 * c]), "=r"(qw[4 * c + 1]), "=r"(qw[4 * c + 2]), "=r"(qw[4 * c + 3]) : "r"(a));
                    }
                    tmem_st32(t_lane + QT_COL + (kq * 2 + half) * 32, qw);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                arrive_lane0(bar(BAR_QT), lane);
            } else { fail(13); ok = false; }
        }
        if constexpr (QRAW) {
            // Q-hat = HIF4(round(Q s)) in place (Algorithm 1 line 1): thread (row, kq) owns the row's 64-channel group kq
            if (wait64(bar(BAR_Q), 0, abort_flag)) {
                const uint32_t row_addr = q_s + (uint32_t)kq * 16384u + (uint32_t)r_loc * 128u;
                const float* sc = args.q_scale ? args.q_scale + (size_t)g * D + kq * 64 : nullptr;
                if (args.in_dtype == HIFA4_F16) hif4_quantize_row64_inplace<__half>(row_addr, r_loc & 7, sc);
                else hif4_quantize_row64_inplace<__nv_bfloat16>(row_addr, r_loc & 7, sc);
            } else { fail(13); ok = false; }
            fence_proxy_async_smem();                          // generic-proxy writes, read by the MMA
            __syncwarp();
            arrive_lane0(bar(BAR_QT), lane);
        }
        if (grp == 0) arrive_lane0(bar(BAR_QKGO), lane);          // S is free for tile 0

        for (int jt = grp; ok && jt < n_tiles; jt += 2) {
            const int j0 = jt * BC;
            const int st = jt & 1;                                 // = grp
            const uint32_t ph = (uint32_t)(jt >> 1) & 1u;          // phase parity of this group's barriers
            if (!wait64(bar(BAR_SF + st), ph, abort_flag)) { fail(8); ok = false; break; }
            tc_fence_after();
            float p[BC];
            if constexpr (F8QK) {
                // bind the two per-group integer sums: acc = (qs0 ks0_j) S0 + (qs1 ks1_j) S1.  The scales have 3
                // significant bits, the sums at most 16: both products are exact, the sum is rounded once.
                if (!wait64(bar(BAR_KSF + (jt & 7)), (uint32_t)(jt >> 3) & 1u, abort_flag)) { fail(15); ok = false; break; }
                const uint32_t ks_s = smem_base + C::KSUM_OFF + (jt & 7) * 512;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {               // 32 keys at a time
                    uint32_t r0[32], r1[32];
                    tmem_ld32(t_lane + S_COL + 32 * hh, r0);
                    tmem_ld32(t_lane + S_COL + 64 + 32 * hh, r1);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float4 ks;                             // ks0_j, ks1_j, ks0_{j+1}, ks1_{j+1}
                        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(ks.x), "=f"(ks.y), "=f"(ks.z), "=f"(ks.w) : "r"(ks_s + 8 * (32 * hh + i)));
                        p[32 * hh + i] = fmaf(qs1 * ks.y, __uint_as_float(r1[i]), (qs0 * ks.x) * __uint_as_float(r0[i]));
                        p[32 * hh + i + 1] = fmaf(qs1 * ks.w, __uint_as_float(r1[i + 1]), (qs0 * ks.z) * __uint_as_float(r0[i + 1]));
                    }
                }
            } else {
                uint32_t r[BC];
                tmem_ld32(t_lane + S_COL, reinterpret_cast<uint32_t(&)[32]>(r[0]));
                tmem_ld32(t_lane + S_COL + 32, reinterpret_cast<uint32_t(&)[32]>(r[32]));
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < BC; ++i) p[i] = __uint_as_float(r[i]);
            }
            tc_fence_before();                                 // S(jt) is in registers: S(jt+1) may overwrite it
            __syncwarp();
            if (jt + 1 < n_tiles) arrive_lane0(bar(BAR_QKGO + (st ^ 1)), lane);

            if (QM) {                                          // Q-Mean correction (line 6): + mu_i * sum_c k~_jc
                if (!wait64(bar(BAR_KSF + (jt & 7)), (uint32_t)(jt >> 3) & 1u, abort_flag)) { fail(15); ok = false; break; }
                const uint32_t ks_s = smem_base + C::KSUM_OFF + (jt & 7) * 256;
                const uint64_t mu2 = pack2(mu_row, mu_row);
#pragma unroll
                for (int i = 0; i < BC / 4; ++i) {
                    float4 ks;
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                 : "=f"(ks.x), "=f"(ks.y), "=f"(ks.z), "=f"(ks.w) : "r"(ks_s + 16 * i));
                    unpack2(fma2(mu2, pack2(ks.x, ks.y), pack2(p[4 * i], p[4 * i + 1])), p[4 * i], p[4 * i + 1]);
                    unpack2(fma2(mu2, pack2(ks.z, ks.w), pack2(p[4 * i + 2], p[4 * i + 3])), p[4 * i + 2], p[4 * i + 3]);
                }
            }
            if ((args.causal && (j0 + BC - 1 > q0)) || (j0 + BC > N)) {   // masked scores become -inf: exp gives exact zeros
#pragma unroll
                for (int i = 0; i < BC; ++i) p[i] = (j0 + i > key_lim) ? -INFINITY : p[i];
            }
            // row maximum = maximum of the tile's single 64-key group: eight chains of eight values
            // (three-input maxima), then one chain over the eight
            float mx;
            {
                float t8[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    float t = max3(p[8 * c], p[8 * c + 1], p[8 * c + 2]);
                    t = max3(t, p[8 * c + 3], p[8 * c + 4]);
                    t = max3(t, p[8 * c + 5], p[8 * c + 6]);
                    t8[c] = fmaxf(t, p[8 * c + 7]);
                }
                mx = max3(t8[0], t8[1], t8[2]);
                mx = max3(mx, t8[3], t8[4]);
                mx = max3(mx, t8[5], t8[6]);
                mx = fmaxf(mx, t8[7]);
            }
            // running maximum after the previous tile, from its owner (the other group)
            if (jt > 0) {
                if (!wait64(bar(BAR_MR + (st ^ 1)), (uint32_t)((jt - 1) >> 1) & 1u, abort_flag)) { fail(12); ok = false; break; }
                m_run = mx_s[(st ^ 1) * 128 + r_loc];
            }
            // running maximum and rescale factor (lines 7-8), both FP16 values.  No branch: r = 1 exactly
            // when the maximum did not move; at jt = 0 (m = -inf) r = 0 is never applied.
            const float m_new = fmaxf(m_run, f16_round(mx * args.c0));
            if (jt + 1 < n_tiles) {                            // hand it to the owner of the next tile
                mx_s[st * 128 + r_loc] = m_new;
                __syncwarp();
                arrive_lane0(bar(BAR_MR + st), lane);
            }
            const float rsc = f16_round(ex2_approx((m_run - m_new) * LOG2E));
            m_run = m_new;
            const float mL = m_run * LOG2E;
            const float A = p_of_score<PF32>(mx, args.c1, mL); // = max of P over the group (monotone map)

            // P = exp(S - m) in FP16 (line 9), P-hat = HIF4(P) (line 10)
            uint8_t* dc = nullptr;
            float* ds = nullptr;
            if (DBG && dbg_slot >= 0 && row < N && j0 < N) {
                const size_t r_idx = (size_t)dbg_slot * 128 + r_loc;
                if (args.dbg.p_codes) dc = args.dbg.p_codes + r_idx * N + j0;
                if (args.dbg.p_step) ds = args.dbg.p_step + r_idx * (N / 4) + j0 / 4;
            }
            uint32_t w[NU * 4];
            const PQuantConst qc = p_quant_const(args.c1, mL, A);
            exp_quantize_units<NU, 0, NU, DBG, PF32>(p, qc, A == 0.f, w, dc, ds);
            // the P-hat columns and [O | l] are free once P V of the previous tile has completed
            if (jt > 0) {
                if (!wait64(bar(BAR_PV + (st ^ 1)), (uint32_t)((jt - 1) >> 1) & 1u, abort_flag)) { fail(10); ok = false; break; }
                tc_fence_after();
            }
            tmem_st32(t_lane + P_COL, w);
            // rescale of the history (line 8): the d channels and the normaliser column (the other columns of
            // the ones block are never read)
            if (jt > 0 && __any_sync(0xffffffffu, rsc != 1.f)) {
                const uint64_t rr = pack2(rsc, rsc);
                auto scale32 = [&](uint32_t (&r)[32]) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float x0, x1;
                        unpack2(mul2(pack2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), rr), x0, x1);
                        r[i] = __float_as_uint(x0);
                        r[i + 1] = __float_as_uint(x1);
                    }
                };
                uint32_t rl[1];
                tmem_ld1(t_lane + D, rl);
#pragma unroll
                for (int cc = 0; cc < D / 64; ++cc) {          // 64 columns per round trip
                    uint32_t r0[32], r1[32];
                    tmem_ld32(t_lane + cc * 64, r0);
                    tmem_ld32(t_lane + cc * 64 + 32, r1);
                    tmem_wait_ld();
                    scale32(r0);
                    tmem_st32(t_lane + cc * 64, r0);
                    scale32(r1);
                    tmem_st32(t_lane + cc * 64 + 32, r1);
                }
                rl[0] = __float_as_uint(__uint_as_float(rl[0]) * rsc);
                tmem_st1(t_lane + D, rl);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (!SELFTEST) arrive_lane0(bar(BAR_PVGO + st), lane);
        }

        // finalize: out = O / l with l rounded to FP16 (line 13); half kq writes channels (d/2)*kq..
        if (ok && wait64(bar(BAR_PV + ((n_tiles - 1) & 1)), (uint32_t)((n_tiles - 1) >> 1) & 1u, abort_flag)) {
            tc_fence_after();
            constexpr int NC = D / 2 / 32;                     // 32-column chunks of this thread's channel half
            uint32_t lr[4], rbuf[2][32];
            tmem_ld4(t_lane + D, lr);
            tmem_ld32(t_lane + kq * (D / 2), rbuf[0]);         // the next chunk is always in flight under the current one
            tmem_wait_ld();
            const float ell = __uint_as_float(lr[0]);
            const float l16 = f16_round(ell);
            // O / l as the correctly rounded quotient from the correctly rounded reciprocal: q0 = O * y,
            // q = fma(fma(-q0, l, O), y, q0) (Markstein's correction step; no value here is near the ends of
            // the FP32 range: l >= 2^-24 is an FP16 value and |O| <= l * max|V|)
            const float rl = __frcp_rn(l16);
            if (DBG && dbg_slot >= 0 && row < N && grp == ((n_tiles - 1) & 1)) {   // the owner of the last tile
                if (args.dbg.l_out) args.dbg.l_out[dbg_slot * 128 + r_loc] = ell;
                if (args.dbg.m_out) args.dbg.m_out[dbg_slot * 128 + r_loc] = m_run;
            }
            const size_t orow = ((size_t)bh_q * N + row) * D + kq * (D / 2);
            // FP32 output goes through a 32 x 32 transpose in shared memory (the K stages are idle by now:
            // every load has landed and every MMA has completed), so that a warp stores four whole
            // 128-byte lines per instruction instead of 32 pieces of 16 bytes.
            const uint32_t stage = k_s + (uint32_t)warp * 4096u;
#pragma unroll
            for (int cc = 0; cc < NC; ++cc) {
                uint32_t (&r)[32] = rbuf[cc & 1];
                if (cc + 1 < NC) tmem_ld32(t_lane + kq * (D / 2) + (cc + 1) * 32, rbuf[(cc + 1) & 1]);
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
                                   kq * (D / 2) + cc * 32 + c4 * 4;
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
                if (cc + 1 < NC) tmem_wait_ld();
            }
        } else if (ok) {
            fail(11);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == W_QK) { __syncwarp(); tmem_dealloc(tmem, TMEM_COLS); }
}

bool make_u8_map(CUtensorMap* m, void* base, uint64_t heads, uint64_t rows, uint64_t cols, uint32_t box_rows);

template <int DH, bool DBG, bool PF32, bool QM, bool SELFTEST = false, bool QRAW = false, bool F8QK = false>
static int launch_ws64(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    using C = WS64<DH, F8QK>;
    CUtensorMap mq, mk, mv;
    if constexpr (F8QK) {
        if (!make_u8_map(&mq, const_cast<void*>(args.q_f8), (uint64_t)sh.B * sh.Hq, sh.N, DH, 128)) return HIFA4_ERR_CUDA;
        if (!make_u8_map(&mk, const_cast<void*>(args.k_f8), (uint64_t)sh.B * sh.Hkv, sh.N, DH, C::BC)) return HIFA4_ERR_CUDA;
    } else {
        if (!make_bf16_map(&mq, QRAW ? const_cast<void*>(args.q_raw) : qkv.q_mma, (uint64_t)sh.B * sh.Hq, sh.N, DH, 128)) return HIFA4_ERR_CUDA;
        if (!make_bf16_map(&mk, qkv.k_mma, (uint64_t)sh.B * sh.Hkv, sh.N, DH, C::BC)) return HIFA4_ERR_CUDA;
    }
    if (!make_bf16_map(&mv, qkv.v_mma, (uint64_t)sh.B * sh.Hkv, DH, sh.N, DH)) return HIFA4_ERR_CUDA;
    auto kern = attention_fwd_ws64_kernel<DH, DBG, PF32, QM, SELFTEST, QRAW, F8QK>;
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
    if (args.q_f8) {                                       // the kind::f8f6f4 experiment: d = 128, plain path only
        if constexpr (DH != 128) return HIFA4_ERR_UNSUPPORTED;
        else {
            if (dbg || args.qmean || args.p_f32 || args.q_raw) return HIFA4_ERR_UNSUPPORTED;
            return launch_ws64<DH, false, false, false, false, false, true>(sh, qkv, args, st);
        }
    }
    if (args.q_raw) {                                      // Q quantized in the kernel: d = 128, no Q-Mean, no dump
        if constexpr (DH != 128) return HIFA4_ERR_UNSUPPORTED;
        else {
            if (dbg || args.qmean) return HIFA4_ERR_UNSUPPORTED;
            if (args.p_f32) return launch_ws64<DH, false, true, false, false, true>(sh, qkv, args, st);
            return launch_ws64<DH, false, false, false, false, true>(sh, qkv, args, st);
        }
    }
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

int launch_attention_ws64_selftest(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    if (sh.d != 128) return HIFA4_ERR_UNSUPPORTED;
    return launch_ws64<128, false, false, false, true>(sh, qkv, args, st);
}

int launch_attention_ws64(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    if (sh.d == 256) return launch_ws64_d<256>(sh, qkv, args, st);
    if (sh.d == 128) return launch_ws64_d<128>(sh, qkv, args, st);
    if (sh.d == 64) return launch_ws64_d<64>(sh, qkv, args, st);
    return HIFA4_ERR_UNSUPPORTED;
}

}  // namespace hifa4
