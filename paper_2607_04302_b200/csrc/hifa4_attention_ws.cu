// Warp-specialised HiFA4 attention forward for d = 128, Bc = 128 (Algorithm 1 lines 4-13).
//
// Persistent kernel: one CTA per SM walks a static list of work items (128 query rows of one (batch,
// query head) each), heaviest first; the tile stream runs through item boundaries, so the next item's Q
// load, its copy to tensor memory and its first S tiles overlap the tail and the epilogue of the current
// one.  4*KS + 2 warps per CTA (KS = 2 or 4):
//   warps 0..4*KS-1  softmax / quantize: warp w owns rows 32*(w%4).. of the tile and keys
//              (128/KS)*(w/4).. of every 128-key tile.  With KS = 2 a thread holds one whole
//              64-key HIF4 group of one row; with KS = 4 half a group (4 level-2 units).  The
//              threads of a row publish their partial score maxima in shared memory; the row
//              maximum and the group maximum both come from those
//   next warp  TMA producer: Q once, then K and V^T tiles through two-stage rings
//   last warp  tcgen05 issuer
// Tensor memory: [O | l] in columns 0..143, the Q-hat image in 144..207, two S buffers of 128
// columns at 256 and 384.  S = Q K^T of tile j+2 is issued right after PV of tile j, so the tensor
// pipe always has work queued.  The softmax warps pull S(j) into registers and write the BF16 image
// of P-hat(j) back over the first 64 columns of the same buffer; both GEMMs take their A operand
// from tensor memory (Q-hat, P-hat) and only K and V^T (with its rows of ones) from shared memory.
// MMAs issued by one thread complete in order, which is what makes the buffer reuse safe: S(j+2)
// is issued after PV(j), whose A operand is P-hat(j).
// Every wait is bounded; a wait that expires raises the abort flag, writes the status word and
// every role falls through to the common exit (tensor memory is freed).
#include "hifa4_attention.cuh"

namespace hifa4 {

namespace ws {
constexpr int D = 128, BC = 128, STAGES = 2;
constexpr int Q_BYTES = 2 * 16384;
constexpr int K_STAGE = 2 * 16384;
constexpr int V_CHUNK = (D + 16) * 128;             // 128 rows of V^T + 16 rows of ones, 64 keys wide
constexpr int V_STAGE = 2 * V_CHUNK;
constexpr int Q_OFF = 0;
constexpr int K_OFF = Q_OFF + 2 * Q_BYTES;        // two Q buffers: the next item's Q loads during this one
constexpr int V_OFF = K_OFF + STAGES * K_STAGE;
constexpr int MISC_OFF = V_OFF + STAGES * V_STAGE;  // barriers, tmem slot, abort flag
constexpr int XCHG_OFF = MISC_OFF + 256;            // partial row maxima [2 parities][4 splits][128 rows]
constexpr int XCHG_BYTES = 2 * 4 * 128 * 4;
constexpr int STG_OFF = XCHG_OFF + XCHG_BYTES;      // per softmax warp: 8 rows x 128 bytes of output staging
constexpr int SMEM_BYTES = STG_OFF + 16 * 1024 + 1024;
constexpr int O_COLS = D + 16, QT_COL = 144, S_COL = 256, TMEM_COLS = 512;
enum { BAR_QFULL = 0, BAR_QFREE = 2, BAR_KF = 4, BAR_KE = 6, BAR_VF = 8, BAR_VE = 10, BAR_SF = 12,
       BAR_PF = 14, BAR_PV = 16, BAR_X = 17, BAR_QT = 25, N_BARS = 26 };
constexpr uint32_t WAIT_POLLS = 1u << 20;           // each poll blocks for a hardware-defined slice
}  // namespace ws

// Bounded waits.  wait_or_abort polls without blocking (softmax warps and the issuer: a late wake-up sits on
// the critical path, and a thread suspended in try_wait was seen to notice a completed phase about 1000 clk
// late).  wait_sleepy lets the hardware suspend the thread for up to a few microseconds per poll, for the
// producer warp, which waits most of the time and has slack.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
#pragma unroll 1
    for (uint32_t i = 0; i < ws::WAIT_POLLS; ++i) {
        if (mbar_test_wait(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    return false;
}
__device__ __forceinline__ bool wait_sleepy(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (uint32_t i = 0; i < ws::WAIT_POLLS / 4; ++i) {
        if (mbar_try_wait_hint(bar, parity, 4000u)) return true;
        if (*abort_flag) return false;
    }
    return false;
}

// One unit of work: 128 query rows of one (batch, query head).
struct WorkItem {
    int qt, h, b, q0, bh_q, bh_kv, n_tiles;
};

// Persistent schedule.  Items are ordered heaviest first (query block descending, all heads and
// batches of a query block together: with a causal mask the work of an item grows with its query
// block).  CTA c of G takes one item per "wave" of G consecutive items, walking the waves in
// alternating direction (c, 2G-1-c, 2G+c, ...), which evens out the totals without a global counter.
struct Schedule {
    int G, c, n_items, n_bh, n_qt, N, causal;
    __device__ __forceinline__ int count() const
    {
        const int full = n_items / G, rem = n_items % G;
        const int pos = (full & 1) ? (G - 1 - c) : c;          // position inside the last, partial wave
        return full + (pos < rem ? 1 : 0);
    }
    __device__ __forceinline__ WorkItem item(int k, const AttnArgs& a) const
    {
        const int idx = k * G + ((k & 1) ? (G - 1 - c) : c);
        WorkItem w;
        w.qt = n_qt - 1 - idx / n_bh;
        const int bh = idx % n_bh;
        w.h = bh % a.Hq;
        w.b = bh / a.Hq;
        w.q0 = w.qt * 128;
        w.bh_q = w.b * a.Hq + w.h;
        w.bh_kv = w.b * a.Hkv + a.map.kv_of[w.h];
        const int last_key = causal ? min(w.q0 + 127, N - 1) : N - 1;
        w.n_tiles = last_key / ws::BC + 1;
        return w;
    }
};

template <int KS, bool DBG, bool QM>
__global__ void __launch_bounds__((4 * KS + 2) * 32, 1)
attention_fwd_ws_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                        const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ AttnArgs args)
{
    using namespace ws;
    constexpr int NSW = 4 * KS;                 // softmax warps
    constexpr int THREADS = (NSW + 2) * 32;
    constexpr int W_TMA = NSW, W_MMA = NSW + 1;
    constexpr int KPT = BC / KS;                // keys per thread and tile
    constexpr int NU = KPT / 8;                 // level-2 units per thread
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_s = smem_base + Q_OFF, k_s = smem_base + K_OFF, v_s = smem_base + V_OFF,
                   bars = smem_base + MISC_OFF;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + MISC_OFF + 8 * N_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + MISC_OFF + 8 * N_BARS + 8);
    float* xmax = reinterpret_cast<float*>(smem_gen + XCHG_OFF);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = args.N;
    Schedule sched;
    sched.G = (int)gridDim.x; sched.c = (int)blockIdx.x;
    sched.n_qt = (N + 127) / 128; sched.n_bh = args.B * args.Hq;
    sched.n_items = sched.n_qt * sched.n_bh; sched.N = N; sched.causal = args.causal;
    const int n_my = sched.count();             // items of this CTA

    if (tid == 0) {
        // A CTA that starts after another one reported a failure does nothing.  One thread reads the status
        // word and publishes the verdict through shared memory, so that all roles of the CTA agree on it
        // and leave through the common exit that frees tensor memory.
        *abort_flag = (args.d_status && *reinterpret_cast<volatile int*>(args.d_status) != 0) ? 2 : 0;
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(BAR_QFULL + s), 1); mbar_init(bar(BAR_QFREE + s), NSW);
            mbar_init(bar(BAR_KF + s), 1); mbar_init(bar(BAR_KE + s), 1);
            mbar_init(bar(BAR_VF + s), 1); mbar_init(bar(BAR_VE + s), 1);
            mbar_init(bar(BAR_SF + s), 1); mbar_init(bar(BAR_PF + s), NSW);
        }
        mbar_init(bar(BAR_PV), 1); mbar_init(bar(BAR_QT), NSW);
        for (int i = 0; i < 8; ++i) mbar_init(bar(BAR_X + i), KS);
        fence_barrier_init();
    }
    if (warp == W_MMA) { tmem_alloc(smem_u32((const void*)tmem_slot), TMEM_COLS); tmem_relinquish(); }
    if (warp == W_TMA && lane == 0) { tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_k); tma_prefetch_desc(&tmap_v); }
    for (int i = tid; i < STAGES * 2 * 128; i += THREADS) {      // ones rows under every V^T chunk
        const int chunk = i / 128, off = (i % 128) * 16;
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};"
                     ::"r"(v_s + chunk * V_CHUNK + D * 128 + off), "r"(0x3F803F80u) : "memory");
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const bool dead = *abort_flag != 0;

    auto fail = [&](int site) {
        *abort_flag = 1;
        if (args.d_status) atomicCAS(args.d_status, 0, HIFA4_ERR_TIMEOUT + 16 * site);
    };

    // Tiles are numbered globally across the items of this CTA (g = 0, 1, ...): ring stages, S buffers
    // and barrier phases follow g, so the tile stream runs through item boundaries without a drain.
    if (dead) {
        // fall through to the common exit
    } else if (warp == W_TMA) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int g = 0;
            bool ok = true;
            for (int k = 0; ok && k < n_my; ++k) {
                const WorkItem it = sched.item(k, args);
                const int qb = k & 1;                      // Q buffer: free once its image sits in tensor memory
                if (!wait_sleepy(bar(BAR_QFREE + qb), ((uint32_t)(k >> 1) & 1u) ^ 1u, abort_flag)) { fail(14); break; }
                mbar_expect_tx(bar(BAR_QFULL + qb), Q_BYTES);
                tma_load_3d(q_s + qb * Q_BYTES, &tmap_q, bar(BAR_QFULL + qb), 0, it.q0, it.bh_q);
                tma_load_3d(q_s + qb * Q_BYTES + 16384, &tmap_q, bar(BAR_QFULL + qb), 64, it.q0, it.bh_q);
                for (int jt = 0; jt < it.n_tiles; ++jt, ++g) {
                    const int st = g & 1;
                    const uint32_t ph = (uint32_t)(g >> 1) & 1u;
                    const int j0 = jt * BC;
                    if (!wait_sleepy(bar(BAR_KE + st), ph ^ 1u, abort_flag)) { fail(1); ok = false; break; }
                    mbar_expect_tx(bar(BAR_KF + st), K_STAGE);
                    tma_load_3d(k_s + st * K_STAGE, &tmap_k, bar(BAR_KF + st), 0, j0, it.bh_kv);
                    tma_load_3d(k_s + st * K_STAGE + 16384, &tmap_k, bar(BAR_KF + st), 64, j0, it.bh_kv);
                    if (!wait_sleepy(bar(BAR_VE + st), ph ^ 1u, abort_flag)) { fail(2); ok = false; break; }
                    mbar_expect_tx(bar(BAR_VF + st), 2 * D * 128);
                    tma_load_3d(v_s + st * V_STAGE, &tmap_v, bar(BAR_VF + st), j0, 0, it.bh_kv);
                    tma_load_3d(v_s + st * V_STAGE + V_CHUNK, &tmap_v, bar(BAR_VF + st), j0 + 64, 0, it.bh_kv);
                }
            }
        }
    } else if (warp == W_MMA) {
        // ------------------------------------------------------------------ tcgen05 issuer
        // The whole warp runs the loop and the waits (warp-uniform control flow keeps the operand
        // arithmetic cheap); one elected lane issues the MMAs and the commits.  S = Q K^T runs two
        // tiles ahead of PV, across item boundaries.
        constexpr uint32_t idesc_s = umma_idesc_bf16(128, BC);
        constexpr uint32_t idesc_o = umma_idesc_bf16(128, O_COLS);
        const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
        const uint32_t k_lo = umma_desc_lo(k_s), v_lo = umma_desc_lo(v_s);
        const bool leader = elect_one();
        int qk_item = 0, qk_jt = 0, qk_g = 0;
        int qk_n = n_my > 0 ? sched.item(0, args).n_tiles : 0;
        bool ok = true;
        auto qk_next = [&]() {                        // S(qk_g) -> buffer qk_g % 2 from K stage qk_g % 2
            if (!ok || qk_item >= n_my) return;
            if (qk_jt == 0 && !wait_or_abort(bar(BAR_QT), (uint32_t)qk_item & 1u, abort_flag)) { if (leader) fail(3); ok = false; return; }
            const int st = qk_g & 1;
            if (!wait_or_abort(bar(BAR_KF + st), (uint32_t)(qk_g >> 1) & 1u, abort_flag)) { if (leader) fail(4); ok = false; return; }
            tc_fence_after();
            const uint32_t d = tm + S_COL + st * 128;
            const uint32_t b0 = k_lo + st * (K_STAGE >> 4);
            if (leader) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)               // 16 channels per step = 8 columns of the Q image
                    umma_bf16_ts_lo(d, tm + QT_COL + kk * 8, b0 + (kk >> 2) * (16384 >> 4) + (kk & 3) * 2, idesc_s,
                                    kk ? 1u : 0u);
                umma_commit(bar(BAR_SF + st));
                umma_commit(bar(BAR_KE + st));
            }
            __syncwarp();
            ++qk_g;
            if (++qk_jt == qk_n) {
                qk_jt = 0;
                if (++qk_item < n_my) qk_n = sched.item(qk_item, args).n_tiles;
            }
        };
        qk_next();
        qk_next();
        int g = 0;
        for (int k = 0; ok && k < n_my; ++k) {
            const int n_tiles = sched.item(k, args).n_tiles;
            for (int jt = 0; ok && jt < n_tiles; ++jt, ++g) {
                const int st = g & 1;
                const uint32_t ph = (uint32_t)(g >> 1) & 1u;
                if (!wait_or_abort(bar(BAR_VF + st), ph, abort_flag)) { if (leader) fail(6); ok = false; break; }
                if (!wait_or_abort(bar(BAR_PF + st), ph, abort_flag)) { if (leader) fail(7); ok = false; break; }
                tc_fence_after();
                const uint32_t a0 = tm + S_COL + st * 128;
                const uint32_t b0 = v_lo + st * (V_STAGE >> 4);
                const uint32_t acc0 = jt > 0 ? 1u : 0u;        // the first PV of an item overwrites [O | l]
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)          // 16 keys per step = 8 columns of packed BF16 pairs
                        umma_bf16_ts_lo(tm, a0 + kk * 8, b0 + (kk >> 2) * (V_CHUNK >> 4) + (kk & 3) * 2, idesc_o,
                                        kk ? 1u : acc0);
                    umma_commit(bar(BAR_PV));
                    umma_commit(bar(BAR_VE + st));
                }
                __syncwarp();
                qk_next();
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax / quantize
        const int kq = warp >> 2, quarter = warp & 3;             // key split, row quarter
        const int r_loc = quarter * 32 + lane;                    // row inside the tile = TMEM lane
        const uint32_t t_lane = tmem + ((uint32_t)(quarter * 32) << 16);
        const float LOG2E = 1.4426950408889634f;
        bool ok = true;

        // Q-hat image of item k: shared memory (swizzled TMA tile) -> tensor memory, so that S = Q K^T
        // reads its A operand from tensor memory and only K from shared memory.  This thread moves
        // 128 / KS channels of its row = 64 / KS columns of packed BF16 pairs.  Callers make sure every
        // QK of the previous item has completed (they have seen S of its last tile).
        auto copy_q = [&](int k) -> bool {
            const int qb = k & 1;
            if (!wait_or_abort(bar(BAR_QFULL + qb), (uint32_t)(k >> 1) & 1u, abort_flag)) { fail(13); return false; }
            constexpr int QC = 64 / KS;
            uint32_t qw[QC];
            const int sw = r_loc & 7;
#pragma unroll
            for (int c = 0; c < QC / 4; ++c) {
                const int chunk = kq * (QC / 4) + c;               // 16-byte chunk of the 256-byte row
                const uint32_t a = q_s + qb * Q_BYTES + (chunk >> 3) * 16384 + (r_loc >> 3) * 1024 + sw * 128 +
                                   (((chunk & 7) ^ sw) << 4);
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(qw[4 * c]), "=r"(qw[4 * c + 1]), "=r"(qw[4 * c + 2]), "=r"(qw[4 * c + 3]) : "r"(a));
            }
            if constexpr (KS == 2) tmem_st32(t_lane + QT_COL + kq * QC, qw);
            else tmem_st16(t_lane + QT_COL + kq * QC, qw);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(bar(BAR_QT)); mbar_arrive(bar(BAR_QFREE + qb)); }
            return true;
        };

        // The scores of the next tile are pulled into registers, reduced and published while the
        // current tile is still being quantized (S is double-buffered), so the row-maximum exchange of
        // a tile is usually complete by the time its turn comes and the KS warps of a row quarter need
        // not run in phase.  g: global tile index; jt, q0: the tile's place in its own item.
        auto fetch_scores = [&](int g, int jt, int q0, float mu, int bh_kv, float (&sc)[KPT]) -> float {
            const int j0 = jt * BC, kb = j0 + kq * KPT;
            const int key_lim = args.causal ? min(q0 + r_loc, N - 1) : N - 1;
            const uint32_t t_src = t_lane + S_COL + (g & 1) * 128 + kq * KPT;
#pragma unroll
            for (int cc = 0; cc < KPT / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(t_src + cc * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) sc[cc * 32 + i] = __uint_as_float(r[i]);
            }
            if (QM && kb < N) {                                // Q-Mean correction (line 6): + mu_i * sum_c k~_jc
                const float4* kp = reinterpret_cast<const float4*>(args.k_sum + (size_t)bh_kv * N + kb);
#pragma unroll
                for (int i = 0; i < KPT / 4; ++i) {
                    const float4 ks = __ldg(kp + i);
                    sc[4 * i] = fmaf(mu, ks.x, sc[4 * i]);
                    sc[4 * i + 1] = fmaf(mu, ks.y, sc[4 * i + 1]);
                    sc[4 * i + 2] = fmaf(mu, ks.z, sc[4 * i + 2]);
                    sc[4 * i + 3] = fmaf(mu, ks.w, sc[4 * i + 3]);
                }
            }
            const bool need_mask = (args.causal && (j0 + BC - 1 > q0)) || (j0 + BC > N);
            if (need_mask) {                                   // masked scores become -inf: exp gives exact zeros
#pragma unroll
                for (int i = 0; i < KPT; ++i) sc[i] = (kb + i > key_lim) ? -INFINITY : sc[i];
            }
            float t4[KPT / 4];
#pragma unroll
            for (int i = 0; i < KPT / 4; ++i) t4[i] = fmaxf(max3(sc[4 * i], sc[4 * i + 1], sc[4 * i + 2]), sc[4 * i + 3]);
#pragma unroll
            for (int w = KPT / 8; w >= 1; w >>= 1)
#pragma unroll
                for (int i = 0; i < w; ++i) t4[i] = fmaxf(t4[i], t4[i + w]);
            xmax[((g & 1) * 4 + kq) * 128 + r_loc] = t4[0];
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_X + quarter * 2 + (g & 1)));
            return t4[0];
        };

        auto mu_of = [&](const WorkItem& w) -> float {        // Q-Mean: mean of this thread's query row
            return (QM && w.q0 + r_loc < N) ? args.q_mu[(size_t)w.bh_q * N + w.q0 + r_loc] : 0.f;
        };
        float pn[KPT];                                        // scores of the next tile
        float mx_next = -INFINITY;
        int g = 0;                                            // global index of the current tile
        if (n_my > 0) {
            const WorkItem first = sched.item(0, args);
            ok = copy_q(0);
            if (ok) {
                if (wait_or_abort(bar(BAR_SF), 0, abort_flag)) {
                    tc_fence_after();
                    mx_next = fetch_scores(0, 0, first.q0, mu_of(first), first.bh_kv, pn);
                    if (first.n_tiles == 1 && n_my > 1) ok = copy_q(1);   // S of the item's last tile has been seen
                } else { fail(8); ok = false; }
            }
        }

        for (int k = 0; ok && k < n_my; ++k) {
            const WorkItem it = sched.item(k, args);
            const int n_tiles = it.n_tiles, q0 = it.q0;
            const int row = q0 + r_loc;
            int dbg_slot = -1;
            if (DBG)
                for (int i = 0; i < args.dbg.n_blocks; ++i)
                    if (args.dbg.blocks[3 * i] == it.b && args.dbg.blocks[3 * i + 1] == it.h && args.dbg.blocks[3 * i + 2] == it.qt)
                        dbg_slot = i;
            float m_run = -INFINITY;
            const bool has_next = k + 1 < n_my;
            const WorkItem nxt = has_next ? sched.item(k + 1, args) : it;   // decoded once per item, not per tile
            const float mu_cur = mu_of(it), mu_nxt = mu_of(nxt);

            for (int jt = 0; ok && jt < n_tiles; ++jt, ++g) {
                const int j0 = jt * BC;
                const uint32_t par = (uint32_t)g & 1u;
                const int sb = g & 1;                              // S / P-hat buffer and its barrier pair
                const uint32_t ph2 = (uint32_t)(g >> 1) & 1u;
                const uint32_t t_s = t_lane + S_COL + sb * 128;
                const int kbase = j0 + kq * KPT;
                float p[KPT];
#pragma unroll
                for (int i = 0; i < KPT; ++i) p[i] = pn[i];
                float mx = mx_next, gmax = mx_next;                // gmax: maximum over this thread's 64-key group
                // row maximum over the 128-key tile (line 7): own keys, then the other splits'
                if (!wait_or_abort(bar(BAR_X + quarter * 2 + sb), ph2, abort_flag)) { fail(9); ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int o = 1; o < KS; ++o) {
                    const float other = xmax[(par * 4 + (kq ^ o)) * 128 + r_loc];
                    mx = fmaxf(mx, other);
                    if (KS == 4 && o == 1) gmax = fmaxf(gmax, other);   // kq ^ 1 is the other half of the group
                }

                const float m_new = fmaxf(m_run, f16_round(mx * args.c0));
                float rsc = 1.f;
                if (jt > 0 && m_new != m_run) rsc = f16_round(ex2_approx((m_run - m_new) * LOG2E));
                m_run = m_new;
                const float mL = m_run * LOG2E;
                const float A = p_of_score(gmax, args.c1, mL);     // = max of P over the group (monotone map)

                // P = exp(S - m) in FP16 (line 9), P-hat = HIF4(P) (line 10); the BF16 image overwrites the
                // first 64 columns of S(g)
                uint8_t* dc = nullptr;
                float* ds = nullptr;
                if (DBG && dbg_slot >= 0 && row < N && kbase < N) {
                    const size_t r_idx = (size_t)dbg_slot * 128 + r_loc;
                    if (args.dbg.p_codes) dc = args.dbg.p_codes + r_idx * N + kbase;
                    if (args.dbg.p_step) ds = args.dbg.p_step + r_idx * (N / 4) + kbase / 4;
                }
                {
                    uint32_t w[NU * 4];
                    const PQuantConst qc = p_quant_const(args.c1, mL, A);
                    constexpr int U_SPLIT = (3 * NU) / 4;
                    exp_quantize_units<NU, 0, U_SPLIT, DBG>(p, qc, A == 0.f, w, dc, ds);
                    // next tile (of this item, or the first of the next item): scores and partial maximum
                    const bool in_item = jt + 1 < n_tiles;
                    if (in_item || has_next) {
                        const int nk = in_item ? k : k + 1, njt = in_item ? jt + 1 : 0;
                        const int n_q0 = in_item ? q0 : nxt.q0, n_nt = in_item ? n_tiles : nxt.n_tiles;
                        if (!wait_or_abort(bar(BAR_SF + (sb ^ 1)), (uint32_t)((g + 1) >> 1) & 1u, abort_flag)) { fail(8); ok = false; break; }
                        tc_fence_after();
                        mx_next = fetch_scores(g + 1, njt, n_q0, in_item ? mu_cur : mu_nxt,
                                               in_item ? it.bh_kv : nxt.bh_kv, pn);
                        // S of the last tile of item nk has been seen, so every QK of that item is complete and
                        // the Q-hat image in tensor memory may be replaced by the next item's
                        if (njt == n_nt - 1 && nk + 1 < n_my) {
                            if (!copy_q(nk + 1)) { ok = false; break; }
                        }
                    }
                    exp_quantize_units<NU, U_SPLIT, NU, DBG>(p, qc, A == 0.f, w, dc, ds);
                    if constexpr (KS == 2) tmem_st32(t_s + kq * (KPT / 2), w);
                    else tmem_st16(t_s + kq * (KPT / 2), w);
                }
                // rescale history (line 8): the KS splits share the 144 columns of [O | l].  It needs PV(g-1)
                // complete; a tile that leaves every running maximum of the warp unchanged skips it (r = 1).
                // Every warp observes every phase of the PV barrier, in order: a parity wait can only tell
                // the last two phases apart, so skipping one would alias.
                if (g > 0) {
                    if (!wait_or_abort(bar(BAR_PV), par ^ 1u, abort_flag)) { fail(10); ok = false; break; }
                    tc_fence_after();
                }
                if (__any_sync(0xffffffffu, rsc != 1.f)) {
                    constexpr int CW = O_COLS / KS;                // 72 or 36 columns per split
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
                    for (int cc = 0; cc < (CW % 32) / 4; ++cc) {
                        uint32_t r[4];
                        tmem_ld4(t_o + (CW / 32) * 32 + cc * 4, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 4; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * rsc);
                        tmem_st4(t_o + (CW / 32) * 32 + cc * 4, r);
                    }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_PF + sb));
            }
            if (!ok) break;

            // finalize the item: out = O / l with l rounded to FP16 (line 13); split kq writes channels
            // KPT*kq..  The next item's first PV cannot be issued before these warps have moved on.
            if (wait_or_abort(bar(BAR_PV), (uint32_t)(g - 1) & 1u, abort_flag)) {
                tc_fence_after();
                uint32_t lr[4];
                tmem_ld4(t_lane + D, lr);
                tmem_wait_ld();
                const float ell = __uint_as_float(lr[0]);
                const float l16 = f16_round(ell);
                // O / l as the correctly rounded quotient from the correctly rounded reciprocal and one
                // correction step (no value here is near the ends of the FP32 range)
                const float rl = __frcp_rn(l16);
                if (DBG && dbg_slot >= 0 && row < N && kq == 0) {
                    if (args.dbg.l_out) args.dbg.l_out[dbg_slot * 128 + r_loc] = ell;
                    if (args.dbg.m_out) args.dbg.m_out[dbg_slot * 128 + r_loc] = m_run;
                }
                const size_t orow = ((size_t)it.bh_q * N + row) * D + kq * KPT;
                const uint32_t stage = smem_base + STG_OFF + (uint32_t)warp * 1024u;
#pragma unroll
                for (int cc = 0; cc < KPT / 32; ++cc) {
                    uint32_t r[32];
                    tmem_ld32(t_lane + kq * KPT + cc * 32, r);
                    tmem_wait_ld();
                    float o[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float a = __uint_as_float(r[i]);
                        const float q0v = a * rl;
                        o[i] = fmaf(fmaf(-q0v, l16, a), rl, q0v);
                    }
                    if (args.out_dtype == HIFA4_F32) {
                        // through shared memory, 8 rows at a time, so that a store instruction writes whole
                        // 128-byte lines
                        const int c4r = lane & 7, sub = lane >> 3;
                        float* obase = reinterpret_cast<float*>(args.out) + ((size_t)it.bh_q * N + q0 + quarter * 32) * D +
                                       kq * KPT + cc * 32 + c4r * 4;
#pragma unroll
                        for (int pass = 0; pass < 4; ++pass) {
                            if ((lane >> 3) == pass) {
#pragma unroll
                                for (int c4 = 0; c4 < 8; ++c4)
                                    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};"
                                                 ::"r"(stage + (lane & 7) * 128 + ((c4 ^ (lane & 7)) << 4)), "f"(o[4 * c4]),
                                                   "f"(o[4 * c4 + 1]), "f"(o[4 * c4 + 2]), "f"(o[4 * c4 + 3]) : "memory");
                            }
                            __syncwarp();
#pragma unroll
                            for (int hh = 0; hh < 2; ++hh) {
                                const int r8 = hh * 4 + sub, rr = pass * 8 + r8;
                                float4 v;
                                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                             : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                                             : "r"(stage + r8 * 128 + ((c4r ^ r8) << 4)));
                                if (q0 + quarter * 32 + rr < N) *reinterpret_cast<float4*>(obase + (size_t)rr * D) = v;
                            }
                            __syncwarp();
                        }
                    } else if (row < N) {
                        {
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
                }
                tc_fence_before();     // [O | l] has been read: the next item's PV may overwrite it
            } else {
                fail(11);
                ok = false;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == W_MMA) { __syncwarp(); tmem_dealloc(tmem, TMEM_COLS); }
}

template <int KS, bool DBG, bool QM>
static int launch_ws(const hifa4_shape& sh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                     const AttnArgs& args, cudaStream_t st)
{
    auto kern = attention_fwd_ws_kernel<KS, DBG, QM>;
    static SmemOptIn opt_in;
    if (!opt_in.ensure(kern, ws::SMEM_BYTES)) return HIFA4_ERR_CUDA;
    int dev = 0, sm_count = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0)
        return HIFA4_ERR_CUDA;
    const long long n_items = (long long)((sh.N + 127) / 128) * sh.Hq * sh.B;
    dim3 grid((unsigned)(n_items < sm_count ? n_items : sm_count));     // persistent: one CTA per SM
    kern<<<grid, (4 * KS + 2) * 32, ws::SMEM_BYTES, st>>>(mq, mk, mv, args);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? HIFA4_OK : HIFA4_ERR_CUDA;
}

int launch_attention_ws(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    CUtensorMap mq, mk, mv;
    if (!make_bf16_map(&mq, qkv.q_mma, (uint64_t)sh.B * sh.Hq, sh.N, ws::D, 128)) return HIFA4_ERR_CUDA;
    if (!make_bf16_map(&mk, qkv.k_mma, (uint64_t)sh.B * sh.Hkv, sh.N, ws::D, ws::BC)) return HIFA4_ERR_CUDA;
    if (!make_bf16_map(&mv, qkv.v_mma, (uint64_t)sh.B * sh.Hkv, ws::D, sh.N, ws::D)) return HIFA4_ERR_CUDA;
    // the P-hat dump code and the Q-Mean correction live in separate instantiations, so that the
    // timed path carries none of either
    const bool dbg = args.dbg.n_blocks > 0;
    if (args.qmean) return dbg ? launch_ws<4, true, true>(sh, mq, mk, mv, args, st) : launch_ws<4, false, true>(sh, mq, mk, mv, args, st);
    return dbg ? launch_ws<4, true, false>(sh, mq, mk, mv, args, st) : launch_ws<4, false, false>(sh, mq, mk, mv, args, st);
}

}  // namespace hifa4
