// Warp-specialised HiFA4 attention forward for d = 128, Bc = 128 (Algorithm 1 lines 4-13).
//
// One CTA = 128 query rows of one (batch, query head), 10 warps:
//   warps 0-7  softmax / quantize: warp w owns rows 32*(w%4).. of the tile and the 64-key HIF4
//              group (w/4) of every 128-key tile, so a thread holds exactly one group of one row;
//              the two threads of a row exchange their partial row maxima through shared memory
//   warp 8     TMA producer: Q once, then K and V^T tiles through two-stage rings
//   warp 9     tcgen05 issuer: S = Q K^T for tile j+1 is issued as soon as the softmax warps
//              have pulled S(j) into registers, then [O | l] += P-hat(j) [V-hat | 1]
// S lives in 128 tensor-memory columns, [O | l] in 144; P-hat goes through one swizzled
// shared-memory tile.  Every wait is bounded; a wait that expires raises the abort flag, writes
// the status word and every role falls through to the common exit (tensor memory is freed).
#include "hifa4_attention.cuh"

namespace hifa4 {

namespace ws {
constexpr int D = 128, BC = 128, STAGES = 2;
constexpr int Q_BYTES = 2 * 16384;
constexpr int K_STAGE = 2 * 16384;
constexpr int V_CHUNK = (D + 16) * 128;
constexpr int V_STAGE = 2 * V_CHUNK;
constexpr int P_BYTES = 2 * 16384;
constexpr int Q_OFF = 0;
constexpr int K_OFF = Q_OFF + Q_BYTES;
constexpr int V_OFF = K_OFF + STAGES * K_STAGE;
constexpr int P_OFF = V_OFF + STAGES * V_STAGE;
constexpr int MISC_OFF = P_OFF + P_BYTES;           // barriers, tmem slot, abort flag
constexpr int XCHG_OFF = MISC_OFF + 256;            // [2 parities][2 groups][128 rows] floats
constexpr int SMEM_BYTES = XCHG_OFF + 2 * 2 * 128 * 4 + 1024;
constexpr int O_COLS = D + 16, S_COL = 256, TMEM_COLS = 512;
constexpr int THREADS = 320;
enum { BAR_Q = 0, BAR_KF = 1, BAR_KE = 3, BAR_VF = 5, BAR_VE = 7, BAR_SF = 9, BAR_SFREE = 10,
       BAR_PF = 11, BAR_PV = 12, BAR_X = 13, N_BARS = 17 };
}  // namespace ws

__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (uint32_t i = 0; i < (1u << 18); ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 255u && *abort_flag) return false;
    }
    return false;
}

__global__ void __launch_bounds__(ws::THREADS, 1)
attention_fwd_ws_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                        const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ AttnArgs args)
{
    using namespace ws;
    if (args.d_status && *reinterpret_cast<volatile int*>(args.d_status) != 0) return;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_s = smem_base + Q_OFF, k_s = smem_base + K_OFF, v_s = smem_base + V_OFF,
                   p_s = smem_base + P_OFF, bars = smem_base + MISC_OFF;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + MISC_OFF + 8 * N_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + MISC_OFF + 8 * N_BARS + 8);
    float* xchg = reinterpret_cast<float*>(smem_gen + XCHG_OFF);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = args.N;
    const int n_qt = (N + 127) / 128;
    const int qt = n_qt - 1 - (int)blockIdx.x;
    const int h = blockIdx.y, b = blockIdx.z;
    const int g = args.map.kv_of[h];
    const int q0 = qt * 128;
    const int bh_q = b * args.Hq + h, bh_kv = b * args.Hkv + g;
    const int last_key = args.causal ? min(q0 + 127, N - 1) : N - 1;
    const int n_tiles = last_key / BC + 1;

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(BAR_Q), 1);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(BAR_KF + s), 1); mbar_init(bar(BAR_KE + s), 1);
            mbar_init(bar(BAR_VF + s), 1); mbar_init(bar(BAR_VE + s), 1);
        }
        mbar_init(bar(BAR_SF), 1); mbar_init(bar(BAR_SFREE), 8);
        mbar_init(bar(BAR_PF), 8); mbar_init(bar(BAR_PV), 1);
        for (int i = 0; i < 4; ++i) mbar_init(bar(BAR_X + i), 2);
        fence_barrier_init();
    }
    if (warp == 9) { tmem_alloc(smem_u32((const void*)tmem_slot), TMEM_COLS); tmem_relinquish(); }
    if (warp == 8 && lane == 0) { tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_k); tma_prefetch_desc(&tmap_v); }
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

    auto fail = [&](int site) {
        *abort_flag = 1;
        if (args.d_status) atomicCAS(args.d_status, 0, HIFA4_ERR_TIMEOUT + 16 * site);
    };

    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(bar(BAR_Q), Q_BYTES);
            tma_load_3d(q_s, &tmap_q, bar(BAR_Q), 0, q0, bh_q);
            tma_load_3d(q_s + 16384, &tmap_q, bar(BAR_Q), 64, q0, bh_q);
            for (int jt = 0; jt < n_tiles; ++jt) {
                const int st = jt & 1;
                const uint32_t ph = (uint32_t)(jt >> 1) & 1u;
                const int j0 = jt * BC;
                if (!wait_or_abort(bar(BAR_KE + st), ph ^ 1u, abort_flag)) { fail(1); break; }
                mbar_expect_tx(bar(BAR_KF + st), K_STAGE);
                tma_load_3d(k_s + st * K_STAGE, &tmap_k, bar(BAR_KF + st), 0, j0, bh_kv);
                tma_load_3d(k_s + st * K_STAGE + 16384, &tmap_k, bar(BAR_KF + st), 64, j0, bh_kv);
                if (!wait_or_abort(bar(BAR_VE + st), ph ^ 1u, abort_flag)) { fail(2); break; }
                mbar_expect_tx(bar(BAR_VF + st), 2 * D * 128);
                tma_load_3d(v_s + st * V_STAGE, &tmap_v, bar(BAR_VF + st), j0, 0, bh_kv);
                tma_load_3d(v_s + st * V_STAGE + V_CHUNK, &tmap_v, bar(BAR_VF + st), j0 + 64, 0, bh_kv);
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = umma_idesc_bf16(128, BC);
            constexpr uint32_t idesc_o = umma_idesc_bf16(128, O_COLS);
            auto issue_qk = [&](int jt) {
                const int st = jt & 1;
#pragma unroll
                for (int s = 0; s < 2; ++s)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16_ss(tmem + S_COL, umma_desc_sw128(q_s + s * 16384 + kk * 32),
                                     umma_desc_sw128(k_s + st * K_STAGE + s * 16384 + kk * 32), idesc_s,
                                     (s | kk) ? 1u : 0u);
                umma_commit(bar(BAR_SF));
                umma_commit(bar(BAR_KE + st));
            };
            bool ok = wait_or_abort(bar(BAR_Q), 0, abort_flag) && wait_or_abort(bar(BAR_KF), 0, abort_flag);
            if (!ok) fail(3);
            if (ok) {
                tc_fence_after();
                issue_qk(0);
                for (int jt = 0; jt < n_tiles; ++jt) {
                    if (jt + 1 < n_tiles) {
                        const int st1 = (jt + 1) & 1;
                        if (!wait_or_abort(bar(BAR_KF + st1), (uint32_t)((jt + 1) >> 1) & 1u, abort_flag)) { fail(4); break; }
                        if (!wait_or_abort(bar(BAR_SFREE), (uint32_t)jt & 1u, abort_flag)) { fail(5); break; }
                        tc_fence_after();
                        issue_qk(jt + 1);
                    }
                    const int st = jt & 1;
                    if (!wait_or_abort(bar(BAR_VF + st), (uint32_t)(jt >> 1) & 1u, abort_flag)) { fail(6); break; }
                    if (!wait_or_abort(bar(BAR_PF), (uint32_t)jt & 1u, abort_flag)) { fail(7); break; }
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < 2; ++c)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_bf16_ss(tmem, umma_desc_sw128(p_s + c * 16384 + kk * 32),
                                         umma_desc_sw128(v_s + st * V_STAGE + c * V_CHUNK + kk * 32), idesc_o,
                                         (jt > 0 || c > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(bar(BAR_PV));
                    umma_commit(bar(BAR_VE + st));
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax / quantize
        const int wg = warp >> 2, quarter = warp & 3;
        const int r_loc = quarter * 32 + lane;                     // row inside the tile = TMEM lane
        const int row = q0 + r_loc;
        const uint32_t t_lane = tmem + ((uint32_t)(quarter * 32) << 16);
        const uint32_t xbar = bar(BAR_X + quarter);
        const float LOG2E = 1.4426950408889634f;
        const int key_lim = args.causal ? min(row, N - 1) : N - 1;
        int dbg_slot = -1;
        for (int i = 0; i < args.dbg.n_blocks; ++i)
            if (args.dbg.blocks[3 * i] == b && args.dbg.blocks[3 * i + 1] == h && args.dbg.blocks[3 * i + 2] == qt)
                dbg_slot = i;
        float m_run = -INFINITY;
        bool ok = true;

        for (int jt = 0; jt < n_tiles; ++jt) {
            const int j0 = jt * BC;
            const uint32_t par = (uint32_t)jt & 1u;
            if (!wait_or_abort(bar(BAR_SF), par, abort_flag)) { fail(8); ok = false; break; }
            tc_fence_after();
            float p[64];
            {
                uint32_t r0[32], r1[32];
                tmem_ld32(t_lane + S_COL + wg * 64, r0);
                tmem_ld32(t_lane + S_COL + wg * 64 + 32, r1);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) { p[i] = __uint_as_float(r0[i]); p[32 + i] = __uint_as_float(r1[i]); }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_SFREE));

            // row maximum over the 128-key tile (line 7): own 64 keys, then the partner's
            const bool need_mask = (args.causal && (j0 + BC - 1 > q0)) || (j0 + BC > N);
            const int kbase = j0 + wg * 64;
            float mx = -INFINITY;
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < 64; ++i) mx = fmaxf(mx, (kbase + i > key_lim) ? -INFINITY : p[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 64; ++i) mx = fmaxf(mx, p[i]);
            }
            xchg[(par * 2 + wg) * 128 + r_loc] = mx;
            __syncwarp();
            if (lane == 0) mbar_arrive(xbar);
            if (!wait_or_abort(xbar, par, abort_flag)) { fail(9); ok = false; break; }
            mx = fmaxf(mx, xchg[(par * 2 + (wg ^ 1)) * 128 + r_loc]);

            const float m_new = fmaxf(m_run, f16_round(mx * args.c0));
            float rsc = 1.f;
            if (jt > 0 && m_new != m_run) rsc = f16_round(ex2_approx((m_run - m_new) * LOG2E));
            m_run = m_new;
            const float mL = m_run * LOG2E;

            // P = exp(S - m) in FP16 (line 9)
#pragma unroll
            for (int i = 0; i < 64; ++i) {
                float e = f16_round(ex2_approx(fmaf(p[i], args.c1, -mL)));
                if (need_mask && (kbase + i > key_lim)) e = 0.f;
                p[i] = e;
            }
            // the P tile and the O accumulator are free once PV(jt-1) has completed
            if (jt > 0) {
                if (!wait_or_abort(bar(BAR_PV), par ^ 1u, abort_flag)) { fail(10); ok = false; break; }
                tc_fence_after();
            }
            // P-hat = HIF4(P) (line 10) -> BF16 image in the swizzled P tile
            uint8_t* dc = nullptr;
            float* ds = nullptr;
            if (dbg_slot >= 0 && row < N && kbase < N) {
                const size_t r_idx = (size_t)dbg_slot * 128 + r_loc;
                if (args.dbg.p_codes) dc = args.dbg.p_codes + r_idx * N + kbase;
                if (args.dbg.p_step) ds = args.dbg.p_step + r_idx * (N / 4) + kbase / 4;
            }
            quantize_p64(p, p_s + wg * 16384, r_loc, dc, ds);
            fence_proxy_async_smem();
            // rescale history (line 8); group 0 owns columns 0..79 of [O | l], group 1 columns 80..143
            if (__any_sync(0xffffffffu, rsc != 1.f)) {
                const uint32_t t_o = t_lane + (wg ? 80 : 0);
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t r[32];
                    tmem_ld32(t_o + cc * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * rsc);
                    tmem_st32(t_o + cc * 32, r);
                }
                if (wg == 0) {
                    uint32_t r[16];
                    tmem_ld16(t_o + 64, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * rsc);
                    tmem_st16(t_o + 64, r);
                }
                tmem_wait_st();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_PF));
        }

        // finalize: out = O / l with l rounded to FP16 (line 13); group g writes channels 64g..64g+63
        if (ok && wait_or_abort(bar(BAR_PV), (uint32_t)(n_tiles - 1) & 1u, abort_flag)) {
            tc_fence_after();
            uint32_t lr[16];
            tmem_ld16(t_lane + D, lr);
            tmem_wait_ld();
            const float ell = __uint_as_float(lr[0]);
            const float l16 = f16_round(ell);
            if (dbg_slot >= 0 && row < N && wg == 0) {
                if (args.dbg.l_out) args.dbg.l_out[dbg_slot * 128 + r_loc] = ell;
                if (args.dbg.m_out) args.dbg.m_out[dbg_slot * 128 + r_loc] = m_run;
            }
            const size_t orow = ((size_t)bh_q * N + row) * D + wg * 64;
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
                uint32_t r[32];
                tmem_ld32(t_lane + wg * 64 + cc * 32, r);
                tmem_wait_ld();
                if (row < N) {
                    float o[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __fdiv_rn(__uint_as_float(r[i]), l16);
                    if (args.out_dtype == HIFA4_F32) {
                        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(args.out) + orow + cc * 32);
#pragma unroll
                        for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                    } else {
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
        } else if (ok) {
            fail(11);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) { __syncwarp(); tmem_dealloc(tmem, TMEM_COLS); }
}

int launch_attention_ws(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    CUtensorMap mq, mk, mv;
    if (!make_bf16_map(&mq, qkv.q_mma, (uint64_t)sh.B * sh.Hq, sh.N, ws::D, 128)) return HIFA4_ERR_CUDA;
    if (!make_bf16_map(&mk, qkv.k_mma, (uint64_t)sh.B * sh.Hkv, sh.N, ws::D, ws::BC)) return HIFA4_ERR_CUDA;
    if (!make_bf16_map(&mv, qkv.v_mma, (uint64_t)sh.B * sh.Hkv, ws::D, sh.N, ws::D)) return HIFA4_ERR_CUDA;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(attention_fwd_ws_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 ws::SMEM_BYTES) != cudaSuccess)
            return HIFA4_ERR_CUDA;
        attr_set = true;
    }
    dim3 grid((sh.N + 127) / 128, sh.Hq, sh.B);
    attention_fwd_ws_kernel<<<grid, ws::THREADS, ws::SMEM_BYTES, st>>>(mq, mk, mv, args);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? HIFA4_OK : HIFA4_ERR_CUDA;
}

}  // namespace hifa4
