// Fused HiFA4 prefill attention forward (Algorithm 1 lines 4-13) for sm_100a.
//
// One CTA owns 128 query rows of one (batch, query head).  Operands are the exact BF16 images
// of the HIF4-quantized Q, K and V^T; both GEMMs run on tcgen05 (kind::f16, FP32 accumulators in
// tensor memory).  Thread r of the CTA owns query row r: it reads its row of S from tensor
// memory, keeps the FP16 running maximum, forms P = exp(S - m) in FP16, quantizes it to HIF4 per
// 64 keys in registers and writes the BF16 image of P-hat into the swizzled shared-memory tile
// the PV MMA consumes.  V^T tiles carry 16 extra rows of ones, so column d of the PV accumulator
// is the row sum of P-hat: the normalizer of P-Reordering comes out of the same MMA.
#include "hifa4_attention.cuh"

namespace hifa4 {

// AUX: the variant that also keeps the row sums of the unquantized P (exactly, in 2^-24 fixed point:
// P is an FP16 value), for the mismatched normalizer and for the mass-error histogram.
template <int D, int BC, bool AUX>
__global__ void __launch_bounds__(128, 1)
attention_fwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                     const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ AttnArgs args)
{
    using C = Cfg<D, BC>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;     // 128-byte swizzle wants 1024
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_s = smem_base + C::Q_OFF, k_s = smem_base + C::K_OFF, v_s = smem_base + C::V_OFF,
                   p_s = smem_base + C::P_OFF;
    const uint32_t bar_q = smem_base + C::BAR_OFF, bar_kv = bar_q + 8, bar_mma = bar_q + 16;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + C::BAR_OFF + 32);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int n_qt = (args.N + 127) / 128;
    const int qt = n_qt - 1 - (int)blockIdx.x;            // heaviest causal tiles are scheduled first
    const int h = blockIdx.y, b = blockIdx.z;
    const int g = args.map.kv_of[h];
    const int q0 = qt * 128;
    const int bh_q = b * args.Hq + h, bh_kv = b * args.Hkv + g;
    const int N = args.N;
    const int row = q0 + tid;                             // this thread's query row

    // ---- set-up: barriers, tensor memory, ones rows under every V^T chunk
    volatile int* dead_flag = reinterpret_cast<volatile int*>(smem_gen + C::BAR_OFF + 40);
    if (tid == 0) {
        // A CTA that starts after another one reported a failure does nothing.  One thread reads the status
        // word and publishes the verdict through shared memory: every thread then takes the same path, and
        // that path still frees the tensor memory allocated below.
        *dead_flag = (args.d_status && *reinterpret_cast<volatile int*>(args.d_status) != 0) ? 1 : 0;
        tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_k); tma_prefetch_desc(&tmap_v);
        mbar_init(bar_q, 1); mbar_init(bar_kv, 1); mbar_init(bar_mma, 1);
        fence_barrier_init();
    }
    if (warp == 0) { tmem_alloc(smem_u32((const void*)tmem_slot), C::TMEM_COLS); tmem_relinquish(); }
    for (int i = tid; i < C::PSUB * 16 * 8; i += 128) {   // 16 rows x 8 chunks of 16 bytes per V chunk
        int c = i / 128, off = (i % 128) * 16;
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};"
                     ::"r"(v_s + c * C::V_CHUNK_BYTES + D * 128 + off), "r"(0x3F803F80u) : "memory");
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's lane quarter
    const uint32_t t_o = t_lane, t_s = t_lane + C::S_COL;

    int dbg_slot = -1;
    for (int i = 0; i < args.dbg.n_blocks; ++i)
        if (args.dbg.blocks[3 * i] == b && args.dbg.blocks[3 * i + 1] == h && args.dbg.blocks[3 * i + 2] == qt)
            dbg_slot = i;

    bool ok = true;
    uint32_t mma_phase = 0;
    int fail_site = 0;
    if (*dead_flag) goto done;

    if (tid == 0) {
        mbar_expect_tx(bar_q, C::KSUB * C::Q_SUB_BYTES);
#pragma unroll
        for (int s = 0; s < C::KSUB; ++s) tma_load_3d(q_s + s * C::Q_SUB_BYTES, &tmap_q, bar_q, 64 * s, q0, bh_q);
    }
    ok = mbar_wait(bar_q, 0);
    if (!__syncthreads_and(ok)) { fail_site = 1; goto fail; }

    {
        const int last_key = args.causal ? min(q0 + 127, N - 1) : N - 1;
        const int n_tiles = last_key / BC + 1;
        float m_run = -INFINITY;                          // FP16 value held in a float
        float ell_p = 0.f;                                // AUX: normalizer accumulated from P (mismatched)
        const float LOG2E = 1.4426950408889634f;
        // Q-Mean correction (line 6): mu of this row, channel sum of every key of the KV head
        const float mu_row = (args.qmean && row < N) ? args.q_mu[(size_t)bh_q * N + row] : 0.f;
        auto ksum_of = [&](int key) { return key < N ? __ldg(args.k_sum + (size_t)bh_kv * N + key) : 0.f; };
        constexpr uint32_t idesc_s = umma_idesc_bf16(128, BC);
        constexpr uint32_t idesc_o = umma_idesc_bf16(128, (C::O_COLS <= 256) ? C::O_COLS : 256);
        constexpr uint32_t idesc_l = umma_idesc_bf16(128, 16);

        for (int jt = 0; jt < n_tiles; ++jt) {
            const int j0 = jt * BC;
            // ---- load K tile and V^T tile
            if (tid == 0) {
                mbar_expect_tx(bar_kv, C::KSUB * C::K_SUB_BYTES + C::PSUB * D * 128);
#pragma unroll
                for (int s = 0; s < C::KSUB; ++s) tma_load_3d(k_s + s * C::K_SUB_BYTES, &tmap_k, bar_kv, 64 * s, j0, bh_kv);
#pragma unroll
                for (int c = 0; c < C::PSUB; ++c) tma_load_3d(v_s + c * C::V_CHUNK_BYTES, &tmap_v, bar_kv, j0 + 64 * c, 0, bh_kv);
            }
            ok = mbar_wait(bar_kv, jt & 1);
            if (!__syncthreads_and(ok)) { fail_site = 2; goto fail; }

            // ---- S = Q-hat K-hat^T (raw accumulators; the softmax scale is applied on the fly)
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int s = 0; s < C::KSUB; ++s)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16_ss(tmem + C::S_COL, umma_desc_sw128(q_s + s * C::Q_SUB_BYTES + kk * 32),
                                     umma_desc_sw128(k_s + s * C::K_SUB_BYTES + kk * 32), idesc_s,
                                     (s | kk) ? 1u : 0u);
                umma_commit(bar_mma);
            }
            ok = mbar_wait(bar_mma, mma_phase & 1);
            ++mma_phase;
            if (!__syncthreads_and(ok)) { fail_site = 3; goto fail; }
            tc_fence_after();

            // ---- row maximum over the tile (Algorithm 1 line 7)
            const bool need_mask = (args.causal && (j0 + BC - 1 > q0)) || (j0 + BC > N);
            const int key_lim = args.causal ? min(row, N - 1) : N - 1;   // last key this row may see
            float mx = -INFINITY;
#pragma unroll
            for (int cc = 0; cc < BC / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(t_s + cc * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float a = __uint_as_float(r[i]);
                    if (args.qmean) a = fmaf(mu_row, ksum_of(j0 + cc * 32 + i), a);
                    if (need_mask && (j0 + cc * 32 + i > key_lim)) a = -INFINITY;
                    mx = fmaxf(mx, a);
                }
            }
            const float m_new = fmaxf(m_run, f16_round(mx * args.c0));
            // ---- rescale history (line 8): r = exp(m - m_new) in FP16; exact no-op when m is unchanged
            if (jt > 0) {
                float rsc = 1.f;
                if (m_new != m_run) rsc = f16_round(ex2_approx((m_run - m_new) * LOG2E));
                if (AUX) ell_p *= rsc;
                if (__any_sync(0xffffffffu, rsc != 1.f)) {
#pragma unroll
                    for (int cc = 0; cc < C::O_COLS / 16; ++cc) {
                        uint32_t r[16];
                        tmem_ld16(t_o + cc * 16, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * rsc);
                        tmem_st16(t_o + cc * 16, r);
                    }
                    tmem_wait_st();
                }
            }
            m_run = m_new;
            const float mL = m_run * LOG2E;

            // ---- P = exp(S - m) in FP16 (line 9), P-hat = HIF4(P) per 64 keys (line 10)
            uint32_t p_fix = 0;                           // AUX: sum of P over the tile in units of 2^-24 (< 2^32)
            double ph_sum = 0.0;                          // AUX: sum of P-hat over the tile (exact)
#pragma unroll
            for (int gq = 0; gq < C::PSUB; ++gq) {
                float p[64];
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t r[32];
                    tmem_ld32(t_s + gq * 64 + cc * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        float a = __uint_as_float(r[i]);
                        if (args.qmean) a = fmaf(mu_row, ksum_of(j0 + gq * 64 + cc * 32 + i), a);
                        float t = fmaf(a, args.c1, -mL);
                        float e = f16_round(ex2_approx(t));
                        if (need_mask && (j0 + gq * 64 + cc * 32 + i > key_lim)) e = 0.f;
                        p[cc * 32 + i] = e;
                    }
                }
                uint8_t* dc = nullptr;
                float* ds = nullptr;
                if (dbg_slot >= 0 && row < N && j0 + gq * 64 < N) {
                    size_t r_idx = (size_t)dbg_slot * 128 + tid;
                    if (args.dbg.p_codes) dc = args.dbg.p_codes + r_idx * N + j0 + gq * 64;
                    if (args.dbg.p_step) ds = args.dbg.p_step + r_idx * (N / 4) + (j0 + gq * 64) / 4;
                }
                float gsum;
                quantize_p64(p, p_s + gq * C::P_SUB_BYTES, tid, dc, ds, AUX ? &gsum : nullptr);
                if (AUX) {
                    ph_sum += (double)gsum;
#pragma unroll
                    for (int i = 0; i < 64; ++i) p_fix += __float2uint_rz(p[i] * 16777216.f);
                }
            }
            if (AUX) {
                const double p_sum = (double)p_fix * (1.0 / 16777216.0);
                ell_p = __double2float_rn((double)ell_p + p_sum);     // one rounding per tile, as for the MMA's l
                if (args.hist && row < N && p_fix != 0) {             // per (row, key tile) mass error of P-hat
                    const double eps = ph_sum / p_sum - 1.0;
                    const double x = floor((eps - args.hist_lo) * args.hist_inv_w);
                    const int bin = x < 0.0 ? args.n_bins : (x >= (double)args.n_bins ? args.n_bins + 1 : (int)x);
                    atomicAdd(args.hist + bin, 1ull);
                }
            }
            fence_proxy_async_smem();                     // P-hat tile -> visible to the MMA's smem reads
            tc_fence_before();
            __syncthreads();

            // ---- [O | l] += P-hat [V-hat | 1]  (line 11)
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < C::PSUB; ++c)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint32_t acc = (jt > 0 || c > 0 || kk > 0) ? 1u : 0u;
                        const uint64_t ad = umma_desc_sw128(p_s + c * C::P_SUB_BYTES + kk * 32);
                        const uint32_t vb = v_s + c * C::V_CHUNK_BYTES + kk * 32;
                        umma_bf16_ss(tmem, ad, umma_desc_sw128(vb), idesc_o, acc);
                        if (C::O_COLS > 256)
                            umma_bf16_ss(tmem + 256, ad, umma_desc_sw128(vb + 256 * 128), idesc_l, acc);
                    }
                umma_commit(bar_mma);
            }
            ok = mbar_wait(bar_mma, mma_phase & 1);
            ++mma_phase;
            if (!__syncthreads_and(ok)) { fail_site = 4; goto fail; }
            tc_fence_after();
        }

        // ---- finalize: out = O / l with l rounded to FP16 (line 13)
        {
            uint32_t lr[16];
            tmem_ld16(t_o + D, lr);
            tmem_wait_ld();
            const float ell = (AUX && args.normalizer) ? ell_p : __uint_as_float(lr[0]);
            const float l16 = f16_round(ell);
            if (dbg_slot >= 0 && row < N) {
                if (args.dbg.l_out) args.dbg.l_out[dbg_slot * 128 + tid] = ell;
                if (args.dbg.m_out) args.dbg.m_out[dbg_slot * 128 + tid] = m_run;
            }
            const size_t orow = ((size_t)bh_q * N + row) * D;
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(t_o + cc * 32, r);
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
        }
    }
    goto done;

fail:
    if (tid == 0 && args.d_status) atomicExch(args.d_status, HIFA4_ERR_TIMEOUT + 16 * fail_site);
    // give copies and MMAs still in flight a bounded chance to land before the CTA's memory goes away
    for (int i = 0; i < 64; ++i) { mbar_try_wait(bar_kv, 0); mbar_try_wait(bar_mma, 0); }

done:
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, C::TMEM_COLS);
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode()
{
    // initialised once, thread-safe (a function-local static); null if the driver lacks the entry point
    static const EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            return (EncodeTiledFn)p;
        return (EncodeTiledFn) nullptr;
    }();
    return fn;
}

bool make_bf16_map(CUtensorMap* m, void* base, uint64_t heads, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[3] = {cols, rows, heads};
    cuuint64_t strides[2] = {cols * 2, rows * cols * 2};
    cuuint32_t box[3] = {64, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_u8_map(CUtensorMap* m, void* base, uint64_t heads, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    EncodeTiledFn enc = get_encode();
    if (!enc || cols != 128) return false;                 // one 128-byte swizzle span per row
    cuuint64_t dims[3] = {cols, rows, heads};
    cuuint64_t strides[2] = {cols, rows * cols};
    cuuint32_t box[3] = {128, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int BC, bool AUX>
static int launch_cfg(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st)
{
    using C = Cfg<D, BC>;
    CUtensorMap mq, mk, mv;
    if (!make_bf16_map(&mq, qkv.q_mma, (uint64_t)sh.B * sh.Hq, sh.N, D, 128)) return HIFA4_ERR_CUDA;
    if (!make_bf16_map(&mk, qkv.k_mma, (uint64_t)sh.B * sh.Hkv, sh.N, D, BC)) return HIFA4_ERR_CUDA;
    if (!make_bf16_map(&mv, qkv.v_mma, (uint64_t)sh.B * sh.Hkv, D, sh.N, D)) return HIFA4_ERR_CUDA;
    auto kern = attention_fwd_kernel<D, BC, AUX>;
    static SmemOptIn opt_in;
    if (!opt_in.ensure(kern, C::SMEM_BYTES)) return HIFA4_ERR_CUDA;
    dim3 grid((sh.N + 127) / 128, sh.Hq, sh.B);
    kern<<<grid, 128, C::SMEM_BYTES, st>>>(mq, mk, mv, args);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? HIFA4_OK : HIFA4_ERR_CUDA;
}

bool attention_qraw_supported(const hifa4_shape& sh, const hifa4_attn_params& prm)
{
    return prm.Bc == 64 && sh.d == 128 && !prm.qmean && !prm.normalizer;
}

int launch_attention(const hifa4_shape& sh, const HeadMap& map, const hifa4_qkv& qkv,
                     const hifa4_attn_params& prm, void* out, const hifa4_debug* dbg,
                     const hifa4_mass_stats* stats, int* d_status, cudaStream_t st, bool selftest,
                     const void* q_raw, const float* q_scale, const F8Operands* f8)
{
    AttnArgs a;
    memset(&a, 0, sizeof(a));
    if (f8) {
        if (prm.Bc != 64 || sh.d != 128 || prm.qmean || prm.normalizer || prm.p_dtype == HIFA4_F32 || stats || selftest ||
            q_raw || (dbg && dbg->n_blocks > 0))
            return HIFA4_ERR_UNSUPPORTED;
        a.q_f8 = f8->q_f8; a.k_f8 = f8->k_f8; a.q_gs = f8->q_gs; a.k_gs = f8->k_gs;
    }
    if (q_raw) {
        if (!attention_qraw_supported(sh, prm) || stats || selftest || (dbg && dbg->n_blocks > 0)) return HIFA4_ERR_UNSUPPORTED;
        a.q_raw = q_raw;
        a.q_scale = q_scale;
        a.in_dtype = sh.in_dtype;
    }
    a.B = sh.B; a.Hq = sh.Hq; a.Hkv = sh.Hkv; a.N = sh.N;
    a.causal = prm.causal ? 1 : 0;
    a.out_dtype = prm.out_dtype;
    const double sigma = prm.softmax_scale != 0.f ? (double)prm.softmax_scale : 1.0 / sqrt((double)sh.d);
    a.c0 = (float)sigma;
    a.c1 = (float)(sigma * 1.4426950408889634074);
    a.out = out;
    a.qmean = prm.qmean ? 1 : 0;
    a.q_mu = qkv.q_mu;
    a.k_sum = qkv.k_sum;
    a.d_status = d_status;
    a.map = map;
    if (dbg && dbg->n_blocks > 0) {
        a.dbg.n_blocks = dbg->n_blocks;
        for (int i = 0; i < 3 * dbg->n_blocks; ++i) a.dbg.blocks[i] = dbg->blocks[i];
        a.dbg.p_codes = dbg->p_codes; a.dbg.p_step = dbg->p_step;
        a.dbg.l_out = dbg->l_out; a.dbg.m_out = dbg->m_out;
    }
    // CTA order of the 64-key kernel: groups of KV heads whose K-hat / V-hat^T images fit in L2 (126 MB) together with
    // room to spare, one group after the other, so that the CTAs in flight share them; inside a group the grid keeps
    // its heaviest-first order.  Causal: the largest divisor of B * Hkv whose images stay within 48 MB (measured on
    // B = 4, Hq = 32, Hkv = 8, d = 128 against one group: +6 % at N = 8192, +5 % at 16384, +1 % at 32768, where
    // single heads, which lose the heaviest-first order across heads, were the earlier choice; no change where
    // everything fits).  Non-causal items are all equal, so nothing is lost by the smallest group: one KV head at a
    // time once the images exceed 50 MB (+4 % at 67 MB, +15 % at 134 MB; no difference below).
    {
        const double per_kv_head = (double)sh.N * sh.d * 4.0;
        const int n_kv = sh.B * sh.Hkv;
        int want = prm.causal ? (int)(48e6 / per_kv_head) : (per_kv_head * n_kv > 50e6 ? 1 : n_kv);
        if (want < 1) want = 1;
        if (sh.q_to_kv || sh.Hq % sh.Hkv) {              // custom head map: whole batch elements only
            int g_b = 1;
            for (int c = 1; c <= sh.B && c * sh.Hkv <= want; ++c)
                if (sh.B % c == 0) g_b = c;
            a.group_heads = g_b * sh.Hq;
        } else {
            int g_kv = 1;
            for (int c = 1; c <= n_kv && c <= want; ++c)
                if (n_kv % c == 0) g_kv = c;
            a.group_heads = g_kv * (sh.Hq / sh.Hkv);
        }
    }
    a.normalizer = prm.normalizer ? 1 : 0;
    a.p_f32 = prm.p_dtype == HIFA4_F32 ? 1 : 0;
    if (selftest) {                               // the instantiation whose wait for P V runs out
        if (a.p_f32 || a.normalizer || a.qmean || stats || dbg || prm.Bc != 64 || sh.d != 128) return HIFA4_ERR_UNSUPPORTED;
        return launch_attention_ws64_selftest(sh, qkv, a, st);
    }
    if (a.p_f32) {                                // variant built for the 64-key warp-specialised kernels only
        if (a.normalizer || stats || prm.Bc != 64 || (sh.d != 128 && sh.d != 256)) return HIFA4_ERR_UNSUPPORTED;
        return launch_attention_ws64(sh, qkv, a, st);
    }
    if (stats) {
        a.hist = stats->hist;
        a.n_bins = stats->n_bins;
        a.hist_lo = stats->lo;
        a.hist_inv_w = (double)stats->n_bins / (stats->hi - stats->lo);
    }
    if (a.normalizer || a.hist) {                 // the one-thread-per-row kernel keeps the sums of P
        if (sh.d == 64 && prm.Bc == 64) return launch_cfg<64, 64, true>(sh, qkv, a, st);
        if (sh.d == 64 && prm.Bc == 128) return launch_cfg<64, 128, true>(sh, qkv, a, st);
        if (sh.d == 128 && prm.Bc == 64) return launch_cfg<128, 64, true>(sh, qkv, a, st);
        if (sh.d == 128 && prm.Bc == 128) return launch_cfg<128, 128, true>(sh, qkv, a, st);
        if (sh.d == 256 && prm.Bc == 64) return launch_cfg<256, 64, true>(sh, qkv, a, st);
        return HIFA4_ERR_UNSUPPORTED;
    }
    if (sh.d == 64 && prm.Bc == 64) return launch_attention_ws64(sh, qkv, a, st);
    if (sh.d == 64 && prm.Bc == 128) return launch_cfg<64, 128, false>(sh, qkv, a, st);
    if (sh.d == 128 && prm.Bc == 64) return launch_attention_ws64(sh, qkv, a, st);
    if (sh.d == 128 && prm.Bc == 128) return launch_attention_ws(sh, qkv, a, st);
    if (sh.d == 256 && prm.Bc == 64) return launch_attention_ws64(sh, qkv, a, st);
    return HIFA4_ERR_UNSUPPORTED;
}

}  // namespace hifa4
