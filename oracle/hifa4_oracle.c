/*
 * HiFA4 CPU oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, step-by-step CPU statement of what the HiFA4 hot path
 * computes, written from the paper (Background "HIF4", Eq. "sqk", Theorem 1,
 * Algorithm 1 "C4V16-Aux", Appendix "Implementation Details").  Only tests,
 * the smoke check and the benchmark's cpu_baseline leg may call it.  It shares
 * no code, table or constant with the CUDA path.
 *
 * Parity unpinned: the paper cites, but does not print, the BF16->HIF4
 * conversion of the HIF4 specification.  hif4_encode_group() below is a
 * reading that uses every format fact the paper states (64-element group,
 * E6M2 level-1 scale, 8 level-2 and 16 level-3 one-bit micro-exponents,
 * sign-magnitude S1P2 elements); its agreement with the official converter
 * cannot be checked here.  Everything else is pinned by tests against brute
 * force, closed forms (Theorem 1) and invariants.
 *
 * Arithmetic conventions: "exact" sums are taken in double (every HIF4 value
 * has at most 6 significant bits, so products and their sums are exact in
 * double for the sizes used); fl32() is a rounding to binary32; rn_f16() is a
 * rounding to binary16 (ties to even, subnormals kept).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* Rounding to narrower binary formats (ties to even).                 */
/* ------------------------------------------------------------------ */

/* Round x to a binary format with `sig` significand bits (implicit one
 * included), minimum normal exponent `emin` and largest finite `maxv`. */
static double round_to_format(double x, int sig, int emin, double maxv)
{
    if (x == 0.0 || isnan(x) || isinf(x)) return x;
    double ax = fabs(x);
    int e;
    frexp(ax, &e);            /* ax = f * 2^e, f in [0.5, 1)  => leading bit 2^(e-1) */
    int lead = e - 1;
    if (lead < emin) lead = emin;               /* subnormal range: fixed quantum */
    double quantum = ldexp(1.0, lead - (sig - 1));
    double r = nearbyint(ax / quantum) * quantum; /* default mode: ties to even */
    if (r > maxv) r = INFINITY;
    return x < 0 ? -r : r;
}

double hifa4_oracle_rn_f16(double x)  { return round_to_format(x, 11, -14, 65504.0); }
double hifa4_oracle_rn_bf16(double x) { return round_to_format(x, 8, -126, 0x1.FEp127); }
static float fl32(double x) { return (float)x; }

/* dtype codes used throughout: 0 = fp16, 1 = bf16, 2 = fp32, 3 = fp64 (no rounding) */
static double round_dtype(double x, int dtype)
{
    switch (dtype) {
    case 0: return hifa4_oracle_rn_f16(x);
    case 1: return hifa4_oracle_rn_bf16(x);
    case 2: return (double)fl32(x);
    default: return x;
    }
}

/* ------------------------------------------------------------------ */
/* HIF4 (Background, "HIF4"): 64 elements + 32 metadata bits.          */
/*   metadata byte 0      : E6M2 level-1 scale code, S = 2^(e-48)(1+M/4) */
/*   metadata byte 1      : 8 level-2 bits a[u], u = i/8               */
/*   metadata bytes 2..3  : 16 level-3 bits b[t], t = i/4              */
/*   element nibble       : sign<<3 | m, magnitude m/4 (S1P2)          */
/*   value_i = +-S * 2^(a[i/8]+b[i/4]) * m_i/4                         */
/* ------------------------------------------------------------------ */

double hifa4_oracle_e6m2_value(int code)
{
    int e = (code >> 2) & 63, M = code & 3;
    return ldexp(1.0 + M / 4.0, e - 48);
}

static double hif4_step(uint32_t meta, int i)
{
    double S = hifa4_oracle_e6m2_value((int)(meta & 0xFF));
    int a = (meta >> (8 + i / 8)) & 1;
    int b = (meta >> (16 + i / 4)) & 1;
    return ldexp(S, a + b - 2);      /* S * 2^(a+b) / 4 */
}

void hifa4_oracle_hif4_decode_group(const uint8_t* nib, uint32_t meta, double* out)
{
    for (int i = 0; i < 64; ++i) {
        int m = nib[i] & 7;
        double v = m * hif4_step(meta, i);
        out[i] = (nib[i] & 8) ? -v : v;
    }
}

/* Encode one group.  x holds 64 finite values.  nib gets one nibble per
 * element (unpacked).  Reading of the conversion:
 *   level 1: the smallest E6M2 value S with 7*S >= max|x| (7*S is the
 *            largest representable magnitude, so the maximum never clips);
 *   level 2/3: every 4-element subgroup takes the smallest shift
 *            k in {0,1,2} with 1.75*S*2^k >= its maximum, made expressible
 *            as a[u]+b[t] under the shared level-2 bit of its pair;
 *   elements: nearest multiple of the step, ties to the even code.      */
void hifa4_oracle_hif4_encode_group(const double* x, uint8_t* nib, uint32_t* meta_out)
{
    double A = 0.0;
    for (int i = 0; i < 64; ++i) if (fabs(x[i]) > A) A = fabs(x[i]);
    if (A == 0.0) { memset(nib, 0, 64); *meta_out = 0; return; }

    int code = 255;
    for (int c = 0; c < 256; ++c)
        if (7.0 * hifa4_oracle_e6m2_value(c) >= A) { code = c; break; }
    double S = hifa4_oracle_e6m2_value(code);

    int need[16];
    for (int t = 0; t < 16; ++t) {
        double At = 0.0;
        for (int i = 4 * t; i < 4 * t + 4; ++i) if (fabs(x[i]) > At) At = fabs(x[i]);
        need[t] = (At <= 1.75 * S) ? 0 : (At <= 3.5 * S) ? 1 : 2;
    }
    uint32_t meta = (uint32_t)code;
    for (int u = 0; u < 8; ++u) {
        int n0 = need[2 * u], n1 = need[2 * u + 1];
        int mx = n0 > n1 ? n0 : n1, mn = n0 < n1 ? n0 : n1;
        int a = (mx == 2 || mn >= 1) ? 1 : 0;
        if (a) meta |= 1u << (8 + u);
        for (int w = 0; w < 2; ++w) {
            int b = need[2 * u + w] - a;
            if (b < 0) b = 0;
            if (b > 1) b = 1;
            if (b) meta |= 1u << (16 + 2 * u + w);
        }
    }
    for (int i = 0; i < 64; ++i) {
        double step = hif4_step(meta, i);
        double ax = fabs(x[i]);
        int m = 0;
        /* count the rounding thresholds (j + 1/2)*step that ax passes; a value
         * exactly on a threshold goes to the even neighbour */
        for (int j = 0; j < 7; ++j) {
            double thr = (j + 0.5) * step;
            if (ax > thr || (ax == thr && (j & 1))) m = j + 1;
        }
        nib[i] = (uint8_t)(m | ((x[i] < 0 && m > 0) ? 8 : 0));
    }
    *meta_out = meta;
}

/* Quantize `rows` rows of `len` values (len % 64 == 0) along the row.
 * codes: [rows][len/2] bytes, even element in the low nibble; meta:
 * [rows][len/64]; deq (optional): dequantized values [rows][len]. */
int hifa4_oracle_hif4_quantize_rows(const double* x, long rows, long len,
                                    uint8_t* codes, uint32_t* meta, double* deq)
{
    if (len % 64) return 1;
    long G = len / 64;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        for (long g = 0; g < G; ++g) {
            uint8_t nib[64];
            uint32_t mt;
            const double* xg = x + r * len + g * 64;
            hifa4_oracle_hif4_encode_group(xg, nib, &mt);
            if (meta) meta[r * G + g] = mt;
            if (codes)
                for (int i = 0; i < 32; ++i)
                    codes[r * (len / 2) + g * 32 + i] = (uint8_t)(nib[2 * i] | (nib[2 * i + 1] << 4));
            if (deq) hifa4_oracle_hif4_decode_group(nib, mt, deq + r * len + g * 64);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* Smooth-QK (Eq. "sqk", Algorithm 1 line 1).                          */
/* ------------------------------------------------------------------ */

/* y[r][c] = round_dtype(fl32(x[r][c] * scale[c]));  scale == NULL => copy.
 * dtype 3 keeps the exact double product (used for the invariance pin). */
void hifa4_oracle_smooth_apply(const float* x, long rows, int d, const float* scale,
                               int dtype, double* y)
{
    for (long r = 0; r < rows; ++r)
        for (int c = 0; c < d; ++c) {
            double v = x[r * d + c];
            if (scale) {
                if (dtype == 3) v = v * (double)scale[c];
                else v = round_dtype((double)(x[r * d + c] * scale[c]), dtype);
            }
            y[r * d + c] = v;
        }
}

static int cmp_float(const void* a, const void* b)
{
    float x = *(const float*)a, y = *(const float*)b;
    return (x > y) - (x < y);
}

/* Calibration ("Calibration-Static Deployment", "Adaptive Applicability
 * Gate").  q_cal [S][Hq][Ncal][d], k_cal [S][Hkv][Ncal][d].
 * Per sample the per-channel statistic is the maximum magnitude over tokens
 * (and, for Q, over the query heads that share the KV head); samples are
 * combined by root-mean-square (the aggregator the paper adopts) or, as the
 * alternatives of its aggregator comparison (table "calib"), by the mean or by
 * the 99th percentile (nearest rank) of the per-sample maxima.
 * s = Kagg^alpha / Qagg^(1-alpha).
 * mode: 0 bypass, 1 strong (alpha .5), 2 mild (.25), 3 gate decides, 4 alpha given;
 * plus 0x100 for the mean aggregator, 0x200 for the 99th percentile.
 * stats[0] = rho_K = max|K| / P99(|K|) (nearest rank), stats[1] = T = max|K|/max|Q|,
 * stats[2] = branch taken (0 bypass, 1 strong, 2 mild), stats[3] = alpha used. */
int hifa4_oracle_smooth_calibrate(const float* q_cal, const float* k_cal, int S, int Hq, int Hkv,
                                  int Ncal, int d, const int* q_to_kv, int mode, double alpha,
                                  float* s, float* inv_s, double* kagg_out, double* qagg_out,
                                  double* stats)
{
    const int aggregator = (mode >> 8) & 3;      /* 0 RMS, 1 mean, 2 99th percentile */
    mode &= 0xFF;
    if (aggregator > 2) return 3;
    double* kms = (double*)malloc(sizeof(double) * 2 * S);
    if (!kms) return 2;
    double* qms = kms + S;
    long nk = (long)S * Hkv * Ncal * d, nq = (long)S * Hq * Ncal * d;
    double kmaxall = 0, qmaxall = 0;
    for (long i = 0; i < nk; ++i) if (fabs(k_cal[i]) > kmaxall) kmaxall = fabs(k_cal[i]);
    for (long i = 0; i < nq; ++i) if (fabs(q_cal[i]) > qmaxall) qmaxall = fabs(q_cal[i]);
    double rho = 0, T = qmaxall > 0 ? kmaxall / qmaxall : 0;
    if (stats || mode == 3) {
        float* tmp = (float*)malloc(sizeof(float) * nk);
        if (!tmp) return 2;
        for (long i = 0; i < nk; ++i) tmp[i] = fabsf(k_cal[i]);
        qsort(tmp, nk, sizeof(float), cmp_float);
        long rank = (long)ceil(0.99 * (double)nk);          /* nearest-rank percentile */
        if (rank < 1) rank = 1;
        double p99 = tmp[rank - 1];
        rho = p99 > 0 ? kmaxall / p99 : 0;
        free(tmp);
    }
    int branch = mode;
    if (mode == 3) branch = (rho >= 6.0 && T >= 2.0) ? (T > 3.0 ? 1 : 2) : 0;
    if (branch == 1) alpha = 0.5;
    if (branch == 2) alpha = 0.25;
    if (stats) { stats[0] = rho; stats[1] = T; stats[2] = branch == 4 ? 4 : branch; stats[3] = branch ? alpha : 0; }

    for (int g = 0; g < Hkv; ++g)
        for (int c = 0; c < d; ++c) {
            double ksum = 0, qsum = 0;
            for (int n = 0; n < S; ++n) {
                double km = 0, qm = 0;
                for (int t = 0; t < Ncal; ++t) {
                    double v = fabs(k_cal[(((long)n * Hkv + g) * Ncal + t) * d + c]);
                    if (v > km) km = v;
                }
                for (int h = 0; h < Hq; ++h) {
                    int gh = q_to_kv ? q_to_kv[h] : h / (Hq / Hkv);
                    if (gh != g) continue;
                    for (int t = 0; t < Ncal; ++t) {
                        double v = fabs(q_cal[(((long)n * Hq + h) * Ncal + t) * d + c]);
                        if (v > qm) qm = v;
                    }
                }
                ksum += km * km;
                qsum += qm * qm;
                kms[n] = km;
                qms[n] = qm;
            }
            double kagg = sqrt(ksum / S), qagg = sqrt(qsum / S);
            if (aggregator == 1) {                       /* mean of the per-sample maxima */
                kagg = qagg = 0;
                for (int n = 0; n < S; ++n) { kagg += kms[n]; qagg += qms[n]; }
                kagg /= S;
                qagg /= S;
            } else if (aggregator == 2) {                /* nearest-rank 99th percentile of them */
                long rank = (long)ceil(0.99 * (double)S);
                if (rank < 1) rank = 1;
                for (int pass = 0; pass < 2; ++pass) {   /* selection by counting: S is small */
                    double* v = pass ? qms : kms;
                    double pick = 0;
                    for (int a = 0; a < S; ++a) {
                        long below = 0, not_above = 0;
                        for (int b2 = 0; b2 < S; ++b2) { below += v[b2] < v[a]; not_above += v[b2] <= v[a]; }
                        if (below < rank && rank <= not_above) { pick = v[a]; break; }
                    }
                    if (pass) qagg = pick; else kagg = pick;
                }
            }
            if (kagg_out) kagg_out[g * d + c] = kagg;
            if (qagg_out) qagg_out[g * d + c] = qagg;
            double sv = 1.0;
            if (branch != 0 && kagg > 0 && qagg > 0) sv = pow(kagg, alpha) / pow(qagg, 1.0 - alpha);
            s[g * d + c] = (float)sv;
            inv_s[g * d + c] = 1.0f / s[g * d + c];
        }
    free(kms);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Q-Mean auxiliary (Algorithm 1 lines 2 and 6; Appendix, "Q-Mean GEMV  */
/* and coordinate consistency").                                       */
/* ------------------------------------------------------------------ */

/* Line 2 on one smoothed query row qt[d] (in place): mu = mean over the d channels, kept in FP16
 * (exact = 1 keeps it in double); q_z = qt - mu rounded to the activation dtype (3 = no rounding). */
double hifa4_oracle_qmean_row(double* qt, int d, int dtype, int exact)
{
    double mu = 0;
    for (int c = 0; c < d; ++c) mu += qt[c];
    mu /= d;
    if (!exact) mu = hifa4_oracle_rn_f16(mu);
    for (int c = 0; c < d; ++c) qt[c] = dtype == 3 ? qt[c] - mu : round_dtype(qt[c] - mu, dtype);
    return mu;
}

/* The key-side vector of line 6: sum over channels of the smoothed key, kept in FP16. */
double hifa4_oracle_ksum_row(const double* kt, int d, int exact)
{
    double a = 0;
    for (int c = 0; c < d; ++c) a += kt[c];
    return exact ? a : hifa4_oracle_rn_f16(a);
}

/* Bulk forms for the parity tests: x [rows][d] raw activations, scale [d] or NULL.
 * qmean_rows: y = q_z (double), mu [rows].  ksum_rows: ks [rows]. */
void hifa4_oracle_qmean_rows(const float* x, long rows, int d, const float* scale, int dtype,
                             double* y, double* mu)
{
    hifa4_oracle_smooth_apply(x, rows, d, scale, dtype, y);
    for (long r = 0; r < rows; ++r) mu[r] = hifa4_oracle_qmean_row(y + r * d, d, dtype, 0);
}

void hifa4_oracle_ksum_rows(const float* x, long rows, int d, const float* scale, int dtype, double* ks)
{
    double* y = (double*)malloc(sizeof(double) * rows * d);
    hifa4_oracle_smooth_apply(x, rows, d, scale, dtype, y);
    for (long r = 0; r < rows; ++r) ks[r] = hifa4_oracle_ksum_row(y + r * d, d, 0);
    free(y);
}

/* ------------------------------------------------------------------ */
/* Algorithm 1 for a set of query rows that share one KV head.         */
/* ------------------------------------------------------------------ */

typedef struct {
    int N, d;             /* keys, head dim                                            */
    int causal, Bc;       /* key-tile width (multiple of 64); causal uses q_pos        */
    int in_dtype;         /* 0 f16, 1 bf16: dtype the smoothed activations round to;
                             3: keep exact products (invariance pin)                   */
    int quant_q, quant_k, quant_v, quant_p;   /* 1 = HIF4, 0 = identity               */
    int v_axis;           /* 0: V groups run along tokens, 1: along channels           */
    int normalizer;       /* 0 consistent (P-Reordering), 1 mismatched                 */
    int qmean;            /* Algorithm 1 lines 2 and 6                                 */
    int state;            /* 0: FP16 softmax state as in the paper, 1: all double      */
    int p_dtype;          /* 0: P rounded to FP16 before quantization, 2: FP32         */
    int out_dtype;        /* 0 f16, 1 bf16, 2 f32, 3 f64                               */
    double softmax_scale; /* 0 => 1/sqrt(d)                                            */
} hifa4_oracle_params;

/* q_rows [R][d] raw queries, q_pos [R] their token index, k,v [N][d] raw,
 * s/inv_s [d] or NULL (bypass).  out [R][d].  Optional dumps (NULL to skip):
 *   p_codes [R][N]  nibble of every P-hat element (0 where a key tile is skipped)
 *   p_step  [R][N/4] step of every 4-key subgroup (0 where skipped or where the group is all zero)
 *   p_raw   [R][N]  P before quantization,  p_hat [R][N] dequantized P-hat
 *   m_trace [R][N/Bc] running max after each processed tile (NaN if skipped)
 *   l_out   [R]     accumulated normalizer before the final division         */
int hifa4_oracle_attention_rows(const hifa4_oracle_params* p, const float* q_rows,
                                const int* q_pos, int R, const float* k, const float* v,
                                const float* s, const float* inv_s, double* out,
                                uint8_t* p_codes, float* p_step, double* p_raw, double* p_hat,
                                double* m_trace, double* l_out)
{
    const int N = p->N, d = p->d, Bc = p->Bc;
    if (N % 64 || d % 64 || Bc % 64 || Bc <= 0) return 1;
    if (p->quant_v && p->v_axis == 0 && N % 64) return 1;
    const double sigma = p->softmax_scale != 0 ? p->softmax_scale : 1.0 / sqrt((double)d);
    const double LOG2E = 1.4426950408889634074;
    const float c0 = fl32(sigma), c1 = fl32(sigma * LOG2E), L = fl32(LOG2E);

    /* lines 1-3: smooth, (Q-Mean), quantize.  K-hat, V-hat as doubles. */
    double* kt = (double*)malloc(sizeof(double) * N * d);     /* K-tilde */
    double* kh = (double*)malloc(sizeof(double) * N * d);
    double* vh = (double*)malloc(sizeof(double) * N * d);
    double* ksum = (double*)calloc(N, sizeof(double));
    if (!kt || !kh || !vh || !ksum) return 2;
    hifa4_oracle_smooth_apply(k, N, d, inv_s, p->in_dtype, kt);
    if (p->quant_k) hifa4_oracle_hif4_quantize_rows(kt, N, d, NULL, NULL, kh);
    else memcpy(kh, kt, sizeof(double) * N * d);
    if (p->qmean)
        for (int j = 0; j < N; ++j) ksum[j] = hifa4_oracle_ksum_row(kt + (long)j * d, d, p->state);
    for (long i = 0; i < (long)N * d; ++i) vh[i] = v[i];
    if (p->quant_v) {
        if (p->v_axis == 1) {
            double* tmp = (double*)malloc(sizeof(double) * N * d);
            memcpy(tmp, vh, sizeof(double) * N * d);
            hifa4_oracle_hif4_quantize_rows(tmp, N, d, NULL, NULL, vh);
            free(tmp);
        } else {                                   /* groups of 64 tokens per channel */
            double* vt = (double*)malloc(sizeof(double) * N * d);
            double* vq = (double*)malloc(sizeof(double) * N * d);
            for (int j = 0; j < N; ++j) for (int c = 0; c < d; ++c) vt[(long)c * N + j] = vh[(long)j * d + c];
            hifa4_oracle_hif4_quantize_rows(vt, d, N, NULL, NULL, vq);
            for (int j = 0; j < N; ++j) for (int c = 0; c < d; ++c) vh[(long)j * d + c] = vq[(long)c * N + j];
            free(vt); free(vq);
        }
    }

    int err = 0;
#pragma omp parallel for schedule(dynamic, 4)
    for (int row = 0; row < R; ++row) {
        double* qt = (double*)malloc(sizeof(double) * d);
        double* qh = (double*)malloc(sizeof(double) * d);
        double* O = (double*)calloc(d, sizeof(double));
        double* acc = (double*)malloc(sizeof(double) * Bc);
        double* P = (double*)malloc(sizeof(double) * Bc);
        double* Ph = (double*)malloc(sizeof(double) * Bc);
        uint8_t* nib = (uint8_t*)malloc(Bc);
        uint32_t* pmeta = (uint32_t*)malloc(sizeof(uint32_t) * (Bc / 64));
        if (!qt || !qh || !O || !acc || !P || !Ph || !nib || !pmeta) { err = 2; goto done; }

        hifa4_oracle_smooth_apply(q_rows + (long)row * d, 1, d, s, p->in_dtype, qt);
        double mu = 0;
        if (p->qmean) mu = hifa4_oracle_qmean_row(qt, d, p->in_dtype, p->state);
        if (p->quant_q) hifa4_oracle_hif4_quantize_rows(qt, 1, d, NULL, NULL, qh);
        else memcpy(qh, qt, sizeof(double) * d);

        double m = -INFINITY, ell = 0;
        const int last_key = p->causal ? q_pos[row] : N - 1;
        if (p_codes) memset(p_codes + (long)row * N, 0, N);
        if (p_step) memset(p_step + (long)row * (N / 4), 0, sizeof(float) * (N / 4));
        if (p_raw) memset(p_raw + (long)row * N, 0, sizeof(double) * N);
        if (p_hat) memset(p_hat + (long)row * N, 0, sizeof(double) * N);
        if (m_trace) for (int t = 0; t < N / Bc + (N % Bc != 0); ++t) m_trace[(long)row * ((N + Bc - 1) / Bc) + t] = NAN;

        for (int j0 = 0; j0 < N && j0 <= last_key; j0 += Bc) {
            const int w = (N - j0 < Bc) ? N - j0 : Bc;       /* ragged last tile: multiple of 64 */
            /* line 5 (+ line 6): raw accumulators */
            double amax = -INFINITY;
            for (int j = 0; j < w; ++j) {
                if (j0 + j > last_key) { acc[j] = -INFINITY; continue; }
                double a = 0;
                for (int c = 0; c < d; ++c) a += qh[c] * kh[(long)(j0 + j) * d + c];
                if (p->qmean) a += mu * ksum[j0 + j];
                if (!p->state) a = (double)fl32(a);
                acc[j] = a;
                if (a > amax) amax = a;
            }
            /* lines 7-9 */
            if (p->state) {
                double m_new = fmax(m, amax * sigma);
                double r = (m == -INFINITY) ? 0.0 : exp(m - m_new);
                for (int c = 0; c < d; ++c) O[c] *= r;
                ell *= r;
                m = m_new;
                for (int j = 0; j < w; ++j) P[j] = (acc[j] == -INFINITY) ? 0.0 : exp(acc[j] * sigma - m);
            } else {
                double m_new = fmax(m, hifa4_oracle_rn_f16((double)(fl32(amax) * c0)));
                double r = (m == -INFINITY) ? 0.0 : hifa4_oracle_rn_f16(exp(m - m_new));
                for (int c = 0; c < d; ++c) O[c] = (double)fl32(r * O[c]);
                ell = (double)fl32(r * ell);
                m = m_new;
                const float mL = fl32(m) * L;
                for (int j = 0; j < w; ++j) {
                    if (acc[j] == -INFINITY) { P[j] = 0.0; continue; }
                    float t = fmaf(fl32(acc[j]), c1, -mL);
                    double e = (double)fl32(exp2((double)t));
                    P[j] = p->p_dtype == 0 ? hifa4_oracle_rn_f16(e) : e;
                }
            }
            /* line 10: quantize P in 64-key groups aligned to the key index */
            for (int g = 0; g < w / 64; ++g) {
                if (p->quant_p) {
                    hifa4_oracle_hif4_encode_group(P + 64 * g, nib + 64 * g, &pmeta[g]);
                    hifa4_oracle_hif4_decode_group(nib + 64 * g, pmeta[g], Ph + 64 * g);
                } else {
                    memcpy(Ph + 64 * g, P + 64 * g, sizeof(double) * 64);
                    memset(nib + 64 * g, 0, 64);
                    pmeta[g] = 0;
                }
            }
            for (int j = 0; j < w; ++j) {
                if (p_codes) p_codes[(long)row * N + j0 + j] = nib[j];
                if (p_step && p->quant_p && (j % 4) == 0)      /* an all-zero group (metadata 0) reports step 0 */
                    p_step[(long)row * (N / 4) + (j0 + j) / 4] =
                        pmeta[j / 64] ? (float)hif4_step(pmeta[j / 64], j % 64) : 0.0f;
                if (p_raw) p_raw[(long)row * N + j0 + j] = P[j];
                if (p_hat) p_hat[(long)row * N + j0 + j] = Ph[j];
            }
            /* line 11: [O | l] += P-hat [V-hat | 1]  (mismatched: l from P) */
            for (int c = 0; c < d; ++c) {
                double a = 0;
                for (int j = 0; j < w; ++j) a += Ph[j] * vh[(long)(j0 + j) * d + c];
                O[c] = p->state ? O[c] + a : (double)fl32(O[c] + a);
            }
            double ls = 0;
            const double* src = p->normalizer == 0 ? Ph : P;
            for (int j = 0; j < w; ++j) ls += src[j];
            ell = p->state ? ell + ls : (double)fl32(ell + ls);
            if (m_trace) m_trace[(long)row * ((N + Bc - 1) / Bc) + j0 / Bc] = m;
        }
        /* line 13 */
        if (l_out) l_out[row] = ell;
        for (int c = 0; c < d; ++c) {
            if (p->state) out[(long)row * d + c] = O[c] / ell;
            else {
                float l16 = fl32(hifa4_oracle_rn_f16(ell));
                out[(long)row * d + c] = round_dtype((double)(fl32(O[c]) / l16), p->out_dtype);
            }
        }
    done:
        free(qt); free(qh); free(O); free(acc); free(P); free(Ph); free(nib); free(pmeta);
    }
    free(kt); free(kh); free(vh); free(ksum);
    return err;
}

int hifa4_oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
