/*
 * RAC reference-aware activation codec -- plain CPU oracle (TEST INFRASTRUCTURE).
 *
 * This file is a slow, scalar restatement of the method, written from the
 * paper's equations.  It exists only so that tests (and the reported CPU
 * baseline of the benchmark) have something independent to compare the CUDA
 * path with.  The product never calls it and it shares no code with the CUDA
 * sources.
 *
 * What follows which passage of the paper (Sec. IV-B, IV-C):
 *   orc_match_spans      Sec. IV-B.1, Eq. 3: w-token windows over the history,
 *                        every hit extended to its longest exact match, at most
 *                        K most recent hits per distinct window, selection by
 *                        lexargmax(length, recency), scan advances by the span
 *                        length or by one.  orc_match_spans_req: the history as a
 *                        list of earlier requests (candidates stay inside one
 *                        request) and the intra-sequence references of uncovered
 *                        repeated tokens.
 *   orc_encode           Sec. IV-C: grouped affine fit (Eq. 6) with the
 *                        zero-variance rule, wire rounding of the coefficients,
 *                        aligned reference and residual (Eq. 7), outlier split
 *                        (unnumbered equation before Eq. 8, outlier values kept
 *                        as FP16), symmetric b-bit quantisation with
 *                        Qmax = 2^(b-1)-1 and round-to-nearest (Eq. 8), packing.
 *   orc_reconstruct      Eq. 9: dequantise, restore outliers, add the aligned
 *                        reference.  Sender and receiver run this same function.
 *   orc_calibrate        "offline calibration" of Sec. IV-C reduced to the one
 *                        thing the codec needs as an input: a per-channel step
 *                        from the RMS of the aligned residual.
 *   orc_calibrate_shared the same with the wire words of every token given
 *                        from outside (Eq. 6 solved over several positions).
 *
 * Readings taken where the paper is silent:
 *   - one fit per (token, group): the "fitting positions" of Eq. 6 are the
 *     channels of one group of one token;
 *   - Round_wire of the coefficients is IEEE binary16 round-to-nearest-even,
 *     saturating at +-65504;
 *   - zero variance means centred Sxx <= 1e-12, or a slope that binary16 cannot
 *     hold (|Sxy| >= 65504*Sxx), or no reference at all;
 *   - scale_mode 0 (the graded variant): the quantiser step is a static
 *     per-channel table (two rows: tokens with a reference, tokens coded
 *     directly) instead of Eq. 8's per-group dynamic scale, so dense values can
 *     clip; step 0 means "code 0";
 *   - scale_mode 1 (Eq. 8 as printed): per (token, group) scale
 *     s = RoundUp_binary16(max|E^d| / Qmax), carried in the record; an all-zero
 *     group carries scale 0 and codes 0 (the "zero marker"); no dense clipping;
 *     the scale, its reciprocal and the scaled value are binary32 operations
 *     (max / Qmax, 1 / s, e * (1/s)) because they decide codes;
 *   - still scale_mode 1, the rest of the quantiser family of Sec. IV-C: the
 *     quantisation group g_q may differ from the alignment group g_a (g_q = d
 *     is the decode mode: one scale per token), the code width may be 8, and
 *     the outlier mask may pick the k_g largest |e| of every quantisation
 *     group (ranked like the per-token form, ties to the lower channel),
 *     serialised as one-byte in-group offsets in ascending order plus binary16
 *     values, which needs g_q <= 256;
 *   - outliers are the k largest |e| per TOKEN (not per group), ranked on the
 *     fp32 bit pattern of |e|, ties to the lower channel, stored with u16
 *     absolute channel indices in ascending order;
 *   - round-to-nearest is ties-to-even;
 *   - the residual, the scaled value, the rounding decision and the
 *     reconstruction are taken in binary32 with one rounding per operation
 *     (fused multiply-add where written as fmaf), because these decide integer
 *     codes and two endpoints must agree bit for bit; the fit itself is done
 *     in binary64.
 *
 * Wire record of one token (all little endian), records back to back:
 *   coef    J  x u32   binary16 alpha in bits 0..15, binary16 beta in bits 16..31
 *   scale   J  x u16   binary16, scale_mode 1 only, padded to a multiple of 4 bytes
 *   codes   d*b/8 B    code of channel c occupies stream bits [c*b, c*b+b),
 *                      stream bit n is bit (n%8) of byte (n/8); two's complement
 *   out_idx k  x u16   ascending
 *   out_val k  x u16   binary16
 *   grp_off Jq*kg x u8 in-group offsets of the per-group outliers, ascending
 *                      within a group, padded to a multiple of 2 bytes
 *   grp_val Jq*kg x u16 binary16                     (Jq = d/g_q, scale has Jq entries)
 *   padding to a multiple of 16 bytes (zero)
 *
 * Parity status: the LS fit, residual identity, quantiser bounds, packing,
 * outlier selection and the matcher are pinned by tests against closed forms,
 * library least squares, brute force and invariants.  The wire layout, the
 * coefficient format, the static step table and the tie rules are this
 * build's own definitions ("parity unpinned" by the paper): only round trips
 * and the properties above pin them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* number formats                                                      */
/* ------------------------------------------------------------------ */

static float bits_to_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static uint32_t f32_to_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

float orc_bf16_to_f32(uint16_t h) { return bits_to_f32((uint32_t)h << 16); }

/* binary32 -> bfloat16, round to nearest even (NaN kept quiet). */
uint16_t orc_f32_to_bf16(float f) {
    uint32_t u = f32_to_bits(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* binary16 -> binary64 (exact). */
double orc_f16_to_f64(uint16_t h) {
    int sign = (h >> 15) & 1;
    int ex = (h >> 10) & 0x1f;
    int man = h & 0x3ff;
    double v;
    if (ex == 0) v = ldexp((double)man, -24);
    else if (ex == 31) v = man ? NAN : INFINITY;
    else v = ldexp((double)(man | 0x400), ex - 25);
    return sign ? -v : v;
}
float orc_f16_to_f32(uint16_t h) { return (float)orc_f16_to_f64(h); }

/* binary64 -> binary16, round to nearest even in ONE rounding, saturating to
 * +-65504 (so never infinity).  NaN gives 0x7e00. */
uint16_t orc_f64_to_f16(double x) {
    if (isnan(x)) return 0x7e00;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a >= 65504.0) return sign | 0x7bff;
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);               /* a = m * 2^e, m in [0.5,1) */
    int ulp_exp = e - 11;             /* 11 significant bits for normals   */
    if (ulp_exp < -24) ulp_exp = -24; /* subnormal spacing 2^-24           */
    double scaled = ldexp(a, -ulp_exp);     /* exact                      */
    double r = nearbyint(scaled);           /* default mode: ties to even  */
    double v = ldexp(r, ulp_exp);
    if (v >= 65520.0) return sign | 0x7bff;
    /* re-encode v, which is exactly representable */
    if (v == 0.0) return sign;
    int e2;
    double m2 = frexp(v, &e2);        /* v = m2 * 2^e2 */
    if (e2 - 1 < -14) {               /* subnormal */
        return sign | (uint16_t)ldexp(v, 24);
    }
    uint16_t ex = (uint16_t)(e2 - 1 + 15);
    uint16_t man = (uint16_t)(ldexp(m2, 11)) & 0x3ff;
    return sign | (uint16_t)(ex << 10) | man;
}

/* smallest binary16 value >= x, for x >= 0 (used for step tables so that the
 * stored step never shrinks the range, mirroring RoundUp_wire of Eq. 8). */
uint16_t orc_f64_to_f16_up(double x) {
    uint16_t h = orc_f64_to_f16(x);
    if (orc_f16_to_f64(h) < x && h < 0x7bff) h++;
    return h;
}

/* ------------------------------------------------------------------ */
/* record geometry                                                     */
/* ------------------------------------------------------------------ */

static int64_t scale_bytes(int d, int qgroup, int scale_mode) {
    return scale_mode == 1 ? (2 * (int64_t)(d / qgroup) + 3) / 4 * 4 : 0;
}

/* in-group offsets of the per-group outliers: one byte each while a group has at most 256 channels, two
 * (little endian) for wider groups; the field is padded to an even number of bytes */
static int goff_width(int qgroup) { return qgroup > 256 ? 2 : 1; }
static int64_t goff_bytes(int64_t ng, int qgroup) { return (ng * goff_width(qgroup) + 1) / 2 * 2; }

/* qgroup 0 means "same as group"; topk_group outliers per quantisation group; coef_fmt 1: the coefficient
 * pairs are shared by the tokens of a segment and travel outside the record */
int64_t orc_record_bytes_full(int d, int group, int bits, int topk, int scale_mode, int qgroup, int topk_group, int coef_fmt) {
    if (qgroup == 0) qgroup = group;
    int64_t ng = (int64_t)(d / qgroup) * topk_group;
    int64_t raw = (coef_fmt == 1 ? 0 : 4 * (int64_t)(d / group)) + scale_bytes(d, qgroup, scale_mode) + ((int64_t)d * bits) / 8 +
                  4 * (int64_t)topk + goff_bytes(ng, qgroup) + 2 * ng;
    return (raw + 15) / 16 * 16;
}

int64_t orc_record_bytes_ext(int d, int group, int bits, int topk, int scale_mode, int qgroup, int topk_group) {
    return orc_record_bytes_full(d, group, bits, topk, scale_mode, qgroup, topk_group, 0);
}

int64_t orc_record_bytes_mode(int d, int group, int bits, int topk, int scale_mode) {
    return orc_record_bytes_ext(d, group, bits, topk, scale_mode, 0, 0);
}

int64_t orc_record_bytes(int d, int group, int bits, int topk) { return orc_record_bytes_mode(d, group, bits, topk, 0); }

static int cfg_ok(int d, int group, int bits, int topk) {
    if (d <= 0 || group <= 0 || d % group) return 0;
    if (bits < 2 || bits > 8) return 0;
    if (((int64_t)d * bits) % 8) return 0;
    if (topk < 0 || topk > d || d > 65536) return 0;
    return 1;
}

/* the quantisation group and the per-group outliers exist in scale_mode 1 only */
static int qcfg_ok(int d, int group, int topk, int scale_mode, int qgroup, int topk_group) {
    if (scale_mode != 0 && scale_mode != 1) return 0;
    if (qgroup < 0 || topk_group < 0) return 0;
    if (scale_mode == 0) return (qgroup == 0 || qgroup == group) && topk_group == 0;
    if (qgroup == 0) qgroup = group;
    if (d % qgroup) return 0;
    if (topk_group && (topk || qgroup > 65536 || topk_group > qgroup)) return 0;
    return 1;
}

static void put_code(uint8_t *codes, int c, int bits, int q) {
    uint32_t v = (uint32_t)q & ((1u << bits) - 1u);
    int64_t bit = (int64_t)c * bits;
    for (int n = 0; n < bits; n++, bit++) {
        if ((v >> n) & 1u) codes[bit >> 3] |= (uint8_t)(1u << (bit & 7));
    }
}

static int get_code(const uint8_t *codes, int c, int bits) {
    uint32_t v = 0;
    int64_t bit = (int64_t)c * bits;
    for (int n = 0; n < bits; n++, bit++) {
        v |= (uint32_t)((codes[bit >> 3] >> (bit & 7)) & 1u) << n;
    }
    if (v & (1u << (bits - 1))) return (int)v - (1 << bits);
    return (int)v;
}

/* exported for the packing tests */
void orc_pack_codes(const int32_t *q, int d, int bits, uint8_t *codes) {
    memset(codes, 0, ((size_t)d * bits) / 8);
    for (int c = 0; c < d; c++) put_code(codes, c, bits, q[c]);
}
void orc_unpack_codes(const uint8_t *codes, int d, int bits, int32_t *q) {
    for (int c = 0; c < d; c++) q[c] = get_code(codes, c, bits);
}

/* ------------------------------------------------------------------ */
/* reference row of one token                                          */
/* ------------------------------------------------------------------ */

/* Returns 1 when the token has a reference, 0 when it is coded directly, and
 * -1 when ref_row points outside the buffer.  r[] receives the reference as
 * binary32 (zeros when there is none).  The optional per-channel transform is
 * the stand-in for the decode predictor of Eq. 5: r <- bf16(gain*r + bias). */
static int resolve_ref(int d, int64_t t, const uint16_t *ref_base, int64_t ref_rows,
                       const int32_t *ref_row, const uint16_t *gain, const uint16_t *bias,
                       float *r) {
    int64_t row = ref_row ? (int64_t)ref_row[t] : t;
    if (!ref_base || row < 0) {
        for (int c = 0; c < d; c++) r[c] = 0.0f;
        return 0;
    }
    if (row >= ref_rows) return -1;
    const uint16_t *src = ref_base + row * (int64_t)d;
    for (int c = 0; c < d; c++) {
        float v = orc_bf16_to_f32(src[c]);
        if (gain) {
            float gsc = orc_f16_to_f32(gain[c]);
            float bsc = orc_f16_to_f32(bias[c]);
            v = orc_bf16_to_f32(orc_f32_to_bf16(fmaf(gsc, v, bsc)));
        }
        r[c] = v;
    }
    return 1;
}

/* ------------------------------------------------------------------ */
/* Eq. 6: least-squares (alpha, beta) of one group                     */
/* ------------------------------------------------------------------ */

/* h, r: g values.  Outputs the unrounded optimum and the two means. */
void orc_fit_group(const float *h, const float *r, int g, int has_ref,
                   double *alpha_star, double *beta_star, double *hbar_out, double *rbar_out) {
    double sr = 0.0, sh = 0.0;
    for (int i = 0; i < g; i++) { sr += (double)r[i]; sh += (double)h[i]; }
    double rbar = sr / g, hbar = sh / g;
    double sxx = 0.0, sxy = 0.0;
    for (int i = 0; i < g; i++) {
        double dr = (double)r[i] - rbar;
        double dh = (double)h[i] - hbar;
        sxx += dr * dr;
        sxy += dr * dh;
    }
    int degenerate = !has_ref || !(sxx > 1e-12) || !(fabs(sxy) < 65504.0 * sxx);
    if (degenerate) { *alpha_star = 0.0; *beta_star = hbar; }
    else { double a = sxy / sxx; *alpha_star = a; *beta_star = hbar - a * rbar; }
    if (hbar_out) *hbar_out = hbar;
    if (rbar_out) *rbar_out = rbar;
}

/* Eq. 6 with several fitting positions: one (alpha, beta) per (segment, group), H_j and R_j being the
 * [positions x g] slices of the segment's tokens (a token coded directly contributes r = 0).
 * seg_off int32[n_seg+1], ascending, seg_off[0] = 0, seg_off[n_seg] = T.
 * coef_out u32[n_seg*J] wire words; diag_* optional double[n_seg*J] (unrounded optimum and the two means).
 * Centred two-pass sums in binary64 over all positions of the segment. */
int orc_fit_segments(int d, int group, const uint16_t *X, int64_t T,
                     const uint16_t *ref_base, int64_t ref_rows, const int32_t *ref_row,
                     const uint16_t *gain, const uint16_t *bias,
                     const int32_t *seg_off, int32_t n_seg, uint32_t *coef_out,
                     double *diag_alpha, double *diag_beta, double *diag_hbar, double *diag_rbar) {
    if (d <= 0 || group <= 0 || d % group || n_seg < 0) return -1;
    if ((gain == NULL) != (bias == NULL)) return -1;
    if (n_seg > 0 && (seg_off[0] != 0 || seg_off[n_seg] != T)) return -1;
    const int J = d / group;
    float *r = (float *)malloc(sizeof(float) * d);
    int err = 0;
    for (int32_t k = 0; k < n_seg && !err; k++) {
        const int64_t t0 = seg_off[k], t1 = seg_off[k + 1];
        if (t1 < t0) { err = -1; break; }
        for (int j = 0; j < J; j++) {
            double sr = 0.0, sh = 0.0;
            int any_ref = 0;
            for (int64_t t = t0; t < t1; t++) {
                int has = resolve_ref(d, t, ref_base, ref_rows, ref_row, gain, bias, r);
                if (has < 0) { err = -2; break; }
                any_ref |= has;
                for (int c = j * group; c < (j + 1) * group; c++) {
                    sr += (double)r[c];
                    sh += (double)orc_bf16_to_f32(X[t * (int64_t)d + c]);
                }
            }
            if (err) break;
            const double n = (double)(t1 - t0) * group;
            double rbar = n > 0 ? sr / n : 0.0, hbar = n > 0 ? sh / n : 0.0;
            double sxx = 0.0, sxy = 0.0;
            for (int64_t t = t0; t < t1; t++) {
                resolve_ref(d, t, ref_base, ref_rows, ref_row, gain, bias, r);
                for (int c = j * group; c < (j + 1) * group; c++) {
                    double dr = (double)r[c] - rbar;
                    double dh = (double)orc_bf16_to_f32(X[t * (int64_t)d + c]) - hbar;
                    sxx += dr * dr;
                    sxy += dr * dh;
                }
            }
            int degenerate = !any_ref || !(sxx > 1e-12) || !(fabs(sxy) < 65504.0 * sxx);
            double as = 0.0, bs = hbar;
            if (!degenerate) { as = sxy / sxx; bs = hbar - as * rbar; }
            coef_out[(int64_t)k * J + j] = (uint32_t)orc_f64_to_f16(as) | ((uint32_t)orc_f64_to_f16(bs) << 16);
            if (diag_alpha) diag_alpha[(int64_t)k * J + j] = as;
            if (diag_beta) diag_beta[(int64_t)k * J + j] = bs;
            if (diag_hbar) diag_hbar[(int64_t)k * J + j] = hbar;
            if (diag_rbar) diag_rbar[(int64_t)k * J + j] = rbar;
        }
    }
    free(r);
    return err;
}

/* ------------------------------------------------------------------ */
/* encode                                                              */
/* ------------------------------------------------------------------ */

static float clampf(float v, float lo, float hi) { return fminf(fmaxf(v, lo), hi); }

/*
 * X            bf16[T,d]
 * ref_base     bf16[ref_rows,d] or NULL (every token direct)
 * ref_row      int32[T] or NULL (identity); negative = direct
 * gain, bias   binary16[d] or both NULL
 * step,inv_step float[2,d]: row 0 for tokens with a reference, row 1 direct
 * forced_coef  u32[T,J] or NULL; when given the fit is skipped and these wire
 *              coefficients are used (tests use this to separate a coefficient
 *              rounding flip from everything downstream of it)
 * payload      T*record bytes out
 * diag_*       optional outputs (NULL to skip): unrounded alpha, beta, the
 *              group means (double[T,J] each), the binary32 residual e[T,d],
 *              the scaled value v[T,d] the rounding decision was taken on
 *              (binary32, e times the reciprocal of the step or scale), and
 *              v_ideal[T,d] = e / s as Eq. 8 prints it, the quotient taken in
 *              binary64 -- a diagnostic that decides no code: tests count the
 *              codes that differ from the rounding of this value (0 where the
 *              channel is an outlier or its step / scale is 0).
 * returns 0, or -1 bad configuration, -2 ref_row out of range.
 */
int orc_encode(int d, int group, int bits, int topk, int scale_mode, int qgroup, int topk_group, int coef_fmt,
               const uint16_t *X, int64_t T,
               const uint16_t *ref_base, int64_t ref_rows, const int32_t *ref_row,
               const uint16_t *gain, const uint16_t *bias,
               const float *step, const float *inv_step,
               const uint32_t *forced_coef,
               uint8_t *payload,
               double *diag_alpha, double *diag_beta, double *diag_hbar, double *diag_rbar,
               float *diag_e, float *diag_v, double *diag_v_ideal, int nthreads) {
    if (!cfg_ok(d, group, bits, topk)) return -1;
    if (!qcfg_ok(d, group, topk, scale_mode, qgroup, topk_group)) return -1;
    if ((gain == NULL) != (bias == NULL)) return -1;
    if (coef_fmt != 0 && coef_fmt != 1) return -1;
    if (coef_fmt == 1 && !forced_coef) return -1;      /* shared coefficients come from outside */
    if (qgroup == 0) qgroup = group;
    const int J = d / group, Jq = d / qgroup;
    const int64_t rec = orc_record_bytes_full(d, group, bits, topk, scale_mode, qgroup, topk_group, coef_fmt);
    const int64_t sbytes = scale_bytes(d, qgroup, scale_mode);
    const int64_t cbytes = coef_fmt == 1 ? 0 : 4 * (int64_t)J;
    const int qmax = (1 << (bits - 1)) - 1;
    int err = 0;
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel num_threads(nthreads)
    {
        float *h = (float *)malloc(sizeof(float) * d);
        float *r = (float *)malloc(sizeof(float) * d);
        float *e = (float *)malloc(sizeof(float) * d);
        uint8_t *is_out = (uint8_t *)malloc(d);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < T; t++) {
            uint8_t *recp = payload + t * rec;
            memset(recp, 0, rec);
            uint32_t *coef = (uint32_t *)recp;
            uint8_t *scales = recp + cbytes;
            uint8_t *codes = scales + sbytes;
            uint8_t *oidx = codes + ((int64_t)d * bits) / 8;
            uint8_t *oval = oidx + 2 * topk;
            uint8_t *goff = oval + 2 * topk;
            uint8_t *gval = goff + goff_bytes((int64_t)Jq * topk_group, qgroup);

            for (int c = 0; c < d; c++) h[c] = orc_bf16_to_f32(X[t * (int64_t)d + c]);
            int has_ref = resolve_ref(d, t, ref_base, ref_rows, ref_row, gain, bias, r);
            if (has_ref < 0) {
#pragma omp atomic write
                err = -2;
                continue;
            }
            /* Eq. 6 + wire rounding, then Eq. 7 in binary32 */
            for (int j = 0; j < J; j++) {
                uint16_t a16, b16;
                double as = 0, bs = 0, hb = 0, rb = 0;
                orc_fit_group(h + j * group, r + j * group, group, has_ref, &as, &bs, &hb, &rb);
                if (forced_coef) {
                    uint32_t w = forced_coef[t * J + j];
                    a16 = (uint16_t)(w & 0xffff); b16 = (uint16_t)(w >> 16);
                } else {
                    a16 = orc_f64_to_f16(as); b16 = orc_f64_to_f16(bs);
                }
                uint32_t w = (uint32_t)a16 | ((uint32_t)b16 << 16);
                if (coef_fmt == 0) memcpy(&coef[j], &w, 4);
                if (diag_alpha) diag_alpha[t * J + j] = as;
                if (diag_beta) diag_beta[t * J + j] = bs;
                if (diag_hbar) diag_hbar[t * J + j] = hb;
                if (diag_rbar) diag_rbar[t * J + j] = rb;
                float a = orc_f16_to_f32(a16), b = orc_f16_to_f32(b16);
                for (int c = j * group; c < (j + 1) * group; c++) {
                    float rt = fmaf(a, r[c], b);
                    e[c] = h[c] - rt;
                }
            }
            /* outlier split: k largest |e| of the token, ties to the lower channel */
            memset(is_out, 0, d);
            for (int n = 0; n < topk; n++) {
                int best = -1; uint32_t bestkey = 0;
                for (int c = 0; c < d; c++) {
                    if (is_out[c]) continue;
                    uint32_t key = f32_to_bits(e[c]) & 0x7fffffffu;
                    if (best < 0 || key > bestkey) { best = c; bestkey = key; }
                }
                is_out[best] = 1;
            }
            {
                int n = 0;
                for (int c = 0; c < d; c++) {
                    if (!is_out[c]) continue;
                    uint16_t ci = (uint16_t)c;
                    uint16_t hv = orc_f64_to_f16((double)clampf(e[c], -65504.0f, 65504.0f));
                    memcpy(oidx + 2 * n, &ci, 2);
                    memcpy(oval + 2 * n, &hv, 2);
                    n++;
                }
            }
            /* per-group form of the mask (Sec. IV-C, "Outlier Metadata"): the k_g largest |e| of every
             * quantisation group, in-group offsets in ascending order, values as binary16 */
            for (int j = 0; j < Jq && topk_group; j++) {
                for (int n = 0; n < topk_group; n++) {
                    int best = -1; uint32_t bestkey = 0;
                    for (int c = j * qgroup; c < (j + 1) * qgroup; c++) {
                        if (is_out[c]) continue;
                        uint32_t key = f32_to_bits(e[c]) & 0x7fffffffu;
                        if (best < 0 || key > bestkey) { best = c; bestkey = key; }
                    }
                    is_out[best] = 1;
                }
                int n = 0;
                for (int c = j * qgroup; c < (j + 1) * qgroup; c++) {
                    if (!is_out[c]) continue;
                    uint16_t hv = orc_f64_to_f16((double)clampf(e[c], -65504.0f, 65504.0f));
                    const int o = c - j * qgroup;
                    if (goff_width(qgroup) == 1) {
                        goff[j * topk_group + n] = (uint8_t)o;
                    } else {
                        goff[2 * (j * topk_group + n)] = (uint8_t)(o & 0xff);
                        goff[2 * (j * topk_group + n) + 1] = (uint8_t)(o >> 8);
                    }
                    memcpy(gval + 2 * (j * topk_group + n), &hv, 2);
                    n++;
                }
            }
            if (scale_mode == 0) {
                /* Eq. 8 with the static table, then packing */
                const float *st = step + (has_ref ? 0 : d);
                const float *ist = inv_step + (has_ref ? 0 : d);
                for (int c = 0; c < d; c++) {
                    int q = 0;
                    float v = 0.0f;
                    double v_ideal = 0.0;
                    if (st[c] != 0.0f && !is_out[c]) {
                        v = e[c] * ist[c];
                        q = (int)rintf(clampf(v, (float)-qmax, (float)qmax));
                        v_ideal = (double)e[c] / (double)st[c];
                    }
                    if (diag_v) diag_v[t * (int64_t)d + c] = v;
                    if (diag_v_ideal) diag_v_ideal[t * (int64_t)d + c] = v_ideal;
                    if (diag_e) diag_e[t * (int64_t)d + c] = e[c];
                    put_code(codes, c, bits, q);
                }
            } else {
                /* Eq. 8 as printed: scale of the group from its dense values, rounded UP in the wire
                 * format so that nothing clips; an all-zero group carries scale 0 and codes 0 */
                for (int j = 0; j < Jq; j++) {
                    float m = 0.0f;
                    for (int c = j * qgroup; c < (j + 1) * qgroup; c++)
                        if (!is_out[c]) m = fmaxf(m, fabsf(e[c]));
                    float s_star = m / (float)qmax;
                    uint16_t s16 = orc_f64_to_f16_up((double)s_star);
                    float sc = orc_f16_to_f32(s16);
                    float isc = sc != 0.0f ? 1.0f / sc : 0.0f;
                    memcpy(scales + 2 * j, &s16, 2);
                    for (int c = j * qgroup; c < (j + 1) * qgroup; c++) {
                        int q = 0;
                        float v = 0.0f;
                        double v_ideal = 0.0;
                        if (!is_out[c]) {
                            v = e[c] * isc;
                            q = (int)rintf(clampf(v, (float)-qmax, (float)qmax));
                            if (sc != 0.0f) v_ideal = (double)e[c] / (double)sc;
                        }
                        if (diag_v) diag_v[t * (int64_t)d + c] = v;
                        if (diag_v_ideal) diag_v_ideal[t * (int64_t)d + c] = v_ideal;
                        if (diag_e) diag_e[t * (int64_t)d + c] = e[c];
                        put_code(codes, c, bits, q);
                    }
                }
            }
        }
        free(h); free(r); free(e); free(is_out);
    }
    return err;
}

/* ------------------------------------------------------------------ */
/* Eq. 9: reconstruct (receiver and sender)                            */
/* ------------------------------------------------------------------ */

/* X_hat bf16[T,d] out.  status (optional, one word) gets bit 1 when a reserved
 * code -2^(b-1) was seen.  returns 0, -1, -2 as orc_encode; -3 when an outlier
 * index is >= d. */
int orc_reconstruct(int d, int group, int bits, int topk, int scale_mode, int qgroup, int topk_group, int coef_fmt,
                    const uint32_t *shared_coef,
                    const uint8_t *payload, int64_t T,
                    const uint16_t *ref_base, int64_t ref_rows, const int32_t *ref_row,
                    const uint16_t *gain, const uint16_t *bias,
                    const float *step, uint16_t *X_hat, uint32_t *status, int nthreads) {
    if (!cfg_ok(d, group, bits, topk)) return -1;
    if ((gain == NULL) != (bias == NULL)) return -1;
    if (!qcfg_ok(d, group, topk, scale_mode, qgroup, topk_group)) return -1;
    if (coef_fmt != 0 && coef_fmt != 1) return -1;
    if (coef_fmt == 1 && !shared_coef) return -1;      /* u32[T,J]: the words of each token's segment */
    if (qgroup == 0) qgroup = group;
    const int J = d / group, Jq = d / qgroup;
    const int64_t rec = orc_record_bytes_full(d, group, bits, topk, scale_mode, qgroup, topk_group, coef_fmt);
    const int64_t sbytes = scale_bytes(d, qgroup, scale_mode);
    const int64_t cbytes = coef_fmt == 1 ? 0 : 4 * (int64_t)J;
    int err = 0;
    uint32_t st_word = 0;
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel num_threads(nthreads)
    {
        float *r = (float *)malloc(sizeof(float) * d);
        float *eh = (float *)malloc(sizeof(float) * d);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < T; t++) {
            const uint8_t *recp = payload + t * rec;
            const uint8_t *scales = recp + cbytes;
            const uint8_t *codes = scales + sbytes;
            const uint8_t *oidx = codes + ((int64_t)d * bits) / 8;
            const uint8_t *oval = oidx + 2 * topk;
            const uint8_t *goff = oval + 2 * topk;
            const uint8_t *gval = goff + goff_bytes((int64_t)Jq * topk_group, qgroup);
            int has_ref = resolve_ref(d, t, ref_base, ref_rows, ref_row, gain, bias, r);
            if (has_ref < 0) {
#pragma omp atomic write
                err = -2;
                continue;
            }
            const float *st = scale_mode == 0 ? step + (has_ref ? 0 : d) : NULL;
            for (int c = 0; c < d; c++) {
                int q = get_code(codes, c, bits);
                if (q == -(1 << (bits - 1))) {
#pragma omp atomic
                    st_word |= 2u;
                }
                float sc;
                if (scale_mode == 0) sc = st[c];
                else { uint16_t s16; memcpy(&s16, scales + 2 * (c / qgroup), 2); sc = orc_f16_to_f32(s16); }
                eh[c] = (float)q * sc;
            }
            for (int n = 0; n < topk; n++) {
                uint16_t ci, hv;
                memcpy(&ci, oidx + 2 * n, 2);
                memcpy(&hv, oval + 2 * n, 2);
                if (ci >= d) {
#pragma omp atomic write
                    err = -3;
                    continue;
                }
                eh[ci] = orc_f16_to_f32(hv);
            }
            for (int n = 0; n < Jq * topk_group; n++) {
                uint16_t hv;
                int o = goff_width(qgroup) == 1 ? goff[n] : (goff[2 * n] | (goff[2 * n + 1] << 8));
                memcpy(&hv, gval + 2 * n, 2);
                if (o >= qgroup) {
#pragma omp atomic write
                    err = -3;
                    continue;
                }
                eh[(n / topk_group) * qgroup + o] = orc_f16_to_f32(hv);
            }
            for (int j = 0; j < J; j++) {
                uint32_t w;
                if (coef_fmt == 1) w = shared_coef[t * J + j];
                else memcpy(&w, recp + 4 * j, 4);
                float a = orc_f16_to_f32((uint16_t)(w & 0xffff));
                float b = orc_f16_to_f32((uint16_t)(w >> 16));
                for (int c = j * group; c < (j + 1) * group; c++) {
                    float rt = fmaf(a, r[c], b);
                    float xh = rt + eh[c];
                    X_hat[t * (int64_t)d + c] = orc_f32_to_bf16(xh);
                }
            }
        }
        free(r); free(eh);
    }
    if (status) *status |= st_word;
    return err;
}

/* ------------------------------------------------------------------ */
/* step tables from a calibration draw                                 */
/* ------------------------------------------------------------------ */

/* For every channel: sigma = sqrt(mean over tokens of e^2), separately over
 * tokens with a reference (row 0) and direct tokens (row 1), e being the
 * binary32 residual of Eq. 7 with wire coefficients.  step = smallest
 * binary16 >= clip_sigmas*sigma/Qmax (held as float), inv_step = 1.0f/step in
 * binary32; a row without tokens, or a channel with sigma 0, gets step 0 and
 * inv_step 0.
 * shared_coef (u32[T,J] or NULL): with Eq. 6 solved over several fitting
 * positions every token uses the wire words of its segment; the residual is
 * then taken with those instead of the token's own fit. */
static int calibrate_impl(int d, int group, int bits,
                          const uint16_t *X, int64_t T,
                          const uint16_t *ref_base, int64_t ref_rows, const int32_t *ref_row,
                          const uint16_t *gain, const uint16_t *bias, const uint32_t *shared_coef,
                          double clip_sigmas, float *step, float *inv_step) {
    if (!cfg_ok(d, group, bits, 0)) return -1;
    const int J = d / group;
    const int qmax = (1 << (bits - 1)) - 1;
    double *acc = (double *)calloc((size_t)2 * d, sizeof(double));
    int64_t cnt[2] = {0, 0};
    float *h = (float *)malloc(sizeof(float) * d);
    float *r = (float *)malloc(sizeof(float) * d);
    int err = 0;
    for (int64_t t = 0; t < T && !err; t++) {
        for (int c = 0; c < d; c++) h[c] = orc_bf16_to_f32(X[t * (int64_t)d + c]);
        int has_ref = resolve_ref(d, t, ref_base, ref_rows, ref_row, gain, bias, r);
        if (has_ref < 0) { err = -2; break; }
        int row = has_ref ? 0 : 1;
        cnt[row]++;
        for (int j = 0; j < J; j++) {
            float a, b;
            if (shared_coef) {
                const uint32_t w = shared_coef[t * (int64_t)J + j];
                a = orc_f16_to_f32((uint16_t)(w & 0xffffu));
                b = orc_f16_to_f32((uint16_t)(w >> 16));
            } else {
                double as, bs;
                orc_fit_group(h + j * group, r + j * group, group, has_ref, &as, &bs, NULL, NULL);
                a = orc_f16_to_f32(orc_f64_to_f16(as));
                b = orc_f16_to_f32(orc_f64_to_f16(bs));
            }
            for (int c = j * group; c < (j + 1) * group; c++) {
                float rt = fmaf(a, r[c], b);
                float e = h[c] - rt;
                acc[row * d + c] += (double)e * (double)e;
            }
        }
    }
    for (int row = 0; row < 2 && !err; row++) {
        for (int c = 0; c < d; c++) {
            float s = 0.0f, is = 0.0f;
            if (cnt[row] > 0) {
                double sigma = sqrt(acc[row * d + c] / (double)cnt[row]);
                double want = clip_sigmas * sigma / (double)qmax;
                if (want > 0.0) {
                    s = orc_f16_to_f32(orc_f64_to_f16_up(want));
                    if (s != 0.0f) is = 1.0f / s;
                }
            }
            step[row * d + c] = s;
            inv_step[row * d + c] = is;
        }
    }
    free(acc); free(h); free(r);
    return err;
}

int orc_calibrate(int d, int group, int bits,
                  const uint16_t *X, int64_t T,
                  const uint16_t *ref_base, int64_t ref_rows, const int32_t *ref_row,
                  const uint16_t *gain, const uint16_t *bias,
                  double clip_sigmas, float *step, float *inv_step) {
    return calibrate_impl(d, group, bits, X, T, ref_base, ref_rows, ref_row, gain, bias, NULL, clip_sigmas, step, inv_step);
}

int orc_calibrate_shared(int d, int group, int bits,
                         const uint16_t *X, int64_t T,
                         const uint16_t *ref_base, int64_t ref_rows, const int32_t *ref_row,
                         const uint16_t *gain, const uint16_t *bias, const uint32_t *shared_coef,
                         double clip_sigmas, float *step, float *inv_step) {
    if (!shared_coef) return -1;
    return calibrate_impl(d, group, bits, X, T, ref_base, ref_rows, ref_row, gain, bias, shared_coef, clip_sigmas, step, inv_step);
}

/* ------------------------------------------------------------------ */
/* Sec. IV-B.1: exact-token span match                                 */
/* ------------------------------------------------------------------ */

static const int32_t *g_sort_tok;
static int g_sort_w;

static int cmp_window_pos(const void *pa, const void *pb) {
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    for (int m = 0; m < g_sort_w; m++) {
        int32_t x = g_sort_tok[a + m], y = g_sort_tok[b + m];
        if (x != y) return x < y ? -1 : 1;
    }
    return a < b ? -1 : (a > b ? 1 : 0);
}

/* compare the history window at position p with the query window at i */
static int cmp_hist_query(const int32_t *hist, int32_t p, const int32_t *query, int64_t i, int w) {
    for (int m = 0; m < w; m++) {
        int32_t x = hist[p + m], y = query[i + m];
        if (x != y) return x < y ? -1 : 1;
    }
    return 0;
}

/*
 * The history is the concatenation of n_req earlier requests: request r holds the
 * tokens [req_off[r], req_off[r+1]) (req_off[0] = 0, req_off[n_req] = n_hist;
 * req_off NULL = one request).  A candidate (r, j, L) lies inside ONE request: its
 * window and its extension stop at the request's end.  Recency is the position in
 * the concatenation (a later request is more recent; inside a request the later
 * start).
 *
 * ref_row  int32[n_query] out: history row of every covered query position, -1 otherwise;
 *          with `intra`, an uncovered position whose token occurred earlier in the
 *          query gets n_hist + (position of the FIRST occurrence of that token in the
 *          query): the "intra-sequence reference" of Sec. IV-B.1.  The first
 *          occurrence itself never gets one, so such references never chain.
 * spans    int32[3*cap]  out (q_start, h_start, len), cap >= n_query/w + 1; may be NULL
 * n_spans  out
 * max_hits K: only the K largest history starts of each distinct window are
 *          candidates; 0 = all of them.
 * first_live  a bounded history ("recent hits"): only windows that START at or after
 *          this history position are candidates; a match still extends forward as far
 *          as it goes.  0 = the whole history.
 * Not thread safe (qsort comparator state).
 */
int orc_match_spans_live(const int32_t *hist, int64_t n_hist, const int32_t *req_off, int32_t n_req,
                         const int32_t *query, int64_t n_query, int w, int max_hits, int intra, int64_t first_live,
                         int32_t *ref_row, int32_t *spans, int32_t *n_spans) {
    if (w < 1 || max_hits < 0 || first_live < 0) return -1;
    if (req_off) {
        if (n_req < 0 || req_off[0] != 0 || req_off[n_req] != n_hist) return -1;
        for (int32_t r = 0; r < n_req; r++) if (req_off[r] > req_off[r + 1]) return -1;
    }
    for (int64_t i = 0; i < n_query; i++) ref_row[i] = -1;
    *n_spans = 0;
    /* end of the request that holds each history position */
    int32_t *end_of = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_hist > 0 ? n_hist : 1));
    if (req_off) {
        for (int32_t r = 0; r < n_req; r++)
            for (int32_t j = req_off[r]; j < req_off[r + 1]; j++) end_of[j] = req_off[r + 1];
    } else {
        for (int64_t j = 0; j < n_hist; j++) end_of[j] = (int32_t)n_hist;
    }
    /* windows that lie inside one request, sorted by content then position */
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_hist > 0 ? n_hist : 1));
    int64_t nwin = 0;
    for (int64_t j = first_live; j + w <= n_hist; j++)
        if (j + w <= end_of[j]) order[nwin++] = (int32_t)j;
    g_sort_tok = hist; g_sort_w = w;
    qsort(order, (size_t)nwin, sizeof(int32_t), cmp_window_pos);

    int64_t i = 0;
    int32_t ns = 0;
    while (i < n_query && nwin > 0) {
        if (i + w > n_query) { i++; continue; }
        /* equal range of the query window in the sorted window list */
        int64_t lo = 0, hi = nwin;
        while (lo < hi) {
            int64_t mid = (lo + hi) / 2;
            if (cmp_hist_query(hist, order[mid], query, i, w) < 0) lo = mid + 1; else hi = mid;
        }
        int64_t first = lo;
        hi = nwin;
        while (lo < hi) {
            int64_t mid = (lo + hi) / 2;
            if (cmp_hist_query(hist, order[mid], query, i, w) <= 0) lo = mid + 1; else hi = mid;
        }
        int64_t last = lo;              /* [first,last): ascending history position */
        if (first == last) { i++; continue; }
        int64_t from = first;
        if (max_hits > 0 && last - first > max_hits) from = last - max_hits;
        int64_t bestL = -1; int32_t bestj = -1;
        for (int64_t k = from; k < last; k++) {
            int32_t j = order[k];
            int64_t L = w;
            while (i + L < n_query && j + L < end_of[j] && query[i + L] == hist[j + L]) L++;
            if (L > bestL || (L == bestL && j > bestj)) { bestL = L; bestj = j; }
        }
        if (spans) { spans[3 * ns] = (int32_t)i; spans[3 * ns + 1] = bestj; spans[3 * ns + 2] = (int32_t)bestL; }
        ns++;
        for (int64_t m = 0; m < bestL; m++) ref_row[i + m] = bestj + (int32_t)m;
        i += bestL;
    }
    *n_spans = ns;
    if (intra) {
        /* plain quadratic scan: the first occurrence of every uncovered position's token */
        for (int64_t q = 0; q < n_query; q++) {
            if (ref_row[q] >= 0) continue;
            for (int64_t f = 0; f < q; f++) {
                if (query[f] == query[q]) { ref_row[q] = (int32_t)(n_hist + f); break; }
            }
        }
    }
    free(order); free(end_of);
    return 0;
}

int orc_match_spans_req(const int32_t *hist, int64_t n_hist, const int32_t *req_off, int32_t n_req,
                        const int32_t *query, int64_t n_query, int w, int max_hits, int intra,
                        int32_t *ref_row, int32_t *spans, int32_t *n_spans) {
    return orc_match_spans_live(hist, n_hist, req_off, n_req, query, n_query, w, max_hits, intra, 0, ref_row, spans, n_spans);
}

int orc_match_spans(const int32_t *hist, int64_t n_hist, const int32_t *query, int64_t n_query,
                    int w, int max_hits, int32_t *ref_row, int32_t *spans, int32_t *n_spans) {
    return orc_match_spans_req(hist, n_hist, NULL, 1, query, n_query, w, max_hits, 0, ref_row, spans, n_spans);
}

int orc_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
