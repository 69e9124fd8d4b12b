// RAC codec kernels for sm_100a: encode (Sec. IV-C, Eq. 6-8 + packing, outlier split), reconstruct (Eq. 9),
// and the residual-RMS pass behind the step tables.
//
// Shape of the streaming kernels: persistent CTAs, one token per CTA iteration, one thread per 32
// consecutive channels.  Rows travel between HBM and shared memory only as 1-D bulk copies (TMA without a
// tensor map): a ring of stages is filled ahead and signalled through mbarriers, finished records and rows
// leave through bulk stores.  Every wait on an mbarrier is bounded; a copy that never lands ends the kernel
// with a status bit instead of a hang.  The arithmetic that decides integers (residual, scaling, rounding)
// is binary32 with one rounding per operation, written with explicit intrinsics / PTX so the compiler
// cannot contract or reorder it.
//
// Shared-memory reads of a thread's 64-byte slab go through a per-lane rotation of the four 16-byte
// pieces (piece (j + lane/2) mod 4 in step j), which makes the 128-bit accesses bank-conflict free
// on a plain linear row.
//
// Kernels: encode_ws_kernel (streaming pass of encode, optionally also the sender-side x_hat),
// outlier_kernel (second launch of encode: the k largest |e| per token), decode_kernel and decode_ws_kernel
// (receiver and sender reconstruction, with and without per-token outliers), calib_kernel +
// calib_finalize_kernel (step tables; in its second form the statistics pass of the segment fit),
// segment_fit_kernel + seg_of_kernel (Eq. 6 over several fitting positions), split_waves_kernel (tokens that
// reference the same prompt go second), recon_error_kernel (error of a sender-path run).  The kernels of the
// per-group-scale quantiser (Eq. 8 as printed) live in rac_codec_dyn.cu; this file holds the C ABI of both.
#include <cstring>

#include "rac_codec_dev.cuh"

namespace rac {

// ------------------------------------------------------------------------------------------------
// geometry / validation (host)
// ------------------------------------------------------------------------------------------------
static bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

int make_geometry(const rac_codec_cfg *cfg, Geometry *g) {
    if (!cfg) return RAC_EINVAL;
    if (cfg->d <= 0 || cfg->group <= 0 || cfg->topk < 0 || cfg->bits <= 0) return RAC_EINVAL;
    if (cfg->qgroup < 0 || cfg->topk_group < 0) return RAC_EINVAL;
    if ((cfg->coef_fmt != 0 && cfg->coef_fmt != 1) || cfg->flags != 0) return RAC_EUNSUPPORTED;
    if (cfg->scale_mode != 0 && cfg->scale_mode != 1) return RAC_EUNSUPPORTED;
    if (cfg->d % cfg->group) return RAC_EINVAL;
    if (cfg->d % 32 || cfg->d > 8192) return RAC_EUNSUPPORTED;
    if (!is_pow2(cfg->group) || cfg->group < 32 || cfg->group > 1024) return RAC_EUNSUPPORTED;
    if (cfg->topk > 16 || cfg->topk > cfg->d) return RAC_EUNSUPPORTED;
    int qgroup = cfg->qgroup ? cfg->qgroup : cfg->group;
    int lpq = 0, qgen = 0;
    if (cfg->scale_mode == 0) {
        // the static table: one grouping, per-token outliers, 2..4 bits
        if (qgroup != cfg->group || cfg->topk_group != 0) return RAC_EUNSUPPORTED;
        if (cfg->bits < 2 || cfg->bits > 4) return RAC_EUNSUPPORTED;
        lpq = cfg->group / 32;
    } else {
        // Eq. 8 takes the scale from the dense values, i.e. after the outliers are known.  The per-token
        // selection runs as a second launch, after the codes exist, so this mode offers the paper's own
        // per-group outliers (picked inside the streaming pass) and not the per-token ones.
        if (cfg->topk != 0) return RAC_EUNSUPPORTED;
        if (cfg->bits != 2 && cfg->bits != 3 && cfg->bits != 4 && cfg->bits != 8) return RAC_EUNSUPPORTED;
        if (cfg->d % qgroup) return RAC_EINVAL;
        if (is_pow2(qgroup) && qgroup >= 32 && qgroup <= 1024) lpq = qgroup / 32;
        else if (qgroup == cfg->d) lpq = 0;   // one scale per token, exchanged through shared memory
        else if (qgroup % 32 == 0) { lpq = 0; qgen = qgroup / 32; }   // any other whole number of lanes: the same exchange
        else return RAC_EUNSUPPORTED;
        if (cfg->topk_group > 8) return RAC_EUNSUPPORTED;
        if (cfg->topk_group > 0 && lpq == 0) return RAC_EUNSUPPORTED;   // a group must lie within one warp
    }
    g->d = cfg->d;
    g->group = cfg->group;
    g->bits = cfg->bits;
    g->topk = cfg->topk;
    g->J = cfg->d / cfg->group;
    g->lpg = cfg->group / 32;
    g->nthreads = ((cfg->d / 32) + 31) / 32 * 32;
    g->code_bytes = cfg->d * cfg->bits / 8;
    g->scale_mode = cfg->scale_mode;
    g->qgroup = qgroup;
    g->Jq = cfg->d / qgroup;
    g->lpq = lpq;
    g->qgen = qgen;
    g->topk_group = cfg->topk_group;
    g->coef_fmt = cfg->coef_fmt;
    g->scale_off = cfg->coef_fmt == 1 ? 0 : 4 * g->J;
    g->codes_off = g->scale_off + (cfg->scale_mode == 1 ? (2 * g->Jq + 3) / 4 * 4 : 0);
    const int ng = g->Jq * g->topk_group;
    g->goff_off = g->codes_off + g->code_bytes + 4 * cfg->topk;
    g->gval_off = g->goff_off + (ng * (qgroup > 256 ? 2 : 1) + 1) / 2 * 2;   // one-byte offsets up to 256 channels, two beyond
    const int raw = g->gval_off + 2 * ng;
    g->rec = (raw + 15) / 16 * 16;
    return RAC_OK;
}

// ------------------------------------------------------------------------------------------------
// calibration pass: per-channel sums of e^2 (the residual of Eq. 7 with wire coefficients)
// ------------------------------------------------------------------------------------------------
// Same front end as the encoder (slab loads, Eq. 6 statistics, wire coefficients); instead of codes, every
// thread accumulates e^2 of its own 32 channels in shared memory, separately for tokens with a reference
// (row 0) and tokens coded directly (row 1).  One CTA barrier per token; the grid is fixed.
// MOMENTS: the first pass of the segment fit instead -- the centred statistics of Eq. 6 of every (token, group)
// go to p.moments and nothing is accumulated.
template <bool MOMENTS>
__global__ void __launch_bounds__(256, 2) calib_kernel(const CodecParams p) {
    constexpr bool SUB = false;  // always over all tokens
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31;
    const int rot = (lane >> 1) & 3;
    const int d = p.d;
    const bool valid = tid * 32 < d;
    const EncSmem L = enc_smem_layout(d, p.stages, nt);
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem);
    const uint32_t sbase = smem_u32(smem);
    const int S = p.stages;
    const uint32_t row_bytes = 2u * (uint32_t)d;

    if (tid == 0) {
        for (int s = 0; s < S; s++) mbar_init(smem_u32(&ctrl->bar[s]), 1);
        mbar_init_fence();
    }
    for (int o = tid; o < 2 * nt * 32; o += nt) reinterpret_cast<float *>(smem + L.acc0)[o] = 0.f;
    __syncthreads();

    const int first = blockIdx.x, stride = gridDim.x;
    const long long n_tok = tokens_to_do<SUB>(p);
    const int n_my = (n_tok > first) ? (int)((n_tok - first + stride - 1) / stride) : 0;
    int next_raw = 0;
    auto raw_row_of = [&](int k) -> int {  // raw ref_row entry of this CTA's k-th token
        long long t = token_at<SUB>(p, first + (long long)k * stride);
        return p.ref_row ? p.ref_row[t] : (int)t;
    };
    if (tid == 0) {
        for (int k = 0; k < S - 1 && k < n_my; k++) {
            long long t = token_at<SUB>(p, first + (long long)k * stride);
            ctrl->tok[k] = t;
            issue_token_loads<SUB>(p, ctrl, sbase + L.stage0 + k * L.stage_bytes, row_bytes, k, resolve_row<SUB>(p, raw_row_of(k)),
                              p.X + t * d, row_bytes);
        }
        if (S - 1 < n_my) next_raw = raw_row_of(S - 1);
    }
    int cnt_ref = 0, cnt_dir = 0;  // tokens per table row (thread 0 only)
    uint32_t off[4];
#pragma unroll
    for (int j = 0; j < 4; j++) off[j] = (uint32_t)(tid * 64 + ((j + rot) & 3) * 16);
    const unsigned int group_mask = __ballot_sync(0xffffffffu, valid);

    int stage = 0, issue_stage = S - 1;
    bool aborted = false;
    uint32_t parity = 0;
    for (int it = 0; it < n_my; it++) {
        if (tid == 0 && it + S - 1 < n_my) {
            const int k = it + S - 1;
            const long long tk = token_at<SUB>(p, first + (long long)k * stride);
            ctrl->tok[issue_stage] = tk;
            issue_token_loads<SUB>(p, ctrl, sbase + L.stage0 + issue_stage * L.stage_bytes, row_bytes, issue_stage,
                              resolve_row<SUB>(p, next_raw), p.X + tk * d, row_bytes);
            if (k + 1 < n_my) next_raw = raw_row_of(k + 1);
        }
        const bool timed_out = !mbar_wait_bounded(smem_u32(&ctrl->bar[stage]), parity);
        if (timed_out && p.status) atomicOr(p.status, RAC_STATUS_TIMEOUT);
        const bool has_ref = ctrl->row[stage] >= 0;
        const long long tok = ctrl->tok[stage];
        const uint32_t xs = sbase + L.stage0 + stage * L.stage_bytes;
        const uint32_t rs = xs + row_bytes;

        if (valid) {
            u64 x2[16], r2[16];
#pragma unroll
            for (int j = 0; j < 4; j++) {
                uint4 w = lds128(xs + off[j]);
                x2[4 * j + 0] = bf16x2_to_p(w.x);
                x2[4 * j + 1] = bf16x2_to_p(w.y);
                x2[4 * j + 2] = bf16x2_to_p(w.z);
                x2[4 * j + 3] = bf16x2_to_p(w.w);
            }
            if (has_ref) {
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    u64 rr[4];
                    load_ref_slot(rs + off[j], p.gain, p.bias, (int)(off[j] >> 1), rr);
#pragma unroll
                    for (int i = 0; i < 4; i++) r2[4 * j + i] = rr[i];
                }
            } else {
#pragma unroll
                for (int i = 0; i < 16; i++) r2[i] = 0ull;
            }
            u64 a2, b2;
            float4 st;
            if (!MOMENTS && p.coef_ext) {
                // shared coefficients: the residual of Eq. 7 with the words of the token's segment
                const uint32_t cw = p.coef_ext[(long long)p.seg_of[tok] * p.J + (tid >> p.lpg_shift)];
                const float a = half_bits_to_float(cw & 0xffffu), b = half_bits_to_float(cw >> 16);
                a2 = pack2(a, a);
                b2 = pack2(b, b);
            } else {
                fit_group(x2, r2, has_ref, p.lpg, p.inv_group, group_mask, p.status, a2, b2, nullptr, &st);
            }
            if (MOMENTS) {
                if (!timed_out && (lane & (p.lpg - 1)) == 0) p.moments[tok * p.J + (tid >> p.lpg_shift)] = st;
            }
            float4 *acc = reinterpret_cast<float4 *>(smem + L.acc0) + (has_ref ? 0 : 8 * nt);
#pragma unroll
            for (int j = 0; j < 4; j++) {
                if (MOMENTS) break;
                const int q = (j + rot) & 3;
#pragma unroll
                for (int hh = 0; hh < 2; hh++) {
                    float e0, e1, e2, e3;
                    unpack2(psub(x2[4 * j + 2 * hh], pfma(a2, r2[4 * j + 2 * hh], b2)), e0, e1);
                    unpack2(psub(x2[4 * j + 2 * hh + 1], pfma(a2, r2[4 * j + 2 * hh + 1], b2)), e2, e3);
                    float4 v = acc[(2 * q + hh) * nt + tid];
                    v.x = __fmaf_rn(e0, e0, v.x);
                    v.y = __fmaf_rn(e1, e1, v.y);
                    v.z = __fmaf_rn(e2, e2, v.z);
                    v.w = __fmaf_rn(e3, e3, v.w);
                    acc[(2 * q + hh) * nt + tid] = v;
                }
            }
        }
        if (tid == 0) { if (has_ref) cnt_ref++; else cnt_dir++; }
        if (__syncthreads_or(timed_out)) { aborted = true; break; }  // one vote: every thread leaves together
        if (++stage == S) { stage = 0; parity ^= 1u; }
        if (++issue_stage == S) issue_stage = 0;
    }

    __syncthreads();
    if (MOMENTS) {
        if (tid == 0 && aborted) {
            for (int s = 0; s < S; s++) {
                mbar_wait_bounded(smem_u32(&ctrl->bar[s]), 0);
                mbar_wait_bounded(smem_u32(&ctrl->bar[s]), 1);
            }
        }
        return;
    }
    // partial sums of this CTA, channel order, then its token counts
    float *out = p.calib_partial + (long long)blockIdx.x * 2 * d;
    const float *acc = reinterpret_cast<const float *>(smem + L.acc0);
    if (valid) {
        for (int rrow = 0; rrow < 2; rrow++)
            for (int f = 0; f < 8; f++)
                for (int cc = 0; cc < 4; cc++)
                    out[rrow * d + tid * 32 + f * 4 + cc] = acc[rrow * nt * 32 + ((f * nt) + tid) * 4 + cc];
    }
    if (tid == 0) {
        int *cnt = reinterpret_cast<int *>(p.calib_partial + (long long)gridDim.x * 2 * d) + 2 * blockIdx.x;
        cnt[0] = cnt_ref;
        cnt[1] = cnt_dir;
        if (aborted) {
            // give copies that may still be in flight a bounded chance to land before the CTA retires
            for (int s = 0; s < S; s++) {
                mbar_wait_bounded(smem_u32(&ctrl->bar[s]), 0);
                mbar_wait_bounded(smem_u32(&ctrl->bar[s]), 1);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// encode
// ------------------------------------------------------------------------------------------------
// Two launches.  (1) The streaming pass (this kernel): statistics, coefficients, residual, codes; every
// warp of the CTA works on its 1024 channels of the token and ends with ONE arrival on the stage's `done`
// mbarrier -- there is no CTA barrier in the loop.  Handing the finished record to the copy engine and
// refilling the stage is the duty of warp (i mod warps) for token i; the other warps are already in the
// next token and only ever wait for data (`full`).  With outliers, every thread also writes the largest
// |e| of its 32 channels to the caller's workspace.  (2) outlier_kernel picks the k largest |e| per token
// from those maxima with one warp per token -- thousands of tokens in flight, so the serial selection
// (threshold, candidates, ranking) costs latency nobody waits for -- and patches the records in place.
struct WsCtrl {
    unsigned long long full[kMaxStages];
    unsigned long long done[kMaxStages];
    int row[kMaxStages];
    int seg[kMaxStages];   // segment of the token in each stage (shared coefficients only)
    int abort;
};

struct WsSmem {
    int stage0, stage_bytes, rec_off, tm_off, tm_bytes, total;
};
__host__ __device__ inline WsSmem ws_smem_layout(int d, int rec, int stages, bool topk) {
    WsSmem s;
    s.stage0 = align_up((int)sizeof(WsCtrl), 128);
    s.rec_off = 4 * d;  // after X row + R row: two record slots, used alternately (by the stage's parity)
    s.tm_off = s.rec_off + 2 * rec;  // two slots of per-slab maxima (outliers only), same alternation
    s.tm_bytes = topk ? align_up((d / 32) * 4, 16) : 0;
    s.stage_bytes = align_up(s.tm_off + 2 * s.tm_bytes, 128);
    s.total = s.stage0 + stages * s.stage_bytes;
    return s;
}

// SUB: the token-list / second-reference-buffer form (see rac_codec_dev.cuh).
// LPG: lanes per alignment group as a compile-time constant (4 = groups of 128 channels, 2 = groups of 64), or 0 to
// read it from the parameters; the constant removes the uniform branches of the shuffle reductions.
// D: the hidden width as a compile-time constant (4096 and 5120 are compiled in), or 0 to read it from the parameters;
// the constant folds the address arithmetic of the rows and stages (downlink call at 131072 x 5120: 0.671 -> 0.658 ms).
// REF: every token has a reference row (identity rows: no row list, a reference buffer): the per-token test and the
// second row of the tables go away (downlink call 0.649 -> 0.634 ms).
template <int BITS, bool TOPK, bool XHAT, int MINB, bool SUB, int LPG = 0, int D = 0, bool REF = false>
__global__ void __launch_bounds__(MINB == 4 ? 160 : 256, MINB) encode_ws_kernel(const CodecParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nwarps = D ? (D / 32 + 31) / 32 : nt >> 5;
    const int rot = (lane >> 1) & 3;
    const int d = D ? D : p.d;
    const bool valid = tid * 32 < d;
    constexpr int S = 2;   // stages of the ring (the host sets p.stages to the same)
    // with the width and the group compiled in, the record geometry is a constant too (those variants are launched for
    // no outliers or eight per token only)
    constexpr bool kGeo = D != 0 && LPG != 0;
    const int Jc = kGeo ? D / (32 * (LPG ? LPG : 1)) : p.J;
    const int codeb = kGeo ? D * BITS / 8 : p.code_bytes;
    const int recb = kGeo ? (4 * (D / (32 * (LPG ? LPG : 1))) + D * BITS / 8 + (TOPK ? 32 : 0) + 15) / 16 * 16 : p.rec;
    const WsSmem L = ws_smem_layout(d, recb, S, TOPK);
    WsCtrl *ctrl = reinterpret_cast<WsCtrl *>(smem);
    const uint32_t sbase = smem_u32(smem);
    constexpr float qmax = (float)((1 << (BITS - 1)) - 1);
    const uint32_t row_bytes = 2u * (uint32_t)d;

    const int first = blockIdx.x, stride = gridDim.x;
    const long long n_tok = tokens_to_do<SUB>(p);
    const int n_my = (n_tok > first) ? (int)((n_tok - first + stride - 1) / stride) : 0;
    auto raw_row_of = [&](int k) -> int {  // raw ref_row entry of this CTA's k-th token
        long long t = token_at<SUB>(p, first + (long long)k * stride);
        return p.ref_row ? p.ref_row[t] : (int)t;
    };
    // one lane: start the copies of this CTA's k-th token into stage s
    auto issue = [&](int k, int s, int raw_row) {
        const long long t = token_at<SUB>(p, first + (long long)k * stride);
        const int row = resolve_row<SUB>(p, raw_row);
        ctrl->row[s] = row;
        if constexpr (SUB) ctrl->seg[s] = p.seg_of ? p.seg_of[t] : 0;
        const uint32_t bar = smem_u32(&ctrl->full[s]);
        const uint32_t base = sbase + L.stage0 + s * L.stage_bytes;
        mbar_arrive_expect_tx(bar, p.test_extra_tx + row_bytes + (row >= 0 ? row_bytes : 0u));
        bulk_load(base, p.X + t * d, row_bytes, bar);
        if (row >= 0) bulk_load(base + row_bytes, ref_row_ptr<SUB>(p, row), row_bytes, bar);
    };

    if (tid == 0) {
        for (int s = 0; s < S; s++) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->done[s]), nwarps);
        }
        ctrl->abort = 0;
        mbar_init_fence();
    }
    // shared coefficients (one pair per segment and group, Eq. 6 over several positions) come from outside the
    // records: no coefficient words in front of the codes
    bool shared = false;
    if constexpr (SUB) shared = p.coef_ext != nullptr;
    const int coff = shared ? 0 : 4 * Jc;
    {
        // padding words of the records are written once and never touched again
        const int raw = coff + codeb + 4 * p.topk;
        for (int s = 0; s < 2 * S; s++)
            for (int o = raw + 4 * tid; o < recb; o += 4 * nt)
                *reinterpret_cast<uint32_t *>(smem + L.stage0 + (s >> 1) * L.stage_bytes + L.rec_off + (s & 1) * recb + o) = 0u;
    }
    __syncthreads();
    if (tid == 0)
        for (int k = 0; k < S && k < n_my; k++) issue(k, k, raw_row_of(k));

    uint32_t off[4];
#pragma unroll
    for (int j = 0; j < 4; j++) off[j] = (uint32_t)(tid * 64 + ((j + rot) & 3) * 16);
    const unsigned int group_mask = __ballot_sync(0xffffffffu, valid);
    const u64 magic2 = pack2(kMagic, kMagic);

    int stage = 0, duty = 0;  // duty: the warp whose turn the tail of this token is
    uint32_t parity = 0;
    bool timed_out = false;
    for (int it = 0; it < n_my; it++) {
        if (*reinterpret_cast<volatile int *>(&ctrl->abort)) break;
        unsigned char *stg = smem + L.stage0 + stage * L.stage_bytes;
        const uint32_t xs = sbase + L.stage0 + stage * L.stage_bytes;
        const uint32_t rs = xs + row_bytes;
        unsigned char *rec = stg + L.rec_off + parity * recb;
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_u32(&ctrl->full[stage]), parity))) { timed_out = true; break; }
        const bool has_ref = REF ? true : ctrl->row[stage] >= 0;

        if (valid) {
            // ---- (1) the slab: 4 slots of 8 channels, slot j holds piece (j + rot) & 3
            u64 x2[16], r2[16];
#pragma unroll
            for (int j = 0; j < 4; j++) {
                uint4 w = lds128(xs + off[j]);
                x2[4 * j + 0] = bf16x2_to_p(w.x);
                x2[4 * j + 1] = bf16x2_to_p(w.y);
                x2[4 * j + 2] = bf16x2_to_p(w.z);
                x2[4 * j + 3] = bf16x2_to_p(w.w);
            }
            if (has_ref) {
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    u64 rr[4];
                    load_ref_slot(rs + off[j], p.gain, p.bias, (int)(off[j] >> 1), rr);
#pragma unroll
                    for (int i = 0; i < 4; i++) r2[4 * j + i] = rr[i];
                }
            } else {
#pragma unroll
                for (int i = 0; i < 16; i++) r2[i] = 0ull;
            }
            // ---- (2) Eq. 6 and wire rounding
            u64 a2, b2;
            constexpr int kShift = LPG == 4 ? 2 : 1;
            const int lpg = LPG ? LPG : p.lpg, lpg_shift = LPG ? kShift : p.lpg_shift;
            if (shared) {
                const uint32_t cw = p.coef_ext[(long long)ctrl->seg[stage] * Jc + (tid >> lpg_shift)];
                const float a = half_bits_to_float(cw & 0xffffu), b = half_bits_to_float(cw >> 16);
                a2 = pack2(a, a);
                b2 = pack2(b, b);
            } else {
                uint32_t coef_word;
                fit_group(x2, r2, has_ref, lpg, p.inv_group, group_mask, p.status, a2, b2, &coef_word);
                if ((lane & (lpg - 1)) == 0) reinterpret_cast<uint32_t *>(rec)[tid >> lpg_shift] = coef_word;
            }

            // ---- (3) Eq. 7 residual, Eq. 8 quantisation with the static table, packing
            const float *inv_tab = p.inv_step + (has_ref ? 0 : d);
            const float *step_tab = p.step + (has_ref ? 0 : d);
            uint32_t words[4];
            float tmax = 0.f;
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const int c = (int)(off[j] >> 1);
                const float4 iv0 = __ldg(reinterpret_cast<const float4 *>(inv_tab + c));
                const float4 iv1 = __ldg(reinterpret_cast<const float4 *>(inv_tab + c + 4));
                const u64 inv2[4] = {pack2(iv0.x, iv0.y), pack2(iv0.z, iv0.w), pack2(iv1.x, iv1.y), pack2(iv1.z, iv1.w)};
                u64 st2[4] = {0ull, 0ull, 0ull, 0ull};
                if (XHAT) {
                    const float4 s0 = __ldg(reinterpret_cast<const float4 *>(step_tab + c));
                    const float4 s1 = __ldg(reinterpret_cast<const float4 *>(step_tab + c + 4));
                    st2[0] = pack2(s0.x, s0.y); st2[1] = pack2(s0.z, s0.w); st2[2] = pack2(s1.x, s1.y); st2[3] = pack2(s1.z, s1.w);
                }
                float ev[8];
                uint32_t xh[4];
                uint32_t w = 0;
                if (BITS == 3) {
                    uint32_t bits8[8];
#pragma unroll
                    for (int i = 0; i < 4; i++) {
                        const u64 rt = pfma(a2, r2[4 * j + i], b2);
                        const u64 e = psub(x2[4 * j + i], rt);
                        float v0, v1, t0, t1;
                        unpack2(pmul(e, inv2[i]), v0, v1);
                        t0 = fminf(fmaxf(v0, -qmax), qmax);
                        t1 = fminf(fmaxf(v1, -qmax), qmax);
                        const u64 tt = padd(pack2(t0, t1), magic2);
                        unpack2(tt, t0, t1);
                        bits8[2 * i] = __float_as_uint(t0);
                        bits8[2 * i + 1] = __float_as_uint(t1);
                        unpack2(e, ev[2 * i], ev[2 * i + 1]);
                        if (XHAT) {
                            // Eq. 9 with the code just chosen: x_hat = bf16(fma(q, step, alpha*r + beta)); a binary16-valued
                            // step makes q*step exact, so the fused form and (alpha*r + beta) + q*step are the same bits
                            float x0, x1;
                            unpack2(pfma(psub(tt, magic2), st2[i], rt), x0, x1);
                            xh[i] = f2_to_bf16x2(x0, x1);
                        }
                    }
                    w = pack8<BITS>(bits8);
                } else {
                    // 4- and 2-bit codes: clamp from below in binary32, round by the magic add, take the integer
                    // out of the mantissa and let the saturating pack clamp from above (its range is
                    // [-2^(BITS-1), 2^(BITS-1)-1], whose upper end is Qmax)
#pragma unroll
                    for (int i = 3; i >= 0; i--) {
                        const u64 rt = pfma(a2, r2[4 * j + i], b2);
                        const u64 e = psub(x2[4 * j + i], rt);
                        float v0, v1, t0, t1;
                        unpack2(pmul(e, inv2[i]), v0, v1);
                        v0 = fmaxf(v0, -qmax);
                        v1 = fmaxf(v1, -qmax);
                        if (XHAT) { v0 = fminf(v0, qmax); v1 = fminf(v1, qmax); }  // the float is used again below
                        const u64 tt = padd(pack2(v0, v1), magic2);
                        unpack2(tt, t0, t1);
                        w = sat_pack2<BITS>((int)__float_as_uint(t1) - 0x4b400000, (int)__float_as_uint(t0) - 0x4b400000, w);
                        unpack2(e, ev[2 * i], ev[2 * i + 1]);
                        if (XHAT) {
                            float x0, x1;
                            unpack2(pfma(psub(tt, magic2), st2[i], rt), x0, x1);
                            xh[i] = f2_to_bf16x2(x0, x1);
                        }
                    }
                }
                words[j] = w;
                // sender-side reconstruction: the thread's own slab of the X row now carries x_hat
                if (XHAT) sts128(xs + off[j], make_uint4(xh[0], xh[1], xh[2], xh[3]));
                if (TOPK) {
                    const float m0 = fmaxf(fmaxf(fabsf(ev[0]), fabsf(ev[1])), fmaxf(fabsf(ev[2]), fabsf(ev[3])));
                    const float m1 = fmaxf(fmaxf(fabsf(ev[4]), fabsf(ev[5])), fmaxf(fabsf(ev[6]), fabsf(ev[7])));
                    tmax = fmaxf(tmax, fmaxf(m0, m1));
                }
            }
            rot_right4(words, rot);  // words[q] is now the code word of piece q
            uint32_t *cw = reinterpret_cast<uint32_t *>(rec + coff) + tid * BITS;
            if (BITS == 4) {
                cw[0] = words[0]; cw[1] = words[1]; cw[2] = words[2]; cw[3] = words[3];
            } else if (BITS == 3) {
                cw[0] = words[0] | (words[1] << 24);
                cw[1] = (words[1] >> 8) | (words[2] << 16);
                cw[2] = (words[2] >> 16) | (words[3] << 8);
            } else {
                cw[0] = words[0] | (words[1] << 16);
                cw[1] = words[2] | (words[3] << 16);
            }
            // (4) the largest |e| of this thread's 32 channels, for the outlier pass
            if (TOPK) reinterpret_cast<float *>(stg + L.tm_off + parity * L.tm_bytes)[tid] = tmax;
        }
        // this warp's share of the token is in shared memory: one arrival per warp
        fence_async_smem();  // the record (and x_hat) bytes written above will be read by the copy engine
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&ctrl->done[stage])) : "memory");

        if (warp == duty) {
            // ---- this warp's turn: hand the record over and refill the stage; the others have moved on
            const int k_next = it + S;
            int raw_next = 0;
            if (lane == 0 && k_next < n_my) raw_next = raw_row_of(k_next);  // in flight while the tail runs
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_u32(&ctrl->done[stage]), parity))) { timed_out = true; break; }
            // ---- refill the stage, then hand the record to the copy engine.  The record sits in the slot of the
            // stage's current parity; the stage's next token writes the other slot, and the one after that
            // cannot start before this warp has arrived for the token in between, which it does only after the
            // wait below.  So the refill need not wait for the record to leave.  (With x_hat the X row itself
            // is the source of a store and must have been read before new data may land on it.)
            if (lane == 0) {
                const long long t = token_at<SUB>(p, first + (long long)it * stride);
                if (TOPK)  // the slab maxima travel like the record: one bulk copy from this parity's slot
                    bulk_store(p.tmax + t * (L.tm_bytes >> 2), xs + L.tm_off + parity * L.tm_bytes, (uint32_t)L.tm_bytes);
                if (XHAT) {
                    bulk_store(p.payload + t * recb, smem_u32(rec), (uint32_t)recb);
                    bulk_store(p.X_hat + t * d, xs, row_bytes);
                    bulk_commit();
                    bulk_wait_read<0>();
                    if (k_next < n_my) issue(k_next, stage, raw_next);
                } else {
                    if (k_next < n_my) issue(k_next, stage, raw_next);
                    bulk_store(p.payload + t * recb, smem_u32(rec), (uint32_t)recb);
                    bulk_commit();
                    bulk_wait_read<0>();
                }
            }
            __syncwarp();
        }
        if (++stage == S) { stage = 0; parity ^= 1u; }
        if (++duty == nwarps) duty = 0;
    }
    if (timed_out) {
        ctrl->abort = 1;
        if (p.status) atomicOr(p.status, RAC_STATUS_TIMEOUT);
    }
    __syncthreads();
    if (lane == 0) bulk_wait_all();  // every lane that stored records waits for its own copies
    if (tid == 0 && *reinterpret_cast<volatile int *>(&ctrl->abort)) {
        // give copies that may still be in flight a bounded chance to land before the CTA retires
        for (int s = 0; s < S; s++) {
            mbar_wait_bounded(smem_u32(&ctrl->full[s]), 0);
            mbar_wait_bounded(smem_u32(&ctrl->full[s]), 1);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// encode, second launch: outlier split (the k largest |e| per token, ties to the lower channel)
// ------------------------------------------------------------------------------------------------
// One warp per token.  Input: the per-thread maxima the streaming pass left in the workspace (one value per
// 32-channel slab); lane l holds the NV consecutive slabs NV*l .. NV*l+NV-1, so lane order is channel order.
// (a) Threshold tau: every lane offers its two largest maxima (two different slabs); k-1 rounds of a warp-wide
// maximum over the heads, the lowest lane that holds it moving on to its second value, then one more maximum.
// The k values seen are maxima of k different slabs, so at least k elements reach tau, and an element that
// reaches it can only sit in a slab whose maximum does.  tau is the exact k-th largest slab maximum unless one
// lane holds three of the k largest, and then only lower: a few more slabs are looked at, the result is the same.
// (b) The slabs that reach tau -- k of them unless maxima tie -- are listed in slab order and their residuals
// recomputed from X, the reference row and the wire coefficients in the record, four lanes per slab, eight
// channels per lane, with the same binary32 operations as the streaming pass (so the same bits).  Elements at or
// above tau are candidates, collected in channel order, one per lane.  (c) While there are more than k, the
// smallest goes (smallest magnitude; among equals the highest channel): the survivors are the k largest with
// ties to the lower channel, still in channel order.  More than 32 candidates (many equal magnitudes, e.g. an
// all-zero residual): k rounds of a maximum over the whole token instead.  (d) The winners go into the record's
// outlier fields in channel order, their dense codes are cleared (E^d = E - O), and with the sender-side
// reconstruction those channels of x_hat are replaced.
constexpr int kOutCap = 32;        // candidates per token: one per lane

// eight values by a run-time index, as a select tree (no local-memory array)
__device__ __forceinline__ float pick8(const float (&v)[8], int i) {
    const float a0 = (i & 1) ? v[1] : v[0], a1 = (i & 1) ? v[3] : v[2], a2 = (i & 1) ? v[5] : v[4], a3 = (i & 1) ? v[7] : v[6];
    const float b0 = (i & 2) ? a1 : a0, b1 = (i & 2) ? a3 : a2;
    return (i & 4) ? b1 : b0;
}

// whole-token path: k rounds of a maximum over all d channels (rare).  Lane r returns the r-th winner:
// channel, residual, aligned reference.
__device__ __noinline__ void select_whole_token(int d, int k, int coef_shift, const uint16_t *xrow, const uint16_t *rrow,
                                                const uint16_t *gain, const uint16_t *bias, const uint32_t *coef,
                                                int lane, int *c_out, float *e_out, float *rt_out) {
    unsigned long long prev = ~0ull, mine = 0ull;
    float minee = 0.f, minert = 0.f;
    for (int r = 0; r < k; r++) {
        unsigned long long best = 0ull;
        float beste = 0.f, bestrt = 0.f;
        for (int c = lane; c < d; c += 32) {
            const float h = __uint_as_float((uint32_t)xrow[c] << 16);
            float rr = 0.f;
            if (rrow) {
                rr = __uint_as_float((uint32_t)rrow[c] << 16);
                if (gain) rr = bf16_round(__fmaf_rn(half_bits_to_float(gain[c]), rr, half_bits_to_float(bias[c])));
            }
            const uint32_t cf = coef[c >> coef_shift];
            const float rtc = __fmaf_rn(half_bits_to_float(cf & 0xffff), rr, half_bits_to_float(cf >> 16));
            const float e = __fsub_rn(h, rtc);
            const unsigned long long comp =
                ((unsigned long long)(__float_as_uint(e) & 0x7fffffffu) << 16) | (unsigned long long)(0xffff - c);
            // a composite is 0 only for |e| == 0 at channel 65535, which d <= 8192 excludes
            if (comp < prev && comp > best) { best = comp; beste = e; bestrt = rtc; }
        }
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            const float othere = __shfl_xor_sync(0xffffffffu, beste, o);
            const float otherrt = __shfl_xor_sync(0xffffffffu, bestrt, o);
            if (other > best) { best = other; beste = othere; bestrt = otherrt; }
        }
        if (lane == r) { mine = best; minee = beste; minert = bestrt; }
        prev = best;
    }
    *c_out = 0xffff - (int)(mine & 0xffffull);
    *e_out = minee;
    *rt_out = minert;
}

// NV: slab maxima per lane (d <= 32*32*NV).  KT: the number of outliers when it is 8 (unrolled), else 0 = p.topk.
// bits: code width (only the clearing of the codes depends on it).  A warp works on kOutPair tokens at a time, phase
// by phase, so that their trips to memory (scattered 32-byte reads of X, the reference row and the record, which
// bound this pass) overlap.
constexpr int kOutPair = 2;

// W: warps per CTA.  7 = four CTAs of 72 registers per SM (56 tokens in flight), the faster shape without x_hat;
// 8 = three CTAs of 80 registers (48 tokens), which the variant that also patches x_hat prefers.
template <int NV, int KT, bool SUB, int W>
__global__ void __launch_bounds__(W * 32, W == 7 ? 4 : 3) outlier_kernel(const CodecParams p, const int bits) {
    constexpr int U = kOutPair;
    __shared__ float s_e[W][U][kOutCap];
    __shared__ float s_rt[W][U][kOutCap];
    __shared__ unsigned short s_c[W][U][kOutCap];
    __shared__ unsigned char s_hot[W][U][32 * NV];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d = p.d, nth = d >> 5;
    const int k = KT ? KT : p.topk;
    const uint32_t cmask = (1u << bits) - 1u;
    const long long tstride = (long long)gridDim.x * W * U;
    const unsigned int lt_mask = (1u << lane) - 1u;
    const int tm_stride = (nth + 3) & ~3;       // rows of slab maxima are padded to 16 bytes
    const bool want_xhat = p.X_hat != nullptr;
    const int my0 = NV * lane;                  // first slab of this lane
    const int my_n = min(NV, max(0, nth - my0));  // how many of its NV slabs exist
    const int coef_shift = 5 + p.lpg_shift;
    bool shared = false;   // coefficient words per segment, outside the records
    if constexpr (SUB) shared = p.coef_ext != nullptr;
    const int coff = shared ? 0 : 4 * p.J;
    // everything this kernel reads was written by the streaming pass launched just before it
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const long long n_tok = tokens_to_do<SUB>(p);

    for (long long ti0 = ((long long)blockIdx.x * W + warp) * U; ti0 < n_tok; ti0 += tstride) {
        long long t[U];
        const uint16_t *xrow[U], *rrow[U];
        const uint32_t *coefp[U];
        unsigned char *rec[U];
        unsigned int tau[U];
        int nh[U], n[U];
        bool live[U];
        // ---- (a) slab maxima, threshold, and the slabs that reach it, in slab order
#pragma unroll
        for (int u = 0; u < U; u++) {
            live[u] = ti0 + u < n_tok;
            t[u] = live[u] ? token_at<SUB>(p, ti0 + u) : 0;
            unsigned int tv[NV];
            {
                const float *tm = p.tmax + t[u] * tm_stride + my0;
                const int lim = live[u] ? my_n : 0;
                if (NV % 4 == 0) {
#pragma unroll
                    for (int j = 0; j < NV / 4; j++) {
                        uint4 v = make_uint4(0u, 0u, 0u, 0u);
                        if (4 * j < lim) v = __ldg(reinterpret_cast<const uint4 *>(tm) + j);   // rows are padded to 16 bytes
                        tv[4 * j + 0] = 4 * j + 0 < lim ? v.x : 0u;
                        tv[4 * j + 1] = 4 * j + 1 < lim ? v.y : 0u;
                        tv[4 * j + 2] = 4 * j + 2 < lim ? v.z : 0u;
                        tv[4 * j + 3] = 4 * j + 3 < lim ? v.w : 0u;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < NV; i++) tv[i] = i < lim ? __float_as_uint(__ldg(tm + i)) : 0u;
                }
            }
            // reference row of the token, by the same rules as the streaming pass (which already reported bad rows)
            const int row = live[u] ? resolve_row<SUB>(p, p.ref_row ? p.ref_row[t[u]] : (int)t[u], false) : -1;
            xrow[u] = p.X + t[u] * d;
            rrow[u] = row >= 0 ? ref_row_ptr<SUB>(p, row) : nullptr;
            rec[u] = p.payload + t[u] * p.rec;
            coefp[u] = reinterpret_cast<const uint32_t *>(rec[u]);
            if constexpr (SUB)
                if (shared) coefp[u] = p.coef_ext + (long long)(live[u] ? p.seg_of[t[u]] : 0) * p.J;
            // threshold.  Bit patterns of non-negative floats order like integers.
            unsigned int m1 = tv[0], m2 = 0u;
#pragma unroll
            for (int i = 1; i < NV; i++) {
                m2 = max(m2, min(m1, tv[i]));
                m1 = max(m1, tv[i]);
            }
#pragma unroll
            for (int r = 1; r < k; r++) {
                const unsigned int top = __reduce_max_sync(0xffffffffu, m1);
                const unsigned int bal = __ballot_sync(0xffffffffu, m1 == top);
                const bool pop = m1 == top && (bal & lt_mask) == 0u;
                m1 = pop ? m2 : m1;
                m2 = pop ? 0u : m2;
            }
            tau[u] = __reduce_max_sync(0xffffffffu, m1);
            // tau == 0: fewer than k slabs hold anything but zeros, every element is a candidate: whole-token path
            nh[u] = 0;
            n[u] = live[u] ? kOutCap + 1 : 0;
            if (tau[u] != 0u) {
                unsigned int hm = 0u;
#pragma unroll
                for (int i = 0; i < NV; i++) hm |= (tv[i] >= tau[u]) ? (1u << i) : 0u;
                int incl = __popc(hm);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int up = __shfl_up_sync(0xffffffffu, incl, o);
                    incl += lane >= o ? up : 0;
                }
                nh[u] = __shfl_sync(0xffffffffu, incl, 31);
                int at = incl - __popc(hm);
                while (hm) {
                    s_hot[warp][u][at++] = (unsigned char)(my0 + __ffs(hm) - 1);
                    hm &= hm - 1u;
                }
                n[u] = 0;
            }
        }
        __syncwarp();
        // ---- (b) candidates: eight slabs per round, four lanes per slab, eight channels per lane.  The first
        // round of every token is loaded before any of them is used.
        auto load_round = [&](int u, int base, int &c0, bool &act, uint4 &xw, uint4 &rw, uint32_t &cf) {
            const int hi = base + (lane >> 2);
            act = hi < nh[u];
            c0 = act ? (int)s_hot[warp][u][hi] * 32 + (lane & 3) * 8 : 0;
            xw = make_uint4(0u, 0u, 0u, 0u);
            rw = xw;
            cf = 0u;
            if (act) {
                xw = __ldg(reinterpret_cast<const uint4 *>(xrow[u] + c0));
                if (rrow[u]) rw = __ldg(reinterpret_cast<const uint4 *>(rrow[u] + c0));
                cf = coefp[u][c0 >> coef_shift];
            }
        };
        auto use_round = [&](int u, int c0, bool act, const uint4 &xw, const uint4 &rw, uint32_t cf) {
            const uint32_t xs[4] = {xw.x, xw.y, xw.z, xw.w};
            const uint32_t rs[4] = {rw.x, rw.y, rw.z, rw.w};
            const float ca = half_bits_to_float(cf & 0xffff), cb = half_bits_to_float(cf >> 16);
            float e[8], rt[8];
            if (rrow[u] && p.gain) {
#pragma unroll
                for (int i = 0; i < 8; i++) {
                    const uint32_t xb = (i & 1) ? (xs[i >> 1] & 0xffff0000u) : (xs[i >> 1] << 16);
                    const uint32_t rb = (i & 1) ? (rs[i >> 1] & 0xffff0000u) : (rs[i >> 1] << 16);
                    const float r = bf16_round(__fmaf_rn(half_bits_to_float(p.gain[c0 + i]), __uint_as_float(rb),
                                                         half_bits_to_float(p.bias[c0 + i])));
                    rt[i] = __fmaf_rn(ca, r, cb);
                    e[i] = __fsub_rn(__uint_as_float(xb), rt[i]);
                }
            } else {
                // without a reference rw is zero, which is the zero reference of a directly coded token
                const u64 a2 = pack2(ca, ca), b2 = pack2(cb, cb);
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    const u64 rt2 = pfma(a2, bf16x2_to_p(rs[i]), b2);
                    unpack2(rt2, rt[2 * i], rt[2 * i + 1]);
                    unpack2(psub(bf16x2_to_p(xs[i]), rt2), e[2 * i], e[2 * i + 1]);
                }
            }
            // which of the lane's eight elements reach the threshold (tau > 0 here; for finite values the
            // comparison of magnitudes is the comparison of their bit patterns)
            const float tauf = __uint_as_float(tau[u]);
            uint32_t m = 0u;
#pragma unroll
            for (int i = 0; i < 8; i++) m |= (fabsf(e[i]) >= tauf) ? (1u << i) : 0u;
            if (!act) m = 0u;
            const int cnt = __popc(m);
            // position of the lane's first candidate (candidates come out in channel order).  Almost always no
            // lane has two, and a ballot does; otherwise a prefix sum over the lanes.
            int pos, total;
            if (!__any_sync(0xffffffffu, cnt > 1)) {
                const unsigned int bal = __ballot_sync(0xffffffffu, cnt != 0);
                pos = n[u] + __popc(bal & lt_mask);
                total = __popc(bal);
            } else {
                int inc2 = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int up = __shfl_up_sync(0xffffffffu, inc2, o);
                    inc2 += lane >= o ? up : 0;
                }
                pos = n[u] + inc2 - cnt;
                total = __shfl_sync(0xffffffffu, inc2, 31);
            }
            while (m) {
                const int i = __ffs(m) - 1;
                m &= m - 1u;
                if (pos < kOutCap) {
                    s_e[warp][u][pos] = pick8(e, i);
                    s_c[warp][u][pos] = (unsigned short)(c0 + i);
                    if (want_xhat) s_rt[warp][u][pos] = pick8(rt, i);
                }
                pos++;
            }
            n[u] += total;
        };
        {
            int c0[U];
            bool act[U];
            uint4 xw[U], rw[U];
            uint32_t cf[U];
#pragma unroll
            for (int u = 0; u < U; u++) load_round(u, 0, c0[u], act[u], xw[u], rw[u], cf[u]);
#pragma unroll
            for (int u = 0; u < U; u++) {
                if (nh[u] > 0) use_round(u, c0[u], act[u], xw[u], rw[u], cf[u]);
                for (int base = 8; base < nh[u] && n[u] <= kOutCap; base += 8) {
                    load_round(u, base, c0[u], act[u], xw[u], rw[u], cf[u]);
                    use_round(u, c0[u], act[u], xw[u], rw[u], cf[u]);
                }
            }
        }
        __syncwarp();
        // ---- (c) one candidate per lane, in channel order; while there are too many the smallest goes
#pragma unroll
        for (int u = 0; u < U; u++) {
            if (!live[u]) continue;
            bool won;
            int wc = 0;
            float we = 0.f, wrt = 0.f;
            if (n[u] <= kOutCap) {
                won = lane < n[u];
                if (won) {
                    wc = s_c[warp][u][lane];
                    we = s_e[warp][u][lane];
                    if (want_xhat) wrt = s_rt[warp][u][lane];
                }
                unsigned int mag = won ? (__float_as_uint(we) & 0x7fffffffu) : 0xffffffffu;
                for (int extra = n[u] - k; extra > 0; extra--) {
                    const unsigned int low = __reduce_min_sync(0xffffffffu, mag);
                    const unsigned int bal = __ballot_sync(0xffffffffu, mag == low);
                    if (lane == 31 - __clz(bal)) { mag = 0xffffffffu; won = false; }   // among equals the highest channel
                }
            } else {
                select_whole_token(d, k, coef_shift, xrow[u], rrow[u], p.gain, p.bias, coefp[u], lane, &wc, &we, &wrt);
                won = lane < k;
            }
            // ---- (d) outlier fields in channel order, dense codes at those channels cleared
            int pos = __popc(__ballot_sync(0xffffffffu, won) & lt_mask);
            if (n[u] > kOutCap) {   // the whole-token path returns its winners by rank, not by channel
                pos = 0;
                for (int y = 0; y < k; y++) {
                    const int cy = __shfl_sync(0xffffffffu, wc, y);
                    pos += cy < wc ? 1 : 0;
                }
            }
            if (won) {
                unsigned short *oidx = reinterpret_cast<unsigned short *>(rec[u] + coff + p.code_bytes);
                const uint32_t hv = float_to_half_bits_sat(we);
                oidx[pos] = (unsigned short)wc;
                oidx[k + pos] = (unsigned short)hv;
                // the sender-side reconstruction of an outlier channel: (alpha*r + beta) + the binary16 value
                if (want_xhat)
                    p.X_hat[t[u] * d + wc] = __bfloat16_as_ushort(__float2bfloat16_rn(__fadd_rn(wrt, half_bits_to_float(hv))));
                uint32_t *codes32 = reinterpret_cast<uint32_t *>(rec[u] + coff);
                const int bit = wc * bits, wd = bit >> 5, sh = bit & 31;
                atomicAnd(&codes32[wd], ~(cmask << sh));
                if (sh + bits > 32) atomicAnd(&codes32[wd + 1], ~(cmask >> (32 - sh)));
            }
        }
        __syncwarp();
    }
}

// step tables from the per-CTA partial sums (fixed summation order -> deterministic)
__global__ void calib_finalize_kernel(const float *partial, int nblocks, int d, int bits, float clip_sigmas, float *step,
                                      float *inv_step) {
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= 2 * d) return;
    int row = c / d;
    const int *cnt = reinterpret_cast<const int *>(partial + (long long)nblocks * 2 * d);
    double sum = 0.0;
    long long n = 0;
    for (int b = 0; b < nblocks; b++) {
        sum += (double)partial[(long long)b * 2 * d + c];
        n += cnt[2 * b + row];
    }
    float s = 0.f, is = 0.f;
    if (n > 0) {
        double qmax = (double)((1 << (bits - 1)) - 1);
        double want = (double)clip_sigmas * sqrt(sum / (double)n) / qmax;
        if (want > 0.0) {
            if (want > 65504.0) want = 65504.0;
            __half h = __double2half(want);
            if ((double)__half2float(h) < want) h = __ushort_as_half((unsigned short)(__half_as_ushort(h) + 1));  // round up
            s = __half2float(h);
            if (s != 0.f) is = __fdiv_rn(1.0f, s);
        }
    }
    step[c] = s;
    inv_step[c] = is;
}

// ------------------------------------------------------------------------------------------------
// reconstruct (receiver and sender)
// ------------------------------------------------------------------------------------------------
// Per token: record and reference row arrive in a stage; every thread dequantises its 32 channels
// (code -> binary32 through the 2^23 trick, times the step), adds the aligned reference, rounds to bf16
// into an output row in shared memory, patches the outliers it owns, and the row leaves as one bulk store.
// The step table row of referenced tokens lives in registers for the whole kernel (a thread always owns
// the same channels); direct tokens read row 1 through L1.
template <int BITS, int KT, bool SUB>
__global__ void __launch_bounds__(256) decode_kernel(const CodecParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int rot = (lane >> 1) & 3;
    const int d = p.d;
    const bool valid = tid * 32 < d;
    const DecSmem L = dec_smem_layout(d, p.rec, p.stages);
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem);
    const uint32_t sbase = smem_u32(smem);
    const int S = p.stages;
    constexpr uint32_t cmask = (1u << BITS) - 1u;
    constexpr uint32_t H = 1u << (BITS - 1);
    // 1 in every one of the 8 fields of a code word, and H in every field
    constexpr uint32_t ones = (BITS == 4) ? 0x11111111u : (BITS == 3) ? 0x00249249u : 0x00005555u;
    constexpr uint32_t highs = ones << (BITS - 1);
    constexpr float kBase = 8388608.0f + (float)H;  // 2^23 + H
    const uint32_t row_bytes = 2u * (uint32_t)d;

    if (tid == 0) {
        for (int s = 0; s < S; s++) mbar_init(smem_u32(&ctrl->bar[s]), 1);
        mbar_init_fence();
    }
    __syncthreads();

    bool shared = false;   // coefficient words per segment, outside the records
    if constexpr (SUB) shared = p.coef_ext != nullptr;
    const int coff = shared ? 0 : 4 * p.J;
    const int first = blockIdx.x, stride = gridDim.x;
    const long long n_tok = tokens_to_do<SUB>(p);
    const int n_my = (n_tok > first) ? (int)((n_tok - first + stride - 1) / stride) : 0;

    int next_raw = 0;
    auto raw_row_of = [&](int k) -> int {
        long long t = token_at<SUB>(p, first + (long long)k * stride);
        return p.ref_row ? p.ref_row[t] : (int)t;
    };
    if (tid == 0) {
        for (int k = 0; k < S - 1 && k < n_my; k++) {
            long long t = token_at<SUB>(p, first + (long long)k * stride);
            issue_token_loads<SUB>(p, ctrl, sbase + L.stage0 + k * L.stage_bytes, L.rec_pad, k, resolve_row<SUB>(p, raw_row_of(k)),
                              p.payload + t * p.rec, (uint32_t)p.rec, t);
        }
        if (S - 1 < n_my) next_raw = raw_row_of(S - 1);
    }

    uint32_t off[4];
#pragma unroll
    for (int j = 0; j < 4; j++) off[j] = (uint32_t)(tid * 64 + ((j + rot) & 3) * 16);
    // step table, row 0, in slot order
    u64 st0[16];
#pragma unroll
    for (int j = 0; j < 4; j++) {
        float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
        if (valid) {
            s0 = __ldg(reinterpret_cast<const float4 *>(p.step + (off[j] >> 1)));
            s1 = __ldg(reinterpret_cast<const float4 *>(p.step + (off[j] >> 1) + 4));
        }
        st0[4 * j + 0] = pack2(s0.x, s0.y);
        st0[4 * j + 1] = pack2(s0.z, s0.w);
        st0[4 * j + 2] = pack2(s1.x, s1.y);
        st0[4 * j + 3] = pack2(s1.z, s1.w);
    }
    const u64 base2 = pack2(kBase, kBase);

    int stage = 0, obuf = 0, issue_stage = S - 1;
    bool aborted = false;
    uint32_t parity = 0;
    for (int it = 0; it < n_my; it++) {
        const long long t = token_at<SUB>(p, first + (long long)it * stride);
        if (tid == 0 && it + S - 1 < n_my) {
            const int k = it + S - 1;
            const long long tk = token_at<SUB>(p, first + (long long)k * stride);
            issue_token_loads<SUB>(p, ctrl, sbase + L.stage0 + issue_stage * L.stage_bytes, L.rec_pad, issue_stage,
                              resolve_row<SUB>(p, next_raw), p.payload + tk * p.rec, (uint32_t)p.rec, tk);
            if (k + 1 < n_my) next_raw = raw_row_of(k + 1);
        }
        const bool timed_out = !mbar_wait_bounded(smem_u32(&ctrl->bar[stage]), parity);
        if (timed_out && p.status) atomicOr(p.status, RAC_STATUS_TIMEOUT);
        const bool has_ref = ctrl->row[stage] >= 0;
        const unsigned char *rec = smem + L.stage0 + stage * L.stage_bytes;
        const uint32_t rs = sbase + L.stage0 + stage * L.stage_bytes + L.rec_pad;
        unsigned char *ob = smem + L.out0 + obuf * (int)row_bytes;
        const uint32_t obs = smem_u32(ob);

        if (valid) {
            uint32_t cf;
            if (shared) cf = p.coef_ext[(long long)ctrl->seg[stage] * p.J + (tid >> p.lpg_shift)];
            else cf = reinterpret_cast<const uint32_t *>(rec)[tid >> p.lpg_shift];
            const float a = half_bits_to_float(cf & 0xffff), b = half_bits_to_float(cf >> 16);
            const u64 a2 = pack2(a, a), b2 = pack2(b, b);
            // code words of the four pieces, in piece order, then rotated into slot order
            const uint32_t *cw = reinterpret_cast<const uint32_t *>(rec + coff) + tid * BITS;
            uint32_t words[4];
            if (BITS == 4) {
                words[0] = cw[0]; words[1] = cw[1]; words[2] = cw[2]; words[3] = cw[3];
            } else if (BITS == 3) {
                uint32_t w0 = cw[0], w1 = cw[1], w2 = cw[2];
                words[0] = w0 & 0xffffffu;
                words[1] = (w0 >> 24) | ((w1 & 0xffffu) << 8);
                words[2] = (w1 >> 16) | ((w2 & 0xffu) << 16);
                words[3] = w2 >> 8;
            } else {
                uint32_t w0 = cw[0], w1 = cw[1];
                words[0] = w0 & 0xffffu; words[1] = w0 >> 16; words[2] = w1 & 0xffffu; words[3] = w1 >> 16;
            }
            uint32_t reserved = 0;
#pragma unroll
            for (int q = 0; q < 4; q++) {
                uint32_t v = words[q] ^ highs;  // field == 0  <=>  code == -2^(BITS-1)
                reserved |= (v - ones) & ~v & highs;
                words[q] = v;                   // fields now hold code + H (offset binary)
            }
            if (reserved && p.status) atomicOr(p.status, RAC_STATUS_RESERVED_CODE);
            rot_left4(words, rot);
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const int c = (int)(off[j] >> 1);
                u64 r2[4], st2[4];
                if (has_ref) {
                    load_ref_slot(rs + off[j], p.gain, p.bias, c, r2);
#pragma unroll
                    for (int i = 0; i < 4; i++) st2[i] = st0[4 * j + i];
                } else {
                    const float4 s0 = __ldg(reinterpret_cast<const float4 *>(p.step + d + c));
                    const float4 s1 = __ldg(reinterpret_cast<const float4 *>(p.step + d + c + 4));
                    st2[0] = pack2(s0.x, s0.y); st2[1] = pack2(s0.z, s0.w); st2[2] = pack2(s1.x, s1.y); st2[3] = pack2(s1.z, s1.w);
#pragma unroll
                    for (int i = 0; i < 4; i++) r2[i] = 0ull;
                }
                const uint32_t w = words[j];
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    // exact integer -> binary32 without a convert: 2^23 + (code + H), minus (2^23 + H)
                    const float q0 = __uint_as_float(0x4b000000u | ((w >> (BITS * (2 * i))) & cmask));
                    const float q1 = __uint_as_float(0x4b000000u | ((w >> (BITS * (2 * i + 1))) & cmask));
                    float x0, x1;
                    unpack2(pfma(psub(pack2(q0, q1), base2), st2[i], pfma(a2, r2[i], b2)), x0, x1);
                    o[i] = f2_to_bf16x2(x0, x1);
                }
                sts128(obs + off[j], make_uint4(o[0], o[1], o[2], o[3]));
            }
            if (KT > 0) {
                // outliers whose channel this thread owns replace what the dense pass wrote
                const unsigned short *oidx = reinterpret_cast<const unsigned short *>(rec + coff + p.code_bytes);
                const unsigned short *oval = oidx + p.topk;
#pragma unroll
                for (int n = 0; n < KT; n++) {
                    if (n < p.topk) {
                        const int c = oidx[n];
                        if ((c >> 5) == tid) {
                            float r = 0.f;
                            if (has_ref) {
                                r = __uint_as_float((uint32_t)(*reinterpret_cast<const unsigned short *>(rec + L.rec_pad + 2 * c)) << 16);
                                if (p.gain) r = bf16_round(__fmaf_rn(half_bits_to_float(p.gain[c]), r, half_bits_to_float(p.bias[c])));
                            }
                            const float xh = __fadd_rn(__fmaf_rn(a, r, b), half_bits_to_float(oval[n]));
                            reinterpret_cast<unsigned short *>(ob)[c] = __bfloat16_as_ushort(__float2bfloat16_rn(xh));
                        }
                    }
                }
            }
        }
        if (KT > 0 && tid == 0) {
            const unsigned short *oidx = reinterpret_cast<const unsigned short *>(rec + coff + p.code_bytes);
            bool bad = false;
            for (int n = 0; n < p.topk; n++) bad |= oidx[n] >= d;
            if (bad && p.status) atomicOr(p.status, RAC_STATUS_OUTLIER_RANGE);
        }
        fence_async_smem();
        if (__syncthreads_or(timed_out)) { aborted = true; break; }  // one vote: every thread leaves together
        if (tid == 0) {
            bulk_store(p.X_hat + t * d, obs, row_bytes);
            bulk_commit();
            bulk_wait_read<1>();
        }
        if (++stage == S) { stage = 0; parity ^= 1u; }
        if (++issue_stage == S) issue_stage = 0;
        if (++obuf == kRecBufs) obuf = 0;
    }
    if (tid == 0) {
        bulk_wait_all();
        if (aborted) {
            for (int s = 0; s < S; s++) {
                mbar_wait_bounded(smem_u32(&ctrl->bar[s]), 0);
                mbar_wait_bounded(smem_u32(&ctrl->bar[s]), 1);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// reconstruct, streaming form: no CTA barrier in the loop
// ------------------------------------------------------------------------------------------------
// Same arithmetic as decode_kernel.  Every warp ends its share of a token with one arrival on the stage's `done`
// mbarrier and moves on, and the warp whose turn it is (token i: warp i mod warps) waits for `done`, sends the
// row off as a bulk store, and refills the stage once the store has read it.
// Records without per-token outliers: the output row is written IN PLACE over the token's reference row in the
// stage (a thread reads its 64-byte slab of r and writes x_hat there), so a stage is record + one row.
// Records with outliers: the output row is a row of its own, so that the reference survives the dense pass; the
// warp whose turn it is prepares the outliers while it waits for the others (lane n takes outlier n: aligned
// reference of that channel + the stored binary16 value) and writes them over the dense results once every warp
// has arrived.  No other thread looks at the outlier fields.  (A first version that let every thread test the
// outlier list for channels it owns cost ~150 warp instructions per 32 channels and lost to the barrier form.)
struct DwSmem {
    int stage0, stage_bytes, rec_pad, total;
};
__host__ __device__ inline DwSmem dw_smem_layout(int d, int rec, int stages, bool out_row) {
    DwSmem s;
    s.stage0 = align_up((int)sizeof(WsCtrl), 128);
    s.rec_pad = align_up(rec, 128);
    s.stage_bytes = s.rec_pad + 2 * d + (out_row ? 2 * d : 0);   // record, reference row (, output row)
    s.total = s.stage0 + stages * s.stage_bytes;
    return s;
}

// KT > 0: records with per-token outliers (the output row is a row of its own behind the reference row).
// ROW1: the call can contain directly coded tokens (a row list, or no reference at all); they take their steps
// from row 1 of the table, which this form keeps in registers as well.
// D: the hidden width as a compile-time constant (5120: -1 % on the reconstruction with directly coded tokens; at 4096
// the constant measured the same at 131072 tokens and 5 % slower at 16384, so that width reads it from the parameters).
template <int BITS, int KT, bool SUB, bool ROW1, int D = 0>
__global__ void __launch_bounds__(256, 2) decode_ws_kernel(const CodecParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nwarps = D ? (D / 32 + 31) / 32 : nt >> 5;
    const int rot = (lane >> 1) & 3;
    const int d = D ? D : p.d;
    const bool valid = tid * 32 < d;
    const int S = D ? (D / 32 > 128 ? 3 : 2) : p.stages;   // the host's rule: three stages for CTAs of more than 128 threads
    const DwSmem L = dw_smem_layout(d, p.rec, S, KT > 0);
    WsCtrl *ctrl = reinterpret_cast<WsCtrl *>(smem);
    const uint32_t sbase = smem_u32(smem);
    constexpr uint32_t cmask = (1u << BITS) - 1u;
    constexpr uint32_t H = 1u << (BITS - 1);
    constexpr uint32_t ones = (BITS == 4) ? 0x11111111u : (BITS == 3) ? 0x00249249u : 0x00005555u;
    constexpr uint32_t highs = ones << (BITS - 1);
    constexpr float kBase = 8388608.0f + (float)H;  // 2^23 + H
    const uint32_t row_bytes = 2u * (uint32_t)d;

    const int first = blockIdx.x, stride = gridDim.x;
    const long long n_tok = tokens_to_do<SUB>(p);
    const int n_my = (n_tok > first) ? (int)((n_tok - first + stride - 1) / stride) : 0;
    auto raw_row_of = [&](int k) -> int {
        long long t = token_at<SUB>(p, first + (long long)k * stride);
        return p.ref_row ? p.ref_row[t] : (int)t;
    };
    auto issue = [&](int k, int s, int raw_row) {
        const long long t = token_at<SUB>(p, first + (long long)k * stride);
        const int row = resolve_row<SUB>(p, raw_row);
        ctrl->row[s] = row;
        const uint32_t bar = smem_u32(&ctrl->full[s]);
        const uint32_t base = sbase + L.stage0 + s * L.stage_bytes;
        mbar_arrive_expect_tx(bar, p.test_extra_tx + (uint32_t)p.rec + (row >= 0 ? row_bytes : 0u));
        bulk_load(base, p.payload + t * p.rec, (uint32_t)p.rec, bar);
        if (row >= 0) bulk_load(base + L.rec_pad, ref_row_ptr<SUB>(p, row), row_bytes, bar);
    };

    if (tid == 0) {
        for (int s = 0; s < S; s++) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->done[s]), nwarps);
        }
        ctrl->abort = 0;
        mbar_init_fence();
    }
    __syncthreads();
    if (tid == 0)
        for (int k = 0; k < S && k < n_my; k++) issue(k, k, raw_row_of(k));

    uint32_t off[4];
#pragma unroll
    for (int j = 0; j < 4; j++) off[j] = (uint32_t)(tid * 64 + ((j + rot) & 3) * 16);
    // step table, row 0, in slot order
    u64 st0[16];
#pragma unroll
    for (int j = 0; j < 4; j++) {
        float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
        if (valid) {
            s0 = __ldg(reinterpret_cast<const float4 *>(p.step + (off[j] >> 1)));
            s1 = __ldg(reinterpret_cast<const float4 *>(p.step + (off[j] >> 1) + 4));
        }
        st0[4 * j + 0] = pack2(s0.x, s0.y);
        st0[4 * j + 1] = pack2(s0.z, s0.w);
        st0[4 * j + 2] = pack2(s1.x, s1.y);
        st0[4 * j + 3] = pack2(s1.z, s1.w);
    }
    // Row 1 (directly coded tokens) as packed binary16 in 16 registers, when binary16 holds every entry of the row
    // exactly -- which is how the calibration writes them.  Otherwise those tokens read the row from memory.
    uint32_t sh1[16];
    bool row1_exact = ROW1;
#pragma unroll
    for (int j = 0; j < 4; j++) {
        float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
        if (ROW1 && valid) {
            s0 = __ldg(reinterpret_cast<const float4 *>(p.step + d + (off[j] >> 1)));
            s1 = __ldg(reinterpret_cast<const float4 *>(p.step + d + (off[j] >> 1) + 4));
        }
        const float v[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const __half2 h = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
            const float2 back = __half22float2(h);
            row1_exact = row1_exact && back.x == v[2 * i] && back.y == v[2 * i + 1];
            sh1[4 * j + i] = *reinterpret_cast<const uint32_t *>(&h);
        }
    }
    if (ROW1) row1_exact = __syncthreads_and(row1_exact) != 0;
    const u64 base2 = pack2(kBase, kBase);

    int stage = 0, duty = 0;
    uint32_t parity = 0;
    bool timed_out = false;
    for (int it = 0; it < n_my; it++) {
        if (*reinterpret_cast<volatile int *>(&ctrl->abort)) break;
        unsigned char *rec = smem + L.stage0 + stage * L.stage_bytes;
        const uint32_t rs = sbase + L.stage0 + stage * L.stage_bytes + L.rec_pad;
        const uint32_t os = KT > 0 ? rs + row_bytes : rs;     // where x_hat goes: its own row, or over the reference
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_u32(&ctrl->full[stage]), parity))) { timed_out = true; break; }
        const bool has_ref = ctrl->row[stage] >= 0;

        if (valid) {
            const uint32_t cf = reinterpret_cast<const uint32_t *>(rec)[tid >> p.lpg_shift];
            const float a = half_bits_to_float(cf & 0xffff), b = half_bits_to_float(cf >> 16);
            const u64 a2 = pack2(a, a), b2 = pack2(b, b);
            // code words of the four pieces, in piece order, then rotated into slot order
            const uint32_t *cw = reinterpret_cast<const uint32_t *>(rec + 4 * p.J) + tid * BITS;
            uint32_t words[4];
            if (BITS == 4) {
                words[0] = cw[0]; words[1] = cw[1]; words[2] = cw[2]; words[3] = cw[3];
            } else if (BITS == 3) {
                uint32_t w0 = cw[0], w1 = cw[1], w2 = cw[2];
                words[0] = w0 & 0xffffffu;
                words[1] = (w0 >> 24) | ((w1 & 0xffffu) << 8);
                words[2] = (w1 >> 16) | ((w2 & 0xffu) << 16);
                words[3] = w2 >> 8;
            } else {
                uint32_t w0 = cw[0], w1 = cw[1];
                words[0] = w0 & 0xffffu; words[1] = w0 >> 16; words[2] = w1 & 0xffffu; words[3] = w1 >> 16;
            }
            uint32_t reserved = 0;
#pragma unroll
            for (int q = 0; q < 4; q++) {
                uint32_t v = words[q] ^ highs;  // field == 0  <=>  code == -2^(BITS-1)
                reserved |= (v - ones) & ~v & highs;
                words[q] = v;                   // fields now hold code + H (offset binary)
            }
            if (reserved && p.status) atomicOr(p.status, RAC_STATUS_RESERVED_CODE);
            rot_left4(words, rot);
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const int c = (int)(off[j] >> 1);
                u64 r2[4], st2[4];
                if (has_ref) {
                    load_ref_slot(rs + off[j], p.gain, p.bias, c, r2);
                } else {
#pragma unroll
                    for (int i = 0; i < 4; i++) r2[i] = 0ull;
                }
                if (has_ref) {
#pragma unroll
                    for (int i = 0; i < 4; i++) st2[i] = st0[4 * j + i];
                } else if (ROW1 && row1_exact) {
#pragma unroll
                    for (int i = 0; i < 4; i++) {
                        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&sh1[4 * j + i]));
                        st2[i] = pack2(f.x, f.y);
                    }
                } else {
                    const float4 s0 = __ldg(reinterpret_cast<const float4 *>(p.step + d + c));
                    const float4 s1 = __ldg(reinterpret_cast<const float4 *>(p.step + d + c + 4));
                    st2[0] = pack2(s0.x, s0.y); st2[1] = pack2(s0.z, s0.w); st2[2] = pack2(s1.x, s1.y); st2[3] = pack2(s1.z, s1.w);
                }
                const uint32_t w = words[j];
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    const float q0 = __uint_as_float(0x4b000000u | ((w >> (BITS * (2 * i))) & cmask));
                    const float q1 = __uint_as_float(0x4b000000u | ((w >> (BITS * (2 * i + 1))) & cmask));
                    float x0, x1;
                    unpack2(pfma(psub(pack2(q0, q1), base2), st2[i], pfma(a2, r2[i], b2)), x0, x1);
                    o[i] = f2_to_bf16x2(x0, x1);
                }
                sts128(os + off[j], make_uint4(o[0], o[1], o[2], o[3]));
            }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&ctrl->done[stage])) : "memory");

        if (warp == duty) {
            const int k_next = it + S;
            int raw_next = 0;
            if (lane == 0 && k_next < n_my) raw_next = raw_row_of(k_next);
            // outliers: lane n prepares outlier n (Eq. 9: aligned reference + binary16 value) while the other warps
            // are still busy; record and reference row do not change any more
            int patch_c = -1;
            unsigned short patch_x = 0;
            if (KT > 0) {
                const unsigned short *oidx = reinterpret_cast<const unsigned short *>(rec + 4 * p.J + p.code_bytes);
                const unsigned short *oval = oidx + p.topk;
                const int c = lane < p.topk ? (int)oidx[lane] : -1;
                const bool ok = c >= 0 && c < d;
                if (ok) {
                    const uint32_t cf = reinterpret_cast<const uint32_t *>(rec)[c >> (5 + p.lpg_shift)];
                    float r = 0.f;
                    if (has_ref) {
                        r = __uint_as_float((uint32_t)(*reinterpret_cast<const unsigned short *>(rec + L.rec_pad + 2 * c)) << 16);
                        if (p.gain) r = bf16_round(__fmaf_rn(half_bits_to_float(p.gain[c]), r, half_bits_to_float(p.bias[c])));
                    }
                    const float xh = __fadd_rn(__fmaf_rn(half_bits_to_float(cf & 0xffff), r, half_bits_to_float(cf >> 16)),
                                               half_bits_to_float(oval[lane]));
                    patch_x = __bfloat16_as_ushort(__float2bfloat16_rn(xh));
                }
                // a malformed record may name a channel twice: the later entry wins, as in a serial pass
                const unsigned int same = __match_any_sync(0xffffffffu, ok ? c : -1 - lane);
                if (ok && (31 - __clz(same)) == lane) patch_c = c;
                if (__any_sync(0xffffffffu, c >= d) && lane == 0 && p.status) atomicOr(p.status, RAC_STATUS_OUTLIER_RANGE);
            }
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_u32(&ctrl->done[stage]), parity))) { timed_out = true; break; }
            if (KT > 0) {
                if (patch_c >= 0)
                    reinterpret_cast<unsigned short *>(rec + L.rec_pad + row_bytes)[patch_c] = patch_x;
                fence_async_smem();
                __syncwarp();
            }
            if (lane == 0) {
                const long long t = token_at<SUB>(p, first + (long long)it * stride);
                bulk_store(p.X_hat + t * d, os, row_bytes);
                bulk_commit();
                bulk_wait_read<0>();      // the row has been read: the stage may be refilled
                if (k_next < n_my) issue(k_next, stage, raw_next);
            }
            __syncwarp();
        }
        if (++stage == S) { stage = 0; parity ^= 1u; }
        if (++duty == nwarps) duty = 0;
    }
    if (timed_out) {
        ctrl->abort = 1;
        if (p.status) atomicOr(p.status, RAC_STATUS_TIMEOUT);
    }
    __syncthreads();
    if (lane == 0) bulk_wait_all();
    if (tid == 0 && *reinterpret_cast<volatile int *>(&ctrl->abort)) {
        for (int s = 0; s < S; s++) {
            mbar_wait_bounded(smem_u32(&ctrl->full[s]), 0);
            mbar_wait_bounded(smem_u32(&ctrl->full[s]), 1);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side: launch plumbing
// ------------------------------------------------------------------------------------------------

static int fill_common(const Geometry &g, CodecParams *p, long long T, const void *ref_base, long long ref_rows,
                       const int32_t *ref_row, const void *gain, const void *bias, uint32_t *status) {
    if (T < 0 || ref_rows < 0) return RAC_EINVAL;
    if ((gain == nullptr) != (bias == nullptr)) return RAC_EINVAL;
    if (ref_base && !ref_row && ref_rows < T) return RAC_EINVAL;
    if (ref_base && !aligned16(ref_base)) return RAC_EALIGN;
    if (gain && (!aligned16(gain) || !aligned16(bias))) return RAC_EALIGN;
    if (ref_rows > 0x7fffffffLL) return RAC_EUNSUPPORTED;
    p->ref_base = static_cast<const uint16_t *>(ref_base);
    p->ref_rows = ref_base ? ref_rows : 0;
    p->ref_row = ref_row;
    p->gain = static_cast<const uint16_t *>(gain);
    p->bias = static_cast<const uint16_t *>(bias);
    p->status = status;
    p->T = T;
    p->d = g.d;
    p->J = g.J;
    p->lpg = g.lpg;
    p->lpg_shift = 0;
    while ((1 << p->lpg_shift) < g.lpg) p->lpg_shift++;
    p->topk = g.topk;
    p->rec = g.rec;
    p->code_bytes = g.code_bytes;
    p->inv_group = 1.0f / (float)g.group;
    p->Jq = g.Jq;
    p->lpq = g.lpq;
    p->qgen = g.qgen;
    p->lpq_shift = 0;
    while ((1 << p->lpq_shift) < g.lpq) p->lpq_shift++;
    p->kg = g.topk_group;
    p->scale_off = g.scale_off;
    p->codes_off = g.codes_off;
    p->goff_off = g.goff_off;
    p->gval_off = g.gval_off;
    p->test_extra_tx = 0;
    return RAC_OK;
}

// Launch of a kernel that runs after the one before it on the stream, allowed to be set up while that one drains
// (programmatic dependent launch): the kernel itself waits for its predecessor's memory before it reads anything.
template <typename K, typename... Args>
static void launch_after(K kernel, unsigned grid, unsigned block, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, args...);
}

// Encode: the streaming kernel, then (with outliers) the selection kernel.  Variant 4 of the streaming kernel
// caps registers at 96 so that four 160-thread CTAs fit on an SM.
static int launch_encode(const Geometry &g, CodecParams &p, long long max_ctas, cudaStream_t stream) {
    if (g.scale_mode == 1) return launch_encode_dyn(g, p, max_ctas, stream);
    const bool topk = g.topk > 0;
    p.stages = 2;
    WsSmem L = ws_smem_layout(g.d, g.rec, p.stages, topk);
    // With x_hat the kernel reads both step tables every token; at four CTAs per SM the shared-memory carve-out
    // leaves too little L1 for them, so that variant runs three CTAs per SM at 128 registers.
    const bool tight = g.nthreads > 96 && g.nthreads <= 160 && !p.X_hat;
    int rc = RAC_EUNSUPPORTED;
    const bool sub = p.tok_list || p.intra_base || p.coef_ext;   // the subset form has one variant per width: it is not the hot path
    // widths 4096 and 5120 with no or eight outliers per token run variants with the whole record geometry compiled in
    const bool geo = (g.d == 5120 || g.d == 4096) && (g.topk == 0 || g.topk == 8);
    const bool allref = p.ref_row == nullptr && p.ref_base != nullptr;   // identity rows: every token has its reference
#define RAC_ENC4(B, K, X, G, W)                                                                                        \
    (tight ? launch_persistent(encode_ws_kernel<B, K, X, 4, false, G, W>, p, g.nthreads, L.total, max_ctas, stream) \
           : launch_persistent(encode_ws_kernel<B, K, X, 2, false, G, W>, p, g.nthreads, L.total, max_ctas, stream))
    // (at those widths the register variant follows from x_hat alone: 96 registers without it, 128 with it)
#define RAC_ENC5(B, K, X, G, W, R) \
    launch_persistent(encode_ws_kernel<B, K, X, (X ? 2 : 4), false, G, W, R>, p, g.nthreads, L.total, max_ctas, stream)
#define RAC_ENC3(B, K, X, G)                                                                              \
    (!geo ? RAC_ENC4(B, K, X, G, 0)                                                                       \
     : g.d == 5120 ? (allref ? RAC_ENC5(B, K, X, G, 5120, true) : RAC_ENC5(B, K, X, G, 5120, false))     \
                   : (allref ? RAC_ENC5(B, K, X, G, 4096, true) : RAC_ENC5(B, K, X, G, 4096, false)))
#define RAC_ENC2(B, K, X)                                                                                           \
    (sub ? launch_persistent(encode_ws_kernel<B, K, X, 2, true, 0>, p, g.nthreads, L.total, max_ctas, stream)      \
     : g.lpg == 4 ? RAC_ENC3(B, K, X, 4) : g.lpg == 2 ? RAC_ENC3(B, K, X, 2) : RAC_ENC4(B, K, X, 0, 0))
#define RAC_ENC(B, K) (p.X_hat ? RAC_ENC2(B, K, true) : RAC_ENC2(B, K, false))
    switch (g.bits) {
        case 4: rc = topk ? RAC_ENC(4, true) : RAC_ENC(4, false); break;
        case 3: rc = topk ? RAC_ENC(3, true) : RAC_ENC(3, false); break;
        case 2: rc = topk ? RAC_ENC(2, true) : RAC_ENC(2, false); break;
    }
#undef RAC_ENC5
#undef RAC_ENC4
#undef RAC_ENC3
#undef RAC_ENC2
#undef RAC_ENC
    if (rc != RAC_OK || !topk) return rc;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc != RAC_OK) return rc;
    // a warp per pair of tokens.  Without x_hat: four CTAs of seven warps per SM (72 registers); with x_hat (more state per
    // token): three CTAs of eight warps (80 registers).  With more work than one round of them, every warp gets the same
    // number of rounds (a grid of whole rounds, not a full grid with a ragged last round).
    // (measured at 131072 x 5120: 0.901 against 0.910 ms; with few rounds the smaller CTAs win: 16384 x 4096 0.105 -> 0.102 ms)
    const bool wide = sub || (p.X_hat != nullptr && p.T > (long long)di.sms * 3 * 8 * kOutPair * 6);
    const int wpc = wide ? 8 : 7;
    const long long per_cta = wpc * kOutPair;
    long long blocks = (p.T + per_cta - 1) / per_cta;
    const long long resident = (long long)di.sms * (wide ? 3 : 4);
    if (blocks > resident) {
        const long long rounds = (blocks + resident - 1) / resident;
        blocks = (blocks + rounds - 1) / rounds;
    }
    const int nth = g.d / 32;
    const unsigned nb = (unsigned)blocks, nt = wpc * 32;
#define RAC_OUT(NV, KT)                                                                    \
    (wide ? launch_after(outlier_kernel<NV, KT, false, 8>, nb, nt, stream, p, g.bits)     \
          : launch_after(outlier_kernel<NV, KT, false, 7>, nb, nt, stream, p, g.bits))
    if (sub) launch_after(outlier_kernel<8, 0, true, 8>, nb, nt, stream, p, g.bits);
    else if (g.topk == 8) {
        if (nth <= 128) RAC_OUT(4, 8);
        else if (nth <= 160) RAC_OUT(5, 8);
        else RAC_OUT(8, 8);
    } else {
        if (nth <= 128) RAC_OUT(4, 0);
        else if (nth <= 160) RAC_OUT(5, 0);
        else RAC_OUT(8, 0);
    }
#undef RAC_OUT
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

static int launch_decode(const Geometry &g, CodecParams &p, cudaStream_t stream) {
    if (g.scale_mode == 1) return launch_decode_dyn(g, p, stream);
    p.stages = 2;
    DecSmem L = dec_smem_layout(g.d, g.rec, p.stages);
    const int kt = g.topk == 0 ? 0 : (g.topk <= 8 ? 8 : 16);
    const bool sub = p.tok_list || p.intra_base || p.coef_ext;
    // The streaming form is the faster one (131072 x 5120: 0.444 against 0.517 ms without outliers, 0.451 against
    // 0.491 ms with eight; 131072 x 4096: 0.37 against 0.43 and 0.40 against 0.46 ms).  The barrier form serves the
    // token-list / second-reference-buffer calls.
    const bool ws = !sub;
    const int wstages = (g.nthreads > 128 ? 3 : 2);
    DwSmem LW = dw_smem_layout(g.d, g.rec, wstages, kt > 0);
    if (ws) p.stages = wstages;
    const bool row1 = p.ref_row != nullptr || p.ref_base == nullptr;   // else every token has its reference row
#define RAC_DECW(B, K, W)                                                                                      \
    (row1 ? launch_persistent(decode_ws_kernel<B, K, false, true, W>, p, g.nthreads, LW.total, p.T, stream)   \
          : launch_persistent(decode_ws_kernel<B, K, false, false, W>, p, g.nthreads, LW.total, p.T, stream))
#define RAC_DEC(B, K)                                                                            \
    (sub ? launch_persistent(decode_kernel<B, K, true>, p, g.nthreads, L.total, p.T, stream)    \
     : ws ? (g.d == 5120 ? RAC_DECW(B, K, 5120) : RAC_DECW(B, K, 0)) \
         : launch_persistent(decode_kernel<B, K, false>, p, g.nthreads, L.total, p.T, stream))
    switch (g.bits * 100 + kt) {
        case 400: return RAC_DEC(4, 0);
        case 408: return RAC_DEC(4, 8);
        case 416: return RAC_DEC(4, 16);
        case 300: return RAC_DEC(3, 0);
        case 308: return RAC_DEC(3, 8);
        case 316: return RAC_DEC(3, 16);
        case 200: return RAC_DEC(2, 0);
        case 208: return RAC_DEC(2, 8);
        case 216: return RAC_DEC(2, 16);
    }
#undef RAC_DEC
#undef RAC_DECW
    return RAC_EUNSUPPORTED;
}

// Tokens whose reference is a row of the same prompt (ref_row >= first_intra_row) form the second wave; both
// lists come out in ascending token order.  One CTA; every warp owns a contiguous range of 32-token tiles
// (coalesced reads), counts its second-wave tokens with ballots, the warps' counts are prefix-summed, and a
// second sweep writes both lists at running offsets.
__global__ void __launch_bounds__(1024) split_waves_kernel(const int32_t *ref_row, int T, long long first_intra_row,
                                                           int32_t *wave1, int32_t *wave2, int32_t *wave_count) {
    __shared__ int s_cnt[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tiles = (T + 31) / 32;
    const int per = (tiles + 31) / 32;
    const int t_lo = min(tiles, warp * per), t_hi = min(tiles, t_lo + per);
    int c2 = 0;
    for (int tg = t_lo; tg < t_hi; tg += 8) {
        int v[8];
#pragma unroll
        for (int u = 0; u < 8; u++) {
            const int i = (tg + u) * 32 + lane;
            v[u] = (tg + u < t_hi && i < T) ? ref_row[i] : -1;
        }
#pragma unroll
        for (int u = 0; u < 8; u++) c2 += __popc(__ballot_sync(0xffffffffu, v[u] >= first_intra_row));
    }
    if (lane == 0) s_cnt[warp] = c2;
    __syncthreads();
    int o2 = 0, total2 = 0;
    for (int w = 0; w < 32; w++) {
        if (w < warp) o2 += s_cnt[w];
        total2 += s_cnt[w];
    }
    int o1 = min(T, t_lo * 32) - o2;
    const unsigned int below = (1u << lane) - 1u;
    for (int tg = t_lo; tg < t_hi; tg += 8) {
        int v[8];
#pragma unroll
        for (int u = 0; u < 8; u++) {
            const int i = (tg + u) * 32 + lane;
            v[u] = (tg + u < t_hi && i < T) ? ref_row[i] : -1;
        }
#pragma unroll
        for (int u = 0; u < 8; u++) {
            const int i = (tg + u) * 32 + lane;
            const bool in = tg + u < t_hi && i < T;
            const bool is2 = in && v[u] >= first_intra_row, is1 = in && !is2;
            const unsigned int b2 = __ballot_sync(0xffffffffu, is2), b1 = __ballot_sync(0xffffffffu, is1);
            if (is2) wave2[o2 + __popc(b2 & below)] = i;
            if (is1) wave1[o1 + __popc(b1 & below)] = i;
            o2 += __popc(b2);
            o1 += __popc(b1);
        }
    }
    if (tid == 0) {
        wave_count[1] = total2;
        wave_count[0] = T - total2;
    }
}

// ------------------------------------------------------------------------------------------------
// Eq. 6 over several fitting positions: one coefficient pair per (segment of tokens, group)
// ------------------------------------------------------------------------------------------------
// Pass 1 (calib_kernel<true>) leaves the centred statistics of every (token, group).  Pass 2: one warp per
// (segment, group) merges them with the pairwise update of means and centred sums, in binary64 and in a fixed
// order (lane l takes tokens l, l+32, ... of the segment in order, then a shuffle tree), applies the
// zero-variance rule and rounds to the wire format.
struct Mom {
    double n, mr, mh, sxx, sxy;
};
__device__ __forceinline__ Mom mom_merge(const Mom &a, const Mom &b) {
    if (b.n == 0.0) return a;
    if (a.n == 0.0) return b;
    Mom o;
    o.n = a.n + b.n;
    const double dr = b.mr - a.mr, dh = b.mh - a.mh, w = b.n / o.n, f = a.n * w;
    o.mr = a.mr + dr * w;
    o.mh = a.mh + dh * w;
    o.sxx = a.sxx + b.sxx + dr * dr * f;
    o.sxy = a.sxy + b.sxy + dr * dh * f;
    return o;
}
__global__ void __launch_bounds__(256) segment_fit_kernel(const float4 *moments, const int32_t *seg_off, long long n_seg,
                                                          int J, int group, long long T, uint32_t *coef_seg) {
    const long long wid = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (wid >= n_seg * J) return;
    const long long k = wid / J;
    const int j = (int)(wid - k * J);
    long long t0 = seg_off[k], t1 = seg_off[k + 1];
    t0 = t0 < 0 ? 0 : (t0 > T ? T : t0);
    t1 = t1 < t0 ? t0 : (t1 > T ? T : t1);
    Mom m = {0.0, 0.0, 0.0, 0.0, 0.0};
    for (long long t = t0 + lane; t < t1; t += 32) {
        const float4 s = moments[t * J + j];
        const Mom one = {(double)group, (double)s.x, (double)s.y, (double)s.z, (double)s.w};
        m = mom_merge(m, one);
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {   // lane l absorbs lane l + o: earlier tokens stay on the left
        Mom b;
        b.n = __shfl_down_sync(0xffffffffu, m.n, o);
        b.mr = __shfl_down_sync(0xffffffffu, m.mr, o);
        b.mh = __shfl_down_sync(0xffffffffu, m.mh, o);
        b.sxx = __shfl_down_sync(0xffffffffu, m.sxx, o);
        b.sxy = __shfl_down_sync(0xffffffffu, m.sxy, o);
        if (lane + o < 32) m = mom_merge(m, b);
    }
    if (lane == 0) {
        double a = 0.0, b = m.mh;
        if (m.sxx > 1e-12 && fabs(m.sxy) < 65504.0 * m.sxx) {
            a = m.sxy / m.sxx;
            b = m.mh - a * m.mr;
        }
        a = fmin(fmax(a, -65504.0), 65504.0);
        b = fmin(fmax(b, -65504.0), 65504.0);
        const uint32_t a16 = __half_as_ushort(__double2half(a)), b16 = __half_as_ushort(__double2half(b));
        coef_seg[k * J + j] = a16 | (b16 << 16);
    }
}
// segment of every token: the last k with seg_off[k] <= t (empty segments have equal offsets and are skipped)
__global__ void seg_of_kernel(const int32_t *seg_off, long long n_seg, long long T, int32_t *seg_of) {
    const long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (t >= T) return;
    long long lo = 0, hi = n_seg;   // invariant: seg_off[lo] <= t (seg_off[0] = 0), answer in [lo, hi)
    while (hi - lo > 1) {
        const long long mid = (lo + hi) >> 1;
        if (seg_off[mid] <= t) lo = mid; else hi = mid;
    }
    seg_of[t] = (int32_t)lo;
}

// ------------------------------------------------------------------------------------------------
// reconstruction error of a sender-path run (input of the byte-cost side of calibration, Sec. IV-C)
// ------------------------------------------------------------------------------------------------
constexpr int kErrGrid = 592;     // fixed, so that the summation order does not depend on the device
constexpr int kErrThreads = 256;

// partial[b] = (sum (x - x_hat)^2, sum x^2, max |x - x_hat|) over the 8-element chunks b, b + grid, ...
__global__ void __launch_bounds__(kErrThreads) recon_error_kernel(const uint4 *X, const uint4 *Xh, long long n8,
                                                                  double *partial) {
    double se = 0.0, sx = 0.0;
    float mx = 0.f;
    for (long long i = blockIdx.x * (long long)kErrThreads + threadIdx.x; i < n8; i += (long long)kErrGrid * kErrThreads) {
        const uint4 a = X[i], b = Xh[i];
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int k = 0; k < 4; k++) {
            const float x0 = __uint_as_float(aw[k] << 16), x1 = __uint_as_float(aw[k] & 0xffff0000u);
            const float y0 = __uint_as_float(bw[k] << 16), y1 = __uint_as_float(bw[k] & 0xffff0000u);
            const float d0 = __fsub_rn(x0, y0), d1 = __fsub_rn(x1, y1);   // exact or one rounding: both are bf16
            se += (double)d0 * (double)d0 + (double)d1 * (double)d1;
            sx += (double)x0 * (double)x0 + (double)x1 * (double)x1;
            mx = fmaxf(mx, fmaxf(fabsf(d0), fabsf(d1)));
        }
    }
    __shared__ double s_se[kErrThreads], s_sx[kErrThreads];
    __shared__ float s_mx[kErrThreads];
    s_se[threadIdx.x] = se; s_sx[threadIdx.x] = sx; s_mx[threadIdx.x] = mx;
    __syncthreads();
    for (int o = kErrThreads / 2; o > 0; o >>= 1) {   // fixed tree: the same order on every run
        if (threadIdx.x < o) {
            s_se[threadIdx.x] += s_se[threadIdx.x + o];
            s_sx[threadIdx.x] += s_sx[threadIdx.x + o];
            s_mx[threadIdx.x] = fmaxf(s_mx[threadIdx.x], s_mx[threadIdx.x + o]);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        partial[3 * blockIdx.x + 0] = s_se[0];
        partial[3 * blockIdx.x + 1] = s_sx[0];
        partial[3 * blockIdx.x + 2] = (double)s_mx[0];
    }
}
__global__ void recon_error_finalize_kernel(const double *partial, double *out) {
    double se = 0.0, sx = 0.0, mx = 0.0;
    for (int b = 0; b < kErrGrid; b++) {
        se += partial[3 * b];
        sx += partial[3 * b + 1];
        mx = fmax(mx, partial[3 * b + 2]);
    }
    out[0] = se; out[1] = sx; out[2] = mx;
}

constexpr int kCalibGrid = 128;  // fixed, so that the summation order does not depend on the device

// A subset of the tokens and a second reference buffer (the *_list entry points); all null/0 otherwise.
struct Subset {
    const int32_t *tok_list = nullptr;
    const int32_t *tok_count = nullptr;
    const void *intra_base = nullptr;
    long long intra_rows = 0;
    const uint32_t *coef_seg = nullptr;
    const int32_t *seg_of = nullptr;
};
static int apply_subset(const Subset &sub, CodecParams *p) {
    if ((sub.tok_list == nullptr) != (sub.tok_count == nullptr)) return RAC_EINVAL;
    if (sub.intra_rows < 0 || (sub.intra_rows > 0 && !sub.intra_base)) return RAC_EINVAL;
    if (sub.intra_base && !aligned16(sub.intra_base)) return RAC_EALIGN;
    if (p->ref_rows + sub.intra_rows > 0x7fffffffLL) return RAC_EUNSUPPORTED;
    p->tok_list = sub.tok_list;
    p->tok_count = sub.tok_count;
    p->intra_base = sub.intra_rows > 0 ? static_cast<const uint16_t *>(sub.intra_base) : nullptr;
    p->intra_rows = sub.intra_rows;
    p->coef_ext = sub.coef_seg;
    p->seg_of = sub.seg_of;
    return RAC_OK;
}

// test hook of rac_selftest_bounded_wait: bytes announced beyond what a stage's copies deliver
struct WaitTest {
    uint32_t extra_tx;
};

static int reconstruct_impl(const rac_codec_cfg *cfg, const void *payload, int64_t T, const void *ref_base,
                            int64_t ref_rows, const int32_t *ref_row, const void *gain, const void *bias,
                            const float *step, void *X_hat, uint32_t *dev_status, void *stream,
                            const Subset &sub = Subset(), const WaitTest *wt = nullptr) {
    Geometry g;
    int rc = make_geometry(cfg, &g);
    if (rc != RAC_OK) return rc;
    CodecParams p = {};
    rc = fill_common(g, &p, T, ref_base, ref_rows, ref_row, gain, bias, dev_status);
    if (rc != RAC_OK) return rc;
    rc = apply_subset(sub, &p);
    if (rc != RAC_OK) return rc;
    if ((g.coef_fmt == 1) != (sub.coef_seg != nullptr) || (sub.coef_seg != nullptr) != (sub.seg_of != nullptr)) return RAC_EINVAL;
    if (T == 0) return RAC_OK;
    if (!payload || !X_hat || (!step && g.scale_mode == 0)) return RAC_EINVAL;   // mode 1 reads no table
    if (!aligned16(payload) || !aligned16(X_hat) || (step && !aligned16(step))) return RAC_EALIGN;
    p.payload = const_cast<uint8_t *>(static_cast<const uint8_t *>(payload));
    p.X_hat = static_cast<uint16_t *>(X_hat);
    p.step = step;
    if (wt) p.test_extra_tx = wt->extra_tx;
    return launch_decode(g, p, static_cast<cudaStream_t>(stream));
}

}  // namespace rac

// ------------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------------
using namespace rac;

extern "C" {

const char *rac_version(void) { return "rac-b200 0.1.0 (sm_100a)"; }

const char *rac_strerror(int err) {
    switch (err) {
        case RAC_OK: return "ok";
        case RAC_EINVAL: return "invalid argument";
        case RAC_EALIGN: return "pointer not 16-byte aligned";
        case RAC_ESIZE: return "caller buffer too small";
        case RAC_EUNSUPPORTED: return "unsupported configuration";
        case RAC_ECUDA: return "CUDA runtime error";
    }
    return "unknown error";
}

size_t rac_record_bytes(const rac_codec_cfg *cfg) {
    Geometry g;
    return make_geometry(cfg, &g) == RAC_OK ? (size_t)g.rec : 0;
}

size_t rac_payload_bytes(const rac_codec_cfg *cfg, int64_t T) {
    if (T < 0) return 0;
    return rac_record_bytes(cfg) * (size_t)T;
}

// ---- header of a serialised payload (host only)
static uint32_t header_sum(const unsigned char *h) {
    uint32_t sum = 0;
    for (int i = 0; i < 14; i++) {
        uint32_t w;
        memcpy(&w, h + 4 * i, 4);
        sum += w;
    }
    return sum;
}

int rac_header_write(const rac_codec_cfg *cfg, int64_t T, void *header) {
    const size_t rec = rac_record_bytes(cfg);
    if (!header || rec == 0 || T < 0) return RAC_EINVAL;
    unsigned char h[RAC_HEADER_BYTES];
    memset(h, 0, sizeof h);
    memcpy(h, "RACP", 4);
    const uint16_t version = 1, size = RAC_HEADER_BYTES;
    memcpy(h + 4, &version, 2);
    memcpy(h + 6, &size, 2);
    memcpy(h + 8, &T, 8);
    const int32_t f[9] = {cfg->d, cfg->group, cfg->bits, cfg->topk, cfg->coef_fmt, cfg->scale_mode, cfg->flags,
                          cfg->qgroup, cfg->topk_group};
    memcpy(h + 16, f, sizeof f);
    const uint32_t rec32 = (uint32_t)rec;
    memcpy(h + 52, &rec32, 4);
    const uint32_t sum = header_sum(h);
    memcpy(h + 56, &sum, 4);
    memcpy(header, h, sizeof h);
    return RAC_OK;
}

int rac_header_parse(const void *header, rac_codec_cfg *cfg_out, int64_t *T_out) {
    if (!header || !cfg_out || !T_out) return RAC_EINVAL;
    const unsigned char *h = static_cast<const unsigned char *>(header);
    uint16_t version, size;
    uint32_t rec32, sum, tail;
    int64_t T;
    int32_t f[9];
    memcpy(&version, h + 4, 2);
    memcpy(&size, h + 6, 2);
    memcpy(&T, h + 8, 8);
    memcpy(f, h + 16, sizeof f);
    memcpy(&rec32, h + 52, 4);
    memcpy(&sum, h + 56, 4);
    memcpy(&tail, h + 60, 4);
    if (memcmp(h, "RACP", 4) != 0 || version != 1 || size != RAC_HEADER_BYTES || tail != 0 || sum != header_sum(h)) return RAC_EINVAL;
    rac_codec_cfg cfg;
    cfg.d = f[0]; cfg.group = f[1]; cfg.bits = f[2]; cfg.topk = f[3]; cfg.coef_fmt = f[4]; cfg.scale_mode = f[5];
    cfg.flags = f[6]; cfg.qgroup = f[7]; cfg.topk_group = f[8];
    const size_t rec = rac_record_bytes(&cfg);
    if (rec == 0 || rec != (size_t)rec32 || T < 0) return RAC_EINVAL;
    *cfg_out = cfg;
    *T_out = T;
    return RAC_OK;
}

size_t rac_encode_workspace_bytes(const rac_codec_cfg *cfg, int64_t T) {
    Geometry g;
    if (make_geometry(cfg, &g) != RAC_OK || T < 0) return 0;
    if (g.topk == 0) return 0;
    return (size_t)T * (size_t)(((g.d / 32) * 4 + 15) / 16 * 16);  // one 16-byte padded row of slab maxima per token
}

static bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return na > 0 && nb > 0 && a0 < b0 + nb && b0 < a0 + na;
}

static int encode_impl(const rac_codec_cfg *cfg, const void *X, int64_t T, const void *ref_base, int64_t ref_rows,
                       const int32_t *ref_row, const void *ref_gain, const void *ref_bias, const float *step,
                       const float *inv_step, void *payload, size_t payload_cap, void *X_hat, void *workspace,
                       size_t workspace_bytes, uint32_t *dev_status, void *stream, const Subset &sub = Subset(),
                       const WaitTest *wt = nullptr) {
    Geometry g;
    int rc = make_geometry(cfg, &g);
    if (rc != RAC_OK) return rc;
    CodecParams p = {};
    rc = fill_common(g, &p, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, dev_status);
    if (rc != RAC_OK) return rc;
    rc = apply_subset(sub, &p);
    if (rc != RAC_OK) return rc;
    if ((g.coef_fmt == 1) != (sub.coef_seg != nullptr) || (sub.coef_seg != nullptr) != (sub.seg_of != nullptr)) return RAC_EINVAL;
    if (T == 0) return RAC_OK;
    if (!X || !payload) return RAC_EINVAL;
    if (g.scale_mode == 0 && (!step || !inv_step)) return RAC_EINVAL;   // the static tables; mode 1 reads neither
    if (!aligned16(X) || !aligned16(payload) || (step && !aligned16(step)) || (inv_step && !aligned16(inv_step))) return RAC_EALIGN;
    if (X_hat && !aligned16(X_hat)) return RAC_EALIGN;
    if (payload_cap < (size_t)g.rec * (size_t)T) return RAC_ESIZE;
    if (X_hat && g.topk > 0 && g.scale_mode == 0) {
        // the outlier pass runs after the streaming pass has written x_hat and reads X and the reference rows
        // again: a token's x_hat must not land on X, nor on a reference row that this call still reads.  With
        // identity rows (ref_row == NULL) every token's reference row is the row it writes.
        const size_t out_bytes = (size_t)T * (size_t)g.d * 2;
        if (ranges_overlap(X_hat, out_bytes, X, out_bytes)) return RAC_EUNSUPPORTED;
        if (ref_base && !ref_row && ranges_overlap(X_hat, out_bytes, ref_base, (size_t)ref_rows * (size_t)g.d * 2))
            return RAC_EUNSUPPORTED;
    }
    const size_t need = rac_encode_workspace_bytes(cfg, T);
    if (need > 0) {
        if (!workspace) return RAC_EINVAL;
        if (!aligned16(workspace)) return RAC_EALIGN;
        if (workspace_bytes < need) return RAC_ESIZE;
    }
    p.X = static_cast<const uint16_t *>(X);
    p.payload = static_cast<uint8_t *>(payload);
    p.X_hat = static_cast<uint16_t *>(X_hat);
    p.step = step;
    p.inv_step = inv_step;
    p.tmax = static_cast<float *>(workspace);
    if (wt) p.test_extra_tx = wt->extra_tx;
    return launch_encode(g, p, T, static_cast<cudaStream_t>(stream));
}

int rac_encode(const rac_codec_cfg *cfg, const void *X, int64_t T, const void *ref_base, int64_t ref_rows,
               const int32_t *ref_row, const void *ref_gain, const void *ref_bias, const float *step,
               const float *inv_step, void *payload, size_t payload_cap, void *workspace, size_t workspace_bytes,
               uint32_t *dev_status, void *stream) {
    return encode_impl(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, inv_step, payload, payload_cap,
                       nullptr, workspace, workspace_bytes, dev_status, stream);
}

int rac_encode_reconstruct(const rac_codec_cfg *cfg, const void *X, int64_t T, const void *ref_base, int64_t ref_rows,
                           const int32_t *ref_row, const void *ref_gain, const void *ref_bias, const float *step,
                           const float *inv_step, void *payload, size_t payload_cap, void *X_hat, void *workspace,
                           size_t workspace_bytes, uint32_t *dev_status, void *stream) {
    if (T > 0 && !X_hat) return RAC_EINVAL;
    return encode_impl(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, inv_step, payload, payload_cap,
                       X_hat, workspace, workspace_bytes, dev_status, stream);
}

int rac_selftest_bounded_wait(const rac_codec_cfg *cfg, int32_t which, const void *in, int64_t T, const void *ref_base,
                              int64_t ref_rows, const float *step, const float *inv_step, void *out, size_t out_cap,
                              void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream) {
    if (T < 1 || T > 1024 || !dev_status) return RAC_EINVAL;
    const WaitTest wt = {16u};   // every stage announces 16 bytes that never come
    if (which == 0)
        return encode_impl(cfg, in, T, ref_base, ref_rows, nullptr, nullptr, nullptr, step, inv_step, out, out_cap, nullptr,
                           workspace, workspace_bytes, dev_status, stream, Subset(), &wt);
    if (which == 1) {
        const size_t need = rac_record_bytes(cfg) ? (size_t)T * (size_t)cfg->d * 2 : 0;
        if (need == 0 || out_cap < need) return need == 0 ? RAC_EINVAL : RAC_ESIZE;
        return reconstruct_impl(cfg, in, T, ref_base, ref_rows, nullptr, nullptr, nullptr, step, out, dev_status, stream,
                                Subset(), &wt);
    }
    return RAC_EINVAL;
}

int rac_decode_reconstruct(const rac_codec_cfg *cfg, const void *payload, int64_t T, const void *ref_base,
                           int64_t ref_rows, const int32_t *ref_row, const void *ref_gain, const void *ref_bias,
                           const float *step, void *X_hat, uint32_t *dev_status, void *stream) {
    return reconstruct_impl(cfg, payload, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, X_hat, dev_status, stream);
}

int rac_sender_reconstruct(const rac_codec_cfg *cfg, const void *payload, int64_t T, const void *ref_base,
                           int64_t ref_rows, const int32_t *ref_row, const void *ref_gain, const void *ref_bias,
                           const float *step, void *X_hat, uint32_t *dev_status, void *stream) {
    return reconstruct_impl(cfg, payload, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, X_hat, dev_status, stream);
}

int rac_encode_reconstruct_list(const rac_codec_cfg *cfg, const void *X, int64_t T, const int32_t *tok_list,
                                const int32_t *tok_count, const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                                const void *intra_base, int64_t intra_rows, const uint32_t *coef_seg, const int32_t *seg_of,
                                const void *ref_gain, const void *ref_bias,
                                const float *step, const float *inv_step, void *payload, size_t payload_cap, void *X_hat,
                                void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream) {
    Subset sub;
    sub.tok_list = tok_list;
    sub.tok_count = tok_count;
    sub.intra_base = intra_base;
    sub.intra_rows = intra_rows;
    sub.coef_seg = coef_seg;
    sub.seg_of = seg_of;
    return encode_impl(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, inv_step, payload, payload_cap,
                       X_hat, workspace, workspace_bytes, dev_status, stream, sub);
}

int rac_decode_reconstruct_list(const rac_codec_cfg *cfg, const void *payload, int64_t T, const int32_t *tok_list,
                                const int32_t *tok_count, const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                                const void *intra_base, int64_t intra_rows, const uint32_t *coef_seg, const int32_t *seg_of,
                                const void *ref_gain, const void *ref_bias,
                                const float *step, void *X_hat, uint32_t *dev_status, void *stream) {
    Subset sub;
    sub.tok_list = tok_list;
    sub.tok_count = tok_count;
    sub.intra_base = intra_base;
    sub.intra_rows = intra_rows;
    sub.coef_seg = coef_seg;
    sub.seg_of = seg_of;
    return reconstruct_impl(cfg, payload, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, X_hat, dev_status, stream,
                            sub);
}

int rac_split_waves(const int32_t *ref_row, int64_t T, int64_t first_intra_row, int32_t *wave1, int32_t *wave2,
                    int32_t *wave_count, void *stream) {
    if (T < 0 || first_intra_row < 0 || !wave_count) return RAC_EINVAL;
    if (T >= (1ll << 30)) return RAC_EUNSUPPORTED;
    if (T > 0 && (!ref_row || !wave1 || !wave2)) return RAC_EINVAL;
    split_waves_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(ref_row, (int)T, first_intra_row, wave1, wave2,
                                                                         wave_count);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

size_t rac_fit_segments_workspace_bytes(const rac_codec_cfg *cfg, int64_t T) {
    Geometry g;
    if (make_geometry(cfg, &g) != RAC_OK || T < 0) return 0;
    return ((size_t)T * (size_t)g.J * sizeof(float4) + 15) / 16 * 16 + 16;
}

int rac_fit_segments(const rac_codec_cfg *cfg, const void *X, int64_t T, const void *ref_base, int64_t ref_rows,
                     const int32_t *ref_row, const void *ref_gain, const void *ref_bias, const int32_t *seg_off,
                     int64_t n_seg, uint32_t *coef_seg, int32_t *seg_of, void *workspace, size_t workspace_bytes,
                     uint32_t *dev_status, void *stream) {
    Geometry g;
    int rc = make_geometry(cfg, &g);
    if (rc != RAC_OK) return rc;
    CodecParams p = {};
    rc = fill_common(g, &p, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, dev_status);
    if (rc != RAC_OK) return rc;
    if (n_seg < 0 || n_seg >= (1ll << 30) || T >= (1ll << 31)) return RAC_EUNSUPPORTED;
    if (n_seg == 0) return T == 0 ? RAC_OK : RAC_EINVAL;
    if (!seg_off || !coef_seg || !workspace || (T > 0 && (!X || !seg_of))) return RAC_EINVAL;
    if (!aligned16(X) || !aligned16(workspace)) return RAC_EALIGN;
    if (workspace_bytes < rac_fit_segments_workspace_bytes(cfg, T)) return RAC_ESIZE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p.X = static_cast<const uint16_t *>(X);
    p.moments = static_cast<float4 *>(workspace);
    if (T > 0) {
        p.stages = 2;
        EncSmem L = enc_smem_layout(g.d, p.stages, g.nthreads);
        rc = launch_persistent(calib_kernel<true>, p, g.nthreads, L.total, T, st);
        if (rc != RAC_OK) return rc;
        seg_of_kernel<<<(unsigned)((T + 255) / 256), 256, 0, st>>>(seg_off, n_seg, T, seg_of);
    }
    const long long warps = n_seg * g.J;
    segment_fit_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, st>>>(p.moments, seg_off, n_seg, g.J, g.group, T,
                                                                            coef_seg);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

size_t rac_recon_error_workspace_bytes(void) { return (size_t)kErrGrid * 3 * sizeof(double); }

int rac_recon_error(const void *X, const void *X_hat, int64_t T, int32_t d, double *out, void *workspace,
                    size_t workspace_bytes, void *stream) {
    if (T < 0 || d <= 0 || !out || !workspace) return RAC_EINVAL;
    if (d % 8) return RAC_EUNSUPPORTED;
    if (T > 0 && (!X || !X_hat)) return RAC_EINVAL;
    if (!aligned16(X) || !aligned16(X_hat) || !aligned16(workspace) || (reinterpret_cast<uintptr_t>(out) & 7u)) return RAC_EALIGN;
    if (workspace_bytes < rac_recon_error_workspace_bytes()) return RAC_ESIZE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double *partial = static_cast<double *>(workspace);
    recon_error_kernel<<<kErrGrid, kErrThreads, 0, st>>>(static_cast<const uint4 *>(X), static_cast<const uint4 *>(X_hat),
                                                       (long long)T * d / 8, partial);
    recon_error_finalize_kernel<<<1, 1, 0, st>>>(partial, out);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

size_t rac_calibrate_workspace_bytes(const rac_codec_cfg *cfg) {
    Geometry g;
    if (make_geometry(cfg, &g) != RAC_OK) return 0;
    return (size_t)kCalibGrid * 2 * (size_t)g.d * sizeof(float) + (size_t)kCalibGrid * 2 * sizeof(int);
}

static int calibrate_impl(const rac_codec_cfg *cfg, const void *X, int64_t T, const void *ref_base, int64_t ref_rows,
                          const int32_t *ref_row, const void *ref_gain, const void *ref_bias, const uint32_t *coef_seg,
                          const int32_t *seg_of, float clip_sigmas, float *step, float *inv_step, void *workspace,
                          size_t workspace_bytes, uint32_t *dev_status, void *stream) {
    Geometry g;
    int rc = make_geometry(cfg, &g);
    if (rc != RAC_OK) return rc;
    CodecParams p = {};
    rc = fill_common(g, &p, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, dev_status);
    if (rc != RAC_OK) return rc;
    if (g.scale_mode != 0) return RAC_EUNSUPPORTED;   // the tables belong to the static quantiser only
    if ((g.coef_fmt == 1) != (coef_seg != nullptr) || (coef_seg != nullptr) != (seg_of != nullptr)) return RAC_EINVAL;
    p.coef_ext = coef_seg;
    p.seg_of = seg_of;
    if (!step || !inv_step || !workspace || !(clip_sigmas > 0.f)) return RAC_EINVAL;
    if (T > 0 && !X) return RAC_EINVAL;
    if (!aligned16(X) || !aligned16(workspace) || !aligned16(step) || !aligned16(inv_step)) return RAC_EALIGN;
    if (workspace_bytes < rac_calibrate_workspace_bytes(cfg)) return RAC_ESIZE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    p.X = static_cast<const uint16_t *>(X);
    p.calib_partial = static_cast<float *>(workspace);
    // every CTA of the fixed grid writes its partials, also when it has no token
    {
        p.stages = 2;
        EncSmem L = enc_smem_layout(g.d, p.stages, g.nthreads);
        DeviceInfo di;
        rc = device_info(&di);
        if (rc != RAC_OK) return rc;
        if (L.total > di.max_smem_optin) return RAC_EUNSUPPORTED;
        if (cudaFuncSetAttribute(calib_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, L.total) != cudaSuccess) return RAC_ECUDA;
        calib_kernel<false><<<kCalibGrid, g.nthreads, L.total, st>>>(p);
        if (cudaGetLastError() != cudaSuccess) return RAC_ECUDA;
    }
    int n = 2 * g.d;
    calib_finalize_kernel<<<(n + 255) / 256, 256, 0, st>>>(p.calib_partial, kCalibGrid, g.d, g.bits, clip_sigmas, step, inv_step);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

int rac_calibrate_steps(const rac_codec_cfg *cfg, const void *X, int64_t T, const void *ref_base, int64_t ref_rows,
                        const int32_t *ref_row, const void *ref_gain, const void *ref_bias, float clip_sigmas,
                        float *step, float *inv_step, void *workspace, size_t workspace_bytes, uint32_t *dev_status,
                        void *stream) {
    return calibrate_impl(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, nullptr, nullptr, clip_sigmas, step,
                          inv_step, workspace, workspace_bytes, dev_status, stream);
}

int rac_calibrate_steps_shared(const rac_codec_cfg *cfg, const void *X, int64_t T, const void *ref_base, int64_t ref_rows,
                               const int32_t *ref_row, const void *ref_gain, const void *ref_bias,
                               const uint32_t *coef_seg, const int32_t *seg_of, float clip_sigmas, float *step,
                               float *inv_step, void *workspace, size_t workspace_bytes, uint32_t *dev_status,
                               void *stream) {
    if (!coef_seg || !seg_of) return RAC_EINVAL;
    return calibrate_impl(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, coef_seg, seg_of, clip_sigmas, step,
                          inv_step, workspace, workspace_bytes, dev_status, stream);
}

}  // extern "C"
