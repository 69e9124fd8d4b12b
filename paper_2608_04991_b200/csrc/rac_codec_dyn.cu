// RAC codec kernels for sm_100a, the quantiser family of Sec. IV-C as printed (scale_mode 1):
//   * Eq. 8: per quantisation group the scale s = RoundUp_binary16(max|E^d| / Qmax) travels in the record, an
//     all-zero group carries scale 0 ("zero marker") and skips the division, nothing clips;
//   * the quantisation group g_q may differ from the alignment group g_a; g_q = d is the decode mode of the
//     paper (one scale per token);
//   * code widths 2, 3, 4 and 8;
//   * the outlier mask of "Outlier Metadata": the k_g largest |e| of every quantisation group leave the dense
//     base (E^d = E - O) BEFORE the scale is taken, and travel as one-byte in-group offsets (ascending) plus
//     binary16 values.
//
// Same streaming shape as the static-table kernels: persistent CTAs, a token per CTA iteration, a thread per 32
// channels, rows in and records out as 1-D bulk copies, bounded mbarrier waits, no CTA barrier in the loop; the
// finished record is handed over by a rotating duty warp.  Because the outliers are picked per GROUP, the
// selection fits into the streaming pass: a group is 1 to 8 lanes of one warp, so k_g rounds of "largest
// magnitude of the group, lowest channel among equals" need only warp shuffles.  The token-wide scale is the
// one place where warps must meet: they exchange their maxima through shared memory and a third mbarrier.
#include <type_traits>

#include "rac_codec_dev.cuh"

namespace rac {

struct DynCtrl {
    unsigned long long full[kMaxStages];    // data of the stage has landed
    unsigned long long done[kMaxStages];    // every warp has finished its share of the token in the stage
    unsigned long long tokmax[kMaxStages];  // every warp has published its largest |e| of the token
    int row[kMaxStages];
    int seg[kMaxStages];                    // segment of the token in each stage (shared coefficients only)
    int abort;
    float wmax[kMaxStages][8];
};

struct DynSmem {
    int stage0, stage_bytes, rec_off, total;
};
__host__ __device__ inline DynSmem dyn_smem_layout(int d, int rec, int stages) {
    DynSmem s;
    s.stage0 = align_up((int)sizeof(DynCtrl), 128);
    s.rec_off = 4 * d;  // after X row + R row: two record slots, used alternately (by the stage's parity)
    s.stage_bytes = align_up(s.rec_off + 2 * rec, 128);
    s.total = s.stage0 + stages * s.stage_bytes;
    return s;
}

__device__ __forceinline__ uint32_t rotl32(uint32_t v, int n) { return __funnelshift_l(v, v, n); }
__device__ __forceinline__ uint32_t rotr32(uint32_t v, int n) { return __funnelshift_r(v, v, n); }

// largest magnitude of 8 values, leaving out those whose bit is set in `skip` (three-input maxima)
__device__ __forceinline__ float abs_max8(const float (&e)[8], uint32_t skip) {
    float v[8];
#pragma unroll
    for (int k = 0; k < 8; k++) v[k] = ((skip >> k) & 1u) ? 0.f : fabsf(e[k]);
    float m0 = 0.f, m1 = 0.f;
    asm("max.f32 %0, %0, %1, %2;" : "+f"(m0) : "f"(v[0]), "f"(v[1]));
    asm("max.f32 %0, %0, %1, %2;" : "+f"(m1) : "f"(v[2]), "f"(v[3]));
    asm("max.f32 %0, %0, %1, %2;" : "+f"(m0) : "f"(v[4]), "f"(v[5]));
    asm("max.f32 %0, %0, %1, %2;" : "+f"(m1) : "f"(v[6]), "f"(v[7]));
    return fmaxf(m0, m1);
}
// rotate the four entries right by rot (new[j] = old[(j - rot) & 3])
__device__ __forceinline__ void rot_right4f(float (&w)[4], int rot) {
    if (rot & 1) { float t = w[3]; w[3] = w[2]; w[2] = w[1]; w[1] = w[0]; w[0] = t; }
    if (rot & 2) { float t = w[0]; w[0] = w[2]; w[2] = t; t = w[1]; w[1] = w[3]; w[3] = t; }
}

// codes of the 8 channels of one slot -> BITS bytes (one word, or two for 8-bit codes)
template <int BITS>
__device__ __forceinline__ void pack_slot(const uint32_t (&t)[8], uint32_t &w0, uint32_t &w1) {
    // t[i]: binary32 bit pattern of (code + 1.5*2^23): the low mantissa bits hold the code in two's complement
    if constexpr (BITS == 8) {
        w0 = __byte_perm(__byte_perm(t[0], t[1], 0x0040), __byte_perm(t[2], t[3], 0x0040), 0x5410);
        w1 = __byte_perm(__byte_perm(t[4], t[5], 0x0040), __byte_perm(t[6], t[7], 0x0040), 0x5410);
    } else {
        w0 = pack8<BITS>(t);
        w1 = 0;
    }
}

// MINB = 4 caps registers at 96 so that four 160-thread CTAs (d = 5120) fit on an SM.
// KG: rounds compiled in (0, 1, 2, 4 or 8; p.kg <= KG is the number taken).
// G, D: lanes per group (alignment and quantisation group alike) and the hidden width as compile-time constants, or 0
// to read them from the parameters; with them the reductions lose their uniform branches and the address arithmetic
// of rows and stages folds.
// QT (with G): the quantisation group is the whole token (one scale per token) instead of the alignment group.
template <int BITS, bool XHAT, int KG, int MINB, bool SUB, int G = 0, int D = 0, bool QT = false>
__global__ void __launch_bounds__(MINB == 4 ? 160 : 256, MINB) encode_dyn_kernel(const CodecParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nwarps = D ? (D / 32 + 31) / 32 : nt >> 5;
    const int rot = (lane >> 1) & 3;
    const int d = D ? D : p.d;
    constexpr int kGShift = G == 32 ? 5 : G == 16 ? 4 : G == 8 ? 3 : G == 4 ? 2 : G == 2 ? 1 : 0;
    const int lpg = G ? G : p.lpg, lpg_shift = G ? kGShift : p.lpg_shift;
    const int lpq = G ? (QT ? 0 : G) : p.lpq, lpq_shift = G ? (QT ? 0 : kGShift) : p.lpq_shift;
    const bool valid = tid * 32 < d;
    const bool qtok = lpq == 0;
    const int S = D ? 2 : p.stages;   // the host sets two stages
    // with the width, the groups and (for up to two outliers per group, where the launcher compiles in the exact count)
    // the outlier count known, the record geometry is a constant: coefficient words, scales, codes, offsets, values
    constexpr bool kGeo = G != 0 && D != 0 && !SUB && KG <= 2;
    constexpr int kJ = kGeo ? D / (32 * (G ? G : 1)) : 0, kJq = QT ? 1 : kJ;   // QT: one scale per token (and KG = 0)
    constexpr int kScaleOff = 4 * kJ, kCodesOff = kScaleOff + (2 * kJq + 3) / 4 * 4, kGoffOff = kCodesOff + D * BITS / 8;
    constexpr int kGvalOff = kGoffOff + (kJq * KG + 1) / 2 * 2, kRec = (kGvalOff + 2 * kJq * KG + 15) / 16 * 16;
    const int recb = kGeo ? kRec : p.rec, kgc = kGeo ? KG : p.kg;
    const int scale_off = kGeo ? kScaleOff : p.scale_off, codes_off = kGeo ? kCodesOff : p.codes_off;
    const int goff_off = kGeo ? kGoffOff : p.goff_off, gval_off = kGeo ? kGvalOff : p.gval_off;
    const DynSmem L = dyn_smem_layout(d, recb, S);
    DynCtrl *ctrl = reinterpret_cast<DynCtrl *>(smem);
    const uint32_t sbase = smem_u32(smem);
    constexpr float qmax = (float)((1 << (BITS - 1)) - 1);
    constexpr int WPT = BITS;  // code words per thread (32 channels)
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
            mbar_init(smem_u32(&ctrl->tokmax[s]), nwarps);
        }
        ctrl->abort = 0;
        mbar_init_fence();
    }
    // padding bytes of the record slots are zero from here on: every field is rewritten per token, the gaps never
    for (int s = 0; s < S; s++)
        for (int o = 4 * tid; o < 2 * recb; o += 4 * nt)
            *reinterpret_cast<uint32_t *>(smem + L.stage0 + s * L.stage_bytes + L.rec_off + o) = 0u;
    __syncthreads();
    if (tid == 0)
        for (int k = 0; k < S && k < n_my; k++) issue(k, k, raw_row_of(k));

    uint32_t off[4];
#pragma unroll
    for (int j = 0; j < 4; j++) off[j] = (uint32_t)(tid * 64 + ((j + rot) & 3) * 16);
    const unsigned int group_mask = __ballot_sync(0xffffffffu, valid);
    const u64 magic2 = pack2(kMagic, kMagic);
    const int qbase = lane & ~(lpq - 1);              // first lane of this lane's quantisation group (lpq > 0)
    const uint32_t qlanes = lpq >= 32 ? 0xffffffffu : ((1u << lpq) - 1u);
    // quantisation group of this thread (qgen: groups of any whole number of lanes, which may cross warps)
    const int jq = qtok ? (p.qgen ? tid / p.qgen : 0) : (tid >> lpq_shift);

    int stage = 0, duty = 0;
    uint32_t parity = 0;
    bool timed_out = false;
    for (int it = 0; it < n_my; it++) {
        if (*reinterpret_cast<volatile int *>(&ctrl->abort)) break;
        unsigned char *stg = smem + L.stage0 + stage * L.stage_bytes;
        const uint32_t xs = sbase + L.stage0 + stage * L.stage_bytes;
        const uint32_t rs = xs + row_bytes;
        unsigned char *rec = stg + L.rec_off + parity * recb;
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_u32(&ctrl->full[stage]), parity))) { timed_out = true; break; }
        const bool has_ref = ctrl->row[stage] >= 0;

        u64 e2[16];        // Eq. 7 residual of this thread's channels, packed pairs in slot order
        u64 r2[16];        // aligned-reference inputs, kept for the sender-side reconstruction
        u64 a2 = 0ull, b2 = 0ull;
        uint32_t sel[KG > 4 ? 8 : 4] = {};   // per round: in-group offset | binary16 value << 16 (same in every lane of the group)
        uint32_t own = 0;                      // rounds whose outlier lives in this thread
        float m = 0.f;
        if (valid) {
            u64 x2[16];
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
            bool shared = false;
            if constexpr (SUB) shared = p.coef_ext != nullptr;
            if (shared) {
                // Eq. 6 was solved over all positions of the token's segment beforehand: the words come from outside
                const uint32_t cw = p.coef_ext[(long long)ctrl->seg[stage] * p.J + (tid >> lpg_shift)];
                const float a = half_bits_to_float(cw & 0xffffu), b = half_bits_to_float(cw >> 16);
                a2 = pack2(a, a);
                b2 = pack2(b, b);
            } else {
                uint32_t coef_word;
                fit_group(x2, r2, has_ref, lpg, p.inv_group, group_mask, p.status, a2, b2, &coef_word);
                if ((lane & (lpg - 1)) == 0) reinterpret_cast<uint32_t *>(rec)[tid >> lpg_shift] = coef_word;
            }
            // residual, and the largest magnitude of each slot of 8 channels
            float sm[4];
#pragma unroll
            for (int j = 0; j < 4; j++) {
                float ev[8];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    e2[4 * j + i] = psub(x2[4 * j + i], pfma(a2, r2[4 * j + i], b2));
                    unpack2(e2[4 * j + i], ev[2 * i], ev[2 * i + 1]);
                }
                sm[j] = abs_max8(ev, 0u);
            }

            // ---- outlier mask: k_g rounds of (largest |e| of the group, lowest channel among equals).  The
            // registers are left alone: what a round needs again is read from the rows in shared memory and formed by
            // the same operations (same bits).  Codes and x_hat of the outliers are patched after the dense pass.
            // Groups of four lanes and more that share one coefficient pair (the usual case) work on a round together:
            // group maximum by shuffles, one ballot for the lowest lane that holds it, that lane names its lowest piece
            // (8 channels) with that maximum and what was taken from it before; four lanes of the group then form one
            // pair of that piece's residuals each, two ballots give the lowest channel that equals the maximum and was
            // not taken, its value comes from the lane that formed it, and the largest of the rest is the piece's new
            // maximum.  Nothing diverges.  Smaller groups (or quantisation groups that span alignment groups) keep the
            // older form: every lane finds ITS candidate beforehand (off the critical path), a round is the group
            // maximum, one ballot, the winner handing out its candidate and looking for its next one.
            if (KG) {
                uint32_t taken = 0;  // channel order within the slab
                if (lpq >= 4 && lpg >= lpq) {
                    const int pi = (lane - qbase) & 3;   // this lane's pair of the piece; with more than four lanes the upper ones repeat the lower four
#pragma unroll
                    for (int n = 0; n < KG; n++) {
                        if (KG <= 2 || n < p.kg) {
                            const float mloc = fmaxf(fmaxf(sm[0], sm[1]), fmaxf(sm[2], sm[3]));
                            float sp[4] = {sm[0], sm[1], sm[2], sm[3]};
                            rot_right4f(sp, rot);
                            const int q = sp[0] == mloc ? 0 : sp[1] == mloc ? 1 : sp[2] == mloc ? 2 : 3;
                            float gm = mloc;
#pragma unroll
                            for (int o = 1; o < 32; o <<= 1)
                                if (lpq > o) gm = fmaxf(gm, __shfl_xor_sync(group_mask, gm, o));
                            const uint32_t gb = (__ballot_sync(group_mask, mloc == gm) >> qbase) & qlanes;
                            const int owner = qbase + (gb ? __ffs(gb) - 1 : 0);
                            const uint32_t info = __shfl_sync(group_mask, (uint32_t)(tid * 64 + q * 16) | (((taken >> (8 * q)) & 0xffu) << 20), owner);
                            const uint32_t wpa = info & 0xfffffu, wtq = info >> 20;
                            const uint32_t ad = wpa + 4u * (uint32_t)pi;
                            u64 rr = 0ull;
                            if (has_ref) rr = load_ref_pair(rs + ad, p.gain, p.bias, (int)(ad >> 1));
                            float e0, e1;
                            unpack2(psub(bf16x2_to_p(lds32(xs + ad)), pfma(a2, rr, b2)), e0, e1);
                            const uint32_t mybits = (((fabsf(e0) == gm ? 1u : 0u) | (fabsf(e1) == gm ? 2u : 0u)) << (2 * pi)) & ~wtq;
                            // the four lanes that hold the piece sit at qbase..qbase+3 of the group
                            const uint32_t b0 = __ballot_sync(group_mask, mybits & (1u << (2 * pi)));
                            const uint32_t b1 = __ballot_sync(group_mask, mybits & (2u << (2 * pi)));
                            const uint32_t g0 = (b0 >> qbase) & 0xfu, g1 = (b1 >> qbase) & 0xfu;
                            // channel 2*l is bit l of g0, channel 2*l+1 bit l of g1: the lowest channel that is set
                            const int k0 = g0 ? 2 * (__ffs(g0) - 1) : 8, k1 = g1 ? 2 * (__ffs(g1) - 1) + 1 : 8;
                            const int k = min(k0, k1) & 7;   // 8 (nothing set: only with NaNs around) -> 0
                            const int kp = k >> 1;
                            const uint32_t gone = (wtq | (1u << k)) >> (2 * pi);
                            const float mine = (k & 1) ? e1 : e0;
                            float rest = fmaxf((gone & 1u) ? 0.f : fabsf(e0), (gone & 2u) ? 0.f : fabsf(e1));
                            const float val = __shfl_sync(group_mask, mine, qbase + kp);
                            rest = fmaxf(rest, __shfl_xor_sync(group_mask, rest, 1));
                            rest = fmaxf(rest, __shfl_xor_sync(group_mask, rest, 2));
                            const int wq = (int)(wpa >> 4) & 3;
                            sel[n] = (uint32_t)((owner - qbase) * 32 + 8 * wq + k) | (float_to_half_bits_sat(val) << 16);
                            if (lane == owner) {
                                own |= 1u << n;
                                taken |= 1u << (8 * wq + k);
                                const int js = (wq - rot) & 3;
#pragma unroll
                                for (int j = 0; j < 4; j++) sm[j] = (j == js) ? rest : sm[j];
                            }
                        }
                    }
                } else {
                    float mloc, cval, cnm;
                    int cq, ck;
                    auto find = [&]() {
                        mloc = fmaxf(fmaxf(sm[0], sm[1]), fmaxf(sm[2], sm[3]));
                        // lowest piece whose maximum is the lane's maximum; piece q sits in slot (q - rot) & 3
                        float sp[4] = {sm[0], sm[1], sm[2], sm[3]};
                        rot_right4f(sp, rot);
                        const int q = sp[0] == mloc ? 0 : sp[1] == mloc ? 1 : sp[2] == mloc ? 2 : 3;
                        const uint32_t pa = (uint32_t)(tid * 64 + q * 16);
                        const uint4 xw = lds128(xs + pa);
                        const uint32_t xws[4] = {xw.x, xw.y, xw.z, xw.w};
                        u64 rr[4] = {0ull, 0ull, 0ull, 0ull};
                        if (has_ref) load_ref_slot(rs + pa, p.gain, p.bias, (int)(pa >> 1), rr);
                        float ev[8];
#pragma unroll
                        for (int i = 0; i < 4; i++) unpack2(psub(bf16x2_to_p(xws[i]), pfma(a2, rr[i], b2)), ev[2 * i], ev[2 * i + 1]);
                        uint32_t tq = (taken >> (8 * q)) & 0xffu;
                        uint32_t eq = 0;
#pragma unroll
                        for (int k = 0; k < 8; k++) eq |= (fabsf(ev[k]) == mloc) ? (1u << k) : 0u;
                        eq &= ~tq;
                        const int k = eq ? __ffs(eq) - 1 : 0;   // eq == 0 only with NaNs around
                        float val = ev[0];
#pragma unroll
                        for (int kk = 1; kk < 8; kk++) val = (kk == k) ? ev[kk] : val;
                        cnm = abs_max8(ev, tq | (1u << k));     // E^d = E - O for this slot's maximum
                        cq = q;
                        ck = k;
                        cval = val;
                    };
                    find();
#pragma unroll
                    for (int n = 0; n < KG; n++) {
                        if (KG <= 2 || n < p.kg) {   // the launcher compiles in exactly k_g rounds for k_g = 1, 2
                            float gm = mloc;
#pragma unroll
                            for (int o = 1; o < 32; o <<= 1)
                                if (lpq > o) gm = fmaxf(gm, __shfl_xor_sync(group_mask, gm, o));
                            const uint32_t gb = (__ballot_sync(group_mask, mloc == gm) >> qbase) & qlanes;
                            const int owner = qbase + (gb ? __ffs(gb) - 1 : 0);   // gb == 0 only with NaNs around
                            uint32_t word = 0;
                            if (lane == owner) {
                                word = (uint32_t)((lane - qbase) * 32 + 8 * cq + ck) | (float_to_half_bits_sat(cval) << 16);
                                own |= 1u << n;
                                taken |= 1u << (8 * cq + ck);
                                const int js = (cq - rot) & 3;
#pragma unroll
                                for (int j = 0; j < 4; j++) sm[j] = (j == js) ? cnm : sm[j];
                                if (KG <= 2 ? n + 1 < KG : n + 1 < p.kg) find();
                            }
                            sel[n] = __shfl_sync(group_mask, word, owner);
                        }
                    }
}
                if ((lane & (lpq - 1)) == 0) {
                    // the group's first lane serialises them in ascending offset order
                    const bool wide = lpq > 8;   // more than 256 channels per group: two-byte offsets
                    unsigned char *go = rec + goff_off + jq * kgc;
                    unsigned short *go2 = reinterpret_cast<unsigned short *>(rec + goff_off) + jq * kgc;
                    unsigned short *gv = reinterpret_cast<unsigned short *>(rec + gval_off) + jq * kgc;
#pragma unroll
                    for (int n = 0; n < KG; n++) {
                        if (KG <= 2 || n < p.kg) {
                            int rank = 0;
#pragma unroll
                            for (int q = 0; q < KG; q++)
                                if ((KG <= 2 || q < p.kg) && (sel[q] & 0xffffu) < (sel[n] & 0xffffu)) rank++;
                            if (wide) go2[rank] = (unsigned short)(sel[n] & 0xffffu);
                            else go[rank] = (unsigned char)(sel[n] & 0xffu);
                            gv[rank] = (unsigned short)(sel[n] >> 16);
                        }
                    }
                }
            }
            // ---- largest dense magnitude of this thread, then of its group
            m = fmaxf(fmaxf(sm[0], sm[1]), fmaxf(sm[2], sm[3]));
            if (!qtok) {
#pragma unroll
                for (int o = 1; o < 32; o <<= 1)
                    if (lpq > o) m = fmaxf(m, __shfl_xor_sync(group_mask, m, o));
            }
        }
        if (qtok && p.qgen) {
            // groups of any whole number of lanes: every thread leaves its maximum in the first word of its own slab of
            // the reference row (read long ago, not needed again), the warps meet once, and every thread takes the
            // largest of its group's entries
            float *mine = reinterpret_cast<float *>(stg + row_bytes + 64 * tid);
            if (valid) *mine = m;
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&ctrl->tokmax[stage])) : "memory");
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_u32(&ctrl->tokmax[stage]), parity))) { timed_out = true; break; }
            if (valid) {
                const int l0 = jq * p.qgen;
                for (int l = 0; l < p.qgen; l++)
                    m = fmaxf(m, *reinterpret_cast<volatile float *>(stg + row_bytes + 64 * (l0 + l)));
            }
        } else if (qtok) {
            // one scale per token: the warps meet once
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            if (lane == 0) {
                ctrl->wmax[stage][warp] = m;
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&ctrl->tokmax[stage])) : "memory");
            }
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_u32(&ctrl->tokmax[stage]), parity))) { timed_out = true; break; }
            for (int w = 0; w < nwarps; w++) m = fmaxf(m, *reinterpret_cast<volatile float *>(&ctrl->wmax[stage][w]));
        }

        if (valid) {
            // ---- Eq. 8: s = RoundUp_binary16(m / Qmax): round to nearest, then one step up if that fell short
            const float s_star = __fdiv_rn(m, qmax);
            uint32_t s16 = float_to_half_bits_sat(s_star);
            if (half_bits_to_float(s16) < s_star && s16 < 0x7bffu) s16++;
            const float sc = half_bits_to_float(s16);
            const float isc = sc != 0.f ? __fdiv_rn(1.0f, sc) : 0.f;   // zero marker: no division, codes 0
            const u64 inv2 = pack2(isc, isc), s2 = pack2(sc, sc);
            if (qtok ? tid == jq * p.qgen : (lane & (lpq - 1)) == 0)
                reinterpret_cast<unsigned short *>(rec + scale_off)[jq] = (unsigned short)s16;

            // No dense value can leave [-Qmax, Qmax] (Eq. 11): s >= max|E^d| / Qmax by the round-up, and the two
            // binary32 roundings of e * (1/s) add a few 2^-24 relative, far from the next half.  The exception is a
            // scale that binary16 cannot hold (s stuck at 65504): then, and only then, the clamp does something.
            // The channels of the outlier mask do exceed the range; their codes and x_hat are replaced below, and
            // the packing keeps only the low bits of every field.  The magic add is written as v*1 + magic so that
            // it stays a second rounding after the product (a plain add could be merged with the multiply).
            const bool clamp = __any_sync(group_mask, s16 >= 0x7bffu);
            const u64 one2 = pack2(1.0f, 1.0f);
            uint32_t words[4][2];
            auto quantise = [&](auto clamp_tag) {
                constexpr bool CLAMP = decltype(clamp_tag)::value;
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    uint32_t t8[8], xh[4];
#pragma unroll
                    for (int i = 0; i < 4; i++) {
                        u64 vv = pmul(e2[4 * j + i], inv2);
                        if (CLAMP) {
                            float v0, v1;
                            unpack2(vv, v0, v1);
                            vv = pack2(fminf(fmaxf(v0, -qmax), qmax), fminf(fmaxf(v1, -qmax), qmax));
                        }
                        const u64 tt = pfma(vv, one2, magic2);
                        float t0, t1;
                        unpack2(tt, t0, t1);
                        t8[2 * i] = __float_as_uint(t0);
                        t8[2 * i + 1] = __float_as_uint(t1);
                        if (XHAT) {
                            // Eq. 9 with the code just chosen: x_hat = bf16((alpha*r + beta) + q*s)
                            float x0, x1;
                            unpack2(pfma(psub(tt, magic2), s2, pfma(a2, r2[4 * j + i], b2)), x0, x1);
                            xh[i] = f2_to_bf16x2(x0, x1);
                        }
                    }
                    pack_slot<BITS>(t8, words[j][0], words[j][1]);
                    if (XHAT) sts128(xs + off[j], make_uint4(xh[0], xh[1], xh[2], xh[3]));
                }
            };
            if (clamp) quantise(std::true_type{});
            else quantise(std::false_type{});
            // slot order -> piece order (words[q] becomes the code word(s) of piece q)
            {
                uint32_t lo[4] = {words[0][0], words[1][0], words[2][0], words[3][0]};
                rot_right4(lo, rot);
                uint32_t *cw = reinterpret_cast<uint32_t *>(rec + codes_off) + tid * WPT;
                if (BITS == 8) {
                    uint32_t hi[4] = {words[0][1], words[1][1], words[2][1], words[3][1]};
                    rot_right4(hi, rot);
#pragma unroll
                    for (int q = 0; q < 4; q++) { cw[2 * q] = lo[q]; cw[2 * q + 1] = hi[q]; }
                } else if (BITS == 4) {
                    cw[0] = lo[0]; cw[1] = lo[1]; cw[2] = lo[2]; cw[3] = lo[3];
                } else if (BITS == 3) {
                    cw[0] = lo[0] | (lo[1] << 24);
                    cw[1] = (lo[1] >> 8) | (lo[2] << 16);
                    cw[2] = (lo[2] >> 16) | (lo[3] << 8);
                } else {
                    cw[0] = lo[0] | (lo[1] << 16);
                    cw[1] = lo[2] | (lo[3] << 16);
                }
            }
            if (KG && own) {
                // the outliers this thread owns: dense code 0 (E^d = E - O), and on the sender side
                // x_hat = bf16((alpha*r + beta) + binary16 value)
                float a, b, unused;
                unpack2(a2, a, unused);
                unpack2(b2, b, unused);
                uint32_t *cw = reinterpret_cast<uint32_t *>(rec + codes_off) + tid * WPT;
#pragma unroll
                for (int n = 0; n < KG; n++) {
                    if ((own >> n) & 1u) {
                        const int c = jq * (lpq * 32) + (int)(sel[n] & 0xffffu);
                        const int bp = (c & 31) * BITS, w = bp >> 5, sh = bp & 31;
                        const unsigned long long mk = (unsigned long long)((1u << BITS) - 1u) << sh;
                        cw[w] &= ~(uint32_t)mk;
                        if (BITS == 3 && sh > 29) cw[w + 1] &= ~(uint32_t)(mk >> 32);
                        if (XHAT) {
                            float r = 0.f;
                            if (has_ref) {
                                r = __uint_as_float((uint32_t)(*reinterpret_cast<const unsigned short *>(stg + row_bytes + 2 * c)) << 16);
                                if (p.gain) r = bf16_round(__fmaf_rn(half_bits_to_float(p.gain[c]), r, half_bits_to_float(p.bias[c])));
                            }
                            const float x = __fadd_rn(__fmaf_rn(a, r, b), half_bits_to_float(sel[n] >> 16));
                            reinterpret_cast<unsigned short *>(stg)[c] = __bfloat16_as_ushort(__float2bfloat16_rn(x));
                        }
                    }
                }
            }
        }
        // this warp's share of the token is in shared memory: one arrival per warp
        fence_async_smem();
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&ctrl->done[stage])) : "memory");

        if (warp == duty) {
            const int k_next = it + S;
            int raw_next = 0;
            if (lane == 0 && k_next < n_my) raw_next = raw_row_of(k_next);
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_u32(&ctrl->done[stage]), parity))) { timed_out = true; break; }
            // The record sits in the slot of the stage's current parity; the stage's next token writes the other
            // slot, and the one after that cannot start before this warp has arrived for the token in between.
            // With x_hat the X row itself is the source of a store and must have been read before the refill.
            if (lane == 0) {
                const long long t = token_at<SUB>(p, first + (long long)it * stride);
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
    if (lane == 0) bulk_wait_all();
    if (tid == 0 && *reinterpret_cast<volatile int *>(&ctrl->abort)) {
        for (int s = 0; s < S; s++) {
            mbar_wait_bounded(smem_u32(&ctrl->full[s]), 0);
            mbar_wait_bounded(smem_u32(&ctrl->full[s]), 1);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// reconstruct (receiver and sender), Eq. 9 with the record's own scales
// ------------------------------------------------------------------------------------------------
// Same shape as the static-table reconstruction: record and reference row arrive in a stage, every thread
// dequantises its 32 channels (code -> binary32 through the 2^23 trick, times its group's scale), adds the
// aligned reference, rounds to bf16 into an output row in shared memory; then the per-group outliers replace
// what the dense pass wrote, and the row leaves as one bulk store.
// G, D: as for the encoder (lanes per group and hidden width compiled in, or 0)
template <int BITS, bool KG, bool SUB, int G = 0, int D = 0>
__global__ void __launch_bounds__(256) decode_dyn_kernel(const CodecParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int rot = (lane >> 1) & 3;
    const int d = D ? D : p.d;
    constexpr int kGShift = G == 32 ? 5 : G == 16 ? 4 : G == 8 ? 3 : G == 4 ? 2 : G == 2 ? 1 : 0;
    const int lpg_shift = G ? kGShift : p.lpg_shift;
    const int lpq = G ? G : p.lpq, lpq_shift = G ? kGShift : p.lpq_shift;
    const bool valid = tid * 32 < d;
    const int S = D ? 2 : p.stages;   // the host sets two stages
    const DecSmem L = dec_smem_layout(d, p.rec, S);
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem);
    const uint32_t sbase = smem_u32(smem);
    constexpr int WPT = BITS;                     // code words per thread
    constexpr int WPP = BITS == 8 ? 2 : 1;        // code words per piece of 8 channels
    constexpr int FPW = 8 / WPP;                  // fields per word
    constexpr uint32_t cmask = (BITS == 8) ? 0xffu : ((1u << BITS) - 1u);
    constexpr uint32_t H = 1u << (BITS - 1);
    constexpr uint32_t ones = (BITS == 8) ? 0x01010101u : (BITS == 4) ? 0x11111111u : (BITS == 3) ? 0x00249249u : 0x00005555u;
    constexpr uint32_t highs = ones << (BITS - 1);
    constexpr float kBase = 8388608.0f + (float)H;  // 2^23 + H
    const uint32_t row_bytes = 2u * (uint32_t)d;
    const int jq = lpq == 0 ? (p.qgen ? tid / p.qgen : 0) : (tid >> lpq_shift);

    if (tid == 0) {
        for (int s = 0; s < S; s++) mbar_init(smem_u32(&ctrl->bar[s]), 1);
        mbar_init_fence();
    }
    __syncthreads();

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
            bool shared = false;
            if constexpr (SUB) shared = p.coef_ext != nullptr;
            if (shared) cf = p.coef_ext[(long long)ctrl->seg[stage] * p.J + (tid >> lpg_shift)];
            else cf = reinterpret_cast<const uint32_t *>(rec)[tid >> lpg_shift];
            const float a = half_bits_to_float(cf & 0xffff), b = half_bits_to_float(cf >> 16);
            const u64 a2 = pack2(a, a), b2 = pack2(b, b);
            const float sc = half_bits_to_float(reinterpret_cast<const unsigned short *>(rec + p.scale_off)[jq]);
            const u64 s2 = pack2(sc, sc);
            // code words of the four pieces, in piece order, then rotated into slot order
            const uint32_t *cw = reinterpret_cast<const uint32_t *>(rec + p.codes_off) + tid * WPT;
            uint32_t lo[4], hi[4] = {0u, 0u, 0u, 0u};
            if (BITS == 8) {
#pragma unroll
                for (int q = 0; q < 4; q++) { lo[q] = cw[2 * q]; hi[q] = cw[2 * q + 1]; }
            } else if (BITS == 4) {
                lo[0] = cw[0]; lo[1] = cw[1]; lo[2] = cw[2]; lo[3] = cw[3];
            } else if (BITS == 3) {
                uint32_t w0 = cw[0], w1 = cw[1], w2 = cw[2];
                lo[0] = w0 & 0xffffffu;
                lo[1] = (w0 >> 24) | ((w1 & 0xffffu) << 8);
                lo[2] = (w1 >> 16) | ((w2 & 0xffu) << 16);
                lo[3] = w2 >> 8;
            } else {
                uint32_t w0 = cw[0], w1 = cw[1];
                lo[0] = w0 & 0xffffu; lo[1] = w0 >> 16; lo[2] = w1 & 0xffffu; lo[3] = w1 >> 16;
            }
            uint32_t reserved = 0;
#pragma unroll
            for (int q = 0; q < 4; q++) {
                uint32_t v = lo[q] ^ highs;  // field == 0  <=>  code == -2^(BITS-1)
                reserved |= (v - ones) & ~v & highs;
                lo[q] = v;                   // fields now hold code + H (offset binary)
                if (BITS == 8) {
                    v = hi[q] ^ highs;
                    reserved |= (v - ones) & ~v & highs;
                    hi[q] = v;
                }
            }
            if (reserved && p.status) atomicOr(p.status, RAC_STATUS_RESERVED_CODE);
            rot_left4(lo, rot);
            if (BITS == 8) rot_left4(hi, rot);
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const int c = (int)(off[j] >> 1);
                u64 r2[4];
                if (has_ref) {
                    load_ref_slot(rs + off[j], p.gain, p.bias, c, r2);
                } else {
#pragma unroll
                    for (int i = 0; i < 4; i++) r2[i] = 0ull;
                }
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    // exact integer -> binary32 without a convert: 2^23 + (code + H), minus (2^23 + H)
                    const int f0 = 2 * i, f1 = 2 * i + 1;
                    const uint32_t w0 = (f0 < FPW) ? lo[j] : hi[j];
                    const uint32_t w1 = (f1 < FPW) ? lo[j] : hi[j];
                    const float q0 = __uint_as_float(0x4b000000u | ((w0 >> (BITS * (f0 % FPW))) & cmask));
                    const float q1 = __uint_as_float(0x4b000000u | ((w1 >> (BITS * (f1 % FPW))) & cmask));
                    float x0, x1;
                    unpack2(pfma(psub(pack2(q0, q1), base2), s2, pfma(a2, r2[i], b2)), x0, x1);
                    o[i] = f2_to_bf16x2(x0, x1);
                }
                sts128(obs + off[j], make_uint4(o[0], o[1], o[2], o[3]));
            }
            if (KG) {
                // outliers of this thread's group that fall into its own 32 channels, in record order
                const bool wide = lpq > 8;   // more than 256 channels per group: two-byte offsets
                const unsigned char *go = rec + p.goff_off + jq * p.kg;
                const unsigned short *go2 = reinterpret_cast<const unsigned short *>(rec + p.goff_off) + jq * p.kg;
                const unsigned short *gv = reinterpret_cast<const unsigned short *>(rec + p.gval_off) + jq * p.kg;
                const int qsize = lpq * 32;
                bool bad = false;
#pragma unroll
                for (int n = 0; n < 8; n++) {
                    if (n < p.kg) {
                        const int o = wide ? (int)go2[n] : (int)go[n];
                        if (o >= qsize) {
                            bad = true;
                        } else if ((o >> 5) == (tid & (lpq - 1))) {
                            const int c = jq * qsize + o;
                            float r = 0.f;
                            if (has_ref) {
                                r = __uint_as_float((uint32_t)(*reinterpret_cast<const unsigned short *>(rec + L.rec_pad + 2 * c)) << 16);
                                if (p.gain) r = bf16_round(__fmaf_rn(half_bits_to_float(p.gain[c]), r, half_bits_to_float(p.bias[c])));
                            }
                            const float xh = __fadd_rn(__fmaf_rn(a, r, b), half_bits_to_float(gv[n]));
                            reinterpret_cast<unsigned short *>(ob)[c] = __bfloat16_as_ushort(__float2bfloat16_rn(xh));
                        }
                    }
                }
                if (bad && p.status) atomicOr(p.status, RAC_STATUS_OUTLIER_RANGE);
            }
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
// host side
// ------------------------------------------------------------------------------------------------
// The 96-register variant (four 160-thread CTAs per SM) exists where it does not spill: without x_hat, and with
// outliers only below 8-bit codes.
template <int B, bool X, int K>
static int launch_encode_variant(bool tight, const Geometry &g, CodecParams &p, int smem, long long max_ctas, cudaStream_t stream) {
    if (p.tok_list || p.intra_base || p.coef_ext)   // the subset form: one variant, not the hot path
        return launch_persistent(encode_dyn_kernel<B, X, K, 2, true>, p, g.nthreads, smem, max_ctas, stream);
    // the paper's code widths (4 and 8 bits) at widths 5120 and 4096 with groups of 128 channels (alignment and
    // quantisation alike) run variants with those compiled in
    if constexpr (B == 4 || B == 8) {
        if (g.d == 5120 && g.lpg == 4 && g.lpq == 4) {
            if constexpr (!X && (K == 0 || B != 8))
                return launch_persistent(encode_dyn_kernel<B, X, K, 4, false, 4, 5120>, p, g.nthreads, smem, max_ctas, stream);
            else
                return launch_persistent(encode_dyn_kernel<B, X, K, 2, false, 4, 5120>, p, g.nthreads, smem, max_ctas, stream);
        }
        if (g.d == 4096 && g.lpg == 4 && g.lpq == 4)
            return launch_persistent(encode_dyn_kernel<B, X, K, 2, false, 4, 4096>, p, g.nthreads, smem, max_ctas, stream);
        if constexpr (K == 0) {   // the paper's decode mode: one scale per token
            if (g.lpg == 4 && g.lpq == 0 && g.qgen == 0) {
                if (g.d == 5120) {
                    if constexpr (!X)
                        return launch_persistent(encode_dyn_kernel<B, X, 0, 4, false, 4, 5120, true>, p, g.nthreads, smem, max_ctas, stream);
                    else
                        return launch_persistent(encode_dyn_kernel<B, X, 0, 2, false, 4, 5120, true>, p, g.nthreads, smem, max_ctas, stream);
                }
                if (g.d == 4096)
                    return launch_persistent(encode_dyn_kernel<B, X, 0, 2, false, 4, 4096, true>, p, g.nthreads, smem, max_ctas, stream);
            }
        }
    }
    if constexpr (!X && (K == 0 || B != 8)) {
        if (tight) return launch_persistent(encode_dyn_kernel<B, X, K, 4, false>, p, g.nthreads, smem, max_ctas, stream);
    }
    return launch_persistent(encode_dyn_kernel<B, X, K, 2, false>, p, g.nthreads, smem, max_ctas, stream);
}

template <int B>
static int launch_encode_bits(const Geometry &g, CodecParams &p, int smem, long long max_ctas, cudaStream_t stream) {
    const bool tight = g.nthreads > 128 && g.nthreads <= 160;
    const int k = g.topk_group;
    if (p.X_hat) {
        return k == 0 ? launch_encode_variant<B, true, 0>(tight, g, p, smem, max_ctas, stream)
             : k == 1 ? launch_encode_variant<B, true, 1>(tight, g, p, smem, max_ctas, stream)
             : k == 2 ? launch_encode_variant<B, true, 2>(tight, g, p, smem, max_ctas, stream)
             : k <= 4 ? launch_encode_variant<B, true, 4>(tight, g, p, smem, max_ctas, stream)
                      : launch_encode_variant<B, true, 8>(tight, g, p, smem, max_ctas, stream);
    }
    return k == 0 ? launch_encode_variant<B, false, 0>(tight, g, p, smem, max_ctas, stream)
         : k == 1 ? launch_encode_variant<B, false, 1>(tight, g, p, smem, max_ctas, stream)
         : k == 2 ? launch_encode_variant<B, false, 2>(tight, g, p, smem, max_ctas, stream)
         : k <= 4 ? launch_encode_variant<B, false, 4>(tight, g, p, smem, max_ctas, stream)
                  : launch_encode_variant<B, false, 8>(tight, g, p, smem, max_ctas, stream);
}

int launch_encode_dyn(const Geometry &g, CodecParams &p, long long max_ctas, cudaStream_t stream) {
    p.stages = 2;
    const DynSmem L = dyn_smem_layout(g.d, g.rec, p.stages);
    switch (g.bits) {
        case 8: return launch_encode_bits<8>(g, p, L.total, max_ctas, stream);
        case 4: return launch_encode_bits<4>(g, p, L.total, max_ctas, stream);
        case 3: return launch_encode_bits<3>(g, p, L.total, max_ctas, stream);
        case 2: return launch_encode_bits<2>(g, p, L.total, max_ctas, stream);
    }
    return RAC_EUNSUPPORTED;
}

int launch_decode_dyn(const Geometry &g, CodecParams &p, cudaStream_t stream) {
    p.stages = 2;
    const DecSmem L = dec_smem_layout(g.d, g.rec, p.stages);
    const bool kg = g.topk_group > 0;
    const bool sub = p.tok_list || p.intra_base || p.coef_ext;
    const bool spec = g.d == 5120 && g.lpg == 4 && g.lpq == 4;   // width and groups of 128 compiled in
#define RAC_DYN_DEC(B) \
    (sub ? (kg ? launch_persistent(decode_dyn_kernel<B, true, true>, p, g.nthreads, L.total, p.T, stream) \
               : launch_persistent(decode_dyn_kernel<B, false, true>, p, g.nthreads, L.total, p.T, stream)) \
     : spec ? (kg ? launch_persistent(decode_dyn_kernel<B, true, false, 4, 5120>, p, g.nthreads, L.total, p.T, stream) \
                  : launch_persistent(decode_dyn_kernel<B, false, false, 4, 5120>, p, g.nthreads, L.total, p.T, stream)) \
         : (kg ? launch_persistent(decode_dyn_kernel<B, true, false>, p, g.nthreads, L.total, p.T, stream) \
               : launch_persistent(decode_dyn_kernel<B, false, false>, p, g.nthreads, L.total, p.T, stream)))
    switch (g.bits) {
        case 8: return RAC_DYN_DEC(8);
        case 4: return RAC_DYN_DEC(4);
        case 3: return RAC_DYN_DEC(3);
        case 2: return RAC_DYN_DEC(2);
    }
#undef RAC_DYN_DEC
    return RAC_EUNSUPPORTED;
}

}  // namespace rac
