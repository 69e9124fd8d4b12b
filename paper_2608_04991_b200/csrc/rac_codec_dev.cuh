// Pieces shared by the RAC codec translation units (sm_100a): kernel parameters, the slab front end (loads,
// Eq. 6 statistics, wire coefficients), packing helpers, and the host-side launch helpers.
#pragma once

#include <math.h>
#include <stdlib.h>

#include <map>
#include <mutex>
#include <tuple>
#include <utility>

#include "rac_common.cuh"

namespace rac {

// ------------------------------------------------------------------------------------------------
// kernel parameters
// ------------------------------------------------------------------------------------------------
struct CodecParams {
    // tensors
    const uint16_t *X;         // encode / calibrate input, bf16[T,d]
    const uint16_t *ref_base;  // bf16[ref_rows,d] or null
    const int32_t *ref_row;    // int32[T] or null
    const uint16_t *gain;      // binary16[d] or null
    const uint16_t *bias;
    const float *step;         // [2,d]
    const float *inv_step;     // [2,d]
    uint8_t *payload;          // encode out / decode in
    uint16_t *X_hat;           // decode out
    float *calib_partial;      // calibrate out: [grid][2][d] sums of e^2, then [grid][2] token counts
    float *tmax;               // encode with outliers: [T][d/32] largest |e| per thread slab (caller workspace)
    uint32_t *status;
    long long T;
    long long ref_rows;
    // geometry
    int d, J, lpg, lpg_shift, topk, rec, code_bytes, stages;
    float inv_group;
    // a subset of the tokens (both null = all T tokens, in order), and a second reference buffer behind ref_base
    const int32_t *tok_list;     // int32[>= *tok_count] token indices in [0, T)
    const int32_t *tok_count;    // device int32[1]
    const uint16_t *intra_base;  // bf16[intra_rows, d]: reference rows ref_rows .. ref_rows + intra_rows - 1, or null
    long long intra_rows;
    // coefficient words shared by the tokens of a segment (Eq. 6 over several fitting positions), outside the record
    const uint32_t *coef_ext;    // u32[n_seg, J] or null (coefficients in the record)
    const int32_t *seg_of;       // int32[T] segment of each token
    float4 *moments;             // segment fit, first pass out: (mean r, mean h, Sxx, Sxy) per (token, group)
    // scale_mode 1 only: quantisation groups, per-group outliers, field offsets in the record
    int Jq, lpq, lpq_shift, kg, scale_off, codes_off, goff_off, gval_off;
    int qgen;   // lanes per quantisation group that is neither a power of two nor the token (lpq == 0 then), else 0
    // only from rac_selftest_bounded_wait: bytes announced on top of what the copies of a stage deliver, so that the
    // (bounded) wait for them cannot complete
    uint32_t test_extra_tx;
};

// scale_mode 1 (defined in rac_codec_dyn.cu)
int launch_encode_dyn(const Geometry &g, CodecParams &p, long long max_ctas, cudaStream_t stream);
int launch_decode_dyn(const Geometry &g, CodecParams &p, cudaStream_t stream);

constexpr int kMaxStages = 4;
constexpr int kRecBufs = 3;
constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it rounds to an integer (ties to even) in the low mantissa bits

// control block at the start of dynamic shared memory
struct Ctrl {
    unsigned long long bar[kMaxStages];
    int row[kMaxStages];        // reference row of the token in each stage, -1 = direct
    int seg[kMaxStages];        // segment of the token in each stage (shared coefficients only)
    long long tok[kMaxStages];  // the token in each stage (segment fit only)
};

__host__ __device__ inline int align_up(int v, int a) { return (v + a - 1) / a * a; }

struct EncSmem {  // calibration kernel
    int stage0, stage_bytes, acc0, total;
};
__host__ __device__ inline EncSmem enc_smem_layout(int d, int stages, int nthreads) {
    EncSmem s;
    s.stage0 = align_up((int)sizeof(Ctrl), 128);
    s.stage_bytes = 4 * d;  // X row + R row
    s.acc0 = s.stage0 + stages * s.stage_bytes;   // e^2 accumulators: 2 table rows x 32 floats per thread
    s.total = s.acc0 + 2 * nthreads * 32 * 4;
    return s;
}

struct DecSmem {
    int ctrl, stage0, stage_bytes, rec_pad, out0, total;
};
__host__ __device__ inline DecSmem dec_smem_layout(int d, int rec, int stages) {
    DecSmem s;
    s.ctrl = 0;
    s.stage0 = align_up((int)sizeof(Ctrl), 128);
    s.rec_pad = align_up(rec, 128);
    s.stage_bytes = s.rec_pad + 2 * d;
    s.out0 = s.stage0 + stages * s.stage_bytes;
    s.total = s.out0 + kRecBufs * 2 * d;
    return s;
}

// ------------------------------------------------------------------------------------------------
// device helpers
// ------------------------------------------------------------------------------------------------
typedef unsigned long long u64;

__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 pfma(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ u64 padd(u64 a, u64 b) {
    u64 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ u64 psub(u64 a, u64 b) {
    u64 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ u64 pmul(u64 a, u64 b) {
    u64 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// a 32-bit word of two bf16 -> packed (even channel, odd channel) binary32, exact
__device__ __forceinline__ u64 bf16x2_to_p(uint32_t w) {
    return pack2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
// bits of a where m is set, bits of b elsewhere
__device__ __forceinline__ uint32_t bitsel(uint32_t a, uint32_t b, uint32_t m) { return (a & m) | (b & ~m); }

// rotate the four entries right by rot (new[j] = old[(j - rot) & 3])
__device__ __forceinline__ void rot_right4(uint32_t (&w)[4], int rot) {
    if (rot & 1) { uint32_t t = w[3]; w[3] = w[2]; w[2] = w[1]; w[1] = w[0]; w[0] = t; }
    if (rot & 2) { uint32_t t = w[0]; w[0] = w[2]; w[2] = t; t = w[1]; w[1] = w[3]; w[3] = t; }
}
// rotate left by rot (new[j] = old[(j + rot) & 3])
__device__ __forceinline__ void rot_left4(uint32_t (&w)[4], int rot) {
    if (rot & 1) { uint32_t t = w[0]; w[0] = w[1]; w[1] = w[2]; w[2] = w[3]; w[3] = t; }
    if (rot & 2) { uint32_t t = w[0]; w[0] = w[2]; w[2] = t; t = w[1]; w[1] = w[3]; w[3] = t; }
}

// low BITS bits of eight integers -> one word, element 0 in the lowest field
template <int BITS>
__device__ __forceinline__ uint32_t pack8(const uint32_t (&b)[8]) {
    if (BITS == 4) {
        uint32_t b01 = bitsel(b[0], b[1] << 4, 0x0fu), b23 = bitsel(b[2], b[3] << 4, 0x0fu);
        uint32_t b45 = bitsel(b[4], b[5] << 4, 0x0fu), b67 = bitsel(b[6], b[7] << 4, 0x0fu);
        return __byte_perm(__byte_perm(b01, b23, 0x0040), __byte_perm(b45, b67, 0x0040), 0x5410);
    } else {
        constexpr uint32_t m1 = (1u << BITS) - 1u, m2 = (1u << (2 * BITS)) - 1u, m4 = (1u << (4 * BITS)) - 1u;
        constexpr uint32_t m8 = (BITS * 8 == 32) ? 0xffffffffu : ((1u << (BITS * 8 % 32)) - 1u);
        uint32_t p0 = bitsel(b[0], b[1] << BITS, m1), p1 = bitsel(b[2], b[3] << BITS, m1);
        uint32_t p2 = bitsel(b[4], b[5] << BITS, m1), p3 = bitsel(b[6], b[7] << BITS, m1);
        uint32_t q0 = bitsel(p0, p1 << (2 * BITS), m2), q1 = bitsel(p2, p3 << (2 * BITS), m2);
        return bitsel(q0, q1 << (4 * BITS), m4) & m8;
    }
}

// Two signed integers saturated to BITS-bit two's complement and packed below the bits of c
// (d = c << 2*BITS | sat(hi) << BITS | sat(lo)); BITS is 4 or 2.
template <int BITS>
__device__ __forceinline__ uint32_t sat_pack2(int hi, int lo, uint32_t c) {
    uint32_t d;
    if (BITS == 4) asm("cvt.pack.sat.s4.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(hi), "r"(lo), "r"(c));
    else asm("cvt.pack.sat.s2.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(hi), "r"(lo), "r"(c));
    return d;
}

// reference values of one slot (8 channels starting at channel c) from shared memory, with the optional
// per-channel transform r <- bf16(gain*r + bias)
__device__ __forceinline__ void load_ref_slot(uint32_t addr, const uint16_t *gain, const uint16_t *bias, int c,
                                              u64 (&r2)[4]) {
    uint4 w = lds128(addr);
    const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
    if (gain) {
        uint4 gw = __ldg(reinterpret_cast<const uint4 *>(gain + c));
        uint4 bw = __ldg(reinterpret_cast<const uint4 *>(bias + c));
        const uint32_t gws[4] = {gw.x, gw.y, gw.z, gw.w};
        const uint32_t bws[4] = {bw.x, bw.y, bw.z, bw.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            float g0 = half_bits_to_float(gws[i] & 0xffff), g1 = half_bits_to_float(gws[i] >> 16);
            float b0 = half_bits_to_float(bws[i] & 0xffff), b1 = half_bits_to_float(bws[i] >> 16);
            float r0 = __uint_as_float(ws[i] << 16), r1 = __uint_as_float(ws[i] & 0xffff0000u);
            r2[i] = pack2(bf16_round(__fmaf_rn(g0, r0, b0)), bf16_round(__fmaf_rn(g1, r1, b1)));
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; i++) r2[i] = bf16x2_to_p(ws[i]);
    }
}

// the same for one pair of channels (c even), operation for operation
__device__ __forceinline__ u64 load_ref_pair(uint32_t addr, const uint16_t *gain, const uint16_t *bias, int c) {
    const uint32_t w = lds32(addr);
    if (gain) {
        const uint32_t gw = __ldg(reinterpret_cast<const uint32_t *>(gain + c));
        const uint32_t bw = __ldg(reinterpret_cast<const uint32_t *>(bias + c));
        const float g0 = half_bits_to_float(gw & 0xffff), g1 = half_bits_to_float(gw >> 16);
        const float b0 = half_bits_to_float(bw & 0xffff), b1 = half_bits_to_float(bw >> 16);
        const float r0 = __uint_as_float(w << 16), r1 = __uint_as_float(w & 0xffff0000u);
        return pack2(bf16_round(__fmaf_rn(g0, r0, b0)), bf16_round(__fmaf_rn(g1, r1, b1)));
    }
    return bf16x2_to_p(w);
}

// SUB = false compiles the plain form (all T tokens in order, one reference buffer); SUB = true the form of the
// *_list entry points.  how many tokens this launch codes, and the idx-th of them:
template <bool SUB>
__device__ __forceinline__ long long tokens_to_do(const CodecParams &p) {
    if constexpr (!SUB) return p.T;
    if (!p.tok_count) return p.T;
    const long long n = *p.tok_count;
    return n < 0 ? 0 : (n > p.T ? p.T : n);
}
template <bool SUB>
__device__ __forceinline__ long long token_at(const CodecParams &p, long long idx) {
    if constexpr (!SUB) return idx;
    if (!p.tok_list) return idx;
    const long long t = p.tok_list[idx];
    return t < 0 ? 0 : (t >= p.T ? p.T - 1 : t);   // a bad entry cannot leave the buffers
}
// Reference row of a token (-1 = coded directly); with SUB in the joint row space [ref_base rows | intra_base
// rows].  `flag` false: do not report rows beyond the buffers (a second pass over tokens already reported).
template <bool SUB>
__device__ __forceinline__ int resolve_row(const CodecParams &p, int raw_row, bool flag = true) {
    if constexpr (!SUB) {
        if (!p.ref_base || raw_row < 0) return -1;
        if (raw_row >= p.ref_rows) {
            if (flag && p.status) atomicOr(p.status, RAC_STATUS_REF_RANGE);
            return -1;
        }
        return raw_row;
    } else {
        if (raw_row < 0 || (!p.ref_base && !p.intra_base)) return -1;
        if (raw_row < p.ref_rows) return raw_row;
        if (p.intra_base && raw_row - p.ref_rows < p.intra_rows) return raw_row;
        if (flag && p.status) atomicOr(p.status, RAC_STATUS_REF_RANGE);
        return -1;
    }
}
template <bool SUB>
__device__ __forceinline__ const uint16_t *ref_row_ptr(const CodecParams &p, long long row) {
    if constexpr (!SUB) return p.ref_base + row * p.d;
    return row < p.ref_rows ? p.ref_base + row * p.d : p.intra_base + (row - p.ref_rows) * p.d;
}
// thread 0: start the copies of one token into a stage: `first` (X row or record) and, if any, its reference row
template <bool SUB>
__device__ __forceinline__ void issue_token_loads(const CodecParams &p, Ctrl *ctrl, uint32_t stage_addr, uint32_t r_off,
                                                  int stage, int row, const void *first_src, uint32_t first_bytes,
                                                  long long tok = 0) {
    ctrl->row[stage] = row;
    if constexpr (SUB) ctrl->seg[stage] = p.seg_of ? p.seg_of[tok] : 0;
    const uint32_t bar = smem_u32(&ctrl->bar[stage]);
    const uint32_t row_bytes = 2u * (uint32_t)p.d;
    mbar_arrive_expect_tx(bar, p.test_extra_tx + first_bytes + (row >= 0 ? row_bytes : 0u));
    bulk_load(stage_addr, first_src, first_bytes, bar);
    if (row >= 0) bulk_load(stage_addr + r_off, ref_row_ptr<SUB>(p, row), row_bytes, bar);
}

// Eq. 6 for the group this thread belongs to: centred two-pass sums over the thread's 32 channels (packed
// binary32, two accumulators per sum), butterflies over the group's lanes, the zero-variance rule, and wire
// rounding of (alpha, beta) to binary16.  Returns the wire coefficients splatted for packed arithmetic; a16/b16
// are their bit patterns.
__device__ __forceinline__ void fit_group(const u64 (&x2)[16], const u64 (&r2)[16], bool has_ref, int lpg, float inv_group,
                                          unsigned int group_mask, uint32_t *status, u64 &a2, u64 &b2,
                                          uint32_t *coef_word = nullptr, float4 *stats = nullptr) {
    u64 sra = 0ull, srb = 0ull, sha = 0ull, shb = 0ull;
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        sra = padd(sra, r2[i]); srb = padd(srb, r2[i + 1]);
        sha = padd(sha, x2[i]); shb = padd(shb, x2[i + 1]);
    }
    float sr, sr_hi, sh, sh_hi;
    unpack2(padd(sra, srb), sr, sr_hi);
    unpack2(padd(sha, shb), sh, sh_hi);
    sr += sr_hi;
    sh += sh_hi;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        if (lpg > o) {
            sr += __shfl_xor_sync(group_mask, sr, o);
            sh += __shfl_xor_sync(group_mask, sh, o);
        }
    }
    if (!(fabsf(sr) <= 3.0e38f) || !(fabsf(sh) <= 3.0e38f)) {
        if (status) atomicOr(status, RAC_STATUS_NONFINITE);
    }
    const float rbar = sr * inv_group, hbar = sh * inv_group;
    const u64 rbar2 = pack2(rbar, rbar), hbar2 = pack2(hbar, hbar);
    u64 sxxa = 0ull, sxxb = 0ull, sxya = 0ull, sxyb = 0ull;
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        u64 dr0 = psub(r2[i], rbar2), dh0 = psub(x2[i], hbar2);
        u64 dr1 = psub(r2[i + 1], rbar2), dh1 = psub(x2[i + 1], hbar2);
        sxxa = pfma(dr0, dr0, sxxa); sxya = pfma(dr0, dh0, sxya);
        sxxb = pfma(dr1, dr1, sxxb); sxyb = pfma(dr1, dh1, sxyb);
    }
    float sxx, sxx_hi, sxy, sxy_hi;
    unpack2(padd(sxxa, sxxb), sxx, sxx_hi);
    unpack2(padd(sxya, sxyb), sxy, sxy_hi);
    sxx += sxx_hi;
    sxy += sxy_hi;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        if (lpg > o) {
            sxx += __shfl_xor_sync(group_mask, sxx, o);
            sxy += __shfl_xor_sync(group_mask, sxy, o);
        }
    }
    if (stats) *stats = make_float4(rbar, hbar, sxx, sxy);
    // zero-variance rule, then wire rounding to binary16
    float a_star = 0.f, b_star = hbar;
    if (has_ref && sxx > 1e-12f && fabsf(sxy) < 65504.0f * sxx) {
        a_star = __fdiv_rn(sxy, sxx);
        b_star = __fmaf_rn(-a_star, rbar, hbar);
    }
    const uint32_t a16 = float_to_half_bits_sat(a_star), b16 = float_to_half_bits_sat(b_star);
    const float a = half_bits_to_float(a16), b = half_bits_to_float(b16);
    a2 = pack2(a, a);
    b2 = pack2(b, b);
    if (coef_word) *coef_word = a16 | (b16 << 16);
}

// ------------------------------------------------------------------------------------------------
// host side: launch plumbing
// ------------------------------------------------------------------------------------------------
struct DeviceInfo {
    int sms = 0;
    int max_smem_optin = 0;
};
inline std::mutex &launch_mutex() {
    static std::mutex m;
    return m;
}
static int device_info(DeviceInfo *out, int *dev_out = nullptr) {
    static DeviceInfo cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return RAC_ECUDA;
    std::lock_guard<std::mutex> lock(launch_mutex());
    if (cache[dev].sms == 0) {
        int sms = 0, smem = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return RAC_ECUDA;
        if (cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return RAC_ECUDA;
        cache[dev].max_smem_optin = smem;
        cache[dev].sms = sms;
    }
    *out = cache[dev];
    if (dev_out) *dev_out = dev;
    return RAC_OK;
}

// Resident CTAs per SM of one kernel at one block size and shared-memory size, looked up once per device.  The
// kernel's shared-memory limit is an attribute of the kernel, not of a launch: it is only ever raised, so that a
// launch with less shared memory between two larger ones leaves it where the larger ones need it.
static int resident_ctas(const void *kernel, int dev, int nthreads, int smem_bytes, int *occ_out) {
    struct Key {
        const void *kernel;
        int dev, nthreads, smem;
        bool operator<(const Key &o) const {
            return std::tie(kernel, dev, nthreads, smem) < std::tie(o.kernel, o.dev, o.nthreads, o.smem);
        }
    };
    static std::map<Key, int> table;
    static std::map<std::pair<const void *, int>, int> limit;   // (kernel, device) -> shared-memory limit set so far
    const Key key{kernel, dev, nthreads, smem_bytes};
    std::lock_guard<std::mutex> lock(launch_mutex());
    auto it = table.find(key);
    if (it == table.end()) {
        int &lim = limit[std::make_pair(kernel, dev)];
        if (smem_bytes > lim) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) return RAC_ECUDA;
            lim = smem_bytes;
        }
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, nthreads, smem_bytes) != cudaSuccess || occ < 1)
            return RAC_ECUDA;
        it = table.emplace(key, occ).first;
    }
    *occ_out = it->second;
    return RAC_OK;
}

template <typename K>
static int launch_persistent(K kernel, const CodecParams &p, int nthreads, int smem_bytes, long long max_ctas,
                             cudaStream_t stream) {
    DeviceInfo di;
    int dev = 0;
    int rc = device_info(&di, &dev);
    if (rc != RAC_OK) return rc;
    if (smem_bytes > di.max_smem_optin) return RAC_EUNSUPPORTED;
    int occ = 0;
    rc = resident_ctas(reinterpret_cast<const void *>(kernel), dev, nthreads, smem_bytes, &occ);
    if (rc != RAC_OK) return rc;
    long long grid = (long long)di.sms * occ;
    if (grid > max_ctas) grid = max_ctas;
    if (grid < 1) grid = 1;
    kernel<<<(unsigned)grid, nthreads, smem_bytes, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace rac
