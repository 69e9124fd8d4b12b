/*
 * rac.h -- C ABI of the B200 (sm_100a) hot path of the RAC reference-aware
 * activation codec.
 *
 * The operations follow the paper's statement of the problem: a boundary hidden
 * state H [T,d] is coded as the residual against a shared, affinely aligned
 * reference (Sec. III-A, Eq. 2; Sec. IV-C), the receiver adds the dequantised
 * residual back (Eq. 9), the sender runs the same reconstruction so that later
 * references stay in sync (Sec. IV-C, first paragraph), and for prefill uplinks
 * the reference row of every token is picked by exact-token span retrieval over
 * a history (Sec. IV-B.1, Eq. 3).
 *
 * Conventions
 *  - Every tensor pointer is a DEVICE pointer owned by the caller.  The library
 *    allocates no device memory and frees none.  `cfg` structs and scalar
 *    arguments are host values.
 *  - Every call is asynchronous on `stream` (a cudaStream_t passed as void*;
 *    NULL is the default stream).  Nothing synchronises the device.
 *  - Return value: RAC_OK or a negative error.  Errors that the host can see
 *    (bad sizes, NULL or misaligned pointers, unsupported configuration) are
 *    returned BEFORE anything is launched and leave every output untouched.
 *  - Anomalies only the device can see never trap: the kernel ORs RAC_STATUS_*
 *    bits into `*dev_status` (device uint32, may be NULL) and finishes.
 *  - bf16 tensors are row major [rows, d]; rows must start on 16-byte
 *    boundaries (d is a multiple of 32, base pointers 16-byte aligned).
 *
 * Wire record of one token (little endian), records back to back in `payload`:
 *     coef    J x u32      binary16 alpha in bits 0..15, binary16 beta in 16..31,  J = d/group (absent with
 *                          coef_fmt 1)
 *     scale   Jq x u16     binary16 scales of the quantisation groups, scale_mode 1 only (Jq = d/qgroup),
 *                          padded to a multiple of 4 bytes
 *     codes   d*bits/8 B   code of channel c in stream bits [c*bits, c*bits+bits); stream bit n is
 *                          bit n%8 of byte n/8; two's complement; -2^(bits-1) is never produced
 *     out_idx topk x u16   channel indices, ascending
 *     out_val topk x u16   binary16 residuals of those channels (their dense code is 0)
 *     grp_off Jq*topk_group x u8   in-group offsets of the per-group outliers, ascending within a group (u16 each
 *                          when a group has more than 256 channels), padded to a multiple of 2 bytes (scale_mode 1 only)
 *     grp_val Jq*topk_group x u16  binary16 residuals of those channels (their dense code is 0)
 *     zero padding to a multiple of 16 bytes
 * rac_record_bytes() gives the stride.  A token range is a contiguous byte range.
 */
#ifndef RAC_H_
#define RAC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RAC_OK            0
#define RAC_EINVAL       -1   /* NULL pointer, negative size, inconsistent arguments           */
#define RAC_EALIGN       -2   /* a pointer that must be 16-byte aligned is not                 */
#define RAC_ESIZE        -3   /* a caller buffer (payload_cap, workspace_bytes) is too small   */
#define RAC_EUNSUPPORTED -4   /* a configuration this build has no kernel for                  */
#define RAC_ECUDA        -5   /* a CUDA runtime call failed (launch error, wrong device, ...)  */

/* bits ORed into *dev_status by the kernels */
#define RAC_STATUS_REF_RANGE     1u   /* a ref_row entry >= ref_rows: the token was coded/decoded as direct   */
#define RAC_STATUS_RESERVED_CODE 2u   /* decode met the code -2^(bits-1); it was dequantised as that value     */
#define RAC_STATUS_NONFINITE     4u   /* encode met a NaN/Inf in X or in the reference; that record is garbage */
#define RAC_STATUS_TIMEOUT       8u   /* an on-chip copy did not complete within the wait limit; the kernel
                                         stopped early and its outputs are incomplete                        */
#define RAC_STATUS_OUTLIER_RANGE 16u  /* decode met an outlier index >= d and ignored that outlier            */

/* Codec configuration (Sec. IV-C: calibration picks (g_a, g_q, q, k) per phase and direction).
 *   d       hidden width; multiple of 32, <= 8192
 *   group   g_a, channels per alignment group; power of two, 32..1024, divides d
 *   bits    code width q: 2, 3 or 4; also 8 in scale_mode 1     (Qmax = 2^(bits-1) - 1, Eq. 8a)
 *   topk    outliers per TOKEN kept as binary16, 0..16 (u16 channel index); scale_mode 0 only
 *   coef_fmt   0 = one binary16 pair per (token, group), in the record
 *              1 = one binary16 pair per (segment, group), outside the record (see rac_fit_segments): the
 *                  record then starts with the scales (scale_mode 1) or with the codes (scale_mode 0)
 *   scale_mode 0 = static per-channel step table `step`/`inv_step` (calibrated clip; dense values may clip);
 *                  g_q == g_a, `qgroup` 0 or == group, `topk_group` 0
 *              1 = Eq. 8 as printed: per quantisation group the scale s = RoundUp_binary16(max|E^d| / Qmax) is
 *                  carried in the record, scale 0 = all-zero group; nothing clips; `step` and `inv_step` are
 *                  not read and may be NULL
 *   flags   must be 0
 *   qgroup  g_q, channels per quantisation group (scale_mode 1): 0 = same as `group`; a power of two 32..1024
 *           that divides d; d itself (the paper's decode mode: one scale per token); or any other multiple of 32
 *           that divides d (without outliers)
 *   topk_group  k_g, outliers per quantisation group (Sec. IV-C "Outlier Metadata"), 0..8, scale_mode 1 with a
 *           power-of-two qgroup (not with qgroup = d unless d is such a value): the k_g largest |e| of every
 *           group (ties to the lower channel) leave the dense base before its scale is taken; in-group offsets in
 *           ascending order (one byte each for groups of up to 256 channels, two bytes little-endian for 512 and
 *           1024; the field is padded to an even size) + binary16 values */
typedef struct {
    int32_t d, group, bits, topk, coef_fmt, scale_mode, flags, qgroup, topk_group;
} rac_codec_cfg;

/* One selected span (Eq. 3): query[q_start .. q_start+len) == history[h_start .. h_start+len). */
typedef struct {
    int32_t q_start, h_start, len;
} rac_span;

const char *rac_version(void);
const char *rac_strerror(int err);

/* Record stride in bytes (0 for an invalid configuration) and payload size of T tokens. */
size_t rac_record_bytes(const rac_codec_cfg *cfg);
size_t rac_payload_bytes(const rac_codec_cfg *cfg, int64_t T);

/* Header of a serialised payload: 64 bytes that say how to read the T records behind them (the record format is
 * this library's own: the paper fixes only two 4-bit values per byte, per-group scales and in-group offsets with
 * binary16 values, Sec. IV-C).  HOST memory, host work only: nothing is launched.
 *   bytes  0..3   "RACP"          4..5  version (1)      6..7  header size (64)
 *          8..15  T (int64)       16..51  d, group, bits, topk, coef_fmt, scale_mode, flags, qgroup, topk_group
 *                                         (int32 each, qgroup as given)
 *         52..55  record bytes    56..59  sum of the fourteen 32-bit words before it, modulo 2^32    60..63  zero
 * All little endian.  rac_header_write returns RAC_EINVAL for an invalid configuration or T < 0.  rac_header_parse
 * returns RAC_EINVAL when magic, version, size, checksum or record size do not fit, and leaves the outputs alone. */
#define RAC_HEADER_BYTES 64
int rac_header_write(const rac_codec_cfg *cfg, int64_t T, void *header /* host, 64 bytes */);
int rac_header_parse(const void *header /* host, 64 bytes */, rac_codec_cfg *cfg_out, int64_t *T_out);

/* ---------------------------------------------------------------------------------------------
 * Span retrieval for prefill uplinks (Sec. IV-B.1, Eq. 3).
 *
 * Every window of `min_ngram` consecutive history tokens is indexed in a hash table (keys are
 * verified token by token, so hash collisions cannot change the result); of each distinct window
 * the `max_hits` most recent (largest) start positions are kept.  For every query position the
 * candidates are extended forward to their longest exact match, bounded by the end of the query
 * and of the history; the longest wins, ties go to the larger history start.  A left-to-right scan
 * then selects spans: at position i with a candidate of length L the span (i, j, L) is emitted and
 * the scan moves to i+L, otherwise to i+1.
 *
 *   hist_tok   int32[n_hist]     history token ids (row j of the history state buffer belongs to token j)
 *   query_tok  int32[n_query]    tokens of the current prompt
 *   min_ngram  w, 1..32
 *   max_hits   K, 1..16; or 0 = no limit: every occurrence of a window is a candidate (the plain longest
 *              match of the paper, the K-hit cap being a bucket policy).  The cost of a query position then
 *              grows with the number of occurrences of its window times the length they match over, so a
 *              history that repeats one token thousands of times is slow; keep the cap for token streams
 *              you do not control.  The persistent index (rac_index_*) takes the same values.
 *   ref_row    int32[n_query]    out: history row of every covered position, -1 elsewhere
 *   spans      rac_span[n_query/min_ngram + 1]  out, in query order; may be NULL
 *   n_spans    int32[1]          out (device)
 *   workspace  >= rac_match_workspace_bytes(n_hist, n_query, max_hits) bytes, 16-byte aligned;
 *              contents are scratch, nothing persists between calls
 * n_hist and n_query must be below 2^30.  n_query == 0 is allowed (only n_spans is written). */
size_t rac_match_workspace_bytes(int64_t n_hist, int64_t n_query, int32_t max_hits);
int rac_match_spans(const int32_t *hist_tok, int64_t n_hist, const int32_t *query_tok, int64_t n_query,
                    int32_t min_ngram, int32_t max_hits, int32_t *ref_row, rac_span *spans, int32_t *n_spans,
                    void *workspace, size_t workspace_bytes, void *stream);

/* Span retrieval for callers that cannot hand over device scratch.  (The paper has no counterpart: this is a
 * convenience of this library.)
 *
 * Who needs it: code that runs where allocating device memory is off the table -- a plug-in called from inside
 * another runtime that owns all device memory and gives out none, a serving loop whose memory budget was fixed
 * at start-up, a callback in which cudaMalloc would synchronise the device at the worst moment.  Such callers
 * can still pass their inputs and outputs, but have nowhere to get the matcher's workspace from.
 *
 * Same operation, arguments and results as rac_match_spans, minus the workspace: the scratch is a fixed array
 * of RAC_MATCH_STATIC_BYTES = 3 MiB inside the library image (every GPU that loads the library holds
 * it until the process ends).  That is enough for, e.g., a 32768-token history with 8192 query tokens and 8
 * hits; a problem whose rac_match_workspace_bytes() exceeds the capacity is refused with RAC_ESIZE and nothing is
 * launched.  The call allocates nothing and frees nothing, on the host side of CUDA or through any library.
 *
 * First call on a device: looks up the device address of the built-in array (one cudaGetSymbolAddress with
 * that device current).  Make that first call outside any stream capture.  The address is kept for the life of the
 * process: after a cudaDeviceReset of that device it is stale, and this entry point must not be used again.
 * All calls on a device share the one array.  Its contents survive from call to call, but every call
 * re-initialises what it reads (hash table, rows, span count), so stale contents never matter.  Two calls that
 * overlap on the GPU (different streams, or several host threads) race on the array and give garbage: keep the
 * calls of one device ordered on one stream. */
#define RAC_MATCH_STATIC_BYTES (3u << 20)
int rac_match_spans_static(const int32_t *hist_tok, int64_t n_hist, const int32_t *query_tok, int64_t n_query,
                           int32_t min_ngram, int32_t max_hits, int32_t *ref_row, rac_span *spans, int32_t *n_spans,
                           void *stream);

/* ---------------------------------------------------------------------------------------------
 * Span retrieval over a growing history of earlier requests (Sec. IV-B.1: the windows of "earlier requests"
 * are indexed, a candidate (r, j, L) lies inside one request r, recency breaks ties) with an index that
 * persists between prompts, plus the intra-sequence references of the same passage.
 *
 * The history is the concatenation of the requests seen so far; row j of the history state buffer belongs to
 * token j of that concatenation.  The index lives in caller memory (`index`, rac_index_bytes() bytes, 16-byte
 * aligned) and holds the hash table, the `max_hits` most recent starts of every distinct window, and the end of
 * the request of every history position.
 *
 *   rac_index_reset    empties the index.
 *   rac_index_append   adds ONE request: the tokens hist_tok[n_before .. n_after).  hist_tok is the device buffer
 *                      of the whole concatenation (tokens below n_before as at earlier calls: the index verifies
 *                      keys against them).  Windows lie inside the request; a request shorter than min_ngram adds
 *                      no window.  n_before must be the n_after of the previous append (0 after a reset); the
 *                      library keeps no host state and cannot check this.  n_after <= capacity.
 *                      Appending requests one by one gives the same index as any other split into calls with the
 *                      same request boundaries: contents do not depend on thread timing.
 *   rac_index_query    the selection of Eq. 3 for one prompt against the indexed history: like rac_match_spans,
 *                      except that a match ends at the end of its request.  With intra != 0, every position that no
 *                      span covers and whose token occurred EARLIER in the prompt gets
 *                      ref_row = n_hist + (position of the first occurrence of that token in the prompt): a
 *                      reference to the reconstruction of that earlier token of the same prompt.  First occurrences
 *                      never get such a reference, so they never chain: all tokens with ref_row < n_hist can be
 *                      coded first and the others second (rac_split_waves and the *_list calls below).
 *                      workspace >= rac_index_query_workspace_bytes(n_query) bytes, scratch.
 * The index only grows.  Old requests are dropped from the RESULTS at no cost with rac_index_query_live (below);
 * to reclaim their memory, reset the index and append the requests that are kept (appending 131072 tokens as 64
 * requests takes about 0.7 ms on a B200), or alternate between two indices.
 * All three are asynchronous on `stream`; calls on one index must be ordered. */
typedef struct {
    int64_t capacity;      /* history tokens the index can hold, 1 .. 2^30 - 1 */
    int32_t min_ngram;     /* w, 1..32 */
    int32_t max_hits;      /* K, 1..16, or 0 = no cap (every occurrence of a window is a candidate) */
} rac_index_cfg;
size_t rac_index_bytes(const rac_index_cfg *cfg);
int rac_index_reset(const rac_index_cfg *cfg, void *index, size_t index_bytes, void *stream);
int rac_index_append(const rac_index_cfg *cfg, void *index, size_t index_bytes, const int32_t *hist_tok,
                     int64_t n_before, int64_t n_after, void *stream);
size_t rac_index_query_workspace_bytes(int64_t n_query);
/* rac_index_query over a bounded history ("recent hits", Sec. IV-B.1): only windows that START at or after history
 * position first_live (0 <= first_live <= n_hist) are candidates; a match still runs forward as far as it goes.
 * Nothing is removed from the index: an old request is dropped by raising first_live past it, at no cost, and the
 * state rows below first_live are never referenced again (the caller may reuse that part of its state buffer; the
 * token buffer must stay readable, the index verifies keys against it).  The K most recent starts of a window that
 * lie in the live part are exactly the leading entries of its list, so the result equals a rebuild from the live
 * requests only.  rac_index_query is this call with first_live = 0. */
int rac_index_query_live(const rac_index_cfg *cfg, const void *index, size_t index_bytes, const int32_t *hist_tok,
                         int64_t n_hist, int64_t first_live, const int32_t *query_tok, int64_t n_query, int32_t intra,
                         int32_t *ref_row, rac_span *spans, int32_t *n_spans, void *workspace, size_t workspace_bytes,
                         void *stream);
int rac_index_query(const rac_index_cfg *cfg, const void *index, size_t index_bytes, const int32_t *hist_tok,
                    int64_t n_hist, const int32_t *query_tok, int64_t n_query, int32_t intra, int32_t *ref_row,
                    rac_span *spans, int32_t *n_spans, void *workspace, size_t workspace_bytes, void *stream);

/* Receiver side of the retrieval: spans travel as control metadata, tokens do not.  Expands
 * `*n_spans` spans into ref_row[n_query] (-1 where no span covers).  Spans reaching outside
 * [0, n_query) are clipped. */
int rac_spans_to_rows(const rac_span *spans, const int32_t *n_spans, int64_t n_query, int32_t *ref_row,
                      void *stream);

/* ---------------------------------------------------------------------------------------------
 * Encode (Sec. IV-C: Eq. 6 grouped affine fit with the zero-variance rule and wire rounding,
 * Eq. 7 aligned residual, outlier split, Eq. 8 symmetric quantisation, packing).
 *
 *   X         bf16[T,d]          activations to send
 *   ref_base  bf16[ref_rows,d]   reference rows; NULL = every token is coded directly
 *   ref_row   int32[T]           row of ref_base used by token t; NULL = row t (needs ref_rows >= T);
 *                                negative = token coded directly (zero reference, alpha = 0,
 *                                beta = group mean, step table row 1)
 *   ref_gain, ref_bias  binary16[d], both or neither: the reference row is first mapped per channel to
 *                                bf16(gain*r + bias) (stand-in for the decode predictor of Eq. 5)
 *   step, inv_step  float[2,d]   quantiser step and its reciprocal per channel; row 0 for tokens with a
 *                                reference, row 1 for direct tokens; step 0 means "code 0".  Steps are meant to
 *                                be binary16-representable values held as float (what rac_calibrate_steps
 *                                writes): code*step is then exact in binary32.  Every reconstruction in the
 *                                library evaluates fma(code, step, alpha*r + beta), so sender and receiver agree
 *                                bit for bit for ANY table; with a step that is not binary16-representable the
 *                                result can differ in its last bf16 bit from (alpha*r + beta) + round(code*step).
 *   payload   >= T*record bytes, 16-byte aligned; payload_cap is its capacity
 *   workspace >= rac_encode_workspace_bytes(cfg, T) bytes of scratch, 16-byte aligned (0 bytes, and NULL
 *             allowed, when cfg->topk == 0).  With outliers the call is two launches: the streaming pass leaves
 *             the largest |e| of every 32-channel slab here (4*d/32 bytes per token, rows padded to 16 bytes) and the
 *             outlier pass reads it.
 * The encoder reads only inv_step on the device: keep inv_step[c] == 0 wherever step[c] == 0 ("code 0").
 * The per-group fit is taken in binary32 on the device; its result, rounded to binary16, is what both
 * ends use, so any rounding difference against a binary64 fit shows up only in `coef`. */
size_t rac_encode_workspace_bytes(const rac_codec_cfg *cfg, int64_t T);
int rac_encode(const rac_codec_cfg *cfg, const void *X, int64_t T,
               const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
               const void *ref_gain, const void *ref_bias,
               const float *step, const float *inv_step,
               void *payload, size_t payload_cap, void *workspace, size_t workspace_bytes,
               uint32_t *dev_status, void *stream);

/* Encode and sender-side reconstruction in one pass (Sec. IV-C: "the sender applies the same wire-format
 * reconstruction as the receiver"; here it reuses the residuals and codes the encoder already holds instead of
 * decoding its own payload again).  Arguments as rac_encode plus
 *   X_hat  bf16[T,d] out: bit-identical to what rac_decode_reconstruct / rac_sender_reconstruct produce from
 *          `payload` with the same reference and step table.  Must not overlap X or payload.  It may be the very
 *          buffer that ref_base points to ONLY with ref_row == NULL (token t reads row t and writes row t; each
 *          row is read completely before it is written), which is how a decode loop keeps its state in place.
 *          With per-token outliers (topk > 0) the outliers are picked in a second launch that reads X and the
 *          reference rows again, after x_hat has been written: there X_hat must not overlap X, the in-place form
 *          above is refused (RAC_EUNSUPPORTED), and with a row list no token may reference a row that this call
 *          writes (the two-wave protocol of the *_list calls keeps to that; it is not checked on the device).
 * Both tables are read here (inv_step for the codes, step for x_hat). */
int rac_encode_reconstruct(const rac_codec_cfg *cfg, const void *X, int64_t T,
                           const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                           const void *ref_gain, const void *ref_bias,
                           const float *step, const float *inv_step,
                           void *payload, size_t payload_cap, void *X_hat, void *workspace, size_t workspace_bytes,
                           uint32_t *dev_status, void *stream);

/* Self-test of the bounded waits (the paper has no counterpart: it is about this library's failure handling).
 * Every wait of the streaming kernels on an mbarrier gives up after a fixed number of polls, sets
 * RAC_STATUS_TIMEOUT in *dev_status and lets the kernel return normally, so that a copy that never lands cannot
 * hang the GPU.  This call runs rac_encode (which = 0: `in` = X bf16[T,d], `out` = payload) or
 * rac_decode_reconstruct (which = 1: `in` = payload, `out` = X_hat bf16[T,d], out_cap in bytes) on at most 1024
 * tokens with identity rows, with every stage announcing 16 bytes more than its copies deliver: no wait can
 * complete, every CTA polls its limit out and takes the give-up path (well under a second per wait).  Expected: RAC_OK
 * from the call, RAC_STATUS_TIMEOUT in *dev_status, `out` unspecified, and the stream usable afterwards.  Nothing
 * faults and nothing waits without a bound. */
int rac_selftest_bounded_wait(const rac_codec_cfg *cfg, int32_t which, const void *in, int64_t T, const void *ref_base,
                              int64_t ref_rows, const float *step, const float *inv_step, void *out, size_t out_cap,
                              void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream);

/* Receiver reconstruction (Eq. 9): X_hat = bf16( (alpha*r + beta) + e_hat ), e_hat = code*step or the
 * stored binary16 outlier.  Arguments as rac_encode.  X_hat bf16[T,d] must not overlap payload.  X_hat
 * may be the very buffer that ref_base points to ONLY with ref_row == NULL (token t reads row t and
 * writes row t; each row is read completely before it is written). */
int rac_decode_reconstruct(const rac_codec_cfg *cfg, const void *payload, int64_t T,
                           const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                           const void *ref_gain, const void *ref_bias, const float *step,
                           void *X_hat, uint32_t *dev_status, void *stream);

/* Sender-side reconstruction (Sec. IV-C: the sender applies the same wire-format reconstruction as the
 * receiver so that subsequent references stay synchronised).  Same device code as
 * rac_decode_reconstruct, hence bit-identical output. */
int rac_sender_reconstruct(const rac_codec_cfg *cfg, const void *payload, int64_t T,
                           const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                           const void *ref_gain, const void *ref_bias, const float *step,
                           void *X_hat, uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Coding a subset of the tokens, with references into the reconstruction of the SAME prompt
 * (the intra-sequence references of Sec. IV-B.1).
 *
 * rac_split_waves: tokens whose ref_row is >= first_intra_row (normally n_hist, see rac_index_query) reference
 * another token of the prompt and must be coded after it; wave1[0 .. wave_count[0]) receives the other tokens,
 * wave2[0 .. wave_count[1]) these, both in ascending order.  wave1, wave2: int32[T]; wave_count: int32[2]
 * (all device memory).
 *
 * The *_list calls are rac_encode_reconstruct / rac_decode_reconstruct restricted to the tokens
 * tok_list[0 .. *tok_count) (device int32 list and device count; both NULL = all T tokens) and with a second
 * reference buffer: a ref_row entry r >= ref_rows names row r - ref_rows of `intra_base` (bf16 [intra_rows, d];
 * NULL/0 = none).  X, payload and X_hat keep their full [T, ...] shapes; only the listed tokens are read and
 * written.  List entries outside [0, T) are clamped into range.  X_hat of the encode call may be NULL (no sender
 * reconstruction).
 * Two-wave protocol, both endpoints: call once with wave 1 (intra_base may already be given: wave 1 never reads
 * it), then with wave 2 and intra_base = X_hat of this prompt, on the same stream.  The rows a wave-2 token
 * references were written by wave 1, and no wave-2 token is referenced by anyone, so the second call reads only
 * finished rows while it writes others.  That is a PRECONDITION on ref_row when it does not come from
 * rac_index_query: an entry >= first_intra_row must name a token whose own entry is below first_intra_row.  A
 * chain (a wave-2 token that references another wave-2 token) is not detected and makes the second call read a
 * row while another CTA writes it. */
int rac_split_waves(const int32_t *ref_row, int64_t T, int64_t first_intra_row, int32_t *wave1, int32_t *wave2,
                    int32_t *wave_count, void *stream);
int rac_encode_reconstruct_list(const rac_codec_cfg *cfg, const void *X, int64_t T, const int32_t *tok_list,
                                const int32_t *tok_count, const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                                const void *intra_base, int64_t intra_rows, const uint32_t *coef_seg, const int32_t *seg_of,
                                const void *ref_gain, const void *ref_bias,
                                const float *step, const float *inv_step, void *payload, size_t payload_cap, void *X_hat,
                                void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream);
int rac_decode_reconstruct_list(const rac_codec_cfg *cfg, const void *payload, int64_t T, const int32_t *tok_list,
                                const int32_t *tok_count, const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                                const void *intra_base, int64_t intra_rows, const uint32_t *coef_seg, const int32_t *seg_of,
                                const void *ref_gain, const void *ref_bias,
                                const float *step, void *X_hat, uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Eq. 6 over several fitting positions: one coefficient pair per (segment of consecutive tokens, group)
 * instead of one per (token, group).  H_j and R_j of Eq. 6 are then the [positions x group] slices of the
 * segment; a token coded directly contributes r = 0.  The pairs are shared by the tokens of the segment and
 * travel once per segment, outside the records: rac_codec_cfg.coef_fmt = 1 gives records without coefficient
 * words, in either scale mode (with the static table: [codes][outlier indices][outlier values]).
 *
 * rac_fit_segments
 *   seg_off   device int32[n_seg + 1], ascending, seg_off[0] = 0, seg_off[n_seg] = T; equal neighbours = an
 *             empty segment (its pairs come out as 0).  Spans of the retrieval and the gaps between them are the
 *             natural segments.
 *   coef_seg  device u32[n_seg, J] out: binary16 alpha | binary16 beta << 16, the zero-variance rule as for a
 *             single token
 *   seg_of    device int32[T] out: the segment of every token
 *   workspace >= rac_fit_segments_workspace_bytes(cfg, T) bytes, 16-byte aligned scratch
 * Sums are merged in binary64 in a fixed order: the same result on every run.
 * Coding: pass coef_seg and seg_of to the *_list calls (with tok_list NULL for all tokens) together with
 * coef_fmt = 1; with coef_fmt = 0 both must be NULL. */
/* The spans of a retrieval and the gaps between them as segments for rac_fit_segments, without a trip to the
 * host: seg_off[0 .. *n_seg] receives the boundaries (0, starts and ends of the spans, T; empty pieces dropped),
 * and seg_off[*n_seg + 1 .. max_seg] is filled with T, so that rac_fit_segments can be called with n_seg = max_seg
 * (the surplus segments are empty).  seg_off: device int32[max_seg + 1]; n_seg: device int32[1].  Spans must be in
 * query order and disjoint (as rac_match_spans / rac_index_query emit them).  At most (max_seg - 1) / 2 spans are
 * used: size max_seg as 2 * (span capacity) + 1. */
int rac_spans_to_segments(const rac_span *spans, const int32_t *n_spans, int64_t T, int64_t max_seg,
                          int32_t *seg_off, int32_t *n_seg, void *stream);
size_t rac_fit_segments_workspace_bytes(const rac_codec_cfg *cfg, int64_t T);
int rac_fit_segments(const rac_codec_cfg *cfg, const void *X, int64_t T, const void *ref_base, int64_t ref_rows,
                     const int32_t *ref_row, const void *ref_gain, const void *ref_bias, const int32_t *seg_off,
                     int64_t n_seg, uint32_t *coef_seg, int32_t *seg_of, void *workspace, size_t workspace_bytes,
                     uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Step tables from a calibration draw (the part of the offline calibration of Sec. IV-C that the
 * codec needs as an input).  Runs the fit and the residual of rac_encode over T calibration tokens and
 * sets, per channel and per table row (0: tokens with a reference, 1: direct tokens),
 *     step = smallest binary16 >= clip_sigmas * sqrt(mean e^2) / Qmax,   inv_step = 1/step (binary32),
 * both 0 for a row without tokens or a channel whose residual is identically 0.
 *   step, inv_step  float[2,d]  out
 *   workspace  >= rac_calibrate_workspace_bytes(cfg) bytes, 16-byte aligned scratch
 * Deterministic for a given device (fixed partition of tokens, fixed summation order). */
size_t rac_calibrate_workspace_bytes(const rac_codec_cfg *cfg);
int rac_calibrate_steps(const rac_codec_cfg *cfg, const void *X, int64_t T,
                        const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                        const void *ref_gain, const void *ref_bias, float clip_sigmas,
                        float *step, float *inv_step, void *workspace, size_t workspace_bytes,
                        uint32_t *dev_status, void *stream);
/* The same for shared coefficients (cfg->coef_fmt = 1, scale_mode 0): the residual of every calibration token is
 * taken with the pair of its segment, coef_seg[seg_of[t]] as rac_fit_segments wrote them over the same T tokens.
 * rac_calibrate_steps wants coef_fmt = 0, this call coef_fmt = 1 and both arrays (RAC_EINVAL otherwise). */
int rac_calibrate_steps_shared(const rac_codec_cfg *cfg, const void *X, int64_t T,
                               const void *ref_base, int64_t ref_rows, const int32_t *ref_row,
                               const void *ref_gain, const void *ref_bias,
                               const uint32_t *coef_seg, const int32_t *seg_of, float clip_sigmas,
                               float *step, float *inv_step, void *workspace, size_t workspace_bytes,
                               uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Reconstruction error of a sender-path run: the measurable half of the offline calibration of Sec. IV-C
 * (there the sender's own reconstruction is run per candidate configuration, and quality is weighed against all
 * the bytes of a record; the bytes are rac_record_bytes(), this call gives the error).
 *   X, X_hat   bf16[T,d], d a multiple of 8
 *   out        device double[3]: sum (x - x_hat)^2, sum x^2, max |x - x_hat|
 *   workspace  >= rac_recon_error_workspace_bytes() bytes, 16-byte aligned scratch
 * Sums are binary64 over a fixed partition in a fixed order: the result is the same on every run. */
size_t rac_recon_error_workspace_bytes(void);
int rac_recon_error(const void *X, const void *X_hat, int64_t T, int32_t d, double *out, void *workspace,
                    size_t workspace_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* RAC_H_ */
