// Exact-token span retrieval for prefill uplinks (Sec. IV-B.1, Eq. 3) on the GPU.
//
// Index: an open-addressing hash table with one slot per DISTINCT w-token window of the history.  A slot
// stores one representative start position (used to verify a key token by token, so hash collisions can
// never change the result) and the K largest start positions of that window in descending order.  A start
// enters its slot's list by a cascade of atomicMax: it is offered to entry 0, the smaller of (offered, found)
// is carried to entry 1, and so on.  Every step keeps the pair it touches, so entry 0 ends as the largest
// value ever offered, entry 1 as the largest of the rest, ...: the final lists do not depend on the order in
// which threads run.
// Query: one thread per query position looks its window up, extends each of the <= K candidates forward
// to the longest exact match and keeps lexargmax(length, start).
// Selection: the left-to-right scan of Eq. 3 visits a position, jumps by the span length if it has a
// candidate and by one otherwise.  "Next position at or after p that has a candidate" is a parallel
// suffix scan; the remaining chain (one hop per selected span) is walked by a single thread, and the
// spans are expanded to per-token rows in parallel.
#include <mutex>

#include "rac_common.cuh"

namespace rac {

struct MatchParams {
    const int32_t *hist;
    const int32_t *query;
    int32_t *ref_row;
    rac_span *spans_out;   // may be null
    int32_t *n_spans;
    // workspace sections
    int32_t *rep;          // [M]      representative start of the slot's window, -1 = empty
    int32_t *top;          // [M*K]    r-th largest start of the slot's window, -1 = none
    int32_t *slot_of;      // [nwin]
    int2 *best;            // [N]      (length, history start) of the best candidate, length 0 = none
    int2 *hop;             // [N]      (next position >= p with a candidate, position after its span)
    rac_span *spans_ws;    // [N/w + 1]
    int32_t *chunk_first;  // [ceil(N/1024)] first position with a candidate in each chunk of 1024 positions
    unsigned short *delta16; // [N]    jump4 - position, 65535 = does not fit
    int32_t *jump2;        // [N]      position after the next two spans at or after each position (n_query if fewer)
    int32_t *jump4;        // [N]      ... after the next four
    int n_hist, n_query, nwin, w, K;
    unsigned int mask;     // M - 1
    const int32_t *end_of; // [n_hist] end of the request that holds each history position; null = one request
    int first_live;        // only windows that start at or after this history position are candidates (0 = all)
    int32_t *next;         // [nwin]   unlimited hits (max_hits = 0) only: another start of the same window, -1 = none;
                           //          top[slot] is then the head of the slot's chain (K = 1 entry per slot)
};

__device__ __forceinline__ unsigned int window_hash(const int32_t *tok, int w) {
    unsigned long long h = 0x9E3779B97F4A7C15ull;
    for (int m = 0; m < w; m++) {
        h ^= (unsigned long long)(unsigned int)tok[m];
        h *= 0xff51afd7ed558ccdull;
        h ^= h >> 32;
    }
    return (unsigned int)h;
}

__device__ __forceinline__ bool same_window(const int32_t *a, const int32_t *b, int w) {
    for (int m = 0; m < w; m++)
        if (a[m] != b[m]) return false;
    return true;
}

// Offers start j to a descending list of K entries (-1 = empty): atomicMax at entry r keeps the larger of
// (offered, found) there and carries the smaller on to entry r + 1.  Whatever the interleaving with other
// threads, the list ends as the K largest values ever offered, in descending order.
__device__ __forceinline__ void cascade_insert(int32_t *lst, int K, int j) {
    int v = j;
    for (int r = 0; r < K && v >= 0; r++) {
        const int old = atomicMax(&lst[r], v);
        v = old < v ? old : v;
    }
}

__global__ void match_init_kernel(MatchParams p, long long table_ints) {
    long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    long long stride = (long long)gridDim.x * blockDim.x;
    for (long long k = i; k < table_ints; k += stride) p.rep[k] = -1;  // rep and top are contiguous
    for (long long k = i; k < p.n_query; k += stride) p.ref_row[k] = -1;
    if (i == 0) *p.n_spans = 0;
}

// one slot per distinct window: claim an empty slot or find the slot that already holds this window
__global__ void match_insert_kernel(MatchParams p) {
    int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= p.nwin) return;
    const int32_t *win = p.hist + j;
    unsigned int s = window_hash(win, p.w) & p.mask;
    int slot = -1;
    for (unsigned int probe = 0; probe <= p.mask; probe++) {
        int cur = atomicCAS(&p.rep[s], -1, j);
        if (cur == -1 || cur == j || same_window(p.hist + cur, win, p.w)) { slot = (int)s; break; }
        s = (s + 1) & p.mask;
    }
    p.slot_of[j] = slot;  // the table has >= 2*nwin slots, so a slot is always found
    if (slot < 0) return;
    // unlimited hits: every start of the window goes onto the slot's chain.  The order of a chain depends on which
    // thread came first; the query looks at ALL of it and keeps lexargmax(length, start), so the result does not.
    if (p.next) p.next[j] = atomicExch(&p.top[slot], j);
    else cascade_insert(p.top + (long long)slot * p.K, p.K, j);
}

__global__ void match_query_kernel(MatchParams p) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.n_query) return;
    int bestL = 0, bestj = -1;
    if (i + p.w <= p.n_query && p.nwin > 0) {
        const int32_t *win = p.query + i;
        unsigned int s = window_hash(win, p.w) & p.mask;
        int slot = -1;
        for (unsigned int probe = 0; probe <= p.mask; probe++) {
            int cur = p.rep[s];
            if (cur < 0) break;  // empty slot ends the probe sequence: the window is not in the history
            if (same_window(p.hist + cur, win, p.w)) { slot = (int)s; break; }
            s = (s + 1) & p.mask;
        }
        if (slot >= 0) {
            // candidate j: extend forward to the longest exact match, keep lexargmax(length, start)
            auto consider = [&](int j) {
                int L = p.w;
                const int hend = p.end_of ? p.end_of[j] : p.n_hist;   // a match stays inside its request
                // eight tokens per trip to memory: the loads of a trip are independent, and a long match is a chain
                // of dependent trips
                const int room = min(p.n_query - i, hend - j);            // L may grow up to this
                bool open = true;
                while (open && L + 8 <= room) {
                    int32_t q[8], h[8];
#pragma unroll
                    for (int u = 0; u < 8; u++) { q[u] = p.query[i + L + u]; h[u] = p.hist[j + L + u]; }
                    unsigned int ne = 0;
#pragma unroll
                    for (int u = 0; u < 8; u++) ne |= (q[u] != h[u]) ? (1u << u) : 0u;
                    if (ne) { L += __ffs(ne) - 1; open = false; }
                    else L += 8;
                }
                while (open && L < room && p.query[i + L] == p.hist[j + L]) L++;
                if (L > bestL || (L == bestL && j > bestj)) { bestL = L; bestj = j; }
            };
            if (p.next) {
                // every occurrence of the window (at most nwin of them: the walk is bounded by construction)
                int j = p.top[slot];
                for (int n = 0; j >= 0 && n < p.nwin; n++) {
                    if (j >= p.first_live) consider(j);
                    j = p.next[j];
                }
            } else {
                const int32_t *lst = p.top + (long long)slot * p.K;
                for (int r = 0; r < p.K; r++) {
                    const int j = lst[r];
                    if (j < p.first_live) break;   // descending: the rest is empty (-1) or older than the live window
                    consider(j);
                }
            }
        }
    }
    p.best[i] = make_int2(bestL, bestj);
}

// Selection.  (1) hop[p] = (s, s + len(s)) with s the first position >= p that has a candidate (n_query if
// none): a suffix scan, done grid-wide in two launches -- first the first candidate of every chunk of 1024
// positions, then every chunk completes its positions with the first candidate of the later chunks as carry --
// which also leaves the jump lengths hop.y - p as 16-bit deltas (65535 = "look it up in hop").  (2) One thread
// of a single CTA follows the chain from 0 and lists the positions it visits: the serial part of Eq. 3, one
// dependent read per selected span; the deltas of a window of positions are staged in shared memory so that each
// read is a shared-memory access instead of a trip to L2.  (3) A grid-wide kernel turns the visited positions into
// spans and per-token rows.
constexpr int kWalkWindow = 96 * 1024;  // positions per window: 192 KiB of shared memory
constexpr int kHopChunk = 1024;         // positions per CTA of the suffix scan

__global__ void __launch_bounds__(kHopChunk) match_chunk_first_kernel(MatchParams p) {
    __shared__ int s_first;
    const int i = blockIdx.x * kHopChunk + threadIdx.x;
    if (threadIdx.x == 0) s_first = p.n_query;
    __syncthreads();
    const bool st = i < p.n_query && p.best[i].x > 0;
    const unsigned int b = __ballot_sync(0xffffffffu, st);
    if (b && (threadIdx.x & 31) == 0) atomicMin(&s_first, i + __ffs(b) - 1);
    __syncthreads();
    if (threadIdx.x == 0) p.chunk_first[blockIdx.x] = s_first;
}

__global__ void __launch_bounds__(kHopChunk) match_hop_kernel(MatchParams p, int nchunks) {
    __shared__ int warp_first[kHopChunk / 32];
    __shared__ int s_carry;
    const int N = p.n_query;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int i = blockIdx.x * kHopChunk + tid;
    const int len = i < N ? p.best[i].x : 0;
    const unsigned int b = __ballot_sync(0xffffffffu, len > 0);
    if (lane == 0) warp_first[warp] = b ? (i + __ffs(b) - 1) : N;
    if (tid == 0) {
        int c = N;   // first candidate of the later chunks
        for (int k = blockIdx.x + 1; k < nchunks; k++) {
            const int f = p.chunk_first[k];
            if (f < N) { c = f; break; }
        }
        s_carry = c;
    }
    __syncthreads();
    if (i >= N) return;
    const unsigned int at_or_after = b >> lane;
    int s;
    if (at_or_after) {
        s = i + __ffs(at_or_after) - 1;
    } else {
        s = s_carry;
        for (int w = warp + 1; w < kHopChunk / 32; w++) {
            if (warp_first[w] < N) { s = warp_first[w]; break; }
        }
    }
    const int nx = s < N ? s + p.best[s].x : N;
    p.hop[i] = make_int2(s, nx);
}

// pointer doubling over "the position after the span at or after i": two spans, then four; the chain walk then
// takes one dependent step per FOUR selected spans
__global__ void match_jump2_kernel(MatchParams p) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.n_query) return;
    const int a = p.hop[i].y;
    p.jump2[i] = a < p.n_query ? p.hop[a].y : p.n_query;
}
__global__ void match_jump4_kernel(MatchParams p) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.n_query) return;
    const int a = p.jump2[i];
    const int b = a < p.n_query ? p.jump2[a] : p.n_query;
    p.jump4[i] = b;
    const int dlt = b - i;
    p.delta16[i] = (unsigned short)(dlt < 65535 ? dlt : 65535);
}

__global__ void __launch_bounds__(1024) match_select_kernel(MatchParams p, int window) {
    extern __shared__ unsigned short s_delta[];
    __shared__ int s_nspans, s_pos;
    const int N = p.n_query;
    const int tid = threadIdx.x;
    if (tid == 0) { s_pos = 0; s_nspans = 0; }
    __syncthreads();

    // (2) the chain, window by window; spans_ws[n].q_start keeps the n-th visited position
    while (true) {
        const int wbeg = s_pos;
        if (wbeg >= N) break;
        const int wend = min(N, wbeg + window);
        // eight deltas per load where the window start allows it (the array itself is 16-byte aligned)
        if ((wbeg & 7) == 0) {
            const int n8 = (wend - wbeg) >> 3;
            const uint4 *src = reinterpret_cast<const uint4 *>(p.delta16 + wbeg);
            uint4 *dst = reinterpret_cast<uint4 *>(s_delta);
            for (int i = tid; i < n8; i += blockDim.x) dst[i] = src[i];
            for (int i = wbeg + (n8 << 3) + tid; i < wend; i += blockDim.x) s_delta[i - wbeg] = p.delta16[i];
        } else {
            for (int i = wbeg + tid; i < wend; i += blockDim.x) s_delta[i - wbeg] = p.delta16[i];
        }
        __syncthreads();
        if (tid == 0) {
            int n = s_nspans, pos = wbeg;
            while (pos < wend) {
                p.spans_ws[n++].q_start = pos;          // start of a group of (up to) four spans
                const int dlt = s_delta[pos - wbeg];
                pos = dlt == 65535 ? p.jump4[pos] : pos + dlt;
            }
            s_nspans = n;
            s_pos = pos;
        }
        __syncthreads();
    }
    if (tid == 0) {
        p.chunk_first[0] = s_nspans;   // the suffix scan is done with this array: it now carries the group count
        *p.n_spans = 0;                // the expansion of the last group sets the real count
    }
}

// (3) grid-wide: a warp per group walks its (up to) four spans -- three dependent lookups each -- and expands them
// to rows; only the last group can hold fewer than four, and its warp sets the span count
__global__ void match_expand_kernel(MatchParams p) {
    const int N = p.n_query;
    const int ng = p.chunk_first[0];
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    for (int g = gw; g < ng; g += warps) {
        int pos = p.spans_ws[g].q_start;
        int m = 0;
        for (; m < 4 && pos < N; m++) {
            const int2 h = p.hop[pos];
            if (h.x >= N) break;               // no candidate at or after pos: the chain ends
            rac_span sp;
            sp.q_start = h.x;
            sp.len = h.y - h.x;
            sp.h_start = p.best[h.x].y;
            if (lane == 0 && p.spans_out) p.spans_out[4 * g + m] = sp;
            for (int q = lane; q < sp.len; q += 32) p.ref_row[sp.q_start + q] = sp.h_start + q;
            pos = h.y;
        }
        if (g == ng - 1 && lane == 0) *p.n_spans = 4 * g + m;
    }
}

__global__ void spans_to_rows_kernel(const rac_span *spans, const int32_t *n_spans, long long n_query, int32_t *ref_row) {
    const int ns = *n_spans;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    for (int s = gw; s < ns; s += warps) {
        long long q0 = spans[s].q_start, len = spans[s].len;
        int h0 = spans[s].h_start;
        for (long long m = lane; m < len; m += 32) {
            long long i = q0 + m;
            if (i >= 0 && i < n_query) ref_row[i] = h0 + (int)m;
        }
    }
}

// Spans and the gaps between them as segments: boundaries in ascending order, empty pieces dropped, the unused
// tail of seg_off filled with T (empty segments).  One CTA; thread k looks at span k.
__global__ void __launch_bounds__(1024) spans_to_segments_kernel(const rac_span *spans, const int32_t *n_spans, int T,
                                                                 int max_seg, int32_t *seg_off, int32_t *n_seg) {
    __shared__ int s_scan[1024];
    __shared__ int s_base;
    const int ns = min(*n_spans, (max_seg - 1) / 2);
    const int tid = threadIdx.x;
    if (tid == 0) { s_base = 1; seg_off[0] = 0; }   // boundary 0 always; every span adds its start (if a gap precedes) and its end
    __syncthreads();
    for (int k0 = 0; k0 < ns; k0 += 1024) {
        const int k = k0 + tid;
        int q0 = 0, q1 = 0, prev_end = 0, cnt = 0;
        if (k < ns) {
            q0 = spans[k].q_start;
            q1 = q0 + spans[k].len;
            prev_end = k > 0 ? spans[k - 1].q_start + spans[k - 1].len : 0;
            cnt = (q0 > prev_end ? 1 : 0) + (q1 > q0 ? 1 : 0);   // boundaries q0 (new only after a gap) and q1
        }
        s_scan[tid] = cnt;
        __syncthreads();
        for (int o = 1; o < 1024; o <<= 1) {
            const int v = tid >= o ? s_scan[tid - o] : 0;
            __syncthreads();
            s_scan[tid] += v;
            __syncthreads();
        }
        int at = s_base + s_scan[tid] - cnt;
        if (k < ns) {
            if (q0 > prev_end) seg_off[at++] = q0;
            if (q1 > q0) seg_off[at] = q1;
        }
        __syncthreads();
        if (tid == 1023) s_base += s_scan[1023];
        __syncthreads();
    }
    int nb = s_base;                      // boundaries written so far, the last one is the end of the last span
    __syncthreads();
    if (tid == 0) {
        if (seg_off[nb - 1] < T) seg_off[nb++] = T;   // the gap behind the last span
        *n_seg = nb - 1;
        s_base = nb;
    }
    __syncthreads();
    for (int i = s_base + tid; i <= max_seg; i += 1024) seg_off[i] = T;
}

__global__ void fill_i32_kernel(int32_t *dst, long long n, int32_t v) {
    long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    long long stride = (long long)gridDim.x * blockDim.x;
    for (; i < n; i += stride) dst[i] = v;
}

// ---------------------------------------------------------------------------------------------
// Persistent index over a growing list of requests
// ---------------------------------------------------------------------------------------------
struct IndexParams {
    const int32_t *hist;
    int32_t *rep;       // [M]
    int32_t *top;       // [M*K]
    int32_t *end_of;    // [capacity]
    int32_t *next;      // [capacity]  no cap on the hits: another start of the same window (chain link), else null
    int32_t *cnt;       // [M]         unused (kept so that the layout of an index does not change)
    int a, b;           // the request: tokens [a, b)
    int w, K;
    unsigned int mask;
};

// Appending a request: every position learns the end of its request; every window of the request finds or claims
// its slot and enters the slot's list by the cascade.  The request's starts are larger than everything already
// there, so the older entries move down (and the oldest fall off) as a by-product.  One launch, any request size.
__global__ void index_append_kernel(IndexParams p) {
    const int j = p.a + blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= p.b) return;
    p.end_of[j] = p.b;
    if (j + p.w > p.b) return;  // the window would leave the request
    const int32_t *win = p.hist + j;
    unsigned int s = window_hash(win, p.w) & p.mask;
    int slot = -1;
    for (unsigned int probe = 0; probe <= p.mask; probe++) {
        int cur = atomicCAS(&p.rep[s], -1, j);
        if (cur == -1 || cur == j || same_window(p.hist + cur, win, p.w)) { slot = (int)s; break; }
        s = (s + 1) & p.mask;
    }
    if (slot < 0) return;
    if (p.next) p.next[j] = atomicExch(&p.top[slot], j);   // every start, on the slot's chain (order irrelevant)
    else cascade_insert(p.top + (long long)slot * p.K, p.K, j);
}

// Intra-sequence references: first occurrence of every token of the prompt (a hash table keyed by a position
// whose token is the key, verified by comparing tokens), then the uncovered positions look theirs up.
__global__ void intra_insert_kernel(const int32_t *query, int n, int32_t *trep, int32_t *tfirst, unsigned int mask) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t tok = query[i];
    unsigned int s = window_hash(&tok, 1) & mask;
    for (unsigned int probe = 0; probe <= mask; probe++) {
        int cur = atomicCAS(&trep[s], -1, i);
        if (cur == -1 || cur == i || query[cur] == tok) { atomicMin(&tfirst[s], i); return; }
        s = (s + 1) & mask;
    }
}
__global__ void intra_assign_kernel(const int32_t *query, int n, const int32_t *trep, const int32_t *tfirst,
                                    unsigned int mask, int n_hist, int32_t *ref_row) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n || ref_row[i] >= 0) return;
    const int32_t tok = query[i];
    unsigned int s = window_hash(&tok, 1) & mask;
    for (unsigned int probe = 0; probe <= mask; probe++) {
        int cur = trep[s];
        if (cur < 0) return;
        if (query[cur] == tok) {
            const int f = tfirst[s];
            if (f < i) ref_row[i] = n_hist + f;
            return;
        }
        s = (s + 1) & mask;
    }
}

__global__ void fill2_i32_kernel(int32_t *a, long long na, int32_t va, int32_t *b, long long nb, int32_t vb) {
    long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    long long stride = (long long)gridDim.x * blockDim.x;
    for (long long k = i; k < na; k += stride) a[k] = va;
    for (long long k = i; k < nb; k += stride) b[k] = vb;
}

static size_t align16(size_t v) { return (v + 15) / 16 * 16; }

// SMs of the current device (grids of the grid-stride kernels are sized from it); looked up once per device
static int sm_count() {
    static int cache[64];
    static std::mutex m;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lock(m);
    if (cache[dev] == 0) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) sms = 148;
        cache[dev] = sms;
    }
    return cache[dev];
}

// the six launches of the selection (suffix scan and pointer doubling grid-wide, chain walk in one CTA, expansion
// grid-wide)
static int launch_selection(const MatchParams &p, cudaStream_t st) {
    const int nchunks = (p.n_query + kHopChunk - 1) / kHopChunk;
    match_chunk_first_kernel<<<nchunks, kHopChunk, 0, st>>>(p);
    match_hop_kernel<<<nchunks, kHopChunk, 0, st>>>(p, nchunks);
    match_jump2_kernel<<<(p.n_query + 255) / 256, 256, 0, st>>>(p);
    match_jump4_kernel<<<(p.n_query + 255) / 256, 256, 0, st>>>(p);
    const int window = p.n_query < kWalkWindow ? p.n_query : kWalkWindow;
    const size_t dyn = ((size_t)window * 2 + 15) / 16 * 16;
    if (dyn > 48 * 1024 &&
        cudaFuncSetAttribute(match_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return RAC_ECUDA;
    match_select_kernel<<<1, 1024, dyn, st>>>(p, window);
    match_expand_kernel<<<sm_count(), 256, 0, st>>>(p);
    return RAC_OK;
}



struct MatchLayout {
    size_t rep, top, slot_of, best, hop, spans, chunk_first, delta16, jump2, jump4, next, total;
    unsigned int M;
};
// K = 0 (unlimited hits): one entry per slot (the head of its chain) and a chain link per history position
static MatchLayout match_layout(long long n_hist, long long n_query, int K) {
    MatchLayout L;
    const bool chains = K == 0;
    if (chains) K = 1;
    unsigned long long M = 1024;
    while (M < 2ull * (unsigned long long)(n_hist > 0 ? n_hist : 1)) M <<= 1;
    L.M = (unsigned int)M;
    size_t o = 0;
    L.rep = o;      o += (size_t)M * 4;                       // rep and top must stay contiguous (one fill)
    L.top = o;      o = align16(o + (size_t)M * K * 4);
    L.slot_of = o;  o = align16(o + (size_t)(n_hist > 0 ? n_hist : 1) * 4);
    L.best = o;     o = align16(o + (size_t)(n_query > 0 ? n_query : 1) * 8);
    L.hop = o;      o = align16(o + (size_t)(n_query > 0 ? n_query : 1) * 8);
    L.spans = o;    o = align16(o + (size_t)(n_query + 1) * sizeof(rac_span));
    L.chunk_first = o; o = align16(o + ((size_t)(n_query > 0 ? n_query : 1) / kHopChunk + 1) * 4);
    L.delta16 = o;  o = align16(o + (size_t)(n_query > 0 ? n_query : 1) * 2);
    L.jump2 = o;    o = align16(o + (size_t)(n_query > 0 ? n_query : 1) * 4);
    L.jump4 = o;    o = align16(o + (size_t)(n_query > 0 ? n_query : 1) * 4);
    L.next = o;     if (chains) o = align16(o + (size_t)(n_hist > 0 ? n_hist : 1) * 4);
    L.total = o;
    return L;
}

// ---------------------------------------------------------------------------------------------
// Scratch for rac_match_spans_static: lives in the library image, so every GPU that loads the library
// holds these bytes until the process exits.  Host code must not pass the symbol itself to a kernel (on
// the host it is only a stand-in); the device address is looked up once per device below.
constexpr size_t kStaticMatchBytes = RAC_MATCH_STATIC_BYTES;  // 3 MiB: a 32768-token history, 8192 query tokens, 8 hits
static __device__ __align__(256) unsigned char g_match_scratch[kStaticMatchBytes];

static std::mutex g_match_scratch_mutex;
static void *g_match_scratch_addr[64];  // device address of g_match_scratch, per device ordinal; null = not looked up yet

// Device address of the scratch array on the CURRENT device (first call per device does the lookup).
static int static_match_scratch(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return RAC_ECUDA;
    std::lock_guard<std::mutex> lock(g_match_scratch_mutex);
    if (!g_match_scratch_addr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_match_scratch) != cudaSuccess || !ptr) return RAC_ECUDA;
        g_match_scratch_addr[dev] = ptr;
    }
    *out = g_match_scratch_addr[dev];
    return RAC_OK;
}

}  // namespace rac

using namespace rac;

extern "C" {

size_t rac_match_workspace_bytes(int64_t n_hist, int64_t n_query, int32_t max_hits) {
    if (n_hist < 0 || n_query < 0 || max_hits < 0 || max_hits > 16) return 0;
    if (n_hist >= (1ll << 30) || n_query >= (1ll << 30)) return 0;
    return match_layout(n_hist, n_query, max_hits).total;
}

int rac_match_spans(const int32_t *hist_tok, int64_t n_hist, const int32_t *query_tok, int64_t n_query,
                    int32_t min_ngram, int32_t max_hits, int32_t *ref_row, rac_span *spans, int32_t *n_spans,
                    void *workspace, size_t workspace_bytes, void *stream) {
    if (n_hist < 0 || n_query < 0 || !n_spans) return RAC_EINVAL;
    if (n_hist >= (1ll << 30) || n_query >= (1ll << 30)) return RAC_EUNSUPPORTED;
    if (min_ngram < 1 || min_ngram > 32) return RAC_EUNSUPPORTED;
    if (max_hits < 0 || max_hits > 16) return RAC_EUNSUPPORTED;
    if ((n_hist > 0 && !hist_tok) || (n_query > 0 && (!query_tok || !ref_row))) return RAC_EINVAL;
    if (!workspace) return RAC_EINVAL;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return RAC_EALIGN;
    MatchLayout L = match_layout(n_hist, n_query, max_hits);
    if (workspace_bytes < L.total) return RAC_ESIZE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    MatchParams p;
    p.end_of = nullptr;
    p.hist = hist_tok;
    p.query = query_tok;
    p.ref_row = ref_row;
    p.spans_out = spans;
    p.n_spans = n_spans;
    p.rep = reinterpret_cast<int32_t *>(ws + L.rep);
    p.top = reinterpret_cast<int32_t *>(ws + L.top);
    p.slot_of = reinterpret_cast<int32_t *>(ws + L.slot_of);
    p.best = reinterpret_cast<int2 *>(ws + L.best);
    p.hop = reinterpret_cast<int2 *>(ws + L.hop);
    p.spans_ws = reinterpret_cast<rac_span *>(ws + L.spans);
    p.chunk_first = reinterpret_cast<int32_t *>(ws + L.chunk_first);
    p.delta16 = reinterpret_cast<unsigned short *>(ws + L.delta16);
    p.jump2 = reinterpret_cast<int32_t *>(ws + L.jump2);
    p.jump4 = reinterpret_cast<int32_t *>(ws + L.jump4);
    p.n_hist = (int)n_hist;
    p.n_query = (int)n_query;
    p.nwin = (int)(n_hist - min_ngram + 1 > 0 ? n_hist - min_ngram + 1 : 0);
    p.w = min_ngram;
    p.K = max_hits > 0 ? max_hits : 1;
    p.first_live = 0;
    p.next = max_hits == 0 ? reinterpret_cast<int32_t *>(ws + L.next) : nullptr;
    p.mask = L.M - 1;

    const long long table_ints = (long long)L.M * (1 + p.K);
    const int tb = 256;
    long long work = table_ints > n_query ? table_ints : n_query;
    int init_blocks = (int)((work + tb - 1) / tb);
    if (init_blocks > sm_count() * 8) init_blocks = sm_count() * 8;
    if (init_blocks < 1) init_blocks = 1;
    match_init_kernel<<<init_blocks, tb, 0, st>>>(p, table_ints);
    if (p.nwin > 0 && n_query > 0) {
        int nb = (p.nwin + tb - 1) / tb;
        match_insert_kernel<<<nb, tb, 0, st>>>(p);
    }
    if (n_query > 0) {
        match_query_kernel<<<(int)((n_query + tb - 1) / tb), tb, 0, st>>>(p);
        if (launch_selection(p, st) != RAC_OK) return RAC_ECUDA;
    }
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

int rac_spans_to_rows(const rac_span *spans, const int32_t *n_spans, int64_t n_query, int32_t *ref_row, void *stream) {
    if (n_query < 0 || !n_spans) return RAC_EINVAL;
    if (n_query == 0) return RAC_OK;
    if (!spans || !ref_row) return RAC_EINVAL;
    if (n_query >= (1ll << 30)) return RAC_EUNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int blocks = (int)((n_query + 255) / 256);
    if (blocks > sm_count() * 8) blocks = sm_count() * 8;
    fill_i32_kernel<<<blocks, 256, 0, st>>>(ref_row, n_query, -1);
    spans_to_rows_kernel<<<sm_count(), 256, 0, st>>>(spans, n_spans, n_query, ref_row);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

int rac_match_spans_static(const int32_t *hist_tok, int64_t n_hist, const int32_t *query_tok, int64_t n_query,
                           int32_t min_ngram, int32_t max_hits, int32_t *ref_row, rac_span *spans, int32_t *n_spans,
                           void *stream) {
    // size check first, with the same layout function the caller-workspace entry point uses
    const size_t need = rac_match_workspace_bytes(n_hist, n_query, max_hits);
    if (need == 0) return (n_hist < 0 || n_query < 0) ? RAC_EINVAL : RAC_EUNSUPPORTED;
    if (need > kStaticMatchBytes) return RAC_ESIZE;  // problem too large for the built-in scratch
    void *scratch = nullptr;
    int rc = static_match_scratch(&scratch);
    if (rc != RAC_OK) return rc;
    // every launch of the matcher re-initialises the table, the rows and the span count, so whatever the
    // previous call left in the scratch is harmless
    return rac_match_spans(hist_tok, n_hist, query_tok, n_query, min_ngram, max_hits, ref_row, spans, n_spans, scratch,
                           kStaticMatchBytes, stream);
}

}  // extern "C"

// ---- persistent index ------------------------------------------------------------------------
namespace {
struct IndexLayout {
    size_t rep, top, cnt, end_of, slot_of, total;
    unsigned int M;
};
bool index_cfg_ok(const rac_index_cfg *c) {
    return c && c->capacity >= 1 && c->capacity < (1ll << 30) && c->min_ngram >= 1 && c->min_ngram <= 32 &&
           c->max_hits >= 0 && c->max_hits <= 16;   // 0 = no cap: chains instead of K-lists
}
IndexLayout index_layout(const rac_index_cfg *c) {
    IndexLayout L;
    unsigned long long M = 1024;
    while (M < 2ull * (unsigned long long)c->capacity) M <<= 1;
    L.M = (unsigned int)M;
    size_t o = 0;
    L.rep = o;      o += (size_t)M * 4;                        // rep and top contiguous: one fill with -1
    L.top = o;      o = align16(o + (size_t)M * (c->max_hits > 0 ? c->max_hits : 1) * 4);
    L.cnt = o;      o = align16(o + (size_t)M * 4);
    L.end_of = o;   o = align16(o + (size_t)c->capacity * 4);
    L.slot_of = o;  o = align16(o + (size_t)c->capacity * 4);
    L.total = o;
    return L;
}
struct QueryLayout {
    size_t best, hop, spans, chunk_first, delta16, jump2, jump4, trep, tfirst, total;
    unsigned int Mq;
};
QueryLayout query_layout(long long n_query) {
    QueryLayout L;
    const size_t n = (size_t)(n_query > 0 ? n_query : 1);
    unsigned long long M = 1024;
    while (M < 2ull * n) M <<= 1;
    L.Mq = (unsigned int)M;
    size_t o = 0;
    L.best = o;    o = align16(o + n * 8);
    L.hop = o;     o = align16(o + n * 8);
    L.spans = o;   o = align16(o + (n + 1) * sizeof(rac_span));
    L.chunk_first = o; o = align16(o + (n / kHopChunk + 1) * 4);
    L.delta16 = o; o = align16(o + n * 2);
    L.jump2 = o;   o = align16(o + n * 4);
    L.jump4 = o;   o = align16(o + n * 4);
    L.trep = o;    o = align16(o + (size_t)M * 4);
    L.tfirst = o;  o = align16(o + (size_t)M * 4);
    L.total = o;
    return L;
}
int grid_for(long long n, int tb) {
    long long b = (n + tb - 1) / tb;
    if (b > (long long)sm_count() * 16) b = (long long)sm_count() * 16;
    return (int)(b < 1 ? 1 : b);
}
}  // namespace

extern "C" {

size_t rac_index_bytes(const rac_index_cfg *cfg) { return index_cfg_ok(cfg) ? index_layout(cfg).total : 0; }

int rac_index_reset(const rac_index_cfg *cfg, void *index, size_t index_bytes, void *stream) {
    if (!index_cfg_ok(cfg)) return cfg ? RAC_EUNSUPPORTED : RAC_EINVAL;
    if (!index) return RAC_EINVAL;
    if (reinterpret_cast<uintptr_t>(index) & 15u) return RAC_EALIGN;
    const IndexLayout L = index_layout(cfg);
    if (index_bytes < L.total) return RAC_ESIZE;
    unsigned char *ix = static_cast<unsigned char *>(index);
    const long long table = (long long)L.M * (1 + (cfg->max_hits > 0 ? cfg->max_hits : 1));
    fill2_i32_kernel<<<grid_for(table, 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<int32_t *>(ix + L.rep), table, -1, reinterpret_cast<int32_t *>(ix + L.cnt), (long long)L.M, 0);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

int rac_index_append(const rac_index_cfg *cfg, void *index, size_t index_bytes, const int32_t *hist_tok,
                     int64_t n_before, int64_t n_after, void *stream) {
    if (!index_cfg_ok(cfg)) return cfg ? RAC_EUNSUPPORTED : RAC_EINVAL;
    if (!index || n_before < 0 || n_after < n_before) return RAC_EINVAL;
    if (n_after > cfg->capacity) return RAC_ESIZE;
    if (reinterpret_cast<uintptr_t>(index) & 15u) return RAC_EALIGN;
    const IndexLayout L = index_layout(cfg);
    if (index_bytes < L.total) return RAC_ESIZE;
    if (n_after == n_before) return RAC_OK;
    if (!hist_tok) return RAC_EINVAL;
    unsigned char *ix = static_cast<unsigned char *>(index);
    IndexParams p;
    p.hist = hist_tok;
    p.rep = reinterpret_cast<int32_t *>(ix + L.rep);
    p.top = reinterpret_cast<int32_t *>(ix + L.top);
    p.cnt = reinterpret_cast<int32_t *>(ix + L.cnt);
    p.end_of = reinterpret_cast<int32_t *>(ix + L.end_of);
    p.next = cfg->max_hits == 0 ? reinterpret_cast<int32_t *>(ix + L.slot_of) : nullptr;
    p.a = (int)n_before;
    p.b = (int)n_after;
    p.w = cfg->min_ngram;
    p.K = cfg->max_hits > 0 ? cfg->max_hits : 1;
    p.mask = L.M - 1;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int tb = 256;
    const int nb = (int)((n_after - n_before + tb - 1) / tb);
    index_append_kernel<<<nb, tb, 0, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

size_t rac_index_query_workspace_bytes(int64_t n_query) {
    if (n_query < 0 || n_query >= (1ll << 30)) return 0;
    return query_layout(n_query).total;
}

int rac_index_query(const rac_index_cfg *cfg, const void *index, size_t index_bytes, const int32_t *hist_tok,
                    int64_t n_hist, const int32_t *query_tok, int64_t n_query, int32_t intra, int32_t *ref_row,
                    rac_span *spans, int32_t *n_spans, void *workspace, size_t workspace_bytes, void *stream) {
    return rac_index_query_live(cfg, index, index_bytes, hist_tok, n_hist, 0, query_tok, n_query, intra, ref_row, spans,
                                n_spans, workspace, workspace_bytes, stream);
}

int rac_index_query_live(const rac_index_cfg *cfg, const void *index, size_t index_bytes, const int32_t *hist_tok,
                         int64_t n_hist, int64_t first_live, const int32_t *query_tok, int64_t n_query, int32_t intra,
                         int32_t *ref_row, rac_span *spans, int32_t *n_spans, void *workspace, size_t workspace_bytes,
                         void *stream) {
    if (!index_cfg_ok(cfg)) return cfg ? RAC_EUNSUPPORTED : RAC_EINVAL;
    if (!index || !n_spans || n_hist < 0 || n_query < 0 || !workspace) return RAC_EINVAL;
    if (first_live < 0 || first_live > n_hist) return RAC_EINVAL;
    if (n_hist > cfg->capacity) return RAC_ESIZE;
    if (n_query >= (1ll << 30) || n_hist + n_query >= (1ll << 31)) return RAC_EUNSUPPORTED;
    if ((n_hist > 0 && !hist_tok) || (n_query > 0 && (!query_tok || !ref_row))) return RAC_EINVAL;
    if ((reinterpret_cast<uintptr_t>(index) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return RAC_EALIGN;
    const IndexLayout L = index_layout(cfg);
    if (index_bytes < L.total) return RAC_ESIZE;
    const QueryLayout Q = query_layout(n_query);
    if (workspace_bytes < Q.total) return RAC_ESIZE;
    const unsigned char *ix = static_cast<const unsigned char *>(index);
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    MatchParams p;
    p.hist = hist_tok;
    p.query = query_tok;
    p.ref_row = ref_row;
    p.spans_out = spans;
    p.n_spans = n_spans;
    p.rep = const_cast<int32_t *>(reinterpret_cast<const int32_t *>(ix + L.rep));
    p.top = const_cast<int32_t *>(reinterpret_cast<const int32_t *>(ix + L.top));
    p.slot_of = nullptr;
    p.best = reinterpret_cast<int2 *>(ws + Q.best);
    p.hop = reinterpret_cast<int2 *>(ws + Q.hop);
    p.spans_ws = reinterpret_cast<rac_span *>(ws + Q.spans);
    p.chunk_first = reinterpret_cast<int32_t *>(ws + Q.chunk_first);
    p.delta16 = reinterpret_cast<unsigned short *>(ws + Q.delta16);
    p.jump2 = reinterpret_cast<int32_t *>(ws + Q.jump2);
    p.jump4 = reinterpret_cast<int32_t *>(ws + Q.jump4);
    p.n_hist = (int)n_hist;
    p.n_query = (int)n_query;
    p.nwin = (int)(n_hist - cfg->min_ngram + 1 > 0 ? n_hist - cfg->min_ngram + 1 : 0);
    p.w = cfg->min_ngram;
    p.K = cfg->max_hits > 0 ? cfg->max_hits : 1;
    p.mask = L.M - 1;
    p.next = cfg->max_hits == 0 ? const_cast<int32_t *>(reinterpret_cast<const int32_t *>(ix + L.slot_of)) : nullptr;
    p.first_live = (int)first_live;
    p.end_of = reinterpret_cast<const int32_t *>(ix + L.end_of);
    const int tb = 256;
    // rows to -1, span count to 0, and (for the intra-sequence pass) the token table to empty
    int32_t *trep = reinterpret_cast<int32_t *>(ws + Q.trep), *tfirst = reinterpret_cast<int32_t *>(ws + Q.tfirst);
    fill2_i32_kernel<<<grid_for(n_query > 1 ? n_query : 1, tb), tb, 0, st>>>(ref_row, n_query, -1, n_spans, 1, 0);
    if (n_query == 0) return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
    match_query_kernel<<<(int)((n_query + tb - 1) / tb), tb, 0, st>>>(p);
    if (launch_selection(p, st) != RAC_OK) return RAC_ECUDA;
    if (intra) {
        fill2_i32_kernel<<<grid_for(Q.Mq, tb), tb, 0, st>>>(trep, (long long)Q.Mq, -1, tfirst, (long long)Q.Mq, 0x7fffffff);
        const int nb = (int)((n_query + tb - 1) / tb);
        intra_insert_kernel<<<nb, tb, 0, st>>>(query_tok, (int)n_query, trep, tfirst, Q.Mq - 1);
        intra_assign_kernel<<<nb, tb, 0, st>>>(query_tok, (int)n_query, trep, tfirst, Q.Mq - 1, (int)n_hist, ref_row);
    }
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}

}  // extern "C"

extern "C" int rac_spans_to_segments(const rac_span *spans, const int32_t *n_spans, int64_t T, int64_t max_seg,
                                     int32_t *seg_off, int32_t *n_seg, void *stream) {
    if (!n_spans || !seg_off || !n_seg || T < 0 || max_seg < 1) return RAC_EINVAL;
    if (T >= (1ll << 30) || max_seg >= (1ll << 30)) return RAC_EUNSUPPORTED;
    if (!spans) return RAC_EINVAL;
    spans_to_segments_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(spans, n_spans, (int)T, (int)max_seg, seg_off,
                                                                               n_seg);
    return cudaGetLastError() == cudaSuccess ? RAC_OK : RAC_ECUDA;
}
