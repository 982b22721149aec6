// S2a: exact outlier thresholds (order statistics) per (b,h) and tensor, in one read of the data.
//
// Wanted: lo = k-th smallest and hi = k-th largest of the N non-NaN values, k = floor(alpha*N/2).
// Only the two tails matter, so the bulk of the data is never histogrammed:
//   1. thr_sample_kernel   a few tokens spread over the sequence give a bracket per tail: a value
//                          below (above) which somewhat more than the wanted tail mass lies.  Problems
//                          small enough to be sampled completely are solved right here.
//   2. thr_scan_kernel     the one pass over all values: entries beyond the brackets ("candidates",
//                          a few per cent) are compacted into per-problem lists (shared-memory lists
//                          per CTA, one global reservation per CTA and tail), NaNs are counted.
//   3. thr_select_kernel   exact radix select of rank k inside the candidate lists.  If a bracket
//                          turned out too tight (fewer than k+1 candidates) or a list overflowed, the
//                          problem is redone exactly by a two-pass radix select over its data, so the
//                          result is always the exact order statistic.
// binary16 patterns are mapped to 16-bit keys that sort like the values.
#include "qaq_internal.cuh"

namespace {

constexpr int SAMPLE_TOKENS = 64;
#ifndef QWARP_FLAGS
#define QWARP_FLAGS 192
#endif
constexpr int SCAN_TOKENS_MAX = 512; // tokens per CTA of the scan (fewer where alpha is large: see scan_tokens_for)
constexpr int WARP_FLAGS = QWARP_FLAGS;      // 16-byte pieces a warp of the scan can set aside before it has to look at them
constexpr int CTA_LIST = 4096;       // candidates per tail a scan CTA can hold
constexpr int SELECT_KEYS = 16384;   // candidates of one tail the select kernel keeps in shared memory

__device__ __forceinline__ uint32_t key_of(unsigned short h) { return (h & 0x8000u) ? (uint32_t)(~h & 0xFFFFu) : (uint32_t)(h | 0x8000u); }
__device__ __forceinline__ unsigned short half_of_key(uint32_t k) { return (k & 0x8000u) ? (unsigned short)(k & 0x7FFFu) : (unsigned short)(~k & 0xFFFFu); }
__device__ __forceinline__ bool is_nan_bits(unsigned short h) { return (h & 0x7FFFu) > 0x7C00u; }
__device__ __forceinline__ __half2 h2_of(uint32_t x) { return *reinterpret_cast<__half2*>(&x); }
__device__ __forceinline__ float float_of_key(uint32_t k) { return __half2float(__ushort_as_half(half_of_key(k))); }

struct Problem {          // per (b,h,tensor), in the workspace
    uint32_t klo, khi;    // bracket keys: candidates are keys < klo and keys > khi
    uint32_t cnt[2];      // candidates found (may exceed the capacity: then the list is incomplete)
    uint32_t nan;         // NaN entries seen by the scan
    uint32_t done;        // solved by the sample kernel
    uint32_t overflow;    // bit `tail`: a scan CTA found more candidates than it can hold, the list has holes
    uint32_t pad;
};

struct ThrArgs {
    const __half* X[2];
    long sb, sh, st;
    int H, T, D;
    double alpha;
    Problem* prob;        // [BH*2]
    unsigned short* list; // [BH*2][2][cap]
    uint32_t cap;
    int scan_tokens;      // tokens per CTA of the scan
    float* thr;           // [BH][4]
};

// rank select (0-based rank `want`) over n 16-bit keys readable through get(i); all threads of the
// CTA (256) call it; hist is 2048 words of shared memory.  Two passes of a radix select: the upper
// 11 bits of the key first, then the lower 5.  binary16 data piles up in a few exponents, so a
// histogram of the upper byte alone would send most lanes of a warp to the same handful of
// counters; 11 bits spread them over 32 bins per octave.  In the first pass every thread sums 8 bins and a
// CTA-wide prefix sum finds the bin holding the wanted rank; the second pass has 32 bins, one per lane of
// warp 0.
template <typename Get>
__device__ uint32_t cta_select(Get get, uint32_t n, uint32_t want, uint32_t* hist, uint32_t* s_tmp) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // ---- first pass: upper 11 bits
    for (int i = threadIdx.x; i < 2048; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) {
        const uint32_t k = get(i);
        if (k <= 0xFFFFu) atomicAdd(&hist[k >> 5], 1u);     // larger: NaN marker
    }
    __syncthreads();
    uint32_t c[8], tot = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) { c[j] = hist[8 * threadIdx.x + j]; tot += c[j]; }
    uint32_t inc = tot;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += t;
    }
    __syncthreads();                                         // every thread has read its bins
    if (lane == 31) hist[warp] = inc;                        // warp totals
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        const uint32_t v = hist[w];
        if (w < warp) before += v;
        all += v;
    }
    uint32_t acc = before + inc - tot;                       // keys in the bins before this thread's eight
    const uint32_t w2 = want < all ? want : (all ? all - 1 : 0);   // defensive clamp
    if (threadIdx.x == 0) { s_tmp[0] = 0; s_tmp[1] = 0; }    // all == 0: no key at all
    __syncthreads();
    if (tot > 0 && w2 >= acc && w2 < acc + tot) {            // exactly one thread
        int bsel = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (w2 >= acc + c[j] && j < 7) { acc += c[j]; bsel = j + 1; }
            else break;
        }
        s_tmp[0] = (uint32_t)(8 * threadIdx.x + bsel);
        s_tmp[1] = w2 - acc;
    }
    __syncthreads();
    const uint32_t prefix = s_tmp[0];
    const uint32_t want1 = s_tmp[1];
    // ---- second pass: lower 5 bits of the keys in that bin
    if (threadIdx.x < 32) hist[threadIdx.x] = 0;
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) {
        const uint32_t k = get(i);
        if (k <= 0xFFFFu && (k >> 5) == prefix) atomicAdd(&hist[k & 31], 1u);
    }
    __syncthreads();
    if (warp == 0) {
        const uint32_t v = hist[lane];
        uint32_t in2 = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, in2, d);
            if (lane >= d) in2 += t;
        }
        const uint32_t all2 = __shfl_sync(0xFFFFFFFFu, in2, 31);
        const uint32_t w3 = want1 < all2 ? want1 : (all2 ? all2 - 1 : 0);
        if (all2 == 0 && lane == 0) s_tmp[0] = 0;
        if (v > 0 && w3 >= in2 - v && w3 < in2) s_tmp[0] = (uint32_t)lane;
    }
    __syncthreads();
    const uint32_t low = s_tmp[0];
    __syncthreads();                                         // s_tmp and hist are free for the next call
    return (prefix << 5) | low;
}

// The same select for keys that sit in shared memory (16-byte aligned), read eight at a time, for
// two ranks at once: both share the first-pass histogram and each gets 32 bins in the second pass.  Every key
// counts here, NaN patterns too: as keys they sort below -inf (sign set) or above +inf, so a caller
// whose ranks are meant among the non-NaN values adds the number of negative NaNs to them.
// s_tmp: 4 words.
__device__ void cta_select_keys(const unsigned short* keys, uint32_t n, uint32_t wantA, uint32_t wantB, uint32_t* hist,
                                uint32_t* s_tmp, uint32_t& outA, uint32_t& outB) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint4* k8 = reinterpret_cast<const uint4*>(keys);
    const uint32_t n8 = (n + 7) / 8;
    for (int i = threadIdx.x; i < 2048; i += blockDim.x) hist[i] = 0;
    if (threadIdx.x < 4) s_tmp[threadIdx.x] = 0;
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < n8; i += blockDim.x) {
        const uint4 r = k8[i];
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t k = (w[j >> 1] >> (16 * (j & 1))) & 0xFFFFu;
            if (8 * i + j < n) atomicAdd(&hist[k >> 5], 1u);
        }
    }
    __syncthreads();
    uint32_t c[8], tot = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) { c[j] = hist[8 * threadIdx.x + j]; tot += c[j]; }
    uint32_t inc = tot;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += t;
    }
    __syncthreads();
    if (lane == 31) hist[warp] = inc;
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        const uint32_t v = hist[w];
        if (w < warp) before += v;
        all += v;
    }
    const uint32_t first = before + inc - tot;               // keys in the bins before this thread's eight
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const uint32_t want = r ? wantB : wantA;
        const uint32_t w2 = want < all ? want : (all ? all - 1 : 0);
        if (tot > 0 && w2 >= first && w2 < first + tot) {    // exactly one thread per rank
            uint32_t acc = first;
            int bsel = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (w2 >= acc + c[j] && j < 7) { acc += c[j]; bsel = j + 1; }
                else break;
            }
            s_tmp[2 * r] = (uint32_t)(8 * threadIdx.x + bsel);
            s_tmp[2 * r + 1] = w2 - acc;
        }
    }
    __syncthreads();
    const uint32_t prefA = s_tmp[0], want1A = s_tmp[1], prefB = s_tmp[2], want1B = s_tmp[3];
    if (threadIdx.x < 64) hist[threadIdx.x] = 0;
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < n8; i += blockDim.x) {
        const uint4 r = k8[i];
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t k = (w[j >> 1] >> (16 * (j & 1))) & 0xFFFFu;
            if (8 * i + j < n) {
                if ((k >> 5) == prefA) atomicAdd(&hist[k & 31], 1u);
                if ((k >> 5) == prefB) atomicAdd(&hist[32 + (k & 31)], 1u);
            }
        }
    }
    __syncthreads();
    if (warp < 2) {                                          // warp 0: rank A, warp 1: rank B
        const uint32_t v = hist[32 * warp + lane];
        uint32_t in2 = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, in2, d);
            if (lane >= d) in2 += t;
        }
        const uint32_t all2 = __shfl_sync(0xFFFFFFFFu, in2, 31);
        const uint32_t want1 = warp ? want1B : want1A;
        const uint32_t w3 = want1 < all2 ? want1 : (all2 ? all2 - 1 : 0);
        if (all2 == 0 && lane == 0) s_tmp[2 * warp] = 0;
        if (v > 0 && w3 >= in2 - v && w3 < in2) s_tmp[2 * warp] = (uint32_t)lane;
    }
    __syncthreads();
    outA = (prefA << 5) | s_tmp[0];
    outB = (prefB << 5) | s_tmp[2];
    __syncthreads();
}

__device__ __forceinline__ unsigned long long rank_k(double alpha, unsigned long long N) {
    unsigned long long k = (unsigned long long)floor(alpha * (double)N / 2.0);
    if (N > 0 && k > (N - 1) / 2) k = (N - 1) / 2;
    return k;
}

// ---- 1. sample: brackets (or the exact answer when the sample is the whole problem)
__global__ void __launch_bounds__(256) thr_sample_kernel(const ThrArgs a) {
    const int bhx = blockIdx.x, bh = bhx >> 1, x = bhx & 1;
    __shared__ __align__(16) unsigned short s_keys[SAMPLE_TOKENS * 128];
    __shared__ uint32_t hist[2048], s_tmp[4], s_cnt[2];
    const int b_idx = bh / a.H, h_idx = bh % a.H;
    const __half* X = a.X[x] + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh;
    const int ns = a.T < SAMPLE_TOKENS ? a.T : SAMPLE_TOKENS;
    const int M = ns * a.D;
    if (threadIdx.x < 2) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    uint32_t nn = 0, nneg = 0;                                  // NaNs, NaNs with the sign set
    for (int i = threadIdx.x; i < M / 8; i += blockDim.x) {    // 16-byte pieces
        const int s = (i * 8) / a.D, c = (i * 8) % a.D;
        const long t = (long)s * a.T / ns;                        // tokens spread over the sequence
        const uint4 r = *reinterpret_cast<const uint4*>(X + (size_t)t * a.st + c);
        uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t mag = w[j] & 0x7FFF7FFFu;
            const uint32_t nan_lo = (mag & 0xFFFFu) > 0x7C00u, nan_hi = (mag >> 16) > 0x7C00u;
            nn += nan_lo + nan_hi;
            nneg += (nan_lo & (w[j] >> 15)) + (nan_hi & (w[j] >> 31));
            // keys of both halves: a set sign flips all 16 bits, a clear one only the sign bit
            const uint32_t neg = ((w[j] >> 15) & 0x00010001u) * 0xFFFFu;
            w[j] ^= neg | 0x80008000u;
        }
        *reinterpret_cast<uint4*>(&s_keys[8 * i]) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    if (nn) { atomicAdd(&s_cnt[0], nn); atomicAdd(&s_cnt[1], nneg); }
    __syncthreads();
    const uint32_t Mv = (uint32_t)M - s_cnt[0];                    // non-NaN sample values
    const uint32_t n_neg_nan = s_cnt[1];
    Problem* pr = a.prob + bhx;
    const bool whole = (ns == a.T);
    if (Mv == 0) {
        if (threadIdx.x == 0) {
            pr->klo = 0; pr->khi = 0xFFFF; pr->cnt[0] = pr->cnt[1] = 0; pr->nan = 0; pr->overflow = 0; pr->done = whole ? 1u : 0u;
            if (whole) { a.thr[(size_t)bh * 4 + 2 * x] = 0.f; a.thr[(size_t)bh * 4 + 2 * x + 1] = 0.f; }
        }
        return;
    }
    uint32_t r_lo, r_hi;
    if (whole) {
        const unsigned long long k = rank_k(a.alpha, Mv);
        r_lo = (uint32_t)k; r_hi = (uint32_t)(Mv - 1 - k);
    } else {
        // rank of 1.25 times the wanted tail mass plus four standard deviations of the sample count (a wider bracket
        // makes the scan set aside more pieces: 2.0 times costs 7 % more time on stationary data; a bracket that
        // turns out too tight only sends that problem to the exact two-pass select)
        const double f2 = 1.25 * 0.5 * a.alpha * (double)Mv;
        uint32_t r = (uint32_t)ceil(f2 + 4.0 * sqrt(f2 + 1.0) + 2.0);
        if (r > (Mv - 1) / 2) r = (Mv - 1) / 2;
        r_lo = r; r_hi = Mv - 1 - r;
    }
    uint32_t klo, khi;
    cta_select_keys(s_keys, (uint32_t)M, r_lo + n_neg_nan, r_hi + n_neg_nan, hist, s_tmp, klo, khi);
    if (threadIdx.x == 0) {
        pr->klo = klo; pr->khi = khi; pr->cnt[0] = pr->cnt[1] = 0; pr->nan = 0; pr->overflow = 0; pr->done = whole ? 1u : 0u;
        if (whole) {
            a.thr[(size_t)bh * 4 + 2 * x] = float_of_key(klo);
            a.thr[(size_t)bh * 4 + 2 * x + 1] = float_of_key(khi);
        }
    }
}

// ---- 2. the one pass over the data: compaction of the tail candidates.
// Almost all entries are inside [lo, hi], so the pass is a cheap filter first: a 16-byte piece whose smallest entry is
// at least lo and whose largest is at most hi (NaN-propagating min / max, so a NaN fails both) is dropped; the others
// (about one in ten at alpha = 1 %) are set aside in a buffer of the warp's own, and when enough of them have come
// together the warp looks at them entry by entry with all lanes busy.  Nothing in the loop needs the other warps:
// no CTA barrier, one shared-memory reservation per warp, tail and batch of set-aside pieces.
__global__ void __launch_bounds__(256) thr_scan_kernel(const ThrArgs a) {
    const int bhx = blockIdx.y, bh = bhx >> 1, x = bhx & 1;
    Problem* pr = a.prob + bhx;
    if (pr->done) return;
    __shared__ unsigned short s_list[2][CTA_LIST];
    __shared__ uint4 s_flag[8][WARP_FLAGS];                   // per warp: pieces with something outside [lo, hi]
    __shared__ uint32_t s_n[2], s_base[2], s_nan;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned lt = (1u << lane) - 1u;
    if (threadIdx.x < 2) s_n[threadIdx.x] = 0;
    if (threadIdx.x == 2) s_nan = 0;
    __syncthreads();
    const float flo = float_of_key(pr->klo), fhi = float_of_key(pr->khi);
    const __half2 lo2 = __float2half2_rn(flo), hi2 = __float2half2_rn(fhi);   // exact: both are binary16 values
    const int b_idx = bh / a.H, h_idx = bh % a.H;
    const int t0 = blockIdx.x * a.scan_tokens, ntok = min(a.T, t0 + a.scan_tokens) - t0;
    const int tok_shift = 31 - __clz(a.D / 8);                   // 16-byte pieces per token is a power of two (4, 8, 16)
    // thread tid looks at piece (tid mod pieces per token) of tokens tid >> tok_shift, + 256 >> tok_shift, ...
    int tok = (int)threadIdx.x >> tok_shift;
    const int tok_step = 256 >> tok_shift;
    const __half* ptr = (x ? a.X[1] : a.X[0]) + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh + (size_t)(t0 + tok) * a.st +
                        (((int)threadIdx.x & ((1 << tok_shift) - 1)) << 3);
    const size_t ptr_step = (size_t)tok_step * a.st;
    uint4* wflag = s_flag[warp];
    uint32_t nflag = 0;      // pieces set aside by this warp (the same in all its lanes)
    uint32_t nnan = 0;

    for (int c0 = 0; c0 < ntok; c0 += 4 * tok_step) {
        // four independent 16-byte loads per thread before any of them is looked at
        uint4 raw[4];
        bool in_range[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            in_range[u] = tok + u * tok_step < ntok;
            raw[u] = make_uint4(0, 0, 0, 0);
            if (in_range[u]) raw[u] = *reinterpret_cast<const uint4*>(ptr + u * ptr_step);
        }
        tok += 4 * tok_step;
        ptr += 4 * ptr_step;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const __half2 v0 = h2_of(raw[u].x), v1 = h2_of(raw[u].y), v2 = h2_of(raw[u].z), v3 = h2_of(raw[u].w);
            const __half2 mn = __hmin2_nan(__hmin2_nan(v0, v1), __hmin2_nan(v2, v3));
            const __half2 mx = __hmax2_nan(__hmax2_nan(v0, v1), __hmax2_nan(v2, v3));
            const bool flag = in_range[u] && !(__hbge2(mn, lo2) && __hble2(mx, hi2));
            const unsigned bal = __ballot_sync(0xFFFFFFFFu, flag);
            if (flag) wflag[nflag + __popc(bal & lt)] = raw[u];
            nflag += (uint32_t)__popc(bal);
        }
        __syncwarp();
        // the next round may set aside 128 more; the last round empties the buffer
        const bool last_round = c0 + 4 * tok_step >= ntok;
        if (!(nflag > (uint32_t)(WARP_FLAGS - 128) || last_round)) continue;
        // whole batches of 32 only (every lane busy); what is left over stays in the buffer for the next time,
        // except in the last round
        const uint32_t ntake = last_round ? nflag : (nflag & ~31u);
        // the warp's set-aside pieces entry by entry: per lane the entries below lo, above hi and NaN; one reservation
        // per tail for the whole batch, then every lane writes its keys
        for (uint32_t i0 = 0; i0 < ntake; i0 += 32) {
            const bool have = i0 + lane < ntake;
            const uint4 r = have ? wflag[i0 + lane] : make_uint4(0, 0, 0, 0);
            const uint32_t w[4] = {r.x, r.y, r.z, r.w};
            uint32_t below = 0, above = 0, nans = 0;              // bit j / 16 + j: low / high half of word j
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const __half2 v = h2_of(w[j]);
                const uint32_t ge = __hge2_mask(v, lo2), le = __hle2_mask(v, hi2);   // a NaN compares false twice
                below |= (~ge & le & 0x00010001u) << j;
                above |= (ge & ~le & 0x00010001u) << j;
                nans |= (~(ge | le) & 0x00010001u) << j;
            }
            if (!have) { below = 0; above = 0; nans = 0; }
            nnan += (uint32_t)__popc(nans);
            const uint32_t pk = (uint32_t)__popc(below) | ((uint32_t)__popc(above) << 16);   // at most 8 each
            uint32_t inc = pk;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= d) inc += t;
            }
            const uint32_t tot = __shfl_sync(0xFFFFFFFFu, inc, 31);
            uint32_t b0 = 0, b1 = 0;
            if (lane == 0) {
                if (tot & 0xFFFFu) b0 = atomicAdd(&s_n[0], tot & 0xFFFFu);
                if (tot >> 16) b1 = atomicAdd(&s_n[1], tot >> 16);
            }
            uint32_t pos[2] = {__shfl_sync(0xFFFFFFFFu, b0, 0) + ((inc - pk) & 0xFFFFu), __shfl_sync(0xFFFFFFFFu, b1, 0) + ((inc - pk) >> 16)};
#pragma unroll
            for (int side = 0; side < 2; ++side) {
                uint32_t m = side ? above : below;
                while (m) {
                    const int bit = __ffs(m) - 1;
                    m &= m - 1;
                    const int j = bit & 3;
                    const uint32_t wj = (j & 2) ? ((j & 1) ? w[3] : w[2]) : ((j & 1) ? w[1] : w[0]);
                    const unsigned short h = (unsigned short)((bit >> 4) ? (wj >> 16) : (wj & 0xFFFFu));
                    if (pos[side] < (uint32_t)CTA_LIST) s_list[side][pos[side]] = (unsigned short)key_of(h);
                    ++pos[side];
                }
            }
        }
        const uint32_t left = nflag - ntake;           // fewer than 32
        uint4 keep = make_uint4(0, 0, 0, 0);
        if ((uint32_t)lane < left) keep = wflag[ntake + lane];
        __syncwarp();
        if ((uint32_t)lane < left) wflag[lane] = keep;
        nflag = left;
        __syncwarp();     // the rest of the buffer is free again
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) nnan += __shfl_xor_sync(0xFFFFFFFFu, nnan, o);
    if (lane == 0 && nnan) atomicAdd(&s_nan, nnan);
    __syncthreads();
    if (threadIdx.x < 2) s_base[threadIdx.x] = s_n[threadIdx.x] ? atomicAdd(&pr->cnt[threadIdx.x], s_n[threadIdx.x]) : 0u;
    if (threadIdx.x == 2 && s_nan) atomicAdd(&pr->nan, s_nan);
    __syncthreads();
#pragma unroll
    for (int side = 0; side < 2; ++side) {
        const uint32_t cnt = s_n[side];
        // a CTA list that overflowed leaves a hole in the global list: the select kernel falls back for that tail
        if (cnt > CTA_LIST) { if (threadIdx.x == 0) atomicOr(&pr->overflow, 1u << side); continue; }
        unsigned short* dst = a.list + ((size_t)bhx * 2 + side) * a.cap;
        for (uint32_t i = threadIdx.x; i < cnt; i += blockDim.x) {
            const uint32_t pos = s_base[side] + i;
            if (pos < a.cap) dst[pos] = s_list[side][i];
        }
    }
}

// ---- 3. exact select among the candidates, exact fallback over the data when that is not possible.
// One CTA per (problem, tail): the two tails are independent order statistics.
__global__ void __launch_bounds__(256) thr_select_kernel(const ThrArgs a) {
    const int bhx = blockIdx.x >> 1, side = blockIdx.x & 1, bh = bhx >> 1, x = bhx & 1;
    Problem* pr = a.prob + bhx;
    if (pr->done) return;
    __shared__ uint32_t hist[2048], s_tmp[4];
    __shared__ __align__(16) unsigned short s_keys[SELECT_KEYS];
    const unsigned long long total = (unsigned long long)a.T * a.D;
    const unsigned long long N = total - pr->nan;
    float res = 0.f;
    if (N > 0) {
        const unsigned long long k = rank_k(a.alpha, N);
        const uint32_t c = pr->cnt[side];
        if (c > k && c <= a.cap && !((pr->overflow >> side) & 1u)) {
            // rank k from below in the low list, rank k from above in the high list
            const uint32_t want = side == 0 ? (uint32_t)k : (uint32_t)(c - 1 - k);
            const unsigned short* l = a.list + ((size_t)bhx * 2 + side) * a.cap;   // 16-byte aligned
            if (c <= (uint32_t)SELECT_KEYS) {
                // the usual case: the list fits in shared memory; bring it in with independent wide loads
                for (uint32_t i = threadIdx.x; i < (c + 7) / 8; i += blockDim.x)
                    reinterpret_cast<uint4*>(s_keys)[i] = reinterpret_cast<const uint4*>(l)[i];
                __syncthreads();
                uint32_t key, same;
                cta_select_keys(s_keys, c, want, want, hist, s_tmp, key, same);
                res = float_of_key(key);
            } else {
                auto getg = [&](uint32_t i) -> uint32_t { return l[i]; };
                res = float_of_key(cta_select(getg, c, want, hist, s_tmp));
            }
        } else {
            // bracket too tight or list overflow: two-pass radix select over this problem's data
            const int b_idx = bh / a.H, h_idx = bh % a.H;
            const __half* X = a.X[x] + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh;
            const int D = a.D;
            auto getx = [&](uint32_t i) -> uint32_t {
                const unsigned short h = __half_as_ushort(X[(size_t)(i / D) * a.st + (i % D)]);
                return is_nan_bits(h) ? 0x10000u : key_of(h);
            };
            res = float_of_key(cta_select(getx, (uint32_t)total, side == 0 ? (uint32_t)k : (uint32_t)(N - 1 - k), hist, s_tmp));
        }
    }
    if (threadIdx.x == 0) a.thr[(size_t)bh * 4 + 2 * x + side] = res;
}

// Tokens per CTA of the scan: as many as keep the expected number of candidates per tail (1.25 times the tail mass
// plus the bracket's slack) well inside the CTA's list; a CTA that overflows sends its problem to the exact fallback.
int scan_tokens_for(double alpha, int D) {
    const double per_token = (0.625 * alpha + 0.004) * D;
    int tokens = SCAN_TOKENS_MAX;
    while (tokens > 64 && per_token * tokens > 0.6 * CTA_LIST) tokens /= 2;
    return tokens;
}

uint32_t list_capacity(const qaq_config* cfg, int n_tokens) {
    // expected candidates per tail: (alpha + margin) * N; keep three times that, at least 4096
    const double N = (double)n_tokens * cfg->head_dim;
    double want = 3.0 * (cfg->outlier_frac * N + 8.0 * sqrt(cfg->outlier_frac * N + 64.0) + 64.0) + 4096.0;
    if (want > N) want = N;
    uint32_t cap = (uint32_t)want;
    return (cap + 63u) & ~63u;
}

}  // namespace

extern "C" qaq_status qaq_thresholds_workspace_bytes(const qaq_config* cfg, size_t* host_out) {
    if (!cfg || !host_out || cfg->batch < 1 || cfg->heads < 1 || cfg->max_tokens < 1) return QAQ_ERR_INVALID_ARG;
    const size_t P = (size_t)cfg->batch * cfg->heads * 2;
    *host_out = P * sizeof(Problem) + P * 2 * (size_t)list_capacity(cfg, cfg->max_tokens) * sizeof(unsigned short) + 256;
    return QAQ_OK;
}

extern "C" qaq_status qaq_outlier_thresholds(const qaq_config* cfg, const void* K, const void* V, long stride_b,
                                             long stride_h, long stride_t, int n_tokens, float* thr, void* ws,
                                             size_t ws_bytes, void* stream) {
    if (!cfg || !K || !V || !thr || !ws || n_tokens < 1) return QAQ_ERR_INVALID_ARG;
    if (!qaq_dim_ok(cfg->head_dim)) return QAQ_ERR_UNSUPPORTED_SHAPE;
    if (!(cfg->outlier_frac >= 0.0 && cfg->outlier_frac <= 1.0)) return QAQ_ERR_INVALID_ARG;
    if ((double)n_tokens * cfg->head_dim >= 4.0e9) return QAQ_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)K & 15) || ((uintptr_t)V & 15) || (stride_b & 7) || (stride_h & 7) || (stride_t & 7) ||
        stride_t < cfg->head_dim)
        return QAQ_ERR_INVALID_ARG;
    size_t need = 0;
    qaq_thresholds_workspace_bytes(cfg, &need);
    if (ws_bytes < need || ((uintptr_t)ws & 15)) return QAQ_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    const int BH = cfg->batch * cfg->heads;
    ThrArgs a;
    a.X[0] = (const __half*)K; a.X[1] = (const __half*)V;
    a.sb = stride_b; a.sh = stride_h; a.st = stride_t;
    a.H = cfg->heads; a.T = n_tokens; a.D = cfg->head_dim; a.alpha = cfg->outlier_frac;
    a.prob = (Problem*)ws;
    // the candidate lists take whatever the workspace offers beyond the problem records
    const size_t head = ((size_t)BH * 2 * sizeof(Problem) + 255) / 256 * 256;
    const size_t per_list = (ws_bytes - head) / ((size_t)BH * 4 * sizeof(unsigned short));
    a.cap = (uint32_t)(per_list > 0x3FFFFFC0u ? 0x3FFFFFC0u : per_list) & ~63u;
    if (a.cap < 64) return QAQ_ERR_WORKSPACE;
    a.list = (unsigned short*)((char*)ws + head);
    a.thr = thr;
    a.scan_tokens = SCAN_TOKENS_MAX;
    thr_sample_kernel<<<BH * 2, 256, 0, s>>>(a);
    if (n_tokens > SAMPLE_TOKENS) {
        a.scan_tokens = scan_tokens_for(cfg->outlier_frac, cfg->head_dim);
        dim3 grid((n_tokens + a.scan_tokens - 1) / a.scan_tokens, BH * 2);
        thr_scan_kernel<<<grid, 256, 0, s>>>(a);
        thr_select_kernel<<<BH * 4, 256, 0, s>>>(a);
    }
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}
