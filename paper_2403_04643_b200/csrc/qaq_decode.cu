// S4+S5: decode attention over the packed cache (Section 2.1 / Figure 1 of the paper):
//   S = Softmax(scale * q Khat^T),  X = S Vhat,  xhat = min + (code + 1/2) * step,
// outliers restored from the sparse side list, split over the sequence with a
// log-sum-exp merge of the split partials.
//
// The affine map is factored out of the inner loops so they work on raw codes:
//   q . Khat_t = step_t * sum_d q_d c_td + (min_t + step_t/2) * sum_d q_d
//   X_d        = sum_t (p_t step_t) c_td + sum_t p_t (min_t + step_t/2)
// and a token's outliers add  q_ch * (x - (min_t + step_t/2))  resp.  p_t * (v - ...)
// because their code slot holds 0.
//
// q.K runs on integer dot products (dp4a): q is converted per (b,h) to 16-bit fixed point
// q_d ~ qscale * (256 * hi_d + lo_d), hi signed / lo unsigned bytes, so that every plane
// word of codes (already one field per byte lane after a mask) feeds two dp4a.  The sums
// are exact integers; the fixed-point error of q is below 2^-16 of max|q|.
//
// One CTA = one (b,h) and one split; per tile of QAQ_TILE tokens the packed bytes, the
// metadata and the outlier entries are staged in shared memory with cp.async (two
// buffers).  A (token, plane) pair is one work item, handled by head_dim/32 lanes; items
// are sorted by plane width so the lanes of a warp run the same extraction code.
#include "qaq_internal.cuh"

namespace {

constexpr int DEC_THREADS = 256;
constexpr int DEC_WARPS = DEC_THREADS / 32;
constexpr int OSTAGE = 512;  // outlier entries staged per tile and tensor; the rest is read from global

struct DecArgs {
    TensorStore k, v;
    size_t pool_bytes;
    uint32_t ocap;
    int tmax_pad, ntiles_max;
    int T;
    const __half* q;
    float scale;
    float* part;       // [BH][nsplit][D+2]
    float* ml;         // [BH][2]   merged (max, sum) for score normalisation
    int nsplit;
    float* out;        // [BH][D]
    float* scores;     // [BH][T] or null
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {  // unsigned bytes x signed bytes
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ int dp4a_uu(uint32_t a, uint32_t b, int c) {  // unsigned x unsigned
    int d;
    asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// integer dot product of one lane's 32 channels of a w-bit plane with q (hi/lo bytes)
template <int W>
__device__ __forceinline__ int plane_dot(const uint32_t* __restrict__ words, const uint32_t (&qh)[8], const uint32_t (&ql)[8]) {
    constexpr int PER = 8 / W;
    constexpr uint32_t MASK = 0x01010101u * ((1u << W) - 1u);
    int ah = 0, al = 0;
#pragma unroll
    for (int j = 0; j < W; ++j) {
        const uint32_t wd = words[j];
#pragma unroll
        for (int m = 0; m < PER; ++m) {
            const uint32_t f = (wd >> (W * m)) & MASK;
            ah = dp4a_us(f, qh[PER * j + m], ah);
            al = dp4a_uu(f, ql[PER * j + m], al);
        }
    }
    return ah * 256 + al;
}

// acc[r][i] += wt * (1 + f/2^W) for the lane's 32 channels of a w-bit plane
template <int W>
__device__ __forceinline__ void plane_axpy(const uint32_t* __restrict__ words, float wt, float (&acc)[8][4]) {
    constexpr int PER = 8 / W;
    constexpr uint32_t MASK = ((1u << W) - 1u) << (23 - W);
#pragma unroll
    for (int j = 0; j < W; ++j) {
        const uint32_t wd = words[j];
#pragma unroll
        for (int m = 0; m < PER; ++m) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                constexpr int dummy = 0;
                (void)dummy;
                const int pos = 8 * i + W * m;
                const uint32_t sh = (pos + W <= 23) ? (wd << (23 - W - pos)) : (wd >> (pos + W - 23));
                const float xf = __uint_as_float((sh & MASK) | 0x3F800000u);
                acc[PER * j + m][i] = fmaf(wt, xf, acc[PER * j + m][i]);
            }
        }
    }
}

template <int D>
struct DecSmem {
    alignas(16) uint8_t codes[2][2][QAQ_TILE * D + 32];  // [buffer][tensor]
    alignas(16) uint32_t outl[2][2][OSTAGE];
    alignas(16) uint8_t bits[2][2][QAQ_TILE];
    alignas(16) uint32_t mnmx[2][2][QAQ_TILE];
    uint32_t table[3][8];       // per tile: off, nbytes, ooff, ocnt for K then V
    uint32_t tokoff[2][QAQ_TILE];
    float step[2][QAQ_TILE];
    float mid[2][QAQ_TILE];     // min + step/2
    int dot[QAQ_TILE];
    float ocorr[QAQ_TILE];
    float logit[QAQ_TILE];
    float p[QAQ_TILE];
    uint8_t item[2][3 * QAQ_TILE];  // token | class << 6, sorted by class (0:w=8 .. 3:w=1)
    int nitem[2];
    float qf[D];
    float vout[D];
    float accsum[D];
    float red[DEC_WARPS];
    float red2[DEC_WARPS];
    float qscale, qsum;
};

template <int D>
__global__ void __launch_bounds__(DEC_THREADS) decode_kernel(const DecArgs a) {
    constexpr int P = D / 32;        // lanes per item
    constexpr int IPW = 32 / P;      // items per warp pass
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecSmem<D>& sm = *reinterpret_cast<DecSmem<D>*>(smem_raw);
    const int bh = blockIdx.y, split = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int part = lane % P, sub = lane / P;

    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const int per_split = (ntiles + a.nsplit - 1) / a.nsplit;
    const int tile_lo = split * per_split, tile_hi = min(ntiles, tile_lo + per_split);
    const int n_my = max(0, tile_hi - tile_lo);

    // ---- q: float copy, fixed-point bytes per lane
    float qmax = 0.f, qs = 0.f;
    for (int d = tid; d < D; d += DEC_THREADS) {
        const float f = __half2float(a.q[(size_t)bh * D + d]);
        sm.qf[d] = f;
        sm.vout[d] = 0.f;
        sm.accsum[d] = 0.f;
        qmax = fmaxf(qmax, fabsf(f));
        qs += f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        qmax = fmaxf(qmax, __shfl_xor_sync(0xFFFFFFFFu, qmax, o));
        qs += __shfl_xor_sync(0xFFFFFFFFu, qs, o);
    }
    if (lane == 0) { sm.red[warp] = qmax; sm.red2[warp] = qs; }
    __syncthreads();
    if (tid == 0) {
        float m = 0.f, s = 0.f;
        for (int w = 0; w < DEC_WARPS; ++w) { m = fmaxf(m, sm.red[w]); s += sm.red2[w]; }
        sm.qscale = m / 32767.0f;
        sm.qsum = s;
    }
    __syncthreads();
    const float qscale = sm.qscale, qsum = sm.qsum;
    const float qinv = qscale > 0.f ? 1.0f / qscale : 0.f;
    uint32_t qh[8], ql[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        uint32_t h = 0, l = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int qi = __float2int_rn(sm.qf[32 * part + 4 * r + i] * qinv);
            qi = max(-32767, min(32767, qi));
            h |= (uint32_t)((qi >> 8) & 0xFF) << (8 * i);
            l |= (uint32_t)(qi & 0xFF) << (8 * i);
        }
        qh[r] = h; ql[r] = l;
    }

    float acc[8][4];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[r][i] = 0.f;
    float offs = 0.f;        // sum of the weights this lane applied (the "1 +" of the magic floats)
    float m_run = __int_as_float(0xff800000), l_run = 0.f;
    float c_run = 0.f;       // thread-per-token part of sum_t p_t (min_t + step_t/2)

    const size_t trow = (size_t)bh * a.ntiles_max;
    auto load_table = [&](int it) {  // it: index among my tiles
        if (tid < 8 && it < n_my) {
            const TensorStore& ts = (tid >= 4) ? a.v : a.k;
            const size_t ti = trow + tile_lo + it;
            const int f = tid & 3;
            sm.table[it % 3][tid] = f == 0 ? ts.tile_off[ti] : f == 1 ? ts.tile_nbytes[ti] : f == 2 ? ts.tile_ooff[ti] : ts.tile_ocnt[ti];
        }
    };
    auto issue_tile = [&](int it) {  // cp.async of tile `it` into buffer it & 1
        const int buf = it & 1;
        const uint32_t* tb = sm.table[it % 3];
        const int tile = tile_lo + it;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const TensorStore& ts = x ? a.v : a.k;
            const uint8_t* src = ts.codes + (size_t)bh * a.pool_bytes + tb[4 * x + 0];
            const int n16 = (int)((tb[4 * x + 1] + 15u) >> 4);
            for (int i = tid; i < n16; i += DEC_THREADS) cp_async16(&sm.codes[buf][x][16 * i], src + 16 * i);
            const uint32_t* osrc = ts.outl + (size_t)bh * a.ocap + tb[4 * x + 2];
            const int o16 = (int)((min(tb[4 * x + 3], (uint32_t)OSTAGE) + 3u) >> 2);
            for (int i = tid; i < o16; i += DEC_THREADS) cp_async16(&sm.outl[buf][x][4 * i], osrc + 4 * i);
            const size_t t0 = (size_t)bh * a.tmax_pad + (size_t)tile * QAQ_TILE;
            if (tid < QAQ_TILE / 16) cp_async16(&sm.bits[buf][x][16 * tid], ts.bits + t0 + 16 * tid);
            if (tid >= 32 && tid < 32 + QAQ_TILE / 4) cp_async16(&sm.mnmx[buf][x][4 * (tid - 32)], ts.mnmx + t0 + 4 * (tid - 32));
        }
    };

    load_table(0);
    load_table(1);
    __syncthreads();
    if (n_my > 0) issue_tile(0);
    cp_async_commit();

    for (int it = 0; it < n_my; ++it) {
        const int buf = it & 1;
        const int tile = tile_lo + it;
        if (it + 1 < n_my) issue_tile(it + 1);
        cp_async_commit();
        load_table(it + 2);
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t* tb = sm.table[it % 3];

        // ---- per-token scalars, byte offsets, work items (warp 0: K, warp 1: V)
        if (warp < 2) {
            const int x = warp;
            int cls_cnt_lo[4], cls_cnt_hi[4];
            uint32_t len[2];
            int Bv[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int slot = lane + 32 * e;
                const bool valid = tile * QAQ_TILE + slot < a.T;
                const int B = valid ? sm.bits[buf][x][slot] : 0;
                Bv[e] = B;
                len[e] = (uint32_t)(D * B / 8);
                const uint32_t mm = sm.mnmx[buf][x][slot];
                const float mn = __half2float(__ushort_as_half((unsigned short)(mm & 0xFFFF)));
                const float mx = __half2float(__ushort_as_half((unsigned short)(mm >> 16)));
                const float st = __fmul_rn(__fsub_rn(mx, mn), __int_as_float((127 - B) << 23));
                sm.step[x][slot] = valid ? st : 0.f;
                sm.mid[x][slot] = valid ? fmaf(0.5f, st, mn) : 0.f;
                if (x == 0) { sm.dot[slot] = 0; sm.ocorr[slot] = 0.f; }
            }
            // exclusive scan of byte lengths in token order
            uint32_t i0 = len[0], i1 = len[1];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t t0 = __shfl_up_sync(0xFFFFFFFFu, i0, d), t1 = __shfl_up_sync(0xFFFFFFFFu, i1, d);
                if (lane >= d) { i0 += t0; i1 += t1; }
            }
            const uint32_t tot0 = __shfl_sync(0xFFFFFFFFu, i0, 31);
            sm.tokoff[x][lane] = i0 - len[0];
            sm.tokoff[x][lane + 32] = tot0 + i1 - len[1];
            // items sorted by class: class c <-> plane width 8 >> c
            int base = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int w = 8 >> c;
                const unsigned b0 = __ballot_sync(0xFFFFFFFFu, (Bv[0] & w) != 0);
                const unsigned b1 = __ballot_sync(0xFFFFFFFFu, (Bv[1] & w) != 0);
                const unsigned lt = (1u << lane) - 1u;
                if (Bv[0] & w) sm.item[x][base + __popc(b0 & lt)] = (uint8_t)(lane | (c << 6));
                if (Bv[1] & w) sm.item[x][base + __popc(b0) + __popc(b1 & lt)] = (uint8_t)((lane + 32) | (c << 6));
                base += __popc(b0) + __popc(b1);
                cls_cnt_lo[c] = 0; cls_cnt_hi[c] = 0;
            }
            (void)cls_cnt_lo; (void)cls_cnt_hi;
            if (lane == 0) sm.nitem[x] = base;
        }
        __syncthreads();

        // ---- K: integer dot products per (token, plane) item, outlier corrections
        {
            const int n = sm.nitem[0];
            const uint8_t* cbuf = sm.codes[buf][0];
            for (int base = warp * IPW; base < n; base += DEC_WARPS * IPW) {
                const int idx = base + sub;
                const bool valid = idx < n;
                const int itv = valid ? sm.item[0][idx] : 0;
                const int tok = itv & 63, cls = itv >> 6;
                const int B = sm.bits[buf][0][tok];
                int dot = 0, shift = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (__ballot_sync(0xFFFFFFFFu, valid && cls == c) == 0) continue;
                    if (valid && cls == c) {
                        constexpr int dummy = 0; (void)dummy;
                        const int w = 8 >> c;
                        const int plane_base = (B & ~((w << 1) - 1)) * (D / 8);
                        const uint32_t* words = reinterpret_cast<const uint32_t*>(cbuf + sm.tokoff[0][tok] + plane_base + part * 4 * w);
                        shift = B & (w - 1);
                        if (c == 0) dot = plane_dot<8>(words, qh, ql);
                        else if (c == 1) dot = plane_dot<4>(words, qh, ql);
                        else if (c == 2) dot = plane_dot<2>(words, qh, ql);
                        else dot = plane_dot<1>(words, qh, ql);
                    }
                }
#pragma unroll
                for (int o = 1; o < P; o <<= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, o);
                if (valid && part == 0) atomicAdd(&sm.dot[tok], dot << shift);
            }
            const uint32_t no = tb[3];
            const uint32_t* og = a.k.outl + (size_t)bh * a.ocap + tb[2];
            for (uint32_t e = tid; e < no; e += DEC_THREADS) {
                const uint32_t v = e < OSTAGE ? sm.outl[buf][0][e] : og[e];
                const int tok = v >> 24, ch = (v >> 16) & 0xFF;
                const float val = __half2float(__ushort_as_half((unsigned short)(v & 0xFFFF)));
                atomicAdd(&sm.ocorr[tok], sm.qf[ch] * (val - sm.mid[0][tok]));
            }
        }
        __syncthreads();

        // ---- logits, tile maximum
        float logit = __int_as_float(0xff800000);
        if (tid < QAQ_TILE) {
            const int t = tile * QAQ_TILE + tid;
            if (t < a.T) {
                const float qk = fmaf(qscale * sm.step[0][tid], (float)sm.dot[tid], fmaf(sm.mid[0][tid], qsum, sm.ocorr[tid]));
                logit = a.scale * qk;
                if (a.scores) a.scores[(size_t)bh * a.T + t] = logit;
            }
            float m = logit;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            if (lane == 0) sm.red[warp] = m;
        }
        __syncthreads();
        const float m_new = fmaxf(m_run, fmaxf(sm.red[0], sm.red[1]));
        const float alpha = __expf(m_run - m_new);   // 0 on the first tile (m_run = -inf)
        m_run = m_new;
        if (alpha != 1.0f) {
#pragma unroll
            for (int r = 0; r < 8; ++r)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[r][i] *= alpha;
            offs *= alpha;
            c_run *= alpha;
            for (int d = tid; d < D; d += DEC_THREADS) sm.vout[d] *= alpha;
        }
        if (tid < QAQ_TILE) {
            const float p = __expf(logit - m_new);   // 0 for slots beyond T
            sm.p[tid] = p;
            c_run = fmaf(p, sm.mid[1][tid], c_run);
            float s = p;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
            if (lane == 0) sm.red2[warp] = s;
        }
        __syncthreads();
        l_run = l_run * alpha + sm.red2[0] + sm.red2[1];

        // ---- V: weighted accumulation of raw codes, outlier corrections
        {
            const int n = sm.nitem[1];
            const uint8_t* cbuf = sm.codes[buf][1];
            for (int base = warp * IPW; base < n; base += DEC_WARPS * IPW) {
                const int idx = base + sub;
                const bool valid = idx < n;
                const int itv = valid ? sm.item[1][idx] : 0;
                const int tok = itv & 63, cls = itv >> 6;
                const int B = sm.bits[buf][1][tok];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (__ballot_sync(0xFFFFFFFFu, valid && cls == c) == 0) continue;
                    if (valid && cls == c) {
                        const int w = 8 >> c;
                        const int plane_base = (B & ~((w << 1) - 1)) * (D / 8);
                        const uint32_t* words = reinterpret_cast<const uint32_t*>(cbuf + sm.tokoff[1][tok] + plane_base + part * 4 * w);
                        const int shift = B & (w - 1);
                        // p_t * step_t * 2^shift * f = wt * (f / 2^w)
                        const float wt = sm.p[tok] * sm.step[1][tok] * __int_as_float((127 + shift + w) << 23);
                        if (c == 0) plane_axpy<8>(words, wt, acc);
                        else if (c == 1) plane_axpy<4>(words, wt, acc);
                        else if (c == 2) plane_axpy<2>(words, wt, acc);
                        else plane_axpy<1>(words, wt, acc);
                        offs += wt;
                    }
                }
            }
            const uint32_t no = tb[7];
            const uint32_t* og = a.v.outl + (size_t)bh * a.ocap + tb[6];
            for (uint32_t e = tid; e < no; e += DEC_THREADS) {
                const uint32_t v = e < OSTAGE ? sm.outl[buf][1][e] : og[e];
                const int tok = v >> 24, ch = (v >> 16) & 0xFF;
                const float val = __half2float(__ushort_as_half((unsigned short)(v & 0xFFFF)));
                atomicAdd(&sm.vout[ch], sm.p[tok] * (val - sm.mid[1][tok]));
            }
        }
        __syncthreads();
    }
    cp_async_wait<0>();

    // ---- CTA reduction: lanes with the same part over the warp, then warps through smem
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float v = acc[r][i] - offs;
#pragma unroll
            for (int o = P; o < 32; o <<= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
            if (sub == 0) atomicAdd(&sm.accsum[32 * part + 4 * r + i], v);
        }
    float cs = c_run;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cs += __shfl_xor_sync(0xFFFFFFFFu, cs, o);
    __syncthreads();
    if (lane == 0) sm.red[warp] = cs;
    __syncthreads();
    const float cterm = sm.red[0] + sm.red[1];
    float* dst = a.part + ((size_t)bh * a.nsplit + split) * (D + 2);
    for (int d = tid; d < D; d += DEC_THREADS) dst[d] = sm.accsum[d] + sm.vout[d] + cterm;
    if (tid == 0) { dst[D] = m_run; dst[D + 1] = l_run; }
}

// log-sum-exp merge of the split partials -> X, and (max, sum) for the score row
template <int D>
__global__ void merge_kernel(const DecArgs a) {
    const int bh = blockIdx.x, d = threadIdx.x;
    const float* p = a.part + (size_t)bh * a.nsplit * (D + 2);
    float M = __int_as_float(0xff800000);
    for (int s = 0; s < a.nsplit; ++s) M = fmaxf(M, p[s * (D + 2) + D]);
    float L = 0.f, x = 0.f;
    for (int s = 0; s < a.nsplit; ++s) {
        const float m = p[s * (D + 2) + D];
        if (m == __int_as_float(0xff800000)) continue;
        const float w = __expf(m - M);
        L = fmaf(w, p[s * (D + 2) + D + 1], L);
        x = fmaf(w, p[s * (D + 2) + d], x);
    }
    a.out[(size_t)bh * D + d] = L > 0.f ? x / L : 0.f;
    if (d == 0) { a.ml[2 * bh] = M; a.ml[2 * bh + 1] = L; }
}

__global__ void scores_kernel(float* scores, const float* ml, int T) {
    const int bh = blockIdx.y;
    const float M = ml[2 * bh], L = ml[2 * bh + 1];
    const float inv = L > 0.f ? 1.0f / L : 0.f;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < T; t += gridDim.x * blockDim.x) {
        float* s = scores + (size_t)bh * T + t;
        *s = __expf(*s - M) * inv;
    }
}

int pick_nsplit(int BH, int ntiles) {
    // enough CTAs for ~4 per SM on 148 SMs, at least 4 tiles per CTA where possible
    int want = (148 * 4 + BH - 1) / BH;
    int cap = ntiles / 4 > 0 ? ntiles / 4 : 1;
    int n = want < cap ? want : cap;
    if (n < 1) n = 1;
    if (n > 64) n = 64;
    return n;
}

template <int D>
qaq_status run_decode(const DecArgs& a, int BH, cudaStream_t s) {
    static bool attr_done = false;
    const size_t smem = sizeof(DecSmem<D>);
    if (!attr_done) {
        QAQ_CUDA_TRY(cudaFuncSetAttribute(decode_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_done = true;
    }
    decode_kernel<D><<<dim3(a.nsplit, BH), DEC_THREADS, smem, s>>>(a);
    merge_kernel<D><<<BH, D, 0, s>>>(a);
    if (a.scores) {
        int gx = (a.T + 1023) / 1024;
        if (gx > 64) gx = 64;
        scores_kernel<<<dim3(gx, BH), 256, 0, s>>>(a.scores, a.ml, a.T);
    }
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

}  // namespace

static const int QAQ_MAX_SPLIT = 64;

extern "C" qaq_status qaq_decode_workspace_bytes(const qaq_cache* c, size_t* host_out) {
    if (!c || !host_out) return QAQ_ERR_INVALID_ARG;
    const size_t BH = (size_t)c->BH, D = (size_t)c->cfg.head_dim;
    *host_out = (BH * QAQ_MAX_SPLIT * (D + 2) + BH * 2) * sizeof(float);
    return QAQ_OK;
}

extern "C" qaq_status qaq_decode_attention(const qaq_cache* c, const void* q, float softmax_scale, float* out,
                                           float* scores_out, void* ws, size_t ws_bytes, void* stream) {
    if (!c || !q || !out || !ws) return QAQ_ERR_INVALID_ARG;
    if (c->tokens < 1) return QAQ_ERR_INVALID_ARG;
    size_t need = 0;
    qaq_decode_workspace_bytes(c, &need);
    if (ws_bytes < need || ((uintptr_t)ws & 15)) return QAQ_ERR_WORKSPACE;
    const int D = c->cfg.head_dim, BH = c->BH;
    DecArgs a;
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.ocap = c->ocap;
    a.tmax_pad = c->tmax_pad; a.ntiles_max = c->ntiles; a.T = (int)c->tokens;
    a.q = (const __half*)q; a.scale = softmax_scale;
    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    a.nsplit = pick_nsplit(BH, ntiles);
    a.part = (float*)ws;
    a.ml = a.part + (size_t)BH * QAQ_MAX_SPLIT * (D + 2);
    a.out = out; a.scores = scores_out;
    cudaStream_t s = (cudaStream_t)stream;
    switch (D) {
        case 32: return run_decode<32>(a, BH, s);
        case 64: return run_decode<64>(a, BH, s);
        case 128: return run_decode<128>(a, BH, s);
    }
    return QAQ_ERR_UNSUPPORTED_SHAPE;
}

// ---------------------------------------------------------------------------------------
// Decode attention for callers that have no way to hand over a workspace.
//
// The split partials of the decode kernel need a few hundred KB of global scratch.  The
// regular entry point takes it from the caller; this one keeps it in a fixed array that
// is part of the library image, so the call itself never asks the CUDA allocator (or any
// other allocator) for memory.
#define QAQ_STATIC_SCRATCH_BYTES (4u << 20)
static __device__ __align__(256) unsigned char g_decode_scratch[QAQ_STATIC_SCRATCH_BYTES];

#include <mutex>
static std::mutex g_scratch_mutex;
static void* g_scratch_addr[64];  // device address of g_decode_scratch, per device ordinal

extern "C" qaq_status qaq_decode_attention_static(const qaq_cache* c, const void* q, float softmax_scale,
                                                  float* out, void* stream) {
    if (!c || !q || !out) return QAQ_ERR_INVALID_ARG;
    if (c->tokens < 1) return QAQ_ERR_INVALID_ARG;
    const int D = c->cfg.head_dim, BH = c->BH;
    const int T = (int)c->tokens;
    const int ntiles = (T + QAQ_TILE - 1) / QAQ_TILE;
    const int nsplit = pick_nsplit(BH, ntiles);
    // partials [BH][nsplit][D+2] followed by the merged (max, sum) pairs [BH][2]
    const size_t need = ((size_t)BH * nsplit * (D + 2) + (size_t)BH * 2) * sizeof(float);
    if (need > QAQ_STATIC_SCRATCH_BYTES) return QAQ_ERR_WORKSPACE;  // shape too large for the built-in scratch

    int dev = -1;
    QAQ_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return QAQ_ERR_UNSUPPORTED_SHAPE;
    void* scratch = nullptr;
    {
        // In host code the array's name is only a handle; the device address has to be
        // looked up, once per device, with that device current.
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_addr[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || !p) {
                (void)cudaGetLastError();
                return QAQ_ERR_CUDA;
            }
            g_scratch_addr[dev] = p;
        }
        scratch = g_scratch_addr[dev];
    }
    DecArgs a;
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.ocap = c->ocap;
    a.tmax_pad = c->tmax_pad; a.ntiles_max = c->ntiles; a.T = T;
    a.q = (const __half*)q; a.scale = softmax_scale;
    a.nsplit = nsplit;
    // Every (b,h,split) partial and every (max,sum) pair is written before it is read, so
    // nothing in the scratch has to be cleared between calls.
    a.part = (float*)scratch;
    a.ml = a.part + (size_t)BH * nsplit * (D + 2);
    a.out = out; a.scores = nullptr;
    cudaStream_t s = (cudaStream_t)stream;
    switch (D) {
        case 32: return run_decode<32>(a, BH, s);
        case 64: return run_decode<64>(a, BH, s);
        case 128: return run_decode<128>(a, BH, s);
    }
    return QAQ_ERR_UNSUPPORTED_SHAPE;
}
