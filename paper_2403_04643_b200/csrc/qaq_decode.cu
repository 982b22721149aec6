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
// One CTA = one run of consecutive tiles of the flattened (b,h, tile) sequence (runs of equal
// length, so every SM gets the same amount of work); each warp works through whole tiles
// (QAQ_TILE tokens) on its own, with its own running max / sum / accumulators and no CTA
// barrier in the tile loop; warps are merged once at the end.  A (token, plane) pair is one
// work item, handled by head_dim/32 lanes that read their words of the plane straight from
// global memory (every packed byte is read once, by one lane); items are grouped by plane
// width so that the lanes of a warp run the same extraction code.
#include "qaq_internal.cuh"

namespace {

constexpr int DEC_WARPS = 4;
constexpr int DEC_THREADS = DEC_WARPS * 32;

struct DecArgs {
    TensorStore k, v;
    size_t pool_bytes;
    uint32_t ocap;
    int tmax_pad, ntiles_max;
    int T;
    const __half* q;
    float scale;
    float* part;       // [ncta][2][D+3]: accumulators, running max, sum of the weights used, exact sum
    float* ml;         // [BH][2]   merged (max, sum) for score normalisation
    int BH, run, ncta; // (b,h) count; tiles per CTA of the flattened (b,h, tile) sequence; CTAs
    float* out;        // [BH][D]
    float* scores;     // [BH][T] or null
};

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

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c) {  // (a & b) | c
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// acc += a * b with a, b binary16 and acc binary32 (one rounding)
__device__ __forceinline__ void fma_f32_f16(float& acc, unsigned short a, unsigned short b) {
    asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(acc) : "h"(a), "h"(b));
}
template <int BYTES>
__device__ __forceinline__ void cp_async(void* smem, const void* gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    if (BYTES == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
    else if (BYTES == 8) asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(s), "l"(gmem));
    else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// W words (4*W bytes) of a plane; the address is ALIGN-byte aligned
template <int W, int ALIGN>
__device__ __forceinline__ void load_words(const uint8_t* __restrict__ p, uint32_t (&w)[8]) {
    if (ALIGN == 16 && W % 4 == 0) {
#pragma unroll
        for (int i = 0; i < W; i += 4) {
            const uint4 v = *reinterpret_cast<const uint4*>(p + 4 * i);
            w[i] = v.x; w[i + 1] = v.y; w[i + 2] = v.z; w[i + 3] = v.w;
        }
    } else if (ALIGN >= 8 && W % 2 == 0) {
#pragma unroll
        for (int i = 0; i < W; i += 2) {
            const uint2 v = *reinterpret_cast<const uint2*>(p + 4 * i);
            w[i] = v.x; w[i + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < W; ++i) w[i] = *reinterpret_cast<const uint32_t*>(p + 4 * i);
    }
}

// integer dot product of one lane's 32 channels of a w-bit plane with q (hi/lo bytes)
template <int W>
__device__ __forceinline__ int plane_dot(const uint32_t (&words)[8], const uint32_t (&qh)[8], const uint32_t (&ql)[8]) {
    constexpr int PER = 8 / W;
    constexpr uint32_t MASK = 0x01010101u * ((1u << W) - 1u);
    int ah[2] = {0, 0}, al[2] = {0, 0};
#pragma unroll
    for (int j = 0; j < W; ++j) {
        const uint32_t wd = words[j];
#pragma unroll
        for (int m = 0; m < PER; ++m) {
            const uint32_t f = (wd >> (W * m)) & MASK;
            const int r = PER * j + m;
            ah[r & 1] = dp4a_us(f, qh[r], ah[r & 1]);
            al[r & 1] = dp4a_uu(f, ql[r], al[r & 1]);
        }
    }
    return (ah[0] + ah[1]) * 256 + (al[0] + al[1]);
}

// acc[r][i] += b * (f - 2^(W-1)) for the lane's 32 channels of a w-bit plane.
// Fields are taken two at a time (the same bit positions of the two 16-bit halves of a word) by
// OR-ing them into the mantissa of a binary16 power of two whose last mantissa bit weighs
// 2^-(W*m) for field slot m: 2^(10-Wm) + f, exactly; subtracting 2^(10-Wm) + 2^(W-1) is exact and
// centres the code, so every slot uses the same weight.  The products go into binary32 accumulators.
template <int W>
__device__ __forceinline__ void plane_axpy(const uint32_t (&words)[8], unsigned short b, float (&acc)[8][4]) {
    constexpr int PER = 8 / W;
#pragma unroll
    for (int j = 0; j < W; ++j) {
        const uint32_t ev = words[j];          // byte lanes 0 and 2 in the low bytes of the halves
        const uint32_t od = words[j] >> 8;     // byte lanes 1 and 3
#pragma unroll
        for (int m = 0; m < PER; ++m) {
            const uint32_t mask = (((1u << W) - 1u) << (W * m)) * 0x00010001u;
            const uint32_t magic = (0x6400u - ((uint32_t)(W * m) << 10)) * 0x00010001u;        // binary16 2^(10-Wm), twice
            const uint32_t cen = magic + (1u << (W - 1 + W * m)) * 0x00010001u;              // ... + 2^(W-1)
            const __half2 c2 = *reinterpret_cast<const __half2*>(&cen);
            uint32_t xe = lop3_and_or(ev, mask, magic), xo = lop3_and_or(od, mask, magic);
            const __half2 ye = __hsub2(*reinterpret_cast<__half2*>(&xe), c2);
            const __half2 yo = __hsub2(*reinterpret_cast<__half2*>(&xo), c2);
            const int r = PER * j + m;
            fma_f32_f16(acc[r][0], __half_as_ushort(__low2half(ye)), b);
            fma_f32_f16(acc[r][2], __half_as_ushort(__high2half(ye)), b);
            fma_f32_f16(acc[r][1], __half_as_ushort(__low2half(yo)), b);
            fma_f32_f16(acc[r][3], __half_as_ushort(__high2half(yo)), b);
        }
    }
}

constexpr int UNIT = QAQ_TILE / 2;   // tokens a warp handles at a time (half a tile)
constexpr int OSTAGE = 192;          // outlier entries per tile and tensor staged in shared memory

// per-warp scratch for the half tile a warp is working on
template <int D>
struct WarpScratch {
    alignas(16) uint8_t bufK[UNIT * D + 16];
    alignas(16) uint8_t bufV[UNIT * D + 16];
    float stepK[UNIT];
    // per token of the whole tile (both halves): the tile's outlier lists are gone through once
    float midK[2 * UNIT];       // min + step/2
    float midV[2 * UNIT];
    float ocorr[2 * UNIT];      // sum over a token's key outliers of q_ch * (x - mid)
    float p[2 * UNIT];          // attention weights, kept at the current scale of the running sums
    float wv[UNIT];             // p_t * step_t * 2^g of the value side
    float vout[D];              // value-outlier corrections
    int dot[UNIT];
    // work items grouped by plane width (8, 4, 2, 1):
    //   byte offset of the plane inside the half tile | shift of the piece << 16 | token << 24
    uint32_t item[2][3 * UNIT];
    alignas(16) uint32_t outl[2][OSTAGE];   // the tile's outlier entries (K, V); longer lists continue in global memory
};

template <int D>
struct DecSmem {
    WarpScratch<D> ws[DEC_WARPS];
    float qf[D];
    float macc[DEC_WARPS][D];
    float mm[DEC_WARPS], ml[DEC_WARPS], mlx[DEC_WARPS];
    float red[DEC_WARPS], red2[DEC_WARPS];
    float qscale, qsum;
};

template <int D, int W, int ALIGN>
__device__ __forceinline__ void k_items(WarpScratch<D>& ws, int first, int n, const uint32_t (&qh)[8],
                                        const uint32_t (&ql)[8], int part, int sub) {
    constexpr int P = D / 32, IPW = 32 / P;
#pragma unroll 1
    for (int i0 = 0; i0 < n; i0 += IPW) {
        uint32_t w0[8];
        const int ia = i0 + sub;
        const bool va = ia < n;
        const uint32_t de = va ? ws.item[0][first + ia] : 0u;
        int da = 0;
        if (va) {
            load_words<W, ALIGN>(ws.bufK + (de & 0xFFFFu) + part * 4 * W, w0);
            da = plane_dot<W>(w0, qh, ql);
        }
#pragma unroll
        for (int o = 1; o < P; o <<= 1) da += __shfl_xor_sync(0xFFFFFFFFu, da, o);
        if (va && part == 0) atomicAdd(&ws.dot[de >> 24], da << ((de >> 16) & 7));
    }
}

template <int D, int W, int ALIGN>
__device__ __forceinline__ void v_items(WarpScratch<D>& ws, int first, int n, float (&acc)[8][4], int part, int sub) {
    constexpr int P = D / 32, IPW = 32 / P;
#pragma unroll 1
    for (int i0 = sub; i0 < n; i0 += IPW) {
        uint32_t w0[8];
        const uint32_t de = ws.item[1][first + i0];
        load_words<W, ALIGN>(ws.bufV + (de & 0xFFFFu) + part * 4 * W, w0);
        // weight of the piece: p_t * step_t * 2^g * 2^shift, in binary16
        const float wt = ws.wv[de >> 24] * __int_as_float((127 + ((de >> 16) & 7)) << 23);
        plane_axpy<W>(w0, __half_as_ushort(__float2half_rn(wt)), acc);
    }
}

// One CTA = one run of consecutive tiles, which meets one or two (b,h): the body below runs once
// per (b,h) segment and leaves one partial per segment.  Every warp works through whole tiles on its
// own, half a tile (32 tokens) at a time: own running max / sum / accumulators, own staging
// buffers, no CTA barrier in the loop; the warps are merged once at the end.  The packed bytes
// of the next half tile are copied to shared memory with cp.async while the current one is being
// processed: the keys during the value phase, the values during the key phase.
template <int D>
__global__ void __launch_bounds__(DEC_THREADS, 4) decode_kernel(const DecArgs a) {
    constexpr int P = D / 32;        // lanes per item
    constexpr int ALIGN = D / 8 >= 16 ? 16 : D / 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecSmem<D>& sm = *reinterpret_cast<DecSmem<D>*>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int part = lane % P, sub = lane / P;
    WarpScratch<D>& ws = sm.ws[warp];

#pragma unroll 1
    for (int seg = 0; seg < 2; ++seg) {
    // this CTA's run of the flattened (b,h, tile) sequence; it touches at most two (b,h).  The block
    // index is read afresh for each segment so that none of this stays in registers over the tile loop.
    int cta;
    asm volatile("mov.u32 %0, %%ctaid.x;" : "=r"(cta));
    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const int flat_lo = cta * a.run, flat_hi = min(a.BH * ntiles, flat_lo + a.run);
    const int bh = flat_lo / ntiles + seg;
    const int tile_lo = max(flat_lo, bh * ntiles) - bh * ntiles, tile_hi = min(flat_hi, (bh + 1) * ntiles) - bh * ntiles;
    if (tile_lo >= tile_hi) continue;   // the same for every thread of the CTA

    // ---- q: float copy, fixed-point bytes per lane
    float qmax = 0.f, qs = 0.f;
    for (int d = tid; d < D; d += DEC_THREADS) {
        const float f = __half2float(a.q[(size_t)bh * D + d]);
        sm.qf[d] = f;
        qmax = fmaxf(qmax, fabsf(f));
        qs += f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        qmax = fmaxf(qmax, __shfl_xor_sync(0xFFFFFFFFu, qmax, o));
        qs += __shfl_xor_sync(0xFFFFFFFFu, qs, o);
    }
    if (lane == 0) { sm.red[warp] = qmax; sm.red2[warp] = qs; }
    for (int d = lane; d < D; d += 32) ws.vout[d] = 0.f;
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
    float m_run = __int_as_float(0xff800000), l_run = 0.f, lx_run = 0.f;   // lx: sum of the unperturbed p
    float c_run = 0.f;       // per-lane part of sum_t p_t * (constant part of the token's values)
    // The binary16 weights of the value side carry a common power-of-two factor 2^g so that the
    // largest possible weight (range/2) sits near 2^12; g only ever decreases.
    int g_run = 24;

    const size_t trow = (size_t)bh * a.ntiles_max;
    const size_t mrow = (size_t)bh * a.tmax_pad;
    const uint8_t* poolK = a.k.codes + (size_t)bh * a.pool_bytes;
    const uint8_t* poolV = a.v.codes + (size_t)bh * a.pool_bytes;

    // ---- tile metadata in registers: table words in lanes 0..7, widths and min/max of tokens lane, lane+32
    struct Meta { uint32_t tb, bits4, mm[4]; };
    auto fetch_meta = [&](int tile) {
        Meta m;
        m.tb = 0; m.bits4 = 0; m.mm[0] = m.mm[1] = m.mm[2] = m.mm[3] = 0;
        if (tile < tile_hi) {
            if (lane < 8) {
                const TensorStore& ts = (lane >= 4) ? a.v : a.k;
                const size_t ti = trow + tile;
                const int f = lane & 3;
                m.tb = f == 0 ? ts.tile_off[ti] : f == 1 ? ts.tile_nbytes[ti] : f == 2 ? ts.tile_ooff[ti] : ts.tile_ocnt[ti];
            }
            const size_t t0 = mrow + (size_t)tile * QAQ_TILE + lane;
            m.bits4 = (uint32_t)a.k.bits[t0] | ((uint32_t)a.k.bits[t0 + 32] << 8) | ((uint32_t)a.v.bits[t0] << 16) |
                      ((uint32_t)a.v.bits[t0 + 32] << 24);
            m.mm[0] = a.k.mnmx[t0]; m.mm[1] = a.k.mnmx[t0 + 32]; m.mm[2] = a.v.mnmx[t0]; m.mm[3] = a.v.mnmx[t0 + 32];
        }
        return m;
    };
    // bytes of the first half (tokens 0..31) of a tile, per tensor (slots beyond T have width 0)
    auto first_half_bytes = [&](const Meta& m, uint32_t& hK, uint32_t& hV) {
        uint32_t k = (m.bits4 & 0xFF) * (D / 8), v = ((m.bits4 >> 16) & 0xFF) * (D / 8);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            k += __shfl_xor_sync(0xFFFFFFFFu, k, o);
            v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        }
        hK = k; hV = v;
    };
    auto stage = [&](uint8_t* dst, const uint8_t* src, uint32_t nbytes) {
#pragma unroll 1
        for (uint32_t o = lane * ALIGN; o < nbytes; o += 32 * ALIGN) cp_async<ALIGN>(dst + o, src + o);
    };

    auto stage_outl = [&](int x, uint32_t first, uint32_t count) {   // entries are 4 bytes, lists start 16-byte aligned
        const uint32_t* src = (x ? a.v.outl : a.k.outl) + (size_t)bh * a.ocap + first;
        const uint32_t n16 = ((count < (uint32_t)OSTAGE ? count : (uint32_t)OSTAGE) + 3u) >> 2;
#pragma unroll 1
        for (uint32_t o = lane; o < n16; o += 32) cp_async<16>(&ws.outl[x][4 * o], src + 4 * o);
    };
    int tile = tile_lo + warp;
    Meta cur = fetch_meta(tile);
    Meta nxt = fetch_meta(tile + DEC_WARPS);
    uint32_t h0K = 0, h0V = 0;
    first_half_bytes(cur, h0K, h0V);
    if (tile < tile_hi) {
        stage(ws.bufK, poolK + __shfl_sync(0xFFFFFFFFu, cur.tb, 0), h0K);
        stage_outl(0, __shfl_sync(0xFFFFFFFFu, cur.tb, 2), __shfl_sync(0xFFFFFFFFu, cur.tb, 3));
        cp_async_commit();
        stage(ws.bufV, poolV + __shfl_sync(0xFFFFFFFFu, cur.tb, 4), h0V);
        stage_outl(1, __shfl_sync(0xFFFFFFFFu, cur.tb, 6), __shfl_sync(0xFFFFFFFFu, cur.tb, 7));
        cp_async_commit();
    }

    for (; tile < tile_hi; tile += DEC_WARPS) {
        const uint32_t offK = __shfl_sync(0xFFFFFFFFu, cur.tb, 0), totK = __shfl_sync(0xFFFFFFFFu, cur.tb, 1);
        const uint32_t ooK = __shfl_sync(0xFFFFFFFFu, cur.tb, 2), ocK = __shfl_sync(0xFFFFFFFFu, cur.tb, 3);
        const uint32_t offV = __shfl_sync(0xFFFFFFFFu, cur.tb, 4), totV = __shfl_sync(0xFFFFFFFFu, cur.tb, 5);
        const uint32_t ooV = __shfl_sync(0xFFFFFFFFu, cur.tb, 6), ocV = __shfl_sync(0xFFFFFFFFu, cur.tb, 7);
        const bool has_next = tile + DEC_WARPS < tile_hi;
        uint32_t n0K = 0, n0V = 0;   // first-half bytes of the next tile

#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
            const int t = tile * QAQ_TILE + UNIT * half + lane;   // this lane's token
            const bool valid = t < a.T;
            // ---- per-token scalars, byte offsets inside the half tile, item lists
            int ncls[2][4];
            float rngV = 0.f, cstV = 0.f;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                const int B = valid ? (int)((cur.bits4 >> (16 * x + 8 * half)) & 0xFF) : 0;
                const uint32_t len = (uint32_t)(D * B / 8);
                const uint32_t mmw = half ? cur.mm[2 * x + 1] : cur.mm[2 * x];
                const float mn = __half2float(__ushort_as_half((unsigned short)(mmw & 0xFFFF)));
                const float mx = __half2float(__ushort_as_half((unsigned short)(mmw >> 16)));
                const float rng = valid ? __fsub_rn(mx, mn) : 0.f;
                const float st = __fmul_rn(rng, __int_as_float((127 - B) << 23));
                const float mid = fmaf(0.5f, st, mn);
                if (x == 0) {
                    ws.stepK[lane] = st;
                    ws.dot[lane] = 0;
                    if (half == 0) {
                        ws.midK[lane] = valid ? mid : 0.f;
                        ws.ocorr[lane] = 0.f;
                        // the lane's token of the second half: its mid is needed already, because all key outliers of
                        // the tile are gone through in this half
                        const bool valid2 = t + UNIT < a.T;
                        const int B2 = valid2 ? (int)((cur.bits4 >> 8) & 0xFF) : 0;
                        const float mn2 = __half2float(__ushort_as_half((unsigned short)(cur.mm[1] & 0xFFFF)));
                        const float mx2 = __half2float(__ushort_as_half((unsigned short)(cur.mm[1] >> 16)));
                        const float st2 = __fmul_rn(valid2 ? __fsub_rn(mx2, mn2) : 0.f, __int_as_float((127 - B2) << 23));
                        ws.midK[UNIT + lane] = valid2 ? fmaf(0.5f, st2, mn2) : 0.f;
                        ws.ocorr[UNIT + lane] = 0.f;
                    }
                } else {
                    // centred planes: piece w contributes a constant step * 2^((B & (2w-1)) - 1)
                    float cst = 0.5f;
#pragma unroll
                    for (int w = 8; w >= 1; w >>= 1)
                        if (B & w) cst += __int_as_float((127 + (B & (2 * w - 1)) - 1) << 23);
                    ws.midV[UNIT * half + lane] = valid ? mid : 0.f;       // value of a zero code slot (outliers)
                    cstV = valid ? fmaf(cst, st, mn) : 0.f;                 // constant part, picked up below
                    ws.wv[lane] = st;                                       // step for now, weight after the softmax
                    rngV = rng;
                }
                uint32_t inc = len;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                    if (lane >= d) inc += u;
                }
                const uint32_t toff = inc - len;
                int base = 0;
                const unsigned lt = (1u << lane) - 1u;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int w = 8 >> c;
                    const unsigned bal = __ballot_sync(0xFFFFFFFFu, (B & w) != 0);
                    if (B & w) {
                        const uint32_t plane = toff + (uint32_t)((B & ~(2 * w - 1)) * (D / 8));
                        ws.item[x][base + __popc(bal & lt)] = plane | ((uint32_t)(B & (w - 1)) << 16) | ((uint32_t)lane << 24);
                    }
                    ncls[x][c] = __popc(bal);
                    base += ncls[x][c];
                }
            }
            // common exponent of the value weights
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) rngV = fmaxf(rngV, __shfl_xor_sync(0xFFFFFFFFu, rngV, o));
            {
                const int e = rngV > 0.f ? ((__float_as_int(rngV) >> 23) & 0xFF) - 127 : -12;
                const int g = 12 - e;
                if (g < g_run) {
                    const float f = __int_as_float((127 + g - g_run) << 23);
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[r][i] *= f;
                    g_run = g;
                }
            }
            cp_async_wait<1>();     // this half's keys have landed (its values may still be in flight)
            __syncwarp();

            // ---- K: integer dot products per (token, plane), outlier corrections
            {
                int first = 0;
                k_items<D, 8, ALIGN>(ws, first, ncls[0][0], qh, ql, part, sub); first += ncls[0][0];
                k_items<D, 4, ALIGN>(ws, first, ncls[0][1], qh, ql, part, sub); first += ncls[0][1];
                k_items<D, 2, (ALIGN > 8 ? 8 : ALIGN)>(ws, first, ncls[0][2], qh, ql, part, sub); first += ncls[0][2];
                k_items<D, 1, 4>(ws, first, ncls[0][3], qh, ql, part, sub);
                // all key outliers of the tile, once, while its first half is worked on
                if (half == 0) {
                    const uint32_t* og = a.k.outl + (size_t)bh * a.ocap + ooK;
#pragma unroll 1
                    for (uint32_t e0 = 0; e0 < ocK; e0 += 32) {
                        const uint32_t e = e0 + lane;
                        if (e < ocK) {
                            const uint32_t v = e < (uint32_t)OSTAGE ? ws.outl[0][e] : __ldg(og + e);
                            const int tok = v >> 24, ch = (v >> 16) & 0xFF;
                            const float val = __half2float(__ushort_as_half((unsigned short)(v & 0xFFFF)));
                            atomicAdd(&ws.ocorr[tok], sm.qf[ch] * (val - ws.midK[tok]));
                        }
                    }
                }
            }
            __syncwarp();
            // ---- the key buffer is free: start the copy of the next unit's keys
            if (half == 0) {
                stage(ws.bufK, poolK + offK + h0K, totK - h0K);
            } else if (has_next) {
                first_half_bytes(nxt, n0K, n0V);
                stage(ws.bufK, poolK + __shfl_sync(0xFFFFFFFFu, nxt.tb, 0), n0K);
                stage_outl(0, __shfl_sync(0xFFFFFFFFu, nxt.tb, 2), __shfl_sync(0xFFFFFFFFu, nxt.tb, 3));
            }
            cp_async_commit();

            // ---- logit of this lane's token; running max / sum; weights
            {
                float lg = __int_as_float(0xff800000);
                if (valid) {
                    const float qk = fmaf(qscale * ws.stepK[lane], (float)ws.dot[lane], fmaf(ws.midK[UNIT * half + lane], qsum, ws.ocorr[UNIT * half + lane]));
                    lg = a.scale * qk;
                    if (a.scores) a.scores[(size_t)bh * a.T + t] = lg;
                }
                float m = lg;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
                const float m_new = fmaxf(m_run, m);
                const float alpha = __expf(m_run - m_new);   // 0 on the first unit (m_run = -inf)
                m_run = m_new;
                if (alpha != 1.0f) {
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[r][i] *= alpha;
                    c_run *= alpha;
                    for (int d = lane; d < D; d += 32) ws.vout[d] *= alpha;
                    if (half == 1) ws.p[lane] *= alpha;       // the first half's weights follow the new scale
                }
                float p = __expf(lg - m_new);                // 0 for slots beyond T
                float sx = p;
                // The value weight p * step * 2^g is used in binary16.  It is rounded to 11 significant
                // bits here, once, and p is adjusted by the same factor, so that the planes, the constant
                // part and the softmax denominator all see the same (slightly perturbed) probability.
                const float wfull = p * ws.wv[lane] * __int_as_float((127 + g_run) << 23);
                const float big = __fmul_rn(wfull, 8193.0f);  // 2^13 + 1: splits off the upper 11 bits (no contraction)
                const float wr = __fsub_rn(big, __fsub_rn(big, wfull));
                if (wfull > 0.f) p *= __fdividef(wr, wfull);
                ws.wv[lane] = wr;
                c_run = fmaf(p, cstV, c_run);
                float s = p;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
                    sx += __shfl_xor_sync(0xFFFFFFFFu, sx, o);
                }
                l_run = l_run * alpha + s;
                lx_run = lx_run * alpha + sx;
                ws.p[UNIT * half + lane] = p;
            }
            cp_async_wait<1>();     // this half's values have landed
            __syncwarp();

            // ---- V: weighted accumulation of centred codes, outlier corrections
            {
                int first = 0;
                v_items<D, 8, ALIGN>(ws, first, ncls[1][0], acc, part, sub); first += ncls[1][0];
                v_items<D, 4, ALIGN>(ws, first, ncls[1][1], acc, part, sub); first += ncls[1][1];
                v_items<D, 2, (ALIGN > 8 ? 8 : ALIGN)>(ws, first, ncls[1][2], acc, part, sub); first += ncls[1][2];
                v_items<D, 1, 4>(ws, first, ncls[1][3], acc, part, sub);
                // all value outliers of the tile, once, when the weights of both halves are known
                if (half == 1) {
                    const uint32_t* og = a.v.outl + (size_t)bh * a.ocap + ooV;
#pragma unroll 1
                    for (uint32_t e0 = 0; e0 < ocV; e0 += 32) {
                        const uint32_t e = e0 + lane;
                        if (e < ocV) {
                            const uint32_t v = e < (uint32_t)OSTAGE ? ws.outl[1][e] : __ldg(og + e);
                            const int tok = v >> 24, ch = (v >> 16) & 0xFF;
                            const float val = __half2float(__ushort_as_half((unsigned short)(v & 0xFFFF)));
                            atomicAdd(&ws.vout[ch], ws.p[tok] * (val - ws.midV[tok]));
                        }
                    }
                }
            }
            __syncwarp();
            // ---- the value buffer is free: start the copy of the next unit's values
            if (half == 0) stage(ws.bufV, poolV + offV + h0V, totV - h0V);
            else if (has_next) {
                stage(ws.bufV, poolV + __shfl_sync(0xFFFFFFFFu, nxt.tb, 4), n0V);
                stage_outl(1, __shfl_sync(0xFFFFFFFFu, nxt.tb, 6), __shfl_sync(0xFFFFFFFFu, nxt.tb, 7));
            }
            cp_async_commit();
        }
        cur = nxt;
        h0K = n0K; h0V = n0V;
        nxt = fetch_meta(tile + 2 * DEC_WARPS);
    }
    cp_async_wait<0>();

    // ---- warp result: lanes with the same part hold partial sums of the same channels
    float cs = c_run;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cs += __shfl_xor_sync(0xFFFFFFFFu, cs, o);
    const float unscale = __int_as_float((127 - g_run) << 23);
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float v = acc[r][i];
#pragma unroll
            for (int o = P; o < 32; o <<= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
            if (sub == 0) sm.macc[warp][32 * part + 4 * r + i] = fmaf(v, unscale, ws.vout[32 * part + 4 * r + i] + cs);
        }
    if (lane == 0) { sm.mm[warp] = m_run; sm.ml[warp] = l_run; sm.mlx[warp] = lx_run; }
    __syncthreads();
    // ---- merge the warps (log-sum-exp) into this segment's partial
    float M = __int_as_float(0xff800000);
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, sm.mm[w]);
    float* dst = a.part + (size_t)(2 * cta + seg) * (D + 3);
    float L = 0.f, LX = 0.f;
    float wgt[DEC_WARPS];
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) {
        wgt[w] = (sm.mm[w] == __int_as_float(0xff800000)) ? 0.f : __expf(sm.mm[w] - M);
        L = fmaf(wgt[w], sm.ml[w], L);
        LX = fmaf(wgt[w], sm.mlx[w], LX);
    }
    for (int d = tid; d < D; d += DEC_THREADS) {
        float x = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) x = fmaf(wgt[w], sm.macc[w][d], x);
        dst[d] = x;
    }
    if (tid == 0) { dst[D] = M; dst[D + 1] = L; dst[D + 2] = LX; }
    __syncthreads();   // the shared arrays are reused by the second segment
    }
}

// log-sum-exp merge of the partials -> X, and (max, sum) for the score row
template <int D>
__global__ void merge_kernel(const DecArgs a) {
    const int bh = blockIdx.x, d = threadIdx.x;
    // the CTAs of decode_kernel whose runs meet this (b,h); a CTA's first segment has slot 0
    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const int c_lo = (bh * ntiles) / a.run, c_hi = ((bh + 1) * ntiles - 1) / a.run;
    // only the first of them can have begun in the (b,h) before
    auto slot = [&](int c) { return a.part + (size_t)(2 * c + (c * a.run < bh * ntiles ? 1 : 0)) * (D + 3); };
    float M = __int_as_float(0xff800000);
    for (int c = c_lo; c <= c_hi; ++c) M = fmaxf(M, slot(c)[D]);
    float L = 0.f, LX = 0.f, x = 0.f;
    for (int c = c_lo; c <= c_hi; ++c) {
        const float* p = slot(c);
        const float m = p[D];
        if (m == __int_as_float(0xff800000)) continue;
        const float w = __expf(m - M);
        L = fmaf(w, p[D + 1], L);
        LX = fmaf(w, p[D + 2], LX);
        x = fmaf(w, p[d], x);
    }
    a.out[(size_t)bh * D + d] = L > 0.f ? x / L : 0.f;
    if (d == 0) { a.ml[2 * bh] = M; a.ml[2 * bh + 1] = LX; }
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

// The flattened sequence of BH * ntiles tiles is cut into runs of `run` consecutive tiles, one CTA
// each: enough CTAs to fill every SM (148 SMs, 4 resident CTAs each) evenly, at least one tile per
// warp where there are that many, and never more than one (b,h) boundary inside a run.
constexpr int DEC_SLOTS = 148 * 4;
struct DecPlan { int run, ncta; };
DecPlan plan_decode(int BH, int ntiles) {
    const long long total = (long long)BH * ntiles;
    long long run = (total + DEC_SLOTS - 1) / DEC_SLOTS;
    const int floor_run = ntiles < DEC_WARPS ? ntiles : DEC_WARPS;
    if (run < floor_run) run = floor_run;
    if (run > ntiles) run = ntiles;
    DecPlan p;
    p.run = (int)run;
    p.ncta = (int)((total + run - 1) / run);
    return p;
}
// floats of workspace for the partials (two slots per CTA) and the merged (max, sum) pairs
size_t decode_ws_floats(int BH, int ncta, int D) { return (size_t)2 * ncta * (D + 3) + (size_t)BH * 2; }

template <int D>
qaq_status run_decode(const DecArgs& a, int BH, cudaStream_t s) {
    const size_t smem = sizeof(DecSmem<D>);
    if (smem > 48 * 1024)
        QAQ_CUDA_TRY(cudaFuncSetAttribute(decode_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_kernel<D><<<a.ncta, DEC_THREADS, smem, s>>>(a);
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

extern "C" qaq_status qaq_decode_workspace_bytes(const qaq_cache* c, size_t* host_out) {
    if (!c || !host_out) return QAQ_ERR_INVALID_ARG;
    // plan_decode never uses more CTAs than max(DEC_SLOTS, BH), whatever the token count
    const int ncta_max = c->BH > DEC_SLOTS ? c->BH : DEC_SLOTS;
    *host_out = decode_ws_floats(c->BH, ncta_max, c->cfg.head_dim) * sizeof(float);
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
    const DecPlan plan = plan_decode(BH, ntiles);
    a.BH = BH; a.run = plan.run; a.ncta = plan.ncta;
    a.part = (float*)ws;
    a.ml = a.part + (size_t)2 * plan.ncta * (D + 3);
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
    const DecPlan plan = plan_decode(BH, ntiles);
    // partials [ncta][2][D+3] followed by the merged (max, sum) pairs [BH][2]
    const size_t need = decode_ws_floats(BH, plan.ncta, D) * sizeof(float);
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
    a.BH = BH; a.run = plan.run; a.ncta = plan.ncta;
    // Every partial that the merge reads and every (max,sum) pair is written before it is read,
    // so nothing in the scratch has to be cleared between calls.
    a.part = (float*)scratch;
    a.ml = a.part + (size_t)2 * plan.ncta * (D + 3);
    a.out = out; a.scores = nullptr;
    cudaStream_t s = (cudaStream_t)stream;
    switch (D) {
        case 32: return run_decode<32>(a, BH, s);
        case 64: return run_decode<64>(a, BH, s);
        case 128: return run_decode<128>(a, BH, s);
    }
    return QAQ_ERR_UNSUPPORTED_SHAPE;
}
