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
// One CTA = one (b,h) and one split of its tiles; each warp works through whole tiles
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
    float* part;       // [BH][nsplit][D+2]
    float* ml;         // [BH][2]   merged (max, sum) for score normalisation
    int nsplit;
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

// W words (4*W bytes) of a plane from global memory; the address is ALIGN-byte aligned
template <int W, int ALIGN>
__device__ __forceinline__ void load_words(const uint8_t* __restrict__ p, uint32_t (&w)[8]) {
    if (ALIGN == 16 && W % 4 == 0) {
#pragma unroll
        for (int i = 0; i < W; i += 4) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(p + 4 * i));
            w[i] = v.x; w[i + 1] = v.y; w[i + 2] = v.z; w[i + 3] = v.w;
        }
    } else if (ALIGN >= 8 && W % 2 == 0) {
#pragma unroll
        for (int i = 0; i < W; i += 2) {
            const uint2 v = __ldg(reinterpret_cast<const uint2*>(p + 4 * i));
            w[i] = v.x; w[i + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < W; ++i) w[i] = __ldg(reinterpret_cast<const uint32_t*>(p + 4 * i));
    }
}

// integer dot product of one lane's 32 channels of a w-bit plane with q (hi/lo bytes)
template <int W>
__device__ __forceinline__ int plane_dot(const uint32_t (&words)[8], const uint32_t (&qh)[8], const uint32_t (&ql)[8]) {
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
__device__ __forceinline__ void plane_axpy(const uint32_t (&words)[8], float wt, float (&acc)[8][4]) {
    constexpr int PER = 8 / W;
    constexpr uint32_t MASK = ((1u << W) - 1u) << (23 - W);
#pragma unroll
    for (int j = 0; j < W; ++j) {
        const uint32_t wd = words[j];
#pragma unroll
        for (int m = 0; m < PER; ++m) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int pos = 8 * i + W * m;
                const uint32_t sh = (pos + W <= 23) ? (wd << (23 - W - pos)) : (wd >> (pos + W - 23));
                const float xf = __uint_as_float((sh & MASK) | 0x3F800000u);
                acc[PER * j + m][i] = fmaf(wt, xf, acc[PER * j + m][i]);
            }
        }
    }
}

// per-warp scratch for the tile a warp is working on
template <int D>
struct WarpScratch {
    float step[2][QAQ_TILE];
    float mid[2][QAQ_TILE];     // min + step/2
    float ocorr[QAQ_TILE];      // sum over a token's key outliers of q_ch * (x - mid)
    float p[QAQ_TILE];
    float vout[D];              // value-outlier corrections
    int dot[QAQ_TILE];
    float wv[QAQ_TILE];         // p_t * step_t of the value side
    // work items grouped by plane width (8, 4, 2, 1):
    //   byte offset of the plane inside the tile | shift of the piece << 16 | token << 24
    uint32_t item[2][3 * QAQ_TILE];
};

template <int D>
struct DecSmem {
    WarpScratch<D> ws[DEC_WARPS];
    float qf[D];
    float macc[DEC_WARPS][D];
    float mm[DEC_WARPS], ml[DEC_WARPS];
    float red[DEC_WARPS], red2[DEC_WARPS];
    float qscale, qsum;
};

// One pass over the key-side items of one plane width: a group of P lanes per item.
template <int D, int W, int ALIGN>
__device__ __forceinline__ void k_items(WarpScratch<D>& ws, const uint8_t* __restrict__ tile, int first, int n,
                                        const uint32_t (&qh)[8], const uint32_t (&ql)[8], int part, int sub) {
    constexpr int P = D / 32, IPW = 32 / P;
    for (int i0 = 0; i0 < n; i0 += 2 * IPW) {
        uint32_t w0[8], w1[8];
        const int ia = i0 + sub, ib = i0 + IPW + sub;
        const bool va = ia < n, vb = ib < n;
        const uint32_t da_ = va ? ws.item[0][first + ia] : 0u, db_ = vb ? ws.item[0][first + ib] : 0u;
        if (va) load_words<W, ALIGN>(tile + (da_ & 0xFFFFu) + part * 4 * W, w0);
        if (vb) load_words<W, ALIGN>(tile + (db_ & 0xFFFFu) + part * 4 * W, w1);
        int da = va ? plane_dot<W>(w0, qh, ql) : 0;
        int db = vb ? plane_dot<W>(w1, qh, ql) : 0;
#pragma unroll
        for (int o = 1; o < P; o <<= 1) {
            da += __shfl_xor_sync(0xFFFFFFFFu, da, o);
            db += __shfl_xor_sync(0xFFFFFFFFu, db, o);
        }
        if (part == 0) {
            if (va) atomicAdd(&ws.dot[da_ >> 24], da << ((da_ >> 16) & 7));
            if (vb) atomicAdd(&ws.dot[db_ >> 24], db << ((db_ >> 16) & 7));
        }
    }
}

template <int D, int W, int ALIGN>
__device__ __forceinline__ void v_items(WarpScratch<D>& ws, const uint8_t* __restrict__ tile, int first, int n,
                                        float (&acc)[8][4], float& offs, int part, int sub) {
    constexpr int P = D / 32, IPW = 32 / P;
    for (int i0 = 0; i0 < n; i0 += 2 * IPW) {
        uint32_t w0[8], w1[8];
        const int ia = i0 + sub, ib = i0 + IPW + sub;
        const bool va = ia < n, vb = ib < n;
        const uint32_t da_ = va ? ws.item[1][first + ia] : 0u, db_ = vb ? ws.item[1][first + ib] : 0u;
        if (va) load_words<W, ALIGN>(tile + (da_ & 0xFFFFu) + part * 4 * W, w0);
        if (vb) load_words<W, ALIGN>(tile + (db_ & 0xFFFFu) + part * 4 * W, w1);
        if (va) {   // p_t * step_t * 2^shift * f = wt * (f / 2^W)
            const float wt = ws.wv[da_ >> 24] * __int_as_float((127 + W) << 23) * __int_as_float((127 + ((da_ >> 16) & 7)) << 23);
            plane_axpy<W>(w0, wt, acc);
            offs += wt;
        }
        if (vb) {
            const float wt = ws.wv[db_ >> 24] * __int_as_float((127 + W) << 23) * __int_as_float((127 + ((db_ >> 16) & 7)) << 23);
            plane_axpy<W>(w1, wt, acc);
            offs += wt;
        }
    }
}

// One CTA = one (b,h) and one split of its tiles; every warp works through whole tiles on
// its own (own running max / sum / accumulators), the warps are merged once at the end.
template <int D>
__global__ void __launch_bounds__(DEC_THREADS, 4) decode_kernel(const DecArgs a) {
    constexpr int P = D / 32;        // lanes per item
    constexpr int ALIGN = D / 8 >= 16 ? 16 : D / 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecSmem<D>& sm = *reinterpret_cast<DecSmem<D>*>(smem_raw);
    const int bh = blockIdx.y, split = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int part = lane % P, sub = lane / P;
    WarpScratch<D>& ws = sm.ws[warp];

    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const int per_split = (ntiles + a.nsplit - 1) / a.nsplit;
    const int tile_lo = split * per_split, tile_hi = min(ntiles, tile_lo + per_split);

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
    float offs = 0.f;        // sum of the weights this lane applied (the "1 +" of the magic floats)
    float m_run = __int_as_float(0xff800000), l_run = 0.f;
    float c_run = 0.f;       // per-lane part of sum_t p_t (min_t + step_t/2)

    const size_t trow = (size_t)bh * a.ntiles_max;
    const size_t mrow = (size_t)bh * a.tmax_pad;

    // Metadata runs ahead of the work: the tile table (lanes 0..7) two tiles ahead, the
    // per-token width / min / max (tokens lane, lane + 32) one tile ahead, and the packed
    // bytes of the next tile are pulled into L1 while the current tile is processed.
    uint32_t tb_next = 0, tb_next2 = 0, bits4 = 0, mmv[4] = {0, 0, 0, 0};
    auto fetch_table = [&](int tile) -> uint32_t {
        uint32_t v = 0;
        if (tile < tile_hi && lane < 8) {
            const TensorStore& ts = (lane >= 4) ? a.v : a.k;
            const size_t ti = trow + tile;
            const int f = lane & 3;
            v = f == 0 ? ts.tile_off[ti] : f == 1 ? ts.tile_nbytes[ti] : f == 2 ? ts.tile_ooff[ti] : ts.tile_ocnt[ti];
        }
        return v;
    };
    auto fetch_tokens = [&](int tile) {
        if (tile < tile_hi) {
            const size_t t0 = mrow + (size_t)tile * QAQ_TILE + lane;
            bits4 = (uint32_t)a.k.bits[t0] | ((uint32_t)a.k.bits[t0 + 32] << 8) | ((uint32_t)a.v.bits[t0] << 16) |
                    ((uint32_t)a.v.bits[t0 + 32] << 24);
            mmv[0] = a.k.mnmx[t0]; mmv[1] = a.k.mnmx[t0 + 32]; mmv[2] = a.v.mnmx[t0]; mmv[3] = a.v.mnmx[t0 + 32];
        }
    };
    auto prefetch_codes = [&](uint32_t tb) {   // tb: table registers of the tile to prefetch
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const uint32_t off = __shfl_sync(0xFFFFFFFFu, tb, 4 * x), nb = __shfl_sync(0xFFFFFFFFu, tb, 4 * x + 1);
            const uint8_t* src = (x ? a.v.codes : a.k.codes) + (size_t)bh * a.pool_bytes + off;
            for (uint32_t o = lane * 128u; o < nb; o += 32u * 128u) asm volatile("prefetch.global.L1 [%0];" ::"l"(src + o));
        }
    };
    uint32_t tb_cur = fetch_table(tile_lo + warp);
    tb_next = fetch_table(tile_lo + warp + DEC_WARPS);
    fetch_tokens(tile_lo + warp);

    for (int tile = tile_lo + warp; tile < tile_hi; tile += DEC_WARPS) {
        // ---- take over the metadata fetched earlier, start the fetches for the tiles ahead
        const uint32_t offK = __shfl_sync(0xFFFFFFFFu, tb_cur, 0), ooK = __shfl_sync(0xFFFFFFFFu, tb_cur, 2), ocK = __shfl_sync(0xFFFFFFFFu, tb_cur, 3);
        const uint32_t offV = __shfl_sync(0xFFFFFFFFu, tb_cur, 4), ooV = __shfl_sync(0xFFFFFFFFu, tb_cur, 6), ocV = __shfl_sync(0xFFFFFFFFu, tb_cur, 7);
        const uint32_t cb4 = bits4;
        const uint32_t cm[4] = {mmv[0], mmv[1], mmv[2], mmv[3]};
        tb_next2 = fetch_table(tile + 2 * DEC_WARPS);
        fetch_tokens(tile + DEC_WARPS);
        if (tile + DEC_WARPS < tile_hi) prefetch_codes(tb_next);
        tb_cur = tb_next;
        tb_next = tb_next2;

        // ---- per-token scalars, byte offsets, item lists (tokens lane and lane + 32)
        int ncls[2][4];
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            uint32_t len[2];
            int Bv[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int slot = lane + 32 * e;
                const bool valid = tile * QAQ_TILE + slot < a.T;
                const int B = valid ? (int)((cb4 >> (16 * x + 8 * e)) & 0xFF) : 0;
                Bv[e] = B;
                len[e] = (uint32_t)(D * B / 8);
                const uint32_t mmw = cm[2 * x + e];
                const float mn = __half2float(__ushort_as_half((unsigned short)(mmw & 0xFFFF)));
                const float mx = __half2float(__ushort_as_half((unsigned short)(mmw >> 16)));
                const float st = __fmul_rn(__fsub_rn(mx, mn), __int_as_float((127 - B) << 23));
                ws.step[x][slot] = valid ? st : 0.f;
                ws.mid[x][slot] = valid ? fmaf(0.5f, st, mn) : 0.f;
                if (x == 0) { ws.dot[slot] = 0; ws.ocorr[slot] = 0.f; }
            }
            uint32_t i0 = len[0], i1 = len[1];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t t0 = __shfl_up_sync(0xFFFFFFFFu, i0, d), t1 = __shfl_up_sync(0xFFFFFFFFu, i1, d);
                if (lane >= d) { i0 += t0; i1 += t1; }
            }
            const uint32_t tot0 = __shfl_sync(0xFFFFFFFFu, i0, 31);
            const uint32_t toff[2] = {i0 - len[0], tot0 + i1 - len[1]};
            int base = 0;
            const unsigned lt = (1u << lane) - 1u;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int w = 8 >> c;
                const unsigned b0 = __ballot_sync(0xFFFFFFFFu, (Bv[0] & w) != 0);
                const unsigned b1 = __ballot_sync(0xFFFFFFFFu, (Bv[1] & w) != 0);
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    if (Bv[e] & w) {
                        const uint32_t plane = toff[e] + (uint32_t)((Bv[e] & ~(2 * w - 1)) * (D / 8));
                        const uint32_t desc = plane | ((uint32_t)(Bv[e] & (w - 1)) << 16) | ((uint32_t)(lane + 32 * e) << 24);
                        ws.item[x][base + (e ? __popc(b0) + __popc(b1 & lt) : __popc(b0 & lt))] = desc;
                    }
                }
                ncls[x][c] = __popc(b0) + __popc(b1);
                base += ncls[x][c];
            }
        }
        __syncwarp();

        // ---- K: integer dot products per (token, plane), outlier corrections
        {
            const uint8_t* tk = a.k.codes + (size_t)bh * a.pool_bytes + offK;
            int first = 0;
            k_items<D, 8, ALIGN>(ws, tk, first, ncls[0][0], qh, ql, part, sub); first += ncls[0][0];
            k_items<D, 4, ALIGN>(ws, tk, first, ncls[0][1], qh, ql, part, sub); first += ncls[0][1];
            k_items<D, 2, (ALIGN > 8 ? 8 : ALIGN)>(ws, tk, first, ncls[0][2], qh, ql, part, sub); first += ncls[0][2];
            k_items<D, 1, 4>(ws, tk, first, ncls[0][3], qh, ql, part, sub);
            const uint32_t* og = a.k.outl + (size_t)bh * a.ocap + ooK;
            for (uint32_t e = lane; e < ocK; e += 32) {
                const uint32_t v = __ldg(og + e);
                const int tok = v >> 24, ch = (v >> 16) & 0xFF;
                const float val = __half2float(__ushort_as_half((unsigned short)(v & 0xFFFF)));
                atomicAdd(&ws.ocorr[tok], sm.qf[ch] * (val - ws.mid[0][tok]));
            }
        }
        __syncwarp();

        // ---- logits of tokens lane, lane + 32; running max / sum; weights
        {
            float lg[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int slot = lane + 32 * e;
                const int t = tile * QAQ_TILE + slot;
                lg[e] = __int_as_float(0xff800000);
                if (t < a.T) {
                    const float qk = fmaf(qscale * ws.step[0][slot], (float)ws.dot[slot], fmaf(ws.mid[0][slot], qsum, ws.ocorr[slot]));
                    lg[e] = a.scale * qk;
                    if (a.scores) a.scores[(size_t)bh * a.T + t] = lg[e];
                }
            }
            float m = fmaxf(lg[0], lg[1]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            const float m_new = fmaxf(m_run, m);
            const float alpha = __expf(m_run - m_new);   // 0 on the first tile (m_run = -inf)
            m_run = m_new;
            if (alpha != 1.0f) {
#pragma unroll
                for (int r = 0; r < 8; ++r)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[r][i] *= alpha;
                offs *= alpha;
                c_run *= alpha;
                for (int d = lane; d < D; d += 32) ws.vout[d] *= alpha;
            }
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int slot = lane + 32 * e;
                const float p = __expf(lg[e] - m_new);   // 0 for slots beyond T
                ws.p[slot] = p;
                ws.wv[slot] = p * ws.step[1][slot];
                c_run = fmaf(p, ws.mid[1][slot], c_run);
                s += p;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
            l_run = l_run * alpha + s;
        }
        __syncwarp();

        // ---- V: weighted accumulation of raw codes, outlier corrections
        {
            const uint8_t* tv = a.v.codes + (size_t)bh * a.pool_bytes + offV;
            int first = 0;
            v_items<D, 8, ALIGN>(ws, tv, first, ncls[1][0], acc, offs, part, sub); first += ncls[1][0];
            v_items<D, 4, ALIGN>(ws, tv, first, ncls[1][1], acc, offs, part, sub); first += ncls[1][1];
            v_items<D, 2, (ALIGN > 8 ? 8 : ALIGN)>(ws, tv, first, ncls[1][2], acc, offs, part, sub); first += ncls[1][2];
            v_items<D, 1, 4>(ws, tv, first, ncls[1][3], acc, offs, part, sub);
            const uint32_t* og = a.v.outl + (size_t)bh * a.ocap + ooV;
            for (uint32_t e = lane; e < ocV; e += 32) {
                const uint32_t v = __ldg(og + e);
                const int tok = v >> 24, ch = (v >> 16) & 0xFF;
                const float val = __half2float(__ushort_as_half((unsigned short)(v & 0xFFFF)));
                atomicAdd(&ws.vout[ch], ws.p[tok] * (val - ws.mid[1][tok]));
            }
        }
        __syncwarp();
    }

    // ---- warp result: lanes with the same part hold partial sums of the same channels
    float cs = c_run;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cs += __shfl_xor_sync(0xFFFFFFFFu, cs, o);
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float v = acc[r][i] - offs;
#pragma unroll
            for (int o = P; o < 32; o <<= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
            if (sub == 0) sm.macc[warp][32 * part + 4 * r + i] = v + ws.vout[32 * part + 4 * r + i] + cs;
        }
    if (lane == 0) { sm.mm[warp] = m_run; sm.ml[warp] = l_run; }
    __syncthreads();
    // ---- merge the warps (log-sum-exp) into this split's partial
    float M = __int_as_float(0xff800000);
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, sm.mm[w]);
    float* dst = a.part + ((size_t)bh * a.nsplit + split) * (D + 2);
    float L = 0.f;
    float wgt[DEC_WARPS];
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) {
        wgt[w] = (sm.mm[w] == __int_as_float(0xff800000)) ? 0.f : __expf(sm.mm[w] - M);
        L = fmaf(wgt[w], sm.ml[w], L);
    }
    for (int d = tid; d < D; d += DEC_THREADS) {
        float x = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) x = fmaf(wgt[w], sm.macc[w][d], x);
        dst[d] = x;
    }
    if (tid == 0) { dst[D] = M; dst[D + 1] = L; }
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
    // about 16 warps per SM on 148 SMs in total (4 warps per CTA), at least one tile per warp
    int want = (148 * 16 + 2 * BH) / (DEC_WARPS * BH);
    int cap = ntiles / DEC_WARPS > 0 ? ntiles / DEC_WARPS : 1;
    int n = want < cap ? want : cap;
    if (n < 1) n = 1;
    if (n > 64) n = 64;
    return n;
}

template <int D>
qaq_status run_decode(const DecArgs& a, int BH, cudaStream_t s) {
    const size_t smem = sizeof(DecSmem<D>);
    if (smem > 48 * 1024)
        QAQ_CUDA_TRY(cudaFuncSetAttribute(decode_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
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
