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
// barrier in the tile loop; warps are merged once at the end.  A tile is stored as sections of
// equal-width pieces (qaq_codec.cuh), so every inner loop runs one extraction routine over the
// items of one section, and a token finds its items by its rank among the tokens that have a
// piece of that width (ballots over the widths; no lists are built).
//
// X = S Vhat runs on integer dot products as well: the value pieces of four tokens share a word
// (one per byte lane), the per-token weights p_t * step_t * 2^shift become 24-bit fixed point
// with one scale per tile (three dp4a per word and field), and the integer sums of a tile are
// added to binary32 accumulators once per tile.  The rounded weight of a token is also what the
// softmax denominator and the constant part of its values use, so numerator and denominator see
// the same slightly perturbed probability.
//
// Outlier corrections are summed in fixed point with integer atomics (scale from the largest
// term of the tile), so that the result does not depend on the order in which lanes arrive.
#include "qaq_codec.cuh"
#include "qaq_internal.cuh"

namespace {

constexpr int DEC_WARPS = 4;
constexpr int DEC_THREADS = DEC_WARPS * 32;
constexpr int DEC_CTAS_PER_SM = 2;   // what the per-warp staging buffers of head_dim 128 leave room for

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

// weighted sums of one lane's 8 channels over the four tokens of a value group:
// acc[cl] += sum_i weight_i * piece_i(channel cl); wt.x / wt.y / wt.z hold the high / middle / low bytes of the four
// 24-bit weights
template <int W>
__device__ __forceinline__ void group_axpy(const uint32_t (&words)[8], const uint4 wt, int (&ahi)[8], int (&amd)[8], int (&alo)[8]) {
    constexpr int PER = 8 / W;
    constexpr uint32_t MASK = 0x01010101u * ((1u << W) - 1u);
#pragma unroll
    for (int k = 0; k < W; ++k) {
#pragma unroll
        for (int m = 0; m < PER; ++m) {
            const uint32_t f = (words[k] >> (W * m)) & MASK;
            ahi[PER * k + m] = dp4a_uu(f, wt.x, ahi[PER * k + m]);
            amd[PER * k + m] = dp4a_uu(f, wt.y, amd[PER * k + m]);
            alo[PER * k + m] = dp4a_uu(f, wt.z, alo[PER * k + m]);
        }
    }
}

constexpr int OSTAGE = 192;          // outlier entries per tile and tensor staged in shared memory

// per-warp scratch for the tile a warp is working on
template <int D>
struct WarpScratch {
    alignas(16) uint8_t bufK[QAQ_TILE * D + 16];
    alignas(16) uint8_t bufV[(qaqc::v_tile_bytes_max(D) + 15) / 16 * 16 + 16];
    int dotw[4][QAQ_TILE];                    // integer q . piece per section and rank
    alignas(16) uint32_t wts[4][QAQ_TILE / 4][4];  // per section and value group: high, middle, low bytes of the four weights
    float midK[QAQ_TILE];       // min + step/2
    float midV[QAQ_TILE];
    float p[QAQ_TILE];          // attention weights of the tile's tokens at the current scale of the running sums
    int iocorr[2][QAQ_TILE];    // fixed-point sums (high, low part) of the key-outlier corrections per token
    int ivout[2][D];            // ... of the value-outlier corrections per channel (zero between tiles)
    float vout[D];              // value-outlier corrections
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

// q . piece for the items of one key section: P = D/32 lanes per item, each 32 channels
template <int D, int W>
__device__ __forceinline__ void k_section(const uint8_t* sec, int n, int* dots, const uint32_t (&qh)[8], const uint32_t (&ql)[8],
                                          int part, int sub) {
    constexpr int P = D / 32, IPW = 32 / P;
#pragma unroll 1
    for (int i0 = 0; i0 < n; i0 += IPW) {
        const int r = i0 + sub;
        int da = 0;
        if (r < n) {
            uint32_t w0[8];
            qaqc::load_words<W>(sec + r * (D * W / 8) + part * 4 * W, w0);
            da = plane_dot<W>(w0, qh, ql);
        }
#pragma unroll
        for (int o = 1; o < P; o <<= 1) da += __shfl_xor_sync(0xFFFFFFFFu, da, o);
        if (r < n && part == 0) dots[r] = da;
    }
}

// weighted accumulation over the groups of one value section: LPG = D/8 lanes per group, each 8 channels
template <int D, int W>
__device__ __forceinline__ void v_section(const uint8_t* sec, int ngroups, const uint32_t (*wts)[4], int (&ahi)[8], int (&amd)[8],
                                          int (&alo)[8], int h, int grp) {
    constexpr int LPG = D / 8, GPW = 32 / LPG;
#pragma unroll 1
    for (int g = grp; g < ngroups; g += GPW) {
        uint32_t w0[8];
        qaqc::load_words<W>(sec + g * (D * W / 2) + h * 4 * W, w0);
        const uint4 wt = *reinterpret_cast<const uint4*>(wts[g]);
        group_axpy<W>(w0, wt, ahi, amd, alo);
    }
}

// Sum of per-entry corrections into integer cells, independent of the order in which lanes arrive: the terms of a
// tile's outlier list are brought to fixed point with one scale for the tile (from the largest term) and added with
// integer atomics.  A term is split into a high part (units of 2^eu, below 2^24 of them) and the exact remainder in
// units of 2^(eu-20), so a cell keeps about 44 bits below the largest term of the tile whatever the other cells hold.
// term(e) gives the cell and the binary32 term of entry e; cells[0][.] / cells[1][.] take the high / low parts.
// Returns the weight of one high unit (0: nothing was added).
constexpr float OUTL_LO = 1048576.0f;     // 2^20 low units per high unit
template <int NCELL, typename F>
__device__ __forceinline__ float outlier_sums(uint32_t count, int lane, int (*cells)[NCELL], F term) {
    float mx = 0.f;
#pragma unroll 1
    for (uint32_t e = lane; e < count; e += 32) {
        int cell; float t;
        term(e, cell, t);
        mx = fmaxf(mx, fabsf(t));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    if (!(mx > 0.f) || !(mx < 3.0e38f)) return 0.f;        // nothing to add (or not finite: left out)
    // largest term below 2^24 units, so that the up to 128 terms of a cell stay inside 32 bits
    const int ex = (__float_as_int(mx) >> 23) & 0xFF;       // mx < 2^(ex-126)
    const int eu = max(-100, min(100, ex - 126 - 24));      // one unit = 2^eu
    const float inv = __int_as_float((127 - eu) << 23), unit = __int_as_float((127 + eu) << 23);
#pragma unroll 1
    for (uint32_t e = lane; e < count; e += 32) {
        int cell; float t;
        term(e, cell, t);
        const float hi = rintf(t * inv);
        const float rem = fmaf(-hi, unit, t);               // exact: |rem| <= unit / 2
        atomicAdd(&cells[0][cell], (int)hi);
        atomicAdd(&cells[1][cell], __float2int_rn(rem * inv * OUTL_LO));
    }
    return unit;
}

// One CTA = one run of consecutive tiles, which meets one or two (b,h): the body below runs once
// per (b,h) segment and leaves one partial per segment.  Every warp works through whole tiles on its
// own: own running max / sum / accumulators, own staging buffers, no CTA barrier in the loop; the
// warps are merged once at the end.  The packed bytes of the next tile are copied to shared memory
// with cp.async while the current one is being processed: the keys during the value phase, the
// values during the key phase.  Lane l looks after tokens l and l + 32 of the tile (logit, softmax
// weight, fixed-point value weight); the section loops spread the items over the lanes.
template <int D>
__global__ void __launch_bounds__(DEC_THREADS, DEC_CTAS_PER_SM) decode_kernel(const DecArgs a) {
    constexpr int P = D / 32;        // lanes per key item
    constexpr int LPG = D / 8;       // lanes per value group
    constexpr int HALF = QAQ_TILE / 2;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecSmem<D>& sm = *reinterpret_cast<DecSmem<D>*>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int part = lane % P, sub = lane / P;
    const int vh = lane % LPG, vgrp = lane / LPG;
    const unsigned lt = (1u << lane) - 1u;
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
    for (int d = lane; d < D; d += 32) { ws.vout[d] = 0.f; ws.ivout[0][d] = 0; ws.ivout[1][d] = 0; }
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

    float X[8];                 // this lane's 8 channels (8*vh ..), summed over the groups this lane has handled
#pragma unroll
    for (int i = 0; i < 8; ++i) X[i] = 0.f;
    float m_run = __int_as_float(0xff800000), l_run = 0.f, lx_run = 0.f;   // lx: sum of the unperturbed p
    float c_run = 0.f;       // per-lane part of sum_t p_t * (min_t + step_t/2) of the values

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
    // a tile's bytes (rounded up to 16, never more than the buffer holds) and its outlier entries
    auto stage = [&](uint8_t* dst, const uint8_t* pool, uint32_t off, uint32_t nbytes, uint32_t cap) {
        nbytes = (min(nbytes, cap) + 15u) & ~15u;
        if ((size_t)off + nbytes > a.pool_bytes) nbytes = 0;      // a table entry that points outside the pool is not followed
#pragma unroll 1
        for (uint32_t o = lane * 16; o < nbytes; o += 32 * 16) cp_async<16>(dst + o, pool + off + o);
    };
    auto stage_outl = [&](int x, uint32_t first, uint32_t count) {   // entries are 4 bytes, lists start 16-byte aligned
        const uint32_t* src = (x ? a.v.outl : a.k.outl) + (size_t)bh * a.ocap + first;
        const uint32_t n16 = ((count < (uint32_t)OSTAGE ? count : (uint32_t)OSTAGE) + 3u) >> 2;
        if ((size_t)first + 4 * n16 > a.ocap) return;
#pragma unroll 1
        for (uint32_t o = lane; o < n16; o += 32) cp_async<16>(&ws.outl[x][4 * o], src + 4 * o);
    };
    auto stage_K = [&](const Meta& m) {
        stage(ws.bufK, poolK, __shfl_sync(0xFFFFFFFFu, m.tb, 0), __shfl_sync(0xFFFFFFFFu, m.tb, 1), QAQ_TILE * D);
        stage_outl(0, __shfl_sync(0xFFFFFFFFu, m.tb, 2), __shfl_sync(0xFFFFFFFFu, m.tb, 3));
        cp_async_commit();
    };
    auto stage_V = [&](const Meta& m) {
        stage(ws.bufV, poolV, __shfl_sync(0xFFFFFFFFu, m.tb, 4), __shfl_sync(0xFFFFFFFFu, m.tb, 5), (uint32_t)sizeof(ws.bufV) - 16u);
        stage_outl(1, __shfl_sync(0xFFFFFFFFu, m.tb, 6), __shfl_sync(0xFFFFFFFFu, m.tb, 7));
        cp_async_commit();
    };
    int tile = tile_lo + warp;
    Meta cur = fetch_meta(tile);
    Meta nxt = fetch_meta(tile + DEC_WARPS);
    if (tile < tile_hi) { stage_K(cur); stage_V(cur); }

    for (; tile < tile_hi; tile += DEC_WARPS) {
        const uint32_t ooK = __shfl_sync(0xFFFFFFFFu, cur.tb, 2), ocK = __shfl_sync(0xFFFFFFFFu, cur.tb, 3);
        const uint32_t ooV = __shfl_sync(0xFFFFFFFFu, cur.tb, 6), ocV = __shfl_sync(0xFFFFFFFFu, cur.tb, 7);
        const bool has_next = tile + DEC_WARPS < tile_hi;
        const int t0 = tile * QAQ_TILE + lane;              // this lane's tokens: t0 and t0 + 32
        const bool val0 = t0 < a.T, val1 = t0 + HALF < a.T;

        // ---- widths, ranks of this lane's tokens in the sections, section sizes
        int B[2][2];          // [tensor][token]
        uint32_t rk[2][2];    // rank in section c in byte c
        int n[2][4];
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            B[x][0] = val0 ? min(8, (int)((cur.bits4 >> (16 * x)) & 0xFF)) : 0;
            B[x][1] = val1 ? min(8, (int)((cur.bits4 >> (16 * x + 8)) & 0xFF)) : 0;
            rk[x][0] = rk[x][1] = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const unsigned b0 = __ballot_sync(0xFFFFFFFFu, (B[x][0] & (8 >> c)) != 0);
                const unsigned b1 = __ballot_sync(0xFFFFFFFFu, (B[x][1] & (8 >> c)) != 0);
                const int n0 = __popc(b0);
                n[x][c] = n0 + __popc(b1);
                rk[x][0] |= (uint32_t)__popc(b0 & lt) << (8 * c);
                rk[x][1] |= (uint32_t)(n0 + __popc(b1 & lt)) << (8 * c);
            }
        }
        uint32_t kb[5], vb[5];
        qaqc::section_bases<D, false>(n[0], kb);
        qaqc::section_bases<D, true>(n[1], vb);

        // ---- per-token scalars
        float stepK[2], stepV[2], midV[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const bool v = j ? val1 : val0;
            const uint32_t mk = cur.mm[j], mv = cur.mm[2 + j];
            const float kmn = __half2float(__ushort_as_half((unsigned short)(mk & 0xFFFF)));
            const float kmx = __half2float(__ushort_as_half((unsigned short)(mk >> 16)));
            const float vmn = __half2float(__ushort_as_half((unsigned short)(mv & 0xFFFF)));
            const float vmx = __half2float(__ushort_as_half((unsigned short)(mv >> 16)));
            stepK[j] = v ? qaqc::step_of(kmn, kmx, B[0][j]) : 0.f;
            stepV[j] = v ? qaqc::step_of(vmn, vmx, B[1][j]) : 0.f;
            ws.midK[lane + HALF * j] = v ? fmaf(0.5f, stepK[j], kmn) : 0.f;
            midV[j] = v ? fmaf(0.5f, stepV[j], vmn) : 0.f;
            ws.midV[lane + HALF * j] = midV[j];
            ws.iocorr[0][lane + HALF * j] = 0;
            ws.iocorr[1][lane + HALF * j] = 0;
        }
        cp_async_wait<1>();     // this tile's keys have landed (its values may still be in flight)
        __syncwarp();

        // ---- K: integer dot products per section
        k_section<D, 8>(ws.bufK + kb[0], n[0][0], ws.dotw[0], qh, ql, part, sub);
        k_section<D, 4>(ws.bufK + kb[1], n[0][1], ws.dotw[1], qh, ql, part, sub);
        k_section<D, 2>(ws.bufK + kb[2], n[0][2], ws.dotw[2], qh, ql, part, sub);
        k_section<D, 1>(ws.bufK + kb[3], n[0][3], ws.dotw[3], qh, ql, part, sub);
        // key outliers: q_ch * (x - mid) per token
        const uint32_t* ogK = a.k.outl + (size_t)bh * a.ocap + ooK;
        const float ounit = outlier_sums(ocK, lane, ws.iocorr, [&](uint32_t e, int& cell, float& t) {
            const uint32_t v = e < (uint32_t)OSTAGE ? ws.outl[0][e] : __ldg(ogK + e);
            cell = (v >> 24) & (QAQ_TILE - 1);
            t = sm.qf[(v >> 16) & (D - 1)] * (__half2float(__ushort_as_half((unsigned short)(v & 0xFFFF))) - ws.midK[cell]);
        });
        __syncwarp();
        // ---- the key buffer is free: start the copy of the next tile's keys
        if (has_next) stage_K(nxt); else cp_async_commit();

        // ---- logits of this lane's tokens; running max / sum
        float lg[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            int dot = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int w = 8 >> c;
                if (B[0][j] & w) dot += ws.dotw[c][(rk[0][j] >> (8 * c)) & 0xFF] << (B[0][j] & (w - 1));
            }
            lg[j] = __int_as_float(0xff800000);
            if (j ? val1 : val0) {
                const int tk = lane + HALF * j;
                const float qk = fmaf(qscale * stepK[j], (float)dot, fmaf(ws.midK[tk], qsum, ounit * fmaf((float)ws.iocorr[1][tk], 1.0f / OUTL_LO, (float)ws.iocorr[0][tk])));
                lg[j] = a.scale * qk;
                if (a.scores) a.scores[(size_t)bh * a.T + t0 + HALF * j] = lg[j];
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
            for (int i = 0; i < 8; ++i) X[i] *= alpha;
            c_run *= alpha;
            for (int d = lane; d < D; d += 32) ws.vout[d] *= alpha;
        }
        // ---- value weights p * step * 2^shift as 24-bit fixed point with one scale for the tile (a token's step
        //      falls with its width, so next to a 2-bit token an 8-bit token of the same p has a weight 64 times
        //      smaller: 16 bits would leave it about 10).  The weight of the
        //      token's lowest piece is rounded once; the other pieces use exact multiples of it, and p is replaced
        //      by what the rounded weight stands for, so that the pieces, the constant part and the softmax
        //      denominator all see the same (slightly perturbed) probability.
        float pe[2], wf[2];
        int top[2];
        float wmax = 0.f;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            pe[j] = __expf(lg[j] - m_new);           // 0 for slots beyond T
            wf[j] = pe[j] * stepV[j];
            const int Bv = B[1][j];
            top[j] = Bv ? Bv - (1 << (31 - __clz(Bv))) : 0;      // shift of the widest piece
            wmax = fmaxf(wmax, wf[j] * __int_as_float((127 + top[j]) << 23));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) wmax = fmaxf(wmax, __shfl_xor_sync(0xFFFFFFFFu, wmax, o));
        // wmax < 2^(ex-126): one unit = 2^(ex-126-24) keeps every shifted weight below 2^24
        const int wex = (__float_as_int(wmax) >> 23) & 0xFF;
        const bool wok = wex > 24 && wex < 255;                    // zero, tiny or non-finite weights: the pieces add nothing
        const float wunit = wok ? __int_as_float((wex - 23) << 23) : 0.f;
        const float winv = wok ? __int_as_float((254 - (wex - 23)) << 23) : 0.f;
        float s = 0.f, sx = 0.f;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int Bv = B[1][j];
            uint32_t iw = (uint32_t)__float2int_rn(wf[j] * winv);
            iw = min(iw, 0xFFFFFFu >> top[j]);
            float p = pe[j];
            if (stepV[j] > 0.f && wok) p = __fdividef((float)iw * wunit, stepV[j]);
            uint8_t* wb = reinterpret_cast<uint8_t*>(ws.wts);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int w = 8 >> c;
                if (Bv & w) {
                    const uint32_t r = (rk[1][j] >> (8 * c)) & 0xFF, wt = iw << (Bv & (w - 1));
                    uint8_t* g = wb + c * (QAQ_TILE / 4) * 16 + (r >> 2) * 16 + (r & 3);
                    g[0] = (uint8_t)(wt >> 16);
                    g[4] = (uint8_t)(wt >> 8);
                    g[8] = (uint8_t)wt;
                }
            }
            c_run = fmaf(p, midV[j], c_run);
            s += p; sx += pe[j];
            ws.p[lane + HALF * j] = p;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
            sx += __shfl_xor_sync(0xFFFFFFFFu, sx, o);
        }
        l_run = l_run * alpha + s;
        lx_run = lx_run * alpha + sx;
        cp_async_wait<1>();     // this tile's values have landed
        __syncwarp();

        // ---- V: integer weighted sums per section, added to the binary32 accumulators once per tile
        if (wok) {
            int ahi[8], amd[8], alo[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { ahi[i] = 0; amd[i] = 0; alo[i] = 0; }
            v_section<D, 8>(ws.bufV + vb[0], (n[1][0] + 3) >> 2, ws.wts[0], ahi, amd, alo, vh, vgrp);
            v_section<D, 4>(ws.bufV + vb[1], (n[1][1] + 3) >> 2, ws.wts[1], ahi, amd, alo, vh, vgrp);
            v_section<D, 2>(ws.bufV + vb[2], (n[1][2] + 3) >> 2, ws.wts[2], ahi, amd, alo, vh, vgrp);
            v_section<D, 1>(ws.bufV + vb[3], (n[1][3] + 3) >> 2, ws.wts[3], ahi, amd, alo, vh, vgrp);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                X[i] = fmaf(fmaf((float)ahi[i], 65536.0f, (float)(amd[i] * 256 + alo[i])), wunit, X[i]);
        }
        // value outliers: p_t * (v - mid) per channel
        const uint32_t* ogV = a.v.outl + (size_t)bh * a.ocap + ooV;
        const float vunit = outlier_sums(ocV, lane, ws.ivout, [&](uint32_t e, int& cell, float& t) {
            const uint32_t v = e < (uint32_t)OSTAGE ? ws.outl[1][e] : __ldg(ogV + e);
            const int tok = (v >> 24) & (QAQ_TILE - 1);
            cell = (v >> 16) & (D - 1);
            t = ws.p[tok] * (__half2float(__ushort_as_half((unsigned short)(v & 0xFFFF))) - ws.midV[tok]);
        });
        __syncwarp();
        if (vunit != 0.f) {
            for (int d = lane; d < D; d += 32) {
                ws.vout[d] = fmaf(fmaf((float)ws.ivout[1][d], 1.0f / OUTL_LO, (float)ws.ivout[0][d]), vunit, ws.vout[d]);
                ws.ivout[0][d] = 0; ws.ivout[1][d] = 0;
            }
        }
        __syncwarp();
        // ---- the value buffer is free: start the copy of the next tile's values
        if (has_next) stage_V(nxt); else cp_async_commit();
        cur = nxt;
        nxt = fetch_meta(tile + 2 * DEC_WARPS);
    }
    cp_async_wait<0>();

    // ---- warp result: lanes with the same vh hold partial sums of the same channels
    float cs = c_run;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cs += __shfl_xor_sync(0xFFFFFFFFu, cs, o);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float v = X[i];
#pragma unroll
        for (int o = LPG; o < 32; o <<= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if (vgrp == 0) sm.macc[warp][8 * vh + i] = v + ws.vout[8 * vh + i] + cs;
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
constexpr int DEC_SLOTS = 148 * DEC_CTAS_PER_SM;
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
