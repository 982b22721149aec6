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
// Both sums over codes run on the integer tensor-core instruction mma.sync.m16n8k32 (u8 x s8 -> s32).  A plane
// word of the cache, after one shift and a byte-replicated mask, holds one w-bit field per byte lane, which is
// exactly an A-operand register of that instruction (four consecutive k), so a decode step - a GEMV, whose cost
// here is taking bit fields apart, not multiplying - spends one instruction per 512 code-times-weight products
// instead of one per four.  The exact integer sums make the result independent of any accumulation order.
//   q.K:  rows = 16 tokens of a section, k = channels; B = q in 16-bit fixed point per (b,h), split into two
//         signed byte digits that sit in columns 0 and 1 (q_d ~ qscale * (256 * hi_d + lo_d)).
//   S.V:  rows = 16 channels, k = 32 tokens of a section (the value pieces of four tokens share a word, one per
//         byte lane); B = the per-token weights p_t * step_t * 2^shift in 23-bit fixed point with one scale per
//         tile, three signed byte digits in columns 0..2.  The integer sums of a tile are added to binary32
//         accumulators once per tile.  The rounded weight of a token is also what the softmax denominator and the
//         constant part of its values use, so numerator and denominator see the same slightly perturbed probability.
//
// One CTA = one run of consecutive tiles of the flattened (b,h, tile) sequence (runs of equal length, so every SM
// gets the same amount of work); each warp works through whole tiles (QAQ_TILE tokens) on its own, with its own
// running max / sum / accumulators and no CTA barrier in the tile loop; warps are merged once at the end.  A tile
// is stored as sections of equal-width pieces behind a header of four masks (qaq_codec.cuh), so every inner loop
// runs one extraction routine over the items of one section, and a token finds its items by its rank among the
// tokens that have a piece of that width (population counts on the masks; no lists are built, the per-token
// widths are not read).  The packed bytes of the next tile are copied to a per-warp shared-memory buffer with
// cp.async while the current one is worked on: the keys during the value phase (at the front of the buffer), the
// values during the key phase (at its back).  The buffer is sized for typical tiles; a tile that does not fit
// beside its neighbour is read in place from global memory by the same loops.
//
// Outlier corrections are summed in fixed point with 32-bit integer atomics in shared memory (a high and a low
// part with fixed scales), so the result does not depend on the order in which lanes arrive.
#include "qaq_decode_common.cuh"

namespace {

using namespace qaqd;

constexpr int DEC_WARPS = 4;
constexpr int DEC_THREADS = DEC_WARPS * 32;
constexpr int DEC_CTAS_PER_SM = 4;

struct DecArgs {
    TensorStore k, v;
    size_t pool_bytes;
    uint32_t ocap;
    int tmax_pad, ntiles_max;
    int T;
    const int* d_count;          // counted kernels only: the token count in device memory (T, run and ncta are then derived from it)
    const __half* q;
    long q_stride, out_stride;   // elements between the rows of consecutive (b,h) in q and in out
    float scale;
    float* part;       // [ncta][2][D+3]: accumulators, running max, sum of the weights used, exact sum
    float* ml;         // [BH][2]   merged (max, sum) for score normalisation
    int BH, run, ncta; // (b,h) count; tiles per CTA of the flattened (b,h, tile) sequence; CTAs
    float* out;        // [BH][D]
    float* scores;     // [BH][scores_stride] or null
    long scores_stride;
};

// The flattened sequence of BH * ntiles tiles is cut into runs of `run` consecutive tiles, one CTA
// each: enough CTAs to fill every SM (148 SMs, 4 resident CTAs each) evenly, at least one tile per
// warp where there are that many, and never more than one (b,h) boundary inside a run.
constexpr int DEC_SLOTS = 148 * DEC_CTAS_PER_SM;
struct DecPlan { int run, ncta; };
__host__ __device__ inline DecPlan plan_decode(int BH, int ntiles) {
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

constexpr int OL_STAGED = 96;     // outlier entries per tile and tensor that come through shared memory; more are read in place

// per-warp scratch for the tile a warp is working on
template <int D>
struct WarpScratch {
    static constexpr int STAGE = 72 * D;      // bytes of the staging buffer (9 KB at head_dim 128: four CTAs per SM)
    alignas(16) uint8_t buf[STAGE];           // keys of a tile from the front, values from the back
    union alignas(16) {                       // the key phase is over (logits taken) before the value weights are written
        int dotw[4][QAQ_TILE];                // integer q . piece per section and rank
        uint32_t wts[4][QAQ_TILE / 4][4];     // per section and value group: the three byte digits of the four weights
    };
    uint32_t olist[2][OL_STAGED];             // the first outlier entries of the tile's keys / values (copied in with the packed words)
    float midK[QAQ_TILE];       // min + step/2
    float midV[QAQ_TILE];
    float p[QAQ_TILE];          // attention weights of the tile's tokens at the current scale of the running sums
    int kcorr[2][QAQ_TILE];     // fixed-point sums (high, low part) of the key-outlier corrections per token (zero between tiles)
    int vcorr[2][D];            // ... of the value-outlier corrections per channel (zero between tiles)
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

// q . piece for the items of one key section: 16 items per instruction row block, lane 4g+t holds the channels
// 4*(t*NR + r) + i (r < NR = D/16) of items g and g+8
template <int D, int W>
__device__ __forceinline__ void k_section(const uint8_t* sec, int n, int* dots, const uint32_t (&qb)[D / 16], int g, int t) {
    constexpr int NR = D / 16, ITEM = D * W / 8;
#pragma unroll 1
    for (int i0 = 0; i0 < n; i0 += 16) {
        const int r0 = i0 + g, r1 = r0 + 8;
        uint32_t x0[NR], x1[NR];
        fetch_regs<W, NR>(sec + r0 * ITEM, t * NR, r0 < n, x0);
        fetch_regs<W, NR>(sec + r1 * ITEM, t * NR, r1 < n, x1);
        int d[4] = {0, 0, 0, 0};
#pragma unroll
        for (int m = 0; m < NR / 2; ++m) mma_u8s8(d, x0[2 * m], x1[2 * m], x0[2 * m + 1], x1[2 * m + 1], qb[2 * m], qb[2 * m + 1]);
        if (t == 0) {          // columns 0 and 1: the high and the low digit of q
            if (r0 < n) dots[r0] = d[0] * 256 + d[1];
            if (r1 < n) dots[r1] = d[2] * 256 + d[3];
        }
    }
}

// weighted sums over the groups of one value section: 8 groups (32 tokens) per instruction, lane 4g+t holds the
// channels (D/8)*g + 2*mb + s (rows g + 8s of row block mb) of groups t and t+4
template <int D, int W>
__device__ __forceinline__ void v_section(const uint8_t* sec, int ngroups, const uint32_t (*wts)[4], int (&acc)[D / 16][4], int g, int t) {
    constexpr int NRV = D / 8, GB = D * W / 2;
#pragma unroll 1
    for (int g0 = 0; g0 < ngroups; g0 += 8) {
        const int ga = g0 + t, gb = ga + 4;
        uint32_t xa[NRV], xb[NRV];
        fetch_regs<W, NRV>(sec + ga * GB, g * NRV, ga < ngroups, xa);
        fetch_regs<W, NRV>(sec + gb * GB, g * NRV, gb < ngroups, xb);
        const uint32_t b0 = (g < 3 && ga < ngroups) ? wts[ga][g] : 0u;
        const uint32_t b1 = (g < 3 && gb < ngroups) ? wts[gb][g] : 0u;
#pragma unroll
        for (int mb = 0; mb < D / 16; ++mb) mma_u8s8(acc[mb], xa[2 * mb], xa[2 * mb + 1], xb[2 * mb], xb[2 * mb + 1], b0, b1);
    }
}

// One CTA = one run of consecutive tiles, which meets one or two (b,h): the body below runs once
// per (b,h) segment and leaves one partial per segment.  Every warp works through whole tiles on its
// own: own running max / sum / accumulators, own staging buffer, no CTA barrier in the loop; the
// warps are merged once at the end.  Lane l looks after tokens l and l + 32 of the tile (logit, softmax
// weight, fixed-point value weight); in the section loops lane 4g+t is lane (g, t) of the tensor-core fragments.
// COUNTED: the token count is read from device memory and the split derived from it here (the grid is then the
// largest one any count needs; CTAs beyond the split find no tiles and leave).
template <int D, bool COUNTED>
__global__ void __launch_bounds__(DEC_THREADS, DEC_CTAS_PER_SM) decode_kernel(const DecArgs a) {
    constexpr int NR = D / 16;       // key operand registers per lane and item
    constexpr int MB = D / 16;       // 16-channel row blocks of the value side
    constexpr int HALF = QAQ_TILE / 2;
    constexpr uint32_t STAGE = WarpScratch<D>::STAGE;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecSmem<D>& sm = *reinterpret_cast<DecSmem<D>*>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int fg = lane >> 2, ft = lane & 3;
    const unsigned lt = (1u << lane) - 1u;
    WarpScratch<D>& ws = sm.ws[warp];
    const int T = COUNTED ? *a.d_count : a.T;
    if (COUNTED && T < 1) return;
    const int run = COUNTED ? plan_decode(a.BH, (T + QAQ_TILE - 1) / QAQ_TILE).run : a.run;

#pragma unroll 1
    for (int seg = 0; seg < 2; ++seg) {
    // this CTA's run of the flattened (b,h, tile) sequence; it touches at most two (b,h).  The block
    // index is read afresh for each segment so that none of this stays in registers over the tile loop.
    int cta;
    asm volatile("mov.u32 %0, %%ctaid.x;" : "=r"(cta));
    const int ntiles = (T + QAQ_TILE - 1) / QAQ_TILE;
    const int flat_lo = cta * run, flat_hi = min(a.BH * ntiles, flat_lo + run);
    const int bh = flat_lo / ntiles + seg;
    const int tile_lo = max(flat_lo, bh * ntiles) - bh * ntiles, tile_hi = min(flat_hi, (bh + 1) * ntiles) - bh * ntiles;
    if (tile_lo >= tile_hi) continue;   // the same for every thread of the CTA

    // ---- q: float copy, fixed-point byte digits per lane
    float qmax = 0.f, qs = 0.f;
    for (int d = tid; d < D; d += DEC_THREADS) {
        const float f = __half2float(a.q[(size_t)bh * a.q_stride + d]);
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
    for (int d = lane; d < D; d += 32) { ws.vcorr[0][d] = 0; ws.vcorr[1][d] = 0; }
    for (int i = lane; i < QAQ_TILE; i += 32) { ws.kcorr[0][i] = 0; ws.kcorr[1][i] = 0; }
    __syncthreads();
    if (tid == 0) {
        float m = 0.f, s = 0.f;
        for (int w = 0; w < DEC_WARPS; ++w) { m = fmaxf(m, sm.red[w]); s += sm.red2[w]; }
        sm.qscale = m / 32639.0f;        // |q| <= 32639 units: both byte digits of 256 * hi + lo stay signed bytes
        sm.qsum = s;
    }
    __syncthreads();
    const float qscale = sm.qscale, qsum = sm.qsum;
    const float qinv = qscale > 0.f ? 1.0f / qscale : 0.f;
    uint32_t qb[NR];             // column fg of the B operand: the high (fg = 0) or low (fg = 1) digit, zero otherwise
#pragma unroll
    for (int r = 0; r < NR; ++r) {
        uint32_t v = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int qi = __float2int_rn(sm.qf[4 * (ft * NR + r) + i] * qinv);
            qi = max(-32639, min(32639, qi));
            const int dg = fg == 0 ? ((qi + 128) >> 8) : qi;     // 256 * hi + lo with lo in [-128, 127]
            v |= (uint32_t)(dg & 0xFF) << (8 * i);
        }
        qb[r] = fg < 2 ? v : 0u;
    }

    float X[MB][2];             // rows fg and fg + 8 of row block mb: this lane's share of the digit columns (summed over ft at the end)
#pragma unroll
    for (int mb = 0; mb < MB; ++mb) { X[mb][0] = 0.f; X[mb][1] = 0.f; }
    // what the accumulator columns of this lane stand for: lane ft = 0 holds the digits 2^16 and 2^8, ft = 1 the units
    const float dig0 = ft == 0 ? 65536.0f : (ft == 1 ? 1.0f : 0.f), dig1 = ft == 0 ? 256.0f : 0.f;
    float m_run = __int_as_float(0xff800000), l_run = 0.f, lx_run = 0.f;   // lx: sum of the unperturbed p
    float c_run = 0.f;       // per-lane part of sum_t p_t * (min_t + step_t/2) of the values
    float vout[(D + 31) / 32];   // value-outlier corrections of channels lane, lane + 32, ...
#pragma unroll
    for (int k = 0; k < (D + 31) / 32; ++k) vout[k] = 0.f;

    const size_t trow = (size_t)bh * a.ntiles_max;
    const size_t mrow = (size_t)bh * a.tmax_pad;
    const uint8_t* poolK = a.k.codes + (size_t)bh * a.pool_bytes;
    const uint8_t* poolV = a.v.codes + (size_t)bh * a.pool_bytes;
    const uint32_t* ogK = a.k.outl + (size_t)bh * a.ocap;
    const uint32_t* ogV = a.v.outl + (size_t)bh * a.ocap;

    // ---- tile metadata in registers: table words in lanes 0..7 (offset and length of the bytes, first entry and
    //      length of the outlier list; keys in lanes 0..3, values in 4..7), min/max of tokens lane, lane+32.
    //      Table entries that point outside the pool or the list are not followed (length 0).
    //      The loads are only issued here; nothing looks at what they return before settle() does, a tile later.
    struct Meta { uint32_t tb, mm[4]; };
    auto fetch_meta = [&](int tile) {
        Meta m;
        m.tb = 0; m.mm[0] = m.mm[1] = m.mm[2] = m.mm[3] = 0;
        if (tile < tile_hi) {
            if (lane < 8) {
                const TensorStore& ts = (lane >= 4) ? a.v : a.k;
                const uint32_t* tab = (lane & 2) ? ((lane & 1) ? ts.tile_ocnt : ts.tile_ooff) : ((lane & 1) ? ts.tile_nbytes : ts.tile_off);
                m.tb = tab[trow + tile];
            }
            const size_t t0 = mrow + (size_t)tile * QAQ_TILE + lane;
            m.mm[0] = a.k.mnmx[t0]; m.mm[1] = a.k.mnmx[t0 + 32]; m.mm[2] = a.v.mnmx[t0]; m.mm[3] = a.v.mnmx[t0 + 32];
        }
        return m;
    };
    // the table words of a tile as they are used: a length becomes 0 where offset and length point outside the pool
    // or the list (lanes 2k, 2k+1 hold an offset and its length)
    auto settle = [&](uint32_t tb) -> uint32_t {
        const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, tb, 1);
        const uint32_t first = (lane & 1) ? other : tb, len = (lane & 1) ? tb : other;
        const bool bad = (lane & 2) ? ((size_t)first + len > a.ocap)
                                    : ((first & 15u) || len < (uint32_t)qaqc::QAQ_TILE_HDR || (size_t)first + ((len + 15u) & ~15u) > a.pool_bytes);
        return lane < 8 ? ((lane & 1) ? (bad ? 0u : len) : first) : 0u;
    };
    // copies nb bytes (a multiple of 16) of a tile to the staging buffer
    auto stage = [&](uint8_t* dst, const uint8_t* src, uint32_t nb) {
        unsigned sa = (unsigned)__cvta_generic_to_shared(dst) + lane * 16;
        const uint8_t* g = src + lane * 16;
#pragma unroll 1
        for (uint32_t o = lane * 16; o < nb; o += 4 * 512, sa += 4 * 512, g += 4 * 512) {      // four copies per round
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (o + 512u * u < nb) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(sa + 512u * u), "l"(g + 512 * u));
        }
    };
    // the first entries of a tile's outlier list, 4 bytes each, into the warp's scratch (part of the copy group open then)
    // (lists of whole tiles start on 16-byte boundaries: four entries per copy, reading up to three entries past the
    // list, which the capacity's read-ahead margin covers; a list that grew with an open tile may start anywhere)
    auto stage_list = [&](uint32_t* dst, const uint32_t* src, uint32_t cnt) {
        if (((uintptr_t)src & 15) == 0) {
            if (lane < OL_STAGED / 4 && 4u * lane < cnt) cp_async<16>(dst + 4 * lane, src + 4 * lane);
        } else {
#pragma unroll
            for (int k = 0; k < OL_STAGED / 32; ++k)
                if (lane + 32 * k < cnt) {
                    const unsigned sa = (unsigned)__cvta_generic_to_shared(dst + lane + 32 * k);
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(sa), "l"(src + lane + 32 * k));
                }
        }
    };
    int tile = tile_lo + warp;
    Meta cur = fetch_meta(tile);
    Meta nxt = fetch_meta(tile + DEC_WARPS);
    cur.tb = settle(cur.tb);
    // what is staged: bytes (rounded up to 16) of the current keys / values in the buffer, 0 = read in place
    uint32_t stK = 0, stV = 0;
    if (tile < tile_hi) {
        const uint32_t nbK = (__shfl_sync(0xFFFFFFFFu, cur.tb, 1) + 15u) & ~15u, nbV = (__shfl_sync(0xFFFFFFFFu, cur.tb, 5) + 15u) & ~15u;
        if (nbK <= STAGE) { stK = nbK; stage(ws.buf, poolK + __shfl_sync(0xFFFFFFFFu, cur.tb, 0), nbK); }
        stage_list(ws.olist[0], ogK + __shfl_sync(0xFFFFFFFFu, cur.tb, 2), __shfl_sync(0xFFFFFFFFu, cur.tb, 3));
        cp_async_commit();
        if (stK + nbV <= STAGE) { stV = nbV; stage(ws.buf + STAGE - nbV, poolV + __shfl_sync(0xFFFFFFFFu, cur.tb, 4), nbV); }
        stage_list(ws.olist[1], ogV + __shfl_sync(0xFFFFFFFFu, cur.tb, 6), __shfl_sync(0xFFFFFFFFu, cur.tb, 7));
        cp_async_commit();
    }

    for (; tile < tile_hi; tile += DEC_WARPS) {
        const uint32_t offK = __shfl_sync(0xFFFFFFFFu, cur.tb, 0), nbK = __shfl_sync(0xFFFFFFFFu, cur.tb, 1);
        const uint32_t ooK = __shfl_sync(0xFFFFFFFFu, cur.tb, 2), ocK = __shfl_sync(0xFFFFFFFFu, cur.tb, 3);
        const uint32_t offV = __shfl_sync(0xFFFFFFFFu, cur.tb, 4), nbV = __shfl_sync(0xFFFFFFFFu, cur.tb, 5);
        const uint32_t ooV = __shfl_sync(0xFFFFFFFFu, cur.tb, 6), ocV = __shfl_sync(0xFFFFFFFFu, cur.tb, 7);
        const bool has_next = tile + DEC_WARPS < tile_hi;
        const int t0 = tile * QAQ_TILE + lane;              // this lane's tokens: t0 and t0 + 32
        const bool val0 = t0 < T, val1 = t0 + HALF < T;
        const uint8_t* tK = stK ? ws.buf : poolK + offK;
        const uint8_t* tV = stV ? ws.buf + STAGE - stV : poolV + offV;
        cp_async_wait<1>();     // this tile's keys have landed (its values may still be in flight)
        __syncwarp();

        // ---- keys: widths, ranks of this lane's tokens in the sections, section sizes (from the tile's header)
        int B[2][2];          // [tensor][token]
        uint32_t rk[2][2];    // rank in section c in byte c
        int n[2][4];
        B[0][0] = B[0][1] = B[1][0] = B[1][1] = 0;
        rk[0][0] = rk[0][1] = rk[1][0] = rk[1][1] = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint2 mk = nbK ? *reinterpret_cast<const uint2*>(tK + 8 * c) : make_uint2(0u, 0u);
            if ((mk.x >> lane) & 1u) B[0][0] |= 8 >> c;
            if ((mk.y >> lane) & 1u) B[0][1] |= 8 >> c;
            const int n0 = __popc(mk.x);
            n[0][c] = n0 + __popc(mk.y);
            rk[0][0] |= (uint32_t)__popc(mk.x & lt) << (8 * c);
            rk[0][1] |= (uint32_t)(n0 + __popc(mk.y & lt)) << (8 * c);
        }
        if (!val0) B[0][0] = 0;
        if (!val1) B[0][1] = 0;
        uint32_t kb[5];
        qaqc::section_bases<D, false>(n[0], kb);
        // a tile that does not hold the sections its masks ask for is not read: its tokens then count with their
        // constant parts only
        const bool okK = kb[4] <= nbK;
        if (!okK) { n[0][0] = n[0][1] = n[0][2] = n[0][3] = 0; }

        // ---- per-token scalars of the keys
        float stepK[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const bool v = j ? val1 : val0;
            const uint32_t mk = cur.mm[j];
            const float kmn = __half2float(__ushort_as_half((unsigned short)(mk & 0xFFFF)));
            const float kmx = __half2float(__ushort_as_half((unsigned short)(mk >> 16)));
            stepK[j] = v ? qaqc::step_of(kmn, kmx, B[0][j]) : 0.f;
            ws.midK[lane + HALF * j] = v ? fmaf(0.5f, stepK[j], kmn) : 0.f;
        }
        __syncwarp();

        // ---- K: integer dot products per section
        k_section<D, 8>(tK + kb[0], n[0][0], ws.dotw[0], qb, fg, ft);
        k_section<D, 4>(tK + kb[1], n[0][1], ws.dotw[1], qb, fg, ft);
        k_section<D, 2>(tK + kb[2], n[0][2], ws.dotw[2], qb, fg, ft);
        k_section<D, 1>(tK + kb[3], n[0][3], ws.dotw[3], qb, fg, ft);
        // key outliers: q_ch * (x - mid) per token
        auto k_outlier = [&](uint32_t v) {
            const int tok = (v >> 24) & (QAQ_TILE - 1);
            const float tm = sm.qf[(v >> 16) & (D - 1)] * (__half2float(__ushort_as_half((unsigned short)(v & 0xFFFF))) - ws.midK[tok]);
            outlier_add(&ws.kcorr[0][tok], &ws.kcorr[1][tok], tm);
        };
#pragma unroll
        for (int k = 0; k < OL_STAGED / 32; ++k)         // the staged entries: independent chains, side by side
            if (lane + 32u * k < ocK) k_outlier(ws.olist[0][lane + 32 * k]);
#pragma unroll 1
        for (uint32_t e = lane + OL_STAGED; e < ocK; e += 32) k_outlier(__ldg(ogK + ooK + e));
        __syncwarp();
        // ---- the front of the buffer is free: start the copy of the next tile's keys (beside this tile's values)
        uint32_t stKn = 0;
        nxt.tb = settle(nxt.tb);       // fetched a tile ago
        if (has_next) {
            const uint32_t nb = (__shfl_sync(0xFFFFFFFFu, nxt.tb, 1) + 15u) & ~15u;
            if (nb + stV <= STAGE) { stKn = nb; stage(ws.buf, poolK + __shfl_sync(0xFFFFFFFFu, nxt.tb, 0), nb); }
            stage_list(ws.olist[0], ogK + __shfl_sync(0xFFFFFFFFu, nxt.tb, 2), __shfl_sync(0xFFFFFFFFu, nxt.tb, 3));
        }
        cp_async_commit();

        // ---- logits of this lane's tokens; running max / sum
        float lg[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            int dot = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int w = 8 >> c;
                if ((B[0][j] & w) && okK) dot += ws.dotw[c][(rk[0][j] >> (8 * c)) & 0xFF] << (B[0][j] & (w - 1));
            }
            lg[j] = __int_as_float(0xff800000);
            const int tk = lane + HALF * j;
            const int kh = ws.kcorr[0][tk], kl = ws.kcorr[1][tk];
            if (kh | kl) { ws.kcorr[0][tk] = 0; ws.kcorr[1][tk] = 0; }
            if (j ? val1 : val0) {
                const float qk = fmaf(qscale * stepK[j], (float)dot, fmaf(ws.midK[tk], qsum, outlier_sum(kh, kl)));
                lg[j] = a.scale * qk;
                if (a.scores) a.scores[(size_t)bh * a.scores_stride + t0 + HALF * j] = lg[j];
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
            for (int mb = 0; mb < MB; ++mb) { X[mb][0] *= alpha; X[mb][1] *= alpha; }
            c_run *= alpha;
#pragma unroll
            for (int k = 0; k < (D + 31) / 32; ++k) vout[k] *= alpha;
        }
        cp_async_wait<1>();     // this tile's values have landed
        __syncwarp();

        // ---- values: widths, ranks, section sizes; per-token scalars
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint2 mv = nbV ? *reinterpret_cast<const uint2*>(tV + 8 * c) : make_uint2(0u, 0u);
            if ((mv.x >> lane) & 1u) B[1][0] |= 8 >> c;
            if ((mv.y >> lane) & 1u) B[1][1] |= 8 >> c;
            const int n0 = __popc(mv.x);
            n[1][c] = n0 + __popc(mv.y);
            rk[1][0] |= (uint32_t)__popc(mv.x & lt) << (8 * c);
            rk[1][1] |= (uint32_t)(n0 + __popc(mv.y & lt)) << (8 * c);
        }
        if (!val0) B[1][0] = 0;
        if (!val1) B[1][1] = 0;
        uint32_t vb[5];
        qaqc::section_bases<D, true>(n[1], vb);
        const bool okV = vb[4] <= nbV;
        if (!okV) { n[1][0] = n[1][1] = n[1][2] = n[1][3] = 0; }
        float stepV[2], midV[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const bool v = j ? val1 : val0;
            const uint32_t mv = cur.mm[2 + j];
            const float vmn = __half2float(__ushort_as_half((unsigned short)(mv & 0xFFFF)));
            const float vmx = __half2float(__ushort_as_half((unsigned short)(mv >> 16)));
            stepV[j] = v ? qaqc::step_of(vmn, vmx, B[1][j]) : 0.f;
            midV[j] = v ? fmaf(0.5f, stepV[j], vmn) : 0.f;
            ws.midV[lane + HALF * j] = midV[j];
        }
        // ---- value weights p * step * 2^shift as 22-bit fixed point with one scale for the tile (a token's step
        //      falls with its width, so next to a 2-bit token an 8-bit token of the same p has a weight 64 times
        //      smaller: 16 bits would leave it about 10).  The weight of the token's lowest piece is rounded once;
        //      the other pieces use exact multiples of it, and p is replaced by what the rounded weight stands for,
        //      so that the pieces, the constant part and the softmax denominator all see the same (slightly
        //      perturbed) probability.
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
        // wmax < 2^(ex-126): one unit = 2^(ex-126-22) keeps every shifted weight at or below 2^22
        const int wex = (__float_as_int(wmax) >> 23) & 0xFF;
        const bool wok = wex > 24 && wex < 255 && okV;             // zero, tiny or non-finite weights: the pieces add nothing
        const float wunit = wok ? __int_as_float((wex - 21) << 23) : 0.f;
        const float winv = wok ? __int_as_float((254 - (wex - 21)) << 23) : 0.f;
        float s = 0.f, sx = 0.f;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int Bv = B[1][j];
            uint32_t iw = (uint32_t)__float2int_rn(wf[j] * winv);
            iw = min(iw, 0x7F0000u >> top[j]);       // the three balanced byte digits of a shifted weight stay signed bytes
            float p = pe[j];
            if (stepV[j] > 0.f && wok) p = __fdividef((float)iw * wunit, stepV[j]);
            uint8_t* wbytes = reinterpret_cast<uint8_t*>(ws.wts);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int w = 8 >> c;
                if (Bv & w) {
                    const uint32_t r = (rk[1][j] >> (8 * c)) & 0xFF, wt = iw << (Bv & (w - 1));
                    // wt = 65536 * d2 + 256 * d1 + d0 with d1, d0 in [-128, 127]
                    const uint32_t r1 = (wt + 128u) >> 8, r2 = (r1 + 128u) >> 8;
                    uint8_t* gp = wbytes + c * (QAQ_TILE / 4) * 16 + (r >> 2) * 16 + (r & 3);
                    gp[0] = (uint8_t)r2;
                    gp[4] = (uint8_t)r1;
                    gp[8] = (uint8_t)wt;
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
        __syncwarp();

        // ---- V: integer weighted sums per section, added to the binary32 accumulators once per tile
        if (wok) {
            int acc[MB][4];
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) { acc[mb][0] = 0; acc[mb][1] = 0; acc[mb][2] = 0; acc[mb][3] = 0; }
            v_section<D, 8>(tV + vb[0], (n[1][0] + 3) >> 2, ws.wts[0], acc, fg, ft);
            v_section<D, 4>(tV + vb[1], (n[1][1] + 3) >> 2, ws.wts[1], acc, fg, ft);
            v_section<D, 2>(tV + vb[2], (n[1][2] + 3) >> 2, ws.wts[2], acc, fg, ft);
            v_section<D, 1>(tV + vb[3], (n[1][3] + 3) >> 2, ws.wts[3], acc, fg, ft);
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
                X[mb][0] = fmaf(fmaf((float)acc[mb][0], dig0, (float)acc[mb][1] * dig1), wunit, X[mb][0]);
                X[mb][1] = fmaf(fmaf((float)acc[mb][2], dig0, (float)acc[mb][3] * dig1), wunit, X[mb][1]);
            }
        }
        // value outliers: p_t * (v - mid) per channel
        auto v_outlier = [&](uint32_t v) {
            const int tok = (v >> 24) & (QAQ_TILE - 1), ch = (v >> 16) & (D - 1);
            const float tm = ws.p[tok] * (__half2float(__ushort_as_half((unsigned short)(v & 0xFFFF))) - ws.midV[tok]);
            outlier_add(&ws.vcorr[0][ch], &ws.vcorr[1][ch], tm);
        };
#pragma unroll
        for (int k = 0; k < OL_STAGED / 32; ++k)
            if (lane + 32u * k < ocV) v_outlier(ws.olist[1][lane + 32 * k]);
#pragma unroll 1
        for (uint32_t e = lane + OL_STAGED; e < ocV; e += 32) v_outlier(__ldg(ogV + ooV + e));
        __syncwarp();
        if (ocV) {
#pragma unroll
            for (int k = 0; k < (D + 31) / 32; ++k) {
                const int d = lane + 32 * k;
                if (d < D) {
                    const int h = ws.vcorr[0][d], l = ws.vcorr[1][d];
                    if (h | l) { vout[k] += outlier_sum(h, l); ws.vcorr[0][d] = 0; ws.vcorr[1][d] = 0; }
                }
            }
        }
        __syncwarp();
        // ---- the back of the buffer is free: start the copy of the next tile's values (beside its keys)
        uint32_t stVn = 0;
        if (has_next) {
            const uint32_t nb = (__shfl_sync(0xFFFFFFFFu, nxt.tb, 5) + 15u) & ~15u;
            if (nb + stKn <= STAGE) { stVn = nb; stage(ws.buf + STAGE - nb, poolV + __shfl_sync(0xFFFFFFFFu, nxt.tb, 4), nb); }
            stage_list(ws.olist[1], ogV + __shfl_sync(0xFFFFFFFFu, nxt.tb, 6), __shfl_sync(0xFFFFFFFFu, nxt.tb, 7));
        }
        cp_async_commit();
        stK = stKn; stV = stVn;
        cur = nxt;
        nxt = fetch_meta(tile + 2 * DEC_WARPS);
    }
    cp_async_wait<0>();

    // ---- warp result: the four lanes ft of a group hold the digit columns of the same channels
    float cs = c_run;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cs += __shfl_xor_sync(0xFFFFFFFFu, cs, o);
#pragma unroll
    for (int k = 0; k < (D + 31) / 32; ++k)
        if (lane + 32 * k < D) sm.macc[warp][lane + 32 * k] = vout[k] + cs;
    __syncwarp();
#pragma unroll
    for (int mb = 0; mb < MB; ++mb)
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
            float v = X[mb][s2];
            v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
            v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
            const int ch = (D / 8) * fg + 2 * mb + s2;     // row fg + 8*s2 of row block mb
            if (ft == 0) sm.macc[warp][ch] += v;
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
template <int D, bool COUNTED>
__global__ void merge_kernel(const DecArgs a) {
    const int bh = blockIdx.x, d = threadIdx.x;
    const int T = COUNTED ? *a.d_count : a.T;
    if (COUNTED && T < 1) { a.out[(size_t)bh * a.out_stride + d] = 0.f; return; }
    const int ntiles = (T + QAQ_TILE - 1) / QAQ_TILE;
    const int run = COUNTED ? plan_decode(a.BH, ntiles).run : a.run;
    // the CTAs of decode_kernel whose runs meet this (b,h); a CTA's first segment has slot 0
    const int c_lo = (bh * ntiles) / run, c_hi = ((bh + 1) * ntiles - 1) / run;
    // only the first of them can have begun in the (b,h) before
    auto slot = [&](int c) { return a.part + (size_t)(2 * c + (c * run < bh * ntiles ? 1 : 0)) * (D + 3); };
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
    a.out[(size_t)bh * a.out_stride + d] = L > 0.f ? x / L : 0.f;
    if (d == 0) { a.ml[2 * bh] = M; a.ml[2 * bh + 1] = LX; }
}

__global__ void scores_kernel(float* scores, long stride, const float* ml, int T, const int* d_count) {
    const int bh = blockIdx.y;
    if (d_count) T = *d_count;
    const float M = ml[2 * bh], L = ml[2 * bh + 1];
    const float inv = L > 0.f ? 1.0f / L : 0.f;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < T; t += gridDim.x * blockDim.x) {
        float* s = scores + (size_t)bh * stride + t;
        *s = __expf(*s - M) * inv;
    }
}

// floats of workspace for the partials (two slots per CTA) and the merged (max, sum) pairs
size_t decode_ws_floats(int BH, int ncta, int D) { return (size_t)2 * ncta * (D + 3) + (size_t)BH * 2; }

template <int D, bool COUNTED = false>
qaq_status run_decode(const DecArgs& a, int BH, cudaStream_t s) {
    const size_t smem = sizeof(DecSmem<D>);
    if (smem > 48 * 1024)
        QAQ_CUDA_TRY(cudaFuncSetAttribute(decode_kernel<D, COUNTED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_kernel<D, COUNTED><<<a.ncta, DEC_THREADS, smem, s>>>(a);
    merge_kernel<D, COUNTED><<<BH, D, 0, s>>>(a);
    if (a.scores) {
        int gx = (a.T + 1023) / 1024;     // counted: a.T holds the capacity
        if (gx > 64) gx = 64;
        scores_kernel<<<dim3(gx, BH), 256, 0, s>>>(a.scores, a.scores_stride, a.ml, a.T, COUNTED ? a.d_count : nullptr);
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
    a.q = (const __half*)q; a.scale = softmax_scale; a.q_stride = c->cfg.head_dim; a.out_stride = c->cfg.head_dim;
    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const DecPlan plan = plan_decode(BH, ntiles);
    a.BH = BH; a.run = plan.run; a.ncta = plan.ncta;
    a.part = (float*)ws;
    a.ml = a.part + (size_t)2 * plan.ncta * (D + 3);
    a.out = out; a.scores = scores_out; a.scores_stride = a.T; a.d_count = nullptr;
    cudaStream_t s = (cudaStream_t)stream;
    switch (D) {
        case 32: return run_decode<32>(a, BH, s);
        case 64: return run_decode<64>(a, BH, s);
        case 128: return run_decode<128>(a, BH, s);
    }
    return QAQ_ERR_UNSUPPORTED_SHAPE;
}

// One query per (b,h) taken from / written to rows that lie q_stride / out_stride elements apart (used by the
// batched entry point for the queries that do not fill a pass of their own); ws as for qaq_decode_attention.
qaq_status qaq_decode_strided(const qaq_cache* c, const void* q, long q_stride, float softmax_scale, float* out, long out_stride,
                              void* ws, cudaStream_t s) {
    const int D = c->cfg.head_dim, BH = c->BH;
    DecArgs a;
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.ocap = c->ocap;
    a.tmax_pad = c->tmax_pad; a.ntiles_max = c->ntiles; a.T = (int)c->tokens;
    a.q = (const __half*)q; a.scale = softmax_scale; a.q_stride = q_stride; a.out_stride = out_stride;
    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const DecPlan plan = plan_decode(BH, ntiles);
    a.BH = BH; a.run = plan.run; a.ncta = plan.ncta;
    a.part = (float*)ws;
    a.ml = a.part + (size_t)2 * plan.ncta * (D + 3);
    a.out = out; a.scores = nullptr; a.scores_stride = 0; a.d_count = nullptr;
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
    a.q = (const __half*)q; a.scale = softmax_scale; a.q_stride = c->cfg.head_dim; a.out_stride = c->cfg.head_dim;
    a.BH = BH; a.run = plan.run; a.ncta = plan.ncta;
    // Every partial that the merge reads and every (max,sum) pair is written before it is read,
    // so nothing in the scratch has to be cleared between calls.
    a.part = (float*)scratch;
    a.ml = a.part + (size_t)2 * plan.ncta * (D + 3);
    a.out = out; a.scores = nullptr; a.scores_stride = 0; a.d_count = nullptr;
    cudaStream_t s = (cudaStream_t)stream;
    switch (D) {
        case 32: return run_decode<32>(a, BH, s);
        case 64: return run_decode<64>(a, BH, s);
        case 128: return run_decode<128>(a, BH, s);
    }
    return QAQ_ERR_UNSUPPORTED_SHAPE;
}

// Decode attention over as many tokens as the device-side count says (qaq_stream_begin / qaq_stream_append): the
// split over CTAs is derived from the count inside the kernels, the grid is the largest any count needs, and nothing
// on the host is read or changed, so the call can be captured in a CUDA graph and replayed while the cache grows.
extern "C" qaq_status qaq_stream_decode(const qaq_cache* c, const void* q, float softmax_scale, float* out,
                                        float* scores_out, long scores_stride, void* ws, size_t ws_bytes, void* stream) {
    if (!c || !q || !out || !ws) return QAQ_ERR_INVALID_ARG;
    if (scores_out && scores_stride < c->cfg.max_tokens) return QAQ_ERR_INVALID_ARG;
    size_t need = 0;
    qaq_decode_workspace_bytes(c, &need);
    if (ws_bytes < need || ((uintptr_t)ws & 15)) return QAQ_ERR_WORKSPACE;
    const int D = c->cfg.head_dim, BH = c->BH;
    DecArgs a;
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.ocap = c->ocap;
    a.tmax_pad = c->tmax_pad; a.ntiles_max = c->ntiles; a.T = (int)c->cfg.max_tokens;
    a.d_count = qaq_d_count(c);
    a.q = (const __half*)q; a.scale = softmax_scale; a.q_stride = D; a.out_stride = D;
    a.BH = BH; a.run = 0; a.ncta = BH > DEC_SLOTS ? BH : DEC_SLOTS;
    a.part = (float*)ws;
    a.ml = a.part + (size_t)2 * a.ncta * (D + 3);
    a.out = out; a.scores = scores_out; a.scores_stride = scores_stride;
    cudaStream_t s = (cudaStream_t)stream;
    switch (D) {
        case 32: return run_decode<32, true>(a, BH, s);
        case 64: return run_decode<64, true>(a, BH, s);
        case 128: return run_decode<128, true>(a, BH, s);
    }
    return QAQ_ERR_UNSUPPORTED_SHAPE;
}
