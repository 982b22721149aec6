// Batched decode attention: up to four queries per (b,h) in one pass over the packed cache (Section 4.2,
// "Integration in text generation process": the cache is read by every query that follows; Section 5.2 for the
// uniform comparison point).  Same arithmetic per query as qaq_decode.cu; what is paid once per packed entry - the
// staging of a tile, the masks that turn section words into operand registers of mma.m16n8k32 - serves all queries:
// the queries are columns of the B operand.
//   q.K:  columns 2j and 2j+1 hold the two signed byte digits of query j (16-bit fixed point, one scale per query),
//         so one instruction per 16 tokens x 32 channels yields the integer dot products of all four queries;
//         fragment lane t of a row holds the two columns of query t.
//   S.V:  the three byte digits of the 22-bit weights of two queries fill six columns; two instructions on the same
//         operand registers serve four queries.
// One CTA (four warps) = one run of consecutive tiles of the flattened (b,h, tile) sequence, all warps on the same
// tile: the 16-item row blocks of the key sections are dealt out to the warps, every thread owns one token for two
// of the queries (logits, softmax weights and weight digits), and on the value side every warp takes its share of
// the 16-channel row blocks for all tokens, so that the accumulators of four queries stay few per thread.  Whole
// tiles are staged two deep with cp.async.  Four barriers per tile; no warp waits on another CTA.
#include "qaq_decode_common.cuh"

namespace {

using namespace qaqd;

constexpr int MQ = 4;                 // queries per pass
constexpr int MQ_WARPS = 4;
constexpr int MQ_THREADS = MQ_WARPS * 32;
constexpr int MQ_CTAS_PER_SM = 3;

struct MultiArgs {
    TensorStore k, v;
    size_t pool_bytes;
    uint32_t ocap;
    int tmax_pad, ntiles_max;
    int T;
    const __half* q;   // [BH][n_q][D]; this pass takes queries q0 .. q0+nq-1
    int n_q, q0, nq;
    float scale;
    float* part;       // [ncta][2][MQ][D+3]: accumulators, running max, sum of the weights used, exact sum
    int BH, run, ncta;
    float* out;        // [BH][n_q][D]
};

template <int D>
struct MultiSmem {
    static constexpr int BUFB = qaqc::v_tile_bytes_max(D);       // a multiple of 16, header included
    alignas(16) uint8_t buf[2][2][BUFB];      // [stage][tensor]: the packed bytes of a tile
    int dotw[4][QAQ_TILE][MQ];                // integer q . piece per section, rank and query
    alignas(16) uint32_t wts[MQ][4][QAQ_TILE / 4][4];  // per query, section and value group: the three byte digits of the four weights
    float midV[QAQ_TILE];                     // min + step/2 of the values
    float p[MQ][QAQ_TILE];                    // attention weights of the tile's tokens at the current scale of the running sums
    int kcorr[2][MQ][QAQ_TILE];               // fixed-point sums (high, low part) of the key-outlier corrections (zero between tiles)
    int vcorr[2][MQ][D];                      // ... of the value-outlier corrections per channel (zero between tiles)
    float qf[MQ][D];
    float xs[MQ][D];
    float red[MQ_WARPS][MQ], red2[MQ_WARPS][MQ], red3[MQ_WARPS][MQ];
    float mloc[2][MQ], wloc[2];               // per token warp: largest logit per query, largest value weight bound
    float mnew[MQ], wunit;                    // of the current tile: running maxima after it, weight of one fixed-point unit
    float qscale[MQ], qsum[MQ];
};

// q . piece for the items of one key section, all queries at once: lane 4g+t holds the channels 4*(t*NR + r) + i
// of items g and g+8, and receives the two digit columns of query t.  Row blocks are numbered through the sections
// (first = number of this section's first block); block b belongs to warp b mod MQ_WARPS.
template <int D, int W>
__device__ __forceinline__ void k_section_mq(const uint8_t* sec, int n, int (*dots)[MQ], const uint32_t (&qb)[D / 16], int g, int t,
                                             int warp, int& first) {
    constexpr int NR = D / 16, ITEM = D * W / 8;
    const int nblk = (n + 15) >> 4;
#pragma unroll 1
    for (int b = (warp - first) & (MQ_WARPS - 1); b < nblk; b += MQ_WARPS) {
        const int r0 = 16 * b + g, r1 = r0 + 8;
        uint32_t x0[NR], x1[NR];
        fetch_regs<W, NR>(sec + r0 * ITEM, t * NR, r0 < n, x0);
        fetch_regs<W, NR>(sec + r1 * ITEM, t * NR, r1 < n, x1);
        int d[4] = {0, 0, 0, 0};
#pragma unroll
        for (int m = 0; m < NR / 2; ++m) mma_u8s8(d, x0[2 * m], x1[2 * m], x0[2 * m + 1], x1[2 * m + 1], qb[2 * m], qb[2 * m + 1]);
        if (r0 < n) dots[r0][t] = d[0] * 256 + d[1];
        if (r1 < n) dots[r1][t] = d[2] * 256 + d[3];
    }
    first += nblk;
}

// weighted sums over the groups of one value section for this warp's MBW row blocks and all queries: the operand
// registers are made once and used by two instructions (queries 0,1 and 2,3)
template <int D, int W, int MBW>
__device__ __forceinline__ void v_section_mq(const uint8_t* sec, int ngroups, const uint32_t (*w0)[4], const uint32_t (*w1)[4],
                                             const uint32_t (*w2)[4], const uint32_t (*w3)[4], int (&acc)[2][MBW][4], int g, int t, int mb0) {
    constexpr int NRV = D / 8, GB = D * W / 2;
    // column g of the B operands: digits 0..2 of the first query of a pair, 3..5 of the second
    const uint32_t (*wa)[4] = g < 3 ? w0 : w1;
    const uint32_t (*wb)[4] = g < 3 ? w2 : w3;
    const int dg = g < 3 ? g : g - 3;
#pragma unroll 1
    for (int g0 = 0; g0 < ngroups; g0 += 8) {
        const int ga = g0 + t, gb = ga + 4;
        uint32_t xa[2 * MBW], xb[2 * MBW];
        fetch_regs<W, 2 * MBW>(sec + ga * GB, g * NRV + 2 * mb0, ga < ngroups, xa);
        fetch_regs<W, 2 * MBW>(sec + gb * GB, g * NRV + 2 * mb0, gb < ngroups, xb);
        const bool ca = g < 6 && ga < ngroups, cb = g < 6 && gb < ngroups;
        const uint32_t b0 = ca ? wa[ga][dg] : 0u, b1 = cb ? wa[gb][dg] : 0u;
        const uint32_t c0 = ca ? wb[ga][dg] : 0u, c1 = cb ? wb[gb][dg] : 0u;
#pragma unroll
        for (int mb = 0; mb < MBW; ++mb) {
            mma_u8s8(acc[0][mb], xa[2 * mb], xa[2 * mb + 1], xb[2 * mb], xb[2 * mb + 1], b0, b1);
            mma_u8s8(acc[1][mb], xa[2 * mb], xa[2 * mb + 1], xb[2 * mb], xb[2 * mb + 1], c0, c1);
        }
    }
}

// Barriers of a tile: [1] its bytes have landed (and the scratch of the tile before is free), [2] key dot products
// and key-outlier sums are complete, [3] the largest logits of the tile are known, [4] value weights are in place.
template <int D>
__global__ void __launch_bounds__(MQ_THREADS, MQ_CTAS_PER_SM) decode_multi_kernel(const MultiArgs a) {
    constexpr int NR = D / 16;                       // key operand registers per lane and item
    constexpr int MBW = D >= 64 ? D / 64 : 1;        // 16-channel row blocks of the value side per warp
    constexpr int VWARPS = (D / 16) / MBW;           // warps that have value row blocks (2 for head_dim 32)
    constexpr int BUFB = MultiSmem<D>::BUFB;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    MultiSmem<D>& sm = *reinterpret_cast<MultiSmem<D>*>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int fg = lane >> 2, ft = lane & 3;
    const int tok = tid & (QAQ_TILE - 1), qh = tid >> 6;   // every thread owns token `tok` of the tile for the queries 2*qh, 2*qh+1
    const int nq = a.nq;
    const float NEG = __int_as_float(0xff800000);

#pragma unroll 1
    for (int seg = 0; seg < 2; ++seg) {
    // this CTA's run of the flattened (b,h, tile) sequence; it touches at most two (b,h)
    const int cta = blockIdx.x;
    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const int flat_lo = cta * a.run, flat_hi = min(a.BH * ntiles, flat_lo + a.run);
    const int bh = flat_lo / ntiles + seg;
    const int tile_lo = max(flat_lo, bh * ntiles) - bh * ntiles, tile_hi = min(flat_hi, (bh + 1) * ntiles) - bh * ntiles;
    if (tile_lo >= tile_hi) continue;   // the same for every thread of the CTA

    // ---- queries: float copies, per-query scale and sum (warp j looks after query j), fixed-point byte digits per lane
    for (int j = 0; j < MQ; ++j)
        for (int d = tid; d < D; d += MQ_THREADS)
            sm.qf[j][d] = j < nq ? __half2float(a.q[((size_t)bh * a.n_q + a.q0 + j) * D + d]) : 0.f;
    for (int i = tid; i < 2 * MQ * D; i += MQ_THREADS) (&sm.vcorr[0][0][0])[i] = 0;
    for (int i = tid; i < 2 * MQ * QAQ_TILE; i += MQ_THREADS) (&sm.kcorr[0][0][0])[i] = 0;
    __syncthreads();
    {
        float qmax = 0.f, qs = 0.f;
        for (int d = lane; d < D; d += 32) { const float f = sm.qf[warp][d]; qmax = fmaxf(qmax, fabsf(f)); qs += f; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            qmax = fmaxf(qmax, __shfl_xor_sync(0xFFFFFFFFu, qmax, o));
            qs += __shfl_xor_sync(0xFFFFFFFFu, qs, o);
        }
        if (lane == 0) { sm.qscale[warp] = qmax / 32639.0f; sm.qsum[warp] = qs; }   // |q| <= 32639 units: both digits stay signed bytes
    }
    __syncthreads();
    uint32_t qb[NR];             // column fg of the B operand: digit (fg & 1) of query fg >> 1
    {
        const int jq = fg >> 1;
        const float qsc = sm.qscale[jq], qinv = qsc > 0.f ? 1.0f / qsc : 0.f;
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            uint32_t v = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int qi = __float2int_rn(sm.qf[jq][4 * (ft * NR + r) + i] * qinv);
                qi = max(-32639, min(32639, qi));
                const int dg = (fg & 1) == 0 ? ((qi + 128) >> 8) : qi;     // 256 * hi + lo with lo in [-128, 127]
                v |= (uint32_t)(dg & 0xFF) << (8 * i);
            }
            qb[r] = v;
        }
    }

    const int mb0 = warp * MBW;  // this warp's value row blocks
    // X[pair][mb][s][0/1]: this lane's share of the digit columns of the first / second query of the pair, channels
    // (D/8)*fg + 2*(mb0+mb) + s (summed over ft at the end)
    float X[2][MBW][2][2];
#pragma unroll
    for (int pr = 0; pr < 2; ++pr)
#pragma unroll
        for (int mb = 0; mb < MBW; ++mb) { X[pr][mb][0][0] = X[pr][mb][0][1] = X[pr][mb][1][0] = X[pr][mb][1][1] = 0.f; }
    // what the two accumulator columns of this lane stand for: columns 0..2 are the digits 2^16, 2^8, 1 of the first
    // query of a pair, columns 3..5 those of the second
    const float sa0 = ft == 0 ? 65536.0f : (ft == 1 ? 1.0f : 0.f), sa1 = ft == 0 ? 256.0f : 0.f;
    const float sb0 = ft == 2 ? 256.0f : 0.f, sb1 = ft == 1 ? 65536.0f : (ft == 2 ? 1.0f : 0.f);
    float m_run[MQ], vout[MQ];
    float l_part[2] = {0.f, 0.f}, lx_part[2] = {0.f, 0.f}, c_part[2] = {0.f, 0.f};   // sums over this thread's token, its two queries
#pragma unroll
    for (int j = 0; j < MQ; ++j) { m_run[j] = NEG; vout[j] = 0.f; }

    const size_t trow = (size_t)bh * a.ntiles_max;
    const size_t mrow = (size_t)bh * a.tmax_pad;
    const uint8_t* poolK = a.k.codes + (size_t)bh * a.pool_bytes;
    const uint8_t* poolV = a.v.codes + (size_t)bh * a.pool_bytes;
    const uint32_t* ogK = a.k.outl + (size_t)bh * a.ocap;
    const uint32_t* ogV = a.v.outl + (size_t)bh * a.ocap;

    // table words of a tile (the same for every thread); entries that point outside the pool or the list are not followed
    struct Tab { uint32_t off[2], nb[2], oo[2], oc[2]; };
    auto fetch_tab = [&](int tile) {
        Tab tb;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            tb.off[x] = tb.nb[x] = tb.oo[x] = tb.oc[x] = 0;
            if (tile < tile_hi) {
                const TensorStore& ts = x ? a.v : a.k;
                const size_t ti = trow + tile;
                tb.off[x] = __ldg(ts.tile_off + ti); tb.nb[x] = __ldg(ts.tile_nbytes + ti);
                tb.oo[x] = __ldg(ts.tile_ooff + ti); tb.oc[x] = __ldg(ts.tile_ocnt + ti);
                if ((tb.off[x] & 15u) || tb.nb[x] < (uint32_t)qaqc::QAQ_TILE_HDR || tb.nb[x] > (uint32_t)BUFB ||
                    (size_t)tb.off[x] + ((tb.nb[x] + 15u) & ~15u) > a.pool_bytes) tb.nb[x] = 0;
                if ((size_t)tb.oo[x] + tb.oc[x] > a.ocap) tb.oc[x] = 0;
            }
        }
        return tb;
    };
    auto stage = [&](const Tab& tb, int st) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const uint32_t nb = (tb.nb[x] + 15u) & ~15u;
            const uint8_t* src = (x ? poolV : poolK) + tb.off[x];
            uint8_t* dst = sm.buf[st][x];
#pragma unroll 1
            for (uint32_t o = tid * 16; o < nb; o += MQ_THREADS * 16) cp_async<16>(dst + o, src + o);
        }
        cp_async_commit();
    };
    // per-token metadata and the first outlier entries of a tile, fetched one tile ahead
    struct Pre { uint32_t mmK, mmV, eK, eV; };
    auto fetch_pre = [&](int tile, const Tab& tb) {
        Pre p;
        p.mmK = p.mmV = 0; p.eK = p.eV = 0;
        if (tile < tile_hi) {
            const size_t t0 = mrow + (size_t)tile * QAQ_TILE + tok;
            p.mmK = __ldg(a.k.mnmx + t0); p.mmV = __ldg(a.v.mnmx + t0);
            if ((uint32_t)tid < tb.oc[0]) p.eK = __ldg(ogK + tb.oo[0] + tid);
            if ((uint32_t)tid < tb.oc[1]) p.eV = __ldg(ogV + tb.oo[1] + tid);
        }
        return p;
    };

    Tab cur = fetch_tab(tile_lo);
    Tab nxt = fetch_tab(tile_lo + 1);
    Pre pcur = fetch_pre(tile_lo, cur);
    stage(cur, 0);

    for (int tile = tile_lo; tile < tile_hi; ++tile) {
        const int st = (tile - tile_lo) & 1;
        cp_async_wait<0>();
        __syncthreads();                                   // [1]
        if (tile + 1 < tile_hi) stage(nxt, st ^ 1); else cp_async_commit();
        const Pre pnxt = fetch_pre(tile + 1, nxt);
        const Tab nxt2 = fetch_tab(tile + 2);
        // value-outlier sums of the tile before (at the scale of the running sums as they are now)
        if (tid < D) {
#pragma unroll
            for (int j = 0; j < MQ; ++j) {
                const int h = sm.vcorr[0][j][tid], l = sm.vcorr[1][j][tid];
                if (h | l) { vout[j] += outlier_sum(h, l); sm.vcorr[0][j][tid] = 0; sm.vcorr[1][j][tid] = 0; }
            }
        }

        // ---- header: which slots have a piece of each width; section sizes and offsets
        const uint8_t* tK = sm.buf[st][0];
        const uint8_t* tV = sm.buf[st][1];
        unsigned long long mk[4], mv[4];
        int n[2][4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            mk[c] = cur.nb[0] ? reinterpret_cast<const unsigned long long*>(tK)[c] : 0ull;
            mv[c] = cur.nb[1] ? reinterpret_cast<const unsigned long long*>(tV)[c] : 0ull;
            n[0][c] = __popcll(mk[c]); n[1][c] = __popcll(mv[c]);
        }
        uint32_t kb[5], vb[5];
        qaqc::section_bases<D, false>(n[0], kb);
        qaqc::section_bases<D, true>(n[1], vb);
        // a tile that does not hold the sections its masks ask for is not read: its tokens then count with their
        // constant parts only
        const bool okK = kb[4] <= cur.nb[0], okV = vb[4] <= cur.nb[1];
        if (!okK) { n[0][0] = n[0][1] = n[0][2] = n[0][3] = 0; }
        if (!okV) { n[1][0] = n[1][1] = n[1][2] = n[1][3] = 0; }

        // ---- token threads: widths, ranks in the sections, steps and midpoints of their token
        const int tg = tile * QAQ_TILE + tok;               // token index
        const bool val = tg < a.T;
        int BK = 0, BV = 0;
        uint32_t rkK = 0, rkV = 0;                           // rank in section c in byte c
        float stepK = 0.f, stepV = 0.f, midK = 0.f, midV = 0.f;
        int topV = 0;
        {
            const unsigned long long below = (1ull << tok) - 1ull;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if ((mk[c] >> tok) & 1ull) BK |= 8 >> c;
                if ((mv[c] >> tok) & 1ull) BV |= 8 >> c;
                rkK |= (uint32_t)__popcll(mk[c] & below) << (8 * c);
                rkV |= (uint32_t)__popcll(mv[c] & below) << (8 * c);
            }
            if (!val) { BK = 0; BV = 0; }
            const float kmn = __half2float(__ushort_as_half((unsigned short)(pcur.mmK & 0xFFFF)));
            const float kmx = __half2float(__ushort_as_half((unsigned short)(pcur.mmK >> 16)));
            const float vmn = __half2float(__ushort_as_half((unsigned short)(pcur.mmV & 0xFFFF)));
            const float vmx = __half2float(__ushort_as_half((unsigned short)(pcur.mmV >> 16)));
            if (val) {
                stepK = qaqc::step_of(kmn, kmx, BK); stepV = qaqc::step_of(vmn, vmx, BV);
                midK = fmaf(0.5f, stepK, kmn); midV = fmaf(0.5f, stepV, vmn);
            }
            if (qh == 0) sm.midV[tok] = midV;
            topV = BV ? BV - (1 << (31 - __clz(BV))) : 0;   // shift of the widest value piece
            // the largest value weight of the tile is at most the largest step * 2^shift (p <= 1)
            float wb = stepV * __int_as_float((127 + topV) << 23);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wb = fmaxf(wb, __shfl_xor_sync(0xFFFFFFFFu, wb, o));
            if (lane == 0 && qh == 0) sm.wloc[warp] = wb;
        }

        // ---- K: integer dot products of all queries, the row blocks of the four sections dealt out to the warps
        {
            int first = 0;
            k_section_mq<D, 8>(tK + kb[0], n[0][0], sm.dotw[0], qb, fg, ft, warp, first);
            k_section_mq<D, 4>(tK + kb[1], n[0][1], sm.dotw[1], qb, fg, ft, warp, first);
            k_section_mq<D, 2>(tK + kb[2], n[0][2], sm.dotw[2], qb, fg, ft, warp, first);
            k_section_mq<D, 1>(tK + kb[3], n[0][3], sm.dotw[3], qb, fg, ft, warp, first);
        }
        // key outliers: q_ch * (x - mid) per token and query; the token's midpoint comes from its metadata
        {
            uint32_t e = tid, v = pcur.eK;
#pragma unroll 1
            for (; e < cur.oc[0]; e += MQ_THREADS) {
                if (e >= MQ_THREADS) v = __ldg(ogK + cur.oo[0] + e);
                const int tok = (v >> 24) & (QAQ_TILE - 1), ch = (v >> 16) & (D - 1);
                int Bt = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) Bt |= (int)((mk[c] >> tok) & 1ull) << (3 - c);
                const uint32_t mm = __ldg(a.k.mnmx + mrow + (size_t)tile * QAQ_TILE + tok);
                const float mn = __half2float(__ushort_as_half((unsigned short)(mm & 0xFFFF)));
                const float mx = __half2float(__ushort_as_half((unsigned short)(mm >> 16)));
                const float dx = __half2float(__ushort_as_half((unsigned short)(v & 0xFFFF))) - fmaf(0.5f, qaqc::step_of(mn, mx, Bt), mn);
                for (int j = 0; j < nq; ++j) outlier_add(&sm.kcorr[0][j][tok], &sm.kcorr[1][j][tok], sm.qf[j][ch] * dx);
            }
        }
        __syncthreads();                                   // [2]

        // ---- logits of this thread's token for its two queries, largest logits of the tile
        float lg[2] = {NEG, NEG};
        {
            int dot[2] = {0, 0};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int w = 8 >> c;
                if ((BK & w) && okK) {
                    const int2 dv = *reinterpret_cast<const int2*>(&sm.dotw[c][(rkK >> (8 * c)) & 0xFF][2 * qh]);
                    const int sh = BK & (w - 1);
                    dot[0] += dv.x << sh; dot[1] += dv.y << sh;
                }
            }
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                const int j = 2 * qh + jj;
                const int kh = sm.kcorr[0][j][tok], kl = sm.kcorr[1][j][tok];
                if (kh | kl) { sm.kcorr[0][j][tok] = 0; sm.kcorr[1][j][tok] = 0; }
                if (val && j < nq) {
                    const float qk = fmaf(sm.qscale[j] * stepK, (float)dot[jj], fmaf(midK, sm.qsum[j], outlier_sum(kh, kl)));
                    lg[jj] = a.scale * qk;
                }
                float m = lg[jj];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
                if (lane == 0) sm.mloc[warp & 1][j] = m;
            }
        }
        __syncthreads();                                   // [3]
        {
            // ---- value weights p * step * 2^shift as 22-bit fixed point with one scale for the tile (the bound on the
            //      largest weight does not depend on the query).  The weight of the token's lowest piece is rounded once;
            //      the other pieces use exact multiples of it, and p is replaced by what the rounded weight stands for,
            //      so that the pieces, the constant part and the softmax denominator all see the same probability.
            const float wmax = fmaxf(sm.wloc[0], sm.wloc[1]);
            const int wex = (__float_as_int(wmax) >> 23) & 0xFF;
            const bool wok = wex > 24 && wex < 255 && okV;     // zero, tiny or non-finite steps: the pieces add nothing
            const float wunit = wok ? __int_as_float((wex - 21) << 23) : 0.f;
            const float winv = wok ? __int_as_float((254 - (wex - 21)) << 23) : 0.f;
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                const int j = 2 * qh + jj;
                const float mr = qh ? m_run[2 + jj] : m_run[jj];
                const float m_new = fmaxf(mr, fmaxf(sm.mloc[0][j], sm.mloc[1][j]));
                if (tok == 0) sm.mnew[j] = m_new;
                const float alpha = m_new == NEG ? 1.0f : __expf(mr - m_new);
                const float pe = m_new == NEG ? 0.f : __expf(lg[jj] - m_new);               // 0 for slots beyond T
                uint32_t iw = (uint32_t)__float2int_rn(fminf(pe * stepV * winv, 8388608.0f));
                iw = min(iw, 0x7F0000u >> topV);                   // the three balanced byte digits of a shifted weight stay signed bytes
                float p = pe;
                if (stepV > 0.f && wok) p = __fdividef((float)iw * wunit, stepV);
                uint8_t* wbytes = reinterpret_cast<uint8_t*>(sm.wts[j]);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int w = 8 >> c;
                    if (BV & w) {
                        const uint32_t r = (rkV >> (8 * c)) & 0xFF, wt = iw << (BV & (w - 1));
                        // wt = 65536 * d2 + 256 * d1 + d0 with d1, d0 in [-128, 127]
                        const uint32_t r1 = (wt + 128u) >> 8, r2 = (r1 + 128u) >> 8;
                        uint8_t* gp = wbytes + c * (QAQ_TILE / 4) * 16 + (r >> 2) * 16 + (r & 3);
                        gp[0] = (uint8_t)r2;
                        gp[4] = (uint8_t)r1;
                        gp[8] = (uint8_t)wt;
                    }
                }
                sm.p[j][tok] = p;
                l_part[jj] = fmaf(l_part[jj], alpha, p);
                lx_part[jj] = fmaf(lx_part[jj], alpha, pe);
                c_part[jj] = fmaf(c_part[jj], alpha, p * midV);
            }
            if (tid == 0) sm.wunit = wunit;
        }
        __syncthreads();                                   // [4]
        float alpha[MQ];
#pragma unroll
        for (int j = 0; j < MQ; ++j) {
            const float m_new = sm.mnew[j];
            alpha[j] = m_new == NEG ? 1.0f : __expf(m_run[j] - m_new);         // 0 on the first tile (m_run = -inf)
            m_run[j] = m_new;
            vout[j] *= alpha[j];
        }
        const float wunit = sm.wunit;
#pragma unroll
        for (int pr = 0; pr < 2; ++pr)
#pragma unroll
            for (int mb = 0; mb < MBW; ++mb)
#pragma unroll
                for (int s2 = 0; s2 < 2; ++s2) { X[pr][mb][s2][0] *= alpha[2 * pr]; X[pr][mb][s2][1] *= alpha[2 * pr + 1]; }

        // ---- V: integer weighted sums per section for this warp's row blocks, added to the binary32 accumulators
        if (wunit != 0.f && warp < VWARPS) {
            int acc[2][MBW][4];
#pragma unroll
            for (int pr = 0; pr < 2; ++pr)
#pragma unroll
                for (int mb = 0; mb < MBW; ++mb) { acc[pr][mb][0] = 0; acc[pr][mb][1] = 0; acc[pr][mb][2] = 0; acc[pr][mb][3] = 0; }
            v_section_mq<D, 8, MBW>(tV + vb[0], (n[1][0] + 3) >> 2, sm.wts[0][0], sm.wts[1][0], sm.wts[2][0], sm.wts[3][0], acc, fg, ft, mb0);
            v_section_mq<D, 4, MBW>(tV + vb[1], (n[1][1] + 3) >> 2, sm.wts[0][1], sm.wts[1][1], sm.wts[2][1], sm.wts[3][1], acc, fg, ft, mb0);
            v_section_mq<D, 2, MBW>(tV + vb[2], (n[1][2] + 3) >> 2, sm.wts[0][2], sm.wts[1][2], sm.wts[2][2], sm.wts[3][2], acc, fg, ft, mb0);
            v_section_mq<D, 1, MBW>(tV + vb[3], (n[1][3] + 3) >> 2, sm.wts[0][3], sm.wts[1][3], sm.wts[2][3], sm.wts[3][3], acc, fg, ft, mb0);
#pragma unroll
            for (int pr = 0; pr < 2; ++pr)
#pragma unroll
                for (int mb = 0; mb < MBW; ++mb)
#pragma unroll
                    for (int s2 = 0; s2 < 2; ++s2) {
                        const float c0 = (float)acc[pr][mb][2 * s2], c1 = (float)acc[pr][mb][2 * s2 + 1];
                        X[pr][mb][s2][0] = fmaf(fmaf(c0, sa0, c1 * sa1), wunit, X[pr][mb][s2][0]);
                        X[pr][mb][s2][1] = fmaf(fmaf(c0, sb0, c1 * sb1), wunit, X[pr][mb][s2][1]);
                    }
        }
        // value outliers: p_t * (v - mid) per channel and query
        {
            uint32_t e = tid, v = pcur.eV;
#pragma unroll 1
            for (; e < cur.oc[1]; e += MQ_THREADS) {
                if (e >= MQ_THREADS) v = __ldg(ogV + cur.oo[1] + e);
                const int tok = (v >> 24) & (QAQ_TILE - 1), ch = (v >> 16) & (D - 1);
                const float dx = __half2float(__ushort_as_half((unsigned short)(v & 0xFFFF))) - sm.midV[tok];
                for (int j = 0; j < nq; ++j) outlier_add(&sm.vcorr[0][j][ch], &sm.vcorr[1][j][ch], sm.p[j][tok] * dx);
            }
        }
        cur = nxt; nxt = nxt2; pcur = pnxt;
    }
    cp_async_wait<0>();
    __syncthreads();

    // ---- the segment's partials: channels from the digit columns of the four lanes ft, sums of the token threads
    if (tid < D) {
#pragma unroll
        for (int j = 0; j < MQ; ++j) {
            const int h = sm.vcorr[0][j][tid], l = sm.vcorr[1][j][tid];
            vout[j] += outlier_sum(h, l);
            sm.vcorr[0][j][tid] = 0; sm.vcorr[1][j][tid] = 0;
        }
    }
#pragma unroll
    for (int pr = 0; pr < 2; ++pr)
#pragma unroll
        for (int mb = 0; mb < MBW; ++mb)
#pragma unroll
            for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    float v = X[pr][mb][s2][w];
                    v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
                    v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
                    if (ft == 0 && warp < VWARPS) sm.xs[2 * pr + w][(D / 8) * fg + 2 * (mb0 + mb) + s2] = v;
                }
#pragma unroll
    for (int jj = 0; jj < 2; ++jj) {
        float l = l_part[jj], lx = lx_part[jj], cs = c_part[jj];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            l += __shfl_xor_sync(0xFFFFFFFFu, l, o);
            lx += __shfl_xor_sync(0xFFFFFFFFu, lx, o);
            cs += __shfl_xor_sync(0xFFFFFFFFu, cs, o);
        }
        // warps 2*qh and 2*qh+1 hold the two halves of the tokens for queries 2*qh, 2*qh+1
        if (lane == 0) { sm.red[warp & 1][2 * qh + jj] = l; sm.red2[warp & 1][2 * qh + jj] = lx; sm.red3[warp & 1][2 * qh + jj] = cs; }
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < MQ; ++j) {
        if (j >= nq) continue;
        float* dst = a.part + ((size_t)(2 * cta + seg) * MQ + j) * (D + 3);
        if (tid < D) dst[tid] = sm.xs[j][tid] + vout[j] + (sm.red3[0][j] + sm.red3[1][j]);
        if (tid == 0) { dst[D] = m_run[j]; dst[D + 1] = sm.red[0][j] + sm.red[1][j]; dst[D + 2] = sm.red2[0][j] + sm.red2[1][j]; }
    }
    __syncthreads();   // the shared arrays are reused by the second segment
    }
}

// log-sum-exp merge of the partials of one (b,h) and query -> X
template <int D>
__global__ void merge_multi_kernel(const MultiArgs a) {
    const int bh = blockIdx.x, j = blockIdx.y, d = threadIdx.x;
    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const int c_lo = (bh * ntiles) / a.run, c_hi = ((bh + 1) * ntiles - 1) / a.run;
    // only the first of the CTAs whose runs meet this (b,h) can have begun in the (b,h) before (then its second segment)
    auto slot = [&](int c) { return a.part + ((size_t)(2 * c + (c * a.run < bh * ntiles ? 1 : 0)) * MQ + j) * (D + 3); };
    const float NEG = __int_as_float(0xff800000);
    float M = NEG;
    for (int c = c_lo; c <= c_hi; ++c) M = fmaxf(M, slot(c)[D]);
    float L = 0.f, x = 0.f;
    for (int c = c_lo; c <= c_hi; ++c) {
        const float* p = slot(c);
        const float m = p[D];
        if (m == NEG) continue;
        const float w = __expf(m - M);
        L = fmaf(w, p[D + 1], L);
        x = fmaf(w, p[d], x);
    }
    a.out[((size_t)bh * a.n_q + a.q0 + j) * D + d] = L > 0.f ? x / L : 0.f;
}

// runs of equal length over the flattened (b,h, tile) sequence, one CTA each, never more than one (b,h) boundary
// inside a run
constexpr int MQ_SLOTS = 148 * MQ_CTAS_PER_SM;
struct MultiPlan { int run, ncta; };
MultiPlan plan_multi(int BH, int ntiles) {
    const long long total = (long long)BH * ntiles;
    long long run = (total + MQ_SLOTS - 1) / MQ_SLOTS;
    if (run < 1) run = 1;
    if (run > ntiles) run = ntiles;
    MultiPlan p;
    p.run = (int)run;
    p.ncta = (int)((total + run - 1) / run);
    return p;
}

template <int D>
qaq_status run_multi(const MultiArgs& a, cudaStream_t s) {
    const size_t smem = sizeof(MultiSmem<D>);
    if (smem > 48 * 1024)
        QAQ_CUDA_TRY(cudaFuncSetAttribute(decode_multi_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_multi_kernel<D><<<a.ncta, MQ_THREADS, smem, s>>>(a);
    merge_multi_kernel<D><<<dim3(a.BH, a.nq), D, 0, s>>>(a);
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

}  // namespace

extern "C" qaq_status qaq_decode_multi_workspace_bytes(const qaq_cache* c, size_t* host_out) {
    if (!c || !host_out) return QAQ_ERR_INVALID_ARG;
    // plan_multi never uses more CTAs than max(MQ_SLOTS, BH), whatever the token count; the passes of a call reuse the
    // space, and the partials of the single-query kernel (at most 2 * max(592, BH) * (head_dim + 3) + 2 * BH floats) fit it too
    const int ncta_max = c->BH > MQ_SLOTS ? c->BH : MQ_SLOTS;
    *host_out = (size_t)2 * ncta_max * MQ * (c->cfg.head_dim + 3) * sizeof(float);
    return QAQ_OK;
}

extern "C" qaq_status qaq_decode_attention_multi(const qaq_cache* c, const void* q, int n_q, float softmax_scale, float* out,
                                                 void* ws, size_t ws_bytes, void* stream) {
    if (!c || !q || !out || !ws || n_q < 1 || n_q > 8) return QAQ_ERR_INVALID_ARG;
    if (c->tokens < 1) return QAQ_ERR_INVALID_ARG;
    size_t need = 0;
    qaq_decode_multi_workspace_bytes(c, &need);
    if (ws_bytes < need || ((uintptr_t)ws & 15)) return QAQ_ERR_WORKSPACE;
    const int D = c->cfg.head_dim, BH = c->BH;
    MultiArgs a;
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.ocap = c->ocap;
    a.tmax_pad = c->tmax_pad; a.ntiles_max = c->ntiles; a.T = (int)c->tokens;
    a.q = (const __half*)q; a.n_q = n_q; a.scale = softmax_scale;
    const int ntiles = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    const MultiPlan plan = plan_multi(BH, ntiles);
    a.BH = BH; a.run = plan.run; a.ncta = plan.ncta;
    a.part = (float*)ws;
    a.out = out;
    cudaStream_t s = (cudaStream_t)stream;
    for (int q0 = 0; q0 < n_q; q0 += MQ) {          // four queries per pass over the cache
        a.q0 = q0; a.nq = n_q - q0 < MQ ? n_q - q0 : MQ;
        qaq_status st;
        if (a.nq <= 2) {
            // one or two queries do not pay for a pass of this kernel (it is laid out for four): the single-query
            // kernel takes them one by one (its partials fit the same workspace)
            for (int j = 0; j < a.nq; ++j) {
                st = qaq_decode_strided(c, (const __half*)q + (size_t)(q0 + j) * D, (long)n_q * D, softmax_scale,
                                        out + (size_t)(q0 + j) * D, (long)n_q * D, ws, s);
                if (st != QAQ_OK) return st;
            }
            continue;
        }
        switch (D) {
            case 32: st = run_multi<32>(a, s); break;
            case 64: st = run_multi<64>(a, s); break;
            case 128: st = run_multi<128>(a, s); break;
            default: return QAQ_ERR_UNSUPPORTED_SHAPE;
        }
        if (st != QAQ_OK) return st;
    }
    return QAQ_OK;
}
