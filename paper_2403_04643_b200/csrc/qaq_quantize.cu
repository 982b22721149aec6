// S1-S3: bit-width selection, outlier split, uniform quantization and bit-packing.
//
// One CTA handles one tile (QAQ_TILE consecutive tokens) of one (b,h); head_dim/32 lanes
// own one token, each lane 32 consecutive channels of K and of V (64 bytes each), held in
// registers from the min/max pass to the packing pass, so K and V are read from HBM once.
//   phase 0  attention-window maximum of the score rows (Section 4.2)
//   phase 1  outlier masks and min/max of the non-outliers in binary16 pair arithmetic
//            (exact: the inputs are binary16), width from the exponents (Section 4.1)
//   phase 2  warp 0: which slots have a piece of each width (ballots), section sizes of the tile,
//            exclusive scan of the outlier counts, space taken from the (b,h) pools by atomicAdd
//   phase 3  codes (binary32: one sub, one mul, round down), pieces written into a shared-memory
//            image of the tile in the section layout of qaq_codec.cuh (values as token-major planes
//            that the copy-out transposes into groups of four tokens), vector stores; outlier
//            entries placed by popc ranks
// A tile that is continued (an append behind a partly filled tile) is built anew: the codes of
// its old tokens are read back from the pool, the image of old and new tokens replaces it.
#include "qaq_codec.cuh"
#include "qaq_internal.cuh"

namespace {

struct QuantArgs {
    const __half* K;
    const __half* V;
    long sb, sh, st;       // element strides of K/V (batch, head, token)
    int H;                 // heads
    int n_new;             // tokens per (b,h) in K/V (and in bits/ring/nvalid rows)
    int t_old;             // tokens already cached (0 for selection only)
    int tok_lo, tok_hi;    // new-token index range handled by this launch
    int first_tile;        // absolute index of the first tile touched by this launch
    const uint8_t* bitsK;  // given widths [BH][n_new] or null
    const uint8_t* bitsV;
    const float* ring;     // [BH][W][n_new]
    const uint8_t* nvalid; // [BH][n_new]
    int W;
    const float* thr;      // [BH][4]
    float cK, cV;
    int bmin, bmax;
    TensorStore k, v;
    size_t pool_bytes;
    uint32_t ocap;
    int tmax_pad, ntiles;
    int* status;
    int* d_count;          // null, or the token count kept in device memory: read instead of t_old / first_tile and
    unsigned* d_ticket;    //   advanced by the last CTA of the launch to finish (small appends only)
    int max_tokens;
    uint8_t* out_bitsK;    // selection only
    uint8_t* out_bitsV;
};

using qaqc::ladder;

__device__ __forceinline__ uint32_t lop3_sel(uint32_t a, uint32_t m, uint32_t c) {  // (a & m) | (c & ~m)
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xE2;" : "=r"(d) : "r"(a), "r"(m), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c) {  // (a & b) | c
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ __half2 as_h2(uint32_t x) { return *reinterpret_cast<__half2*>(&x); }
__device__ __forceinline__ uint32_t as_u32(__half2 x) { return *reinterpret_cast<uint32_t*>(&x); }
// One lane's 32 channels of one token and tensor: outlier masks, masked min / max.
//   v[k] holds channels 2k, 2k+1 (binary16 pairs).  On return every outlier entry of v has
//   been replaced by -inf: in the code computation that yields code byte 0 without a mask
//   (the outlier's own value is re-read from memory when its list entry is written).
//   inl : bit k = channel 2k is an inlier, bit 16+k = channel 2k+1 is an inlier
__device__ __forceinline__ void analyze32(uint32_t (&v)[16], __half2 lo2, __half2 hi2, uint32_t& inl, __half2& mn2,
                                          __half2& mx2) {
    uint32_t mnacc = 0x7C007C00u, mxacc = 0xFC00FC00u, bits = 0;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const __half2 x = as_h2(v[k]);
        const uint32_t m = __hge2_mask(x, lo2) & __hle2_mask(x, hi2);
        mnacc = as_u32(__hmin2(as_h2(mnacc), as_h2(lop3_sel(v[k], m, 0x7C007C00u))));
        v[k] = lop3_sel(v[k], m, 0xFC00FC00u);
        mxacc = as_u32(__hmax2(as_h2(mxacc), as_h2(v[k])));
        bits = lop3_and_or(m, 0x00010001u << k, bits);
    }
    inl = bits;
    mn2 = as_h2(mnacc);
    mx2 = as_h2(mxacc);
}

// space from a (b,h) pool: `whole` tiles take a rounded-up amount in one atomic; a tile that is
// being continued takes the exact amount and is padded to the unit when it closes.  `taken` is
// what the pool end moved by (to be given back if the space turns out not to fit).
__device__ __forceinline__ uint32_t pool_take(uint32_t* pool, uint32_t amount, uint32_t unit_mask, bool whole, bool closes,
                                              uint32_t& taken) {
    uint32_t base;
    if (whole) {
        taken = (amount + unit_mask) & ~unit_mask;
        base = atomicAdd(pool, taken);
    } else {
        base = atomicAdd(pool, amount);
        taken = amount;
        if (closes) {
            const uint32_t pad = (0u - (base + amount)) & unit_mask;
            if (pad) atomicAdd(pool, pad);
            taken += pad;
        }
    }
    return base;
}

// One CTA = one tile of 64 tokens of one (b,h); P = D/32 lanes own a token, each lane 32
// consecutive channels (64 bytes) of K and of V, kept in registers across all phases.
// Order of work (barriers in brackets): loads, attention window, outlier masks and ranges,
// widths [A] warp 0 finds the section sizes of the tile, scans the outlier counts and takes pool
// space with four atomics in flight at once while every warp computes its codes [B] pieces into a
// shared-memory image of the tile [C] the image goes out with 16-byte stores; outlier entries and
// per-token metadata follow.  Slots below the first new token of a continued tile hold the tile's
// old tokens: their widths come from the metadata, their codes from the tile as it is stored.
// XSEL: -1 = keys and values in one CTA; 0 / 1 = this launch handles only the keys / only the values of a tile
// (half the registers and shared memory per CTA, so more tiles are in flight per SM).
template <int D, bool SELECT_ONLY, int XSEL>
#ifndef QSPLIT_CTAS
#define QSPLIT_CTAS 6
#endif
#ifndef QSPLIT_MIN_CTAS
#define QSPLIT_MIN_CTAS 4096
#endif
__global__ void __launch_bounds__(2 * D, XSEL < 0 ? (D == 128 ? 3 : 4) : (D == 128 ? QSPLIT_CTAS : 6)) quant_kernel(const QuantArgs a) {
    constexpr int X0 = XSEL < 0 ? 0 : XSEL, X1 = XSEL < 0 ? 2 : XSEL + 1;
    constexpr int P = D / 32;            // lanes per token
    constexpr int NT = 2 * D;            // threads
    constexpr int IMG = qaqc::v_tile_bytes_max(D);
    constexpr bool COUNTED = XSEL < 0 && !SELECT_ONLY;   // the launches that may take the token count from device memory
    const int bh = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid / P, p = tid % P;
    int t_old = a.t_old, first_tile = a.first_tile;
    if (COUNTED && a.d_count) {
        t_old = *a.d_count;                // the same value in every thread of the launch: it is written only by tick()
        first_tile = t_old / QAQ_TILE;
        if (t_old + a.tok_hi > a.max_tokens) {             // no room: nothing is stored, the count stays
            if (tid == 0) atomicMax(a.status, (int)QAQ_ERR_CAPACITY);
            return;
        }
    }
    const int tile = first_tile + blockIdx.x;
    // counted launches: the last CTA to get here moves the count on.  Every thread of every CTA has used the count it
    // read by then (the barrier), and nothing else of the launch reads it afterwards.
    auto tick = [&]() {
        if (COUNTED && a.d_count) {
            __syncthreads();
            if (tid == 0) {
                __threadfence();
                const unsigned n = gridDim.x * gridDim.y;
                if (atomicInc(a.d_ticket, n - 1) == n - 1) *a.d_count = t_old + a.tok_hi;
            }
        }
    };

    const int abs_lo = max(tile * QAQ_TILE, t_old + a.tok_lo);
    const int abs_hi = min((tile + 1) * QAQ_TILE, t_old + a.tok_hi);
    const int s_lo = abs_lo - tile * QAQ_TILE, s_hi = abs_hi - tile * QAQ_TILE;
    const bool valid = slot >= s_lo && slot < s_hi;       // a new token
    const bool old = !SELECT_ONLY && slot < s_lo;         // a token the tile already holds
    const int tn = tile * QAQ_TILE + slot - t_old;        // index among the new tokens

    __shared__ uint8_t s_bits[2][QAQ_TILE];   // widths of the tile's slots (0: empty)
    __shared__ uint32_t s_cnt[2][QAQ_TILE];   // outlier counts of the new tokens, then exclusive offsets
    __shared__ qaqc::TileMasks s_tm[2];
    __shared__ uint32_t s_rank[2][QAQ_TILE];   // ranks of the slots in the four sections, one per byte
    __shared__ uint32_t s_sec[2][5];           // byte offsets of the sections
    __shared__ uint32_t s_tot[2], s_base[2], s_obase[2], s_olimit[2], s_otot[2];
    constexpr uint32_t OUT_STAGE = 4 * D;      // outliers of a tile whose (slot, channel) are listed on chip in entry order; more go out one by one
    __shared__ unsigned short s_work[SELECT_ONLY ? 1 : X1 - X0][SELECT_ONLY ? 1 : OUT_STAGE];
    __shared__ int s_skip;
    __shared__ __align__(16) uint8_t s_img[SELECT_ONLY ? 1 : X1 - X0][SELECT_ONLY ? 16 : IMG];  // the tile as it will be stored

    const float* thr = a.thr + (size_t)bh * 4;
    const bool given = a.bitsK != nullptr;
    const size_t ti = (size_t)bh * a.ntiles + tile;
    const size_t mt = (size_t)bh * a.tmax_pad + (size_t)tile * QAQ_TILE + slot;

    // ---- loads first (independent of everything else)
    const int b_idx = bh / a.H, h_idx = bh % a.H;
    uint32_t vk[16], vv[16];
    {
        const __half* Kr = a.K + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh + (size_t)(valid ? tn : 0) * a.st + 32 * p;
        const __half* Vr = a.V + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh + (size_t)(valid ? tn : 0) * a.st + 32 * p;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 x = make_uint4(0, 0, 0, 0), y = make_uint4(0, 0, 0, 0);
            if (valid) {
                if (XSEL != 1) x = *reinterpret_cast<const uint4*>(Kr + 8 * i);
                if (XSEL != 0) y = *reinterpret_cast<const uint4*>(Vr + 8 * i);
            }
            vk[4 * i] = x.x; vk[4 * i + 1] = x.y; vk[4 * i + 2] = x.z; vk[4 * i + 3] = x.w;
            vv[4 * i] = y.x; vv[4 * i + 1] = y.y; vv[4 * i + 2] = y.z; vv[4 * i + 3] = y.w;
        }
    }
    // the padding of the value groups has to read as zero
    if (!SELECT_ONLY && XSEL != 0) {
        uint4* z = reinterpret_cast<uint4*>(s_img[X1 - X0 - 1]);
        for (int o = tid; o < IMG / 16; o += NT) z[o] = make_uint4(0, 0, 0, 0);
    }

    // ---- attention window: the P lanes of a token take its rows p, p+P, ... and combine by shuffles
    float shat = __int_as_float(0xff800000);
    int nv_tok = 0;
    {
        if (XSEL != 0 && !given && valid) {
            nv_tok = a.nvalid[(size_t)bh * a.n_new + tn];
            nv_tok = nv_tok < a.W ? nv_tok : a.W;
            // every row of the window is read (the ring is allocated in full), rows the token has no score in are
            // left out of the maximum: the loads then depend on nothing and go out together
            const float* r = a.ring + (size_t)bh * a.W * a.n_new + tn;
            int i = p;
            for (; i + 7 * P < a.W; i += 8 * P) {
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = __ldg(r + (size_t)(i + u * P) * a.n_new);
#pragma unroll
                for (int u = 0; u < 8; ++u) if (i + u * P < nv_tok) shat = fmaxf(shat, v[u]);
            }
            for (; i < a.W; i += P) {
                const float v = __ldg(r + (size_t)i * a.n_new);
                if (i < nv_tok) shat = fmaxf(shat, v);
            }
        }
#pragma unroll
        for (int o = 1; o < P; o <<= 1) shat = fmaxf(shat, __shfl_xor_sync(0xFFFFFFFFu, shat, o));
    }

    // ---- outlier masks and range of the rest (register work, needs nothing from shared memory)
    uint32_t inl[2], cntx[2];
    float mnf[2], mxf[2];
#pragma unroll
    for (int x = X0; x < X1; ++x) {
        // thresholds as binary16 bounds that decide exactly like the binary32 ones on binary16 data
        const __half lo = __float2half_ru(thr[2 * x]), hi = __float2half_rd(thr[2 * x + 1]);
        __half2 mn2, mx2;
        analyze32(x ? vv : vk, __half2half2(lo), __half2half2(hi), inl[x], mn2, mx2);
        const __half lmin = __hmin(__low2half(mn2), __high2half(mn2));
        const __half lmax = __hmax(__low2half(mx2), __high2half(mx2));
        __half2 pk = __halves2half2(lmin, __hneg(lmax));
#pragma unroll
        for (int o = 1; o < P; o <<= 1) pk = __hmin2(pk, as_h2(__shfl_xor_sync(0xFFFFFFFFu, as_u32(pk), o)));
        float mn = __low2float(pk), mx = -__high2float(pk);
        if (mn > mx) { mn = 0.f; mx = 0.f; }   // no entry inside [lo, hi]
        uint32_t cnt = 32u - (uint32_t)__popc(inl[x]);
#pragma unroll
        for (int o = 1; o < P; o <<= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
        mnf[x] = mn; mxf[x] = mx; cntx[x] = cnt;
    }

    // ---- widths
    int Bx[2];
#pragma unroll
    for (int x = X0; x < X1; ++x) {
        int B;
        if (given) {
            B = valid ? (x ? a.bitsV : a.bitsK)[(size_t)bh * a.n_new + tn] : 0;
            B = B < 1 ? 1 : (B > 8 ? 8 : B);
        } else {
            const float r = __fsub_rn(mxf[x], mnf[x]);
            if (x == 0) {
                B = ladder(r, a.cK, a.bmin, a.bmax);
            } else {
                B = (nv_tok == 0) ? a.bmax : ladder(__fmul_rn(r, shat), a.cV, a.bmin, a.bmax);
            }
        }
        Bx[x] = valid ? B : 0;
        if (old) {
            const int bo = (x ? a.v : a.k).bits[mt];
            Bx[x] = bo > 8 ? 8 : bo;
        }
        if (p == 0) {                                   // every slot of the tile is written: empty ones count nothing
            s_bits[x][slot] = (uint8_t)Bx[x];
            s_cnt[x][slot] = valid ? cntx[x] : 0u;
            if (SELECT_ONLY && valid) (x ? a.out_bitsV : a.out_bitsK)[(size_t)bh * a.n_new + tn] = (uint8_t)B;
        }
    }
    if (SELECT_ONLY) return;
    __syncthreads();   // [A] widths and outlier counts visible

    // ---- warp 0: section masks of the tile, ranks and section offsets, space for the bytes; warp 1: scan of the
    //      outlier counts, space for the entries (the two halves do not depend on each other; the atomics - lane 2x of
    //      warp 0 and lane 2x + 1 of warp 1 for tensor x - stay in flight while every warp computes its codes)
    const bool starts = (s_lo == 0), closes = (s_hi == QAQ_TILE), whole = starts && closes;
    uint32_t my_base = 0, my_amount = 0, my_taken = 0;
    if (warp == 0) {
        uint32_t amount[2];
#pragma unroll
        for (int x = X0; x < X1; ++x) {
            const uint32_t b0 = s_bits[x][lane], b1 = s_bits[x][lane + 32];
            qaqc::TileMasks tm;
            uint32_t rk0 = 0, rk1 = 0;       // ranks of slots lane and lane + 32
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const unsigned lo = __ballot_sync(0xFFFFFFFFu, (b0 & (8u >> c)) != 0), hi = __ballot_sync(0xFFFFFFFFu, (b1 & (8u >> c)) != 0);
                tm.m[c] = (unsigned long long)lo | ((unsigned long long)hi << 32);
                const unsigned below = (1u << lane) - 1u;
                rk0 |= (uint32_t)__popc(lo & below) << (8 * c);
                rk1 |= (uint32_t)(__popc(lo) + __popc(hi & below)) << (8 * c);
            }
            s_rank[x][lane] = rk0; s_rank[x][lane + 32] = rk1;
            uint32_t base[5];
            if (x == 0) qaqc::section_bases<D, false>(tm, base); else qaqc::section_bases<D, true>(tm, base);
            if (lane == 0) {
#pragma unroll
                for (int c = 0; c < 5; ++c) s_sec[x][c] = base[c];
            }
            // a continued tile stays where it is and takes only what it grows by behind its end
            const uint32_t old_nb = starts ? 0u : (x ? a.v : a.k).tile_nbytes[ti];
            amount[x] = base[4] - old_nb;
            if (lane == 0) { s_tm[x] = tm; s_tot[x] = base[4]; }
        }
        if (!(lane & 1) && lane >= 2 * X0 && lane < 2 * X1) {
            const int x = lane >> 1;
            my_amount = x ? amount[1] : amount[0];
            my_base = pool_take(&(x ? a.v : a.k).pool_end[bh], my_amount, 15u, whole, closes, my_taken);
        }
    } else if (warp == 1) {
        uint32_t amount[2];
#pragma unroll
        for (int x = X0; x < X1; ++x) {
            const uint32_t c0 = s_cnt[x][lane], c1 = s_cnt[x][lane + 32];
            uint32_t ic0 = c0, ic1 = c1;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t u0 = __shfl_up_sync(0xFFFFFFFFu, ic0, d), u1 = __shfl_up_sync(0xFFFFFFFFu, ic1, d);
                if (lane >= d) { ic0 += u0; ic1 += u1; }
            }
            const uint32_t ctot0 = __shfl_sync(0xFFFFFFFFu, ic0, 31), ctot1 = __shfl_sync(0xFFFFFFFFu, ic1, 31);
            s_cnt[x][lane] = ic0 - c0; s_cnt[x][lane + 32] = ctot0 + ic1 - c1;
            amount[x] = ctot0 + ctot1;
            if (lane == 0) s_otot[x] = ctot0 + ctot1;
        }
        if ((lane & 1) && lane >= 2 * X0 && lane < 2 * X1) {
            const int x = lane >> 1;
            my_amount = x ? amount[1] : amount[0];
            my_base = pool_take(&(x ? a.v : a.k).opool_end[bh], my_amount, 3u, whole, closes, my_taken);
        }
    }

    // ---- codes of the new tokens (every warp; needs only registers): channels 4j..4j+3 in the byte lanes of creg[j]
    uint32_t cregs[2][8];
#pragma unroll
    for (int x = X0; x < X1; ++x) qaqc::codes32(x ? vv : vk, mnf[x], mxf[x], Bx[x], cregs[x]);
    __syncthreads();   // [B] section masks visible

    // ---- old tokens of a continued tile: their codes from the tile as it is stored (read before anything is written)
    if (!starts) {
#pragma unroll
        for (int x = X0; x < X1; ++x) {
            if (!old) continue;
            const TensorStore& ts = x ? a.v : a.k;
            const uint8_t* src = ts.codes + (size_t)bh * a.pool_bytes + ts.tile_off[ti];
            qaqc::TileMasks om;
#pragma unroll
            for (int c = 0; c < 4; ++c) om.m[c] = s_tm[x].m[c] & ((1ull << s_lo) - 1ull);
            uint32_t ob[5];
            if (x == 0) { qaqc::section_bases<D, false>(om, ob); qaqc::read_pieces<D, false>(src, om, ob, slot, Bx[x], p, cregs[x]); }
            else        { qaqc::section_bases<D, true>(om, ob);  qaqc::read_pieces<D, true>(src, om, ob, slot, Bx[x], p, cregs[x]); }
        }
    }
    // ---- header and pieces into the shared-memory image of the tile (the values as token-major planes, which the
    //      copy to global memory turns into groups of four tokens)
    uint32_t vbase[5] = {0, 0, 0, 0, 0};
#pragma unroll
    for (int x = X0; x < X1; ++x) {
        if (tid < 4) qaqc::write_header(s_img[x - X0], s_tm[x], tid);
        const qaqc::PackedRanks rk{s_rank[x][slot & (QAQ_TILE - 1)]};
        if (x == 0) {
            uint32_t base[5];
#pragma unroll
            for (int c = 0; c < 5; ++c) base[c] = s_sec[x][c];
            if (valid || old) qaqc::write_pieces<D, false>(s_img[x - X0], rk, base, Bx[x], p, cregs[x]);
        } else {
#pragma unroll
            for (int c = 0; c < 5; ++c) vbase[c] = s_sec[x][c];
            if (valid || old) qaqc::write_planes_v<D>(s_img[x - X0], rk, vbase, Bx[x], p, cregs[x]);
        }
    }
    // ---- where the outliers of the new tokens are: (slot, channel) in (token, channel) order - entries of lanes
    //      p' < p of a token come first - listed in shared memory; their place needs only the scan of the counts.
    //      The values are fetched and the entries written afterwards by all threads, one entry each.
#pragma unroll
    for (int x = X0; x < X1; ++x) {
        uint32_t ob = valid ? ~inl[x] : 0u;
        const uint32_t mine = (uint32_t)__popc(ob);
        uint32_t before = 0;
#pragma unroll
        for (int d = 1; d < P; ++d) {
            const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, mine, d);
            if (p >= d) before += o;
        }
        if (ob) {
            const uint32_t all = ob;
            const uint32_t lp0 = s_cnt[x][slot & (QAQ_TILE - 1)] + before;
            while (ob) {
                const int bit = __ffs(ob) - 1;
                ob &= ob - 1;
                const int k = bit & 15, hi = bit >> 4;
                const int c = 2 * k + hi;                                   // channel inside the lane's 32
                // entries of lower channels: pairs k' < k, plus channel 2k when this is 2k+1
                const uint32_t lower = (((1u << k) - 1u) * 0x00010001u) | (hi ? (1u << k) : 0u);
                const uint32_t lp = lp0 + (uint32_t)__popc(all & lower);
                if (lp < OUT_STAGE) s_work[x - X0][lp] = (unsigned short)(((slot & (QAQ_TILE - 1)) << 8) | (32 * p + c));
            }
        }
    }
    // ---- allocation results (the atomics were issued before the codes were computed).  A pool without room:
    //      the space is given back, nothing about the tile is published and the CTA stops; the device status
    //      reports the lost tokens.
    if (warp == 0) {          // the byte pools
        bool fail = false;
        const bool mine = !(lane & 1) && lane >= 2 * X0 && lane < 2 * X1;
        const int x = lane >> 1;
        const TensorStore& ts = x ? a.v : a.k;
        if (mine) {
            const uint32_t off = starts ? my_base : ts.tile_off[ti];
            fail = (size_t)my_base + my_taken + 16 > a.pool_bytes || (size_t)off + s_tot[x] + 16 > a.pool_bytes;
            s_base[x] = off;
        }
        const bool any_fail = __any_sync(0xFFFFFFFFu, fail);
        if (mine) {
            if (any_fail) {
                if (my_taken) atomicSub(&ts.pool_end[bh], my_taken);
            } else {
                if (starts) ts.tile_off[ti] = my_base;
                ts.tile_nbytes[ti] = s_tot[x];
            }
        }
        if (lane == 0) {
            s_skip = any_fail ? 1 : 0;
            if (any_fail) atomicMax(a.status, (int)QAQ_ERR_CAPACITY);
        }
    } else if (warp == 1) {   // the outlier lists: what fits is known now, the table is written once the byte pools have answered
        if ((lane & 1) && lane >= 2 * X0 && lane < 2 * X1) {
            const int x = lane >> 1;
            const uint32_t room = my_base + 8 < a.ocap ? a.ocap - 8 - my_base : 0;  // 8 entries of read-ahead margin
            const uint32_t stored = my_amount < room ? my_amount : room;
            if (stored < my_amount) atomicMax(a.status, (int)QAQ_ERR_CAPACITY);
            s_obase[x] = my_base;
            s_olimit[x] = my_base + stored;
        }
    }
    __syncthreads();   // [C] image complete, pool positions known, every old byte of the tile has been read
    if (warp == 1 && (lane & 1) && lane >= 2 * X0 && lane < 2 * X1) {
        const int x = lane >> 1;
        const TensorStore& ts = x ? a.v : a.k;
        if (s_skip) {
            if (my_taken) atomicSub(&ts.opool_end[bh], my_taken);
        } else {
            const uint32_t stored = s_olimit[x] - s_obase[x];
            if (starts) { ts.tile_ooff[ti] = my_base; ts.tile_ocnt[ti] = stored; }
            else ts.tile_ocnt[ti] += stored;
        }
    }
    if (s_skip) { tick(); return; }

    // ---- the image goes out with vector stores; outlier list; per-token metadata
#pragma unroll
    for (int x = X0; x < X1; ++x) {
        const TensorStore& ts = x ? a.v : a.k;
        uint8_t* dst = ts.codes + (size_t)bh * a.pool_bytes + s_base[x];
        const uint32_t nb = (s_tot[x] + 15u) & ~15u;     // tiles start 16-byte aligned and own a rounded amount
        // the value of the first listed outlier of this thread is on its way (read again from the input: the
        // registers hold -inf in its place) while the image goes out
        const uint32_t ntot = s_otot[x], nst = ntot < OUT_STAGE ? ntot : OUT_STAGE;
        const __half* X = (x ? a.V : a.K) + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh;
        uint32_t w_first = 0;
        unsigned short v_first = 0;
        if ((uint32_t)tid < nst) {
            w_first = s_work[x - X0][tid];
            v_first = __half_as_ushort(X[(size_t)(tile * QAQ_TILE + (int)(w_first >> 8) - t_old) * a.st + (w_first & 0xFFu)]);
        }
        for (uint32_t o = tid * 16; o < nb; o += NT * 16) {
            uint4 v;
            if (x == 0 || o < (uint32_t)qaqc::QAQ_TILE_HDR) v = *reinterpret_cast<const uint4*>(s_img[x - X0] + o);
            else v = qaqc::group_unit_v<D>(s_img[x - X0], vbase, o);
            *reinterpret_cast<uint4*>(dst + o) = v;
        }
        // outlier entries: one listed outlier per thread (value read again from the input: the registers hold -inf in
        // its place), stores next to each other; a tile with more outliers than are listed writes the rest one by one
        {
            if ((uint32_t)tid < nst) {
                const uint32_t pos = s_obase[x] + tid;
                if (pos < s_olimit[x]) ts.outl[(size_t)bh * a.ocap + pos] = (uint32_t)v_first | ((w_first & 0xFFu) << 16) | ((w_first >> 8) << 24);
            }
            for (uint32_t i = tid + NT; i < nst; i += NT) {
                const uint32_t w = s_work[x - X0][i], sl = w >> 8, ch = w & 0xFFu;
                const uint32_t pos = s_obase[x] + i;
                if (pos < s_olimit[x])
                    ts.outl[(size_t)bh * a.ocap + pos] = (uint32_t)__half_as_ushort(X[(size_t)(tile * QAQ_TILE + (int)sl - t_old) * a.st + ch]) |
                                                          (ch << 16) | (sl << 24);
            }
            if (ntot > OUT_STAGE) {
                // rare.  Nothing of the listing pass is kept in registers for this: the lane reads its 32 channels
                // again and repeats the outlier test (same bounds, same bit order as analyze32)
                const __half2 lo2 = __half2half2(__float2half_ru(thr[2 * x])), hi2 = __half2half2(__float2half_rd(thr[2 * x + 1]));
                const __half* row = X + (size_t)(valid ? tn : 0) * a.st + 32 * p;
                uint32_t ob = 0;
                if (valid) {
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const __half2 v = as_h2(reinterpret_cast<const uint32_t*>(row)[k]);
                        ob |= (~(__hge2_mask(v, lo2) & __hle2_mask(v, hi2)) & 0x00010001u) << k;
                    }
                }
                const uint32_t mine = (uint32_t)__popc(ob);
                uint32_t lp0 = s_cnt[x][slot & (QAQ_TILE - 1)];
#pragma unroll
                for (int d = 1; d < P; ++d) {
                    const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, mine, d);
                    if (p >= d) lp0 += o;
                }
                const uint32_t all = ob;
                while (ob) {
                    const int bit = __ffs(ob) - 1;
                    ob &= ob - 1;
                    const int k = bit & 15, hi = bit >> 4;
                    const int c = 2 * k + hi;
                    const uint32_t lower = (((1u << k) - 1u) * 0x00010001u) | (hi ? (1u << k) : 0u);
                    const uint32_t lp = lp0 + (uint32_t)__popc(all & lower);
                    if (lp >= OUT_STAGE && s_obase[x] + lp < s_olimit[x])
                        ts.outl[(size_t)bh * a.ocap + s_obase[x] + lp] = (uint32_t)__half_as_ushort(row[c]) | ((uint32_t)(32 * p + c) << 16) |
                                                                           ((uint32_t)(slot & (QAQ_TILE - 1)) << 24);
                }
            }
        }
        if (valid && p == 0) {
            ts.bits[mt] = (uint8_t)Bx[x];
            ts.mnmx[mt] = (uint32_t)__half_as_ushort(__float2half_rn(mnf[x])) | ((uint32_t)__half_as_ushort(__float2half_rn(mxf[x])) << 16);
        }
    }
    tick();
}


template <bool SELECT_ONLY, int XSEL>
qaq_status launch_x(int D, dim3 grid, const QuantArgs& a, cudaStream_t s) {
    switch (D) {
        case 32: quant_kernel<32, SELECT_ONLY, XSEL><<<grid, 64, 0, s>>>(a); break;
        case 64: quant_kernel<64, SELECT_ONLY, XSEL><<<grid, 128, 0, s>>>(a); break;
        case 128: quant_kernel<128, SELECT_ONLY, XSEL><<<grid, 256, 0, s>>>(a); break;
        default: return QAQ_ERR_UNSUPPORTED_SHAPE;
    }
    return QAQ_OK;
}

template <bool SELECT_ONLY>
qaq_status launch(int D, dim3 grid, const QuantArgs& a, cudaStream_t s) {
    qaq_status st;
    if (SELECT_ONLY || grid.x * grid.y < QSPLIT_MIN_CTAS) {
        st = launch_x<SELECT_ONLY, -1>(D, grid, a, s);
    } else {   // large launches: keys and values of a tile in separate CTAs
        st = launch_x<SELECT_ONLY, 0>(D, grid, a, s);
        if (st == QAQ_OK) st = launch_x<SELECT_ONLY, 1>(D, grid, a, s);
    }
    if (st != QAQ_OK) return st;
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

qaq_status check_dense(const void* K, const void* V, long sb, long sh, long st, int D) {
    if (!K || !V) return QAQ_ERR_INVALID_ARG;
    if (((uintptr_t)K & 15) || ((uintptr_t)V & 15)) return QAQ_ERR_INVALID_ARG;  // 16-byte vector loads
    if (st < D || (sb & 7) || (sh & 7) || (st & 7) || sb < 0 || sh < 0) return QAQ_ERR_INVALID_ARG;
    return QAQ_OK;
}

}  // namespace

qaq_status qaq_launch_select(const qaq_config* cfg, const qaq_policy* pol, const void* K, const void* V, long sb,
                             long sh, long st, int n, const float* ring, const uint8_t* nvalid, const float* thr,
                             uint8_t* bitsK, uint8_t* bitsV, cudaStream_t s) {
    QuantArgs a{};
    a.K = (const __half*)K; a.V = (const __half*)V; a.sb = sb; a.sh = sh; a.st = st;
    a.H = cfg->heads; a.n_new = n; a.t_old = 0; a.tok_lo = 0; a.tok_hi = n; a.first_tile = 0;
    a.ring = ring; a.nvalid = nvalid; a.W = cfg->window; a.thr = thr;
    a.cK = pol->cK; a.cV = pol->cV; a.bmin = cfg->bits_min; a.bmax = cfg->bits_max;
    a.out_bitsK = bitsK; a.out_bitsV = bitsV;
    dim3 grid((n + QAQ_TILE - 1) / QAQ_TILE, cfg->batch * cfg->heads);
    return launch<true>(cfg->head_dim, grid, a, s);
}

qaq_status qaq_launch_append(qaq_cache* c, const void* K, const void* V, long sb, long sh, long st, int n_new,
                             const uint8_t* bitsK, const uint8_t* bitsV, const qaq_policy* pol, const float* ring,
                             const uint8_t* nvalid, const float* thr, cudaStream_t s) {
    QuantArgs a{};
    a.K = (const __half*)K; a.V = (const __half*)V; a.sb = sb; a.sh = sh; a.st = st;
    a.H = c->cfg.heads; a.n_new = n_new; a.t_old = (int)c->tokens;
    a.bitsK = bitsK; a.bitsV = bitsV; a.ring = ring; a.nvalid = nvalid; a.W = c->cfg.window; a.thr = thr;
    a.cK = pol ? pol->cK : 0.f; a.cV = pol ? pol->cV : 0.f; a.bmin = c->cfg.bits_min; a.bmax = c->cfg.bits_max;
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.ocap = c->ocap;
    a.tmax_pad = c->tmax_pad; a.ntiles = c->ntiles; a.status = c->d_status;
    const int D = c->cfg.head_dim, BH = c->BH;
    // Tiles are placed by atomic bump allocation, so a tile that stays open (partly filled)
    // must be the last thing allocated in its pool: the head of the range (completing an
    // open tile), the whole tiles, and a trailing partial tile go in separate launches.
    const int t0 = (int)c->tokens, t1 = t0 + n_new;
    int cur = t0;
    qaq_status stt;
    if (cur % QAQ_TILE != 0) {  // head: finish (or extend) the open tile
        const int end = min(t1, (cur / QAQ_TILE + 1) * QAQ_TILE);
        a.tok_lo = cur - t0; a.tok_hi = end - t0; a.first_tile = cur / QAQ_TILE;
        if ((stt = launch<false>(D, dim3(1, BH), a, s)) != QAQ_OK) return stt;
        cur = end;
    }
    const int full_end = t1 / QAQ_TILE * QAQ_TILE;
    if (cur < full_end) {       // body: whole tiles
        a.tok_lo = cur - t0; a.tok_hi = full_end - t0; a.first_tile = cur / QAQ_TILE;
        if ((stt = launch<false>(D, dim3((full_end - cur) / QAQ_TILE, BH), a, s)) != QAQ_OK) return stt;
        cur = full_end;
    }
    if (cur < t1) {             // tail: a new, partly filled tile
        a.tok_lo = cur - t0; a.tok_hi = t1 - t0; a.first_tile = cur / QAQ_TILE;
        if ((stt = launch<false>(D, dim3(1, BH), a, s)) != QAQ_OK) return stt;
    }
    c->tokens = t1;
    return QAQ_OK;
}

extern "C" qaq_status qaq_select_bits(const qaq_config* cfg, const qaq_policy* policy, const void* K, const void* V,
                                      long stride_b, long stride_h, long stride_t, int n_tokens,
                                      const float* score_ring, const uint8_t* nvalid, const float* thr,
                                      uint8_t* bitsK, uint8_t* bitsV, void* stream) {
    if (!cfg || !policy || !score_ring || !nvalid || !thr || !bitsK || !bitsV || n_tokens < 0) return QAQ_ERR_INVALID_ARG;
    if (!qaq_dim_ok(cfg->head_dim)) return QAQ_ERR_UNSUPPORTED_SHAPE;
    if (cfg->bits_min < 1 || cfg->bits_max > 8 || cfg->bits_min > cfg->bits_max || cfg->window < 1) return QAQ_ERR_UNSUPPORTED_SHAPE;
    qaq_status st = check_dense(K, V, stride_b, stride_h, stride_t, cfg->head_dim);
    if (st != QAQ_OK) return st;
    if (n_tokens == 0) return QAQ_OK;
    return qaq_launch_select(cfg, policy, K, V, stride_b, stride_h, stride_t, n_tokens, score_ring, nvalid, thr, bitsK,
                             bitsV, (cudaStream_t)stream);
}

extern "C" qaq_status qaq_quantize_append(qaq_cache* c, const void* K_new, const void* V_new, long stride_b,
                                          long stride_h, long stride_t, int n_new, const uint8_t* bitsK,
                                          const uint8_t* bitsV, const qaq_policy* policy, const float* score_ring,
                                          const uint8_t* nvalid, const float* thr, void* stream) {
    if (!c || !thr || n_new < 0) return QAQ_ERR_INVALID_ARG;
    if ((bitsK == nullptr) != (bitsV == nullptr)) return QAQ_ERR_INVALID_ARG;
    if (!bitsK && (!policy || !score_ring || !nvalid)) return QAQ_ERR_INVALID_ARG;
    qaq_status st = check_dense(K_new, V_new, stride_b, stride_h, stride_t, c->cfg.head_dim);
    if (st != QAQ_OK) return st;
    if (c->tokens + n_new > c->cfg.max_tokens) return QAQ_ERR_CAPACITY;
    if (n_new == 0) return QAQ_OK;
    return qaq_launch_append(c, K_new, V_new, stride_b, stride_h, stride_t, n_new, bitsK, bitsV, policy, score_ring,
                             nvalid, thr, (cudaStream_t)stream);
}

// One new token per (b,h) with the token count taken from (and advanced in) device memory: the open tile (or a new one)
// of every (b,h) is rebuilt by one CTA, as in the head / tail launch of qaq_launch_append.  Nothing on the host changes,
// so the call can be captured in a CUDA graph and replayed.
extern "C" qaq_status qaq_stream_append(qaq_cache* c, const void* k_new, const void* v_new, long stride_b, long stride_h,
                                        const uint8_t* bitK, const uint8_t* bitV, const qaq_policy* policy,
                                        const float* score_col, const uint8_t* nvalid, const float* thr, void* stream) {
    if (!c || !thr) return QAQ_ERR_INVALID_ARG;
    if ((bitK == nullptr) != (bitV == nullptr)) return QAQ_ERR_INVALID_ARG;
    if (!bitK && (!policy || !score_col || !nvalid)) return QAQ_ERR_INVALID_ARG;
    const int D = c->cfg.head_dim;
    qaq_status st = check_dense(k_new, v_new, stride_b, stride_h, D, D);
    if (st != QAQ_OK) return st;
    QuantArgs a{};
    a.K = (const __half*)k_new; a.V = (const __half*)v_new; a.sb = stride_b; a.sh = stride_h; a.st = D;
    a.H = c->cfg.heads; a.n_new = 1; a.tok_lo = 0; a.tok_hi = 1;
    a.bitsK = bitK; a.bitsV = bitV; a.ring = score_col; a.nvalid = nvalid; a.W = c->cfg.window; a.thr = thr;
    a.cK = policy ? policy->cK : 0.f; a.cV = policy ? policy->cV : 0.f; a.bmin = c->cfg.bits_min; a.bmax = c->cfg.bits_max;
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.ocap = c->ocap;
    a.tmax_pad = c->tmax_pad; a.ntiles = c->ntiles; a.status = c->d_status;
    a.d_count = qaq_d_count(c); a.d_ticket = qaq_d_ticket(c); a.max_tokens = (int)c->cfg.max_tokens;
    st = launch_x<false, -1>(D, dim3(1, c->BH), a, (cudaStream_t)stream);
    if (st != QAQ_OK) return st;
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}
