// S1-S3: bit-width selection, outlier split, uniform quantization and bit-packing.
//
// One CTA handles one tile (QAQ_TILE consecutive tokens) of one (b,h); head_dim/32 lanes
// own one token, each lane 32 consecutive channels of K and of V (64 bytes each), held in
// registers from the min/max pass to the packing pass, so K and V are read from HBM once.
//   phase 0  attention-window maximum of the score rows (Section 4.2)
//   phase 1  outlier masks and min/max of the non-outliers in binary16 pair arithmetic
//            (exact: the inputs are binary16), width from the exponents (Section 4.1)
//   phase 2  warp 0: exclusive scans of byte lengths and outlier counts over the tile,
//            space taken from the (b,h) pools by atomicAdd
//   phase 3  codes (binary32: one sub, one mul, round down), planes built lane-locally,
//            vector stores; outlier entries placed by popc ranks
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
    uint8_t* out_bitsK;    // selection only
    uint8_t* out_bitsV;
};

// B = min{b in [bmin,bmax] : v <= c * 2^b}, bmax if none; c * 2^b is an exact power-of-two
// scaling.  For positive normal v and c the answer is read off the exponents: with
// v = mv * 2^ev, c = mc * 2^ec (mv, mc in [1,2)) the smallest b is ev - ec if mv <= mc,
// else ev - ec + 1.
__device__ __forceinline__ int ladder(float v, float c, int bmin, int bmax) {
    if (!(c > 0.f)) return bmax;
    if (v <= __fmul_rn(c, (float)(1 << bmin))) return bmin;
    const int vb = __float_as_int(v), cb = __float_as_int(c);
    if (cb < 0x00800000 || vb < 0x00800000) {  // subnormal operand: plain ladder
        for (int b = bmin; b <= bmax; ++b)
            if (v <= __fmul_rn(c, (float)(1 << b))) return b;
        return bmax;
    }
    int b = (vb >> 23) - (cb >> 23) + (((vb & 0x7FFFFF) > (cb & 0x7FFFFF)) ? 1 : 0);
    return b < bmin ? bmin : (b > bmax ? bmax : b);
}

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
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ __half2 as_h2(uint32_t x) { return *reinterpret_cast<__half2*>(&x); }
__device__ __forceinline__ uint32_t as_u32(__half2 x) { return *reinterpret_cast<uint32_t*>(&x); }
// binary32 (x - c) with x a binary16 value: one rounding, same as widening x exactly and subtracting
__device__ __forceinline__ float sub_f32_f16(unsigned short x, float c) {
    float d;
    asm("sub.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(x), "f"(c));
    return d;
}

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

template <int BYTES>
__device__ __forceinline__ void store_words(uint8_t* dst, const uint32_t* w, int nwords) {
    // nwords * 4 bytes to dst, which is BYTES-aligned (BYTES in {4, 8, 16})
    if (BYTES == 16 && nwords % 4 == 0) {
        for (int i = 0; i < nwords; i += 4) *reinterpret_cast<uint4*>(dst + 4 * i) = make_uint4(w[i], w[i + 1], w[i + 2], w[i + 3]);
    } else if (BYTES >= 8 && nwords % 2 == 0) {
        for (int i = 0; i < nwords; i += 2) *reinterpret_cast<uint2*>(dst + 4 * i) = make_uint2(w[i], w[i + 1]);
    } else {
        for (int i = 0; i < nwords; ++i) *reinterpret_cast<uint32_t*>(dst + 4 * i) = w[i];
    }
}

// space from a (b,h) pool: `whole` tiles take a rounded-up amount in one atomic; a tile that is
// being continued takes the exact amount and is padded to the unit when it closes
__device__ __forceinline__ uint32_t pool_take(uint32_t* pool, uint32_t amount, uint32_t unit_mask, bool whole, bool closes) {
    uint32_t base;
    if (whole) {
        base = atomicAdd(pool, (amount + unit_mask) & ~unit_mask);
    } else {
        base = atomicAdd(pool, amount);
        if (closes) {
            const uint32_t pad = (0u - (base + amount)) & unit_mask;
            if (pad) atomicAdd(pool, pad);
        }
    }
    return base;
}

// One CTA = one tile of 64 tokens of one (b,h); P = D/32 lanes own a token, each lane 32
// consecutive channels (64 bytes) of K and of V, kept in registers across all phases.
// Order of work (barriers in brackets): loads, attention window, outlier masks and ranges,
// widths [A] warp 0 scans the tile and takes pool space with four atomics in flight at once
// while every warp computes its codes [B] planes into a shared-memory image of the tile
// [C] the image goes out with 16-byte stores; outlier entries and per-token metadata follow.
// XSEL: -1 = keys and values in one CTA; 0 / 1 = this launch handles only the keys / only the values of a tile
// (half the registers and shared memory per CTA, so more tiles are in flight per SM).
template <int D, bool SELECT_ONLY, int XSEL>
__global__ void __launch_bounds__(2 * D, XSEL < 0 ? (D == 128 ? 3 : 4) : (D == 128 ? 5 : 6)) quant_kernel(const QuantArgs a) {
    constexpr int X0 = XSEL < 0 ? 0 : XSEL, X1 = XSEL < 0 ? 2 : XSEL + 1;
    constexpr int P = D / 32;            // lanes per token
    constexpr int ALIGN = D / 8 >= 16 ? 16 : D / 8;  // alignment of a token's bytes inside a tile
    constexpr int NT = 2 * D;            // threads
    const int bh = blockIdx.y;
    const int tile = a.first_tile + blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid / P, p = tid % P;

    const int abs_lo = max(tile * QAQ_TILE, a.t_old + a.tok_lo);
    const int abs_hi = min((tile + 1) * QAQ_TILE, a.t_old + a.tok_hi);
    const int s_lo = abs_lo - tile * QAQ_TILE, s_hi = abs_hi - tile * QAQ_TILE;
    const bool valid = slot >= s_lo && slot < s_hi;
    const int tn = tile * QAQ_TILE + slot - a.t_old;  // index among the new tokens

    __shared__ uint32_t s_len[2][QAQ_TILE];   // bytes, then exclusive byte offsets
    __shared__ uint32_t s_cnt[2][QAQ_TILE];   // outlier counts, then exclusive offsets
    __shared__ uint32_t s_tot[2], s_base[2], s_obase[2], s_olimit[2];
    __shared__ int s_skip;
    __shared__ __align__(16) uint8_t s_img[SELECT_ONLY ? 1 : X1 - X0][SELECT_ONLY ? 16 : QAQ_TILE * D];  // packed tile (K and V)

    const float* thr = a.thr + (size_t)bh * 4;
    const bool given = a.bitsK != nullptr;

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

    // ---- attention window: the P lanes of a token take its rows p, p+P, ... and combine by shuffles
    float shat = __int_as_float(0xff800000);
    int nv_tok = 0;
    {
        if (XSEL != 0 && !given && valid) {
            nv_tok = a.nvalid[(size_t)bh * a.n_new + tn];
            nv_tok = nv_tok < a.W ? nv_tok : a.W;
            const float* r = a.ring + (size_t)bh * a.W * a.n_new + tn;
            for (int i = p; i < nv_tok; i += P) shat = fmaxf(shat, r[(size_t)i * a.n_new]);
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
        if (p == 0) {                                   // every slot of the tile is written: empty ones count nothing
            s_len[x][slot] = valid ? (uint32_t)(D * B / 8) : 0u;
            s_cnt[x][slot] = valid ? cntx[x] : 0u;
            if (SELECT_ONLY && valid) (x ? a.out_bitsV : a.out_bitsK)[(size_t)bh * a.n_new + tn] = (uint8_t)B;
        }
    }
    if (SELECT_ONLY) return;
    __syncthreads();   // [A] byte lengths and outlier counts visible

    // ---- warp 0: scans over the tile; lanes 0..3 each take space from one pool (four atomics in flight)
    const bool starts = (s_lo == 0), closes = (s_hi == QAQ_TILE), whole = starts && closes;
    uint32_t my_base = 0, my_amount = 0;
    if (warp == 0) {
        uint32_t amount[2][2];   // [tensor][0: bytes, 1: outliers]
#pragma unroll
        for (int x = X0; x < X1; ++x) {
            uint32_t l0 = s_len[x][lane], l1 = s_len[x][lane + 32];
            uint32_t c0 = s_cnt[x][lane], c1 = s_cnt[x][lane + 32];
            uint32_t il0 = l0, il1 = l1, ic0 = c0, ic1 = c1;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                uint32_t t0 = __shfl_up_sync(0xFFFFFFFFu, il0, d), t1 = __shfl_up_sync(0xFFFFFFFFu, il1, d);
                uint32_t u0 = __shfl_up_sync(0xFFFFFFFFu, ic0, d), u1 = __shfl_up_sync(0xFFFFFFFFu, ic1, d);
                if (lane >= d) { il0 += t0; il1 += t1; ic0 += u0; ic1 += u1; }
            }
            const uint32_t tot0 = __shfl_sync(0xFFFFFFFFu, il0, 31), tot1 = __shfl_sync(0xFFFFFFFFu, il1, 31);
            const uint32_t ctot0 = __shfl_sync(0xFFFFFFFFu, ic0, 31), ctot1 = __shfl_sync(0xFFFFFFFFu, ic1, 31);
            s_len[x][lane] = il0 - l0; s_len[x][lane + 32] = tot0 + il1 - l1;
            s_cnt[x][lane] = ic0 - c0; s_cnt[x][lane + 32] = ctot0 + ic1 - c1;
            amount[x][0] = tot0 + tot1; amount[x][1] = ctot0 + ctot1;
            if (lane == 0) s_tot[x] = amount[x][0];
        }
        if (lane >= 2 * X0 && lane < 2 * X1) {
            const int x = lane >> 1, pool = lane & 1;
            const TensorStore& ts = x ? a.v : a.k;
            my_amount = x ? amount[1][pool] : amount[0][pool];
            my_base = pool_take(pool ? &ts.opool_end[bh] : &ts.pool_end[bh], my_amount, pool ? 3u : 15u, whole, closes);
        }
    }

    // ---- codes (every warp; needs only registers): channels 4j..4j+3 in the byte lanes of creg[j]
    uint32_t cregs[2][8];
#pragma unroll
    for (int x = X0; x < X1; ++x) {
        const uint32_t (&v)[16] = x ? vv : vk;
        const int B = Bx[x];
        const float mn = mnf[x];
        const float step = __fmul_rn(__fsub_rn(mxf[x], mn), __int_as_float((127 - B) << 23));
        const float inv = step > 0.f ? __fdiv_rn(1.0f, step) : 0.f;
        // zero step (constant token): every code is 0, and -inf * 0 = NaN must not clamp to the top code
        const float topf = step > 0.f ? (float)((1 << B) - 1) : 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t f[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t pair = v[2 * j + (i >> 1)];
                const unsigned short h = (i & 1) ? (unsigned short)(pair >> 16) : (unsigned short)(pair & 0xFFFF);
                float t = __fmul_rn(sub_f32_f16(h, mn), inv);            // -inf for an outlier
                t = fminf(t, topf);
                f[i] = __float_as_uint(__fadd_rd(t, 8388608.0f));   // 2^23 + floor(t): the code is the low byte (0 for -inf)
            }
            cregs[x][j] = prmt(prmt(f[0], f[1], 0x0040u), prmt(f[2], f[3], 0x0040u), 0x5410u);
        }
    }
    __syncthreads();   // [B] offsets inside the tile visible

    // ---- planes into the shared-memory image of the tile
#pragma unroll
    for (int x = X0; x < X1; ++x) {
        const uint32_t (&creg)[8] = cregs[x];
        const int B = Bx[x];
        uint8_t* tok = s_img[x - X0] + s_len[x][slot & (QAQ_TILE - 1)];
        if (B & 8) {
            store_words<ALIGN>(tok + p * 32, creg, 8);
        }
        if (B & 4) {
            const int sh = B & 3;
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                w[j] = ((creg[2 * j] >> sh) & 0x0F0F0F0Fu) | (((creg[2 * j + 1] >> sh) & 0x0F0F0F0Fu) << 4);
            store_words<ALIGN>(tok + (B & 8) * (D / 8) + p * 16, w, 4);
        }
        if (B & 2) {
            const int sh = B & 1;
            uint32_t w[2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                uint32_t acc = 0;
#pragma unroll
                for (int m = 0; m < 4; ++m) acc |= ((creg[4 * j + m] >> sh) & 0x03030303u) << (2 * m);
                w[j] = acc;
            }
            store_words<(ALIGN > 8 ? 8 : ALIGN)>(tok + (B & 12) * (D / 8) + p * 8, w, 2);
        }
        if (B & 1) {
            uint32_t acc = 0;
#pragma unroll
            for (int m = 0; m < 8; ++m) acc |= (creg[m] & 0x01010101u) << m;
            *reinterpret_cast<uint32_t*>(tok + (B & 14) * (D / 8) + p * 4) = acc;
        }
    }
    // ---- allocation results (the atomics were issued before the codes were computed)
    if (warp == 0 && lane >= 2 * X0 && lane < 2 * X1) {
        const int x = lane >> 1, pool = lane & 1;
        const TensorStore& ts = x ? a.v : a.k;
        const size_t ti = (size_t)bh * a.ntiles + tile;
        if (lane == 2 * X0) s_skip = 0;
        if (pool == 0) {
            if ((size_t)my_base + my_amount + 16 > a.pool_bytes) { atomicMax(a.status, (int)QAQ_ERR_CAPACITY); s_skip = 1; }
            if (starts) { ts.tile_off[ti] = my_base; ts.tile_nbytes[ti] = my_amount; }
            else ts.tile_nbytes[ti] += my_amount;
            s_base[x] = my_base;
        } else {
            const uint32_t room = my_base + 8 < a.ocap ? a.ocap - 8 - my_base : 0;  // 8 entries of read-ahead margin
            const uint32_t stored = my_amount < room ? my_amount : room;
            if (stored < my_amount) atomicMax(a.status, (int)QAQ_ERR_CAPACITY);
            if (starts) { ts.tile_ooff[ti] = my_base; ts.tile_ocnt[ti] = stored; }
            else ts.tile_ocnt[ti] += stored;
            s_obase[x] = my_base;
            s_olimit[x] = my_base + stored;
        }
    }
    __syncthreads();   // [C] image complete, pool positions known
    if (s_skip) return;

    // ---- the image goes out with vector stores; outlier list; per-token metadata
#pragma unroll
    for (int x = X0; x < X1; ++x) {
        const TensorStore& ts = x ? a.v : a.k;
        uint8_t* dst = ts.codes + (size_t)bh * a.pool_bytes + s_base[x];
        const uint32_t nb = s_tot[x];
        for (uint32_t o = tid * ALIGN; o < nb; o += NT * ALIGN) {
            if (ALIGN == 16) *reinterpret_cast<uint4*>(dst + o) = *reinterpret_cast<const uint4*>(s_img[x - X0] + o);
            else if (ALIGN == 8) *reinterpret_cast<uint2*>(dst + o) = *reinterpret_cast<const uint2*>(s_img[x - X0] + o);
            else *reinterpret_cast<uint32_t*>(dst + o) = *reinterpret_cast<const uint32_t*>(s_img[x - X0] + o);
        }
        // outliers in (token, channel) order: entries of lanes p' < p come first
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
            const uint32_t pos0 = s_obase[x] + s_cnt[x][slot & (QAQ_TILE - 1)] + before;
            const __half* row = (x ? a.V : a.K) + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh + (size_t)tn * a.st + 32 * p;
            while (ob) {
                const int bit = __ffs(ob) - 1;
                ob &= ob - 1;
                const int k = bit & 15, hi = bit >> 4;
                const int c = 2 * k + hi;                                   // channel inside the lane's 32
                // entries of lower channels: pairs k' < k, plus channel 2k when this is 2k+1
                const uint32_t lower = (((1u << k) - 1u) * 0x00010001u) | (hi ? (1u << k) : 0u);
                const uint32_t pos = pos0 + (uint32_t)__popc(all & lower);
                if (pos < s_olimit[x])
                    ts.outl[(size_t)bh * a.ocap + pos] = (uint32_t)__half_as_ushort(row[c]) | ((uint32_t)(32 * p + c) << 16) |
                                                          ((uint32_t)(slot & (QAQ_TILE - 1)) << 24);
            }
        }
        if (valid && p == 0) {
            const size_t t = (size_t)bh * a.tmax_pad + (size_t)tile * QAQ_TILE + slot;
            ts.bits[t] = (uint8_t)Bx[x];
            ts.mnmx[t] = (uint32_t)__half_as_ushort(__float2half_rn(mnf[x])) | ((uint32_t)__half_as_ushort(__float2half_rn(mxf[x])) << 16);
        }
    }
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
    if (SELECT_ONLY || grid.x * grid.y < 4096) {
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
