// The one copy of the codec arithmetic and of the tile layout, used by the quantize, re-quantize,
// export and decode kernels (not part of the ABI).
//
// Codes (Section 4.1 of the paper: the range [min,max] of a token's non-outlier entries is cut into 2^B equal
// segments): step = (max-min) * 2^-B, code = min(2^B-1, floor((x-min) * (1/step))) in binary32 with separately
// rounded operations; an outlier's code slot holds 0.
//
// Pieces.  A B-bit code is cut into the power-of-two pieces of B's binary representation, widest first, the
// widest holding the most significant bits (7 = 4+2+1): the piece of width w (w in {8,4,2,1}, present iff B & w)
// is (code >> (B & (w-1))) & (2^w - 1).
//
// Tile layout in the code pool.  A tile (QAQ_TILE consecutive tokens of one (b,h) and tensor) is stored as four
// sections, one per piece width, in the order 8, 4, 2, 1.  Section w holds the w-bit pieces of the tokens that
// have one, in token order; the position of a token among them is its rank r_w.
//   keys:    item r of section w is the plane of that token: head_dim*w/8 bytes; channel d = 32p + 4j + i sits in
//            little-endian word p*w + j*w/8 of the plane at bit 8i + w*(j mod 8/w)  (after one shift and a
//            byte-replicated mask a word has one field per byte lane: the operand of dp4a against four channels
//            of the query).
//   values:  items are stored in groups of four (the last group of a section is padded with zero bytes):
//            group G = items 4G..4G+3, head_dim*w/2 bytes, made of 32-bit words whose byte lane i belongs to item
//            4G+i and whose bit field m (bits w*m .. w*m+w-1 of every byte) is one channel, so that a masked word is
//            four tokens of one channel, one per byte: the A operand of the integer tensor-core instruction
//            mma.m16n8k32 with rows = channels and k = tokens.  Channel c sits in word c / (8/w), field
//            c % (8/w): seen per token, a group interleaves byte by byte the four tokens' rows of packed fields
//            (consecutive channels, lowest bits first).  The MMA lane with group id g takes the head_dim/8
//            channels from g*head_dim/8 on as its rows, one vector load per group.
// The sections are preceded by a header of QAQ_TILE_HDR bytes: the four 64-bit masks "slot t has a piece of width
// 8, 4, 2, 1" (widths, ranks and section sizes of a tile can be read off them without the per-token metadata).
// A tile therefore takes the header plus sum_t head_dim*B_t/8 bytes for keys, and that plus the group padding for
// values.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

#include "qaq.h"

namespace qaqc {

// ------------------------------------------------------------------------------------------ small helpers
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// binary32 (x - c) with x a binary16 value: one rounding, same as widening x exactly and subtracting
__device__ __forceinline__ float sub_f32_f16(unsigned short x, float c) {
    float d;
    asm("sub.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(x), "f"(c));
    return d;
}

// B = min{b in [bmin,bmax] : v <= c * 2^b}, bmax if none (the bit count of Section 4.1 without a logarithm;
// c * 2^b is an exact power-of-two scaling).  For positive normal v and c the answer is read off the exponents:
// with v = mv * 2^ev, c = mc * 2^ec (mv, mc in [1,2)) the smallest b is ev - ec if mv <= mc, else ev - ec + 1.
__device__ __forceinline__ int ladder(float v, float c, int bmin, int bmax) {
    if (!(c > 0.f)) return bmax;
    if (v <= __fmul_rn(c, (float)(1 << bmin))) return bmin;
    const int vb = __float_as_int(v), cb = __float_as_int(c);
    if (cb < 0x00800000 || vb < 0x00800000) {  // subnormal operand: plain ladder
        for (int b = bmin; b <= bmax; ++b)
            if (v <= __fmul_rn(c, (float)(1 << b))) return b;
        return bmax;
    }
    const int b = (vb >> 23) - (cb >> 23) + (((vb & 0x7FFFFF) > (cb & 0x7FFFFF)) ? 1 : 0);
    return b < bmin ? bmin : (b > bmax ? bmax : b);
}

// step of a token from its stored range and width (exact scaling)
__device__ __forceinline__ float step_of(float mn, float mx, int B) {
    return __fmul_rn(__fsub_rn(mx, mn), __int_as_float((127 - B) << 23));
}

// Codes of 32 channels held as 16 binary16 pairs (v[k] = channels 2k, 2k+1; outliers already replaced by -inf,
// which yields code 0): creg[j] = codes of channels 4j..4j+3, one per byte.
__device__ __forceinline__ void codes32(const uint32_t (&v)[16], float mn, float mx, int B, uint32_t (&creg)[8]) {
    const float step = step_of(mn, mx, B);
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
            float t = __fmul_rn(sub_f32_f16(h, mn), inv);   // -inf for an outlier
            t = fminf(t, topf);
            f[i] = __float_as_uint(__fadd_rd(t, 8388608.0f));   // 2^23 + floor(t): the code is the low byte (0 for -inf)
        }
        creg[j] = prmt(prmt(f[0], f[1], 0x0040u), prmt(f[2], f[3], 0x0040u), 0x5410u);
    }
}

// outliers (entries outside [lo2, hi2], NaN included) of 16 binary16 pairs replaced by -inf
__device__ __forceinline__ void mask_outliers32(uint32_t (&v)[16], __half2 lo2, __half2 hi2) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const __half2 x = *reinterpret_cast<const __half2*>(&v[k]);
        const uint32_t m = __hge2_mask(x, lo2) & __hle2_mask(x, hi2);
        v[k] = (v[k] & m) | (0xFC00FC00u & ~m);
    }
}

// ------------------------------------------------------------------------------------------ tile layout
constexpr int QAQ_TILE_HDR = 32;

// Which slots of a tile have a piece of width 8 >> c (c = 0..3): one 64-bit mask per width.
struct TileMasks {
    unsigned long long m[4];
};

// largest tile: the header, 64 tokens at 8 bits plus the worst padding of the value groups (three items in each of the four
// sections), rounded up to a multiple of 16 so that images of tiles can sit back to back in shared memory
__host__ __device__ constexpr int v_tile_bytes_max(int D) {
    return (QAQ_TILE_HDR + QAQ_TILE_TOKENS * D + 3 * (D * 15 / 8) + 15) / 16 * 16;
}

// Byte offsets of the four sections inside a tile (base[4] = bytes of the tile).
template <int D, bool IS_V>
__device__ __forceinline__ void section_bases(const int (&n)[4], uint32_t (&base)[5]) {
    uint32_t o = QAQ_TILE_HDR;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int w = 8 >> c;
        base[c] = o;
        o += IS_V ? (uint32_t)((n[c] + 3) >> 2) * (uint32_t)(D * w / 2) : (uint32_t)n[c] * (uint32_t)(D * w / 8);
    }
    base[4] = o;
}
template <int D, bool IS_V>
__device__ __forceinline__ void section_bases(const TileMasks& tm, uint32_t (&base)[5]) {
    int n[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) n[c] = __popcll(tm.m[c]);
    section_bases<D, IS_V>(n, base);
}
// the header of a tile image (16-byte aligned, shared or global memory)
__device__ __forceinline__ void write_header(uint8_t* img, const TileMasks& tm, int c) {
    reinterpret_cast<unsigned long long*>(img)[c] = tm.m[c];
}
__device__ __forceinline__ int rank_in(const TileMasks& tm, int c, int slot) {
    return __popcll(tm.m[c] & ((1ull << slot) - 1ull));
}
// The ranks of one slot in the four sections, either taken from the masks when asked for or handed over packed
// (rank in section c in byte c; a tile has at most 64 items per section).
struct MaskRanks {
    const TileMasks& tm;
    int slot;
    __device__ __forceinline__ int operator()(int c) const { return rank_in(tm, c, slot); }
};
struct PackedRanks {
    uint32_t rk;
    __device__ __forceinline__ int operator()(int c) const { return (int)((rk >> (8 * c)) & 0xFFu); }
};

template <int NW>
__device__ __forceinline__ void store_words(uint8_t* p, const uint32_t* w) {   // p is min(16, 4*NW)-byte aligned
    if (NW % 4 == 0) {
#pragma unroll
        for (int i = 0; i < NW; i += 4) *reinterpret_cast<uint4*>(p + 4 * i) = make_uint4(w[i], w[i + 1], w[i + 2], w[i + 3]);
    } else if (NW == 2) {
        *reinterpret_cast<uint2*>(p) = make_uint2(w[0], w[1]);
    } else {
        *reinterpret_cast<uint32_t*>(p) = w[0];
    }
}
template <int NW>
__device__ __forceinline__ void load_words(const uint8_t* p, uint32_t* w) {
    if (NW % 4 == 0) {
#pragma unroll
        for (int i = 0; i < NW; i += 4) {
            const uint4 v = *reinterpret_cast<const uint4*>(p + 4 * i);
            w[i] = v.x; w[i + 1] = v.y; w[i + 2] = v.z; w[i + 3] = v.w;
        }
    } else if (NW == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        w[0] = v.x; w[1] = v.y;
    } else {
        w[0] = *reinterpret_cast<const uint32_t*>(p);
    }
}

// The pieces of one thread's 32 channels (block p of the token in `slot`, codes one per byte in creg) written
// into a tile image (shared or global memory, 16-byte aligned).
template <int D, bool IS_V, typename Ranks>
__device__ __forceinline__ void write_pieces(uint8_t* img, const Ranks& rk, const uint32_t (&base)[5], int B, int p,
                                             const uint32_t (&creg)[8]) {
    if (!IS_V) {
        if (B & 8) store_words<8>(img + base[0] + rk(0) * D + p * 32, creg);
        if (B & 4) {
            const int sh = B & 3;
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)     // the odd register goes straight to the high nibbles: one shift by 4 - sh
                w[j] = ((creg[2 * j] >> sh) & 0x0F0F0F0Fu) | ((creg[2 * j + 1] << (4 - sh)) & 0xF0F0F0F0u);
            store_words<4>(img + base[1] + rk(1) * (D / 2) + p * 16, w);
        }
        if (B & 2) {
            const int sh = B & 1;
            uint32_t w[2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                uint32_t acc = (creg[4 * j] >> sh) & 0x03030303u;
#pragma unroll
                for (int m = 1; m < 4; ++m) acc |= (creg[4 * j + m] << (2 * m - sh)) & (0x03030303u << (2 * m));
                w[j] = acc;
            }
            store_words<2>(img + base[2] + rk(2) * (D / 4) + p * 8, w);
        }
        if (B & 1) {
            uint32_t acc = 0;
#pragma unroll
            for (int m = 0; m < 8; ++m) acc |= (creg[m] & 0x01010101u) << m;
            *reinterpret_cast<uint32_t*>(img + base[3] + rk(3) * (D / 8) + p * 4) = acc;
        }
    } else {
        // values: byte lane (rank & 3) of the words of group rank >> 2; channel 32p + 4j + b is byte b of creg[j]
        if (B & 8) {
            const int r = rk(0);
            uint8_t* grp = img + base[0] + (r >> 2) * (D * 4) + (r & 3);
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int b = 0; b < 4; ++b) grp[4 * (32 * p + 4 * j + b)] = (uint8_t)(creg[j] >> (8 * b));
        }
        if (B & 4) {
            const int sh = B & 3, r = rk(1);
            uint8_t* grp = img + base[1] + (r >> 2) * (D * 2) + (r & 3);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t x = (creg[j] >> sh) & 0x0F0F0F0Fu;
                const uint32_t y = x | (x >> 4);     // byte 0: channels 4j, 4j+1; byte 2: channels 4j+2, 4j+3
                grp[4 * (16 * p + 2 * j)] = (uint8_t)y;
                grp[4 * (16 * p + 2 * j + 1)] = (uint8_t)(y >> 16);
            }
        }
        if (B & 2) {
            const int sh = B & 1, r = rk(2);
            uint8_t* grp = img + base[2] + (r >> 2) * D + (r & 3);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t x = (creg[j] >> sh) & 0x03030303u;
                const uint32_t z = x | (x >> 6);
                grp[4 * (8 * p + j)] = (uint8_t)(z | (z >> 12));    // the four 2-bit fields of channels 4j..4j+3
            }
        }
        if (B & 1) {
            const int r = rk(3);
            uint8_t* grp = img + base[3] + (r >> 2) * (D / 2) + (r & 3);
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const uint32_t n0 = (((creg[j] & 0x01010101u) * 0x01020408u) >> 24) & 15u;
                const uint32_t n1 = (((creg[j + 1] & 0x01010101u) * 0x01020408u) >> 24) & 15u;
                grp[4 * (4 * p + j / 2)] = (uint8_t)(n0 | (n1 << 4));
            }
        }
    }
}

template <int D, bool IS_V>
__device__ __forceinline__ void write_pieces(uint8_t* img, const TileMasks& tm, const uint32_t (&base)[5], int slot, int B,
                                             int p, const uint32_t (&creg)[8]) {
    write_pieces<D, IS_V>(img, MaskRanks{tm, slot}, base, B, p, creg);
}

// The inverse: codes of one thread's 32 channels (one per byte) put together from the token's pieces.
template <int D, bool IS_V>
__device__ __forceinline__ void read_pieces(const uint8_t* img, const TileMasks& tm, const uint32_t (&base)[5], int slot, int B,
                                            int p, uint32_t (&creg)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) creg[j] = 0;
    if (!IS_V) {
        if (B & 8) load_words<8>(img + base[0] + rank_in(tm, 0, slot) * D + p * 32, creg);
        if (B & 4) {
            const int sh = B & 3;
            uint32_t w[4];
            load_words<4>(img + base[1] + rank_in(tm, 1, slot) * (D / 2) + p * 16, w);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                creg[2 * j] |= (w[j] & 0x0F0F0F0Fu) << sh;
                creg[2 * j + 1] |= ((w[j] >> 4) & 0x0F0F0F0Fu) << sh;
            }
        }
        if (B & 2) {
            const int sh = B & 1;
            uint32_t w[2];
            load_words<2>(img + base[2] + rank_in(tm, 2, slot) * (D / 4) + p * 8, w);
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int m = 0; m < 4; ++m) creg[4 * j + m] |= ((w[j] >> (2 * m)) & 0x03030303u) << sh;
        }
        if (B & 1) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(img + base[3] + rank_in(tm, 3, slot) * (D / 8) + p * 4);
#pragma unroll
            for (int m = 0; m < 8; ++m) creg[m] |= (w >> m) & 0x01010101u;
        }
    } else {
        if (B & 8) {
            const int r = rank_in(tm, 0, slot);
            const uint8_t* grp = img + base[0] + (r >> 2) * (D * 4) + (r & 3);
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int b = 0; b < 4; ++b) creg[j] |= (uint32_t)grp[4 * (32 * p + 4 * j + b)] << (8 * b);
        }
        if (B & 4) {
            const int sh = B & 3, r = rank_in(tm, 1, slot);
            const uint8_t* grp = img + base[1] + (r >> 2) * (D * 2) + (r & 3);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t b0 = grp[4 * (16 * p + 2 * j)], b1 = grp[4 * (16 * p + 2 * j + 1)];
                const uint32_t x = (b0 & 15u) | ((b0 >> 4) << 8) | ((b1 & 15u) << 16) | ((b1 >> 4) << 24);
                creg[j] |= x << sh;
            }
        }
        if (B & 2) {
            const int sh = B & 1, r = rank_in(tm, 2, slot);
            const uint8_t* grp = img + base[2] + (r >> 2) * D + (r & 3);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t b = grp[4 * (8 * p + j)];
                const uint32_t u = b | (b << 12);
                creg[j] |= ((u | (u << 6)) & 0x03030303u) << sh;
            }
        }
        if (B & 1) {
            const int r = rank_in(tm, 3, slot);
            const uint8_t* grp = img + base[3] + (r >> 2) * (D / 2) + (r & 3);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t b = ((uint32_t)grp[4 * (4 * p + j / 2)] >> (4 * (j & 1))) & 15u;
                creg[j] |= (b * 0x00204081u) & 0x01010101u;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------ values, fast writer
// The quantizer builds the values of a tile in two steps so that it never stores single bytes of a word that four
// tokens share.  Step 1 (write_planes_v): every token writes its row of packed w-bit fields (consecutive channels,
// lowest bits first) on its own with vector stores: the item of rank r of section c takes the quarter (r & 3) of
// its group.  Step 2 (group_unit_v): 16 bytes of the final layout, words 4u .. 4u+3 of a group, are the 4x4 byte
// transpose of word u of the group's four rows.
template <int D, typename Ranks>
__device__ __forceinline__ void write_planes_v(uint8_t* img, const Ranks& rk, const uint32_t (&base)[5], int B, int p,
                                               const uint32_t (&creg)[8]) {
    if (B & 8) {
        const int r = rk(0);
        store_words<8>(img + base[0] + (r >> 2) * (D * 4) + (r & 3) * D + 32 * p, creg);
    }
    if (B & 4) {
        const int sh = B & 3, r = rk(1);
        uint32_t y[8], w[4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t x = (creg[j] >> sh) & 0x0F0F0F0Fu;
            y[j] = x | (x >> 4);                     // byte 0: channels 4j, 4j+1; byte 2: channels 4j+2, 4j+3
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) w[m] = prmt(y[2 * m], y[2 * m + 1], 0x6420u);
        store_words<4>(img + base[1] + (r >> 2) * (D * 2) + (r & 3) * (D / 2) + 16 * p, w);
    }
    if (B & 2) {
        const int sh = B & 1, r = rk(2);
        // the four 2-bit fields of a register gathered into one byte by a multiplication: field b (bit 8b + sh) times
        // 2^(24 - 6b - sh) lands at bit 24 + 2b, and no other product of a field and a term reaches the top byte
        const uint32_t msk = 0x03030303u << sh, mul = 0x01041040u >> sh;
        uint32_t t[8], w[2];
#pragma unroll
        for (int j = 0; j < 8; ++j) t[j] = (creg[j] & msk) * mul;
#pragma unroll
        for (int k = 0; k < 2; ++k)
            w[k] = prmt(prmt(t[4 * k], t[4 * k + 1], 0x0073u), prmt(t[4 * k + 2], t[4 * k + 3], 0x0073u), 0x5410u);
        store_words<2>(img + base[2] + (r >> 2) * D + (r & 3) * (D / 4) + 8 * p, w);
    }
    if (B & 1) {
        const int r = rk(3);
        // the low bits of a register's four bytes gathered into a nibble by a multiplication (bit 8b times 2^(24 - 7b)
        // lands at bit 24 + b); odd registers are placed four bits higher, so that a pair fills the top byte
        uint32_t t[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            t[k] = (((creg[2 * k] & 0x01010101u) * 0x01020408u) & 0x0F000000u) | (((creg[2 * k + 1] & 0x01010101u) * 0x10204080u) & 0xF0000000u);
        const uint32_t w = prmt(prmt(t[0], t[1], 0x0073u), prmt(t[2], t[3], 0x0073u), 0x5410u);
        *reinterpret_cast<uint32_t*>(img + base[3] + (r >> 2) * (D / 2) + (r & 3) * (D / 8) + 4 * p) = w;
    }
}

// 16 bytes at offset o (a multiple of 16, QAQ_TILE_HDR <= o < base[4]) of the final layout of a values tile, from
// the rows that write_planes_v left in the image
template <int D, int C>
__device__ __forceinline__ uint4 group_unit_c(const uint8_t* img, uint32_t sec, uint32_t rel) {
    constexpr int W = 8 >> C, GB = D * W / 2;
    const uint32_t G = rel / GB, u = (rel % GB) >> 4;
    const uint8_t* grp = img + sec + G * GB + 4 * u;
    uint32_t in[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) in[i] = *reinterpret_cast<const uint32_t*>(grp + i * (GB / 4));
    const uint32_t t0 = prmt(in[0], in[1], 0x5140u), t1 = prmt(in[2], in[3], 0x5140u);
    const uint32_t t2 = prmt(in[0], in[1], 0x7362u), t3 = prmt(in[2], in[3], 0x7362u);
    return make_uint4(prmt(t0, t1, 0x5410u), prmt(t0, t1, 0x7632u), prmt(t2, t3, 0x5410u), prmt(t2, t3, 0x7632u));
}
template <int D>
__device__ __forceinline__ uint4 group_unit_v(const uint8_t* img, const uint32_t (&base)[5], uint32_t o) {
    if (o >= base[3]) return group_unit_c<D, 3>(img, base[3], o - base[3]);
    if (o >= base[2]) return group_unit_c<D, 2>(img, base[2], o - base[2]);
    if (o >= base[1]) return group_unit_c<D, 1>(img, base[1], o - base[1]);
    return group_unit_c<D, 0>(img, base[0], o - base[0]);
}

// The w-bit piece (w = 8 >> c) of channel d of the item of rank r in section c (for the canonical export).
template <bool IS_V>
__device__ __forceinline__ uint32_t piece_at(const uint8_t* tile, const uint32_t (&base)[5], int D, int c, int r, int d) {
    const int w = 8 >> c, per = 8 / w;
    if (!IS_V) {
        const uint8_t* item = tile + base[c] + (size_t)r * (D * w / 8);
        const int p = d >> 5, j = (d >> 2) & 7, i = d & 3;
        const uint32_t word = *reinterpret_cast<const uint32_t*>(item + 4 * (p * w + j * w / 8));
        return (word >> (8 * i + w * (j & (per - 1)))) & ((1u << w) - 1u);
    } else {
        const uint8_t* grp = tile + base[c] + (size_t)(r >> 2) * (D * w / 2);
        return ((uint32_t)grp[4 * (d / per) + (r & 3)] >> (w * (d & (per - 1)))) & ((1u << w) - 1u);
    }
}

}  // namespace qaqc
