// Further quantization of cached tokens to lower widths (Section 4.2 of the paper,
// "Integration in text generation process"): in every generation step the widths of all
// cached tokens are computed again; a token whose new width is lower than its current one is
// quantized further.  The quantizer is nested (min and range kept, the B'-bit code is the
// B-bit code without its low B-B' bits), so this needs nothing but the packed cache itself:
//   range = max - min from the token's metadata  ->  new width by the rules of Section 4.1
//   code >>= (B - B'),  planes rebuilt for B',  the tile rewritten in place (it only shrinks).
// Widths are never raised here (that needs the unquantized copy the paper keeps in CPU memory).
//
// One CTA = one tile (QAQ_TILE tokens) of one (b,h), both tensors; head_dim/32 lanes own a
// token, each lane the codes of 32 consecutive channels, one byte per code in 8 registers.
// All of a tile's old bytes are in registers before the first new byte is written (the new
// planes are built in a shared-memory image of the tile first), so rewriting in place is safe.
// Pool space freed inside closed tiles is not handed back; an open (last, partly filled) tile
// gives its bytes back to the pool so that later appends continue right behind it.
#include "qaq_internal.cuh"

namespace {

struct RequantArgs {
    TensorStore k, v;
    size_t pool_bytes;
    int tmax_pad, ntiles;
    int H, T;                // heads; cached tokens
    long ncols;              // row length of bitsK/bitsV/ring/nvalid (>= T)
    const uint8_t* bitsK;    // requested widths [BH][ncols] or null
    const uint8_t* bitsV;
    const float* ring;       // [BH][W][ncols]
    const uint8_t* nvalid;   // [BH][ncols]
    int W;
    float cK, cV;
    int bmin, bmax;
};

// B = min{b in [bmin,bmax] : v <= c * 2^b}, bmax if none (c * 2^b is an exact scaling)
__device__ __forceinline__ int ladder(float v, float c, int bmin, int bmax) {
    if (!(c > 0.f)) return bmax;
    for (int b = bmin; b <= bmax; ++b)
        if (v <= __fmul_rn(c, (float)(1 << b))) return b;
    return bmax;
}

// NW words from / to an address that is ALIGN-byte aligned (ALIGN in {4, 8, 16})
template <int NW, int ALIGN>
__device__ __forceinline__ void load_words(const uint8_t* __restrict__ p, uint32_t* w) {
    if (ALIGN == 16 && NW % 4 == 0) {
#pragma unroll
        for (int i = 0; i < NW; i += 4) {
            const uint4 v = *reinterpret_cast<const uint4*>(p + 4 * i);
            w[i] = v.x; w[i + 1] = v.y; w[i + 2] = v.z; w[i + 3] = v.w;
        }
    } else if (ALIGN >= 8 && NW % 2 == 0) {
#pragma unroll
        for (int i = 0; i < NW; i += 2) {
            const uint2 v = *reinterpret_cast<const uint2*>(p + 4 * i);
            w[i] = v.x; w[i + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < NW; ++i) w[i] = *reinterpret_cast<const uint32_t*>(p + 4 * i);
    }
}
template <int NW, int ALIGN>
__device__ __forceinline__ void store_words(uint8_t* p, const uint32_t* w) {
    if (ALIGN == 16 && NW % 4 == 0) {
#pragma unroll
        for (int i = 0; i < NW; i += 4) *reinterpret_cast<uint4*>(p + 4 * i) = make_uint4(w[i], w[i + 1], w[i + 2], w[i + 3]);
    } else if (ALIGN >= 8 && NW % 2 == 0) {
#pragma unroll
        for (int i = 0; i < NW; i += 2) *reinterpret_cast<uint2*>(p + 4 * i) = make_uint2(w[i], w[i + 1]);
    } else {
#pragma unroll
        for (int i = 0; i < NW; ++i) *reinterpret_cast<uint32_t*>(p + 4 * i) = w[i];
    }
}

// A token's bytes are the planes of the power-of-two pieces of its width, widest first, each
// holding the next lower bits of the codes; a lane's 32 channels of a w-bit plane are w words at
// plane + p * 4w.  creg[j] holds the codes of channels 4j..4j+3, one per byte.
template <int D, int ALIGN>
__device__ __forceinline__ void read_planes(const uint8_t* tok, int B, int p, uint32_t (&creg)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) creg[j] = 0;
    if (B & 8) load_words<8, ALIGN>(tok + p * 32, creg);
    if (B & 4) {
        const int sh = B & 3;
        uint32_t w[4];
        load_words<4, ALIGN>(tok + (B & 8) * (D / 8) + p * 16, w);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            creg[2 * j] |= (w[j] & 0x0F0F0F0Fu) << sh;
            creg[2 * j + 1] |= ((w[j] >> 4) & 0x0F0F0F0Fu) << sh;
        }
    }
    if (B & 2) {
        const int sh = B & 1;
        uint32_t w[2];
        load_words<2, (ALIGN > 8 ? 8 : ALIGN)>(tok + (B & 12) * (D / 8) + p * 8, w);
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int m = 0; m < 4; ++m) creg[4 * j + m] |= ((w[j] >> (2 * m)) & 0x03030303u) << sh;
    }
    if (B & 1) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(tok + (B & 14) * (D / 8) + p * 4);
#pragma unroll
        for (int m = 0; m < 8; ++m) creg[m] |= (w >> m) & 0x01010101u;
    }
}
template <int D, int ALIGN>
__device__ __forceinline__ void write_planes(uint8_t* tok, int B, int p, const uint32_t (&creg)[8]) {
    if (B & 8) store_words<8, ALIGN>(tok + p * 32, creg);
    if (B & 4) {
        const int sh = B & 3;
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            w[j] = ((creg[2 * j] >> sh) & 0x0F0F0F0Fu) | (((creg[2 * j + 1] >> sh) & 0x0F0F0F0Fu) << 4);
        store_words<4, ALIGN>(tok + (B & 8) * (D / 8) + p * 16, w);
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
        store_words<2, (ALIGN > 8 ? 8 : ALIGN)>(tok + (B & 12) * (D / 8) + p * 8, w);
    }
    if (B & 1) {
        uint32_t acc = 0;
#pragma unroll
        for (int m = 0; m < 8; ++m) acc |= (creg[m] & 0x01010101u) << m;
        *reinterpret_cast<uint32_t*>(tok + (B & 14) * (D / 8) + p * 4) = acc;
    }
}

template <int D>
__global__ void __launch_bounds__(2 * D) requant_kernel(const RequantArgs a) {
    constexpr int P = D / 32;
    constexpr int ALIGN = D / 8 >= 16 ? 16 : D / 8;
    constexpr int NT = 2 * D;
    const int tile = blockIdx.x, bh = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid / P, p = tid % P;
    const int tok = tile * QAQ_TILE + slot;
    const bool valid = tok < a.T;
    const bool given = a.bitsK != nullptr;

    __shared__ float s_part[P][QAQ_TILE];
    __shared__ uint8_t s_nv[QAQ_TILE];
    __shared__ uint32_t s_old[2][QAQ_TILE], s_new[2][QAQ_TILE];   // byte lengths, then exclusive offsets in the tile
    __shared__ uint32_t s_tot[2];                                  // new bytes of the tile
    __shared__ __align__(16) uint8_t s_img[2][QAQ_TILE * D];

    // ---- attention window of the tile's tokens (value rule); P threads share a token's rows
    {
        const int g = tid / QAQ_TILE, tk = tid % QAQ_TILE;
        const int t2 = tile * QAQ_TILE + tk;
        float m = __int_as_float(0xff800000);
        int nv = 0;
        if (!given && t2 < a.T) {
            nv = a.nvalid[(size_t)bh * a.ncols + t2];
            nv = nv < a.W ? nv : a.W;
            const float* r = a.ring + (size_t)bh * a.W * a.ncols + t2;
            for (int i = g; i < nv; i += P) m = fmaxf(m, r[(size_t)i * a.ncols]);
        }
        s_part[g][tk] = m;
        if (g == 0) s_nv[tk] = (uint8_t)nv;
    }
    // ---- current widths and ranges
    const size_t mt = (size_t)bh * a.tmax_pad + tok;
    int Bo[2] = {0, 0};
    float rng[2] = {0.f, 0.f};
    if (valid) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const TensorStore& ts = x ? a.v : a.k;
            Bo[x] = ts.bits[mt];
            const uint32_t mm = ts.mnmx[mt];
            const float mn = __half2float(__ushort_as_half((unsigned short)(mm & 0xFFFF)));
            const float mx = __half2float(__ushort_as_half((unsigned short)(mm >> 16)));
            rng[x] = __fsub_rn(mx, mn);
        }
    }
    __syncthreads();   // window partials visible

    // ---- new widths: the rule's (or the caller's) width where it is lower, else the current one
    int Bn[2];
    bool changed[2];
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        int B = 8;
        if (valid) {
            if (given) {
                B = (x ? a.bitsV : a.bitsK)[(size_t)bh * a.ncols + tok];
                B = B < 1 ? 1 : B;
            } else if (x == 0) {
                B = ladder(rng[0], a.cK, a.bmin, a.bmax);
            } else {
                float sh = __int_as_float(0xff800000);
#pragma unroll
                for (int g = 0; g < P; ++g) sh = fmaxf(sh, s_part[g][slot]);
                B = (s_nv[slot] == 0) ? a.bmax : ladder(__fmul_rn(rng[1], sh), a.cV, a.bmin, a.bmax);
            }
        }
        Bn[x] = B < Bo[x] ? B : Bo[x];
        if (p == 0) {
            s_old[x][slot] = (uint32_t)(D * Bo[x] / 8);
            s_new[x][slot] = (uint32_t)(D * Bn[x] / 8);
        }
        changed[x] = __syncthreads_or(Bn[x] != Bo[x]) != 0;   // also makes the lengths visible
    }
    if (!changed[0] && !changed[1]) return;

    // ---- warp 0: exclusive offsets of the tokens inside the tile, before and after
    if (warp == 0) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            uint32_t o0 = s_old[x][lane], o1 = s_old[x][lane + 32], n0 = s_new[x][lane], n1 = s_new[x][lane + 32];
            uint32_t io0 = o0, io1 = o1, in0 = n0, in1 = n1;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t a0 = __shfl_up_sync(0xFFFFFFFFu, io0, d), a1 = __shfl_up_sync(0xFFFFFFFFu, io1, d);
                const uint32_t b0 = __shfl_up_sync(0xFFFFFFFFu, in0, d), b1 = __shfl_up_sync(0xFFFFFFFFu, in1, d);
                if (lane >= d) { io0 += a0; io1 += a1; in0 += b0; in1 += b1; }
            }
            const uint32_t to0 = __shfl_sync(0xFFFFFFFFu, io0, 31), tn0 = __shfl_sync(0xFFFFFFFFu, in0, 31);
            const uint32_t tn1 = __shfl_sync(0xFFFFFFFFu, in1, 31);
            s_old[x][lane] = io0 - o0; s_old[x][lane + 32] = to0 + io1 - o1;
            s_new[x][lane] = in0 - n0; s_new[x][lane + 32] = tn0 + in1 - n1;
            if (lane == 0) s_tot[x] = tn0 + tn1;
        }
    }
    __syncthreads();

    // ---- old planes -> codes -> low bits dropped -> new planes in the shared-memory image
    const size_t ti = (size_t)bh * a.ntiles + tile;
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        if (!changed[x]) continue;
        const TensorStore& ts = x ? a.v : a.k;
        uint32_t creg[8];
        if (valid) {
            const uint8_t* src = ts.codes + (size_t)bh * a.pool_bytes + ts.tile_off[ti] + s_old[x][slot];
            read_planes<D, ALIGN>(src, Bo[x], p, creg);
            const int drop = Bo[x] - Bn[x];
            const uint32_t keep = 0x01010101u * (0xFFu >> drop);
#pragma unroll
            for (int j = 0; j < 8; ++j) creg[j] = (creg[j] >> drop) & keep;
            write_planes<D, ALIGN>(s_img[x] + s_new[x][slot], Bn[x], p, creg);
        }
    }
    __syncthreads();   // every old byte of the tile has been read, the image is complete

    // ---- the image replaces the tile; widths and tile length follow
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        if (!changed[x]) continue;
        const TensorStore& ts = x ? a.v : a.k;
        const uint32_t off = ts.tile_off[ti];
        uint8_t* dst = ts.codes + (size_t)bh * a.pool_bytes + off;
        const uint32_t nb = s_tot[x];
        for (uint32_t o = tid * ALIGN; o < nb; o += NT * ALIGN) {
            if (ALIGN == 16) *reinterpret_cast<uint4*>(dst + o) = *reinterpret_cast<const uint4*>(s_img[x] + o);
            else if (ALIGN == 8) *reinterpret_cast<uint2*>(dst + o) = *reinterpret_cast<const uint2*>(s_img[x] + o);
            else *reinterpret_cast<uint32_t*>(dst + o) = *reinterpret_cast<const uint32_t*>(s_img[x] + o);
        }
        if (valid && p == 0) ts.bits[mt] = (uint8_t)Bn[x];
        if (tid == 0) {
            ts.tile_nbytes[ti] = nb;
            // an open tile is the last thing in its pool: appends continue right behind its bytes
            if (tile == a.T / QAQ_TILE && (a.T % QAQ_TILE) != 0) ts.pool_end[bh] = off + nb;
        }
    }
}

}  // namespace

extern "C" qaq_status qaq_requantize_down(qaq_cache* c, const uint8_t* bitsK, const uint8_t* bitsV,
                                          const qaq_policy* policy, const float* score_ring, const uint8_t* nvalid,
                                          long n_cols, void* stream) {
    if (!c) return QAQ_ERR_INVALID_ARG;
    if ((bitsK == nullptr) != (bitsV == nullptr)) return QAQ_ERR_INVALID_ARG;
    if (!bitsK && (!policy || !score_ring || !nvalid)) return QAQ_ERR_INVALID_ARG;
    if (c->tokens == 0) return QAQ_OK;
    if (n_cols < c->tokens) return QAQ_ERR_INVALID_ARG;
    RequantArgs a{};
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.tmax_pad = c->tmax_pad; a.ntiles = c->ntiles;
    a.H = c->cfg.heads; a.T = (int)c->tokens; a.ncols = n_cols;
    a.bitsK = bitsK; a.bitsV = bitsV; a.ring = score_ring; a.nvalid = nvalid; a.W = c->cfg.window;
    a.cK = policy ? policy->cK : 0.f; a.cV = policy ? policy->cV : 0.f;
    a.bmin = c->cfg.bits_min; a.bmax = c->cfg.bits_max;
    const dim3 grid((unsigned)((c->tokens + QAQ_TILE - 1) / QAQ_TILE), (unsigned)c->BH);
    cudaStream_t s = (cudaStream_t)stream;
    switch (c->cfg.head_dim) {
        case 32: requant_kernel<32><<<grid, 64, 0, s>>>(a); break;
        case 64: requant_kernel<64><<<grid, 128, 0, s>>>(a); break;
        case 128: requant_kernel<128><<<grid, 256, 0, s>>>(a); break;
        default: return QAQ_ERR_UNSUPPORTED_SHAPE;
    }
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}
