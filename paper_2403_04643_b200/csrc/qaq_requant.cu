// Re-quantization of cached tokens (Section 4.2 of the paper, "Integration in text generation
// process"): in every generation step the widths of all cached tokens are computed again.
//   lower width:  the token is quantized further.  The quantizer is nested (min and range kept,
//                 the B'-bit code is the B-bit code without its low B-B' bits), so this needs
//                 nothing but the packed cache:  code >>= (B - B').
//   higher width: the paper takes the unquantized values from a copy kept in CPU memory and
//                 quantizes them again.  Here the caller passes that copy (any memory the GPU can
//                 read, e.g. mapped pinned host memory: only the rows of the raised tokens are
//                 touched); min, max and the outliers of the token stay what they were, the codes
//                 are computed as at append time.  Without a copy, widths are only lowered.
// The new widths come from the caller or from the rules of Section 4.1 applied to the stored
// range (max - min of the token's metadata) with the current score window and policy scalars.
//
// One CTA = one tile (QAQ_TILE tokens) of one (b,h), both tensors; head_dim/32 lanes own a
// token, each lane the codes of 32 consecutive channels, one byte per code in 8 registers.
// All of a tile's old bytes are in registers before the first new byte is written (the new
// planes are built in a shared-memory image of the tile first), so a tile that does not grow is
// rewritten in place.  A closed tile that grows takes a new place at the end of its pool (the
// old bytes stay unused); the open (last, partly filled) tile is handled in a launch of its own
// after the closed ones and is kept - or made again - the last thing in its pool, so that later
// appends continue right behind it.
#include "qaq_codec.cuh"
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
    // raising widths: the unquantized values [B,H,T,D] (element strides), the thresholds, the tile to start at
    const __half* Ks;
    const __half* Vs;
    long sb, sh, st;
    const float* thr;        // [BH][4]
    int first_tile;
    int* status;
};

using qaqc::ladder;

// Codes of one lane's 32 channels computed from the unquantized row, as at append time:
// code = min(2^B - 1, floor((x - min) * (1/step))) in binary32, 0 for an outlier (outside [lo, hi]).
__device__ __forceinline__ void fresh_codes(const __half* row, float lo, float hi, float mn, float mx, int B, uint32_t (&creg)[8]) {
    uint32_t v[16];
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
        const uint4 raw = *reinterpret_cast<const uint4*>(row + 8 * q4);
        v[4 * q4] = raw.x; v[4 * q4 + 1] = raw.y; v[4 * q4 + 2] = raw.z; v[4 * q4 + 3] = raw.w;
    }
    qaqc::mask_outliers32(v, __half2half2(__float2half_ru(lo)), __half2half2(__float2half_rd(hi)));
    qaqc::codes32(v, mn, mx, B, creg);
}

// UP: widths may be raised (the unquantized copy is there).  Either way a tile whose bytes grow - raised widths,
// or lowered ones that need more padding of the value groups than before - takes a new place at the end of its
// pool; closed tiles are handled by one launch, the open tile by a launch of its own after it.
template <int D, bool UP>
__global__ void __launch_bounds__(2 * D) requant_kernel(const RequantArgs a) {
    constexpr int P = D / 32;
    constexpr int NT = 2 * D;
    constexpr int IMG = qaqc::v_tile_bytes_max(D);
    const int tile = a.first_tile + blockIdx.x, bh = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid / P, p = tid % P;
    const int tok = tile * QAQ_TILE + slot;
    const bool valid = tok < a.T;
    const bool given = a.bitsK != nullptr;

    __shared__ float s_part[P][QAQ_TILE];
    __shared__ uint8_t s_nv[QAQ_TILE];
    __shared__ uint8_t s_bo[2][QAQ_TILE], s_bn[2][QAQ_TILE];      // widths before and after
    __shared__ qaqc::TileMasks s_tmo[2], s_tmn[2];
    __shared__ uint32_t s_tot[2], s_off[2];                        // new bytes of the tile, where they go in the pool
    __shared__ int s_skip[2];
    __shared__ __align__(16) uint8_t s_img[2][IMG];

    // the padding of the value groups has to read as zero
    for (int o = tid; o < IMG / 16; o += NT) reinterpret_cast<uint4*>(s_img[1])[o] = make_uint4(0, 0, 0, 0);

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
    float rng[2] = {0.f, 0.f}, mnf[2] = {0.f, 0.f}, mxf[2] = {0.f, 0.f};
    if (valid) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const TensorStore& ts = x ? a.v : a.k;
            Bo[x] = ts.bits[mt];
            Bo[x] = Bo[x] > 8 ? 8 : Bo[x];
            const uint32_t mm = ts.mnmx[mt];
            mnf[x] = __half2float(__ushort_as_half((unsigned short)(mm & 0xFFFF)));
            mxf[x] = __half2float(__ushort_as_half((unsigned short)(mm >> 16)));
            rng[x] = __fsub_rn(mxf[x], mnf[x]);
        }
    }
    __syncthreads();   // window partials visible

    // ---- new widths: the rule's (or the caller's) width; without the unquantized copy only where it is lower
    int Bn[2];
    bool changed[2];
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        int B = 8;
        if (valid) {
            if (given) {
                B = (x ? a.bitsV : a.bitsK)[(size_t)bh * a.ncols + tok];
                B = B < 1 ? 1 : (B > 8 ? 8 : B);
            } else if (x == 0) {
                B = ladder(rng[0], a.cK, a.bmin, a.bmax);
            } else {
                float sh = __int_as_float(0xff800000);
#pragma unroll
                for (int g = 0; g < P; ++g) sh = fmaxf(sh, s_part[g][slot]);
                B = (s_nv[slot] == 0) ? a.bmax : ladder(__fmul_rn(rng[1], sh), a.cV, a.bmin, a.bmax);
            }
        }
        Bn[x] = !valid ? 0 : ((UP || B < Bo[x]) ? B : Bo[x]);
        if (p == 0) {
            s_bo[x][slot] = (uint8_t)Bo[x];
            s_bn[x][slot] = (uint8_t)Bn[x];
        }
        changed[x] = __syncthreads_or(Bn[x] != Bo[x]) != 0;   // also makes the widths visible
    }
    // An open tile has to be the last thing in its pool.  If closed tiles of this (b,h) have just been moved
    // behind it, it moves to the end as well, whether its own tokens change or not.
    const bool open = tile == a.T / QAQ_TILE && (a.T % QAQ_TILE) != 0;
    bool relocate[2] = {false, false};
    if (open) {
        const size_t ti0 = (size_t)bh * a.ntiles + tile;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const TensorStore& ts = x ? a.v : a.k;
            relocate[x] = ts.tile_off[ti0] + ts.tile_nbytes[ti0] != ts.pool_end[bh];
            changed[x] = changed[x] || relocate[x];
        }
    }
    if (!changed[0] && !changed[1]) return;

    // ---- warp 0: which slots have a piece of each width, before and after; size and place of the new tile
    if (warp == 0) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const uint32_t o0 = s_bo[x][lane], o1 = s_bo[x][lane + 32], n0 = s_bn[x][lane], n1 = s_bn[x][lane + 32];
            qaqc::TileMasks mo, mn_;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mo.m[c] = (unsigned long long)__ballot_sync(0xFFFFFFFFu, (o0 & (8u >> c)) != 0) |
                          ((unsigned long long)__ballot_sync(0xFFFFFFFFu, (o1 & (8u >> c)) != 0) << 32);
                mn_.m[c] = (unsigned long long)__ballot_sync(0xFFFFFFFFu, (n0 & (8u >> c)) != 0) |
                           ((unsigned long long)__ballot_sync(0xFFFFFFFFu, (n1 & (8u >> c)) != 0) << 32);
            }
            if (lane == 0) {
                s_tmo[x] = mo; s_tmn[x] = mn_;
                uint32_t nbase[5];
                if (x == 0) qaqc::section_bases<D, false>(mn_, nbase); else qaqc::section_bases<D, true>(mn_, nbase);
                // where the new tile goes: in place unless it grows
                const TensorStore& ts = x ? a.v : a.k;
                const size_t ti0 = (size_t)bh * a.ntiles + tile;
                const uint32_t nb = nbase[4], off = ts.tile_off[ti0], old_nb = ts.tile_nbytes[ti0];
                const uint32_t old_own = open ? old_nb : ((old_nb + 15u) & ~15u);   // closed tiles own a rounded amount
                uint32_t noff = off;
                int skip = 0;
                if (changed[x] && (nb > old_own || relocate[x])) {
                    if (open && off + old_nb == ts.pool_end[bh]) {
                        // still the last thing in its pool: it grows where it is
                        if ((size_t)off + nb + 16 > a.pool_bytes) skip = 1;
                        else ts.pool_end[bh] = off + nb;
                    } else if (open) {
                        // behind everything else, 16-byte aligned, and exactly as long as its bytes: the last thing
                        // in the pool again (this launch has one CTA per (b,h), nobody else touches the pool)
                        noff = (ts.pool_end[bh] + 15u) & ~15u;
                        if ((size_t)noff + nb + 16 > a.pool_bytes) skip = 1;
                        else ts.pool_end[bh] = noff + nb;
                    } else {
                        // the end of the pool need not be aligned while a tile is open: take 16 bytes more and align;
                        // space that does not fit is given back
                        const uint32_t take = ((nb + 15u) & ~15u) + 16u;
                        const uint32_t at = atomicAdd(&ts.pool_end[bh], take);
                        noff = (at + 15u) & ~15u;
                        if ((size_t)at + take + 16 > a.pool_bytes) { skip = 1; atomicSub(&ts.pool_end[bh], take); }
                    }
                    if (skip) atomicMax(a.status, (int)QAQ_ERR_CAPACITY);
                }
                s_tot[x] = nb; s_off[x] = noff; s_skip[x] = skip;
            }
        }
    }
    __syncthreads();
    // no room in the pool: that tensor's tile stays as it is
    if (s_skip[0]) changed[0] = false;
    if (s_skip[1]) changed[1] = false;

    // ---- old pieces -> codes -> low bits dropped -> new pieces in the shared-memory image
    const size_t ti = (size_t)bh * a.ntiles + tile;
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        if (!changed[x]) continue;
        const TensorStore& ts = x ? a.v : a.k;
        if (tid < 4) qaqc::write_header(s_img[x], s_tmn[x], tid);
        uint32_t creg[8];
        if (valid) {
            if (UP && Bn[x] > Bo[x]) {
                // raised: codes from the unquantized row, with the token's stored min / max and the thresholds
                const __half* row = (x ? a.Vs : a.Ks) + (size_t)(bh / a.H) * a.sb + (size_t)(bh % a.H) * a.sh +
                                    (size_t)tok * a.st + 32 * p;
                fresh_codes(row, a.thr[(size_t)bh * 4 + 2 * x], a.thr[(size_t)bh * 4 + 2 * x + 1], mnf[x], mxf[x], Bn[x], creg);
            } else {
                const uint8_t* src = ts.codes + (size_t)bh * a.pool_bytes + ts.tile_off[ti];
                const qaqc::TileMasks mo = s_tmo[x];
                uint32_t ob[5];
                if (x == 0) { qaqc::section_bases<D, false>(mo, ob); qaqc::read_pieces<D, false>(src, mo, ob, slot, Bo[x], p, creg); }
                else        { qaqc::section_bases<D, true>(mo, ob);  qaqc::read_pieces<D, true>(src, mo, ob, slot, Bo[x], p, creg); }
                const int drop = Bo[x] - Bn[x];
                const uint32_t keep = 0x01010101u * (0xFFu >> drop);
#pragma unroll
                for (int j = 0; j < 8; ++j) creg[j] = (creg[j] >> drop) & keep;
            }
            const qaqc::TileMasks mn_ = s_tmn[x];
            uint32_t nbs[5];
            if (x == 0) { qaqc::section_bases<D, false>(mn_, nbs); qaqc::write_pieces<D, false>(s_img[0], mn_, nbs, slot, Bn[x], p, creg); }
            else        { qaqc::section_bases<D, true>(mn_, nbs);  qaqc::write_pieces<D, true>(s_img[1], mn_, nbs, slot, Bn[x], p, creg); }
        }
    }
    __syncthreads();   // every old byte of the tile has been read, the image is complete

    // ---- the image replaces the tile; widths and tile length follow
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        if (!changed[x]) continue;
        const TensorStore& ts = x ? a.v : a.k;
        const uint32_t off = s_off[x];
        uint8_t* dst = ts.codes + (size_t)bh * a.pool_bytes + off;
        const uint32_t nb = s_tot[x], nb16 = (nb + 15u) & ~15u;
        for (uint32_t o = tid * 16; o < nb16; o += NT * 16)
            *reinterpret_cast<uint4*>(dst + o) = *reinterpret_cast<const uint4*>(s_img[x] + o);
        if (valid && p == 0) ts.bits[mt] = (uint8_t)Bn[x];
        if (tid == 0) {
            // an open tile that is still the last thing in its pool gives back what it no longer needs:
            // appends continue right behind its bytes
            const uint32_t old_off = ts.tile_off[ti], old_nb = ts.tile_nbytes[ti];
            if (open && off == old_off && nb < old_nb && old_off + old_nb == ts.pool_end[bh]) ts.pool_end[bh] = off + nb;
            ts.tile_off[ti] = off;
            ts.tile_nbytes[ti] = nb;
        }
    }
}

template <bool UP>
qaq_status launch_requant(int D, dim3 grid, const RequantArgs& a, cudaStream_t s) {
    switch (D) {
        case 32: requant_kernel<32, UP><<<grid, 64, 0, s>>>(a); break;
        case 64: requant_kernel<64, UP><<<grid, 128, 0, s>>>(a); break;
        case 128: requant_kernel<128, UP><<<grid, 256, 0, s>>>(a); break;
        default: return QAQ_ERR_UNSUPPORTED_SHAPE;
    }
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

// a pointer the GPU can read: device memory, managed memory or mapped (pinned) host memory
const void* device_view(const void* p) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    if (at.type == cudaMemoryTypeUnregistered) return nullptr;   // pageable host memory
    return at.devicePointer;
}

}  // namespace

extern "C" qaq_status qaq_requantize(qaq_cache* c, const void* K_full, const void* V_full, long stride_b, long stride_h,
                                     long stride_t, const float* thr, const uint8_t* bitsK, const uint8_t* bitsV,
                                     const qaq_policy* policy, const float* score_ring, const uint8_t* nvalid,
                                     long n_cols, void* stream) {
    if (!c) return QAQ_ERR_INVALID_ARG;
    if ((bitsK == nullptr) != (bitsV == nullptr)) return QAQ_ERR_INVALID_ARG;
    if (!bitsK && (!policy || !score_ring || !nvalid)) return QAQ_ERR_INVALID_ARG;
    if ((K_full == nullptr) != (V_full == nullptr)) return QAQ_ERR_INVALID_ARG;
    const bool up = K_full != nullptr;
    if (c->tokens == 0) return QAQ_OK;
    if (n_cols < c->tokens) return QAQ_ERR_INVALID_ARG;
    RequantArgs a{};
    a.k = c->t[0]; a.v = c->t[1]; a.pool_bytes = c->pool_bytes; a.tmax_pad = c->tmax_pad; a.ntiles = c->ntiles;
    a.H = c->cfg.heads; a.T = (int)c->tokens; a.ncols = n_cols;
    a.bitsK = bitsK; a.bitsV = bitsV; a.ring = score_ring; a.nvalid = nvalid; a.W = c->cfg.window;
    a.cK = policy ? policy->cK : 0.f; a.cV = policy ? policy->cV : 0.f;
    a.bmin = c->cfg.bits_min; a.bmax = c->cfg.bits_max;
    a.status = c->d_status;
    cudaStream_t s = (cudaStream_t)stream;
    const int D = c->cfg.head_dim;
    const int ntile = (int)((c->tokens + QAQ_TILE - 1) / QAQ_TILE);
    if (up) {
        if (!thr) return QAQ_ERR_INVALID_ARG;
        if (stride_t < D || (stride_b & 7) || (stride_h & 7) || (stride_t & 7) || stride_b < 0 || stride_h < 0) return QAQ_ERR_INVALID_ARG;
        a.Ks = (const __half*)device_view(K_full); a.Vs = (const __half*)device_view(V_full);
        if (!a.Ks || !a.Vs || ((uintptr_t)a.Ks & 15) || ((uintptr_t)a.Vs & 15)) return QAQ_ERR_INVALID_ARG;
        a.sb = stride_b; a.sh = stride_h; a.st = stride_t; a.thr = thr;
    }
    // closed tiles first (a tile that grows moves to the end of its pool), then the open tile, which has to be
    // the last thing in its pool when this call is over
    const int closed = (int)(c->tokens / QAQ_TILE);
    qaq_status st = QAQ_OK;
    if (closed > 0) {
        a.first_tile = 0;
        const dim3 grid((unsigned)closed, (unsigned)c->BH);
        if ((st = up ? launch_requant<true>(D, grid, a, s) : launch_requant<false>(D, grid, a, s)) != QAQ_OK) return st;
    }
    if (closed < ntile) {
        a.first_tile = closed;
        const dim3 grid(1, (unsigned)c->BH);
        st = up ? launch_requant<true>(D, grid, a, s) : launch_requant<false>(D, grid, a, s);
    }
    return st;
}

extern "C" qaq_status qaq_requantize_down(qaq_cache* c, const uint8_t* bitsK, const uint8_t* bitsV,
                                          const qaq_policy* policy, const float* score_ring, const uint8_t* nvalid,
                                          long n_cols, void* stream) {
    return qaq_requantize(c, nullptr, nullptr, 0, 0, 0, nullptr, bitsK, bitsV, policy, score_ring, nvalid, n_cols, stream);
}

// ---------------------------------------------------------------------------------------
// Compaction of the code pools.  Tiles that grew in qaq_requantize were placed anew at the end
// of their pool and left their old bytes behind; this closes the gaps again: the tiles of a
// (b,h) pool are moved down, in the order in which they lie in memory, until they are
// contiguous (16-byte aligned each), the open tile last.  One CTA per (b,h) and tensor works
// through its tiles one after the other; a tile is copied forward in 4 KB pieces, every piece
// read completely before it is written, so that overlapping source and destination are safe.
namespace {

constexpr int COMPACT_MAX_TILES = 4096;

struct CompactArgs {
    TensorStore t[2];
    size_t pool_bytes;
    int ntiles, T;
};

__global__ void __launch_bounds__(256) compact_kernel(const CompactArgs a) {
    const int bh = blockIdx.x;
    const TensorStore& ts = a.t[blockIdx.y];
    __shared__ unsigned long long s_key[COMPACT_MAX_TILES];   // current offset << 32 | tile index
    const int nt = (a.T + QAQ_TILE - 1) / QAQ_TILE;
    int n2 = 1;
    while (n2 < nt) n2 <<= 1;
    const size_t row = (size_t)bh * a.ntiles;
    for (int i = threadIdx.x; i < n2; i += blockDim.x)
        s_key[i] = i < nt ? ((unsigned long long)ts.tile_off[row + i] << 32) | (unsigned)i : ~0ull;
    __syncthreads();
    // bitonic sort by current offset
    for (int k = 2; k <= n2; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < n2; i += blockDim.x) {
                const int l = i ^ j;
                if (l > i) {
                    const unsigned long long x = s_key[i], y = s_key[l];
                    const bool up = (i & k) == 0;
                    if ((x > y) == up) { s_key[i] = y; s_key[l] = x; }
                }
            }
            __syncthreads();
        }
    uint8_t* pool = ts.codes + (size_t)bh * a.pool_bytes;
    uint32_t dst = 0;
    for (int s = 0; s < nt; ++s) {
        const uint32_t src = (uint32_t)(s_key[s] >> 32);
        const int tile = (int)(s_key[s] & 0xFFFFFFFFu);
        const uint32_t n = ts.tile_nbytes[row + tile];
        const uint32_t n16 = (n + 15u) & ~15u;
        if (src != dst) {                                  // dst < src: tiles before this one only moved down
            for (uint32_t o = 0; o < n16; o += 256 * 16) {
                const uint32_t b = o + threadIdx.x * 16;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (b < n16) v = *reinterpret_cast<const uint4*>(pool + src + b);
                __syncthreads();
                if (b < n16) *reinterpret_cast<uint4*>(pool + dst + b) = v;
            }
            if (threadIdx.x == 0) ts.tile_off[row + tile] = dst;
        }
        // closed tiles own a 16-byte rounded amount; the open tile, which is the last one, its exact bytes
        const bool open = tile == a.T / QAQ_TILE && (a.T % QAQ_TILE) != 0;
        dst += open ? n : n16;
        __syncthreads();                                   // the next tile's source may be this tile's old place
    }
    if (threadIdx.x == 0) ts.pool_end[bh] = dst;
}

__global__ void pool_use_kernel(TensorStore tk, TensorStore tv, int BH, unsigned int* out) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < BH; i += gridDim.x * blockDim.x) {
        atomicMax(&out[0], tk.pool_end[i]);
        atomicMax(&out[1], tv.pool_end[i]);
    }
}

}  // namespace

extern "C" qaq_status qaq_cache_compact(qaq_cache* c, void* stream) {
    if (!c) return QAQ_ERR_INVALID_ARG;
    if (c->tokens == 0) return QAQ_OK;
    const long nt = (c->tokens + QAQ_TILE - 1) / QAQ_TILE;
    if (nt > COMPACT_MAX_TILES) return QAQ_ERR_UNSUPPORTED_SHAPE;
    CompactArgs a;
    a.t[0] = c->t[0]; a.t[1] = c->t[1]; a.pool_bytes = c->pool_bytes; a.ntiles = c->ntiles; a.T = (int)c->tokens;
    compact_kernel<<<dim3((unsigned)c->BH, 2), 256, 0, (cudaStream_t)stream>>>(a);
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

extern "C" qaq_status qaq_cache_pool_use(const qaq_cache* c, long* host_used, long* host_capacity, void* stream) {
    if (!c || !host_used) return QAQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    unsigned int* d = (unsigned int*)c->d_status + 2;      // two spare words behind the status word
    QAQ_CUDA_TRY(cudaMemsetAsync(d, 0, 8, s));
    pool_use_kernel<<<32, 256, 0, s>>>(c->t[0], c->t[1], c->BH, d);
    QAQ_CUDA_TRY(cudaGetLastError());
    unsigned int h[2] = {0, 0};
    QAQ_CUDA_TRY(cudaMemcpyAsync(h, d, 8, cudaMemcpyDeviceToHost, s));
    QAQ_CUDA_TRY(cudaStreamSynchronize(s));
    host_used[0] = (long)h[0]; host_used[1] = (long)h[1];
    if (host_capacity) *host_capacity = (long)c->pool_bytes;
    return QAQ_OK;
}
