// S1-S3: bit-width selection, outlier split, uniform quantization and bit-packing.
//
// One CTA handles one tile (QAQ_TILE consecutive tokens) of one (b,h); a group of
// head_dim/4 lanes owns one token (4 channels per lane, held in registers from the
// min/max pass to the packing pass, so K and V are read from HBM exactly once).
//   phase 0  thread per token: attention-window maximum of the score rows (Section 4.2)
//   phase 1  group per token: outlier flags, min/max of the non-outliers (shuffle
//            reductions), width ladder (Section 4.1), outlier count (ballot/popc)
//   phase 2  warp 0: exclusive scans of byte lengths and outlier counts over the tile,
//            space taken from the (b,h) pools by atomicAdd
//   phase 3  group per token: codes, plane packing, stores; outlier compaction
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

__device__ __forceinline__ int ladder(float v, float c, int bmin, int bmax) {
    // B = min{b : v <= c * 2^b}; c * 2^b is exact (power-of-two scaling)
    if (!(c > 0.f)) return bmax;
    for (int b = bmin; b <= bmax; ++b)
        if (v <= __fmul_rn(c, (float)(1 << b))) return b;
    return bmax;
}

template <int D, bool SELECT_ONLY>
__global__ void __launch_bounds__(256) quant_kernel(const QuantArgs a) {
    constexpr int G = D / 4;         // lanes per token
    constexpr int TPW = 32 / G;      // tokens handled concurrently by a warp
    constexpr int NI = 8 / TPW;      // iterations: 8 token slots per warp
    const int bh = blockIdx.y;
    const int tile = a.first_tile + blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane % G, sub = lane / G;
    const unsigned gmask = (G == 32) ? 0xFFFFFFFFu : (((1u << G) - 1u) << (sub * G));
    const unsigned lt_in_group = gmask & ((1u << lane) - 1u);

    // new-token index range of this tile
    const int abs_lo = max(tile * QAQ_TILE, a.t_old + a.tok_lo);
    const int abs_hi = min((tile + 1) * QAQ_TILE, a.t_old + a.tok_hi);
    const int s_lo = abs_lo - tile * QAQ_TILE, s_hi = abs_hi - tile * QAQ_TILE;  // slots in the tile

    __shared__ float s_shat[QAQ_TILE];
    __shared__ uint8_t s_bits[2][QAQ_TILE];
    __shared__ float s_mn[2][QAQ_TILE], s_mx[2][QAQ_TILE];
    __shared__ uint32_t s_len[2][QAQ_TILE];   // bytes, then exclusive byte offsets
    __shared__ uint32_t s_cnt[2][QAQ_TILE];   // outlier counts, then exclusive offsets
    __shared__ uint32_t s_base[2], s_obase[2], s_olimit[2];
    __shared__ int s_skip;

    const float* thr = a.thr + (size_t)bh * 4;
    const float loK = thr[0], hiK = thr[1], loV = thr[2], hiV = thr[3];
    const bool given = a.bitsK != nullptr;

    // ---- phase 0: attention window (max of the valid score rows of each token)
    if (threadIdx.x < QAQ_TILE) {
        const int slot = threadIdx.x;
        float m = __int_as_float(0x7f800000);  // +inf: no score seen
        if (!given && slot >= s_lo && slot < s_hi) {
            const int tn = tile * QAQ_TILE + slot - a.t_old;
            int nv = a.nvalid[(size_t)bh * a.n_new + tn];
            nv = nv < a.W ? nv : a.W;
            if (nv > 0) {
                const float* r = a.ring + (size_t)bh * a.W * a.n_new + tn;
                m = r[0];
                for (int i = 1; i < nv; ++i) m = fmaxf(m, r[(size_t)i * a.n_new]);
            }
        }
        s_shat[slot] = m;
        s_len[0][slot] = 0; s_len[1][slot] = 0; s_cnt[0][slot] = 0; s_cnt[1][slot] = 0;
        s_bits[0][slot] = 0; s_bits[1][slot] = 0;
    }
    __syncthreads();

    // ---- phase 1: load, outlier flags, masked range, widths
    const int b_idx = bh / a.H, h_idx = bh % a.H;
    const __half* Kb = a.K + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh;
    const __half* Vb = a.V + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh;
    uint2 rawK[NI], rawV[NI];
#pragma unroll
    for (int j = 0; j < NI; ++j) {
        const int slot = warp * 8 + j * TPW + sub;
        const bool valid = slot >= s_lo && slot < s_hi;
        rawK[j] = make_uint2(0, 0); rawV[j] = make_uint2(0, 0);
        if (valid) {
            const size_t tn = (size_t)(tile * QAQ_TILE + slot - a.t_old);
            rawK[j] = *reinterpret_cast<const uint2*>(Kb + tn * a.st + 4 * g);
            rawV[j] = *reinterpret_cast<const uint2*>(Vb + tn * a.st + 4 * g);
        }
    }
#pragma unroll
    for (int j = 0; j < NI; ++j) {
        const int slot = warp * 8 + j * TPW + sub;
        const bool valid = slot >= s_lo && slot < s_hi;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const uint2 raw = x ? rawV[j] : rawK[j];
            const float lo = x ? loV : loK, hi = x ? hiV : hiK;
            const float2 f01 = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
            const float2 f23 = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
            const float xv[4] = {f01.x, f01.y, f23.x, f23.y};
            float mn = __int_as_float(0x7f800000), mx = __int_as_float(0xff800000);
            unsigned cnt = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const bool o = !(lo <= xv[i] && xv[i] <= hi);
                if (!o) { mn = fminf(mn, xv[i]); mx = fmaxf(mx, xv[i]); }
                cnt += __popc(__ballot_sync(0xFFFFFFFFu, o && valid) & gmask);
            }
#pragma unroll
            for (int d = 1; d < G; d <<= 1) {
                mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, d));
                mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, d));
            }
            if (mn > mx) { mn = 0.f; mx = 0.f; }  // no non-outlier entry
            int B;
            if (given) {
                B = valid ? (x ? a.bitsV : a.bitsK)[(size_t)bh * a.n_new + (tile * QAQ_TILE + slot - a.t_old)] : 0;
            } else {
                const float r = __fsub_rn(mx, mn);
                if (x == 0) {
                    B = ladder(r, a.cK, a.bmin, a.bmax);
                } else {
                    const float sh = s_shat[slot & (QAQ_TILE - 1)];
                    B = isinf(sh) ? a.bmax : ladder(__fmul_rn(r, sh), a.cV, a.bmin, a.bmax);
                }
            }
            if (valid && g == 0) {
                s_bits[x][slot] = (uint8_t)B;
                s_mn[x][slot] = mn; s_mx[x][slot] = mx;
                s_len[x][slot] = (uint32_t)(D * B / 8);
                s_cnt[x][slot] = cnt;
                if (SELECT_ONLY) (x ? a.out_bitsV : a.out_bitsK)[(size_t)bh * a.n_new + (tile * QAQ_TILE + slot - a.t_old)] = (uint8_t)B;
            }
        }
    }
    if (SELECT_ONLY) return;
    __syncthreads();

    // ---- phase 2: scans over the tile and pool allocation
    if (warp == 0) {
        const bool starts = (s_lo == 0), closes = (s_hi == QAQ_TILE), whole = starts && closes;
        if (lane == 0) s_skip = 0;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const TensorStore& ts = x ? a.v : a.k;
            // two slots per lane: (lane, lane + 32)
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
            if (lane == 0) {
                const uint32_t bytes = tot0 + tot1, cnt = ctot0 + ctot1;
                const size_t ti = (size_t)bh * a.ntiles + tile;
                // packed codes
                uint32_t base;
                if (whole) {
                    base = atomicAdd(&ts.pool_end[bh], (bytes + 15u) & ~15u);
                } else {
                    base = atomicAdd(&ts.pool_end[bh], bytes);
                    if (closes) {
                        const uint32_t pad = (0u - (base + bytes)) & 15u;
                        if (pad) atomicAdd(&ts.pool_end[bh], pad);
                    }
                }
                if ((size_t)base + bytes + 16 > a.pool_bytes) { atomicMax(a.status, (int)QAQ_ERR_CAPACITY); s_skip = 1; }
                if (starts) { ts.tile_off[ti] = base; ts.tile_nbytes[ti] = bytes; }
                else ts.tile_nbytes[ti] += bytes;
                s_base[x] = base;
                // outliers
                uint32_t obase;
                if (whole) {
                    obase = atomicAdd(&ts.opool_end[bh], (cnt + 3u) & ~3u);
                } else {
                    obase = atomicAdd(&ts.opool_end[bh], cnt);
                    if (closes) {
                        const uint32_t pad = (0u - (obase + cnt)) & 3u;
                        if (pad) atomicAdd(&ts.opool_end[bh], pad);
                    }
                }
                const uint32_t room = obase + 8 < a.ocap ? a.ocap - 8 - obase : 0;  // 8 entries of read-ahead margin
                const uint32_t stored = cnt < room ? cnt : room;
                if (stored < cnt) atomicMax(a.status, (int)QAQ_ERR_CAPACITY);
                if (starts) { ts.tile_ooff[ti] = obase; ts.tile_ocnt[ti] = stored; }
                else ts.tile_ocnt[ti] += stored;
                s_obase[x] = obase;
                s_olimit[x] = obase + stored;
            }
        }
    }
    __syncthreads();
    if (s_skip) return;

    // ---- phase 3: codes, planes, stores
    const int p = g >> 3, r = g & 7;
#pragma unroll
    for (int j = 0; j < NI; ++j) {
        const int slot = warp * 8 + j * TPW + sub;
        const bool valid = slot >= s_lo && slot < s_hi;
        const int sl = slot & (QAQ_TILE - 1);
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const TensorStore& ts = x ? a.v : a.k;
            const uint2 raw = x ? rawV[j] : rawK[j];
            const float lo = x ? loV : loK, hi = x ? hiV : hiK;
            const float2 f01 = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
            const float2 f23 = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
            const float xv[4] = {f01.x, f01.y, f23.x, f23.y};
            const unsigned short hv[4] = {(unsigned short)(raw.x & 0xFFFF), (unsigned short)(raw.x >> 16),
                                          (unsigned short)(raw.y & 0xFFFF), (unsigned short)(raw.y >> 16)};
            const int B = valid ? s_bits[x][sl] : 0;
            const float mn = valid ? s_mn[x][sl] : 0.f, mx = valid ? s_mx[x][sl] : 0.f;
            const float step = __fmul_rn(__fsub_rn(mx, mn), __int_as_float((127 - B) << 23));
            const float inv = step > 0.f ? __fdiv_rn(1.0f, step) : 0.f;
            const int top = (1 << B) - 1;
            uint32_t reg = 0;
            bool o[4];
            unsigned bal[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                o[i] = !(lo <= xv[i] && xv[i] <= hi);
                int c = 0;
                if (!o[i]) {
                    c = __float2int_rd(__fmul_rn(__fsub_rn(xv[i], mn), inv));
                    c = c > top ? top : c;
                    c = c < 0 ? 0 : c;
                }
                reg |= (uint32_t)c << (8 * i);
                bal[i] = __ballot_sync(0xFFFFFFFFu, o[i] && valid);
            }
            // planes, widest first
            uint8_t* tok = ts.codes + (size_t)bh * a.pool_bytes + s_base[x] + s_len[x][sl];
#pragma unroll
            for (int w = 8; w >= 1; w >>= 1) {
                const int per = 8 / w;                 // slots per byte lane
                const int m = r & (per - 1);
                const int shift = B & (w - 1);
                uint32_t word = ((reg >> shift) & (0x01010101u * ((1u << w) - 1u))) << (w * m);
#pragma unroll
                for (int d = 1; d < per; d <<= 1) word |= __shfl_xor_sync(0xFFFFFFFFu, word, d);
                if (valid && (B & w) && m == 0) {
                    const int plane_base = (B & ~((w << 1) - 1)) * (D / 8);
                    *reinterpret_cast<uint32_t*>(tok + plane_base + 4 * (p * w + ((r * w) >> 3))) = word;
                }
            }
            // outliers in (token, channel) order
            uint32_t before = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) before += __popc(bal[i] & lt_in_group);
            uint32_t pos = s_obase[x] + s_cnt[x][sl] + before;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (o[i] && valid) {
                    if (pos < s_olimit[x])
                        ts.outl[(size_t)bh * a.ocap + pos] = (uint32_t)hv[i] | ((uint32_t)(4 * g + i) << 16) | ((uint32_t)sl << 24);
                    ++pos;
                }
            }
            if (valid && g == 0) {
                const size_t t = (size_t)bh * a.tmax_pad + (size_t)tile * QAQ_TILE + sl;
                ts.bits[t] = (uint8_t)B;
                ts.mnmx[t] = (uint32_t)__half_as_ushort(__float2half_rn(mn)) |
                             ((uint32_t)__half_as_ushort(__float2half_rn(mx)) << 16);
            }
        }
    }
}

template <bool SELECT_ONLY>
qaq_status launch(int D, dim3 grid, const QuantArgs& a, cudaStream_t s) {
    switch (D) {
        case 32: quant_kernel<32, SELECT_ONLY><<<grid, 256, 0, s>>>(a); break;
        case 64: quant_kernel<64, SELECT_ONLY><<<grid, 256, 0, s>>>(a); break;
        case 128: quant_kernel<128, SELECT_ONLY><<<grid, 256, 0, s>>>(a); break;
        default: return QAQ_ERR_UNSUPPORTED_SHAPE;
    }
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

qaq_status check_dense(const void* K, const void* V, long sb, long sh, long st, int D) {
    if (!K || !V) return QAQ_ERR_INVALID_ARG;
    if (((uintptr_t)K & 7) || ((uintptr_t)V & 7)) return QAQ_ERR_INVALID_ARG;  // 8-byte vector loads
    if (st < D || (sb & 3) || (sh & 3) || (st & 3) || sb < 0 || sh < 0) return QAQ_ERR_INVALID_ARG;
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
