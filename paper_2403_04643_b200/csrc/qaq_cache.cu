// Cache object: allocation, reset, statistics, canonical export, host-buffer wrappers.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include "qaq_codec.cuh"
#include "qaq_internal.cuh"

extern "C" const char* qaq_status_string(qaq_status s) {
    switch (s) {
        case QAQ_OK: return "ok";
        case QAQ_ERR_INVALID_ARG: return "invalid argument";
        case QAQ_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case QAQ_ERR_CAPACITY: return "capacity exceeded";
        case QAQ_ERR_CUDA: return "CUDA error";
        case QAQ_ERR_WORKSPACE: return "workspace too small or misaligned";
    }
    return "unknown status";
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static qaq_status check_cfg(const qaq_config* cfg) {
    if (!cfg) return QAQ_ERR_INVALID_ARG;
    if (cfg->batch < 1 || cfg->heads < 1 || cfg->max_tokens < 1 || cfg->window < 1) return QAQ_ERR_INVALID_ARG;
    if (!(cfg->outlier_frac >= 0.0 && cfg->outlier_frac <= 1.0)) return QAQ_ERR_INVALID_ARG;
    if (!qaq_dim_ok(cfg->head_dim)) return QAQ_ERR_UNSUPPORTED_SHAPE;
    if (cfg->bits_min < 1 || cfg->bits_max > 8 || cfg->bits_min > cfg->bits_max) return QAQ_ERR_UNSUPPORTED_SHAPE;
    if (cfg->window > 255) return QAQ_ERR_UNSUPPORTED_SHAPE;
    return QAQ_OK;
}

extern "C" qaq_status qaq_cache_create(const qaq_config* cfg, qaq_cache** out) {
    if (!out) return QAQ_ERR_INVALID_ARG;
    *out = nullptr;
    qaq_status st = check_cfg(cfg);
    if (st != QAQ_OK) return st;
    qaq_cache* c = (qaq_cache*)calloc(1, sizeof(qaq_cache));
    if (!c) return QAQ_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->BH = cfg->batch * cfg->heads;
    c->tmax_pad = (int)align_up((size_t)cfg->max_tokens, QAQ_TILE);
    c->ntiles = c->tmax_pad / QAQ_TILE;
    const int D = cfg->head_dim;
    // worst case per tile: every token at 8 bits or the largest padding of the value groups, plus alignment
    // padding per tile and a read-ahead margin
    c->pool_bytes = align_up((size_t)c->ntiles * (size_t)qaqc::v_tile_bytes_max(D) + 16 * (size_t)c->ntiles + 256, 256);
    if (c->pool_bytes >= ((size_t)1 << 32)) { free(c); return QAQ_ERR_UNSUPPORTED_SHAPE; }
    long ocap = cfg->max_outliers_per_bh;
    if (ocap <= 0) {
        double want = 2.0 * cfg->outlier_frac * (double)c->tmax_pad * D + 1024.0;
        ocap = (long)want;
    }
    ocap += 4L * c->ntiles + 64;  // per-tile alignment padding + read-ahead margin
    if ((double)ocap > 4.0e9) { free(c); return QAQ_ERR_UNSUPPORTED_SHAPE; }
    c->ocap = (uint32_t)align_up((size_t)ocap, 64);

    const size_t BH = (size_t)c->BH;
    size_t off = 0;
    auto carve = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    size_t o_codes[2], o_bits[2], o_mnmx[2], o_toff[2], o_tnb[2], o_tooff[2], o_tocnt[2], o_outl[2], o_pe[2], o_ope[2];
    // three regions: pools that need no initialisation; tables that start at zero; what qaq_cache_reset clears
    // (one contiguous range, one memset)
    for (int x = 0; x < 2; ++x) {
        o_codes[x] = carve(BH * c->pool_bytes);
        o_outl[x] = carve(BH * (size_t)c->ocap * 4);
    }
    for (int x = 0; x < 2; ++x) {
        o_mnmx[x] = carve(BH * c->tmax_pad * 4);
        o_toff[x] = carve(BH * c->ntiles * 4);
        o_tooff[x] = carve(BH * c->ntiles * 4);
    }
    for (int x = 0; x < 2; ++x) {
        o_bits[x] = carve(BH * c->tmax_pad);
        o_tnb[x] = carve(BH * c->ntiles * 4);
        o_tocnt[x] = carve(BH * c->ntiles * 4);
        o_pe[x] = carve(BH * 4);
        o_ope[x] = carve(BH * 4);
    }
    size_t o_status = carve(256);
    c->slab_bytes = off;
    if (cudaMalloc(&c->slab, c->slab_bytes) != cudaSuccess) { (void)cudaGetLastError(); free(c); return QAQ_ERR_CUDA; }
    char* base = (char*)c->slab;
    for (int x = 0; x < 2; ++x) {
        TensorStore& t = c->t[x];
        t.codes = (uint8_t*)(base + o_codes[x]);
        t.bits = (uint8_t*)(base + o_bits[x]);
        t.mnmx = (uint32_t*)(base + o_mnmx[x]);
        t.tile_off = (uint32_t*)(base + o_toff[x]);
        t.tile_nbytes = (uint32_t*)(base + o_tnb[x]);
        t.tile_ooff = (uint32_t*)(base + o_tooff[x]);
        t.tile_ocnt = (uint32_t*)(base + o_tocnt[x]);
        t.outl = (uint32_t*)(base + o_outl[x]);
        t.pool_end = (uint32_t*)(base + o_pe[x]);
        t.opool_end = (uint32_t*)(base + o_ope[x]);
    }
    c->d_status = (int*)(base + o_status);
    c->reset_off = o_bits[0];
    c->reset_bytes = off - o_bits[0];
    // metadata and tables start at zero; code pools need no initialisation
    if (cudaMemset(base + o_mnmx[0], 0, off - o_mnmx[0]) != cudaSuccess) {
        (void)cudaGetLastError(); cudaFree(c->slab); free(c); return QAQ_ERR_CUDA;
    }
    c->tokens = 0;
    *out = c;
    return QAQ_OK;
}

extern "C" qaq_status qaq_cache_destroy(qaq_cache* c) {
    if (!c) return QAQ_OK;
    for (int i = 0; i < 8; ++i)
        if (c->stage[i]) cudaFree(c->stage[i]);
    if (c->slab) cudaFree(c->slab);
    free(c);
    return QAQ_OK;
}

extern "C" qaq_status qaq_cache_reset(qaq_cache* c, void* stream) {
    if (!c) return QAQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    // widths, tile lengths, outlier counts, pool ends and the status word: one contiguous range
    QAQ_CUDA_TRY(cudaMemsetAsync((char*)c->slab + c->reset_off, 0, c->reset_bytes, s));
    c->tokens = 0;
    return QAQ_OK;
}

namespace {
__global__ void set_count_kernel(int* count, unsigned* ticket, int value) { *count = value; *ticket = 0u; }
}  // namespace

// The token count moves to device memory (qaq_stream_begin) and back (qaq_stream_end); between the two the
// qaq_stream_* calls read and advance it there, and the host counter is stale.
extern "C" qaq_status qaq_stream_begin(qaq_cache* c, void* stream) {
    if (!c) return QAQ_ERR_INVALID_ARG;
    set_count_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(qaq_d_count(c), qaq_d_ticket(c), (int)c->tokens);
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

extern "C" qaq_status qaq_stream_end(qaq_cache* c, void* stream) {
    if (!c) return QAQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    int count = -1;
    QAQ_CUDA_TRY(cudaMemcpyAsync(&count, qaq_d_count(c), sizeof(int), cudaMemcpyDeviceToHost, s));
    QAQ_CUDA_TRY(cudaStreamSynchronize(s));
    if (count < 0 || count > c->cfg.max_tokens) return QAQ_ERR_INVALID_ARG;
    c->tokens = count;
    return QAQ_OK;
}

int g_qaq_last_cuda_error = 0;

extern "C" const char* qaq_last_cuda_error(void) { return cudaGetErrorName((cudaError_t)g_qaq_last_cuda_error); }

extern "C" long qaq_cache_tokens(const qaq_cache* c) { return c ? c->tokens : -1; }

extern "C" qaq_status qaq_policy_from_hyper(double sigmaS_max, double sigmaX_max, double qnorm2, long T,
                                            qaq_policy* host_out) {
    if (!host_out || !(sigmaS_max >= 0.0) || !(sigmaX_max >= 0.0)) return QAQ_ERR_INVALID_ARG;
    const double c = 2.0 * sqrt(3.0);
    host_out->cK = 0.f;
    host_out->cV = 0.f;
    if (T >= 2 && qnorm2 > 0.0) {
        double t = (double)T;
        double var_k = log(t * t * t / (t - 1.0) * sigmaS_max * sigmaS_max + 1.0) / qnorm2;
        host_out->cK = (float)(c * sqrt(var_k));
    }
    if (T >= 1) host_out->cV = (float)(c * sigmaX_max / sqrt((double)T));
    return QAQ_OK;
}

// ------------------------------------------------------------------ statistics
struct StatsDev {
    unsigned long long hist[2][9];
    unsigned long long code_bytes[2];
    unsigned long long outliers[2];
    unsigned long long stored_bytes[2];   // bytes the tiles occupy (values: with the padding of their groups)
};

__global__ void stats_kernel(TensorStore tk, TensorStore tv, int T, int tmax_pad, int ntiles, int D, StatsDev* out) {
    __shared__ unsigned long long sh[2][9];
    __shared__ unsigned long long so[2], sb[2];
    if (threadIdx.x < 18) ((unsigned long long*)sh)[threadIdx.x] = 0;
    if (threadIdx.x < 2) { so[threadIdx.x] = 0; sb[threadIdx.x] = 0; }
    __syncthreads();
    const int bh = blockIdx.x;
    for (int x = 0; x < 2; ++x) {
        const TensorStore& ts = x ? tv : tk;
        for (int t = threadIdx.x; t < T; t += blockDim.x) {
            int b = ts.bits[(size_t)bh * tmax_pad + t];
            atomicAdd(&sh[x][b > 8 ? 8 : b], 1ULL);
        }
        int nt = (T + QAQ_TILE - 1) / QAQ_TILE;
        for (int i = threadIdx.x; i < nt; i += blockDim.x) {
            atomicAdd(&so[x], (unsigned long long)ts.tile_ocnt[(size_t)bh * ntiles + i]);
            atomicAdd(&sb[x], (unsigned long long)ts.tile_nbytes[(size_t)bh * ntiles + i]);
        }
    }
    __syncthreads();
    if (threadIdx.x < 18) {
        int x = threadIdx.x / 9, b = threadIdx.x % 9;
        atomicAdd(&out->hist[x][b], sh[x][b]);
        atomicAdd(&out->code_bytes[x], sh[x][b] * (unsigned long long)(D * b / 8));
    }
    if (threadIdx.x < 2) {
        atomicAdd(&out->outliers[threadIdx.x], so[threadIdx.x]);
        atomicAdd(&out->stored_bytes[threadIdx.x], sb[threadIdx.x]);
    }
}

static qaq_status ensure_stage(qaq_cache* c, int slot, size_t bytes) {
    if (c->stage_bytes[slot] >= bytes) return QAQ_OK;
    if (c->stage[slot]) { cudaFree(c->stage[slot]); c->stage[slot] = nullptr; c->stage_bytes[slot] = 0; }
    QAQ_CUDA_TRY(cudaMalloc(&c->stage[slot], bytes));
    c->stage_bytes[slot] = bytes;
    return QAQ_OK;
}

extern "C" qaq_status qaq_cache_stats(const qaq_cache* cc, qaq_stats* host_out, void* stream) {
    if (!cc || !host_out) return QAQ_ERR_INVALID_ARG;
    qaq_cache* c = const_cast<qaq_cache*>(cc);
    cudaStream_t s = (cudaStream_t)stream;
    qaq_status st = ensure_stage(c, 7, sizeof(StatsDev));
    if (st != QAQ_OK) return st;
    StatsDev* d = (StatsDev*)c->stage[7];
    QAQ_CUDA_TRY(cudaMemsetAsync(d, 0, sizeof(StatsDev), s));
    stats_kernel<<<c->BH, 256, 0, s>>>(c->t[0], c->t[1], (int)c->tokens, c->tmax_pad, c->ntiles, c->cfg.head_dim, d);
    QAQ_CUDA_TRY(cudaGetLastError());
    StatsDev h;
    int dev_status = 0;
    QAQ_CUDA_TRY(cudaMemcpyAsync(&h, d, sizeof(h), cudaMemcpyDeviceToHost, s));
    QAQ_CUDA_TRY(cudaMemcpyAsync(&dev_status, c->d_status, 4, cudaMemcpyDeviceToHost, s));
    QAQ_CUDA_TRY(cudaStreamSynchronize(s));
    memset(host_out, 0, sizeof(*host_out));
    host_out->tokens = c->tokens;
    const long BH = c->BH, T = c->tokens, D = c->cfg.head_dim;
    const long nt = (T + QAQ_TILE - 1) / QAQ_TILE;
    double bits_total = 0.0;
    long resident = 0;
    for (int x = 0; x < 2; ++x) {
        host_out->code_bytes[x] = (long)h.code_bytes[x];
        host_out->outliers[x] = (long)h.outliers[x];
        for (int b = 0; b < 9; ++b) host_out->hist[x][b] = (long)h.hist[x][b];
        bits_total += 8.0 * (double)h.code_bytes[x] + 16.0 * (double)h.outliers[x];
        resident += (long)h.stored_bytes[x] + 4 * (long)h.outliers[x] + BH * T * 5 + BH * nt * 16;
    }
    host_out->resident_bytes = resident;
    double orig_bits = 16.0 * 2.0 * (double)BH * (double)T * (double)D;
    host_out->cr_paper = bits_total > 0 ? orig_bits / bits_total : 0.0;
    host_out->cr_total = resident > 0 ? (orig_bits / 8.0) / (double)resident : 0.0;
    host_out->device_status = dev_status;
    return QAQ_OK;
}

// ------------------------------------------------------------------ canonical export
// (1) per-token byte lengths and outlier counts -> (2) per-(b,h) exclusive scans ->
// (3) gather of codes and outliers into token order.
__global__ void export_count_kernel(TensorStore ts, int T, int tmax_pad, int D, uint32_t* off) {
    const int bh = blockIdx.y, tile = blockIdx.x;
    const int t = tile * QAQ_TILE + threadIdx.x;
    const size_t rowbase = (size_t)bh * (T + 1);
    if (threadIdx.x < QAQ_TILE && t < T) {
        if (off) off[rowbase + t + 1] = (uint32_t)D * ts.bits[(size_t)bh * tmax_pad + t] / 8;
    }
}

__global__ void export_ocount_kernel(TensorStore ts, int T, int ntiles, uint32_t ocap, uint32_t* rowptr) {
    const int bh = blockIdx.y, tile = blockIdx.x;
    const uint32_t n = ts.tile_ocnt[(size_t)bh * ntiles + tile];
    const uint32_t o0 = ts.tile_ooff[(size_t)bh * ntiles + tile];
    const uint32_t* e = ts.outl + (size_t)bh * ocap + o0;
    for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) {
        int t = tile * QAQ_TILE + (int)(e[i] >> 24);
        if (t < T) atomicAdd(&rowptr[(size_t)bh * (T + 1) + t + 1], 1u);
    }
}

// in-place inclusive scan of a[1..T] (a[0] = 0) per (b,h): one block per (b,h)
__global__ void export_scan_kernel(uint32_t* a, int T) {
    __shared__ uint32_t sm[256];
    __shared__ uint32_t carry;
    uint32_t* row = a + (size_t)blockIdx.x * (T + 1);
    if (threadIdx.x == 0) { carry = 0; row[0] = 0; }
    __syncthreads();
    for (int base = 0; base < T; base += 256) {
        int i = base + threadIdx.x;
        uint32_t v = i < T ? row[i + 1] : 0;
        sm[threadIdx.x] = v;
        __syncthreads();
        for (int d = 1; d < 256; d <<= 1) {
            uint32_t add = threadIdx.x >= d ? sm[threadIdx.x - d] : 0;
            __syncthreads();
            sm[threadIdx.x] += add;
            __syncthreads();
        }
        if (i < T) row[i + 1] = sm[threadIdx.x] + carry;
        __syncthreads();
        if (threadIdx.x == 0) carry += sm[255];
        __syncthreads();
    }
}

// one canonical byte of a token: byte y of its string (the planes of its pieces, widest first; inside the plane of
// a w-bit piece channel d = 32p + 4j + i sits in word p*w + j*w/8 at bit 8i + w*(j mod 8/w)), put together from the
// pieces as the tile stores them
template <bool IS_V>
__device__ uint32_t canonical_byte(const uint8_t* tile, const qaqc::TileMasks& tm, const uint32_t (&base)[5], int D, int slot,
                                   int B, uint32_t y) {
    for (int c = 0; c < 4; ++c) {
        const int w = 8 >> c;
        if (!(B & w)) continue;
        const uint32_t plen = (uint32_t)D * w / 8;
        if (y >= plen) { y -= plen; continue; }
        const int per = 8 / w, cw = y >> 2, i = y & 3, p = cw / w, rr = cw % w;
        const int r = qaqc::rank_in(tm, c, slot);
        uint32_t v = 0;
        for (int mm = 0; mm < per; ++mm) v |= qaqc::piece_at<IS_V>(tile, base, D, c, r, 32 * p + 4 * (rr * per + mm) + i) << (w * mm);
        return v;
    }
    return 0;
}

__global__ void export_gather_kernel(TensorStore ts, int is_v, int T, int tmax_pad, int ntiles, int D, size_t pool_bytes, uint32_t ocap,
                                     uint8_t* bits, float* mn, float* step, const uint32_t* off, uint8_t* codes,
                                     long codes_stride, const uint32_t* rowptr, uint8_t* ch, __half* val, long outl_stride) {
    const int bh = blockIdx.y, tile = blockIdx.x;
    __shared__ uint32_t s_in[QAQ_TILE + 1];
    __shared__ uint8_t s_b[QAQ_TILE];
    __shared__ unsigned int s_m[4][2];
    const int t0 = tile * QAQ_TILE;
    if (threadIdx.x < QAQ_TILE) {
        const int t = t0 + threadIdx.x;
        int B = t < T ? ts.bits[(size_t)bh * tmax_pad + t] : 0;
        B = B > 8 ? 8 : B;
        s_b[threadIdx.x] = (uint8_t)B;
        for (int c = 0; c < 4; ++c) {
            const unsigned int bal = __ballot_sync(0xFFFFFFFFu, (B & (8 >> c)) != 0);
            if ((threadIdx.x & 31) == 0) s_m[c][threadIdx.x >> 5] = bal;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t acc = 0;
        for (int k = 0; k < QAQ_TILE; ++k) {
            s_in[k] = acc;
            acc += (uint32_t)D * s_b[k] / 8;
        }
        s_in[QAQ_TILE] = acc;
    }
    __syncthreads();
    if (threadIdx.x < QAQ_TILE && t0 + (int)threadIdx.x < T) {
        const int t = t0 + threadIdx.x;
        const int B = s_b[threadIdx.x];
        const uint32_t mm = ts.mnmx[(size_t)bh * tmax_pad + t];
        const float fmn = __half2float(__ushort_as_half((unsigned short)(mm & 0xFFFF)));
        const float fmx = __half2float(__ushort_as_half((unsigned short)(mm >> 16)));
        if (bits) bits[(size_t)bh * T + t] = (uint8_t)B;
        if (mn) mn[(size_t)bh * T + t] = fmn;
        if (step) step[(size_t)bh * T + t] = qaqc::step_of(fmn, fmx, B);
    }
    if (codes && off) {
        const uint8_t* src = ts.codes + (size_t)bh * pool_bytes + ts.tile_off[(size_t)bh * ntiles + tile];
        uint8_t* dst = codes + (size_t)bh * codes_stride + off[(size_t)bh * (T + 1) + t0];
        qaqc::TileMasks tm;
        for (int c = 0; c < 4; ++c) tm.m[c] = (unsigned long long)s_m[c][0] | ((unsigned long long)s_m[c][1] << 32);
        int n[4];
        for (int c = 0; c < 4; ++c) n[c] = __popcll(tm.m[c]);
        uint32_t base[5];
        {   // section offsets for any head_dim (the templates of the codec header fix it at compile time)
            uint32_t o = qaqc::QAQ_TILE_HDR;
            for (int c = 0; c < 4; ++c) {
                const int w = 8 >> c;
                base[c] = o;
                o += is_v ? (uint32_t)((n[c] + 3) >> 2) * (uint32_t)(D * w / 2) : (uint32_t)n[c] * (uint32_t)(D * w / 8);
            }
            base[4] = o;
        }
        for (int k0 = 0; k0 < QAQ_TILE; k0 += 4) {
            const int k = k0 + (threadIdx.x >> 6);
            const uint32_t len = s_in[k + 1] - s_in[k];
            for (uint32_t y = threadIdx.x & 63; y < len; y += 64)
                dst[s_in[k] + y] = (uint8_t)(is_v ? canonical_byte<true>(src, tm, base, D, k, s_b[k], y)
                                                  : canonical_byte<false>(src, tm, base, D, k, s_b[k], y));
        }
    }
    if (rowptr && (ch || val)) {
        const uint32_t n = ts.tile_ocnt[(size_t)bh * ntiles + tile];
        const uint32_t* e = ts.outl + (size_t)bh * ocap + ts.tile_ooff[(size_t)bh * ntiles + tile];
        const uint32_t dst0 = rowptr[(size_t)bh * (T + 1) + t0];
        for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) {
            uint32_t v = e[i];
            if ((long)(dst0 + i) < outl_stride) {
                if (ch) ch[(size_t)bh * outl_stride + dst0 + i] = (uint8_t)((v >> 16) & 0xFF);
                if (val) val[(size_t)bh * outl_stride + dst0 + i] = __ushort_as_half((unsigned short)(v & 0xFFFF));
            }
        }
    }
}

extern "C" qaq_status qaq_cache_export(const qaq_cache* c, int tensor, uint8_t* bits, float* mn, float* step,
                                       uint32_t* off, uint8_t* codes, long codes_stride, uint32_t* rowptr,
                                       uint8_t* ch, void* val, long outl_stride, void* stream) {
    if (!c || tensor < 0 || tensor > 1) return QAQ_ERR_INVALID_ARG;
    if (codes && !off) return QAQ_ERR_INVALID_ARG;
    if ((ch || val) && !rowptr) return QAQ_ERR_INVALID_ARG;
    const int T = (int)c->tokens;
    if (T == 0) return QAQ_OK;
    cudaStream_t s = (cudaStream_t)stream;
    const TensorStore& ts = c->t[tensor];
    const int nt = (T + QAQ_TILE - 1) / QAQ_TILE;
    dim3 grid(nt, c->BH);
    if (off) {
        QAQ_CUDA_TRY(cudaMemsetAsync(off, 0, (size_t)c->BH * (T + 1) * 4, s));
        export_count_kernel<<<grid, QAQ_TILE, 0, s>>>(ts, T, c->tmax_pad, c->cfg.head_dim, off);
        export_scan_kernel<<<c->BH, 256, 0, s>>>(off, T);
    }
    if (rowptr) {
        QAQ_CUDA_TRY(cudaMemsetAsync(rowptr, 0, (size_t)c->BH * (T + 1) * 4, s));
        export_ocount_kernel<<<grid, 128, 0, s>>>(ts, T, c->ntiles, c->ocap, rowptr);
        export_scan_kernel<<<c->BH, 256, 0, s>>>(rowptr, T);
    }
    export_gather_kernel<<<grid, 256, 0, s>>>(ts, tensor, T, c->tmax_pad, c->ntiles, c->cfg.head_dim, c->pool_bytes, c->ocap, bits, mn,
                                              step, off, codes, codes_stride, rowptr, ch, (__half*)val, outl_stride);
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

// ------------------------------------------------------------------ host-buffer wrappers
extern "C" qaq_status qaq_quantize_append_host(qaq_cache* c, const void* K_new, const void* V_new, int n_new,
                                               const qaq_policy* policy, const float* score_ring,
                                               const uint8_t* nvalid, const float* thr, void* stream) {
    if (!c || !K_new || !V_new || !policy || !score_ring || !nvalid || !thr || n_new < 1) return QAQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t BH = (size_t)c->BH, D = (size_t)c->cfg.head_dim, W = (size_t)c->cfg.window;
    const size_t kv_bytes = BH * (size_t)n_new * D * 2, ring_bytes = BH * W * (size_t)n_new * 4, nv_bytes = BH * (size_t)n_new;
    qaq_status st;
    if ((st = ensure_stage(c, 0, kv_bytes)) != QAQ_OK) return st;
    if ((st = ensure_stage(c, 1, kv_bytes)) != QAQ_OK) return st;
    if ((st = ensure_stage(c, 2, ring_bytes)) != QAQ_OK) return st;
    if ((st = ensure_stage(c, 3, nv_bytes)) != QAQ_OK) return st;
    if ((st = ensure_stage(c, 4, BH * 16)) != QAQ_OK) return st;
    QAQ_CUDA_TRY(cudaMemcpyAsync(c->stage[0], K_new, kv_bytes, cudaMemcpyHostToDevice, s));
    QAQ_CUDA_TRY(cudaMemcpyAsync(c->stage[1], V_new, kv_bytes, cudaMemcpyHostToDevice, s));
    QAQ_CUDA_TRY(cudaMemcpyAsync(c->stage[2], score_ring, ring_bytes, cudaMemcpyHostToDevice, s));
    QAQ_CUDA_TRY(cudaMemcpyAsync(c->stage[3], nvalid, nv_bytes, cudaMemcpyHostToDevice, s));
    QAQ_CUDA_TRY(cudaMemcpyAsync(c->stage[4], thr, BH * 16, cudaMemcpyHostToDevice, s));
    const long H = c->cfg.heads;
    st = qaq_quantize_append(c, c->stage[0], c->stage[1], H * n_new * (long)D, n_new * (long)D, (long)D, n_new, nullptr,
                             nullptr, policy, (const float*)c->stage[2], (const uint8_t*)c->stage[3],
                             (const float*)c->stage[4], stream);
    if (st != QAQ_OK) return st;
    QAQ_CUDA_TRY(cudaStreamSynchronize(s));
    return QAQ_OK;
}

extern "C" qaq_status qaq_decode_attention_host(qaq_cache* c, const void* q, float softmax_scale, float* out, void* stream) {
    if (!c || !q || !out) return QAQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t BH = (size_t)c->BH, D = (size_t)c->cfg.head_dim;
    size_t wsb = 0;
    qaq_status st = qaq_decode_workspace_bytes(c, &wsb);
    if (st != QAQ_OK) return st;
    if ((st = ensure_stage(c, 5, BH * D * 2 + BH * D * 4)) != QAQ_OK) return st;
    if ((st = ensure_stage(c, 6, wsb)) != QAQ_OK) return st;
    char* dq = (char*)c->stage[5];
    // q first, output after it (both 16-byte aligned: BH*D*2 is a multiple of 64)
    float* dout = (float*)(dq + BH * D * 2);
    QAQ_CUDA_TRY(cudaMemcpyAsync(dq, q, BH * D * 2, cudaMemcpyHostToDevice, s));
    st = qaq_decode_attention(c, dq, softmax_scale, dout, nullptr, c->stage[6], wsb, stream);
    if (st != QAQ_OK) return st;
    QAQ_CUDA_TRY(cudaMemcpyAsync(out, dout, BH * D * 4, cudaMemcpyDeviceToHost, s));
    QAQ_CUDA_TRY(cudaStreamSynchronize(s));
    return QAQ_OK;
}
