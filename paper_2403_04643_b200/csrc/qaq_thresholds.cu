// S2a: exact outlier thresholds (order statistics) per (b,h) and tensor.
//
// binary16 patterns are mapped to 16-bit keys that sort like the values.  Two passes of
// an 8-bit radix select find the key of rank k from below and of rank k from above:
//   pass 1  256-bin histogram of the high key byte (shared-memory bins per CTA, merged
//           with global atomics);
//   pass 2  every CTA locates the two high-byte bins holding the wanted ranks, then
//           histograms the low byte of the keys that fall into them;
//   pass 3  one warp per (b,h,tensor) finishes the select and writes binary32 thresholds.
// NaNs are not counted.  k = floor(alpha * N / 2), N = number of counted values.
#include "qaq_internal.cuh"

namespace {

constexpr int THR_CHUNK_TOKENS = 256;  // tokens per CTA

__device__ __forceinline__ uint32_t key_of(unsigned short h) { return (h & 0x8000u) ? (uint32_t)(~h & 0xFFFFu) : (uint32_t)(h | 0x8000u); }
__device__ __forceinline__ unsigned short half_of_key(uint32_t k) { return (k & 0x8000u) ? (unsigned short)(k & 0x7FFFu) : (unsigned short)(~k & 0xFFFFu); }
__device__ __forceinline__ bool is_nan_bits(unsigned short h) { return (h & 0x7FFFu) > 0x7C00u; }

struct ThrArgs {
    const __half* X[2];
    long sb, sh, st;
    int H, T, D;
    double alpha;
    uint32_t* hist1;  // [BH*2][256]
    uint32_t* hist2;  // [BH*2][2][256]
    float* thr;       // [BH][4]
};

// rank search in a 256-bin histogram: bin holding rank `want` (0-based), and the rank inside it
__device__ void find_bin(const uint32_t* hist, unsigned long long want, int* bin, unsigned long long* within) {
    unsigned long long acc = 0;
    int b = 0;
    for (; b < 255; ++b) {
        unsigned long long n = hist[b];
        if (acc + n > want) break;
        acc += n;
    }
    *bin = b;
    *within = want - acc;
}

template <int PASS>
__global__ void __launch_bounds__(256) thr_hist_kernel(const ThrArgs a) {
    const int bhx = blockIdx.y;  // (b,h) * 2 + tensor
    const int bh = bhx >> 1, x = bhx & 1;
    __shared__ uint32_t sh[2][256];
    __shared__ int s_bin[2];
    sh[0][threadIdx.x] = 0;
    sh[1][threadIdx.x] = 0;
    if (PASS == 2 && threadIdx.x == 0) {
        const uint32_t* h1 = a.hist1 + (size_t)bhx * 256;
        unsigned long long N = 0;
        for (int b = 0; b < 256; ++b) N += h1[b];
        int bl = 0, bu = 0;
        if (N > 0) {
            unsigned long long k = (unsigned long long)floor(a.alpha * (double)N / 2.0);
            if (k > (N - 1) / 2) k = (N - 1) / 2;
            unsigned long long w;
            find_bin(h1, k, &bl, &w);
            find_bin(h1, N - 1 - k, &bu, &w);
        }
        s_bin[0] = bl; s_bin[1] = bu;
    }
    __syncthreads();
    const int b_idx = bh / a.H, h_idx = bh % a.H;
    const __half* X = a.X[x] + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh;
    const int t0 = blockIdx.x * THR_CHUNK_TOKENS, t1 = min(a.T, t0 + THR_CHUNK_TOKENS);
    const int per_tok = a.D / 4;  // uint2 (4 halves) per token
    const int n = (t1 - t0) * per_tok;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int t = t0 + i / per_tok, c = (i % per_tok) * 4;
        const uint2 raw = *reinterpret_cast<const uint2*>(X + (size_t)t * a.st + c);
        const unsigned short hv[4] = {(unsigned short)(raw.x & 0xFFFF), (unsigned short)(raw.x >> 16),
                                      (unsigned short)(raw.y & 0xFFFF), (unsigned short)(raw.y >> 16)};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (is_nan_bits(hv[j])) continue;
            const uint32_t key = key_of(hv[j]);
            if (PASS == 1) {
                atomicAdd(&sh[0][key >> 8], 1u);
            } else {
                if ((int)(key >> 8) == s_bin[0]) atomicAdd(&sh[0][key & 255], 1u);
                if ((int)(key >> 8) == s_bin[1]) atomicAdd(&sh[1][key & 255], 1u);
            }
        }
    }
    __syncthreads();
    if (PASS == 1) {
        if (sh[0][threadIdx.x]) atomicAdd(&a.hist1[(size_t)bhx * 256 + threadIdx.x], sh[0][threadIdx.x]);
    } else {
        if (sh[0][threadIdx.x]) atomicAdd(&a.hist2[((size_t)bhx * 2 + 0) * 256 + threadIdx.x], sh[0][threadIdx.x]);
        if (sh[1][threadIdx.x]) atomicAdd(&a.hist2[((size_t)bhx * 2 + 1) * 256 + threadIdx.x], sh[1][threadIdx.x]);
    }
}

__global__ void thr_final_kernel(const ThrArgs a, int n_problems) {
    const int bhx = blockIdx.x * blockDim.x + threadIdx.x;
    if (bhx >= n_problems) return;
    const uint32_t* h1 = a.hist1 + (size_t)bhx * 256;
    unsigned long long N = 0;
    for (int b = 0; b < 256; ++b) N += h1[b];
    float lo = 0.f, hi = 0.f;
    if (N > 0) {
        unsigned long long k = (unsigned long long)floor(a.alpha * (double)N / 2.0);
        if (k > (N - 1) / 2) k = (N - 1) / 2;
        int bl, bu, ll, lu;
        unsigned long long wl, wu, dummy;
        find_bin(h1, k, &bl, &wl);
        find_bin(h1, N - 1 - k, &bu, &wu);
        find_bin(a.hist2 + ((size_t)bhx * 2 + 0) * 256, wl, &ll, &dummy);
        find_bin(a.hist2 + ((size_t)bhx * 2 + 1) * 256, wu, &lu, &dummy);
        lo = __half2float(__ushort_as_half(half_of_key(((uint32_t)bl << 8) | (uint32_t)ll)));
        hi = __half2float(__ushort_as_half(half_of_key(((uint32_t)bu << 8) | (uint32_t)lu)));
    }
    a.thr[(size_t)(bhx >> 1) * 4 + (bhx & 1) * 2 + 0] = lo;
    a.thr[(size_t)(bhx >> 1) * 4 + (bhx & 1) * 2 + 1] = hi;
}

}  // namespace

extern "C" qaq_status qaq_thresholds_workspace_bytes(const qaq_config* cfg, size_t* host_out) {
    if (!cfg || !host_out || cfg->batch < 1 || cfg->heads < 1) return QAQ_ERR_INVALID_ARG;
    *host_out = (size_t)cfg->batch * cfg->heads * 2 * 3 * 256 * sizeof(uint32_t);
    return QAQ_OK;
}

extern "C" qaq_status qaq_outlier_thresholds(const qaq_config* cfg, const void* K, const void* V, long stride_b,
                                             long stride_h, long stride_t, int n_tokens, float* thr, void* ws,
                                             size_t ws_bytes, void* stream) {
    if (!cfg || !K || !V || !thr || !ws || n_tokens < 1) return QAQ_ERR_INVALID_ARG;
    if (!qaq_dim_ok(cfg->head_dim)) return QAQ_ERR_UNSUPPORTED_SHAPE;
    if (!(cfg->outlier_frac >= 0.0 && cfg->outlier_frac <= 1.0)) return QAQ_ERR_INVALID_ARG;
    if (((uintptr_t)K & 7) || ((uintptr_t)V & 7) || (stride_b & 3) || (stride_h & 3) || (stride_t & 3) ||
        stride_t < cfg->head_dim)
        return QAQ_ERR_INVALID_ARG;
    size_t need = 0;
    qaq_thresholds_workspace_bytes(cfg, &need);
    if (ws_bytes < need || ((uintptr_t)ws & 15)) return QAQ_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    const int BH = cfg->batch * cfg->heads;
    ThrArgs a;
    a.X[0] = (const __half*)K; a.X[1] = (const __half*)V;
    a.sb = stride_b; a.sh = stride_h; a.st = stride_t;
    a.H = cfg->heads; a.T = n_tokens; a.D = cfg->head_dim; a.alpha = cfg->outlier_frac;
    a.hist1 = (uint32_t*)ws;
    a.hist2 = a.hist1 + (size_t)BH * 2 * 256;
    a.thr = thr;
    QAQ_CUDA_TRY(cudaMemsetAsync(ws, 0, need, s));
    dim3 grid((n_tokens + THR_CHUNK_TOKENS - 1) / THR_CHUNK_TOKENS, BH * 2);
    thr_hist_kernel<1><<<grid, 256, 0, s>>>(a);
    thr_hist_kernel<2><<<grid, 256, 0, s>>>(a);
    thr_final_kernel<<<(BH * 2 + 63) / 64, 64, 0, s>>>(a, BH * 2);
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}
