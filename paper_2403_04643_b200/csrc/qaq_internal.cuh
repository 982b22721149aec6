// Internal definitions shared by the libqaq translation units (not part of the ABI).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qaq.h"

#define QAQ_TILE QAQ_TILE_TOKENS

// Device storage of one tensor (K or V) of the cache.  Tokens are grouped in tiles of
// QAQ_TILE consecutive tokens; a tile's packed codes are contiguous, tokens in order, and
// start 16-byte aligned somewhere in the (b,h) pool (tiles are placed by a bump allocator,
// so their order in memory is not the token order).  Per-token metadata is 5 bytes:
// the width and the binary16 min and max of the non-outlier entries (step = (max-min)*2^-B
// is recomputed where needed).  Outliers of a tile are contiguous 32-bit entries
//   value(binary16) | channel << 16 | token-in-tile << 24,  sorted by (token, channel).
struct TensorStore {
    uint8_t* codes;         // [BH][pool_bytes]
    uint8_t* bits;          // [BH][tmax_pad]
    uint32_t* mnmx;         // [BH][tmax_pad]  half(min) | half(max) << 16
    uint32_t* tile_off;     // [BH][ntiles]    byte offset of the tile in its pool
    uint32_t* tile_nbytes;  // [BH][ntiles]
    uint32_t* tile_ooff;    // [BH][ntiles]    first outlier entry of the tile
    uint32_t* tile_ocnt;    // [BH][ntiles]
    uint32_t* outl;         // [BH][ocap]
    uint32_t* pool_end;     // [BH] bump pointer, bytes
    uint32_t* opool_end;    // [BH] bump pointer, entries
};

struct qaq_cache {
    qaq_config cfg;
    int BH;
    int tmax_pad;       // max_tokens rounded up to a tile
    int ntiles;         // tmax_pad / QAQ_TILE
    size_t pool_bytes;  // per (b,h)
    uint32_t ocap;      // outlier entries per (b,h)
    TensorStore t[2];
    int* d_status;      // sticky device-side status; the two words behind it: see qaq_d_count / qaq_d_ticket
    void* slab;         // the one allocation everything above lives in
    size_t slab_bytes;
    size_t reset_off, reset_bytes;   // the range of the slab that qaq_cache_reset clears
    long tokens;        // host counter
    // lazily sized staging for the *_host entry points
    void* stage[8];
    size_t stage_bytes[8];
};

// the CUDA error behind the most recent QAQ_ERR_CUDA of this process (qaq_last_cuda_error)
extern int g_qaq_last_cuda_error;

#define QAQ_CUDA_TRY(expr)                                  \
    do {                                                    \
        cudaError_t _e = (expr);                            \
        if (_e != cudaSuccess) { g_qaq_last_cuda_error = (int)_e; (void)cudaGetLastError(); return QAQ_ERR_CUDA; } \
    } while (0)

// the token count in device memory that the qaq_stream_* calls work with (valid between qaq_stream_begin and
// qaq_stream_end), and the arrival counter of the kernel that advances it (zero between launches)
static inline int* qaq_d_count(const qaq_cache* c) { return c->d_status + 1; }
static inline unsigned* qaq_d_ticket(const qaq_cache* c) { return (unsigned*)(c->d_status + 2); }

static inline bool qaq_dim_ok(int D) { return D == 32 || D == 64 || D == 128; }

// launchers implemented in the kernel translation units
qaq_status qaq_launch_select(const qaq_config* cfg, const qaq_policy* pol, const void* K, const void* V, long sb,
                             long sh, long st, int n, const float* ring, const uint8_t* nvalid, const float* thr,
                             uint8_t* bitsK, uint8_t* bitsV, cudaStream_t s);
qaq_status qaq_launch_append(qaq_cache* c, const void* K, const void* V, long sb, long sh, long st, int n_new,
                             const uint8_t* bitsK, const uint8_t* bitsV, const qaq_policy* pol, const float* ring,
                             const uint8_t* nvalid, const float* thr, cudaStream_t s);
// single-query decode on strided query / output rows (qaq_decode.cu); ws: qaq_decode_workspace_bytes bytes
qaq_status qaq_decode_strided(const qaq_cache* c, const void* q, long q_stride, float softmax_scale, float* out, long out_stride,
                              void* ws, cudaStream_t s);
