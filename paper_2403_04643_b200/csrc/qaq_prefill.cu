// Score window after a prefill (Section 4.2 of the paper, "Attention score prediction": the
// predicted score of a token is the maximum over the scores of the preceding n queries).  Right
// after a prefill of T tokens those are the attention rows of its last n queries on the
// unquantized binary16 keys:
//   row of query i (position T-n+i):  softmax over the tokens t <= T-n+i of  scale * q_i . k_t.
// Rows are written newest first (row r = query n-1-r), so that the rows in which token t exists
// are 0..nvalid[t]-1 with nvalid[t] = min(n, T-t); entries of tokens a query cannot see are 0.
//
// This is the one dense contraction on the path ([n x D] x [D x T] per (b,h)), so the logits run
// on the tensor cores (mma.sync m16n8k16, binary16 in, binary32 accumulate); with n <= 64 rows it is
// bound by reading K once.  Sequences of up to 4096 tokens take one kernel whose CTAs form a
// thread-block cluster per (b,h) (logits stay in shared memory, row statistics travel through
// distributed shared memory, the ring is written once); longer ones take two kernels: logits +
// per-chunk (max, sum of exponentials) of every row, then the rows are normalised in place with
// the merged (max, sum).
#include <cooperative_groups.h>

#include "qaq_internal.cuh"

namespace {

constexpr int PW_WARPS = 4;
constexpr int PW_CHUNK = 256;          // tokens per CTA: 64 per warp, 8 at a time
constexpr int PW_MAXQ = 64;            // rows (queries) at most

struct PrefillArgs {
    const __half* Q;     // [BH][n][D]
    const __half* K;
    long sb, sh, st;
    int H, T, n;
    float scale;
    float* ring;         // [BH][n][T]
    uint8_t* nvalid;     // [BH][T]
    float* qnorm2;       // [BH][n] or null
    float2* part;        // [BH][nchunk][n] (max, sum of exp) of the visible logits of a chunk
    int nchunk;
};

__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// The contraction index is permuted the same way in both operands: lane c (of the four lanes that
// share a row / a token) owns channels [c*D/4, (c+1)*D/4), read with 16-byte loads; k-step ks takes
// words 2ks and 2ks+1 of them.
template <int D>
__global__ void __launch_bounds__(PW_WARPS * 32) window_logits_kernel(const PrefillArgs a) {
    constexpr int WPL = D / 8;          // 32-bit words per lane and row
    constexpr int KS = D / 16;          // k-steps
    const int bh = blockIdx.y, chunk = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const int b_idx = bh / a.H, h_idx = bh % a.H;
    const __half* Kb = a.K + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh;
    const __half* Qb = a.Q + (size_t)bh * a.n * D;
    __shared__ float2 s_part[PW_WARPS][PW_MAXQ];

    if (a.qnorm2 && chunk == 0) {
        for (int i = threadIdx.x; i < a.n; i += blockDim.x) {
            float s = 0.f;
            for (int d = 0; d < D; ++d) { const float f = a.scale * __half2float(Qb[(size_t)i * D + d]); s = fmaf(f, f, s); }
            a.qnorm2[(size_t)bh * a.n + i] = s;
        }
    }
    const int t_warp = chunk * PW_CHUNK + warp * (PW_CHUNK / PW_WARPS);
    const float NEG = __int_as_float(0xff800000);

    for (int mp = 0; mp * 32 < a.n; ++mp) {            // two 16-row tiles of queries at a time
        uint32_t afr[2][KS][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const int r0 = mp * 32 + mt * 16 + g, r1 = r0 + 8;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const uint32_t* q0 = reinterpret_cast<const uint32_t*>(Qb + (size_t)r0 * D + c * (D / 4)) + 2 * ks;
                const uint32_t* q1 = reinterpret_cast<const uint32_t*>(Qb + (size_t)r1 * D + c * (D / 4)) + 2 * ks;
                afr[mt][ks][0] = r0 < a.n ? q0[0] : 0u;
                afr[mt][ks][1] = r1 < a.n ? q1[0] : 0u;
                afr[mt][ks][2] = r0 < a.n ? q0[1] : 0u;
                afr[mt][ks][3] = r1 < a.n ? q1[1] : 0u;
            }
        }
        // running (max, sum) of this lane's share of rows (mt, g) and (mt, g+8)
        float rm[2][2], rs[2][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) { rm[mt][0] = rm[mt][1] = NEG; rs[mt][0] = rs[mt][1] = 0.f; }

#pragma unroll 2
        for (int step = 0; step < PW_CHUNK / PW_WARPS / 8; ++step) {
            const int t0 = t_warp + 8 * step;
            if (t0 >= a.T) break;
            uint32_t bw[WPL];
            {
                const int t = t0 + g;
                const uint4* src = reinterpret_cast<const uint4*>(Kb + (size_t)(t < a.T ? t : 0) * a.st + c * (D / 4));
#pragma unroll
                for (int i = 0; i < WPL / 4; ++i) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (t < a.T) v = src[i];
                    bw[4 * i] = v.x; bw[4 * i + 1] = v.y; bw[4 * i + 2] = v.z; bw[4 * i + 3] = v.w;
                }
            }
            float acc[2][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) mma_16816(acc[mt], afr[mt][ks], bw[2 * ks], bw[2 * ks + 1]);
            }
            // acc[mt][0..1]: row g, tokens t0+2c, t0+2c+1;  acc[mt][2..3]: row g+8
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int hr = 0; hr < 2; ++hr) {
                    const int i = mp * 32 + mt * 16 + g + 8 * hr;          // query
                    if (i >= a.n) continue;
                    const int last = a.T - a.n + i;                         // last token the query sees
                    float* row = a.ring + ((size_t)bh * a.n + (a.n - 1 - i)) * a.T;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int t = t0 + 2 * c + e;
                        if (t >= a.T) continue;
                        const float l = a.scale * acc[mt][2 * hr + e];
                        row[t] = l;
                        if (t <= last) {
                            const float mnew = fmaxf(rm[mt][hr], l);
                            rs[mt][hr] = rs[mt][hr] * __expf(rm[mt][hr] - mnew) + __expf(l - mnew);
                            rm[mt][hr] = mnew;
                        }
                    }
                }
        }
        // merge the four lanes of a row, then the warps, into the chunk's partial
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int hr = 0; hr < 2; ++hr) {
                float m = rm[mt][hr], s = rs[mt][hr];
#pragma unroll
                for (int o = 1; o < 4; o <<= 1) {
                    const float m2 = __shfl_xor_sync(0xFFFFFFFFu, m, o), s2 = __shfl_xor_sync(0xFFFFFFFFu, s, o);
                    const float mn = fmaxf(m, m2);
                    s = (m == NEG ? 0.f : s * __expf(m - mn)) + (m2 == NEG ? 0.f : s2 * __expf(m2 - mn));
                    m = mn;
                }
                const int il = mt * 16 + g + 8 * hr;                        // row inside this pair of tiles
                if (c == 0) s_part[warp][il] = make_float2(m, s);
            }
        __syncthreads();
        for (int il = threadIdx.x; il < 32; il += blockDim.x) {
            const int i = mp * 32 + il;
            if (i >= a.n) continue;
            float m = NEG, s = 0.f;
            for (int w = 0; w < PW_WARPS; ++w) {
                const float2 p = s_part[w][il];
                const float mn = fmaxf(m, p.x);
                s = (m == NEG ? 0.f : s * __expf(m - mn)) + (p.x == NEG ? 0.f : p.y * __expf(p.x - mn));
                m = mn;
            }
            a.part[((size_t)bh * a.nchunk + chunk) * a.n + i] = make_float2(m, s);
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256) window_normalize_kernel(const PrefillArgs a) {
    const int bh = blockIdx.y, chunk = blockIdx.x;
    __shared__ float s_m[PW_MAXQ], s_inv[PW_MAXQ];
    const float NEG = __int_as_float(0xff800000);
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) {
        float m = NEG, s = 0.f;
        for (int ch = 0; ch < a.nchunk; ++ch) {
            const float2 p = a.part[((size_t)bh * a.nchunk + ch) * a.n + i];
            const float mn = fmaxf(m, p.x);
            s = (m == NEG ? 0.f : s * __expf(m - mn)) + (p.x == NEG ? 0.f : p.y * __expf(p.x - mn));
            m = mn;
        }
        s_m[i] = m;
        s_inv[i] = s > 0.f ? 1.0f / s : 0.f;
    }
    __syncthreads();
    const int t_lo = chunk * PW_CHUNK;
    const int nt = min(PW_CHUNK, a.T - t_lo);
    for (int k = threadIdx.x; k < nt; k += blockDim.x) {      // a thread takes a token through all rows
        const int t = t_lo + k;
        float* p = a.ring + (size_t)bh * a.n * a.T + t;
#pragma unroll 4
        for (int r = 0; r < a.n; ++r) {
            const int i = a.n - 1 - r;
            p[(size_t)r * a.T] = (t <= a.T - a.n + i) ? __expf(p[(size_t)r * a.T] - s_m[i]) * s_inv[i] : 0.f;
        }
        a.nvalid[(size_t)bh * a.T + t] = (uint8_t)min(a.n, a.T - t);
    }
}

// ---- one pass: the CTAs of one (b,h) form a thread-block cluster.  Each keeps the logits of its 512 tokens in
// shared memory, the per-row (max, sum) of the CTAs are exchanged through distributed shared memory, and the
// normalised rows are written once: K is read once and the ring written once (no logits in global memory, no
// workspace).  Used while a (b,h) fits a portable cluster (up to 8 x 512 tokens); longer sequences take the two
// kernels above.
constexpr int PC_WARPS = 16;            // 32 tokens per warp
constexpr int PC_MINCTA = 2;            // two CTAs per SM (64 registers per thread)
constexpr int PC_CHUNK = 512;           // tokens per CTA
constexpr int PC_MAXCTA = 8;            // portable cluster size
constexpr int PC_PITCH = PC_CHUNK + 8;  // row pitch of the logits tile in floats (spreads the rows of a fragment over the banks)

template <int D>
__global__ void __launch_bounds__(PC_WARPS * 32, PC_MINCTA) window_cluster_kernel(const PrefillArgs a) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    constexpr int WPL = D / 8;
    constexpr int KS = D / 16;
    extern __shared__ __align__(16) float s_l[];            // [n][PC_PITCH] logits of this CTA's tokens, then the queries
    // the queries as A-operand fragments, one uint4 per (16-row tile, k step, lane): every warp reads the same ones
    uint4* s_q = reinterpret_cast<uint4*>(s_l + (size_t)a.n * PC_PITCH);
    __shared__ float s_part[PC_WARPS][32];                   // per warp: maximum of every row of the current 32 over its tokens
    __shared__ float s_mcta[PW_MAXQ];                        // maximum of every row over this CTA's tokens
    __shared__ float2 s_all[PC_MAXCTA][PW_MAXQ];             // (max, sum of exponentials) of every row over the tokens of every CTA
                                                             // of the cluster: each CTA writes its entries into all the copies
    __shared__ float s_inv[PW_MAXQ];
    const int bh = blockIdx.y, chunk = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const int b_idx = bh / a.H, h_idx = bh % a.H;
    const __half* Kb = a.K + (size_t)b_idx * a.sb + (size_t)h_idx * a.sh;
    const __half* Qb = a.Q + (size_t)bh * a.n * D;
    const float NEG = __int_as_float(0xff800000);

    if (a.qnorm2 && chunk == 0) {
        for (int i = threadIdx.x; i < a.n; i += blockDim.x) {
            float s = 0.f;
            for (int d = 0; d < D; ++d) { const float f = a.scale * __half2float(Qb[(size_t)i * D + d]); s = fmaf(f, f, s); }
            a.qnorm2[(size_t)bh * a.n + i] = s;
        }
    }
    const int t_cta = chunk * PC_CHUNK;
    const int t_warp = t_cta + warp * (PC_CHUNK / PC_WARPS);
    // this warp's keys are on their way to L2 while the queries are laid out
    constexpr int LPT = D >= 64 ? D / 64 : 1;                                    // 128-byte lines per token
    for (int ln = lane; ln < (PC_CHUNK / PC_WARPS) * LPT; ln += 32) {
        const int t = t_warp + ln / LPT;
        if (t < a.T) asm volatile("prefetch.global.L2 [%0];" ::"l"(Kb + (size_t)t * a.st + (ln % LPT) * 64));
    }
    // first half of a cluster barrier: by the time the row statistics are exchanged every CTA of the cluster is known
    // to be running (its shared memory may be written)
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

    const int ntile = 2 * ((a.n + 31) / 32);
    for (int idx = threadIdx.x; idx < ntile * KS * 32; idx += blockDim.x) {
        const int ln = idx & 31, ks = (idx >> 5) % KS, tile = idx / (32 * KS);
        const int r0 = tile * 16 + (ln >> 2), r1 = r0 + 8, cc = ln & 3;
        // k step ks of lane (., cc): words 2 (ks mod 2), + 1 of the 16-byte piece 4 (ks / 2) + cc of the row
        const int w0 = 4 * (4 * (ks >> 1) + cc) + 2 * (ks & 1);
        const uint32_t* q0 = reinterpret_cast<const uint32_t*>(Qb + (size_t)r0 * D) + w0;
        const uint32_t* q1 = reinterpret_cast<const uint32_t*>(Qb + (size_t)r1 * D) + w0;
        uint4 f;
        f.x = r0 < a.n ? q0[0] : 0u;
        f.y = r1 < a.n ? q1[0] : 0u;
        f.z = r0 < a.n ? q0[1] : 0u;
        f.w = r1 < a.n ? q1[1] : 0u;
        s_q[idx] = f;
    }
    __syncthreads();

    for (int mp = 0; mp * 32 < a.n; ++mp) {            // two 16-row tiles of queries at a time
        float rm[2][2];                 // running maximum of rows g, g + 8 of the two tiles over the tokens this lane sees
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) rm[mt][0] = rm[mt][1] = NEG;

#pragma unroll 1
        for (int step = 0; step < PC_CHUNK / PC_WARPS / 8; step += 2) {    // two groups of 8 tokens per set of query fragments
            const int t0 = t_warp + 8 * step;
            if (t0 >= a.T) break;
            // lane (g, c) holds, of token t0 + g (and t0 + 8 + g), the 16-byte pieces c, c + 4, ...: the four lanes of a
            // token read 64 consecutive bytes at a time, and the words of piece 4i + c are the B operands of k steps
            // 2i and 2i + 1 (the queries are laid out to match)
            uint32_t bw[2][WPL];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int t = t0 + 8 * h + g;
                const uint4* src = reinterpret_cast<const uint4*>(Kb + (size_t)(t < a.T ? t : 0) * a.st) + c;
#pragma unroll
                for (int i = 0; i < WPL / 4; ++i) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (t < a.T) v = src[4 * i];
                    bw[h][4 * i] = v.x; bw[h][4 * i + 1] = v.y; bw[h][4 * i + 2] = v.z; bw[h][4 * i + 3] = v.w;
                }
            }
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                float acc[2][4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { acc[0][i] = 0.f; acc[1][i] = 0.f; }
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const uint4 f = s_q[((2 * mp + mt) * KS + ks) * 32 + lane];
                    const uint32_t fr[4] = {f.x, f.y, f.z, f.w};
                    mma_16816(acc[0], fr, bw[0][2 * ks], bw[0][2 * ks + 1]);
                    mma_16816(acc[1], fr, bw[1][2 * ks], bw[1][2 * ks + 1]);
                }
                // acc[h][0..1]: row g, tokens t0+8h+2c, +1;  acc[h][2..3]: row g+8
#pragma unroll
                for (int hr = 0; hr < 2; ++hr) {
                    const int i = mp * 32 + mt * 16 + g + 8 * hr;          // query
                    if (i >= a.n) continue;
                    const int last = a.T - a.n + i;                         // last token the query sees
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int t = t0 + 8 * h + 2 * c;
                        const float l0 = a.scale * acc[h][2 * hr], l1 = a.scale * acc[h][2 * hr + 1];
                        *reinterpret_cast<float2*>(&s_l[(size_t)i * PC_PITCH + (t - t_cta)]) = make_float2(l0, l1);
                        if (t <= last) rm[mt][hr] = fmaxf(rm[mt][hr], l0);       // last < T: one bound does for both
                        if (t + 1 <= last) rm[mt][hr] = fmaxf(rm[mt][hr], l1);
                    }
                }
            }
        }
        // merge the four lanes of a row, then the warps, into this CTA's maximum of the row
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int hr = 0; hr < 2; ++hr) {
                float m = rm[mt][hr];
                m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
                m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
                if (c == 0) s_part[warp][mt * 16 + g + 8 * hr] = m;
            }
        __syncthreads();
        if (threadIdx.x < 32 && mp * 32 + (int)threadIdx.x < a.n) {
            float m = NEG;
#pragma unroll
            for (int w = 0; w < PC_WARPS; ++w) m = fmaxf(m, s_part[w][threadIdx.x]);
            s_mcta[mp * 32 + threadIdx.x] = m;
        }
        __syncthreads();
    }
    // ---- the logits become exponentials relative to the CTA's row maximum, in place (one exponential per entry in
    //      all; entries a query cannot see become 0), and every row gets its sum over this CTA's tokens
    const int nt = min(PC_CHUNK, a.T - t_cta);
    const unsigned ncta = cluster.num_blocks(), rank = cluster.block_rank();
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");       // second half of the barrier begun at the start
    for (int i = warp; i < a.n; i += PC_WARPS) {
        const int last = a.T - a.n + i;
        const float m = s_mcta[i];
        float* rowl = s_l + (size_t)i * PC_PITCH;
        float sum = 0.f;
        for (int k = 4 * lane; k < nt; k += 128) {       // the pitch covers the four of a ragged end; what is there is not used
            const float4 l = *reinterpret_cast<const float4*>(rowl + k);
            float4 e;
            e.x = (t_cta + k <= last) ? __expf(l.x - m) : 0.f;
            e.y = (t_cta + k + 1 <= last) ? __expf(l.y - m) : 0.f;
            e.z = (t_cta + k + 2 <= last) ? __expf(l.z - m) : 0.f;
            e.w = (t_cta + k + 3 <= last) ? __expf(l.w - m) : 0.f;
            *reinterpret_cast<float4*>(rowl + k) = e;
            sum += (e.x + e.y) + (e.z + e.w);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        if (lane < (int)ncta) *cluster.map_shared_rank(&s_all[rank][i], lane) = make_float2(m, sum);
    }
    // ---- every CTA of the (b,h) has the row statistics of all of them (the remote stores are complete at the cluster
    //      barrier, and nothing is read from or written to another CTA afterwards): merge them
    cluster.sync();
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) {
        float m = NEG, s = 0.f;
        for (unsigned r = 0; r < ncta; ++r) {
            const float2 p = s_all[r][i];
            const float mn = fmaxf(m, p.x);
            s = (m == NEG ? 0.f : s * __expf(m - mn)) + (p.x == NEG ? 0.f : p.y * __expf(p.x - mn));
            m = mn;
        }
        // what this CTA's exponentials are multiplied by: exp(own maximum - maximum of the row) / sum of the row
        const float own = s_mcta[i];
        s_inv[i] = (s > 0.f && own != NEG) ? __expf(own - m) / s : 0.f;
    }
    __syncthreads();
    // ---- normalised rows, newest first, written once; rows-per-token counts
    const bool vec_ok = (a.T & 3) == 0 && ((uintptr_t)a.ring & 15) == 0;      // rows start 16-byte aligned, no ragged end
    for (int r = warp; r < a.n; r += PC_WARPS) {
        const int i = a.n - 1 - r;
        const float f = s_inv[i];
        float* row = a.ring + ((size_t)bh * a.n + r) * a.T + t_cta;
        const float* src = s_l + (size_t)i * PC_PITCH;
        if (vec_ok) {     // four tokens per lane and store
            for (int k = 4 * lane; k < nt; k += 128) {
                float4 o = *reinterpret_cast<const float4*>(src + k);
                o.x *= f; o.y *= f; o.z *= f; o.w *= f;
                *reinterpret_cast<float4*>(row + k) = o;
            }
        } else {
            for (int k = lane; k < nt; k += 32) row[k] = src[k] * f;
        }
    }
    for (int k = threadIdx.x; k < nt; k += blockDim.x) a.nvalid[(size_t)bh * a.T + t_cta + k] = (uint8_t)min(a.n, a.T - (t_cta + k));
}

// Upper quantile of a list of binary32 values (the squared query norms): exact 4 x 8-bit radix select on
// order-preserving keys by one CTA.  NaNs are not counted.
constexpr int QS_THREADS = 1024;
__device__ __forceinline__ uint32_t order_key(float f) {
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__global__ void __launch_bounds__(QS_THREADS) quantile_kernel(const float* __restrict__ v, long n, double upper_frac, float* out) {
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long s_count;
    __shared__ uint32_t s_prefix;
    __shared__ unsigned long long s_rank;
    const int tid = threadIdx.x;
    if (tid == 0) s_count = 0;
    __syncthreads();
    unsigned long long mine = 0;
    for (long i = tid; i < n; i += QS_THREADS) mine += (v[i] == v[i]) ? 1ull : 0ull;
    atomicAdd(&s_count, mine);
    __syncthreads();
    const unsigned long long N = s_count;
    if (N == 0) { if (tid == 0) *out = 0.f; return; }
    if (tid == 0) {
        unsigned long long k = (unsigned long long)floor(upper_frac * (double)N);
        if (k > N - 1) k = N - 1;
        s_rank = N - 1 - k;          // ascending rank of the answer
        s_prefix = 0;
    }
    __syncthreads();
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t prefix = s_prefix, pmask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (long i = tid; i < n; i += QS_THREADS) {
            const float f = v[i];
            if (f == f) {
                const uint32_t key = order_key(f);
                if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 0xFF], 1u);
            }
        }
        __syncthreads();
        if (tid == 0) {
            unsigned long long r = s_rank;
            int b = 0;
            for (; b < 255; ++b) {
                if (r < hist[b]) break;
                r -= hist[b];
            }
            s_rank = r;
            s_prefix = prefix | ((uint32_t)b << shift);
        }
        __syncthreads();
    }
    if (tid == 0) {
        const uint32_t key = s_prefix;
        const uint32_t u = (key & 0x80000000u) ? (key & 0x7FFFFFFFu) : ~key;
        *out = __uint_as_float(u);
    }
}

}  // namespace

extern "C" qaq_status qaq_prefill_window_workspace_bytes(const qaq_config* cfg, int n_tokens, size_t* host_out) {
    if (!cfg || !host_out || n_tokens < 1 || cfg->batch < 1 || cfg->heads < 1 || cfg->window < 1) return QAQ_ERR_INVALID_ARG;
    const size_t nchunk = ((size_t)n_tokens + PW_CHUNK - 1) / PW_CHUNK;
    *host_out = (size_t)cfg->batch * cfg->heads * nchunk * (size_t)cfg->window * sizeof(float2);
    return QAQ_OK;
}

extern "C" qaq_status qaq_prefill_window(const qaq_config* cfg, const void* Q, const void* K, long stride_b, long stride_h,
                                         long stride_t, int n_tokens, float softmax_scale, float* score_ring,
                                         uint8_t* nvalid, float* qnorm2, void* ws, size_t ws_bytes, void* stream) {
    if (!cfg || !Q || !K || !score_ring || !nvalid || !ws || n_tokens < 1) return QAQ_ERR_INVALID_ARG;
    if (!qaq_dim_ok(cfg->head_dim) || cfg->window < 1 || cfg->window > PW_MAXQ) return QAQ_ERR_UNSUPPORTED_SHAPE;
    if (((uintptr_t)K & 15) || ((uintptr_t)Q & 15) || (stride_b & 7) || (stride_h & 7) || (stride_t & 7) ||
        stride_t < cfg->head_dim || stride_b < 0 || stride_h < 0)
        return QAQ_ERR_INVALID_ARG;
    size_t need = 0;
    qaq_prefill_window_workspace_bytes(cfg, n_tokens, &need);
    if (ws_bytes < need || ((uintptr_t)ws & 7)) return QAQ_ERR_WORKSPACE;
    PrefillArgs a;
    a.Q = (const __half*)Q; a.K = (const __half*)K; a.sb = stride_b; a.sh = stride_h; a.st = stride_t;
    a.H = cfg->heads; a.T = n_tokens; a.n = cfg->window; a.scale = softmax_scale;
    a.ring = score_ring; a.nvalid = nvalid; a.qnorm2 = qnorm2; a.part = (float2*)ws;
    a.nchunk = (n_tokens + PW_CHUNK - 1) / PW_CHUNK;
    cudaStream_t s = (cudaStream_t)stream;
    const int ncl = (n_tokens + PC_CHUNK - 1) / PC_CHUNK;
    if (ncl <= PC_MAXCTA) {
        // one pass: the CTAs of a (b,h) are one cluster
        const size_t smem = (size_t)cfg->window * PC_PITCH * sizeof(float) +
                            (size_t)(2 * ((cfg->window + 31) / 32)) * (cfg->head_dim / 16) * 32 * sizeof(uint4);   // logits, query fragments
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3((unsigned)ncl, (unsigned)(cfg->batch * cfg->heads));
        lc.blockDim = dim3(PC_WARPS * 32);
        lc.dynamicSmemBytes = smem;
        lc.stream = s;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = (unsigned)ncl; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        lc.attrs = at; lc.numAttrs = 1;
        switch (cfg->head_dim) {
            case 32:
                QAQ_CUDA_TRY(cudaFuncSetAttribute(window_cluster_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
                QAQ_CUDA_TRY(cudaLaunchKernelEx(&lc, window_cluster_kernel<32>, a)); break;
            case 64:
                QAQ_CUDA_TRY(cudaFuncSetAttribute(window_cluster_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
                QAQ_CUDA_TRY(cudaLaunchKernelEx(&lc, window_cluster_kernel<64>, a)); break;
            case 128:
                QAQ_CUDA_TRY(cudaFuncSetAttribute(window_cluster_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
                QAQ_CUDA_TRY(cudaLaunchKernelEx(&lc, window_cluster_kernel<128>, a)); break;
            default: return QAQ_ERR_UNSUPPORTED_SHAPE;
        }
        QAQ_CUDA_TRY(cudaGetLastError());
        return QAQ_OK;
    }
    const dim3 grid((unsigned)a.nchunk, (unsigned)(cfg->batch * cfg->heads));
    switch (cfg->head_dim) {
        case 32: window_logits_kernel<32><<<grid, PW_WARPS * 32, 0, s>>>(a); break;
        case 64: window_logits_kernel<64><<<grid, PW_WARPS * 32, 0, s>>>(a); break;
        case 128: window_logits_kernel<128><<<grid, PW_WARPS * 32, 0, s>>>(a); break;
        default: return QAQ_ERR_UNSUPPORTED_SHAPE;
    }
    window_normalize_kernel<<<grid, 256, 0, s>>>(a);
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}

extern "C" qaq_status qaq_qnorm2_quantile(const float* values, long n, double upper_frac, float* out, void* stream) {
    if (!values || !out || n < 1 || !(upper_frac >= 0.0 && upper_frac < 1.0)) return QAQ_ERR_INVALID_ARG;
    quantile_kernel<<<1, QS_THREADS, 0, (cudaStream_t)stream>>>(values, n, upper_frac, out);
    QAQ_CUDA_TRY(cudaGetLastError());
    return QAQ_OK;
}
