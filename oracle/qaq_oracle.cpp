// QAQ oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, one-definition-at-a-time CPU restatement of the QAQ hot path
// (quality-adaptive KV-cache quantization + attention over the quantized cache,
// arXiv 2403.04643).  Only tests, the smoke check and the benchmark's CPU-baseline
// leg may call it; the CUDA library never does and shares no code with it.
//
// Every function cites the passage of the paper it restates.  Steps are taken in
// the paper's order and notation: no blocking, fusion or reordering.  Per-(batch,
// head) problems are independent (Section 2.1: the tensors live "within each head in
// every layer"), so every routine works on ONE (b,h) and ONE tensor (K or V) unless
// said otherwise; the batch helper only loops over (b,h), optionally on threads.
//
// Arithmetic conventions (fixed so that integer results are reproducible):
//   * inputs are IEEE binary16 bit patterns (uint16_t), widened exactly to binary32;
//   * every binary32 operation that decides an integer (a bit-width, a code, an
//     outlier flag) is a single correctly rounded operation, in the order written
//     here; compile with -ffp-contract=off so no fused multiply-add sneaks in;
//   * attention (Section 2.1) accumulates in binary64.
//
// Parity status: everything here is pinned by tests/test_oracle_pins.py except the
// paper's task-accuracy results (Tables 1-3, Figures 2/4/5), which need model weights
// and public evaluation data that are not available: "parity unpinned" for those.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

// ---- binary16 -> binary32, exact (IEEE 754-2008 interchange formats) ----------
float half_to_float(uint16_t h) {
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1Fu;
    uint32_t man = h & 0x3FFu;
    uint32_t bits;
    if (exp == 0) {
        if (man == 0) {
            bits = sign;  // +-0
        } else {          // subnormal: value = man * 2^-24
            float v = std::ldexp((float)man, -24);
            uint32_t vb;
            std::memcpy(&vb, &v, 4);
            bits = vb | sign;
        }
    } else if (exp == 31) {
        bits = sign | 0x7F800000u | (man << 13);  // inf / nan
    } else {
        bits = sign | ((exp + 112u) << 23) | (man << 13);
    }
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
}

// ---- chunk planes: the storage order of one token's codes ----------------------
// The paper fixes no storage layout (memory is "calculated by the quantized bit",
// Section 2.1).  This build's documented layout: a B-bit code is cut into the
// power-of-two pieces of B's binary representation, widest piece first, the widest
// piece holding the most significant bits.  The piece of width w (w in {8,4,2,1})
// of all D channels forms one "plane" of D*w/8 bytes; planes are concatenated.
// Inside a plane, channel d = 32*p + 4*r + i  (p = d/32, r = (d%32)/4, i = d%4)
// sits in 32-bit little-endian word  p*w + (r*w)/8  at bit  8*i + w*(r % (8/w)).
struct Piece { int w; int shift; };
int pieces_of(int B, Piece out[4]) {
    int n = 0;
    for (int w = 8; w >= 1; w >>= 1) {
        if (B & w) { out[n].w = w; out[n].shift = B & (w - 1); ++n; }
    }
    return n;
}

inline void put_bits(uint8_t* bytes, long bitpos, int w, uint32_t f) {
    for (int b = 0; b < w; ++b) {
        long pos = bitpos + b;
        if ((f >> b) & 1u) bytes[pos >> 3] |= (uint8_t)(1u << (pos & 7));
    }
}
inline uint32_t get_bits(const uint8_t* bytes, long bitpos, int w) {
    uint32_t f = 0;
    for (int b = 0; b < w; ++b) {
        long pos = bitpos + b;
        f |= (uint32_t)((bytes[pos >> 3] >> (pos & 7)) & 1u) << b;
    }
    return f;
}
inline long plane_bitpos(int d, int w) {
    int p = d / 32, r = (d % 32) / 4, i = d % 4;
    long word = (long)p * w + (r * w) / 8;
    return word * 32 + 8 * i + w * (r % (8 / w));
}

}  // namespace

extern "C" {

float qaq_oracle_half_to_float(uint16_t h) { return half_to_float(h); }

// Bytes of one token at width B: D*B/8 (D is a multiple of 32).
long qaq_oracle_token_bytes(int D, int B) { return (long)D * B / 8; }

// ---- O0: outlier thresholds (Section 4.2 "Outliers") ---------------------------
// Outliers are the values beyond the alpha% quantile at the maximum and minimum
// ends.  Reading: alpha is the total proportion, alpha/2 per tail; the thresholds
// are order statistics of the N values of this (b,h) tensor: k = floor(alpha*N/2),
// lo = sorted[k], hi = sorted[N-1-k]; a value is an outlier iff it lies strictly
// outside [lo, hi].  NaNs are left out of the population.
void qaq_oracle_thresholds(const uint16_t* x, long n, double alpha, float* lo, float* hi) {
    std::vector<float> v;
    v.reserve((size_t)n);
    for (long i = 0; i < n; ++i) {
        float f = half_to_float(x[i]);
        if (!std::isnan(f)) v.push_back(f);
    }
    if (v.empty()) { *lo = 0.f; *hi = 0.f; return; }
    std::sort(v.begin(), v.end());
    long N = (long)v.size();
    long k = (long)std::floor(alpha * (double)N / 2.0);
    if (k > (N - 1) / 2) k = (N - 1) / 2;
    if (k < 0) k = 0;
    *lo = v[(size_t)k];
    *hi = v[(size_t)(N - 1 - k)];
}

// ---- policy scalars (Section 4.1) ------------------------------------------------
// Key bound:   sigma2(K_t) <= log(T^3/(T-1) * sigma2(S)_max + 1) / sum_d Q_d^2
// Value bound: sigma(V_t)  <= sigma(X)_max / (sqrt(T) * |S_t|)
// Bit count:   B = ceil(log2((max-min) / (2*sqrt(3)*sigma)))
// The bit count is evaluated as a ladder  B = min{b : range <= c * 2^b}  with
//   cK = 2*sqrt(3)*sigmaK            (keys:   range        <= cK * 2^b)
//   cV = 2*sqrt(3)*sigmaX/sqrt(T)    (values: range * S_t  <= cV * 2^b)
// computed in binary64 and rounded once to binary32.  T < 2 has no key bound
// (division by zero in the paper's expression): cK = 0 makes every key take b_max.
void qaq_oracle_policy(double sigmaS_max, double sigmaX_max, double qnorm2, long T, float* cK,
                       float* cV) {
    double two_root3 = 2.0 * std::sqrt(3.0);
    if (T >= 2 && qnorm2 > 0.0) {
        double t = (double)T;
        double var_k = std::log(t * t * t / (t - 1.0) * sigmaS_max * sigmaS_max + 1.0) / qnorm2;
        *cK = (float)(two_root3 * std::sqrt(var_k));
    } else {
        *cK = 0.f;
    }
    *cV = (T >= 1) ? (float)(two_root3 * sigmaX_max / std::sqrt((double)T)) : 0.f;
}

// ---- O1: attention window (Sections 3.2, 4.2 "Attention score prediction") -----
// The predicted score of a token is the maximum of its preceding n scores.
// ring is [W][T] (row i = i-th stored score row); nvalid[t] <= W rows are valid
// for token t (rows 0..nvalid-1).  nvalid == 0: no score known, shat = +inf so the
// value rule saturates at b_max (aggressive quantization only after low scores
// have been observed).
void qaq_oracle_window_max(const float* ring, const uint8_t* nvalid, int W, long T, float* shat) {
    for (long t = 0; t < T; ++t) {
        int nv = nvalid[t] < W ? nvalid[t] : W;
        if (nv == 0) { shat[t] = INFINITY; continue; }
        float m = ring[t];
        for (int i = 1; i < nv; ++i) m = std::max(m, ring[(long)i * T + t]);
        shat[t] = m;
    }
}

// ---- O2: range of the non-outlier values of one token (Section 4.2) -----------
// With the outliers set aside the range of a token shrinks a lot, which is the point of
// setting them aside: min and max are taken over the entries that are not outliers.
// No such entry: range [0,0].
void qaq_oracle_masked_range(const uint16_t* x, int D, float lo, float hi, float* mn, float* mx) {
    bool any = false;
    float a = 0.f, b = 0.f;
    for (int d = 0; d < D; ++d) {
        float v = half_to_float(x[d]);
        bool outlier = !(lo <= v && v <= hi);
        if (outlier) continue;
        if (!any) { a = b = v; any = true; }
        else { a = std::min(a, v); b = std::max(b, v); }
    }
    *mn = a;
    *mx = b;
}

// ---- O3: bit ladder (Section 4.1 "Determining quantization bits") -------------
// B = ceil(log2(range / (2 sqrt3 sigma))) clamped to [bmin, bmax]
//   = min{ b in [bmin,bmax] : range <= c * 2^b },  b_max if none.
// c * 2^b is an exact power-of-two scaling; c <= 0 -> b_max.
int qaq_oracle_bits_ladder(float range, float c, int bmin, int bmax) {
    if (!(c > 0.f)) return bmax;
    for (int b = bmin; b <= bmax; ++b) {
        if (range <= std::ldexp(c, b)) return b;
    }
    return bmax;
}

// Key width: range only (the key bound has no S_t in it).
int qaq_oracle_key_bits(float mn, float mx, float cK, int bmin, int bmax) {
    float r = mx - mn;
    return qaq_oracle_bits_ladder(r, cK, bmin, bmax);
}
// Value width: range times predicted score, one binary32 multiply.
int qaq_oracle_value_bits(float mn, float mx, float shat, float cV, int bmin, int bmax) {
    float r = mx - mn;
    if (std::isinf(shat)) return bmax;
    float rv = r * shat;
    return qaq_oracle_bits_ladder(rv, cV, bmin, bmax);
}

// S1 for one (b,h): bitsK[t], bitsV[t].  thr = {loK, hiK, loV, hiV}.
void qaq_oracle_select_bits(const uint16_t* K, const uint16_t* V, long T, int D, const float* thr,
                            const float* ring, const uint8_t* nvalid, int W, float cK, float cV,
                            int bmin, int bmax, uint8_t* bitsK, uint8_t* bitsV) {
    std::vector<float> shat((size_t)T);
    qaq_oracle_window_max(ring, nvalid, W, T, shat.data());
    for (long t = 0; t < T; ++t) {
        float mn, mx;
        qaq_oracle_masked_range(K + t * D, D, thr[0], thr[1], &mn, &mx);
        bitsK[t] = (uint8_t)qaq_oracle_key_bits(mn, mx, cK, bmin, bmax);
        qaq_oracle_masked_range(V + t * D, D, thr[2], thr[3], &mn, &mx);
        bitsV[t] = (uint8_t)qaq_oracle_value_bits(mn, mx, shat[(size_t)t], cV, bmin, bmax);
    }
}

// ---- O4: uniform quantizer of one token (Section 4.1) --------------------------
// [min,max] is split into 2^B equal segments; a value is rounded to the midpoint of
// its segment.  Segments are half-open [min + c*step, min + (c+1)*step); x = max
// falls into the last one.  step = range * 2^-B (exact), inv = 1/step (one division),
// code = min(2^B - 1, floor((x - min) * inv)).  Outliers take code 0.
void qaq_oracle_token_codes(const uint16_t* x, int D, float lo, float hi, int B, float* mn_out,
                            float* step_out, uint8_t* codes, uint8_t* is_outlier) {
    float mn, mx;
    qaq_oracle_masked_range(x, D, lo, hi, &mn, &mx);
    float r = mx - mn;
    float step = std::ldexp(r, -B);
    float inv = step > 0.f ? 1.0f / step : 0.f;
    int top = (1 << B) - 1;
    for (int d = 0; d < D; ++d) {
        float v = half_to_float(x[d]);
        bool outlier = !(lo <= v && v <= hi);
        is_outlier[d] = outlier ? 1 : 0;
        if (outlier) { codes[d] = 0; continue; }
        float rel = v - mn;
        float sc = rel * inv;
        int c = (int)std::floor(sc);
        if (c > top) c = top;
        if (c < 0) c = 0;
        codes[d] = (uint8_t)c;
    }
    *mn_out = mn;
    *step_out = step;
}

// Midpoint reconstruction: xhat = min + (code + 1/2) * step, one fused rounding.
float qaq_oracle_dequant(uint8_t code, float mn, float step) {
    return std::fmaf((float)code + 0.5f, step, mn);
}

// ---- O5: pack / unpack one token (layout documented at the top) ---------------
void qaq_oracle_pack_token(const uint8_t* codes, int D, int B, uint8_t* bytes) {
    long nbytes = qaq_oracle_token_bytes(D, B);
    std::memset(bytes, 0, (size_t)nbytes);
    Piece pc[4];
    int np = pieces_of(B, pc);
    long plane_base = 0;  // in bits
    for (int k = 0; k < np; ++k) {
        int w = pc[k].w;
        for (int d = 0; d < D; ++d) {
            uint32_t f = ((uint32_t)codes[d] >> pc[k].shift) & ((1u << w) - 1u);
            put_bits(bytes, plane_base + plane_bitpos(d, w), w, f);
        }
        plane_base += (long)D * w;
    }
}
void qaq_oracle_unpack_token(const uint8_t* bytes, int D, int B, uint8_t* codes) {
    Piece pc[4];
    int np = pieces_of(B, pc);
    for (int d = 0; d < D; ++d) codes[d] = 0;
    long plane_base = 0;
    for (int k = 0; k < np; ++k) {
        int w = pc[k].w;
        for (int d = 0; d < D; ++d) {
            uint32_t f = get_bits(bytes, plane_base + plane_bitpos(d, w), w);
            codes[d] |= (uint8_t)(f << pc[k].shift);
        }
        plane_base += (long)D * w;
    }
}

// ---- S2+S3 for one (b,h) tensor: outlier split, quantize, pack ----------------
// Outputs (canonical form): mn[T], step[T], off[T+1] (byte offsets, exclusive prefix
// sum of D*B/8), stream (tokens concatenated), rowptr[T+1], ch[], val[] (outliers
// in (token, channel) order, value = the original binary16 bits, so that an outlier
// comes back without any quantization error).  Returns the number of outliers, or -1 if out_cap
// or stream_cap is too small.
long qaq_oracle_quantize(const uint16_t* x, long T, int D, float lo, float hi, const uint8_t* bits,
                         float* mn, float* step, uint32_t* off, uint8_t* stream, long stream_cap,
                         uint32_t* rowptr, uint8_t* ch, uint16_t* val, long out_cap) {
    std::vector<uint8_t> codes((size_t)D), flag((size_t)D);
    long pos = 0, nout = 0;
    for (long t = 0; t < T; ++t) {
        int B = bits[t];
        qaq_oracle_token_codes(x + t * D, D, lo, hi, B, &mn[t], &step[t], codes.data(), flag.data());
        long nb = qaq_oracle_token_bytes(D, B);
        if (pos + nb > stream_cap) return -1;
        off[t] = (uint32_t)pos;
        qaq_oracle_pack_token(codes.data(), D, B, stream + pos);
        pos += nb;
        rowptr[t] = (uint32_t)nout;
        for (int d = 0; d < D; ++d) {
            if (!flag[(size_t)d]) continue;
            if (nout >= out_cap) return -1;
            ch[nout] = (uint8_t)d;
            val[nout] = x[t * D + d];
            ++nout;
        }
    }
    off[T] = (uint32_t)pos;
    rowptr[T] = (uint32_t)nout;
    return nout;
}

// Dense reconstruction xhat[T][D] (binary32) of one quantized (b,h) tensor.
void qaq_oracle_reconstruct(long T, int D, const uint8_t* bits, const float* mn, const float* step,
                            const uint32_t* off, const uint8_t* stream, const uint32_t* rowptr,
                            const uint8_t* ch, const uint16_t* val, float* xhat) {
    std::vector<uint8_t> codes((size_t)D);
    for (long t = 0; t < T; ++t) {
        qaq_oracle_unpack_token(stream + off[t], D, bits[t], codes.data());
        for (int d = 0; d < D; ++d) xhat[t * D + d] = qaq_oracle_dequant(codes[(size_t)d], mn[t], step[t]);
        for (uint32_t o = rowptr[t]; o < rowptr[t + 1]; ++o) xhat[t * D + ch[o]] = half_to_float(val[o]);
    }
}

// ---- O9: further quantization to lower widths (Section 4.2, "Integration in text
// generation process") ------------------------------------------------------------
// In every generation step the widths of all cached tokens are computed again with the
// current scores and token count; a token whose new width is lower than its current one
// is quantized further, to the lower width.  Reading: the quantizer of O4 is nested -
// with min and range kept, the B'-bit code of a value is its B-bit code without the low
// B-B' bits - so "further" means code >>= (B-B') and step *= 2^(B-B'), which is what
// quantizing the original values at B' directly would have given.  A new width that is
// not lower leaves the token as it is (raising a width needs the unquantized copy the
// paper keeps in CPU memory; that transfer is not part of this path).
//
// Widths from the stored form: the range of a token is step * 2^B (exact), so the rules
// of O3 apply without the original values.
void qaq_oracle_reselect_bits(long T, const uint8_t* bits, const float* step, int is_value, const float* ring,
                              const uint8_t* nvalid, int W, float c, int bmin, int bmax, uint8_t* bits_new) {
    std::vector<float> shat((size_t)T);
    if (is_value) qaq_oracle_window_max(ring, nvalid, W, T, shat.data());
    for (long t = 0; t < T; ++t) {
        float r = std::ldexp(step[t], bits[t]);
        int b;
        if (!is_value) b = qaq_oracle_bits_ladder(r, c, bmin, bmax);
        else if (std::isinf(shat[(size_t)t])) b = bmax;
        else b = qaq_oracle_bits_ladder(r * shat[(size_t)t], c, bmin, bmax);
        bits_new[t] = (uint8_t)b;
    }
}
// One (b,h) tensor in canonical form (bits, step, off, stream) -> the same with every token
// at width min(bits[t], max(1, bits_req[t])).  min[], the outlier lists and the code slots of
// outliers (0) are unchanged.  Returns the new stream length, or -1 if cap is too small.
long qaq_oracle_requantize_down(long T, int D, const uint8_t* bits, const float* step, const uint32_t* off,
                                const uint8_t* stream, const uint8_t* bits_req, uint8_t* bits_out, float* step_out,
                                uint32_t* off_out, uint8_t* stream_out, long cap) {
    std::vector<uint8_t> codes((size_t)D);
    long pos = 0;
    for (long t = 0; t < T; ++t) {
        int B = bits[t];
        int want = bits_req[t] < 1 ? 1 : bits_req[t];
        int Bn = want < B ? want : B;
        int drop = B - Bn;
        qaq_oracle_unpack_token(stream + off[t], D, B, codes.data());
        for (int d = 0; d < D; ++d) codes[(size_t)d] = (uint8_t)(codes[(size_t)d] >> drop);
        long nb = qaq_oracle_token_bytes(D, Bn);
        if (pos + nb > cap) return -1;
        off_out[t] = (uint32_t)pos;
        qaq_oracle_pack_token(codes.data(), D, Bn, stream_out + pos);
        pos += nb;
        bits_out[t] = (uint8_t)Bn;
        step_out[t] = std::ldexp(step[t], drop);
    }
    off_out[T] = (uint32_t)pos;
    return pos;
}

// ---- O7: attention (Section 2.1, Figure 1) --------------------------------------
// S = Softmax(scale * Q Khat^T),  X = S Vhat, on dense binary32 Khat, Vhat [T][D],
// Q binary16 [D]; all sums in binary64; the softmax subtracts the row maximum.
void qaq_oracle_attention_dense(const uint16_t* q, const float* Khat, const float* Vhat, long T,
                                int D, double scale, double* X, double* S) {
    std::vector<double> a((size_t)T);
    double amax = -INFINITY;
    for (long t = 0; t < T; ++t) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += (double)half_to_float(q[d]) * (double)Khat[t * D + d];
        a[(size_t)t] = scale * acc;
        amax = std::max(amax, a[(size_t)t]);
    }
    double denom = 0.0;
    for (long t = 0; t < T; ++t) { a[(size_t)t] = std::exp(a[(size_t)t] - amax); denom += a[(size_t)t]; }
    for (int d = 0; d < D; ++d) X[d] = 0.0;
    for (long t = 0; t < T; ++t) {
        double s = a[(size_t)t] / denom;
        if (S) S[t] = s;
        for (int d = 0; d < D; ++d) X[d] += s * (double)Vhat[t * D + d];
    }
}

// Attention of one (b,h) read from the quantized structures.
void qaq_oracle_decode(const uint16_t* q, long T, int D, double scale,
                       const uint8_t* bitsK, const float* mnK, const float* stepK, const uint32_t* offK,
                       const uint8_t* streamK, const uint32_t* rowptrK, const uint8_t* chK, const uint16_t* valK,
                       const uint8_t* bitsV, const float* mnV, const float* stepV, const uint32_t* offV,
                       const uint8_t* streamV, const uint32_t* rowptrV, const uint8_t* chV, const uint16_t* valV,
                       double* X, double* S) {
    std::vector<float> Kh((size_t)T * D), Vh((size_t)T * D);
    qaq_oracle_reconstruct(T, D, bitsK, mnK, stepK, offK, streamK, rowptrK, chK, valK, Kh.data());
    qaq_oracle_reconstruct(T, D, bitsV, mnV, stepV, offV, streamV, rowptrV, chV, valV, Vh.data());
    qaq_oracle_attention_dense(q, Kh.data(), Vh.data(), T, D, scale, X, S);
}

// Attention on the original binary16 K, V (the unquantized reference of Section 2.1).
void qaq_oracle_attention_fp16(const uint16_t* q, const uint16_t* K, const uint16_t* V, long T, int D,
                               double scale, double* X, double* S) {
    std::vector<float> Kf((size_t)T * D), Vf((size_t)T * D);
    for (long i = 0; i < T * D; ++i) { Kf[(size_t)i] = half_to_float(K[i]); Vf[(size_t)i] = half_to_float(V[i]); }
    qaq_oracle_attention_dense(q, Kf.data(), Vf.data(), T, D, scale, X, S);
}

// ---- O8: memory accounting (Sections 2.1, 5.2) ----------------------------------
// "KV cache memory ... is calculated by the quantized bit".  For one tensor:
// code_bits = sum_t D * B_t;  CR_paper = 16*2*T*D / (code_bits + 16 * n_outliers).
double qaq_oracle_code_bits(const uint8_t* bits, long T, int D) {
    double s = 0.0;
    for (long t = 0; t < T; ++t) s += (double)D * bits[t];
    return s;
}
double qaq_oracle_cr_paper(double code_bits_k, double code_bits_v, long n_out_k, long n_out_v, long T, int D) {
    double orig = 16.0 * 2.0 * (double)T * D;
    return orig / (code_bits_k + code_bits_v + 16.0 * (double)(n_out_k + n_out_v));
}

// ---- batch helper used by the timing leg and the parity tests -------------------
// Runs thresholds (optional) -> select (optional) -> quantize(K), quantize(V) ->
// decode (optional) for every (b,h) of a [BH][T][D] batch; (b,h) problems are spread
// over n_threads.  Per-(b,h) output arrays are [BH][...] with the given capacities.
struct QaqOracleBatch {
    long BH, T; int D, W, bmin, bmax;
    double alpha, scale; float cK, cV;
    int use_given_thr, use_given_bits, run_decode;
    const uint16_t *K, *V, *q; const float* ring; const uint8_t* nvalid;
    float* thr;               // [BH][4] in/out
    uint8_t *bitsK, *bitsV;   // [BH][T] in/out
    float *mnK, *stepK, *mnV, *stepV;       // [BH][T]
    uint32_t *offK, *offV, *rowptrK, *rowptrV;  // [BH][T+1]
    uint8_t *streamK, *streamV; long stream_cap;  // [BH][stream_cap]
    uint8_t *chK, *chV; uint16_t *valK, *valV; long out_cap;  // [BH][out_cap]
    long *noutK, *noutV;      // [BH]
    double *X, *S;            // [BH][D], [BH][T] (S may be null)
};

static void run_one(const QaqOracleBatch* p, long bh) {
    long T = p->T; int D = p->D;
    const uint16_t* K = p->K + bh * T * D;
    const uint16_t* V = p->V + bh * T * D;
    float* thr = p->thr + bh * 4;
    if (!p->use_given_thr) {
        qaq_oracle_thresholds(K, T * D, p->alpha, &thr[0], &thr[1]);
        qaq_oracle_thresholds(V, T * D, p->alpha, &thr[2], &thr[3]);
    }
    uint8_t* bK = p->bitsK + bh * T; uint8_t* bV = p->bitsV + bh * T;
    if (!p->use_given_bits) {
        qaq_oracle_select_bits(K, V, T, D, thr, p->ring + bh * (long)p->W * T, p->nvalid + bh * T, p->W,
                               p->cK, p->cV, p->bmin, p->bmax, bK, bV);
    }
    p->noutK[bh] = qaq_oracle_quantize(K, T, D, thr[0], thr[1], bK, p->mnK + bh * T, p->stepK + bh * T,
                                       p->offK + bh * (T + 1), p->streamK + bh * p->stream_cap, p->stream_cap,
                                       p->rowptrK + bh * (T + 1), p->chK + bh * p->out_cap,
                                       p->valK + bh * p->out_cap, p->out_cap);
    p->noutV[bh] = qaq_oracle_quantize(V, T, D, thr[2], thr[3], bV, p->mnV + bh * T, p->stepV + bh * T,
                                       p->offV + bh * (T + 1), p->streamV + bh * p->stream_cap, p->stream_cap,
                                       p->rowptrV + bh * (T + 1), p->chV + bh * p->out_cap,
                                       p->valV + bh * p->out_cap, p->out_cap);
    if (p->run_decode && p->noutK[bh] >= 0 && p->noutV[bh] >= 0) {
        qaq_oracle_decode(p->q + bh * D, T, D, p->scale,
                          bK, p->mnK + bh * T, p->stepK + bh * T, p->offK + bh * (T + 1),
                          p->streamK + bh * p->stream_cap, p->rowptrK + bh * (T + 1), p->chK + bh * p->out_cap,
                          p->valK + bh * p->out_cap,
                          bV, p->mnV + bh * T, p->stepV + bh * T, p->offV + bh * (T + 1),
                          p->streamV + bh * p->stream_cap, p->rowptrV + bh * (T + 1), p->chV + bh * p->out_cap,
                          p->valV + bh * p->out_cap,
                          p->X + bh * D, p->S ? p->S + bh * T : nullptr);
    }
}

// Returns the number of threads actually used.
int qaq_oracle_run_batch(const QaqOracleBatch* p, int n_threads) {
    if (n_threads < 1) n_threads = 1;
    if ((long)n_threads > p->BH) n_threads = (int)p->BH;
    if (n_threads == 1) {
        for (long bh = 0; bh < p->BH; ++bh) run_one(p, bh);
        return 1;
    }
    std::vector<std::thread> th;
    for (int i = 0; i < n_threads; ++i) {
        th.emplace_back([p, i, n_threads]() {
            for (long bh = i; bh < p->BH; bh += n_threads) run_one(p, bh);
        });
    }
    for (auto& t : th) t.join();
    return n_threads;
}

}  // extern "C"
