// Checkpoint writer (Section IV-D, offload side): lay out the clustered directory from the tags, then gather
// each block's rows from the paged pool, compute per-group fp16 scales, quantise and pack the record.
// The inverse direction of restore: an HBM-bound stream through the same kind of bulk-copy pipeline.
#include <cuda_fp16.h>

#include <algorithm>

#include "common.cuh"

namespace patchkv {

constexpr int kPlanThreads = kScanThreads;
constexpr int kGatherThreads = 256;

// One CTA per layer: offsets of the runs [bf16][int8][int4][k4v4], ascending block index inside a run.  The four
// tags are counted and ranked together: one counting pass (warp votes) for the runs' bases, then one prefix sum per
// 1024 blocks over four 16-bit counters packed into a 64-bit word.
__global__ void __launch_bounds__(kPlanThreads)
plan_checkpoint_kernel(const uint8_t* tags, int NB, unsigned long long elems, int group,
                       unsigned long long* blk_off, unsigned long long* layer_bytes, int32_t* status) {
    __shared__ unsigned long long warp_sums[33];
    __shared__ unsigned int tag_total[4];
    const int l = blockIdx.x;
    const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint8_t* tg = tags + (long long)l * NB;
    unsigned long long* off = blk_off + (long long)l * NB;
    if (threadIdx.x < 4) tag_total[threadIdx.x] = 0;
    __syncthreads();
    bool bad = false;
    for (int j0 = 0; j0 < NB; j0 += kPlanThreads) {
        const int j = j0 + threadIdx.x;
        const int tag = j < NB ? tg[j] : 255;
        bad = bad || (j < NB && tag > PATCHKV_TAG_K4V4);
#pragma unroll
        for (int t = 0; t <= PATCHKV_TAG_K4V4; t++) {
            const unsigned c = __popc(__ballot_sync(0xFFFFFFFFu, tag == t));
            if (lane == 0 && c) atomicAdd(&tag_total[t], c);
        }
    }
    __syncthreads();
    unsigned long long rec[4], base[4], end = 0;
#pragma unroll
    for (int t = 0; t <= PATCHKV_TAG_K4V4; t++) {
        rec[t] = record_bytes(t, elems, group);
        base[t] = end;
        end += (unsigned long long)tag_total[t] * rec[t];
    }
    unsigned int run[4] = {0, 0, 0, 0};                     // blocks of each tag in the chunks before this one
    for (int j0 = 0; j0 < NB; j0 += kPlanThreads) {
        const int j = j0 + threadIdx.x;
        const int tag = j < NB ? tg[j] : 255;
        const bool mine = tag <= PATCHKV_TAG_K4V4;
        const unsigned long long v = mine ? 1ull << (16 * tag) : 0ull;
        unsigned long long inc = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= (unsigned)d) inc += o;
        }
        __syncthreads();                                    // warp_sums free to overwrite
        if (lane == 31) warp_sums[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const unsigned long long w = warp_sums[lane];   // kPlanThreads / 32 = 32 warps: one per lane
            unsigned long long winc = w;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, winc, d);
                if (lane >= (unsigned)d) winc += o;
            }
            warp_sums[lane] = winc - w;
            if (lane == 31) warp_sums[32] = winc;
        }
        __syncthreads();
        const unsigned long long excl = warp_sums[warp] + inc - v, total = warp_sums[32];
        if (mine) {
            const unsigned int rank = (unsigned int)(excl >> (16 * tag)) & 0xFFFFu;
            unsigned int before = run[0];
            unsigned long long b = base[0], r = rec[0];
#pragma unroll
            for (int t = 1; t <= PATCHKV_TAG_K4V4; t++) if (tag == t) { before = run[t]; b = base[t]; r = rec[t]; }
            off[j] = b + (unsigned long long)(before + rank) * r;
        } else if (j < NB) {
            off[j] = ~0ull;
        }
#pragma unroll
        for (int t = 0; t <= PATCHKV_TAG_K4V4; t++) run[t] += (unsigned int)(total >> (16 * t)) & 0xFFFFu;
    }
    if (bad) atomicCAS(status, 0, (int)PATCHKV_E_BOUNDS);
    if (threadIdx.x == 0) layer_bytes[l] = end;
}

struct GatherParams {
    int32_t L, H, D, B, P, G;
    const uint16_t* k_base;
    const uint16_t* v_base;
    long long stride_layer, stride_page, stride_token, stride_head;
    int32_t n_pages, n, nb, src_shift, n_table;
    int32_t layer_begin;                    // first layer of this launch (grid = nb * layers of the launch)
    const int32_t* block_table;
    const uint8_t* tags;
    const unsigned long long* blk_off;
    void* const* layer_payload;
    const unsigned long long* layer_bytes;
    int32_t* status;
};

// Eight bf16 channels -> one chunk of a section.  `seg` = lanes per scale group (group / 8, a power of two).
template <int FMT>
__device__ __forceinline__ void encode_chunk(const uint4& w, uint8_t* codes, uint8_t* scales, size_t elem0,
                                             size_t scale_index, int seg, bool write) {
    if (FMT == FMT_BF16) {
        if (write) *reinterpret_cast<uint4*>(codes + 2 * elem0) = w;
        return;
    }
    float x[8];
    x[0] = __uint_as_float(w.x << 16); x[1] = __uint_as_float(w.x & 0xFFFF0000u);
    x[2] = __uint_as_float(w.y << 16); x[3] = __uint_as_float(w.y & 0xFFFF0000u);
    x[4] = __uint_as_float(w.z << 16); x[5] = __uint_as_float(w.z & 0xFFFF0000u);
    x[6] = __uint_as_float(w.w << 16); x[7] = __uint_as_float(w.w & 0xFFFF0000u);
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; i++) amax = fmaxf(amax, fabsf(x[i]));
    for (int d = 1; d < seg; d <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
    const float qmax = FMT == FMT_INT8 ? 127.0f : 7.0f;
    const __half s16 = __float2half_rn(__fdiv_rn(amax, qmax));
    const float s = __half2float(s16);
    // code = rint(fp32(x / s)), ties to even.  x has 8 significant bits and s has 11, so x / s is either exactly a
    // half-integer or at least 2^-12 away from one; the fp32 rounding of the quotient (< 2^-16 here) therefore never
    // crosses a rounding boundary, and the code is the exact quotient rounded to the nearest integer, ties to even.
    // That is computed without a division per element: t = x * (1/s) is within 2^-16 of the quotient, so rint(t) is
    // right unless the quotient is an exact tie, which the exact remainder x - k*s (one fma) detects and repairs.
    const float r = s > 0.0f ? __frcp_rn(s) : 0.0f;
    const float half_s = s > 0.0f ? 0.5f * s : -1.0f;      // -1: a zero group has no ties to look for
    const float magic = 12582912.0f;                       // 1.5 * 2^23: adding it rounds to an integer, ties to even
    // tm = x * r + magic in one fused operation rounds the product to an integer k (low byte of tm = the code).
    // |x * r| <= qmax * (1 + 2^-11) < qmax + 0.5 whenever s is a normal fp16, so no clamp is needed then; a subnormal
    // s can be far below amax / qmax and takes the clamped path below.  Two lanes per instruction throughout.
    uint32_t kb[8];
    float df[8];
    const f32x2 r2 = pack2(r, r), m2 = pack2(magic, magic), ns2 = pack2(-s, -s);
    bool any_tie = false;
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
        const f32x2 x2 = pack2(x[i], x[i + 1]);
        const f32x2 tm = fma2(x2, r2, m2);
        const f32x2 d2 = fma2(sub2(tm, m2), ns2, x2);      // x - k*s, exact: a multiple of ulp(s) no larger than s
        float a0, a1;
        unpack2(tm, a0, a1);
        kb[i] = __float_as_uint(a0); kb[i + 1] = __float_as_uint(a1);
        unpack2(d2, df[i], df[i + 1]);
        any_tie = any_tie || fabsf(df[i]) == half_s || fabsf(df[i + 1]) == half_s;
    }
    if (any_tie) {                                         // rare: an exact half-integer quotient sitting on an odd k
#pragma unroll
        for (int i = 0; i < 8; i++)
            if (fabsf(df[i]) == half_s && (kb[i] & 1u)) kb[i] += df[i] > 0.0f ? 1u : 0xFFFFFFFFu;
    }
    if ((__half_as_ushort(s16) & 0x7C00u) == 0 && s > 0.0f) {      // subnormal scale: |k| may exceed qmax
#pragma unroll
        for (int i = 0; i < 8; i++) {
            const float k = fminf(fmaxf(__uint_as_float(kb[i]) - magic, -qmax), qmax);
            kb[i] = __float_as_uint(k + magic);
        }
    }
    if (!write) return;
    // byte k of a word <- low byte of kb[k]
    const uint32_t w0 = __byte_perm(__byte_perm(kb[0], kb[1], 0x0040), __byte_perm(kb[2], kb[3], 0x0040), 0x5410);
    const uint32_t w1 = __byte_perm(__byte_perm(kb[4], kb[5], 0x0040), __byte_perm(kb[6], kb[7], 0x0040), 0x5410);
    if (FMT == FMT_INT8) {
        *reinterpret_cast<uint2*>(codes + elem0) = make_uint2(w0, w1);
    } else {
        // keep the low nibble of every byte and squeeze four bytes into sixteen bits: channel 2k -> low nibble of byte k
        uint32_t a = w0 & 0x0F0F0F0Fu, b = w1 & 0x0F0F0F0Fu;
        a = (a | (a >> 4)) & 0x00FF00FFu; a = (a | (a >> 8)) & 0x0000FFFFu;
        b = (b | (b >> 4)) & 0x00FF00FFu; b = (b | (b >> 8)) & 0x0000FFFFu;
        *reinterpret_cast<uint32_t*>(codes + (elem0 >> 1)) = a | (b << 16);
    }
    if (((threadIdx.x & 31) & (seg - 1)) == 0) *reinterpret_cast<__half*>(scales + 2 * scale_index) = s16;
}

// One CTA per (layer, block).
__global__ void __launch_bounds__(kGatherThreads)
quantize_gather_kernel(const GatherParams p) {
    extern __shared__ long long tok_off[];                  // block_tokens entries
    const int l = p.layer_begin + blockIdx.x / p.nb, j = blockIdx.x % p.nb;
    const int tag = __ldg(p.tags + (size_t)l * p.nb + j);
    const unsigned long long off = __ldg(p.blk_off + (size_t)l * p.nb + j);
    const unsigned long long lbytes = __ldg(p.layer_bytes + l);
    uint8_t* base = reinterpret_cast<uint8_t*>(
        static_cast<uintptr_t>(__ldg(reinterpret_cast<const unsigned long long*>(p.layer_payload) + l)));
    const unsigned long long elems = (unsigned long long)p.B * p.H * p.D;
    const unsigned long long rec = record_bytes(tag, elems, p.G);
    bool bad = rec == 0 || off > lbytes || rec > lbytes - off || base == nullptr ||
               ((reinterpret_cast<uintptr_t>(base) + off) & 15u) != 0;
    const int valid = min(p.B, p.n - j * p.B);
    for (int t = threadIdx.x; t < p.B; t += kGatherThreads) {
        long long o = -1;                                   // past the end of the suffix: encodes as zeros
        if (t < valid) {
            const long long u = (long long)j * p.B + t + p.src_shift;
            const long long lp = u / p.P;
            const int page = lp < p.n_table ? __ldg(p.block_table + lp) : -1;
            if (page < 0 || page >= p.n_pages) bad = true;
            o = (long long)l * p.stride_layer + (long long)page * p.stride_page + (u - lp * p.P) * p.stride_token;
        }
        tok_off[t] = o;
    }
    if (__syncthreads_or(bad)) {                            // skip the block whole, latch the error
        if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)PATCHKV_E_BOUNDS);
        return;
    }
    const int kf = k_format(tag), vf = v_format(tag);
    uint8_t* kc = base + off;
    uint8_t* ks = kc + code_bytes(kf, elems);
    uint8_t* vc = ks + scale_bytes(kf, elems, p.G);
    uint8_t* vs = vc + code_bytes(vf, elems);
    const int cpv = p.D >> 3;                               // 8-channel chunks per head vector
    const int seg = p.G >> 3;                               // lanes per scale group
    const int gpv = p.D / p.G;
    const bool cpv_pow2 = (cpv & (cpv - 1)) == 0, h_pow2 = (p.H & (p.H - 1)) == 0;
    const int cpv_shift = 31 - __clz(cpv), h_shift = 31 - __clz(p.H), seg_shift = 31 - __clz(seg);
    const int units = p.B * p.H * cpv;
    const int padded = (units + kGatherThreads - 1) / kGatherThreads * kGatherThreads;
#pragma unroll 1
    for (int sec = 0; sec < 2; sec++) {
        const int fmt = sec ? vf : kf;
        const uint16_t* pool = sec ? p.v_base : p.k_base;
        uint8_t* codes = sec ? vc : kc;
        uint8_t* scales = sec ? vs : ks;
#pragma unroll 4
        for (int u = threadIdx.x; u < padded; u += kGatherThreads) {
            const bool in = u < units;
            const int vec = cpv_pow2 ? (u >> cpv_shift) : u / cpv;
            const int cx = u - vec * cpv;
            const int t = h_pow2 ? (vec >> h_shift) : vec / p.H;
            const int h = vec - t * p.H;
            uint4 w = make_uint4(0, 0, 0, 0);
            if (in) {
                const long long to = tok_off[t];
                if (to >= 0) w = __ldg(reinterpret_cast<const uint4*>(pool + to + (long long)h * p.stride_head + 8 * cx));
            }
            const size_t elem0 = (size_t)vec * p.D + 8 * cx;
            const size_t sidx = (size_t)vec * gpv + (cx >> seg_shift);
            switch (fmt) {
                case FMT_BF16: encode_chunk<FMT_BF16>(w, codes, scales, elem0, sidx, seg, in); break;
                case FMT_INT8: encode_chunk<FMT_INT8>(w, codes, scales, elem0, sidx, seg, in); break;
                default:       encode_chunk<FMT_INT4>(w, codes, scales, elem0, sidx, seg, in); break;
            }
        }
    }
}

__device__ __forceinline__ uint32_t absmax_bf16x2(uint32_t a, uint32_t b) {     // max(|a|, |b|) per half; sign bits arbitrary
    uint32_t d;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// The codes of a span element by element, with a tie test on the exact remainder and the clamp a subnormal scale
// needs: the rare path of quantise_span (a span whose scale is a subnormal fp16).
template <int FMT, int NC>
__device__ __forceinline__ void quantise_span_exact(const uint4* w, float s, float r, bool subnormal, uint32_t* out) {
    const float qmax = FMT == FMT_INT8 ? 127.0f : 7.0f;
    const float half_s = 0.5f * s, magic = 12582912.0f;
#pragma unroll
    for (int c = 0; c < NC; c++) {
        const uint32_t word[4] = {w[c].x, w[c].y, w[c].z, w[c].w};
        uint32_t lo = 0, hi = 0;                            // int8: bytes 0..3 / 4..7; int4: nibbles 0..7 in lo
#pragma unroll
        for (int i = 0; i < 8; i++) {
            const float x = __uint_as_float((i & 1) ? (word[i >> 1] & 0xFFFF0000u) : (word[i >> 1] << 16));
            const float tm = __fmaf_rn(x, r, magic);
            const float d = __fmaf_rn(__fsub_rn(tm, magic), -s, x);     // x - k*s, exact
            uint32_t kb = __float_as_uint(tm);
            if (fabsf(d) == half_s && (kb & 1u)) kb += d > 0.0f ? 1u : 0xFFFFFFFFu;      // a tie sitting on an odd k
            if (subnormal) kb = __float_as_uint(fminf(fmaxf(__uint_as_float(kb) - magic, -qmax), qmax) + magic);
            if (FMT == FMT_INT8) {
                if (i < 4) lo |= (kb & 0xFFu) << (8 * i); else hi |= (kb & 0xFFu) << (8 * (i - 4));
            } else {
                lo |= (kb & 0xFu) << (4 * i);
            }
        }
        if (FMT == FMT_INT8) { out[2 * c] = lo; out[2 * c + 1] = hi; } else out[c] = lo;
    }
}

// Quantises a span of NC consecutive 8-channel chunks (8 * NC channels of one head vector, all inside one scale
// group), so that the scale arithmetic is paid once per 8 * NC elements.  `seg` = lanes that share a scale group.
// Register c of `w` holds chunk (c + rot) & (NC - 1) of the span (neighbouring threads read their chunks from shared
// memory in a rotated order so that a quarter-warp's 128-bit loads fall into distinct banks); the codes come back
// packed in registers in that same order (int8: two words per chunk; int4: one word per chunk), with the fp16 scale.
//
// scale = fp16(amax / qmax): the fp32 quotient comes from q0 = amax * y, q = q0 + (amax - q0 * qmax) * y with
// y = fp32(1 / qmax) and fused operations, which is the correctly rounded quotient for every bf16-valued amax and
// qmax = 7 or 127 (checked over all 32 640 finite values).  code = rint(x / s), ties to even: x has 8 significant
// bits and s has 11, so x / s is either exactly a half-integer or at least 2^-12 away from one.  With r = 1/s to
// within an ulp, t = x * r and one correction t' = t + (x - t*s) * r (the remainder is exact) give a quotient that
// is within 2^-15 of x / s and *equal* to it whenever x / s is a half-integer (an fp32 value, which the correction
// reproduces exactly); adding 1.5 * 2^23 then rounds it to the integer the exact quotient rounds to, ties to even,
// and leaves the code in the low byte.  Four packed fp32 operations per pair of elements, no tie test.  A span whose
// scale is a subnormal fp16 (its codes may need the clamp) takes the element-wise path above.
template <int FMT, int NC>
__device__ __forceinline__ void quantise_span(const uint4* w, int seg, uint32_t* out, __half* scale) {
    uint32_t mx = 0;
#pragma unroll
    for (int c = 0; c < NC; c++) {
        mx = absmax_bf16x2(mx, w[c].x); mx = absmax_bf16x2(mx, w[c].y);
        mx = absmax_bf16x2(mx, w[c].z); mx = absmax_bf16x2(mx, w[c].w);
    }
    mx &= 0x7FFF7FFFu;
    uint32_t amax_bits = max(mx << 16, mx & 0xFFFF0000u);
    for (int d = 1; d < seg; d <<= 1) amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, d));
    const float amax = __uint_as_float(amax_bits);
    const float qmax = FMT == FMT_INT8 ? 127.0f : 7.0f;
    const float y = 1.0f / qmax;                            // a compile-time constant, rounded to nearest
    const float q0 = __fmul_rn(amax, y);
    float q = __fmaf_rn(__fmaf_rn(-q0, qmax, amax), y, q0);
    if (amax_bits >= 0x7F800000u) q = amax;                 // inf, nan: as the division gives
    const __half s16 = __float2half_rn(q);
    const float s = __half2float(s16);
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(s));
    r = s > 0.0f ? r : 0.0f;
    const float magic = 12582912.0f;                       // 1.5 * 2^23: adding it rounds to an integer, ties to even
    const uint32_t exp16 = __half_as_ushort(s16) & 0x7C00u;
    const bool subnormal = exp16 == 0 && s > 0.0f;          // |k| may exceed qmax
    // an infinite scale (amax beyond 65504 * qmax) has r = 0 and every code 0: keep inf * 0 out of the remainder
    const float s_rem = exp16 == 0x7C00u ? 0.0f : s;
    const f32x2 r2 = pack2(r, r), m2 = pack2(magic, magic), ns2 = pack2(-s_rem, -s_rem);
#pragma unroll
    for (int c = 0; c < NC; c++) {
        const uint32_t word[4] = {w[c].x, w[c].y, w[c].z, w[c].w};
        uint32_t kb[8];
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const f32x2 x2 = pack2(__uint_as_float(word[j] << 16), __uint_as_float(word[j] & 0xFFFF0000u));
            const f32x2 t = mul2(x2, r2);
            const f32x2 tq = fma2(fma2(t, ns2, x2), r2, t);
            const f32x2 tm = add2(tq, m2);                  // low byte of each half = the code
            float t0, t1;
            unpack2(tm, t0, t1);
            kb[2 * j] = __float_as_uint(t0); kb[2 * j + 1] = __float_as_uint(t1);
        }
        if (FMT == FMT_INT8) {
            out[2 * c] = __byte_perm(__byte_perm(kb[0], kb[1], 0x0040), __byte_perm(kb[2], kb[3], 0x0040), 0x5410);
            out[2 * c + 1] = __byte_perm(__byte_perm(kb[4], kb[5], 0x0040), __byte_perm(kb[6], kb[7], 0x0040), 0x5410);
        } else {
            // even channels -> low nibbles, odd channels -> high nibbles of the same bytes
            const uint32_t ev = __byte_perm(__byte_perm(kb[0], kb[2], 0x0040), __byte_perm(kb[4], kb[6], 0x0040), 0x5410);
            const uint32_t od = __byte_perm(__byte_perm(kb[1], kb[3], 0x0040), __byte_perm(kb[5], kb[7], 0x0040), 0x5410);
            out[c] = (ev & 0x0F0F0F0Fu) | ((od << 4) & 0xF0F0F0F0u);
        }
    }
    if (subnormal) quantise_span_exact<FMT, NC>(w, s, r, subnormal, out);
    *scale = s16;
}

__device__ __forceinline__ void sts64(uint32_t a, uint32_t x, uint32_t y) {
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(a), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t x) {
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(a), "r"(x) : "memory");
}

// One pass of a consumer warp over 32 consecutive spans of a quantised unit: quantise, put the codes back into the
// warp's own part of the stage in record order, and copy them out with 16-byte stores that cover the warp's piece of
// the record contiguously.  `region` = shared address of the warp's 32 spans, `u0` = index of its first span.
template <int FMT, int NC>
__device__ __forceinline__ void encode_pass(uint32_t region, int u0, int units, int staged, uint8_t* codes,
                                            uint8_t* scales, int seg, int seg_shift, int rot, int lane) {
    constexpr int kSpanOut = FMT == FMT_INT8 ? 8 * NC : 4 * NC;     // bytes of codes per span
    const int u = u0 + lane;
    uint4 w[NC];
    if (u0 + 32 <= staged) {
#pragma unroll
        for (int k = 0; k < NC; k++) w[k] = lds128(region + 16u * (uint32_t)(lane * NC + ((k + rot) & (NC - 1))));
    } else {
#pragma unroll
        for (int k = 0; k < NC; k++)                        // rows past the end of the suffix encode as zeros
            w[k] = u < staged ? lds128(region + 16u * (uint32_t)(lane * NC + ((k + rot) & (NC - 1)))) : make_uint4(0, 0, 0, 0);
    }
    uint32_t out[FMT == FMT_INT8 ? 2 * NC : NC];
    __half s16;
    quantise_span<FMT, NC>(w, seg, out, &s16);
    __syncwarp();                                           // every lane holds its input: the region can be reused
    if (u < units) {
#pragma unroll
        for (int k = 0; k < NC; k++) {
            const int lc = (k + rot) & (NC - 1);
            if (FMT == FMT_INT8) sts64(region + (uint32_t)(lane * kSpanOut + 8 * lc), out[2 * k], out[2 * k + 1]);
            else sts32(region + (uint32_t)(lane * kSpanOut + 4 * lc), out[k]);
        }
        if ((lane & (seg - 1)) == 0) *reinterpret_cast<__half*>(scales + 2 * (size_t)(u >> seg_shift)) = s16;
    }
    __syncwarp();
    const int bytes = min(32, units - u0) * kSpanOut;       // a multiple of 16 (checked at launch)
#pragma unroll
    for (int o = 0; o < 32 * kSpanOut; o += 512) {
        const int b = o + 16 * lane;
        if (b < bytes) *reinterpret_cast<uint4*>(codes + (size_t)u0 * kSpanOut + b) = lds128(region + b);
    }
}

// ---------------------------------------------------------------- persistent bulk-copy pipeline
// The block encoder as a persistent kernel: one producer warp takes rounds of consecutive (layer, block) entries (the
// first dealt out statically, the rest claimed from the launch's work counter in shrinking rounds), looks up and
// validates the directory entries and source pages a round of up to 32 blocks ahead, one block per lane, and stages
// the blocks' K and V rows into a shared-memory ring with bulk asynchronous
// copies that complete on an mbarrier; the consumer warps quantise from shared memory and write the record with
// warp-contiguous stores.  A stage (a unit) carries up to kWMaxSub pieces -- a piece is a run of tokens of one section
// of one block -- so that geometries with small rows still move about 32 KiB per barrier round trip, and the
// consumer warps share out the unit's passes (32 spans each) whatever piece they fall into, so that every warp is
// busy whatever the pieces' sizes.  Reads of several units are in flight per CTA at all times.  Every wait is bounded.
constexpr int kWPipeConsumerWarps = 8;                      // (twelve were slower: 0.93 against 0.99 on K8/V8 blocks)
constexpr int kWPipeThreads = 32 * (kWPipeConsumerWarps + 1);
constexpr int kWPipeMaxStages = 8;
constexpr int kWPipeMaxPages = 4;                          // logical pages one block may touch in this kernel
constexpr int kWMaxSub = 8;                                // pieces per unit

struct WPipeCfg {
    int32_t unit_tokens;                                    // rows of a piece at most (<= 32: one row per producer lane)
    int32_t cap_rows;                                       // rows a stage holds
    int32_t stage_bytes, n_stages, heads_contiguous, total_items;
    int32_t spans_per_row;                                  // H * D / (8 * NC)
    int32_t round_div;                                      // a round: left / (round_div * CTAs) blocks, 1 .. 32
    int32_t* sched;                                         // this launch's work counters: [0] blocks handed out, [1] CTAs gone
    uint32_t wait_limit;                                    // polls before a barrier wait gives up
    int32_t stall_after;                                    // self-test only: consumer warp 0 withholds the `empty`
                                                            // arrival of its unit number stall_after (-1: never)
    // bytes of a block's / a token's codes and scales per format, and of a record per tag
    uint32_t blk_codes[3], blk_scales[3], tok_codes[3], tok_scales[3], rec_bytes[4];
};
struct WSub {                                               // 32 bytes: one piece of a unit
    unsigned long long codes, scales;                       // where the piece's codes / scales go in the record
    int32_t fmt, rows;                                      // rows: total | valid << 16 (rows past the suffix are zeros)
    int32_t row0, pass0;                                    // first row of the piece in the stage, its first pass
};
constexpr int kWMetaBytes = 16 + 32 * kWMaxSub;             // {n_sub (< 0: no more work), n_pass, passes per piece if
                                                            // all alike else 0, -}, then the pieces

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

template <int NC>
__global__ void __launch_bounds__(kWPipeThreads, 2)
quantize_gather_pipe_kernel(const __grid_constant__ GatherParams p, const __grid_constant__ WPipeCfg cfg) {
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ uint64_t full_bar[kWPipeMaxStages], empty_bar[kWPipeMaxStages];
    __shared__ int abort_flag;
    const int S = cfg.n_stages;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; s++) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kWPipeConsumerWarps); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile int* abortp = &abort_flag;
    const int off_meta = cfg.stage_bytes - kWMetaBytes;
    const int row_bytes = p.H * p.D * 2, vec_bytes = p.D * 2;

    if (threadIdx.x < 32) {
        // ================================================================ producer warp
        const int lane = threadIdx.x;
        const uint32_t hd = (uint32_t)p.H * p.D;
        uint32_t q = 0;                                     // units published
        int stage = 0;
        uint32_t phase = 0;
        bool alive = true;
        // the unit being filled
        bool open = false;
        int open_rows = 0, open_sub = 0, open_pass = 0, open_ppp = 0;   // open_ppp: passes per piece if all alike, else 0
        auto close_unit = [&]() {
            __syncwarp();                                   // the pieces' descriptors and byte counts come from other lanes
            if (lane == 0) {
                *reinterpret_cast<int4*>(ring + (size_t)stage * cfg.stage_bytes + off_meta) = make_int4(open_sub, open_pass, open_ppp, 0);
                mbar_arrive(&full_bar[stage]);
            }
            __syncwarp();
            q++;
            if (++stage == S) { stage = 0; phase ^= 1; }
            open = false; open_rows = 0; open_sub = 0; open_pass = 0;
        };
        auto open_unit = [&]() -> bool {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&empty_bar[stage], phase ^ 1, abortp, cfg.wait_limit))) return false;
            open = true;
            return true;
        };
        // Directory entries and source pages are looked up and validated thirty-two blocks at a time, one block per
        // lane, a whole round before they are used: the loads of the next round are issued when the current round
        // starts, so their latency never sits in front of a copy, and the per-block work left on the serial path is
        // a handful of shuffles.  Section sizes per format come precomputed (no divisions here).
        struct Pre {
            unsigned long long rec;                         // address of the block's record, 0: skip the block
            long long layer_off;                            // l * stride_layer
            int tag, valid, slot0;                          // slot0: first source slot counted from the first page
            int pages[kWPipeMaxPages];
            long long o0;                                   // simple blocks: where the block's first row lies in the pool
            int simple;                                     // all rows of the block follow one another in one page
        };
        auto lookup = [&](long long first, int count, Pre& r) {
            const long long item = first + lane;
            r.rec = 0; r.layer_off = 0; r.tag = 0; r.valid = 0; r.slot0 = 0; r.o0 = 0; r.simple = 0;
#pragma unroll
            for (int k = 0; k < kWPipeMaxPages; k++) r.pages[k] = 0;
            if (lane < count) {
                const int it = (int)item;
                const int l = p.layer_begin + it / p.nb, j = it - (it / p.nb) * p.nb;
                const int tag = __ldg(p.tags + (size_t)l * p.nb + j);
                const unsigned long long off = __ldg(p.blk_off + (size_t)l * p.nb + j);
                const unsigned long long lbytes = __ldg(p.layer_bytes + l);
                const unsigned long long base = __ldg(reinterpret_cast<const unsigned long long*>(p.layer_payload) + l);
                const int u0 = j * p.B + p.src_shift;       // token indices fit 32 bits (checked at launch)
                const int lp0 = u0 / p.P;
                const int valid = min(p.B, p.n - j * p.B);
                const int last = (u0 + valid - 1) / p.P - lp0;
                bool bad = tag < 0 || tag > PATCHKV_TAG_K4V4;
                const unsigned long long rec = bad ? 0 : (unsigned long long)cfg.rec_bytes[tag];
                bad = bad || off > lbytes || rec > lbytes - off || base == 0 || ((base + off) & 15u) != 0;
#pragma unroll
                for (int k = 0; k < kWPipeMaxPages; k++) {
                    if (k <= last) {
                        const int page = lp0 + k < p.n_table ? __ldg(p.block_table + lp0 + k) : -1;
                        if (page < 0 || page >= p.n_pages) bad = true;
                        r.pages[k] = page;
                    }
                }
                r.rec = bad ? 1 : base + off;               // 1: latch the error when the block's turn comes
                r.layer_off = (long long)l * p.stride_layer;
                r.tag = tag; r.valid = valid; r.slot0 = u0 - lp0 * p.P;
                r.simple = !bad && last == 0 && cfg.heads_contiguous && p.stride_token == (long long)hd && p.B <= cfg.unit_tokens;
                r.o0 = r.layer_off + (long long)r.pages[0] * p.stride_page + (long long)r.slot0 * p.stride_token;
            }
        };
        // Blocks are handed out in rounds of consecutive blocks, one block per lane: the first round statically (CTA b
        // takes blocks b * r0 ...), the rest from the launch's work counter, shrinking towards the end of the list so
        // that CTAs whose blocks were cheaper (bf16 blocks are copies) take more of them.  The claim for the round after
        // the next one is issued when a round starts and read a round later, so its latency is never waited for.
        const int r0 = (int)max(1ll, min(32ll, (long long)cfg.total_items / ((long long)cfg.round_div * gridDim.x)));
        const long long static_items = (long long)r0 * gridDim.x;
        long long seen = static_items;                     // blocks known to be handed out already
        long long c_first = 0;                              // the pending claim (lane 0)
        int c_round = 0;
        auto claim = [&]() {
            if (lane == 0) {
                const long long left = (long long)cfg.total_items - seen;
                c_round = (int)max(1ll, min(32ll, left / ((long long)cfg.round_div * gridDim.x)));
                c_first = static_items + atomicAdd(cfg.sched, c_round);
            }
        };
        claim();
        Pre cur, nxt;
        long long cur_first = (long long)blockIdx.x * r0;
        int cur_n = (int)max(0ll, min((long long)r0, (long long)cfg.total_items - cur_first));
        lookup(cur_first, cur_n, cur);
        nxt = cur;
#pragma unroll 1
        while (cur_n > 0 && alive) {
            const long long nxt_first = __shfl_sync(0xFFFFFFFFu, c_first, 0);
            const int nxt_round = __shfl_sync(0xFFFFFFFFu, c_round, 0);
            seen = max(seen, nxt_first + nxt_round);
            const int nxt_n = (int)max(0ll, min((long long)nxt_round, (long long)cfg.total_items - nxt_first));
            if (nxt_n > 0) { lookup(nxt_first, nxt_n, nxt); claim(); }
            const uint32_t bad_mask = __ballot_sync(0xFFFFFFFFu, cur.rec == 1);
            const uint32_t simple_mask = __ballot_sync(0xFFFFFFFFu, cur.simple != 0);
#pragma unroll 1
            for (int ri = 0; ri < cur_n && alive; ri++) {
            if ((bad_mask >> ri) & 1u) {                    // skip the block whole, latch the error
                if (lane == 0) atomicCAS(p.status, 0, (int)PATCHKV_E_BOUNDS);
                continue;
            }
            if ((simple_mask >> ri) & 1u) {
                // The block's rows are one contiguous run of the pool (the usual case: a block inside one page): the
                // lane that looked the block up writes the two pieces' descriptors and issues their copies from its own
                // registers; the warp only keeps the books of the unit.
#pragma unroll 1
                for (int sec = 0; sec < 2; sec++) {
                    if (open && (open_rows + p.B > cfg.cap_rows || open_sub == kWMaxSub)) close_unit();
                    if (!open && !open_unit()) { alive = false; break; }
                    if (lane == ri) {
                        const int kf = k_format(cur.tag), vf = v_format(cur.tag);
                        const int fmt = sec ? vf : kf;
                        uint8_t* sp = ring + (size_t)stage * cfg.stage_bytes;
                        uint8_t* codes = reinterpret_cast<uint8_t*>(static_cast<uintptr_t>(cur.rec)) +
                                         (sec ? cfg.blk_codes[kf] + cfg.blk_scales[kf] : 0u);
                        WSub m;
                        m.codes = reinterpret_cast<unsigned long long>(codes);
                        m.scales = reinterpret_cast<unsigned long long>(codes + cfg.blk_codes[fmt]);
                        m.fmt = fmt; m.rows = p.B | (cur.valid << 16); m.row0 = open_rows; m.pass0 = open_pass;
                        *reinterpret_cast<WSub*>(sp + off_meta + 16 + 32 * open_sub) = m;
                        const uint32_t bytes = (uint32_t)cur.valid * row_bytes;
                        mbar_expect_tx(&full_bar[stage], bytes);
                        bulk_g2s(sp + (size_t)open_rows * row_bytes, (sec ? p.v_base : p.k_base) + cur.o0, bytes, &full_bar[stage]);
                    }
                    const int piece_passes = (p.B * cfg.spans_per_row + 31) >> 5;
                    open_ppp = open_sub == 0 ? piece_passes : (open_ppp == piece_passes ? open_ppp : 0);
                    open_rows += p.B; open_sub++;
                    open_pass += piece_passes;
                    if (open_rows >= cfg.cap_rows) close_unit();
                }
                continue;
            }
            const unsigned long long rec = __shfl_sync(0xFFFFFFFFu, cur.rec, ri);
            const long long layer_off = __shfl_sync(0xFFFFFFFFu, cur.layer_off, ri);
            const int tag = __shfl_sync(0xFFFFFFFFu, cur.tag, ri);
            const int valid = __shfl_sync(0xFFFFFFFFu, cur.valid, ri);
            const int slot0 = __shfl_sync(0xFFFFFFFFu, cur.slot0, ri);
            int pages[kWPipeMaxPages];
#pragma unroll
            for (int k = 0; k < kWPipeMaxPages; k++) pages[k] = __shfl_sync(0xFFFFFFFFu, cur.pages[k], ri);
            const int kf = k_format(tag), vf = v_format(tag);
            uint8_t* sec_codes[2];
            uint8_t* sec_scales[2];
            sec_codes[0] = reinterpret_cast<uint8_t*>(static_cast<uintptr_t>(rec));
            sec_scales[0] = sec_codes[0] + cfg.blk_codes[kf];
            sec_codes[1] = sec_scales[0] + cfg.blk_scales[kf];
            sec_scales[1] = sec_codes[1] + cfg.blk_codes[vf];
#pragma unroll 1
            for (int t0 = 0; t0 < p.B && alive; t0 += cfg.unit_tokens) {
                const int rows_total = min(cfg.unit_tokens, p.B - t0);
                const int rows_valid = max(0, min(rows_total, valid - t0));
                // where this lane's row of the piece lies in the pool (the same for K and V)
                long long o = 0;
                if (lane < rows_valid) {
                    int us = slot0 + t0 + lane, page = pages[0];
#pragma unroll
                    for (int k = 1; k < kWPipeMaxPages; k++) if (us >= p.P) { us -= p.P; page = pages[k]; }
                    o = layer_off + (long long)page * p.stride_page + (long long)us * p.stride_token;
                }
                const long long o_prev = __shfl_up_sync(0xFFFFFFFFu, o, 1);
                // rows that follow one another in the pool (consecutive slots of one page) travel as one copy: a lane
                // whose row does not continue its predecessor's starts a run and copies all of it
                const bool head = lane < rows_valid && (lane == 0 || o != o_prev + (long long)hd);
                const uint32_t heads = __ballot_sync(0xFFFFFFFFu, head);
                const uint32_t later = lane == 31 ? 0u : heads >> (lane + 1);
                const int run_end = later ? lane + __ffs(later) : rows_valid;
#pragma unroll 1
                for (int sec = 0; sec < 2; sec++) {
                    if (open && (open_rows + rows_total > cfg.cap_rows || open_sub == kWMaxSub)) close_unit();
                    if (!open && !open_unit()) { alive = false; break; }
                    const int fmt = sec ? vf : kf;
                    const uint16_t* pool = sec ? p.v_base : p.k_base;
                    uint8_t* sp = ring + (size_t)stage * cfg.stage_bytes;
                    uint8_t* dst = sp + (size_t)open_rows * row_bytes;
                    if (lane == 0) {
                        WSub m;
                        m.codes = reinterpret_cast<unsigned long long>(sec_codes[sec] + (size_t)t0 * cfg.tok_codes[fmt]);
                        m.scales = reinterpret_cast<unsigned long long>(sec_scales[sec] + (size_t)t0 * cfg.tok_scales[fmt]);
                        m.fmt = fmt; m.rows = rows_total | (rows_valid << 16); m.row0 = open_rows; m.pass0 = open_pass;
                        *reinterpret_cast<WSub*>(sp + off_meta + 16 + 32 * open_sub) = m;
                        if (rows_valid) mbar_expect_tx(&full_bar[stage], (uint32_t)rows_valid * row_bytes);
                    }
                    __syncwarp();
                    if (cfg.heads_contiguous) {
                        if (head) bulk_g2s(dst + (size_t)lane * row_bytes, pool + o, (uint32_t)(run_end - lane) * row_bytes, &full_bar[stage]);
                    } else {
                        for (int ib = 0; ib < rows_valid * p.H; ib += 32) {
                            const int i = ib + lane;
                            const int t = i / p.H, h = i - t * p.H;
                            const long long ot = __shfl_sync(0xFFFFFFFFu, o, t & 31);
                            if (i < rows_valid * p.H)
                                bulk_g2s(dst + (size_t)i * vec_bytes, pool + ot + (long long)h * p.stride_head, vec_bytes, &full_bar[stage]);
                        }
                    }
                    const int piece_passes = (rows_total * cfg.spans_per_row + 31) >> 5;
                    open_ppp = open_sub == 0 ? piece_passes : (open_ppp == piece_passes ? open_ppp : 0);
                    open_rows += rows_total; open_sub++;
                    open_pass += piece_passes;
                    if (open_rows >= cfg.cap_rows) close_unit();
                }
            }
            }
            cur = nxt; cur_n = nxt_n;
        }
        if (open) close_unit();                             // also after a wait gave up: its copies must be able to land
        if (alive) {                                        // tell the consumers that the list is exhausted
            if (__all_sync(0xFFFFFFFFu, mbar_wait(&empty_bar[stage], phase ^ 1, abortp, cfg.wait_limit))) {
                if (lane == 0) {
                    *reinterpret_cast<int4*>(ring + (size_t)stage * cfg.stage_bytes + off_meta) = make_int4(-1, 0, 0, 0);
                    mbar_arrive(&full_bar[stage]);
                }
            } else alive = false;
        }
        if (!alive) {
            // a wait gave up: let the copies already issued land (bounded), so that no bulk copy is still writing
            // this CTA's shared memory after it exits
            const uint32_t issued = q < (uint32_t)S ? q : (uint32_t)S;
            for (uint32_t k = 0; k < issued; k++) {
                const uint32_t qq = q - 1 - k;
                for (uint32_t i = 0; i < cfg.wait_limit; i++) {
                    if (mbar_try_wait(&full_bar[qq % S], (qq / S) & 1)) break;
                    __nanosleep(100);
                }
            }
            if (lane == 0) atomicCAS(p.status, 0, (int)PATCHKV_E_TIMEOUT);
        }
    } else {
        // ================================================================ consumer warps
        const int c = threadIdx.x - 32;
        const int lane = c & 31;
        const int seg = p.G / (8 * NC);                     // lanes per scale group (>= 1: a span never crosses a group)
        const int seg_shift = 31 - __clz(seg);
        const int rot = NC > 1 ? (lane / (8 / NC)) & (NC - 1) : 0;
        int stage = 0;
        uint32_t phase = 0;
        int units_done = 0;
        while (true) {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&full_bar[stage], phase, abortp, cfg.wait_limit))) break;
            const uint32_t src = smem_u32(ring + (size_t)stage * cfg.stage_bytes);
            const uint32_t meta = src + off_meta;
            const uint4 hdr = lds128(meta);
            const int n_sub = (int)hdr.x, n_pass = (int)hdr.y, ppp = (int)hdr.z;
            if (n_sub < 0) break;
#pragma unroll 1
            for (int pass = c >> 5; pass < n_pass; pass += kWPipeConsumerWarps) {
                int i = 0;                                  // the piece this pass belongs to
                if (ppp) {
                    for (int q = pass; q >= ppp; q -= ppp) i++;
                } else {
                    while (i + 1 < n_sub) {
                        int next0;
                        asm volatile("ld.shared.s32 %0, [%1];" : "=r"(next0) : "r"(meta + 16 + 32 * (i + 1) + 28));
                        if (next0 > pass) break;
                        i++;
                    }
                }
                const uint4 m0 = lds128(meta + 16 + 32 * i), m1 = lds128(meta + 32 + 32 * i);
                uint8_t* codes = reinterpret_cast<uint8_t*>(static_cast<uintptr_t>(((unsigned long long)m0.y << 32) | m0.x));
                uint8_t* scales = reinterpret_cast<uint8_t*>(static_cast<uintptr_t>(((unsigned long long)m0.w << 32) | m0.z));
                const int fmt = (int)m1.x;
                const int units = (int)(m1.y & 0xFFFFu) * cfg.spans_per_row, staged = (int)(m1.y >> 16) * cfg.spans_per_row;
                const int u0 = (pass - (int)m1.w) * 32;
                const uint32_t piece = src + (uint32_t)m1.z * (uint32_t)row_bytes;
                if (fmt == FMT_BF16) {
                    // a copy: 16 bytes per lane, lanes side by side
                    const int n16 = units * NC, have16 = staged * NC;
#pragma unroll
                    for (int k = 0; k < NC; k++) {
                        const int w = u0 * NC + 32 * k + lane;
                        if (w < n16)
                            reinterpret_cast<uint4*>(codes)[w] = w < have16 ? lds128(piece + 16u * (uint32_t)w) : make_uint4(0, 0, 0, 0);
                    }
                } else {
                    const uint32_t region = piece + 16u * NC * (uint32_t)u0;
                    if (fmt == FMT_INT8) encode_pass<FMT_INT8, NC>(region, u0, units, staged, codes, scales, seg, seg_shift, rot, lane);
                    else                 encode_pass<FMT_INT4, NC>(region, u0, units, staged, codes, scales, seg, seg_shift, rot, lane);
                }
            }
            // the stage was rewritten with ordinary stores above; order them before the bulk copy that refills it
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            // (self-test: warp 0 keeps one arrival to itself, so that the producer's wait for this stage runs out)
            if (lane == 0 && !(c == 0 && units_done == cfg.stall_after)) mbar_arrive(&empty_bar[stage]);
            units_done++;
            if (++stage == S) { stage = 0; phase ^= 1; }
        }
        if (c == 0 && *abortp) atomicCAS(p.status, 0, (int)PATCHKV_E_TIMEOUT);
    }
    // the last CTA to leave hands the slot of work counters back at zero for the next launch that uses it
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(cfg.sched + 1, 1) == (int)gridDim.x - 1) {
            cfg.sched[0] = 0;
            cfg.sched[1] = 0;
            __threadfence();
        }
    }
}

}  // namespace patchkv

using namespace patchkv;

extern "C" int patchkv_plan_checkpoint(patchkv_ctx* ctx, const patchkv_geom* g, int n_suffix_tokens,
                                       const uint8_t* tags, uint64_t* blk_off, uint64_t* layer_bytes, void* stream) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (!g || g->struct_size != sizeof(patchkv_geom)) return fail(ctx, PATCHKV_E_INVALID, "plan: geometry null or struct_size mismatch");
    if (g->n_layers <= 0 || g->n_layers > 65535 || g->n_kv_heads <= 0 || g->head_dim <= 0 || g->block_tokens <= 0 ||
        g->group <= 0 || g->head_dim % g->group || n_suffix_tokens < 0)
        return fail(ctx, PATCHKV_E_INVALID, "plan: bad geometry");
    if (!layer_bytes) return fail(ctx, PATCHKV_E_INVALID, "plan: null output");
    const int NB = (n_suffix_tokens + g->block_tokens - 1) / g->block_tokens;
    if (NB > 0 && (!tags || !blk_off)) return fail(ctx, PATCHKV_E_INVALID, "plan: null pointer");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    plan_checkpoint_kernel<<<g->n_layers, kPlanThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        tags, NB, (unsigned long long)g->block_tokens * g->n_kv_heads * g->head_dim, g->group,
        reinterpret_cast<unsigned long long*>(blk_off), reinterpret_cast<unsigned long long*>(layer_bytes), ctx->d_status);
    PKV_CUDA(ctx, cudaGetLastError());
    return PATCHKV_OK;
}

namespace patchkv {

// Validates the arguments of a gather and fills the launch parameters (layer_payload / layer range set by the caller).
static int fill_gather(patchkv_ctx* ctx, const patchkv_geom* g, const patchkv_pool* pool, const patchkv_session* s,
                       GatherParams* p, int* nb_out) {
    static thread_local RestoreParams rp;                  // reused only for the shared geometry / pool validation
    int rc = fill_geometry(ctx, g, pool, &rp);
    if (rc != PATCHKV_OK) return rc;
    if (rp.scalar_only)
        return fail(ctx, PATCHKV_E_UNSUPPORTED, "quantize_gather: needs D % 8, G % 8, B*H <= 2048 and record sections that are "
                                                "multiples of 16 bytes");
    if (!s || s->struct_size != sizeof(patchkv_session)) return fail(ctx, PATCHKV_E_INVALID, "session: null or struct_size mismatch");
    if (s->n_suffix_tokens < 0 || s->dst_shift < 0 || s->dst_shift >= g->page_tokens || s->n_table < 0)
        return fail(ctx, PATCHKV_E_INVALID, "session: n_suffix_tokens >= 0, 0 <= dst_shift < P, n_table >= 0");
    const int G = g->group;
    if (!(G == 8 || G == 16 || G == 32 || G == 64 || G == 128 || G == 256))
        return fail(ctx, PATCHKV_E_UNSUPPORTED, "quantize_gather: group must be 8, 16, 32, 64, 128 or 256");
    if (g->block_tokens > 2048) return fail(ctx, PATCHKV_E_UNSUPPORTED, "quantize_gather: block_tokens > 2048");
    const int nb = (s->n_suffix_tokens + g->block_tokens - 1) / g->block_tokens;
    *nb_out = nb;
    if (nb == 0) return PATCHKV_OK;
    if (!s->block_table || !s->tags || !s->blk_off || !s->layer_bytes)
        return fail(ctx, PATCHKV_E_INVALID, "session: null pointer");
    if ((long long)nb * g->n_layers > 0x7fff0000LL) return fail(ctx, PATCHKV_E_UNSUPPORTED, "quantize_gather: too many blocks");
    p->L = g->n_layers; p->H = g->n_kv_heads; p->D = g->head_dim; p->B = g->block_tokens; p->P = g->page_tokens; p->G = G;
    p->k_base = static_cast<const uint16_t*>(pool->k_base);
    p->v_base = static_cast<const uint16_t*>(pool->v_base);
    p->stride_layer = pool->stride_layer; p->stride_page = pool->stride_page;
    p->stride_token = pool->stride_token; p->stride_head = pool->stride_head;
    p->n_pages = pool->n_pages; p->n = s->n_suffix_tokens; p->nb = nb; p->src_shift = s->dst_shift; p->n_table = s->n_table;
    p->layer_begin = 0;
    p->block_table = s->block_table; p->tags = s->tags;
    p->blk_off = reinterpret_cast<const unsigned long long*>(s->blk_off);
    p->layer_payload = const_cast<void* const*>(s->layer_payload);
    p->layer_bytes = reinterpret_cast<const unsigned long long*>(s->layer_bytes);
    p->status = ctx->d_status;
    return PATCHKV_OK;
}

template <int NC>
static cudaError_t launch_wpipe(const GatherParams& p, const WPipeCfg& cfg, int grid, int smem, cudaStream_t stream) {
    cudaError_t e = cudaFuncSetAttribute(quantize_gather_pipe_kernel<NC>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    quantize_gather_pipe_kernel<NC><<<grid, kWPipeThreads, smem, stream>>>(p, cfg);
    return cudaGetLastError();
}

// Launches the block encoder for `layers` layers starting at p.layer_begin.
static int launch_gather(patchkv_ctx* ctx, const patchkv_geom* g, const patchkv_pool* pool, const GatherParams& p,
                         int layers, cudaStream_t stream) {
    // persistent pipeline, two CTAs per SM: stages of about 32 KiB of rows and about 64 KiB of reads in flight per
    // CTA (measured: a third stage costs the 30/50/20 mix of tags 9 % and gains uniform K4/V4 payloads 3 %; stages of
    // 16 KiB cost 3 to 10 %)
    {
        const long long row_bytes = (long long)g->n_kv_heads * g->head_dim * 2;
        const int hc = pool->stride_head == g->head_dim ? 1 : 0;
        const long long pages_per_block = (g->block_tokens + g->page_tokens - 1) / g->page_tokens + 1;
        // a piece: up to 32 tokens of one section of one block; a stage: as many pieces as fit into about 32 KiB
        int ut = (int)std::min<long long>(g->block_tokens, std::max<long long>(1, 32768 / row_bytes));
        ut = std::min(ut, 32);
        const int cap_rows = (int)std::max<long long>(ut, std::min<long long>(32768 / row_bytes, (long long)kWMaxSub * ut));
        const long long stage_bytes = ((long long)cap_rows * row_bytes + kWMetaBytes + 127) & ~127ll;
        const int budget = std::min(ctx->max_smem_optin, 227 * 1024) / 2 - 2048;
        const int n_stages = (int)std::min<long long>(std::min<long long>(kWPipeMaxStages, budget / stage_bytes),
                                                      std::max<long long>(2, (65536 + stage_bytes / 2) / stage_bytes));
        if (!(ctx->flags & PATCHKV_FLAG_DIRECT_LOADS) && row_bytes % 16 == 0 &&
            pages_per_block <= kWPipeMaxPages && n_stages >= 2 && g->group >= 8 && (g->n_kv_heads * g->head_dim) % 32 == 0 &&
            (long long)p.nb * g->block_tokens + g->page_tokens < 0x7fffffffLL) {
            const int nc = g->group >= 32 ? 4 : g->group == 16 ? 2 : 1;
            WPipeCfg cfg;
            cfg.unit_tokens = ut; cfg.cap_rows = cap_rows; cfg.stage_bytes = (int)stage_bytes; cfg.n_stages = n_stages;
            cfg.heads_contiguous = hc;
            cfg.total_items = p.nb * layers;
            cfg.spans_per_row = g->n_kv_heads * g->head_dim / (8 * nc);
            cfg.wait_limit = kWaitLimit; cfg.stall_after = -1;
            if (ctx->selftest_stall_after >= 0) {          // armed by patchkv_selftest_stall_next_launch: this launch only
                cfg.wait_limit = ctx->selftest_wait_limit;
                cfg.stall_after = ctx->selftest_stall_after;
                ctx->selftest_stall_after = -1;
            }
            const uint64_t elems = (uint64_t)g->block_tokens * g->n_kv_heads * g->head_dim, hd = (uint64_t)g->n_kv_heads * g->head_dim;
            for (int f = 0; f < 3; f++) {
                cfg.blk_codes[f] = (uint32_t)code_bytes(f, elems); cfg.blk_scales[f] = (uint32_t)scale_bytes(f, elems, g->group);
                cfg.tok_codes[f] = (uint32_t)code_bytes(f, hd); cfg.tok_scales[f] = (uint32_t)scale_bytes(f, hd, g->group);
            }
            for (int t = 0; t < 4; t++) cfg.rec_bytes[t] = (uint32_t)record_bytes(t, elems, g->group);
            const int smem = (int)(stage_bytes * n_stages);
            const int grid = std::min(cfg.total_items, 2 * ctx->sm_count);
            cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
            PKV_CUDA(ctx, cudaStreamIsCapturing(stream, &cap));
            int slot = 0;
            const int rc = sched_slot(ctx, stream, cap != cudaStreamCaptureStatusNone, &slot);
            if (rc != PATCHKV_OK) return rc;
            cfg.sched = ctx->d_sched + 2 * slot;
            cfg.round_div = 4;
            const cudaError_t e = nc == 4 ? launch_wpipe<4>(p, cfg, grid, smem, stream)
                                : nc == 2 ? launch_wpipe<2>(p, cfg, grid, smem, stream) : launch_wpipe<1>(p, cfg, grid, smem, stream);
            PKV_CUDA(ctx, e);
            return PATCHKV_OK;
        }
    }
    // direct loads: one CTA per (layer, block)
    quantize_gather_kernel<<<p.nb * layers, kGatherThreads, g->block_tokens * sizeof(long long), stream>>>(p);
    PKV_CUDA(ctx, cudaGetLastError());
    return PATCHKV_OK;
}

}  // namespace patchkv

extern "C" int patchkv_quantize_gather(patchkv_ctx* ctx, const patchkv_geom* g, const patchkv_pool* pool,
                                       const patchkv_session* s, void* stream) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    GatherParams p;
    int nb = 0;
    int rc = fill_gather(ctx, g, pool, s, &p, &nb);
    if (rc != PATCHKV_OK || nb == 0) return rc;
    if (!s->layer_payload) return fail(ctx, PATCHKV_E_INVALID, "session: null layer_payload");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    return launch_gather(ctx, g, pool, p, g->n_layers, static_cast<cudaStream_t>(stream));
}

// Offload to a CPU-resident checkpoint: plan, then per layer encode into a device staging slot and copy the finished
// layer payload to pinned host memory on the copy stream while the next layer is being encoded.
extern "C" int patchkv_checkpoint_to_host(patchkv_ctx* ctx, const patchkv_geom* g, const patchkv_pool* pool,
                                          const patchkv_session* s, void* const* host_layer_payload,
                                          const uint64_t* host_layer_capacity, uint64_t* host_layer_bytes,
                                          void* stream_) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (!host_layer_payload || !host_layer_capacity || !host_layer_bytes)
        return fail(ctx, PATCHKV_E_INVALID, "checkpoint_to_host: null host array");
    GatherParams p;
    int nb = 0;
    int rc = fill_gather(ctx, g, pool, s, &p, &nb);
    if (rc != PATCHKV_OK) return rc;
    const int L = g->n_layers;
    if (nb == 0) { for (int l = 0; l < L; l++) host_layer_bytes[l] = 0; return PATCHKV_OK; }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (ctx->host_call_pending) {                           // the ring and the metadata arena may still be in use
        PKV_CUDA(ctx, cudaEventSynchronize(ctx->ev_done));
        ctx->host_call_pending = false;
    }
    // 1. directory of the clustered layout, and its per-layer sizes back on the host (the one synchronisation)
    plan_checkpoint_kernel<<<L, kPlanThreads, 0, stream>>>(
        s->tags, nb, (unsigned long long)g->block_tokens * g->n_kv_heads * g->head_dim, g->group,
        reinterpret_cast<unsigned long long*>(const_cast<uint64_t*>(s->blk_off)),
        reinterpret_cast<unsigned long long*>(const_cast<uint64_t*>(s->layer_bytes)), ctx->d_status);
    PKV_CUDA(ctx, cudaGetLastError());
    rc = ensure_host_workspace(ctx, (size_t)L * 16 + 256, 16);
    if (rc != PATCHKV_OK) return rc;
    uint64_t* h_bytes = reinterpret_cast<uint64_t*>(ctx->h_meta);
    PKV_CUDA(ctx, cudaMemcpyAsync(h_bytes, s->layer_bytes, (size_t)L * 8, cudaMemcpyDeviceToHost, stream));
    PKV_CUDA(ctx, cudaStreamSynchronize(stream));
    size_t slot_bytes = 16;
    for (int l = 0; l < L; l++) {
        host_layer_bytes[l] = h_bytes[l];
        if (h_bytes[l] > host_layer_capacity[l]) return fail(ctx, PATCHKV_E_INVALID, "checkpoint_to_host: host buffer too small");
        if (h_bytes[l] && (!host_layer_payload[l] || (reinterpret_cast<uintptr_t>(host_layer_payload[l]) & 15u)))
            return fail(ctx, PATCHKV_E_INVALID, "checkpoint_to_host: host buffer null or not 16-byte aligned");
        slot_bytes = std::max<size_t>(slot_bytes, h_bytes[l]);
    }
    rc = ensure_host_workspace(ctx, (size_t)L * 16 + 256, slot_bytes);
    if (rc != PATCHKV_OK) return rc;
    const int n_slots = (int)ctx->slots.size();
    // 2. staged layer pointers: layer l encodes into slot l % n_slots
    void** h_ptrs = reinterpret_cast<void**>(ctx->h_meta + (size_t)L * 8);
    for (int l = 0; l < L; l++) h_ptrs[l] = ctx->slots[l % n_slots].base;
    void** d_ptrs = reinterpret_cast<void**>(ctx->d_meta);
    PKV_CUDA(ctx, cudaEventRecord(ctx->ev_begin, stream));
    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_begin, 0));
    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->decode_stream, ctx->ev_begin, 0));
    // From here on work is enqueued on the internal streams; every exit goes through `join`, which makes the caller's
    // stream wait for both of them and marks the ring as in use, also when a later step fails.
    auto join = [&](int code) -> int {
        cudaError_t e = cudaEventRecord(ctx->ev_begin, ctx->decode_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_begin, 0);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_done, ctx->copy_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->ev_done, 0);
        if (e == cudaSuccess) ctx->host_call_pending = true;
        else {
            cudaGetLastError();
            cudaStreamSynchronize(ctx->decode_stream);
            cudaStreamSynchronize(ctx->copy_stream);
            if (code == PATCHKV_OK) code = fail(ctx, PATCHKV_E_CUDA, std::string("checkpoint_to_host: ") + cudaGetErrorString(e));
        }
        return code;
    };
    auto enqueue = [&]() -> int {
    PKV_CUDA(ctx, cudaMemcpyAsync(d_ptrs, h_ptrs, (size_t)L * 8, cudaMemcpyHostToDevice, ctx->decode_stream));
    p.layer_payload = d_ptrs;
    // 3. encode layer l on the decode stream, copy it out on the copy stream; events order slot reuse
    for (int l = 0; l < L; l++) {
        Staging& slot = ctx->slots[l % n_slots];
        if (l >= n_slots) PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->decode_stream, slot.freed, 0));
        p.layer_begin = l;
        rc = launch_gather(ctx, g, pool, p, 1, ctx->decode_stream);
        if (rc != PATCHKV_OK) return rc;
        PKV_CUDA(ctx, cudaEventRecord(slot.copied, ctx->decode_stream));
        PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, slot.copied, 0));
        if (h_bytes[l])
            PKV_CUDA(ctx, cudaMemcpyAsync(host_layer_payload[l], slot.base, h_bytes[l], cudaMemcpyDeviceToHost, ctx->copy_stream));
        PKV_CUDA(ctx, cudaEventRecord(slot.freed, ctx->copy_stream));
    }
    return PATCHKV_OK;
    };
    return join(enqueue());
}

// ---------------------------------------------------------------- precision planner (Eqs. 13-14)
namespace patchkv {

// One thread per block walks its tokens in ascending order with separately rounded fp32 operations, so the tag is
// decided in one fixed precision and order (the same sequence a scalar host program would take).
__global__ void plan_precision_kernel(const float* attn, const float* resid, int n, int B, int NB, float alpha,
                                      float tau_L, float tau_H, float eps4, uint8_t* tags, float* risk) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= NB) return;
    float zmax = 0.0f, zsum = 0.0f, emax = 0.0f;
    int cnt = 0;
    const int e = min(n, (j + 1) * B);
    for (int i = j * B; i < e; i++) {
        const float a = __ldg(attn + i), r = __ldg(resid + i);
        const float z = __fsqrt_rn(__fmul_rn(a, r));
        if (z > zmax) zmax = z;
        if (r > emax) emax = r;
        zsum = __fadd_rn(zsum, z);
        cnt++;
    }
    const float mean = __fdiv_rn(zsum, (float)cnt);
    const float rb = __fadd_rn(__fmul_rn(alpha, zmax), __fmul_rn(__fsub_rn(1.0f, alpha), mean));
    if (risk) risk[j] = rb;
    uint8_t tag;
    if (rb >= tau_H) tag = PATCHKV_TAG_BF16;
    else if (rb >= tau_L) tag = PATCHKV_TAG_INT8;
    else tag = emax <= eps4 ? PATCHKV_TAG_INT4 : PATCHKV_TAG_INT8;
    tags[j] = tag;
}

}  // namespace patchkv

extern "C" int patchkv_plan_precision(patchkv_ctx* ctx, const float* attn, const float* resid, int n_suffix_tokens,
                                      int block_tokens, float alpha, float tau_L, float tau_H, float eps4,
                                      uint8_t* tags, float* risk, void* stream) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (n_suffix_tokens < 0 || block_tokens <= 0 || !(alpha >= 0.0f && alpha <= 1.0f) || !(tau_L < tau_H))
        return fail(ctx, PATCHKV_E_INVALID, "plan_precision: need n >= 0, B > 0, 0 <= alpha <= 1, tau_L < tau_H");
    const int NB = (int)(((long long)n_suffix_tokens + block_tokens - 1) / block_tokens);
    if (NB == 0) return PATCHKV_OK;
    if (!attn || !resid || !tags) return fail(ctx, PATCHKV_E_INVALID, "plan_precision: null pointer");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    plan_precision_kernel<<<(NB + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        attn, resid, n_suffix_tokens, block_tokens, NB, alpha, tau_L, tau_H, eps4, tags, risk);
    PKV_CUDA(ctx, cudaGetLastError());
    return PATCHKV_OK;
}
