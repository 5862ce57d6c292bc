// Checkpoint writer (Section IV-D, offload side): lay out the clustered directory from the tags, then gather
// each block's rows from the paged pool, compute per-group fp16 scales, quantise and pack the record.
// The inverse direction of restore; HBM-bound streaming with a warp-shuffle maximum per scale group.
#include <cuda_fp16.h>

#include <algorithm>

#include "common.cuh"

namespace patchkv {

constexpr int kPlanThreads = 1024;
constexpr int kGatherThreads = 256;

// Exclusive prefix sum of v over a 1024-thread CTA; *total receives the CTA sum.
__device__ __forceinline__ int plan_exclusive_scan(int v, int* warp_sums, int* total) {
    const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= (unsigned)d) inc += o;
    }
    __syncthreads();
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int w = warp_sums[lane];
        int winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xFFFFFFFFu, winc, d);
            if (lane >= (unsigned)d) winc += o;
        }
        warp_sums[lane] = winc - w;
        if (lane == 31) warp_sums[32] = winc;
    }
    __syncthreads();
    *total = warp_sums[32];
    return warp_sums[warp] + inc - v;
}

// One CTA per layer: offsets of the runs [bf16][int8][int4][k4v4], ascending block index inside a run.
__global__ void __launch_bounds__(kPlanThreads)
plan_checkpoint_kernel(const uint8_t* tags, int NB, unsigned long long elems, int group,
                       unsigned long long* blk_off, unsigned long long* layer_bytes, int32_t* status) {
    __shared__ int warp_sums[33];
    const int l = blockIdx.x;
    const uint8_t* tg = tags + (long long)l * NB;
    unsigned long long* off = blk_off + (long long)l * NB;
    unsigned long long base = 0;
    for (int tag = 0; tag <= PATCHKV_TAG_K4V4; tag++) {
        const unsigned long long rec = record_bytes(tag, elems, group);
        int run = 0;
        for (int j0 = 0; j0 < NB; j0 += kPlanThreads) {
            const int j = j0 + threadIdx.x;
            const int mine = j < NB && tg[j] == tag;
            int tot;
            const int rank = plan_exclusive_scan(mine, warp_sums, &tot) + run;
            run += tot;
            if (mine) off[j] = base + (unsigned long long)rank * rec;
        }
        base += (unsigned long long)run * rec;
    }
    bool bad = false;
    for (int j = threadIdx.x; j < NB; j += kPlanThreads)
        if (tg[j] > PATCHKV_TAG_K4V4) { off[j] = ~0ull; bad = true; }
    if (bad) atomicCAS(status, 0, (int)PATCHKV_E_BOUNDS);
    if (threadIdx.x == 0) layer_bytes[l] = base;
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

// NC consecutive 8-channel chunks (8 * NC channels of one head vector, all inside one scale group) per thread: the
// scale arithmetic and the addressing are paid once per 8 * NC elements.  `seg` = lanes per scale group.
template <int FMT, int NC>
__device__ __forceinline__ void encode_span(const uint4* w, uint8_t* codes, uint8_t* scales, size_t elem0,
                                            size_t scale_index, int seg, bool write) {
    if (FMT == FMT_BF16) {
        if (write) {
#pragma unroll
            for (int c = 0; c < NC; c++) reinterpret_cast<uint4*>(codes + 2 * elem0)[c] = w[c];
        }
        return;
    }
    // group maximum straight from the bf16 bit patterns (|x| as an integer compare is monotone for finite values)
    uint32_t amax_bits = 0;
#pragma unroll
    for (int c = 0; c < NC; c++) {
        const uint32_t ww[4] = {w[c].x, w[c].y, w[c].z, w[c].w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            amax_bits = max(amax_bits, (ww[i] << 16) & 0x7FFF0000u);
            amax_bits = max(amax_bits, ww[i] & 0x7FFF0000u);
        }
    }
    for (int d = 1; d < seg; d <<= 1) amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, d));
    const float amax = __uint_as_float(amax_bits);
    const float qmax = FMT == FMT_INT8 ? 127.0f : 7.0f;
    const __half s16 = __float2half_rn(__fdiv_rn(amax, qmax));
    const float s = __half2float(s16);
    const float r = s > 0.0f ? __frcp_rn(s) : 0.0f;
    const float half_s = s > 0.0f ? 0.5f * s : -1.0f;
    const float magic = 12582912.0f;
    const bool subnormal = (__half_as_ushort(s16) & 0x7C00u) == 0 && s > 0.0f;
    const f32x2 r2 = pack2(r, r), m2 = pack2(magic, magic), ns2 = pack2(-s, -s);
    uint32_t out[2 * NC];
#pragma unroll
    for (int c = 0; c < NC; c++) {
        float x[8];
        x[0] = __uint_as_float(w[c].x << 16); x[1] = __uint_as_float(w[c].x & 0xFFFF0000u);
        x[2] = __uint_as_float(w[c].y << 16); x[3] = __uint_as_float(w[c].y & 0xFFFF0000u);
        x[4] = __uint_as_float(w[c].z << 16); x[5] = __uint_as_float(w[c].z & 0xFFFF0000u);
        x[6] = __uint_as_float(w[c].w << 16); x[7] = __uint_as_float(w[c].w & 0xFFFF0000u);
        uint32_t kb[8];
        float df[8];
        bool any_tie = false;
#pragma unroll
        for (int i = 0; i < 8; i += 2) {
            const f32x2 x2 = pack2(x[i], x[i + 1]);
            const f32x2 tm = fma2(x2, r2, m2);
            const f32x2 d2 = fma2(sub2(tm, m2), ns2, x2);
            float a0, a1;
            unpack2(tm, a0, a1);
            kb[i] = __float_as_uint(a0); kb[i + 1] = __float_as_uint(a1);
            unpack2(d2, df[i], df[i + 1]);
            any_tie = any_tie || fabsf(df[i]) == half_s || fabsf(df[i + 1]) == half_s;
        }
        if (any_tie) {
#pragma unroll
            for (int i = 0; i < 8; i++)
                if (fabsf(df[i]) == half_s && (kb[i] & 1u)) kb[i] += df[i] > 0.0f ? 1u : 0xFFFFFFFFu;
        }
        if (subnormal) {
#pragma unroll
            for (int i = 0; i < 8; i++) {
                const float k = fminf(fmaxf(__uint_as_float(kb[i]) - magic, -qmax), qmax);
                kb[i] = __float_as_uint(k + magic);
            }
        }
        out[2 * c] = __byte_perm(__byte_perm(kb[0], kb[1], 0x0040), __byte_perm(kb[2], kb[3], 0x0040), 0x5410);
        out[2 * c + 1] = __byte_perm(__byte_perm(kb[4], kb[5], 0x0040), __byte_perm(kb[6], kb[7], 0x0040), 0x5410);
    }
    if (!write) return;
    if (FMT == FMT_INT8) {
        if (NC == 1) *reinterpret_cast<uint2*>(codes + elem0) = make_uint2(out[0], out[1]);
        else {
#pragma unroll
            for (int c = 0; c < NC / 2; c++)
                reinterpret_cast<uint4*>(codes + elem0)[c] = make_uint4(out[4 * c], out[4 * c + 1], out[4 * c + 2], out[4 * c + 3]);
        }
    } else {
        uint32_t nib[NC];
#pragma unroll
        for (int c = 0; c < NC; c++) {
            uint32_t a = out[2 * c] & 0x0F0F0F0Fu, b = out[2 * c + 1] & 0x0F0F0F0Fu;
            a = (a | (a >> 4)) & 0x00FF00FFu; a = (a | (a >> 8)) & 0x0000FFFFu;
            b = (b | (b >> 4)) & 0x00FF00FFu; b = (b | (b >> 8)) & 0x0000FFFFu;
            nib[c] = a | (b << 16);
        }
        if (NC == 1) *reinterpret_cast<uint32_t*>(codes + (elem0 >> 1)) = nib[0];
        else if (NC == 2) *reinterpret_cast<uint2*>(codes + (elem0 >> 1)) = make_uint2(nib[0], nib[NC - 1]);
        else *reinterpret_cast<uint4*>(codes + (elem0 >> 1)) = make_uint4(nib[0], nib[1 % NC], nib[2 % NC], nib[3 % NC]);
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

// The same block encoder with the block's K and V rows staged in shared memory by bulk asynchronous copies: every
// row of the block is in flight at once (no registers held for loads), and the encode loop reads 16-byte chunks
// from shared memory.  One CTA per (layer, block); three CTAs per SM at the 8B-shaped geometry.
template <int NC>
__global__ void __launch_bounds__(kGatherThreads)
quantize_gather_staged_kernel(const GatherParams p, int sec_bytes, int heads_contiguous) {
    extern __shared__ __align__(128) uint8_t stage[];       // [K rows][V rows][tok_off]
    __shared__ uint64_t bar[2];
    __shared__ int abort_flag;
    long long* tok_off = reinterpret_cast<long long*>(stage + 2 * (size_t)sec_bytes);
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
    if (threadIdx.x == 0) {
        mbar_init(&bar[0], 1); mbar_init(&bar[1], 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int t = threadIdx.x; t < p.B; t += kGatherThreads) {
        long long o = -1;
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
    // ---- stage: valid rows by bulk copies (one per token, or one per (token, head) when heads are strided),
    //      rows past the end of the suffix as zeros
    const int row_bytes = p.H * p.D * 2, vec_bytes = p.D * 2;
    if (threadIdx.x == 0) {
        mbar_arrive_expect_tx(&bar[0], (uint32_t)valid * row_bytes);
        mbar_arrive_expect_tx(&bar[1], (uint32_t)valid * row_bytes);
    }
    const int copies = heads_contiguous ? valid : valid * p.H;
    for (int i = threadIdx.x; i < 2 * copies; i += kGatherThreads) {
        const int sec = i >= copies, c = sec ? i - copies : i;
        const uint16_t* pool = sec ? p.v_base : p.k_base;
        uint8_t* dst = stage + (size_t)sec * sec_bytes;
        if (heads_contiguous) bulk_g2s(dst + (size_t)c * row_bytes, pool + tok_off[c], row_bytes, &bar[sec]);
        else {
            const int t = c / p.H, h = c - t * p.H;
            bulk_g2s(dst + (size_t)c * vec_bytes, pool + tok_off[t] + (long long)h * p.stride_head, vec_bytes, &bar[sec]);
        }
    }
    for (int i = valid * row_bytes / 16 + threadIdx.x; i < sec_bytes / 16; i += kGatherThreads) {
        reinterpret_cast<uint4*>(stage)[i] = make_uint4(0, 0, 0, 0);
        reinterpret_cast<uint4*>(stage + sec_bytes)[i] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();

    const int kf = k_format(tag), vf = v_format(tag);
    uint8_t* kc = base + off;
    uint8_t* ks = kc + code_bytes(kf, elems);
    uint8_t* vc = ks + scale_bytes(kf, elems, p.G);
    uint8_t* vs = vc + code_bytes(vf, elems);
    const int spv = p.D / (8 * NC);                         // spans of 8 * NC channels per head vector
    const int seg = p.G / (8 * NC);                         // lanes per scale group (>= 1: a span never crosses a group)
    const int gpv = p.D / p.G;
    const int seg_shift = 31 - __clz(seg);
    const bool spv_pow2 = (spv & (spv - 1)) == 0;
    const int spv_shift = 31 - __clz(spv);
    const int units = p.B * p.H * spv;                      // spans of one section, in record order
    const int padded = (units + kGatherThreads - 1) / kGatherThreads * kGatherThreads;
    volatile int* abortp = &abort_flag;
#pragma unroll 1
    for (int sec = 0; sec < 2; sec++) {
        // bounded wait for this section's rows; the verdict is CTA-uniform through the shared flag
        const bool ok = mbar_wait(&bar[sec], 0, abortp);
        if (__syncthreads_or(!ok)) {
            if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)PATCHKV_E_TIMEOUT);
            // let the other section's copies land (bounded) before the CTA's shared memory is released
            for (uint32_t i = 0; i < kWaitLimit && !mbar_try_wait(&bar[1], 0); i++) __nanosleep(100);
            return;
        }
        const int fmt = sec ? vf : kf;
        uint8_t* codes = sec ? vc : kc;
        uint8_t* scales = sec ? vs : ks;
        const uint32_t src = smem_u32(stage + (size_t)sec * sec_bytes);
#pragma unroll 1
        for (int u = threadIdx.x; u < padded; u += kGatherThreads) {
            const bool in = u < units;
            uint4 w[NC];
#pragma unroll
            for (int c = 0; c < NC; c++) w[c] = in ? lds128(src + 16u * (uint32_t)(u * NC + c)) : make_uint4(0, 0, 0, 0);
            const int vec = spv_pow2 ? (u >> spv_shift) : u / spv;
            const int sx = u - vec * spv;
            const size_t elem0 = (size_t)u * 8 * NC;
            const size_t sidx = (size_t)vec * gpv + (sx >> seg_shift);
            switch (fmt) {
                case FMT_BF16: encode_span<FMT_BF16, NC>(w, codes, scales, elem0, sidx, seg, in); break;
                case FMT_INT8: encode_span<FMT_INT8, NC>(w, codes, scales, elem0, sidx, seg, in); break;
                default:       encode_span<FMT_INT4, NC>(w, codes, scales, elem0, sidx, seg, in); break;
            }
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
    if ((long long)nb * g->n_layers > 0x7fffffffLL) return fail(ctx, PATCHKV_E_UNSUPPORTED, "quantize_gather: too many blocks");
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

// Launches the block encoder for `layers` layers starting at p.layer_begin.
static int launch_gather(patchkv_ctx* ctx, const patchkv_geom* g, const patchkv_pool* pool, const GatherParams& p,
                         int layers, cudaStream_t stream) {
    // staged variant: both sections of a block in shared memory, at least two CTAs per SM
    const long long sec_bytes = (long long)g->block_tokens * g->n_kv_heads * g->head_dim * 2;
    const long long smem = 2 * sec_bytes + (long long)g->block_tokens * 8 + 16;
    if (!(ctx->flags & PATCHKV_FLAG_DIRECT_LOADS) && smem <= 100 * 1024 && sec_bytes % 16 == 0) {
        const int hc = pool->stride_head == g->head_dim ? 1 : 0;
        // channels per thread: the whole scale group up to 32 channels
        if (g->group >= 32) {
            PKV_CUDA(ctx, cudaFuncSetAttribute(quantize_gather_staged_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            quantize_gather_staged_kernel<4><<<p.nb * layers, kGatherThreads, smem, stream>>>(p, (int)sec_bytes, hc);
        } else if (g->group == 16) {
            PKV_CUDA(ctx, cudaFuncSetAttribute(quantize_gather_staged_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            quantize_gather_staged_kernel<2><<<p.nb * layers, kGatherThreads, smem, stream>>>(p, (int)sec_bytes, hc);
        } else {
            PKV_CUDA(ctx, cudaFuncSetAttribute(quantize_gather_staged_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            quantize_gather_staged_kernel<1><<<p.nb * layers, kGatherThreads, smem, stream>>>(p, (int)sec_bytes, hc);
        }
    } else {
        quantize_gather_kernel<<<p.nb * layers, kGatherThreads, g->block_tokens * sizeof(long long), stream>>>(p);
    }
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
    PKV_CUDA(ctx, cudaEventRecord(ctx->ev_done, ctx->copy_stream));
    PKV_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->ev_done, 0));
    ctx->host_call_pending = true;
    return PATCHKV_OK;
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
