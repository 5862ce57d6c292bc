// Fused restore of reused suffix blocks: dequantise by precision tag, RoPE phase correction of K (Eq. 3),
// placement into destination KV pages through the block table (Section IV-D).  HBM-bound streaming codec:
// no tensor cores, coalesced 128/64/32-bit code loads, 128-bit bf16 stores, persistent grid over block records.
#include <cuda_fp16.h>
#include <math.h>

#include <algorithm>
#include <functional>
#include <thread>

#include "common.cuh"

namespace patchkv {

constexpr int kThreads = 256;
constexpr int kCtasPerSm = 6;

// ---------------------------------------------------------------- conversions
__device__ __forceinline__ float fp16_bits_to_f32(uint16_t h) { return __half2float(__ushort_as_half(h)); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));   // first source -> upper half
    return r;
}
__device__ __forceinline__ uint4 pack8(const float* v) {
    return make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
}

// Eight consecutive channels of one (token, head) vector, as stored.
struct Chunk {
    uint4 w;        // bf16: 16 bytes; int8: x,y; int4: x
    uint16_t s;     // fp16 scale bits (quantised formats)
};

template <int FMT>
__device__ __forceinline__ Chunk load_chunk(const uint8_t* codes, const uint8_t* scales, uint32_t vec, int D,
                                            int groups_per_vec, int c0, int g0) {
    Chunk c;
    c.w = make_uint4(0, 0, 0, 0);
    c.s = 0;
    const size_t e = (size_t)vec * D + c0;
    if (FMT == FMT_BF16) {
        c.w = __ldg(reinterpret_cast<const uint4*>(codes + 2 * e));
    } else if (FMT == FMT_INT8) {
        const uint2 t = __ldg(reinterpret_cast<const uint2*>(codes + e));
        c.w.x = t.x; c.w.y = t.y;
        c.s = __ldg(reinterpret_cast<const uint16_t*>(scales) + (size_t)vec * groups_per_vec + g0);
    } else {
        c.w.x = __ldg(reinterpret_cast<const uint32_t*>(codes + (e >> 1)));
        c.s = __ldg(reinterpret_cast<const uint16_t*>(scales) + (size_t)vec * groups_per_vec + g0);
    }
    return c;
}

template <int FMT>
__device__ __forceinline__ void chunk_to_f32(const Chunk& c, float* v) {
    if (FMT == FMT_BF16) {
        v[0] = __uint_as_float(c.w.x << 16); v[1] = __uint_as_float(c.w.x & 0xFFFF0000u);
        v[2] = __uint_as_float(c.w.y << 16); v[3] = __uint_as_float(c.w.y & 0xFFFF0000u);
        v[4] = __uint_as_float(c.w.z << 16); v[5] = __uint_as_float(c.w.z & 0xFFFF0000u);
        v[6] = __uint_as_float(c.w.w << 16); v[7] = __uint_as_float(c.w.w & 0xFFFF0000u);
    } else {
        // magic-number floats 2^23 + (code + bias); subtracting 2^23 + bias and multiplying by the scale are
        // both exact (< 2^8 times an 11-bit significand), done two lanes at a time
        uint32_t m[8];
        float bias;
        if (FMT == FMT_INT8) {
            const uint32_t x = c.w.x ^ 0x80808080u, y = c.w.y ^ 0x80808080u;
            m[0] = __byte_perm(x, 0x4B000000u, 0x7650); m[1] = __byte_perm(x, 0x4B000000u, 0x7651);
            m[2] = __byte_perm(x, 0x4B000000u, 0x7652); m[3] = __byte_perm(x, 0x4B000000u, 0x7653);
            m[4] = __byte_perm(y, 0x4B000000u, 0x7650); m[5] = __byte_perm(y, 0x4B000000u, 0x7651);
            m[6] = __byte_perm(y, 0x4B000000u, 0x7652); m[7] = __byte_perm(y, 0x4B000000u, 0x7653);
            bias = 8388736.0f;      // 2^23 + 128
        } else {
            const uint32_t x = c.w.x ^ 0x88888888u;
            const uint32_t lo = x & 0x0F0F0F0Fu, hi = (x >> 4) & 0x0F0F0F0Fu;   // even / odd channels
            m[0] = __byte_perm(lo, 0x4B000000u, 0x7650); m[1] = __byte_perm(hi, 0x4B000000u, 0x7650);
            m[2] = __byte_perm(lo, 0x4B000000u, 0x7651); m[3] = __byte_perm(hi, 0x4B000000u, 0x7651);
            m[4] = __byte_perm(lo, 0x4B000000u, 0x7652); m[5] = __byte_perm(hi, 0x4B000000u, 0x7652);
            m[6] = __byte_perm(lo, 0x4B000000u, 0x7653); m[7] = __byte_perm(hi, 0x4B000000u, 0x7653);
            bias = 8388616.0f;      // 2^23 + 8
        }
        const float s = fp16_bits_to_f32(c.s);
        const f32x2 b2 = pack2(bias, bias), s2 = pack2(s, s);
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const f32x2 q = sub2(pack2(__uint_as_float(m[2 * i]), __uint_as_float(m[2 * i + 1])), b2);
            unpack2(mul2(q, s2), v[2 * i], v[2 * i + 1]);
        }
    }
}

// (a, b) -> (a c - b s, a s + b c), every operation rounded on its own.
__device__ __forceinline__ void rotate_pair(float& a, float& b, float c, float s) {
    const float ac = __fmul_rn(a, c), bs = __fmul_rn(b, s), as = __fmul_rn(a, s), bc = __fmul_rn(b, c);
    a = __fsub_rn(ac, bs);
    b = __fadd_rn(as, bc);
}
// The same for eight HALF-style pairs (a[i], b[i]) against (tc[i], ts[i]).  The four products of two pairs are
// formed two lanes per instruction; the sum and the difference stay scalar __fadd_rn / __fsub_rn, which are
// never merged with a multiply (packed add/sub were observed to be contracted with the products).
__device__ __forceinline__ void rotate8_half(float* a, float* b, const float* tc, const float* ts) {
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
        const f32x2 A = pack2(a[i], a[i + 1]), B = pack2(b[i], b[i + 1]);
        const f32x2 C = pack2(tc[i], tc[i + 1]), S = pack2(ts[i], ts[i + 1]);
        float ac0, ac1, bs0, bs1, as0, as1, bc0, bc1;
        unpack2(mul2(A, C), ac0, ac1);
        unpack2(mul2(B, S), bs0, bs1);
        unpack2(mul2(A, S), as0, as1);
        unpack2(mul2(B, C), bc0, bc1);
        a[i] = __fsub_rn(ac0, bs0); a[i + 1] = __fsub_rn(ac1, bs1);
        b[i] = __fadd_rn(as0, bc0); b[i + 1] = __fadd_rn(as1, bc1);
    }
}
// Four INTERLEAVED pairs (v[2i], v[2i+1]) against (tc[i], ts[i]).
__device__ __forceinline__ void rotate4_interleaved(float* v, const float* tc, const float* ts) {
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const f32x2 X = pack2(v[2 * i], v[2 * i + 1]);
        float xc, yc, xs, ys;
        unpack2(mul2(X, pack2(tc[i], tc[i])), xc, yc);
        unpack2(mul2(X, pack2(ts[i], ts[i])), xs, ys);
        v[2 * i] = __fsub_rn(xc, ys);
        v[2 * i + 1] = __fadd_rn(xs, yc);
    }
}

// Which two 8-channel chunks of a head vector a thread owns, and how they rotate.
struct ThreadMap {
    int ty, TY;         // vector lane of this thread, vector lanes per CTA
    int cA, cB;         // first channel of chunk A / chunk B (cB < 0: absent)
    int gA, gB;         // scale group of each chunk
    bool rotA, rotB;    // chunk holds rotary channels (HALF: A and B are partners and rotate together)
    int tab;            // HALF: table index of the first pair; INTERLEAVED: unused
    int t0, h0;         // (token, head) of vector index ty inside a unit, and the step of one loop iteration:
    int dt, dh;         // vector ty + k*TY is (t0 + k*dt + carries, (h0 + k*dh) mod H)
};

// The per-thread channel map, fixed for a launch: `n_threads` threads split into TX = ceil(D / 16) channel lanes times
// TY vector lanes; thread `tid` owns chunk A and chunk B of every vector its lane visits.
template <bool INTER>
__device__ __forceinline__ ThreadMap make_thread_map(const RestoreParams& p, int n_threads, int tid, bool* lane_active) {
    ThreadMap tm;
    const int TX = (p.D + 15) >> 4;
    tm.TY = n_threads / TX;
    const int tx = tid % TX;
    tm.ty = tid / TX;
    *lane_active = tm.ty < tm.TY;
    if (!INTER) {
        const int n_rot = p.Dr >> 4;
        if (tx < n_rot) { tm.cA = 8 * tx; tm.cB = (p.Dr >> 1) + 8 * tx; tm.rotA = tm.rotB = true; tm.tab = 8 * tx; }
        else { tm.cA = p.Dr + 16 * (tx - n_rot); tm.cB = tm.cA + 8; tm.rotA = tm.rotB = false; tm.tab = 0; }
    } else {
        tm.cA = 16 * tx; tm.cB = tm.cA + 8;
        tm.rotA = tm.cA < p.Dr; tm.rotB = tm.cB < p.Dr; tm.tab = 0;
    }
    if (tm.cB >= p.D) { tm.cB = -1; if (INTER) tm.rotB = false; }
    tm.gA = tm.cA / p.G;
    tm.gB = tm.cB >= 0 ? tm.cB / p.G : 0;
    tm.t0 = tm.ty / p.H; tm.h0 = tm.ty - tm.t0 * p.H;
    tm.dt = tm.TY / p.H; tm.dh = tm.TY - tm.dt * p.H;
    return tm;
}

// This thread's eight cos / sin entries of one session's table (HALF: pairs tab .. tab+7; INTERLEAVED: four pairs
// of chunk A, then four of chunk B).
template <bool INTER>
__device__ __forceinline__ void load_rotation(const RestoreParams& p, int session, const ThreadMap& tm, float* tc, float* ts) {
#pragma unroll
    for (int i = 0; i < 8; i++) {
        int idx;
        if (!INTER) idx = tm.tab + i;
        else idx = (i < 4) ? (tm.cA >> 1) + i : ((tm.cB >= 0 ? tm.cB : 0) >> 1) + (i - 4);
        idx = min(idx, PATCHKV_MAX_ROTARY_DIM / 2 - 1);
        tc[i] = p.cs[session][0][idx];
        ts[i] = p.cs[session][1][idx];
    }
}

template <int KF, int VF, bool INTER>
__device__ __forceinline__ void restore_vectors(const RestoreParams& p, const uint8_t* rec, int nvec,
                                                const long long* vec_off, const ThreadMap& tm,
                                                const float* tc, const float* ts, bool rotate) {
    const uint64_t elems = (uint64_t)p.B * p.H * p.D;
    const uint8_t* kc = rec;
    const uint8_t* ks = kc + code_bytes(KF, elems);
    const uint8_t* vc = ks + scale_bytes(KF, elems, p.G);
    const uint8_t* vs = vc + code_bytes(VF, elems);
    const int gpv = p.D / p.G;
    const bool hasB = tm.cB >= 0;
    const bool rotA = rotate && tm.rotA, rotB = rotate && tm.rotB;

#pragma unroll 2
    for (int vec = tm.ty; vec < nvec; vec += tm.TY) {
        const long long off = vec_off[vec];
        Chunk ka = load_chunk<KF>(kc, ks, vec, p.D, gpv, tm.cA, tm.gA);
        Chunk kb = ka, va, vb;
        if (hasB) kb = load_chunk<KF>(kc, ks, vec, p.D, gpv, tm.cB, tm.gB);
        va = load_chunk<VF>(vc, vs, vec, p.D, gpv, tm.cA, tm.gA);
        vb = va;
        if (hasB) vb = load_chunk<VF>(vc, vs, vec, p.D, gpv, tm.cB, tm.gB);

        // ---- K: dequantise, rotate, round once
        uint16_t* kd = p.k_base + off;
        {
            float a[8], b[8];
            chunk_to_f32<KF>(ka, a);
            chunk_to_f32<KF>(kb, b);
            if (!INTER) {
                if (rotA) rotate8_half(a, b, tc, ts);
            } else {
                if (rotA) rotate4_interleaved(a, tc, ts);
                if (rotB) rotate4_interleaved(b, tc + 4, ts + 4);
            }
            // a bf16 code that is not rotated is copied bit for bit
            const uint4 oa = (KF == FMT_BF16 && !rotA) ? ka.w : pack8(a);
            *reinterpret_cast<uint4*>(kd + tm.cA) = oa;
            if (hasB) {
                const uint4 ob = (KF == FMT_BF16 && !rotB) ? kb.w : pack8(b);
                *reinterpret_cast<uint4*>(kd + tm.cB) = ob;
            }
        }
        // ---- V: dequantise and round once; never rotated
        uint16_t* vd = p.v_base + off;
        {
            float a[8];
            uint4 oa = va.w;
            if (VF != FMT_BF16) { chunk_to_f32<VF>(va, a); oa = pack8(a); }
            *reinterpret_cast<uint4*>(vd + tm.cA) = oa;
            if (hasB) {
                uint4 ob = vb.w;
                if (VF != FMT_BF16) { chunk_to_f32<VF>(vb, a); ob = pack8(a); }
                *reinterpret_cast<uint4*>(vd + tm.cB) = ob;
            }
        }
    }
}

template <bool INTER>
__global__ void __launch_bounds__(kThreads)
restore_kernel(const __grid_constant__ RestoreParams p) {
    __shared__ long long vec_off[PATCHKV_MAX_BLOCK_VECTORS];

    bool lane_active;
    const ThreadMap tm = make_thread_map<INTER>(p, kThreads, threadIdx.x, &lane_active);

    float tc[8], ts[8];
    int cur_session = -1;

    for (int item = blockIdx.x; item < p.total_items; item += gridDim.x) {
        int si = 0;
#pragma unroll 1
        for (int k = 1; k < p.n_sessions; k++) if (item >= p.s[k].item_begin) si = k;
        const SessionDev& S = p.s[si];
        const int local = item - S.item_begin;
        const int l = p.layer_begin + local / S.list_nb;
        const int r = local - (l - p.layer_begin) * S.list_nb;
        if (r >= __ldg(S.reuse_cnt + l)) continue;                     // uniform over the CTA

        if (si != cur_session) { cur_session = si; load_rotation<INTER>(p, si, tm, tc, ts); }

        // ---- directory entry of the block; every thread reads the same words (broadcast)
        const int j = __ldg(S.reuse_idx + (size_t)l * S.list_nb + r);
        bool bad = j < 0 || j >= S.nb;
        int tag = 0;
        unsigned long long off = 0, rec = 0, lbytes = 0;
        const uint8_t* base = nullptr;
        if (!bad) {
            tag = __ldg(S.tags + (size_t)l * S.nb + j);
            off = __ldg(S.blk_off + (size_t)l * S.nb + j);
            lbytes = __ldg(S.layer_bytes + l);
            base = reinterpret_cast<const uint8_t*>(
                static_cast<uintptr_t>(__ldg(reinterpret_cast<const unsigned long long*>(S.layer_payload) + l)));
            rec = record_bytes(tag, (uint64_t)p.B * p.H * p.D, p.G);
            bad = rec == 0 || off > lbytes || rec > lbytes - off || base == nullptr ||
                  ((reinterpret_cast<uintptr_t>(base) + off) & 15u) != 0;
        }
        const int valid = bad ? 0 : min(p.B, S.n - j * p.B);
        const int nvec = valid * p.H;

        __syncthreads();                                                // previous item's vec_off no longer in use
        // ---- destination offset of every (token, head) vector; all pages validated before any write
        for (int i = threadIdx.x; i < nvec; i += kThreads) {
            const int t = i / p.H, h = i - t * p.H;
            const long long u = (long long)j * p.B + t + S.dst_shift;
            const long long lp = u / p.P;
            int page = -1;
            if (lp < S.n_table) page = __ldg(S.block_table + lp);
            if (page < 0 || page >= p.n_pages) bad = true;
            vec_off[i] = (long long)l * p.stride_layer + (long long)page * p.stride_page +
                         (u - lp * p.P) * p.stride_token + (long long)h * p.stride_head;
        }
        if (__syncthreads_or(bad)) {                                    // skip the block whole, latch the error
            if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)PATCHKV_E_BOUNDS);
            continue;
        }
        if (!lane_active) continue;

        const uint8_t* recp = base + off;
        const bool rotate = S.delta != 0;
        switch (tag) {
            case PATCHKV_TAG_BF16: restore_vectors<FMT_BF16, FMT_BF16, INTER>(p, recp, nvec, vec_off, tm, tc, ts, rotate); break;
            case PATCHKV_TAG_INT8: restore_vectors<FMT_INT8, FMT_INT8, INTER>(p, recp, nvec, vec_off, tm, tc, ts, rotate); break;
            case PATCHKV_TAG_INT4: restore_vectors<FMT_INT8, FMT_INT4, INTER>(p, recp, nvec, vec_off, tm, tc, ts, rotate); break;
            default:               restore_vectors<FMT_INT4, FMT_INT4, INTER>(p, recp, nvec, vec_off, tm, tc, ts, rotate); break;
        }
    }
}

// ---------------------------------------------------------------- any geometry
// One element (or one rotary pair) per thread, byte and halfword accesses only: the kernel for geometries that the
// vector kernels above and below do not take (head_dim, group or rotary_dim not multiples of 8 / 16, record sections that
// are not multiples of 16 bytes, blocks of more than 2048 (token, head) vectors).  Same arithmetic, same validation,
// same results; speed is not its purpose.
__device__ __forceinline__ float scalar_dequant(int fmt, const uint8_t* codes, const uint8_t* scales, size_t e, size_t sidx,
                                                uint16_t* bits) {
    if (fmt == FMT_BF16) {
        const uint16_t b = (uint16_t)codes[2 * e] | ((uint16_t)codes[2 * e + 1] << 8);
        *bits = b;
        return __uint_as_float((uint32_t)b << 16);
    }
    const uint16_t sb = (uint16_t)scales[2 * sidx] | ((uint16_t)scales[2 * sidx + 1] << 8);
    int q;
    if (fmt == FMT_INT8) q = (int)(int8_t)codes[e];
    else {
        const uint32_t byte = codes[e >> 1];
        const uint32_t nib = (e & 1) ? byte >> 4 : byte & 15u;
        q = (int)(nib ^ 8u) - 8;                        // two's-complement nibble
    }
    return __fmul_rn((float)q, fp16_bits_to_f32(sb));   // exact: at most 8 x 11 significant bits
}
__device__ __forceinline__ uint16_t bf16_bits_rn(float x) { return (uint16_t)(pack_bf16x2(x, 0.0f) & 0xFFFFu); }

template <bool INTER>
__global__ void __launch_bounds__(kThreads)
restore_scalar_kernel(const __grid_constant__ RestoreParams p) {
    pdl_wait();
    const uint64_t elems = (uint64_t)p.B * p.H * p.D;
    const int half = p.Dr >> 1, slots = half + (p.D - p.Dr), gpv = p.D / p.G;
    for (int item = blockIdx.x; item < p.total_items; item += gridDim.x) {
        int si = 0;
#pragma unroll 1
        for (int k = 1; k < p.n_sessions; k++) if (item >= p.s[k].item_begin) si = k;
        const SessionDev& S = p.s[si];
        const int local = item - S.item_begin;
        const int l = p.layer_begin + local / S.list_nb;
        const int r = local - (l - p.layer_begin) * S.list_nb;
        if (r >= __ldg(S.reuse_cnt + l)) continue;                     // uniform over the CTA
        const int j = __ldg(S.reuse_idx + (size_t)l * S.list_nb + r);
        bool bad = j < 0 || j >= S.nb;
        int tag = 0;
        unsigned long long off = 0, rec = 0, lbytes = 0;
        const uint8_t* base = nullptr;
        if (!bad) {
            tag = __ldg(S.tags + (size_t)l * S.nb + j);
            off = __ldg(S.blk_off + (size_t)l * S.nb + j);
            lbytes = __ldg(S.layer_bytes + l);
            base = reinterpret_cast<const uint8_t*>(
                static_cast<uintptr_t>(__ldg(reinterpret_cast<const unsigned long long*>(S.layer_payload) + l)));
            rec = record_bytes(tag, elems, p.G);
            // (no alignment rule here: records of these geometries are not multiples of 16 bytes to begin with)
            bad = rec == 0 || off > lbytes || rec > lbytes - off || base == nullptr;
        }
        const int valid = bad ? 0 : min(p.B, S.n - j * p.B);
        // every destination page is validated before any write
        for (int t = threadIdx.x; t < valid; t += kThreads) {
            const long long u = (long long)j * p.B + t + S.dst_shift;
            const long long lp = u / p.P;
            const int page = lp < S.n_table ? __ldg(S.block_table + lp) : -1;
            if (page < 0 || page >= p.n_pages) bad = true;
        }
        if (__syncthreads_or(bad)) {                                    // skip the block whole, latch the error
            if (threadIdx.x == 0) atomicCAS(p.status, 0, (int)PATCHKV_E_BOUNDS);
            continue;
        }
        const int kf = k_format(tag), vf = v_format(tag);
        const uint8_t* kc = base + off;
        const uint8_t* ks = kc + code_bytes(kf, elems);
        const uint8_t* vc = ks + scale_bytes(kf, elems, p.G);
        const uint8_t* vs = vc + code_bytes(vf, elems);
        const bool rotate = S.delta != 0;
        const long long work = (long long)valid * p.H * slots;
        for (long long w = threadIdx.x; w < work; w += kThreads) {
            const int vec = (int)(w / slots), s = (int)(w - (long long)vec * slots);
            const int t = vec / p.H, h = vec - t * p.H;
            const long long u = (long long)j * p.B + t + S.dst_shift;
            const long long lp = u / p.P;
            const long long dst = (long long)l * p.stride_layer + (long long)__ldg(S.block_table + lp) * p.stride_page +
                                  (u - lp * p.P) * p.stride_token + (long long)h * p.stride_head;
            // the one or two channels of this slot: a rotary pair, or one channel outside the rotary dimension
            int c0, c1 = -1;
            if (s < half) { c0 = INTER ? 2 * s : s; c1 = INTER ? 2 * s + 1 : s + half; }
            else c0 = p.Dr + (s - half);
            const size_t e0 = (size_t)vec * p.D + c0, g0 = (size_t)vec * gpv + c0 / p.G;
            uint16_t kb0 = 0, kb1 = 0, vb0 = 0, vb1 = 0;
            float ka = scalar_dequant(kf, kc, ks, e0, g0, &kb0);
            const float va = scalar_dequant(vf, vc, vs, e0, g0, &vb0);
            p.v_base[dst + c0] = vf == FMT_BF16 ? vb0 : bf16_bits_rn(va);          // V is never rotated
            if (c1 >= 0) {
                const size_t e1 = (size_t)vec * p.D + c1, g1 = (size_t)vec * gpv + c1 / p.G;
                float kbv = scalar_dequant(kf, kc, ks, e1, g1, &kb1);
                const float vb = scalar_dequant(vf, vc, vs, e1, g1, &vb1);
                p.v_base[dst + c1] = vf == FMT_BF16 ? vb1 : bf16_bits_rn(vb);
                if (rotate) {
                    rotate_pair(ka, kbv, p.cs[si][0][s], p.cs[si][1][s]);
                    p.k_base[dst + c0] = bf16_bits_rn(ka);
                    p.k_base[dst + c1] = bf16_bits_rn(kbv);
                } else {                                                    // a bf16 code that is not rotated is copied bit for bit
                    p.k_base[dst + c0] = kf == FMT_BF16 ? kb0 : bf16_bits_rn(ka);
                    p.k_base[dst + c1] = kf == FMT_BF16 ? kb1 : bf16_bits_rn(kbv);
                }
            } else {
                p.k_base[dst + c0] = kf == FMT_BF16 ? kb0 : bf16_bits_rn(ka);
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------- bulk-copy pipeline
// A resolver warp takes rounds of blocks from the global work counter and resolves the directory entry and the
// destination pages of each block one round ahead; an issuing warp stages the resolved blocks into a shared-memory
// ring with bulk asynchronous copies that complete on an mbarrier.  What one copy (one "unit") carries depends on the
// size of the block's record: a record that fits a stage travels whole, K and V sections together, and records of the
// same tag that lie next to each other in the payload (same-tag runs are contiguous in the checkpoint) share a unit and
// a copy; a record larger than a stage is staged one K or V section at a time, a few tokens per unit.
// Eight consumer warps dequantise / rotate from shared memory and write the bf16 rows to the pool with 128-bit
// stores.  Directory latency and HBM read latency are hidden by the ring instead of by occupancy.  Every wait is
// bounded.
constexpr int kPipeConsumers = 256;
constexpr int kPipeProducers = 64;                          // warp 0 feeds the ring, warp 1 resolves the next round of blocks
constexpr int kPipeThreads = kPipeConsumers + kPipeProducers;
constexpr int kMaxStages = 8;
constexpr int kMaxUnitTokens = 128;                         // tokens one unit may carry (rows of its token table)
constexpr int kMaxUnitRecords = 8;                          // records one unit may carry

// Header of a staged unit (32 bytes at the end of the stage).  Section bases are byte offsets from the start of the stage
// for the first record of the unit; a token's table row adds the offset of its own record.
struct StageMeta {
    int32_t nvec;                   // (token, head) vectors in the unit; < 0: no more work
    int32_t fmt;                    // K format | V format << 4
    int32_t flags;                  // bit0: unit holds K rows, bit1: rotate K, bit2: unit holds V rows
    int32_t session;
    uint32_t k_codes, k_scales, v_codes, v_scales;
};
// One row of a unit's token table: where the token's rows go in the pool (element offset without the head term), the byte
// offset of its record inside the unit, and its index inside that record (or inside the staged slice of a section).
struct TokenRow { long long dst; uint32_t rec_off; uint32_t tok; };
constexpr int kMaxItemPages = 8;                            // destination pages one block may touch in this kernel
struct ItemDesc {                                           // one resolved, validated block (valid == 0: nothing to do)
    const uint8_t* rec;
    int32_t valid, tag, l, si, slot0;
    int32_t pages[kMaxItemPages];
};

template <int FMT>
__device__ __forceinline__ Chunk lds_chunk(uint32_t codes, uint32_t scales, int vec, int D, int gpv, int c0, int g0) {
    Chunk c;
    c.w = make_uint4(0, 0, 0, 0);
    c.s = 0;
    const uint32_t e = (uint32_t)vec * D + c0;
    if (FMT == FMT_BF16) {
        c.w = lds128(codes + 2 * e);
    } else if (FMT == FMT_INT8) {
        const uint2 t = lds64(codes + e);
        c.w.x = t.x; c.w.y = t.y;
        c.s = lds16(scales + 2 * ((uint32_t)vec * gpv + g0));
    } else {
        c.w.x = lds32(codes + (e >> 1));
        c.s = lds16(scales + 2 * ((uint32_t)vec * gpv + g0));
    }
    return c;
}

// One section (K or V) of a staged unit: `codes` / `scales` are the shared-memory addresses of the section in the unit's
// first record, `tok_tab` the unit's token table.
template <int FMT, bool INTER>
__device__ __forceinline__ void consume_unit(const RestoreParams& p, uint32_t codes, uint32_t scales,
                                             uint32_t tok_tab, int nvec, uint16_t* dst_base,
                                             const ThreadMap& tm, int gpv, const float* tc, const float* ts, bool rotate) {
    const bool hasB = tm.cB >= 0;
    const bool rotA = rotate && tm.rotA, rotB = rotate && tm.rotB;
    int t = tm.t0, h = tm.h0;                              // (token, head) of `vec`, advanced without divisions
#pragma unroll 1
    for (int vec = tm.ty; vec < nvec; vec += tm.TY) {
        const uint4 row = lds128(tok_tab + 16u * (uint32_t)t);
        const int rv = (int)row.w * p.H + h;               // vector index inside the token's record
        const Chunk ca = lds_chunk<FMT>(codes + row.z, scales + row.z, rv, p.D, gpv, tm.cA, tm.gA);
        Chunk cb = ca;
        if (hasB) cb = lds_chunk<FMT>(codes + row.z, scales + row.z, rv, p.D, gpv, tm.cB, tm.gB);
        uint16_t* d = dst_base + (long long)(((unsigned long long)row.y << 32) | row.x) + (long long)h * p.stride_head;
        t += tm.dt; h += tm.dh;
        if (h >= p.H) { h -= p.H; t++; }
        uint4 oa = ca.w, ob = cb.w;
        if (FMT != FMT_BF16 || rotA || rotB) {
            float a[8], b[8];
            chunk_to_f32<FMT>(ca, a);
            chunk_to_f32<FMT>(cb, b);
            if (!INTER) {
                if (rotA) rotate8_half(a, b, tc, ts);
            } else {
                if (rotA) rotate4_interleaved(a, tc, ts);
                if (rotB) rotate4_interleaved(b, tc + 4, ts + 4);
            }
            if (FMT != FMT_BF16 || rotA) oa = pack8(a);      // a bf16 code that is not rotated is copied bit for bit
            if (FMT != FMT_BF16 || rotB) ob = pack8(b);
        }
        *reinterpret_cast<uint4*>(d + tm.cA) = oa;
        if (hasB) *reinterpret_cast<uint4*>(d + tm.cB) = ob;
    }
}

template <bool INTER>
__global__ void __launch_bounds__(kPipeThreads, 2)
restore_pipe_kernel(const __grid_constant__ RestoreParams p) {
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages];
    __shared__ int abort_flag;
    __shared__ ItemDesc descs[2][32];                    // two rounds of resolved blocks: one being issued, one being resolved
    __shared__ int round_blocks[2];                      // blocks in each round buffer (-1: the work list is exhausted)
    __shared__ uint64_t rfull_bar[2], rempty_bar[2];

    const int S = p.n_stages;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; s++) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kPipeConsumers / 32); }
        for (int b = 0; b < 2; b++) { mbar_init(&rfull_bar[b], 1); mbar_init(&rempty_bar[b], 1); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int off_tab = p.stage_data_bytes;              // stage layout: [data][token table][header]
    const int off_meta = p.stage_bytes - 32;
    volatile int* abortp = &abort_flag;
    // Launched with programmatic stream serialisation: everything above overlaps the tail of the kernel before this
    // one in the stream (usually the selection that writes the reuse lists); nothing below may run before that
    // kernel has completed and its writes are visible.  Without the launch attribute this is a no-op.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (threadIdx.x >= 32 && threadIdx.x < kPipeProducers) {
        // ================================================================ resolver warp
        // Takes rounds of blocks from the global work counter and resolves them one lane per block (directory
        // entry, record extent, destination pages: three dependent global loads), into the round buffer the issuing
        // warp is not reading.  The directory latency of a round is spent while the previous round is being issued.
        // Rounds shrink towards the end of the list (a fraction of what is left per CTA, at most round_cap blocks, at
        // least one) so that CTAs with heavier tags do not leave a long tail; a round is consecutive entries of one list.
        const int lane = threadIdx.x - 32;
        const uint64_t elems = (uint64_t)p.B * p.H * p.D;
        int rb = 0;
        uint32_t rphase = 0;
        // The lookups of a round form a chain of dependent global loads, each a microsecond when the memory system is
        // busy, so the chain is kept short: the first round is dealt out statically (CTA b takes blocks b * r0 ..., the
        // counter hands out what follows), the size of a round comes from the previous claim's answer instead of a
        // fresh read of the counter, and loads that do not depend on one another are issued together (the list entry
        // with the list length; the destination pages with the directory entry).
        const int r0 = (int)max(1ll, min((long long)p.round_cap, (long long)p.total_items / ((long long)p.round_div * gridDim.x)));
        const long long static_items = (long long)r0 * gridDim.x;
        long long seen = static_items;                   // blocks known to be handed out already
        bool first_round = true;
#pragma unroll 1
        while (true) {
            long long first = 0;
            int round = 0;
            if (first_round) {
                first = (long long)blockIdx.x * r0;
                round = r0;
                first_round = false;
            } else {
                if (lane == 0) {
                    const long long left = (long long)p.total_items - seen;
                    round = (int)max(1ll, min((long long)p.round_cap, left / ((long long)p.round_div * gridDim.x)));
                    first = static_items + atomicAdd(p.sched, round);
                }
                first = __shfl_sync(0xFFFFFFFFu, first, 0);
                round = __shfl_sync(0xFFFFFFFFu, round, 0);
                seen = max(seen, first + round);
            }
            ItemDesc d;
            d.valid = 0;
            const long long item = first + lane;
            if (lane < round && item < p.total_items) {
                int si = 0;
#pragma unroll 1
                for (int k = 1; k < p.n_sessions; k++) if (item >= p.s[k].item_begin) si = k;
                const SessionDev& Sd = p.s[si];
                const int local = (int)item - Sd.item_begin;
                const int l = p.layer_begin + local / Sd.list_nb;
                const int r = local - (l - p.layer_begin) * Sd.list_nb;
                // r < list_nb, so the list entry can be read before the list length is known
                const int cnt = __ldg(Sd.reuse_cnt + l);
                const int j = __ldg(Sd.reuse_idx + (size_t)l * Sd.list_nb + r);
                if (r < cnt) {
                    bool bad = j < 0 || j >= Sd.nb;
                    if (!bad) {
                        const int valid = min(p.B, Sd.n - j * p.B);
                        const long long u0 = (long long)j * p.B + Sd.dst_shift;
                        const long long lp0 = u0 / p.P, lp1 = (u0 + valid - 1) / p.P;
                        const int tag = __ldg(Sd.tags + (size_t)l * Sd.nb + j);
                        const unsigned long long off = __ldg(Sd.blk_off + (size_t)l * Sd.nb + j);
                        const unsigned long long lbytes = __ldg(Sd.layer_bytes + l);
                        const uint8_t* base = reinterpret_cast<const uint8_t*>(static_cast<uintptr_t>(
                            __ldg(reinterpret_cast<const unsigned long long*>(Sd.layer_payload) + l)));
                        // every destination page is validated before any write
                        for (long long lp = lp0; lp <= lp1; lp++) {
                            const int page = lp < Sd.n_table ? __ldg(Sd.block_table + lp) : -1;
                            if (page < 0 || page >= p.n_pages) bad = true;
                            d.pages[lp - lp0] = page;
                        }
                        const unsigned long long rbytes = record_bytes(tag, elems, p.G);
                        bad = bad || rbytes == 0 || off > lbytes || rbytes > lbytes - off || base == nullptr ||
                              ((reinterpret_cast<uintptr_t>(base) + off) & 15u) != 0;
                        d.rec = base + off;
                        d.valid = bad ? 0 : valid; d.tag = tag; d.l = l; d.si = si;
                        d.slot0 = (int)(u0 - lp0 * p.P);
                    }
                    if (bad) { d.valid = 0; atomicCAS(p.status, 0, (int)PATCHKV_E_BOUNDS); }
                }
            }
            // hand the round over once the issuing warp has finished with this buffer (bounded, warp-uniform)
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&rempty_bar[rb], rphase ^ 1, abortp, p.wait_limit))) break;
            descs[rb][lane] = d;
            if (lane == 0) round_blocks[rb] = first >= p.total_items ? -1 : round;
            __syncwarp();
            if (lane == 0) mbar_arrive(&rfull_bar[rb]);
            if (first >= p.total_items) break;
            rb ^= 1;
            if (rb == 0) rphase ^= 1;
        }
    } else if (threadIdx.x < 32) {
        // ================================================================ issuing warp
        // Feeds the shared-memory ring from the resolved rounds without touching global memory itself: per unit it
        // waits for a free stage, writes the unit's token table and header, and starts the bulk copy (two for a section
        // of a quantised format: codes and scales).  Lane i keeps block i of the round; a unit of whole records is built
        // by chaining blocks of the round whose records follow one another in the payload.
        const int lane = threadIdx.x;
        uint32_t q = 0;                                  // units issued
        int stage = 0;                                   // q % S, and the parity of q / S, kept without divisions
        uint32_t phase = 0;
        int ib = 0;
        uint32_t iphase = 0;
        bool alive = true;
#pragma unroll 1
        while (alive) {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&rfull_bar[ib], iphase, abortp, p.wait_limit))) { alive = false; break; }
            if (round_blocks[ib] < 0) break;
            const ItemDesc* rd = descs[ib];
            // this lane's block of the round
            const unsigned long long my_rec = reinterpret_cast<unsigned long long>(rd[lane].rec);
            const int my_valid = rd[lane].valid, my_tag = rd[lane].tag, my_l = rd[lane].l, my_si = rd[lane].si;
            uint32_t todo = __ballot_sync(0xFFFFFFFFu, my_valid != 0);
#pragma unroll 1
            while (todo && alive) {
                const int di = __ffs(todo) - 1;
                todo &= todo - 1;
                const ItemDesc& d = rd[di];
                const int valid = d.valid, tag = d.tag, l = d.l, si = d.si;
                const int kf = k_format(tag), vf = v_format(tag);
                const bool shifted = p.s[si].delta != 0;
                const int cap_records = p.unit_records[tag];
                if (cap_records > 0) {
                    // ---- whole records: this block and up to cap_records - 1 blocks of the round that follow it in the
                    //      payload (same tag, same layer and session).  Only the last member may be a partial block.
                    const uint32_t rbytes = p.rec_bytes[tag];
                    int members = 1, tokens = valid;
                    int my_member = lane == 0 ? di : -1;     // lane c remembers member c of the unit
                    unsigned long long want = reinterpret_cast<unsigned long long>(d.rec) + rbytes;
                    bool open = valid == p.B;
#pragma unroll 1
                    while (open && members < cap_records) {
                        const uint32_t hit = __ballot_sync(0xFFFFFFFFu, ((todo >> lane) & 1u) && my_rec == want && my_tag == tag &&
                                                                          my_l == l && my_si == si);
                        if (!hit) break;
                        const int nx = __ffs(hit) - 1;
                        todo &= ~(1u << nx);
                        if (lane == members) my_member = nx;
                        const int nv = __shfl_sync(0xFFFFFFFFu, my_valid, nx);
                        members++;
                        tokens += nv;
                        want += rbytes;
                        open = nv == p.B;
                    }
                    if (!__all_sync(0xFFFFFFFFu, mbar_wait(&empty_bar[stage], phase ^ 1, abortp, p.wait_limit))) { alive = false; break; }
                    uint8_t* sp = ring + (size_t)stage * p.stage_bytes;
                    TokenRow* tab = reinterpret_cast<TokenRow*>(sp + off_tab);
                    for (int i0 = 0; i0 < tokens; i0 += 32) {
                        const int i = i0 + lane;
                        const int m = p.B_shift >= 0 ? i >> p.B_shift : i / p.B;      // member the token belongs to
                        const int src = __shfl_sync(0xFFFFFFFFu, my_member, min(m, members - 1));
                        if (i < tokens) {
                            const ItemDesc& dm = rd[src];
                            const int tr = i - m * p.B;
                            const int us = dm.slot0 + tr;
                            const int pi = p.P_shift >= 0 ? us >> p.P_shift : us / p.P;
                            TokenRow row;
                            row.dst = (long long)l * p.stride_layer + (long long)dm.pages[pi] * p.stride_page +
                                      (long long)(us - pi * p.P) * p.stride_token;
                            row.rec_off = (uint32_t)m * rbytes;
                            row.tok = (uint32_t)tr;
                            tab[i] = row;
                        }
                    }
                    if (lane == 0) {
                        StageMeta m;
                        m.nvec = tokens * p.H; m.fmt = kf | (vf << 4); m.session = si;
                        m.flags = 1 | 4 | (shifted ? 2 : 0);
                        m.k_codes = 0; m.k_scales = p.blk_codes[kf];
                        m.v_codes = m.k_scales + p.blk_scales[kf]; m.v_scales = m.v_codes + p.blk_codes[vf];
                        *reinterpret_cast<StageMeta*>(sp + off_meta) = m;
                    }
                    __syncwarp();
                    if (lane == 0) {
                        const uint32_t bytes = (uint32_t)members * rbytes;
                        mbar_arrive_expect_tx(&full_bar[stage], bytes);
                        bulk_g2s(sp, d.rec, bytes, &full_bar[stage]);
                    }
                    q++;
                    if (++stage == S) { stage = 0; phase ^= 1; }
                    continue;
                }
                // ---- a record larger than a stage: one section at a time, unit_tokens tokens per unit
                const uint8_t* sec_codes[2];
                const uint8_t* sec_scales[2];
                sec_codes[0] = d.rec;
                sec_scales[0] = sec_codes[0] + p.blk_codes[kf];
                sec_codes[1] = sec_scales[0] + p.blk_scales[kf];
                sec_scales[1] = sec_codes[1] + p.blk_codes[vf];
#pragma unroll 1
                for (int sec = 0; sec < 2 && alive; sec++) {
                    const int fmt = sec ? vf : kf;
                    const uint32_t ctok = p.tok_codes[fmt], stok = p.tok_scales[fmt];
#pragma unroll 1
                    for (int t0 = 0; t0 < valid; t0 += p.unit_tokens) {
                        const int nt = min(p.unit_tokens, valid - t0);
                        // the verdict is made warp-uniform: the lanes meet again at __syncwarp below
                        if (!__all_sync(0xFFFFFFFFu, mbar_wait(&empty_bar[stage], phase ^ 1, abortp, p.wait_limit))) { alive = false; break; }
                        uint8_t* sp = ring + (size_t)stage * p.stage_bytes;
                        TokenRow* tab = reinterpret_cast<TokenRow*>(sp + off_tab);
                        for (int i = lane; i < nt; i += 32) {                // one destination row per token
                            const int us = d.slot0 + t0 + i;               // slot counted from the first page
                            const int pi = p.P_shift >= 0 ? us >> p.P_shift : us / p.P;
                            TokenRow row;
                            row.dst = (long long)l * p.stride_layer + (long long)d.pages[pi] * p.stride_page +
                                      (long long)(us - pi * p.P) * p.stride_token;
                            row.rec_off = 0;
                            row.tok = (uint32_t)i;
                            tab[i] = row;
                        }
                        const uint32_t cb = nt * ctok, sb = nt * stok;
                        if (lane == 0) {
                            StageMeta m;
                            m.nvec = nt * p.H; m.fmt = fmt | (fmt << 4); m.session = si;
                            m.flags = sec == 0 ? (1 | (shifted ? 2 : 0)) : 4;
                            m.k_codes = 0; m.k_scales = cb; m.v_codes = 0; m.v_scales = cb;
                            *reinterpret_cast<StageMeta*>(sp + off_meta) = m;
                        }
                        __syncwarp();
                        if (lane == 0) {
                            mbar_arrive_expect_tx(&full_bar[stage], cb + sb);
                            bulk_g2s(sp, sec_codes[sec] + (size_t)t0 * ctok, cb, &full_bar[stage]);
                            if (sb) bulk_g2s(sp + cb, sec_scales[sec] + (size_t)t0 * stok, sb, &full_bar[stage]);
                        }
                        q++;
                        if (++stage == S) { stage = 0; phase ^= 1; }
                    }
                }
            }
            __syncwarp();                                 // every lane is done with this round buffer
            if (lane == 0) mbar_arrive(&rempty_bar[ib]);
            ib ^= 1;
            if (ib == 0) iphase ^= 1;
        }
        // tell the consumers that the work list is exhausted: one empty unit
        if (alive) {
            if (__all_sync(0xFFFFFFFFu, mbar_wait(&empty_bar[stage], phase ^ 1, abortp, p.wait_limit))) {
                if (lane == 0) {
                    StageMeta m;
                    memset(&m, 0, sizeof(m));
                    m.nvec = -1;
                    *reinterpret_cast<StageMeta*>(ring + (size_t)stage * p.stage_bytes + off_meta) = m;
                    mbar_arrive(&full_bar[stage]);
                }
                q++;
                if (++stage == S) { stage = 0; phase ^= 1; }
            } else alive = false;
        }
        if (!alive) {
            // a wait gave up: before leaving, let the copies already issued land (bounded), so that no bulk copy
            // is still writing this CTA's shared memory after it exits
            const uint32_t issued = q < (uint32_t)S ? q : (uint32_t)S;
            for (uint32_t k = 0; k < issued; k++) {
                const uint32_t qq = q - 1 - k;
                for (uint32_t i = 0; i < p.wait_limit; i++) {
                    if (mbar_try_wait(&full_bar[qq % S], (qq / S) & 1)) break;
                    __nanosleep(100);
                }
            }
            if (lane == 0) atomicCAS(p.status, 0, (int)PATCHKV_E_TIMEOUT);
        }
    } else {
        // ================================================================ consumer warps
        // All eight warps work on one unit at a time, in issue order.  (Every waiter has to see every phase of a stage's
        // barriers - a parity wait cannot tell a phase from the one two before it - so the warps are never split into
        // groups that would each visit only some uses of a stage.)
        const int c = threadIdx.x - kPipeProducers;
        bool lane_active;
        const ThreadMap tm = make_thread_map<INTER>(p, kPipeConsumers, c, &lane_active);
        const int gpv = p.D / p.G;
        float tc[8], ts[8];
        int cur_session = -1;
        int stage = 0;
        uint32_t phase = 0;
        int units_done = 0;
        while (true) {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&full_bar[stage], phase, abortp, p.wait_limit))) break;
            uint8_t* sp = ring + (size_t)stage * p.stage_bytes;
            const uint32_t base = smem_u32(sp);
            const uint4 mw = lds128(base + off_meta), mo = lds128(base + off_meta + 16);
            const int nvec = (int)mw.x, fmts = (int)mw.y, flags = (int)mw.z, session = (int)mw.w;
            if (nvec < 0) break;
            if (session != cur_session) { cur_session = session; load_rotation<INTER>(p, cur_session, tm, tc, ts); }
            if (lane_active) {
                const uint32_t tab = base + off_tab;
#pragma unroll 1
                for (int sec = 0; sec < 2; sec++) {
                    if (!(flags & (sec ? 4 : 1))) continue;
                    const int fmt = sec ? fmts >> 4 : fmts & 15;
                    const uint32_t codes = base + (sec ? mo.z : mo.x), scales = base + (sec ? mo.w : mo.y);
                    uint16_t* dst = sec ? p.v_base : p.k_base;
                    const bool rotate = sec == 0 && (flags & 2) != 0;
                    switch (fmt) {
                        case FMT_BF16: consume_unit<FMT_BF16, INTER>(p, codes, scales, tab, nvec, dst, tm, gpv, tc, ts, rotate); break;
                        case FMT_INT8: consume_unit<FMT_INT8, INTER>(p, codes, scales, tab, nvec, dst, tm, gpv, tc, ts, rotate); break;
                        default:       consume_unit<FMT_INT4, INTER>(p, codes, scales, tab, nvec, dst, tm, gpv, tc, ts, rotate); break;
                    }
                }
            }
            __syncwarp();
            // (self-test: the arrivals of one unit are withheld, so that the issuing warp's wait for this stage runs out)
            if ((c & 31) == 0 && units_done != p.stall_after) mbar_arrive(&empty_bar[stage]);
            units_done++;
            if (++stage == S) { stage = 0; phase ^= 1; }
        }
        if (c == 0 && *abortp) atomicCAS(p.status, 0, (int)PATCHKV_E_TIMEOUT);
    }
    // The last CTA to leave hands the slot of work counters back at zero, so the next launch that uses the slot (the
    // next one on the same stream, or the next replay of the same graph node) needs no reset of its own.
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(p.sched + 1, 1) == (int)gridDim.x - 1) {
            p.sched[0] = 0;
            p.sched[1] = 0;
            __threadfence();
        }
    }
}

// ---------------------------------------------------------------- host side
void build_rope_table(const patchkv_geom* g, int delta, float* cos_out, float* sin_out) {
    const int half = g->rotary_dim / 2;
    for (int i = 0; i < half; i++) {
        const double theta = g->inv_freq ? (double)g->inv_freq[i]
                                         : pow(g->rope_base, -2.0 * (double)i / (double)g->rotary_dim);
        const double phi = (double)delta * theta;
        cos_out[i] = (float)cos(phi);
        sin_out[i] = (float)sin(phi);
    }
}

int fill_geometry(patchkv_ctx* ctx, const patchkv_geom* g, const patchkv_pool* pool, RestoreParams* p) {
    if (!g || !pool || g->struct_size != sizeof(patchkv_geom) || pool->struct_size != sizeof(patchkv_pool))
        return fail(ctx, PATCHKV_E_INVALID, "geometry / pool: null or struct_size mismatch");
    if (g->n_layers <= 0 || g->n_kv_heads <= 0 || g->head_dim <= 0 || g->block_tokens <= 0 || g->page_tokens <= 0 ||
        g->group <= 0 || g->rotary_dim < 0 || g->rotary_dim > g->head_dim || (g->head_dim & 1) || (g->rotary_dim & 1) ||
        g->head_dim % g->group != 0)
        return fail(ctx, PATCHKV_E_INVALID, "geometry: need L,H,D,B,P,G > 0, D and Dr even, Dr <= D, G | D");
    if (g->rope_style != PATCHKV_ROPE_HALF && g->rope_style != PATCHKV_ROPE_INTERLEAVED)
        return fail(ctx, PATCHKV_E_INVALID, "geometry: unknown rope_style");
    if (!g->inv_freq && g->rotary_dim > 0 && !(g->rope_base > 0.0))
        return fail(ctx, PATCHKV_E_INVALID, "geometry: rope_base must be positive");
    if (g->rotary_dim > PATCHKV_MAX_ROTARY_DIM)
        return fail(ctx, PATCHKV_E_UNSUPPORTED, "geometry outside kernel limits: rotary_dim <= 256");
    // The vector kernels own 8-channel chunks (one scale per chunk, a rotary chunk and its partner in one thread) and
    // read record sections with 16-byte accesses; anything else goes to the element-wise kernel.
    const int rot_mult = g->rope_style == PATCHKV_ROPE_HALF ? 16 : 8;
    const long long vecs = (long long)g->block_tokens * g->n_kv_heads;
    p->scalar_only = (g->head_dim % 8 || g->group % 8 || g->rotary_dim % rot_mult || vecs > PATCHKV_MAX_BLOCK_VECTORS ||
                      g->head_dim > 16 * kThreads || (vecs * g->head_dim) % 32 != 0 ||
                      (vecs * (g->head_dim / g->group)) % 8 != 0) ? 1 : 0;
    if (!pool->k_base || !pool->v_base || pool->n_pages <= 0)
        return fail(ctx, PATCHKV_E_INVALID, "pool: null base or n_pages <= 0");
    if ((reinterpret_cast<uintptr_t>(pool->k_base) | reinterpret_cast<uintptr_t>(pool->v_base)) & 15u)
        return fail(ctx, PATCHKV_E_INVALID, "pool: bases must be 16-byte aligned");
    if (pool->stride_layer < 0 || pool->stride_page < 0 || pool->stride_token < 0 || pool->stride_head < 0)
        return fail(ctx, PATCHKV_E_INVALID, "pool: strides must be non-negative");
    if ((pool->stride_layer | pool->stride_page | pool->stride_token | pool->stride_head) & 7)
        p->scalar_only = 1;                                // the vector kernels store 16 bytes at a time
    p->L = g->n_layers; p->H = g->n_kv_heads; p->D = g->head_dim; p->Dr = g->rotary_dim; p->rope_style = g->rope_style;
    p->B = g->block_tokens; p->P = g->page_tokens; p->G = g->group;
    p->k_base = static_cast<uint16_t*>(pool->k_base);
    p->v_base = static_cast<uint16_t*>(pool->v_base);
    p->stride_layer = pool->stride_layer; p->stride_page = pool->stride_page;
    p->stride_token = pool->stride_token; p->stride_head = pool->stride_head;
    p->n_pages = pool->n_pages;
    p->status = ctx->d_status;
    return PATCHKV_OK;
}

// Static shared memory of the pipeline kernel (descriptor buffers, barriers), asked of the runtime once.
static long long pipe_static_smem(bool inter) {
    static long long cached[2] = {-1, -1};
    if (cached[inter] < 0) {
        cudaFuncAttributes fa;
        cudaError_t e = inter ? cudaFuncGetAttributes(&fa, restore_pipe_kernel<true>) : cudaFuncGetAttributes(&fa, restore_pipe_kernel<false>);
        if (e != cudaSuccess) { cudaGetLastError(); return 6 * 1024; }
        cached[inter] = (long long)fa.sharedSizeBytes;
    }
    return cached[inter];
}

// Sizes the shared-memory ring for a geometry and decides, per tag, what a unit carries.  Returns false when the
// bulk-copy pipeline does not apply: per-token code / scale runs that are not multiples of 16 bytes, or a token row
// too large for one stage.
static bool plan_pipeline(const patchkv_ctx* ctx, RestoreParams* p) {
    if (ctx->flags & PATCHKV_FLAG_DIRECT_LOADS) return false;
    const long long hd = (long long)p->H * p->D;
    if (hd % 32 != 0 || (hd / p->G) % 8 != 0) return false;
    if ((p->B + p->P - 2) / p->P + 1 > kMaxItemPages) return false;   // pages one block can straddle
    // two CTAs per SM: each may use half of what an SM offers, less its static shared memory (descriptor buffers,
    // barriers) and the 1 KiB the system reserves per CTA
    long long budget = (long long)ctx->smem_per_sm / 2 - pipe_static_smem(p->rope_style == PATCHKV_ROPE_INTERLEAVED) - 1024;
    if (budget > 112 * 1024) budget = 112 * 1024;
    if (budget > ctx->max_smem_optin) budget = ctx->max_smem_optin;
    // Three stages of about 36 KiB each (measured: fewer, larger units beat more, smaller ones as long as three fit).
    long long stage_total = budget / 3 / 128 * 128;
    if (stage_total > 40 * 1024) stage_total = 40 * 1024;
    const uint64_t elems = (uint64_t)p->B * hd;
    for (int f = 0; f < 3; f++) {                     // section sizes per format: no divisions in the issuing warp
        p->blk_codes[f] = (uint32_t)code_bytes(f, elems); p->blk_scales[f] = (uint32_t)scale_bytes(f, elems, p->G);
        p->tok_codes[f] = (uint32_t)code_bytes(f, hd); p->tok_scales[f] = (uint32_t)scale_bytes(f, hd, p->G);
    }
    for (int t = 0; t < 4; t++) p->rec_bytes[t] = (uint32_t)record_bytes(t, elems, p->G);
    // A record that fits the data area of a stage travels whole, and as many records of a same-tag run as fit (at most
    // kMaxUnitRecords, at most kMaxUnitTokens tokens) share a unit; a larger record is staged a section slice at a time.
    // The token table grows with the tokens a unit may carry, so the two sizes are settled together.
    long long rows = std::min<long long>(p->B, kMaxUnitTokens), cap = 0, ut = 0;
    for (int pass = 0; pass < 3; pass++) {
        cap = (stage_total - 32 - 16 * rows) / 16 * 16;
        if (cap < 2 * hd) return false;               // not even one token of a bf16 section
        ut = std::min<long long>(std::min<long long>(p->B, cap / (2 * hd)), std::max<long long>(1, 256 / p->H));
        ut = std::min<long long>(ut, kMaxUnitTokens);
        long long want = ut;
        for (int t = 0; t < 4; t++) {
            long long m = 0;
            if (p->B <= kMaxUnitTokens && (long long)p->rec_bytes[t] <= cap)
                m = std::min<long long>(std::min<long long>(kMaxUnitRecords, cap / p->rec_bytes[t]), kMaxUnitTokens / p->B);
            p->unit_records[t] = (int32_t)m;
            want = std::max(want, m * p->B);
        }
        if (want == rows) break;
        rows = want;
    }
    cap = (stage_total - 32 - 16 * rows) / 16 * 16;
    for (int t = 0; t < 4; t++)
        while (p->unit_records[t] > 0 && ((long long)p->unit_records[t] * p->rec_bytes[t] > cap || (long long)p->unit_records[t] * p->B > rows))
            p->unit_records[t]--;
    if (ut < 1 || 2 * ut * hd > cap || ut > rows) return false;
    p->unit_tokens = (int32_t)ut;
    p->stage_data_bytes = (int32_t)cap;
    p->stage_bytes = (int32_t)((cap + 16 * rows + 32 + 127) / 128 * 128);
    long long stages = budget / p->stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return false;
    p->n_stages = (int32_t)stages;
    p->B_shift = (p->B & (p->B - 1)) == 0 ? 31 - __builtin_clz((unsigned)p->B) : -1;
    p->P_shift = (p->P & (p->P - 1)) == 0 ? 31 - __builtin_clz((unsigned)p->P) : -1;
    // Self-scheduled rounds.  The resolver's chain of dependent lookups (about 5 us under load) has to stay shorter than
    // the time the CTA spends issuing the previous round, so a round carries about 100 KiB of traffic (a block moves
    // about 1.6 x its bf16 size) - measured best at 2 blocks for 64-KiB records, 4 for 32- and 16-KiB records; larger
    // rounds only cost balance, a deeper ring of resolved rounds was slower at every size (it commits work too early).
    // Rounds shrink towards the end of the list: a fraction 1 / round_div of what is left per CTA.
    const long long rec_bf16 = 4ll * p->B * hd;
    const long long traffic = rec_bf16 * 13 / 8;
    long long rcap = (105 * 1024 + traffic - 1) / traffic;
    rcap = std::max<long long>(rcap, rec_bf16 >= 64 * 1024 ? 2 : 4);
    p->round_cap = (int32_t)std::min<long long>(rcap, 32);
    p->round_div = (int32_t)std::max<long long>(2, std::min<long long>(8, rec_bf16 / 8192));
    return true;
}

// The slot of work counters a pipeline launch on `stream` uses.  Launches that share a slot must never overlap on the
// GPU, so a slot belongs to whatever serialises them: the two internal streams (slots 0 and 1), one caller stream each
// (slots 2 ...), or one captured launch (a graph node can be replayed from any stream, next to anything).
int sched_slot(patchkv_ctx* ctx, cudaStream_t stream, bool capturing, int* slot) {
    if (stream == ctx->decode_stream && !capturing) { *slot = 0; return PATCHKV_OK; }
    if (stream == ctx->direct_stream && !capturing) { *slot = 1; return PATCHKV_OK; }
    if (capturing) {
        if (ctx->sched_captured >= kSchedCaptureSlots)
            return fail(ctx, PATCHKV_E_UNSUPPORTED, "too many launches captured into CUDA graphs by this context");
        *slot = kSchedStreamSlots + ctx->sched_captured++;
        return PATCHKV_OK;
    }
    // cudaStreamPerThread is one handle for a different stream in every host thread
    const uint64_t handle = reinterpret_cast<uintptr_t>(stream);
    const uint64_t owner = stream == cudaStreamPerThread ? (uint64_t)std::hash<std::thread::id>()(std::this_thread::get_id()) : 0;
    for (size_t i = 0; i < ctx->sched_streams.size(); i++)
        if (ctx->sched_streams[i].first == handle && ctx->sched_streams[i].second == owner) { *slot = 2 + (int)i; return PATCHKV_OK; }
    if ((int)ctx->sched_streams.size() >= kSchedStreamSlots - 2)
        return fail(ctx, PATCHKV_E_UNSUPPORTED, "this context has been used from too many different streams");
    ctx->sched_streams.emplace_back(handle, owner);
    *slot = 1 + (int)ctx->sched_streams.size();
    return PATCHKV_OK;
}

template <bool INTER>
static int launch_pipe(patchkv_ctx* ctx, RestoreParams* p, int grid, int smem, cudaStream_t stream, bool pdl) {
    PKV_CUDA(ctx, cudaFuncSetAttribute(restore_pipe_kernel<INTER>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kPipeThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
    PKV_CUDA(ctx, cudaLaunchKernelEx(&cfg, restore_pipe_kernel<INTER>, *p));
    return PATCHKV_OK;
}

int launch_restore(patchkv_ctx* ctx, RestoreParams* p, cudaStream_t stream) {
    if (p->total_items <= 0) return PATCHKV_OK;
    const bool inter = p->rope_style == PATCHKV_ROPE_INTERLEAVED;
    if (p->scalar_only) {
        int grid = ctx->sm_count * kCtasPerSm;
        if (grid > p->total_items) grid = p->total_items;
        if (inter) restore_scalar_kernel<true><<<grid, kThreads, 0, stream>>>(*p);
        else restore_scalar_kernel<false><<<grid, kThreads, 0, stream>>>(*p);
        PKV_CUDA(ctx, cudaGetLastError());
        return PATCHKV_OK;
    }
    if (plan_pipeline(ctx, p)) {
        const int smem = p->n_stages * p->stage_bytes;
        int grid = ctx->sm_count * 2;
        if (grid > p->total_items) grid = p->total_items;
        if (p->grid_cap > 0 && grid > p->grid_cap) grid = p->grid_cap;
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        PKV_CUDA(ctx, cudaStreamIsCapturing(stream, &cap));
        const bool capturing = cap != cudaStreamCaptureStatusNone;
        int slot = 0;
        int rc = sched_slot(ctx, stream, capturing, &slot);
        if (rc != PATCHKV_OK) return rc;
        p->sched = ctx->d_sched + 2 * slot;
        p->wait_limit = kWaitLimit;
        p->stall_after = -1;
        if (ctx->selftest_stall_after >= 0) {            // armed by patchkv_selftest_stall_next_launch: this launch only
            p->wait_limit = ctx->selftest_wait_limit;
            p->stall_after = ctx->selftest_stall_after;
            ctx->selftest_stall_after = -1;
        }
        // The kernel's prologue (barrier set-up, thread map, rotation table) may run under the tail of the kernel in
        // front of it in the stream; it waits for that kernel before it touches memory.
        return inter ? launch_pipe<true>(ctx, p, grid, smem, stream, true) : launch_pipe<false>(ctx, p, grid, smem, stream, true);
    }
    int grid = ctx->sm_count * kCtasPerSm;
    if (grid > p->total_items) grid = p->total_items;
    if (inter) restore_kernel<true><<<grid, kThreads, 0, stream>>>(*p);
    else restore_kernel<false><<<grid, kThreads, 0, stream>>>(*p);
    PKV_CUDA(ctx, cudaGetLastError());
    return PATCHKV_OK;
}

}  // namespace patchkv

using namespace patchkv;

extern "C" int patchkv_restore(patchkv_ctx* ctx, const patchkv_geom* geom, const patchkv_pool* pool,
                               const patchkv_session* sessions, int n_sessions, void* stream) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (n_sessions < 0 || n_sessions > PATCHKV_MAX_SESSIONS || (n_sessions > 0 && !sessions))
        return fail(ctx, PATCHKV_E_INVALID, "restore: n_sessions must be 0..PATCHKV_MAX_SESSIONS");
    static thread_local RestoreParams p;
    int rc = fill_geometry(ctx, geom, pool, &p);
    if (rc != PATCHKV_OK) return rc;
    p.n_sessions = n_sessions; p.layer_begin = 0; p.layer_end = geom->n_layers; p.grid_cap = 0;
    long long items = 0;
    for (int i = 0; i < n_sessions; i++) {
        const patchkv_session& s = sessions[i];
        if (s.struct_size != sizeof(patchkv_session)) return fail(ctx, PATCHKV_E_INVALID, "session: struct_size mismatch");
        if (s.n_suffix_tokens < 0 || s.dst_shift < 0 || s.dst_shift >= geom->page_tokens || s.n_table < 0)
            return fail(ctx, PATCHKV_E_INVALID, "session: n_suffix_tokens >= 0, 0 <= dst_shift < P, n_table >= 0");
        const int nb = (s.n_suffix_tokens + geom->block_tokens - 1) / geom->block_tokens;
        if (nb > 0 && (!s.block_table || !s.tags || !s.blk_off || !s.layer_payload || !s.layer_bytes || !s.reuse_idx || !s.reuse_cnt))
            return fail(ctx, PATCHKV_E_INVALID, "session: null pointer");
        SessionDev& d = p.s[i];
        d.block_table = s.block_table; d.tags = s.tags;
        d.blk_off = reinterpret_cast<const unsigned long long*>(s.blk_off);
        d.layer_payload = s.layer_payload;
        d.layer_bytes = reinterpret_cast<const unsigned long long*>(s.layer_bytes);
        d.reuse_idx = s.reuse_idx; d.reuse_cnt = s.reuse_cnt;
        d.n = s.n_suffix_tokens; d.nb = nb; d.list_nb = nb; d.delta = s.delta; d.dst_shift = s.dst_shift; d.n_table = s.n_table;
        d.item_begin = (int32_t)items;
        items += (long long)nb * geom->n_layers;
        if (items > 0x7fff0000LL) return fail(ctx, PATCHKV_E_UNSUPPORTED, "restore: more than 2^31 work items");
        build_rope_table(geom, s.delta, p.cs[i][0], p.cs[i][1]);
    }
    p.total_items = (int32_t)items;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    return launch_restore(ctx, &p, static_cast<cudaStream_t>(stream));
}
