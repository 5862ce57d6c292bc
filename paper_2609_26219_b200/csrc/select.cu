// Repair-set selection (Section IV-B Eq. 9, Section IV-C Eqs. 10-12) at block granularity:
//   1. exact per-block attention mass from stored fp16 attention (integer units of 2^-24, so any reduction
//      order gives the same bits): 128-bit streaming loads, per-thread integer accumulation over rows,
//      warp-shuffle segmented reduction over the octets of a block, one 64-bit atomic per block per CTA;
//   2. per layer one CTA: radix select of the k-th largest candidate mass (8 passes of 8 bits over u64 keys),
//      ties resolved towards the lower block index by a prefix count, then union with the dirty window and
//      prefix-sum compaction into ascending repair / reuse lists.
#include <cuda_fp16.h>

#include "common.cuh"

namespace patchkv {

// ---------------------------------------------------------------- block mass
// Units of 2^-24 of a finite fp16 in [0, 2): exact through fp32 (value * 2^24 <= 2^25 is an integer).
__device__ __forceinline__ uint32_t units2_fast(uint32_t w) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
    return __float2uint_rz(f.x * 16777216.0f) + __float2uint_rz(f.y * 16777216.0f);
}
// Any fp16 bit pattern: negative non-zero / inf / NaN count as zero and raise *bad.
__device__ __forceinline__ unsigned long long units_any(uint32_t h, bool* bad) {
    h &= 0xFFFFu;
    if ((h & 0x7FFFu) == 0) return 0;
    const uint32_t e = (h >> 10) & 31u, m = h & 1023u;
    if ((h & 0x8000u) || e == 31u) { *bad = true; return 0; }
    return e == 0 ? (unsigned long long)m : (unsigned long long)(1024u + m) << (e - 1);
}

struct MassParams {
    const uint16_t* attn;
    long long stride_layer, stride_head, stride_query;
    int Hq, Q, n, B, NB;
    int rows_per_cta;
    unsigned long long* mass;   // [L][NB], zeroed before the launch
    long long mass_stride;      // elements between the rows of two layers (0: every layer adds into one row, which is
                                // the layer-summed mass of LAYERS_SHARED; exact, so the order of the adds is immaterial)
    int32_t* status;
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Exact running sum of one thread's octet over rows, in units of 2^-24.
struct OctetSum {
    unsigned long long acc = 0;
    uint32_t acc32 = 0;
    float facc = 0.0f;
    int n32 = 0, nf = 0;
    bool bad = false;

    __device__ __forceinline__ void add(const uint4& w) {
        const uint32_t any = w.x | w.y | w.z | w.w;
        if ((any & 0xE000E000u) == 0) {
            // every entry in [0, 2^-7): multiples of 2^-24 below 2^-7, so the eight add up exactly in fp32 (< 2^-4)
            // and fifteen such rows still fit 24 bits (< 1): one float->int conversion per 15 rows
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
            const float2 c = __half22float2(*reinterpret_cast<const __half2*>(&w.z));
            const float2 d = __half22float2(*reinterpret_cast<const __half2*>(&w.w));
            facc += ((a.x + a.y) + (b.x + b.y)) + ((c.x + c.y) + (d.x + d.y));
            if (++nf == 15) { acc += __float2uint_rz(facc * 16777216.0f); facc = 0.0f; nf = 0; }
        } else if ((any & 0xC000C000u) == 0 && (any & 0x00003000u) != 0x00003000u && (any & 0x30000000u) != 0x30000000u) {
            // no entry has exponent bits 13 and 12 both set: every entry is in [0, 2^-3), the eight add up exactly in
            // fp32 (< 1, multiples of 2^-24) and one conversion serves the octet.  A warp lands here whenever one lane
            // holds a large attention weight, which is about every other row of a Zipf-shaped map.
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
            const float2 c = __half22float2(*reinterpret_cast<const __half2*>(&w.z));
            const float2 d = __half22float2(*reinterpret_cast<const __half2*>(&w.w));
            acc32 += __float2uint_rz((((a.x + a.y) + (b.x + b.y)) + ((c.x + c.y) + (d.x + d.y))) * 16777216.0f);
            if (++n32 == 8) { acc += acc32; acc32 = 0; n32 = 0; }
        } else if ((any & 0xC000C000u) == 0) {                       // every entry in [0, 2)
            acc32 += units2_fast(w.x) + units2_fast(w.y) + units2_fast(w.z) + units2_fast(w.w);
            if (++n32 == 8) { acc += acc32; acc32 = 0; n32 = 0; }    // 8 * 8 * 2^25 = 2^31
        } else {
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int i = 0; i < 4; i++) acc += units_any(ww[i], &bad) + units_any(ww[i] >> 16, &bad);
        }
    }
    __device__ __forceinline__ unsigned long long total() const {
        return acc + acc32 + __float2uint_rz(facc * 16777216.0f);
    }
};

constexpr int kMassBatch = 8;      // rows whose loads are issued before any of them is consumed

// One thread owns one octet (8 consecutive key positions, all in one block because B % 8 == 0) and walks the
// rows (head, query) assigned to its CTA, eight 128-bit loads in flight at a time.
// grid = (octet tiles, row groups, layers).
__global__ void __launch_bounds__(256)
block_mass_octet_kernel(const MassParams p) {
    pdl_wait();
    pdl_trigger();
    const int oct = blockIdx.x * blockDim.x + threadIdx.x;
    const int col = oct * 8;
    const int l = blockIdx.z;
    const int R = p.Hq * p.Q;
    const int r0 = blockIdx.y * p.rows_per_cta;
    const int r1 = min(R, r0 + p.rows_per_cta);
    const bool in_range = col < p.n;
    const int n_valid = in_range ? min(8, p.n - col) : 0;

    OctetSum sum;
    if (in_range) {
        const uint16_t* base = p.attn + (long long)l * p.stride_layer + col;
        int h = r0 / p.Q, q = r0 - h * p.Q;
        if (n_valid == 8 && p.Q % kMassBatch == 0 && r0 % kMassBatch == 0 && (r1 - r0) % kMassBatch == 0) {
            // regular shape: a batch of eight rows lies inside one head, no wrap test per load
            for (int r = r0; r < r1; r += kMassBatch) {
                const uint16_t* row = base + (long long)h * p.stride_head + (long long)q * p.stride_query;
                q += kMassBatch;
                if (q == p.Q) { q = 0; h++; }
                uint4 w[kMassBatch];
#pragma unroll
                for (int i = 0; i < kMassBatch; i++) w[i] = __ldcs(reinterpret_cast<const uint4*>(row + (long long)i * p.stride_query));
#pragma unroll
                for (int i = 0; i < kMassBatch; i++) sum.add(w[i]);
            }
        } else if (n_valid == 8) {
            for (int r = r0; r < r1; r += kMassBatch) {
                uint4 w[kMassBatch];
#pragma unroll
                for (int i = 0; i < kMassBatch; i++) {
                    w[i] = make_uint4(0, 0, 0, 0);              // a zero row adds nothing
                    if (r + i < r1) {
                        w[i] = __ldcs(reinterpret_cast<const uint4*>(base + (long long)h * p.stride_head +
                                                                     (long long)q * p.stride_query));
                        if (++q == p.Q) { q = 0; h++; }
                    }
                }
#pragma unroll
                for (int i = 0; i < kMassBatch; i++) sum.add(w[i]);
            }
        } else {                                                // ragged last octet of a row: element loads
            for (int r = r0; r < r1; r++) {
                const uint16_t* row = base + (long long)h * p.stride_head + (long long)q * p.stride_query;
                uint16_t e[8];
#pragma unroll
                for (int i = 0; i < 8; i++) e[i] = i < n_valid ? __ldg(row + i) : (uint16_t)0;
                sum.add(make_uint4(e[0] | (uint32_t)e[1] << 16, e[2] | (uint32_t)e[3] << 16,
                                   e[4] | (uint32_t)e[5] << 16, e[6] | (uint32_t)e[7] << 16));
                if (++q == p.Q) { q = 0; h++; }
            }
        }
    }
    if (sum.bad) atomicCAS(p.status, 0, (int)PATCHKV_E_BADINPUT);
    unsigned long long acc = sum.total();

    // segmented reduction over the octets of one block (segments are aligned groups of B/8 lanes)
    const int opb = p.B >> 3;
    const unsigned lane = threadIdx.x & 31u;
    if (opb <= 32 && (opb & (opb - 1)) == 0) {
        for (int d = 1; d < opb; d <<= 1) {
            const unsigned long long o = __shfl_down_sync(0xFFFFFFFFu, acc, d);
            if ((lane & (2 * d - 1)) == 0) acc += o;     // only segment-aligned lanes keep a full sum
        }
        if (in_range && (lane & (opb - 1)) == 0 && acc) atomicAdd(p.mass + (long long)l * p.mass_stride + col / p.B, acc);
    } else if (in_range && acc) {
        atomicAdd(p.mass + (long long)l * p.mass_stride + col / p.B, acc);
    }
}

// Token granularity through a bulk-copy ring (regular shapes: 16-byte aligned rows, Q a multiple of 8, n a multiple of
// 8).  The reads in flight of the kernel below are what its registers hold (eight 128-bit loads per thread at 64
// registers: 32 warps per SM); here a producer warp stages batches of eight rows x 2048 tokens (32 KiB) into a ring
// of three stages with bulk asynchronous copies, so 192 KiB per SM are in flight whatever the consumers need, and the
// eight consumer warps add up from shared memory.  Persistent grid: the launch's (layer, column tile, batch of rows)
// list is cut into one contiguous piece per CTA, so a thread keeps its eight sums in registers across batches and
// goes to memory (one 64-bit atomic per token) only when its piece crosses into another (layer, column tile).
constexpr int kTokPipeConsumers = 256;
constexpr int kTokPipeThreads = kTokPipeConsumers + 32;
constexpr int kTokPipeStages = 3;
constexpr int kTokPipeRows = 8;                                // rows per stage: one batch inside one head
constexpr int kTokPipeCols = 8 * kTokPipeConsumers;            // tokens per column tile
constexpr int kTokPipeStageBytes = kTokPipeRows * kTokPipeCols * 2;

struct TokPipeParams {
    MassParams m;
    int col_tiles;              // ceil(n / kTokPipeCols)
    int batches_per_tile;       // Hq * Q / kTokPipeRows
    long long total_batches;    // L * col_tiles * batches_per_tile
    uint32_t wait_limit;        // polls before a barrier wait gives up
    int32_t stall_after;        // self-test only: consumer warp 0 withholds the `empty` arrival of its batch number
                                // stall_after (-1: never), so that the producer's wait for that stage runs out
};

__global__ void __launch_bounds__(kTokPipeThreads, 2)
token_mass_pipe_kernel(const __grid_constant__ TokPipeParams tp) {
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ uint64_t full_bar[kTokPipeStages], empty_bar[kTokPipeStages];
    __shared__ int abort_flag;
    const MassParams& p = tp.m;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTokPipeStages; s++) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kTokPipeConsumers / 32); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_wait();
    pdl_trigger();
    volatile int* abortp = &abort_flag;
    // this CTA's piece of the batch list
    const long long first = tp.total_batches * blockIdx.x / gridDim.x, last = tp.total_batches * (blockIdx.x + 1) / gridDim.x;
    long long tile = first / tp.batches_per_tile;              // (layer, column tile) index
    int batch = (int)(first - tile * tp.batches_per_tile);
    int l = (int)(tile / tp.col_tiles), ct = (int)(tile - (long long)l * tp.col_tiles);
    const int bpq = p.Q / kTokPipeRows;                        // batches per head

    if (threadIdx.x < 32) {
        // ================================================================ producer warp
        const int lane = threadIdx.x;
        int stage = 0;
        uint32_t phase = 0, issued = 0;
        bool alive = true;
        for (long long i = first; i < last && alive; i++) {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&empty_bar[stage], phase ^ 1, abortp, tp.wait_limit))) { alive = false; break; }
            const int col0 = ct * kTokPipeCols;
            const uint32_t bytes = (uint32_t)min(kTokPipeCols, p.n - col0) * 2u;
            const int h = batch / bpq, q0 = (batch - h * bpq) * kTokPipeRows;
            if (lane == 0) mbar_arrive_expect_tx(&full_bar[stage], bytes * kTokPipeRows);
            __syncwarp();
            if (lane < kTokPipeRows)
                bulk_g2s(ring + (size_t)stage * kTokPipeStageBytes + (size_t)lane * (kTokPipeCols * 2),
                         p.attn + (long long)l * p.stride_layer + (long long)h * p.stride_head +
                             (long long)(q0 + lane) * p.stride_query + col0,
                         bytes, &full_bar[stage]);
            issued++;
            if (++stage == kTokPipeStages) { stage = 0; phase ^= 1; }
            if (++batch == tp.batches_per_tile) { batch = 0; if (++ct == tp.col_tiles) { ct = 0; l++; } }
        }
        if (!alive) {
            // a wait gave up: let the copies already issued land (bounded) before the CTA and its shared memory go
            const uint32_t n_wait = issued < (uint32_t)kTokPipeStages ? issued : (uint32_t)kTokPipeStages;
            for (uint32_t k = 0; k < n_wait; k++) {
                const uint32_t qq = issued - 1 - k;
                for (uint32_t it = 0; it < tp.wait_limit; it++) {
                    if (mbar_try_wait(&full_bar[qq % kTokPipeStages], (qq / kTokPipeStages) & 1)) break;
                    __nanosleep(100);
                }
            }
            if (lane == 0) atomicCAS(p.status, 0, (int)PATCHKV_E_TIMEOUT);
        }
    } else {
        // ================================================================ consumer warps
        // An fp16 below 1/2 is x = u * 2^-24 with u < 2^23, and fma(x, 2^15, 2^14) in fp32 -- one mixed-precision
        // instruction on the fp16 operand, no conversion -- is exactly 2^14 + u * 2^-9: its bit pattern is
        // 0x46800000 + u.  So a token's sum is kept as a 32-bit integer sum of those patterns (one fma per element, one
        // three-input integer add per two elements), and the bias leaves when the sum moves to the token's 64-bit total
        // (after at most 256 rows: the arithmetic is modular and the true partial sum stays below 2^31).  Whether a
        // batch may go this way is decided once per batch: the largest half of its 32 words as an unsigned 16-bit
        // integer (the order of non-negative fp16; a set sign bit counts as large) must be below 0x3800 = 1/2.
        // Otherwise the batch is taken word by word, and a word with an entry of 1/2 or more, a negative, an infinity
        // or a NaN takes the general conversion.
        const int c = threadIdx.x - 32;
        uint32_t a32[8];
        unsigned long long acc[8];
#pragma unroll
        for (int k = 0; k < 8; k++) { a32[k] = 0; acc[k] = 0; }
        uint32_t biased = 0;                                    // rows whose biased patterns a32 holds
        bool bad = false;
        int stage = 0, since_fold = 0;
        uint32_t phase = 0;
        auto pattern2 = [](uint32_t word, uint32_t& p0, uint32_t& p1) {
            unsigned short lo, hi;
            asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(word));
            float t0, t1;
            asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(t0) : "h"(lo), "h"((unsigned short)0x7800), "f"(16384.0f));
            asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(t1) : "h"(hi), "h"((unsigned short)0x7800), "f"(16384.0f));
            p0 = __float_as_uint(t0); p1 = __float_as_uint(t1);
        };
        auto fold = [&]() {
#pragma unroll
            for (int k = 0; k < 8; k++) { acc[k] += (uint32_t)(a32[k] - biased * 0x46800000u); a32[k] = 0; }
            biased = 0; since_fold = 0;
        };
        auto to_memory = [&]() {                                // this thread's eight sums of (l, ct) -> the mass row
            fold();
            const int col = ct * kTokPipeCols + 8 * c;
            if (col < p.n) {
#pragma unroll
                for (int k = 0; k < 8; k++)
                    if (acc[k]) atomicAdd(p.mass + (long long)l * p.mass_stride + col + k, acc[k]);
            }
#pragma unroll
            for (int k = 0; k < 8; k++) acc[k] = 0;
        };
        bool dirty = false;                                     // sums not yet in memory
        for (long long i = first; i < last; i++) {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&full_bar[stage], phase, abortp, tp.wait_limit))) break;
            const uint32_t src = smem_u32(ring + (size_t)stage * kTokPipeStageBytes) + 16u * (uint32_t)c;
            if (ct * kTokPipeCols + 8 * c < p.n) {
                uint4 w[kTokPipeRows];
#pragma unroll
                for (int r = 0; r < kTokPipeRows; r++) w[r] = lds128(src + (uint32_t)r * (kTokPipeCols * 2));
                uint32_t mx = 0;
#pragma unroll
                for (int r = 0; r < kTokPipeRows; r += 2) {
                    mx = __vimax3_u16x2(mx, w[r].x, w[r].y);
                    mx = __vimax3_u16x2(mx, w[r].z, w[r].w);
                    mx = __vimax3_u16x2(mx, w[r + 1].x, w[r + 1].y);
                    mx = __vimax3_u16x2(mx, w[r + 1].z, w[r + 1].w);
                }
                if ((mx & 0xFFFFu) < 0x3800u && (mx >> 16) < 0x3800u) {
#pragma unroll
                    for (int r = 0; r < kTokPipeRows; r += 2) {
                        const uint32_t wa[4] = {w[r].x, w[r].y, w[r].z, w[r].w};
                        const uint32_t wb[4] = {w[r + 1].x, w[r + 1].y, w[r + 1].z, w[r + 1].w};
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            uint32_t a0, a1, b0, b1;
                            pattern2(wa[k], a0, a1);
                            pattern2(wb[k], b0, b1);
                            a32[2 * k] += a0 + b0; a32[2 * k + 1] += a1 + b1;
                        }
                    }
                    biased += kTokPipeRows;
                } else
#pragma unroll
                for (int r = 0; r < kTokPipeRows; r++) {
                    const uint32_t ww[4] = {w[r].x, w[r].y, w[r].z, w[r].w};
                    const uint32_t m4 = __vimax3_u16x2(__vimax3_u16x2(ww[0], ww[1], ww[2]), ww[3], 0u);
                    if ((m4 & 0xFFFFu) < 0x3800u && (m4 >> 16) < 0x3800u) {
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            uint32_t a0, a1;
                            pattern2(ww[k], a0, a1);
                            a32[2 * k] += a0; a32[2 * k + 1] += a1;
                        }
                        biased++;
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; k++) { acc[2 * k] += units_any(ww[k], &bad); acc[2 * k + 1] += units_any(ww[k] >> 16, &bad); }
                    }
                }
            }
            __syncwarp();
            if ((c & 31) == 0 && !(c == 0 && i - first == tp.stall_after)) mbar_arrive(&empty_bar[stage]);
            if (++stage == kTokPipeStages) { stage = 0; phase ^= 1; }
            dirty = true;
            since_fold += kTokPipeRows;
            if (since_fold == 256) fold();
            if (++batch == tp.batches_per_tile) {
                to_memory();
                dirty = false;
                batch = 0;
                if (++ct == tp.col_tiles) { ct = 0; l++; }
            }
        }
        if (dirty) to_memory();
        if (bad) atomicCAS(p.status, 0, (int)PATCHKV_E_BADINPUT);
        if (c == 0 && *abortp) atomicCAS(p.status, 0, (int)PATCHKV_E_TIMEOUT);
    }
}

// Token granularity (the score of Eq. 10 per token): one thread owns eight consecutive tokens and keeps one exact sum
// per token over the rows of its CTA.  Same loads and the same exact-fp32 fast path as the block kernel.
__global__ void __launch_bounds__(256, 4)
token_mass_octet_kernel(const MassParams p) {
    pdl_wait();
    pdl_trigger();
    const int oct = blockIdx.x * blockDim.x + threadIdx.x;
    const int col = oct * 8;
    const int l = blockIdx.z;
    const int R = p.Hq * p.Q;
    const int r0 = blockIdx.y * p.rows_per_cta;
    const int r1 = min(R, r0 + p.rows_per_cta);
    if (col + 8 > p.n) {                                   // ragged tail: element loads
        bool bad = false;
        for (int i = 0; i < 8 && col + i < p.n; i++) {
            unsigned long long acc = 0;
            for (int r = r0; r < r1; r++) {
                const int h = r / p.Q, q = r - h * p.Q;
                acc += units_any(__ldg(p.attn + (long long)l * p.stride_layer + (long long)h * p.stride_head +
                                       (long long)q * p.stride_query + col + i), &bad);
            }
            if (acc) atomicAdd(p.mass + (long long)l * p.mass_stride + col + i, acc);
        }
        if (bad) atomicCAS(p.status, 0, (int)PATCHKV_E_BADINPUT);
        return;
    }
    float facc[8];
    unsigned long long acc[8];
#pragma unroll
    for (int i = 0; i < 8; i++) { facc[i] = 0.0f; acc[i] = 0; }
    int nf = 0;
    bool bad = false;
    const uint16_t* base = p.attn + (long long)l * p.stride_layer + col;
    int h = r0 / p.Q, q = r0 - h * p.Q;
    if (p.Q % kMassBatch == 0 && r0 % kMassBatch == 0 && (r1 - r0) % kMassBatch == 0) {
        // Regular shape (the usual one): a batch of eight rows never straddles a head, so the row pointers are
        // base + i * stride_query with no wrap test per load, and the fp32 sums are flushed by position in the row
        // loop (every 64 rows) instead of by a counter.
        for (int rc = r0; rc < r1; rc += 64) {
            const int re = min(r1, rc + 64);
            for (int r = rc; r < re; r += kMassBatch) {
                const uint16_t* row = base + (long long)h * p.stride_head + (long long)q * p.stride_query;
                q += kMassBatch;
                if (q == p.Q) { q = 0; h++; }
                uint4 w[kMassBatch];
#pragma unroll
                for (int i = 0; i < kMassBatch; i++) w[i] = __ldcs(reinterpret_cast<const uint4*>(row + (long long)i * p.stride_query));
#pragma unroll
                for (int i = 0; i < kMassBatch; i++) {
                    const uint32_t ww[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
                    const uint32_t m = ww[0] | ww[1] | ww[2] | ww[3];
                    if ((m & 0xE000E000u) == 0) {           // every entry below 2^-7: exact in fp32 for 64 rows
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww[k]));
                            facc[2 * k] += f.x; facc[2 * k + 1] += f.y;
                        }
                    } else if ((m & 0xC000C000u) == 0) {    // every entry in [0, 2): value * 2^24 is exact in fp32
#pragma unroll
                        for (int k = 0; k < 4; k++) {
                            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww[k]));
                            acc[2 * k] += __float2uint_rz(f.x * 16777216.0f);
                            acc[2 * k + 1] += __float2uint_rz(f.y * 16777216.0f);
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; k++) { acc[2 * k] += units_any(ww[k], &bad); acc[2 * k + 1] += units_any(ww[k] >> 16, &bad); }
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < 8; k++) { acc[k] += __float2uint_rz(facc[k] * 16777216.0f); facc[k] = 0.0f; }
        }
    } else
    for (int r = r0; r < r1; r += kMassBatch) {
        uint4 w[kMassBatch];
#pragma unroll
        for (int i = 0; i < kMassBatch; i++) {
            w[i] = make_uint4(0, 0, 0, 0);
            if (r + i < r1) {
                w[i] = __ldcs(reinterpret_cast<const uint4*>(base + (long long)h * p.stride_head + (long long)q * p.stride_query));
                if (++q == p.Q) { q = 0; h++; }
            }
        }
#pragma unroll
        for (int i = 0; i < kMassBatch; i++) {
            const uint32_t ww[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
            if (((ww[0] | ww[1] | ww[2] | ww[3]) & 0xE000E000u) == 0) {
                // every entry below 2^-7: 64 such rows add up exactly in fp32 (< 1/2, multiples of 2^-24)
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww[k]));
                    facc[2 * k] += f.x; facc[2 * k + 1] += f.y;
                }
                if (++nf == 64) {
#pragma unroll
                    for (int k = 0; k < 8; k++) { acc[k] += __float2uint_rz(facc[k] * 16777216.0f); facc[k] = 0.0f; }
                    nf = 0;
                }
            } else if (((ww[0] | ww[1] | ww[2] | ww[3]) & 0xC000C000u) == 0) {
                // every entry in [0, 2): value * 2^24 is an integer below 2^25, exact in fp32 (a warp takes this path
                // whenever one of its lanes holds a large attention weight, so it has to stay cheap)
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww[k]));
                    acc[2 * k] += __float2uint_rz(f.x * 16777216.0f);
                    acc[2 * k + 1] += __float2uint_rz(f.y * 16777216.0f);
                }
            } else {
#pragma unroll
                for (int k = 0; k < 4; k++) { acc[2 * k] += units_any(ww[k], &bad); acc[2 * k + 1] += units_any(ww[k] >> 16, &bad); }
            }
        }
    }
    if (bad) atomicCAS(p.status, 0, (int)PATCHKV_E_BADINPUT);
#pragma unroll
    for (int k = 0; k < 8; k++) {
        const unsigned long long v = acc[k] + __float2uint_rz(facc[k] * 16777216.0f);
        if (v) atomicAdd(p.mass + (long long)l * p.mass_stride + col + k, v);
    }
}

// Any B, any strides, any alignment: one thread per key position.
__global__ void __launch_bounds__(256)
block_mass_generic_kernel(const MassParams p) {
    pdl_wait();
    pdl_trigger();
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int l = blockIdx.z;
    const int R = p.Hq * p.Q;
    const int r0 = blockIdx.y * p.rows_per_cta;
    const int r1 = min(R, r0 + p.rows_per_cta);
    if (col >= p.n) return;
    unsigned long long acc = 0;
    bool bad = false;
    for (int r = r0; r < r1; r++) {
        const int h = r / p.Q, q = r - h * p.Q;
        const uint16_t x = __ldg(p.attn + (long long)l * p.stride_layer + (long long)h * p.stride_head +
                                 (long long)q * p.stride_query + col);
        acc += units_any(x, &bad);
    }
    if (bad) atomicCAS(p.status, 0, (int)PATCHKV_E_BADINPUT);
    if (acc) atomicAdd(p.mass + (long long)l * p.mass_stride + col / p.B, acc);
}

__global__ void sum_layers_kernel(const unsigned long long* mass, int L, int NB, unsigned long long* out) {
    pdl_wait();
    pdl_trigger();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= NB) return;
    unsigned long long s = 0;
    int l = 0;
    for (; l + 8 <= L; l += 8) {                         // eight loads in flight, then the adds
        unsigned long long v[8];
#pragma unroll
        for (int u = 0; u < 8; u++) v[u] = mass[(long long)(l + u) * NB + j];
#pragma unroll
        for (int u = 0; u < 8; u++) s += v[u];
    }
    for (; l < L; l++) s += mass[(long long)l * NB + j];
    out[j] = s;
}

// ---------------------------------------------------------------- top-k + union + lists
struct TopkParams {
    const unsigned long long* mass;     // [L][NB], or [NB] when shared
    int shared;                         // 1: every layer ranks on mass[0..NB)
    int spill_keys;                     // candidates the kernel may keep in its dynamic shared memory
    const unsigned int* coarse_hist;    // select_kernel<true>: [rankings][kCoarseCodes] counts of coarse_hist_kernel
    int NB, n_dirty, top_k;
    uint8_t* mask;
    int32_t* repair_idx; int32_t* repair_cnt;
    int32_t* reuse_idx;  int32_t* reuse_cnt;
};

constexpr int kSelThreads = kScanThreads;

// Norm of Eq. 10 as the share of the row total: one CTA per row, exact u64 total, quotient in double, one rounding
// to fp32.  Reported only; the ranking uses the exact masses.
__global__ void __launch_bounds__(256)
normalise_kernel(const unsigned long long* mass, int NB, float* score) {
    pdl_wait();
    pdl_trigger();
    __shared__ unsigned long long part[8];
    const unsigned long long* m = mass + (long long)blockIdx.x * NB;
    unsigned long long t = 0;
    for (int j = threadIdx.x; j < NB; j += 256) t += m[j];
    for (int d = 16; d > 0; d >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, d);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = t;
    __syncthreads();
    unsigned long long total = 0;
#pragma unroll
    for (int w = 0; w < 8; w++) total += part[w];
    const double dt = (double)total;
    for (int j = threadIdx.x; j < NB; j += 256)
        score[(long long)blockIdx.x * NB + j] = total ? (float)__ddiv_rn((double)m[j], dt) : 0.0f;
}

constexpr int kKeysPerThread = 8;      // candidate masses cached in registers: covers NB - n_dirty <= 8192

// ---- ranking many candidates (the tokens of the token-level form): the first cut is made by many CTAs
constexpr int kCoarseCodes = 2048;
constexpr int kSelList = 1024;         // keys of the deciding code that are ranked from a list, one per thread

// A monotone 11-bit code of a 64-bit key: the key itself below 64, else the position of its leading one and the five
// bits under it.  Keys that share a code share every bit down to position `low` (coarse_prefix).
__device__ __forceinline__ unsigned coarse_code(unsigned long long x) {
    if (x < 64ull) return (unsigned)x;
    const int e = 64 - __clzll((long long)x);            // 7 .. 64: x in [2^(e-1), 2^e)
    return 64u + (unsigned)(e - 7) * 32u + ((unsigned)(x >> (e - 6)) & 31u);
}
__device__ __forceinline__ unsigned long long coarse_prefix(unsigned code, int* low) {
    if (code < 64u) { *low = 0; return code; }
    const int e = 7 + (int)((code - 64u) >> 5);
    *low = e - 6;
    return (unsigned long long)(32u + ((code - 64u) & 31u)) << (e - 6);
}

// Histogram of the candidates' coarse codes, one slice of the candidates per CTA: grid = (slices, rankings).  Masses
// spread over many octaves, so the codes spread the keys over many counters; each CTA counts in shared memory and adds
// its non-zero counters to the ranking's row of `hist` (zeroed before the launch).
__global__ void __launch_bounds__(kSelThreads)
coarse_hist_kernel(const unsigned long long* mass, int shared, int NB, int n_dirty, unsigned int* hist) {
    __shared__ unsigned int h[kCoarseCodes];
    pdl_wait();
    pdl_trigger();
    const int r = blockIdx.y;
    const unsigned long long* key = mass + (shared ? 0 : (long long)r * NB);
    const int nd = min(n_dirty, NB), ncand = NB - nd;
    const int per = ((ncand + (int)gridDim.x - 1) / (int)gridDim.x + kSelThreads - 1) / kSelThreads * kSelThreads;
    const int c0 = blockIdx.x * per, c1 = min(ncand, c0 + per);
    for (int i = threadIdx.x; i < kCoarseCodes; i += kSelThreads) h[i] = 0;
    __syncthreads();
    const unsigned lane = threadIdx.x & 31u;
    for (int cb = c0; cb < c1; cb += kSelThreads) {          // (uniform trip count: the ballots below are warp-wide)
        const int c = cb + threadIdx.x;
        const bool live = c < c1;
        const unsigned code = live ? coarse_code(key[nd + c]) : 0u;
        const unsigned act = __ballot_sync(0xFFFFFFFFu, live);
        if (live) {
            const unsigned peers = __match_any_sync(act, code);
            if (lane == (unsigned)(__ffs(peers) - 1)) atomicAdd(&h[code], (unsigned)__popc(peers));
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kCoarseCodes; i += kSelThreads)
        if (h[i]) atomicAdd(hist + (long long)r * kCoarseCodes + i, h[i]);
}

// Radix select, 8 bits per pass from byte `top_byte` down, over the candidates of one CTA: kr[] are the register-cached
// keys, later(c) fetches a candidate of a later round.  After the pass over byte b, *s_prefix holds the bytes >= b of the
// k-th largest key and *s_krem how many keys with that prefix are still to be taken; after the last pass *s_eq is the
// number of keys equal to the k-th largest.  K is the integer type the keys fit (32-bit keys halve the arithmetic).
template <typename K, int KPT, typename Later>
__device__ __forceinline__ void radix_select_passes(const K (&kr)[KPT], Later later, int iters, int ncand, int top_byte,
                                                    unsigned int* hist, unsigned long long* s_prefix, int* s_krem, int* s_eq) {
    const unsigned lane = threadIdx.x & 31u;
    constexpr int kTopByte = (int)sizeof(K) - 1;
    for (int b = top_byte; b >= 0; b--) {
        if (threadIdx.x < 256) hist[threadIdx.x] = 0;
        __syncthreads();
        const K prefix = (K)*s_prefix;
        const int need = *s_krem;
        // In the high bytes most keys share one digit (a long tail of small masses), and thousands of atomics on one
        // counter serialise; a warp whose live lanes all hold the same digit adds its count with one atomic.
        auto count_digit = [&](bool live, K x) {
            const unsigned digit = (unsigned)(x >> (8 * b)) & 255u;
            const unsigned act = __ballot_sync(0xFFFFFFFFu, live);
            if (live) {
                int same;
                __match_all_sync(act, digit, &same);
                if (!same) atomicAdd(&hist[digit], 1u);
                else if (lane == (unsigned)(__ffs(act) - 1)) atomicAdd(&hist[digit], (unsigned)__popc(act));
            }
        };
#pragma unroll
        for (int i = 0; i < KPT; i++) {
            if (i >= iters) break;                   // (uniform) rounds that hold no candidate cost nothing
            const int c = threadIdx.x + i * kSelThreads;
            const K x = kr[i];
            count_digit(c < ncand && (b == kTopByte || ((K)(x ^ prefix) >> (8 * (b + 1))) == 0), x);
        }
        for (int i = KPT; i < iters; i++) {
            const int c = threadIdx.x + i * kSelThreads;
            const K x = c < ncand ? (K)later(c) : (K)0;
            count_digit(c < ncand && (b == kTopByte || ((K)(x ^ prefix) >> (8 * (b + 1))) == 0), x);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane owns the 8 digits 255-8*lane ... 248-8*lane; a warp scan finds the digit where the running
            // count from the top first reaches `need`
            int cnt[8], sum = 0;
#pragma unroll
            for (int t = 0; t < 8; t++) { cnt[t] = (int)hist[255 - 8 * (int)lane - t]; sum += cnt[t]; }
            int inc = sum;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= (unsigned)d) inc += o;
            }
            int cum = inc - sum;
            if (cum < need && need <= inc) {
#pragma unroll
                for (int t = 0; t < 8; t++) {
                    if (cum < need && need <= cum + cnt[t]) {
                        *s_prefix = (unsigned long long)prefix | ((unsigned long long)(255 - 8 * (int)lane - t) << (8 * b));
                        *s_krem = need - cum;
                        *s_eq = cnt[t];              // after the last pass: how many keys equal the k-th largest
                    }
                    cum += cnt[t];
                }
            }
        }
        __syncthreads();
    }
}

// COARSE: the histogram of coarse_hist_kernel makes the first cut, and the few candidates that share the code of the k-th
// largest key are ranked from a list in shared memory, one key per thread; the passes over all candidates remain for
// masses so full of ties that the list would overflow.  (A separate instantiation, so that the kernel of the block form,
// which runs under the restore kernel's CTAs, keeps its small shared-memory footprint.)
template <bool COARSE>
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const TopkParams p) {
    // Candidates cached in registers per thread.  The many-candidate instantiation keeps one and reads the rest from
    // shared memory: it runs as a single CTA that executes its code once, cold, and the loops over register-cached
    // rounds are unrolled code that would have to be fetched instruction by instruction.
    constexpr int KPT = COARSE ? 1 : kKeysPerThread;
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long s_list[COARSE ? kSelList : 1];
    __shared__ int s_code, s_list_n;
    __shared__ int warp_sums[33];
    __shared__ unsigned long long s_prefix;
    __shared__ int s_krem, s_eq;
    __shared__ unsigned int s_or[2];

    // The kernel that follows in the stream (the restore, launched with programmatic stream serialisation) may be
    // brought onto the SMs now; it still waits for this grid to finish before it reads the lists written here.
    pdl_wait();
    pdl_trigger();
    extern __shared__ unsigned long long spill[];        // candidates beyond the register-cached ones (p.spill_keys of them)
    const int l = blockIdx.x;
    const unsigned long long* key = p.mass + (p.shared ? 0 : (long long)l * p.NB);
    const int NB = p.NB, n_dirty = min(p.n_dirty, NB);
    const int ncand = NB - n_dirty;
    const int k = min(p.top_k, ncand);
    const bool take_all = k == ncand, take_none = k == 0;
    const int iters = (ncand + kSelThreads - 1) / kSelThreads;
    const unsigned lane = threadIdx.x & 31u;

    // candidate c = threadIdx.x + i * kSelThreads is block n_dirty + c; the first KPT rounds live in registers,
    // the next p.spill_keys candidates in shared memory, anything beyond that is re-read from global memory
    unsigned long long kreg[KPT];
#pragma unroll
    for (int i = 0; i < KPT; i++) {
        const int c = threadIdx.x + i * kSelThreads;
        kreg[i] = c < ncand ? key[n_dirty + c] : 0ull;
    }
    const int reg_keys = KPT * kSelThreads;
    {
        // eight loads in flight per thread: the copy into shared memory is a chain of global-memory latencies otherwise
        const int spill_end = min(ncand, reg_keys + p.spill_keys);
        for (int c0 = reg_keys + threadIdx.x; c0 < spill_end; c0 += 8 * kSelThreads) {
            unsigned long long v[8];
#pragma unroll
            for (int u = 0; u < 8; u++) {
                const int c = c0 + u * kSelThreads;
                v[u] = c < spill_end ? key[n_dirty + c] : 0ull;
            }
#pragma unroll
            for (int u = 0; u < 8; u++) {
                const int c = c0 + u * kSelThreads;
                if (c < spill_end) spill[c - reg_keys] = v[u];
            }
        }
    }
    auto later_key = [&](int c) -> unsigned long long {      // a candidate of a later round (a thread reads back its own writes only)
        return c - reg_keys < p.spill_keys ? spill[c - reg_keys] : key[n_dirty + c];
    };

    unsigned long long T = 0;
    int krem = 0, n_eq = 0;                      // keys equal to T: krem of them are taken, n_eq exist
    bool ranked = take_all || take_none;
    if (COARSE && !ranked) {
        // thread t owns the codes 2047 - 2t and 2046 - 2t; a scan from the top finds the code where the count reaches k
        const unsigned int* ch = p.coarse_hist + (long long)l * kCoarseCodes;
        const int c0 = (int)ch[kCoarseCodes - 1 - 2 * (int)threadIdx.x], c1 = (int)ch[kCoarseCodes - 2 - 2 * (int)threadIdx.x];
        if (threadIdx.x == 0) s_list_n = 0;
        int tot;
        int cum = cta_exclusive_scan(c0 + c1, warp_sums, &tot);
        if (cum < k && k <= cum + c0) { s_code = kCoarseCodes - 1 - 2 * (int)threadIdx.x; s_krem = k - cum; s_eq = c0; }
        cum += c0;
        if (cum < k && k <= cum + c1) { s_code = kCoarseCodes - 2 - 2 * (int)threadIdx.x; s_krem = k - cum; s_eq = c1; }
        __syncthreads();
        const unsigned code_k = (unsigned)s_code;
        const int n_code = s_eq;                         // candidates that share the code of the k-th largest
        int low = 0;                                     // bits of the k-th largest key not known yet
        const unsigned long long prefix0 = coarse_prefix(code_k, &low);
        if (low == 0 || n_code <= kSelList) {
            if (low > 0) {
#pragma unroll
                for (int i = 0; i < KPT; i++) {
                    if (i >= iters) break;
                    if (threadIdx.x + i * kSelThreads < ncand && coarse_code(kreg[i]) == code_k) s_list[atomicAdd(&s_list_n, 1)] = kreg[i];
                }
                for (int i = KPT; i < iters; i++) {
                    const int c = threadIdx.x + i * kSelThreads;
                    if (c < ncand) {
                        const unsigned long long x = later_key(c);
                        if (coarse_code(x) == code_k) s_list[atomicAdd(&s_list_n, 1)] = x;
                    }
                }
            }
            if (threadIdx.x == 0) s_prefix = prefix0;
            __syncthreads();
            const bool have = (int)threadIdx.x < n_code && low > 0;
            const unsigned long long mine = have ? s_list[threadIdx.x] : 0ull;
            if (low > 0 && n_code <= 256) {
                // a short list is ranked directly: the key that has exactly need - 1 keys in front of it (larger, or equal
                // and earlier in the list) is the k-th largest; three barriers instead of three per radix pass
                const int need = s_krem;
                int front = 0;
                if (have)
                    for (int j = 0; j < n_code; j++) {
                        const unsigned long long x = s_list[j];
                        front += (x > mine || (x == mine && j < (int)threadIdx.x)) ? 1 : 0;
                    }
                if (have && front == need - 1) s_prefix = mine;
                __syncthreads();
                const unsigned long long kth = s_prefix;
                const int larger = __syncthreads_count(have && mine > kth);
                const int equal = __syncthreads_count(have && mine == kth);
                T = kth; krem = need - larger; n_eq = equal;
                low = 0;
                ranked = true;
            }
            // radix select over the remaining bits of the listed keys, up to 8 per pass from the top
            while (low > 0) {
                const int width = min(8, low), shift = low - width;
                if (threadIdx.x < 256) hist[threadIdx.x] = 0;
                __syncthreads();
                const unsigned long long prefix = s_prefix;
                const int need = s_krem;
                if (have && ((mine ^ prefix) >> low) == 0) atomicAdd(&hist[(unsigned)(mine >> shift) & ((1u << width) - 1u)], 1u);
                __syncthreads();
                if (threadIdx.x < 32) {
                    int cnt[8], sum = 0;
#pragma unroll
                    for (int t = 0; t < 8; t++) { cnt[t] = (int)hist[255 - 8 * (int)lane - t]; sum += cnt[t]; }
                    int inc = sum;
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        const int o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                        if (lane >= (unsigned)d) inc += o;
                    }
                    int cm = inc - sum;
                    if (cm < need && need <= inc) {
#pragma unroll
                        for (int t = 0; t < 8; t++) {
                            if (cm < need && need <= cm + cnt[t]) {
                                s_prefix = prefix | ((unsigned long long)(255 - 8 * (int)lane - t) << shift);
                                s_krem = need - cm;
                                s_eq = cnt[t];
                            }
                            cm += cnt[t];
                        }
                    }
                }
                __syncthreads();
                low = shift;
            }
            if (!ranked) { T = s_prefix; krem = s_krem; n_eq = s_eq; }
            ranked = true;
        }
        __syncthreads();                                 // (the shared words are set again below)
    }
    if (!ranked) {
        // highest byte that is non-zero in any candidate: the passes above it would all pick digit 0
        unsigned long long orv = 0;
#pragma unroll
        for (int i = 0; i < KPT; i++) orv |= kreg[i];
        for (int i = KPT; i < iters; i++) {
            const int c = threadIdx.x + i * kSelThreads;
            if (c < ncand) orv |= later_key(c);
        }
        if (threadIdx.x == 0) { s_or[0] = 0; s_or[1] = 0; s_prefix = 0; s_krem = k; s_eq = ncand; }
        __syncthreads();
        const unsigned lo = __reduce_or_sync(0xFFFFFFFFu, (unsigned)orv);
        const unsigned hi = __reduce_or_sync(0xFFFFFFFFu, (unsigned)(orv >> 32));
        if (lane == 0) { if (lo) atomicOr(&s_or[0], lo); if (hi) atomicOr(&s_or[1], hi); }
        __syncthreads();
        const unsigned long long all_or = ((unsigned long long)s_or[1] << 32) | s_or[0];
        const int top_byte = all_or ? (63 - __clzll((long long)all_or)) >> 3 : -1;

        if (!COARSE && iters == 1) {
            // One candidate per thread (the block form: at most 1024 blocks per layer): the k-th largest key by bisection
            // on its bits from the top, one counting barrier per bit.  As soon as exactly k keys lie at or above the
            // trial value the selection is decided and the remaining bits do not matter (masses spread over many
            // octaves: a dozen steps); masses full of ties go through every bit and end with the exact key and the
            // number of its equals.
            const bool cand = (int)threadIdx.x < ncand;
            const unsigned long long x = kreg[0];
            unsigned long long t = 0;
            bool exact_k = false;
            for (int bit = all_or ? 63 - __clzll((long long)all_or) : -1; bit >= 0; bit--) {
                const unsigned long long trial = t | (1ull << bit);
                const int c = __syncthreads_count(cand && x >= trial);
                if (c >= k) { t = trial; if (c == k) { exact_k = true; break; } }
            }
            T = t;
            if (exact_k) { krem = 0; n_eq = 0; }         // x >= T takes exactly k keys: no equals to rank
            else {
                const int larger = __syncthreads_count(cand && x > t);
                n_eq = __syncthreads_count(cand && x == t);
                krem = k - larger;
            }
        } else if ((all_or >> 32) == 0) {
            // every candidate fits 32 bits (masses of a few thousand rows): the same passes on 32-bit keys
            unsigned int k32[KPT];
#pragma unroll
            for (int i = 0; i < KPT; i++) k32[i] = (unsigned int)kreg[i];
            radix_select_passes<unsigned int, KPT>(k32, later_key, iters, ncand, top_byte, hist, &s_prefix, &s_krem, &s_eq);
        } else {
            radix_select_passes<unsigned long long, KPT>(kreg, later_key, iters, ncand, top_byte, hist, &s_prefix, &s_krem, &s_eq);
        }
        if (COARSE || iters != 1) {
            T = s_prefix;
            krem = s_krem;                       // keys equal to T to take, lowest block index first
            n_eq = s_eq;
        }
    }
    // Ranking among equal keys (a prefix count in index order) is needed only when some of them stay out.
    const bool ties_matter = !take_all && !take_none && n_eq > krem;

    // ---- emit mask and ascending lists: the dirty window first, then the candidates in index order
    uint8_t* mask = p.mask + (long long)l * NB;
    int32_t* ridx = p.repair_idx + (long long)l * NB;
    int32_t* fidx = p.reuse_idx + (long long)l * NB;
    const bool lists = p.repair_idx != nullptr;          // the token-level stage only needs the mask
    for (int j = threadIdx.x; j < n_dirty; j += kSelThreads) { mask[j] = 1; if (lists) ridx[j] = j; }
    int run_sel = 0, run_eq = 0;
    auto emit = [&](int i, unsigned long long x) {       // round i of the candidates; x: this thread's key of the round
        const int c = threadIdx.x + i * kSelThreads;
        const bool in = c < ncand;
        bool sel = false;
        if (take_all) sel = in;
        else if (!take_none) {
            sel = in && x >= T;
            if (ties_matter) {
                const int eq = in && x == T;
                int tot_eq;
                const int rank = cta_exclusive_scan(eq, warp_sums, &tot_eq) + run_eq;
                run_eq += tot_eq;
                sel = in && (x > T || (eq && rank < krem));
            }
        }
        int before = 0;
        if (lists) {                                     // the mask alone needs no compaction
            int tot_sel;
            before = cta_exclusive_scan(sel ? 1 : 0, warp_sums, &tot_sel) + run_sel;
            run_sel += tot_sel;
        }
        if (in) {
            const int j = n_dirty + c;
            mask[j] = sel ? 1 : 0;
            if (lists) {
                if (sel) ridx[n_dirty + before] = j;
                else fidx[c - before] = j;
            }
        }
    };
#pragma unroll
    for (int i = 0; i < KPT; i++) {
        if (i >= iters) break;
        emit(i, kreg[i]);
    }
    for (int i = KPT; i < iters; i++) {
        const int c = threadIdx.x + i * kSelThreads;
        emit(i, c < ncand ? later_key(c) : 0ull);
    }
    if (!lists) return;
    const int n_r = n_dirty + run_sel, n_f = NB - n_r;
    for (int i = n_r + threadIdx.x; i < NB; i += kSelThreads) ridx[i] = -1;
    for (int i = n_f + threadIdx.x; i < NB; i += kSelThreads) fidx[i] = -1;
    if (threadIdx.x == 0) { p.repair_cnt[l] = n_r; p.reuse_cnt[l] = n_f; }
}

// BlockRound of Eq. 12: a block is repaired when any of its tokens is in D u H.  One CTA per layer turns the token
// mask into the block mask and the ascending repair / reuse lists.
__global__ void __launch_bounds__(kSelThreads)
block_round_kernel(const uint8_t* token_mask, long long mask_stride, int n, int B, int NB, uint8_t* mask, int32_t* repair_idx,
                   int32_t* repair_cnt, int32_t* reuse_idx, int32_t* reuse_cnt) {
    __shared__ int warp_sums[33];
    pdl_wait();
    pdl_trigger();                                        // see select_kernel
    const int l = blockIdx.x;
    const uint8_t* tm = token_mask + (long long)l * mask_stride;      // stride 0: one request-level token set for every layer
    uint8_t* bm = mask + (long long)l * NB;
    int32_t* ridx = repair_idx + (long long)l * NB;
    int32_t* fidx = reuse_idx + (long long)l * NB;
    int run = 0;
    for (int j0 = 0; j0 < NB; j0 += kSelThreads) {
        const int j = j0 + threadIdx.x;
        int hit = 0;
        if (j < NB) {
            const int e = min(n, (j + 1) * B);
            if ((B & 15) == 0 && e == (j + 1) * B && ((reinterpret_cast<uintptr_t>(tm) + (size_t)j * B) & 15u) == 0) {
                for (int i = j * B; i < e; i += 16) {
                    const uint4 w = *reinterpret_cast<const uint4*>(tm + i);
                    hit |= (w.x | w.y | w.z | w.w) != 0;
                }
            } else {
                for (int i = j * B; i < e; i++) hit |= tm[i];
            }
        }
        int tot;
        const int before = cta_exclusive_scan(hit, warp_sums, &tot) + run;
        run += tot;
        if (j < NB) {
            bm[j] = (uint8_t)hit;
            if (hit) ridx[before] = j;
            else fidx[j - before] = j;
        }
    }
    const int n_r = run, n_f = NB - run;
    for (int i = n_r + threadIdx.x; i < NB; i += kSelThreads) ridx[i] = -1;
    for (int i = n_f + threadIdx.x; i < NB; i += kSelThreads) fidx[i] = -1;
    if (threadIdx.x == 0) { repair_cnt[l] = n_r; reuse_cnt[l] = n_f; }
}

// Shared memory for the candidates that select_kernel cannot keep in registers (it would otherwise re-read them from
// global memory in every radix pass).
static int select_spill(patchkv_ctx* ctx, int ncand, int* keys, int* bytes, int keys_per_thread = kKeysPerThread) {
    long long want = (long long)ncand - (long long)keys_per_thread * kSelThreads;
    const long long cap = ((long long)ctx->max_smem_optin - 4096 - 8 * kSelList) / 8;
    if (want < 0) want = 0;
    if (want > cap) want = cap;
    *keys = (int)want;
    *bytes = (int)want * 8;
    if (*bytes > 48 * 1024) {
        PKV_CUDA(ctx, cudaFuncSetAttribute(select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, *bytes));
        PKV_CUDA(ctx, cudaFuncSetAttribute(select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, *bytes));
    }
    return PATCHKV_OK;
}

static int ensure_mass_ws(patchkv_ctx* ctx, size_t elems) {
    if (elems <= ctx->mass_ws_elems) return PATCHKV_OK;
    PKV_CUDA(ctx, cudaDeviceSynchronize());
    if (ctx->d_mass_ws) { cudaFree(ctx->d_mass_ws); ctx->d_mass_ws = nullptr; ctx->mass_ws_elems = 0; }
    PKV_CUDA(ctx, cudaMalloc(&ctx->d_mass_ws, elems * sizeof(unsigned long long)));
    ctx->mass_ws_elems = elems;
    return PATCHKV_OK;
}

}  // namespace patchkv

using namespace patchkv;

// Copies of the selection outputs into the caller's pinned host mirrors, in stream order after the kernels.
static cudaError_t mirror_to_host(const patchkv_select_args* a, int L, int NB, cudaStream_t stream) {
    const size_t cells = (size_t)L * NB;
    cudaError_t e = cudaSuccess;
    if (a->host_repair_mask && cells && e == cudaSuccess)
        e = cudaMemcpyAsync(a->host_repair_mask, a->repair_mask, cells, cudaMemcpyDeviceToHost, stream);
    if (a->host_repair_idx && cells && e == cudaSuccess)
        e = cudaMemcpyAsync(a->host_repair_idx, a->repair_idx, cells * 4, cudaMemcpyDeviceToHost, stream);
    if (a->host_reuse_idx && cells && e == cudaSuccess)
        e = cudaMemcpyAsync(a->host_reuse_idx, a->reuse_idx, cells * 4, cudaMemcpyDeviceToHost, stream);
    if (a->host_repair_cnt && e == cudaSuccess)
        e = cudaMemcpyAsync(a->host_repair_cnt, a->repair_cnt, (size_t)L * 4, cudaMemcpyDeviceToHost, stream);
    if (a->host_reuse_cnt && e == cudaSuccess)
        e = cudaMemcpyAsync(a->host_reuse_cnt, a->reuse_cnt, (size_t)L * 4, cudaMemcpyDeviceToHost, stream);
    if (a->sync_to_host && e == cudaSuccess) e = cudaStreamSynchronize(stream);
    return e;
}

extern "C" int patchkv_select_repair(patchkv_ctx* ctx, const patchkv_select_args* a, void* stream_) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (!a || a->struct_size != sizeof(patchkv_select_args)) return fail(ctx, PATCHKV_E_INVALID, "select: null args or struct_size mismatch");
    if (a->n_layers <= 0 || a->n_suffix_tokens < 0 || a->block_tokens <= 0 || a->top_k < 0)
        return fail(ctx, PATCHKV_E_INVALID, "select: need L > 0, n >= 0, B > 0, top_k >= 0");
    if (a->layer_mode != PATCHKV_LAYERS_INDEPENDENT && a->layer_mode != PATCHKV_LAYERS_SHARED)
        return fail(ctx, PATCHKV_E_INVALID, "select: unknown layer_mode");
    if (a->kind != PATCHKV_SCORE_ATTN_F16 && a->kind != PATCHKV_SCORE_BLOCK_MASS)
        return fail(ctx, PATCHKV_E_INVALID, "select: unknown kind");
    if (!a->repair_mask || !a->repair_idx || !a->repair_cnt || !a->reuse_idx || !a->reuse_cnt)
        return fail(ctx, PATCHKV_E_INVALID, "select: null output");
    const int L = a->n_layers, n = a->n_suffix_tokens, B = a->block_tokens;
    const int NB = (int)(((long long)n + B - 1) / B);
    long long nd = a->dirty_tokens < 0 ? 0 : a->dirty_tokens;
    if (nd > n) nd = n;
    const int n_dirty = (int)((nd + B - 1) / B);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");

    const bool shared = a->layer_mode == PATCHKV_LAYERS_SHARED && L > 1;
    const bool from_attn = a->kind == PATCHKV_SCORE_ATTN_F16;
    // (request-level ranking with nobody asking for the per-layer masses: every layer adds straight into the summed row)
    const bool sum_direct = shared && from_attn && !a->mass_out;
    size_t ws_need = (from_attn && !a->mass_out && !sum_direct ? (size_t)L * NB : 0) + (shared ? (size_t)NB : 0);
    if (ws_need) { int rc = ensure_mass_ws(ctx, ws_need); if (rc != PATCHKV_OK) return rc; }
    unsigned long long* ws = ctx->d_mass_ws;

    const unsigned long long* mass = reinterpret_cast<const unsigned long long*>(a->mass);
    if (from_attn) {
        if (a->n_q_heads < 0 || a->n_queries < 0 || (NB > 0 && a->n_q_heads > 0 && a->n_queries > 0 && !a->attn))
            return fail(ctx, PATCHKV_E_INVALID, "select: attention shape / pointer");
        unsigned long long* m = a->mass_out ? reinterpret_cast<unsigned long long*>(a->mass_out) : ws;
        if (!a->mass_out && !sum_direct) ws += (size_t)L * NB;
        const long long rows = (long long)a->n_q_heads * a->n_queries;
        if (NB > 0) PKV_CUDA(ctx, cudaMemsetAsync(m, 0, (size_t)(sum_direct ? 1 : L) * NB * sizeof(unsigned long long), stream));
        if (NB > 0 && rows > 0) {
            if (rows > 0x7fffffffLL) return fail(ctx, PATCHKV_E_UNSUPPORTED, "select: Hq * Q too large");
            MassParams mp;
            mp.attn = static_cast<const uint16_t*>(a->attn);
            mp.stride_layer = a->attn_stride_layer; mp.stride_head = a->attn_stride_head; mp.stride_query = a->attn_stride_query;
            mp.Hq = a->n_q_heads; mp.Q = a->n_queries; mp.n = n; mp.B = B; mp.NB = NB;
            mp.mass = m; mp.mass_stride = sum_direct ? 0 : NB; mp.status = ctx->d_status;
            const bool octet = (B % 8 == 0) && ((reinterpret_cast<uintptr_t>(a->attn) & 15u) == 0) &&
                               ((a->attn_stride_layer | a->attn_stride_head | a->attn_stride_query) & 7) == 0;
            const int cols = octet ? (n + 7) / 8 : n;
            const int tiles = (cols + 255) / 256;
            // enough CTAs for ~8 waves of 8 CTAs per SM, at least 16 rows each so that atomics stay rare
            long long want = (long long)ctx->sm_count * 64;
            long long groups = want / ((long long)tiles * L);
            if (groups < 1) groups = 1;
            long long rpc = (rows + groups - 1) / groups;
            rpc = (rpc + kMassBatch - 1) / kMassBatch * kMassBatch;     // whole batches of rows per CTA
            if (rpc < 16) rpc = 16;
            if (rpc > rows) rpc = rows;
            groups = (rows + rpc - 1) / rpc;
            if (groups > 65535 || L > 65535) return fail(ctx, PATCHKV_E_UNSUPPORTED, "select: grid too large");
            mp.rows_per_cta = (int)rpc;
            dim3 grid(tiles, (unsigned)groups, L);
            PKV_CUDA(ctx, launch_pdl(octet ? block_mass_octet_kernel : block_mass_generic_kernel, grid, dim3(256), 0, stream, mp));
        }
        mass = m;
    } else if (NB > 0 && !mass) {
        return fail(ctx, PATCHKV_E_INVALID, "select: null mass");
    }

    TopkParams tp;
    tp.mass = mass; tp.shared = 0;
    if (shared && NB > 0) {
        if (!sum_direct) PKV_CUDA(ctx, launch_pdl(sum_layers_kernel, dim3((NB + 255) / 256), dim3(256), 0, stream, mass, L, NB, ws));
        tp.mass = ws; tp.shared = 1;
    }
    tp.NB = NB; tp.n_dirty = n_dirty; tp.top_k = a->top_k;
    tp.mask = a->repair_mask; tp.repair_idx = a->repair_idx; tp.repair_cnt = a->repair_cnt;
    tp.reuse_idx = a->reuse_idx; tp.reuse_cnt = a->reuse_cnt;
    if (a->score_out && NB > 0)
        PKV_CUDA(ctx, launch_pdl(normalise_kernel, dim3(tp.shared ? 1 : L), dim3(256), 0, stream, tp.mass, NB, a->score_out));
    int spill_bytes = 0;
    tp.coarse_hist = nullptr;
    int rc2 = select_spill(ctx, NB - n_dirty, &tp.spill_keys, &spill_bytes);
    if (rc2 != PATCHKV_OK) return rc2;
    PKV_CUDA(ctx, launch_pdl(select_kernel<false>, dim3(L), dim3(kSelThreads), (size_t)spill_bytes, stream, tp));
    PKV_CUDA(ctx, mirror_to_host(a, L, NB, stream));
    return PATCHKV_OK;
}

// ---------------------------------------------------------------- token-level selection
extern "C" int patchkv_select_repair_tokens(patchkv_ctx* ctx, const patchkv_select_args* a, void* stream_) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (!a || a->struct_size != sizeof(patchkv_select_args)) return fail(ctx, PATCHKV_E_INVALID, "select: null args or struct_size mismatch");
    if (a->n_layers <= 0 || a->n_layers > 65535 || a->n_suffix_tokens < 0 || a->block_tokens <= 0 || a->top_k < 0)
        return fail(ctx, PATCHKV_E_INVALID, "select: need 0 < L <= 65535, n >= 0, B > 0, top_k >= 0");
    if (a->layer_mode != PATCHKV_LAYERS_INDEPENDENT && a->layer_mode != PATCHKV_LAYERS_SHARED)
        return fail(ctx, PATCHKV_E_INVALID, "select: unknown layer_mode");
    if (a->kind != PATCHKV_SCORE_ATTN_F16 && a->kind != PATCHKV_SCORE_TOKEN_MASS)
        return fail(ctx, PATCHKV_E_INVALID, "select: kind must be ATTN_F16 or TOKEN_MASS");
    if (!a->repair_mask || !a->repair_idx || !a->repair_cnt || !a->reuse_idx || !a->reuse_cnt)
        return fail(ctx, PATCHKV_E_INVALID, "select: null output");
    const int L = a->n_layers, n = a->n_suffix_tokens, B = a->block_tokens;
    const int NB = (int)(((long long)n + B - 1) / B);
    long long nd = a->dirty_tokens < 0 ? 0 : a->dirty_tokens;
    if (nd > n) nd = n;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");

    const bool shared = a->layer_mode == PATCHKV_LAYERS_SHARED && L > 1;
    const bool from_attn = a->kind == PATCHKV_SCORE_ATTN_F16;
    // workspace: [token mass L*n (if computed here and not handed out)] [summed mass n (shared)] [code histogram] [token
    // mask L*n bytes]; what has to start at zero (masses computed here, the histogram) is contiguous: one memset
    // (request-level ranking with nobody asking for the per-layer masses: every layer adds straight into the summed row)
    const bool sum_direct = shared && from_attn && !a->mass_out;
    const size_t mass_elems = from_attn && !a->mass_out && !sum_direct ? (size_t)L * n : 0;
    const size_t sum_elems = shared ? (size_t)n : 0;
    const size_t mask_words = ((size_t)L * n + 7) / 8;
    // many candidates: the first cut of the ranking is a histogram made by several CTAs (coarse_hist_kernel)
    const long long nd_tokens = std::min<long long>(std::max<long long>(a->dirty_tokens, 0), n);
    const bool coarse = (long long)n - nd_tokens >= 4 * kSelThreads;
    const size_t hist_words = coarse ? ((size_t)(shared ? 1 : L) * kCoarseCodes + 1) / 2 : 0;
    int rc = ensure_mass_ws(ctx, mass_elems + sum_elems + mask_words + hist_words + 1);
    if (rc != PATCHKV_OK) return rc;
    unsigned long long* ws = ctx->d_mass_ws;
    unsigned long long* ws_sum = ws + mass_elems;
    unsigned int* coarse_hist = reinterpret_cast<unsigned int*>(ws_sum + sum_elems);
    uint8_t* tok_mask = reinterpret_cast<uint8_t*>(ws_sum + sum_elems + hist_words);
    const bool mass_in_ws = from_attn && !a->mass_out && n > 0;       // the masses are computed into the workspace
    if (mass_in_ws) PKV_CUDA(ctx, cudaMemsetAsync(ws, 0, (mass_elems + sum_elems + hist_words) * 8, stream));
    else if (coarse) PKV_CUDA(ctx, cudaMemsetAsync(coarse_hist, 0, hist_words * 8, stream));

    const unsigned long long* mass = reinterpret_cast<const unsigned long long*>(a->mass);
    if (from_attn) {
        if (a->n_q_heads < 0 || a->n_queries < 0 || (n > 0 && a->n_q_heads > 0 && a->n_queries > 0 && !a->attn))
            return fail(ctx, PATCHKV_E_INVALID, "select: attention shape / pointer");
        unsigned long long* m = a->mass_out ? reinterpret_cast<unsigned long long*>(a->mass_out) : (sum_direct ? ws_sum : ws);
        const long long rows = (long long)a->n_q_heads * a->n_queries;
        if (rows > 0x7fffffffLL) return fail(ctx, PATCHKV_E_UNSUPPORTED, "select: Hq * Q too large");
        if (n > 0 && !mass_in_ws) PKV_CUDA(ctx, cudaMemsetAsync(m, 0, (size_t)L * n * sizeof(unsigned long long), stream));
        if (n > 0 && rows > 0) {
            MassParams mp;                         // token granularity: a block of one token
            mp.attn = static_cast<const uint16_t*>(a->attn);
            mp.stride_layer = a->attn_stride_layer; mp.stride_head = a->attn_stride_head; mp.stride_query = a->attn_stride_query;
            mp.Hq = a->n_q_heads; mp.Q = a->n_queries; mp.n = n; mp.B = 1; mp.NB = n;
            mp.mass = m; mp.mass_stride = sum_direct ? 0 : n; mp.status = ctx->d_status;
            const bool octet = ((reinterpret_cast<uintptr_t>(a->attn) & 15u) == 0) &&
                               ((a->attn_stride_layer | a->attn_stride_head | a->attn_stride_query) & 7) == 0;
            if (octet && n % 8 == 0 && a->n_queries % kTokPipeRows == 0 && !(ctx->flags & PATCHKV_FLAG_DIRECT_LOADS)) {
                // regular shape: rows staged through shared memory by bulk copies, one contiguous piece of the list per CTA
                TokPipeParams tpp;
                tpp.m = mp;
                tpp.col_tiles = (n + kTokPipeCols - 1) / kTokPipeCols;
                tpp.batches_per_tile = (int)(rows / kTokPipeRows);
                tpp.total_batches = (long long)L * tpp.col_tiles * tpp.batches_per_tile;
                tpp.wait_limit = kWaitLimit; tpp.stall_after = -1;
                if (ctx->selftest_stall_after >= 0) {      // armed by patchkv_selftest_stall_next_launch: this launch only
                    tpp.wait_limit = ctx->selftest_wait_limit;
                    tpp.stall_after = ctx->selftest_stall_after;
                    ctx->selftest_stall_after = -1;
                }
                const int smem = kTokPipeStages * kTokPipeStageBytes;
                const int grid = (int)std::min<long long>(tpp.total_batches, 2ll * ctx->sm_count);
                PKV_CUDA(ctx, cudaFuncSetAttribute(token_mass_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
                PKV_CUDA(ctx, launch_pdl(token_mass_pipe_kernel, dim3(grid), dim3(kTokPipeThreads), smem, stream, tpp));
            } else {
            const int cols = octet ? (n + 7) / 8 : n;
            const int tiles = (cols + 255) / 256;
            // few row groups (every thread ends with one 64-bit atomic per token), a whole number of batches each,
            // and a grid that fills its last wave: among the candidates the one with the best wave efficiency
            int occ = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, token_mass_octet_kernel, 256, 0) != cudaSuccess || occ < 1) {
                cudaGetLastError();
                occ = 2;
            }
            const long long slots = (long long)ctx->sm_count * occ, per_group = (long long)tiles * L;
            long long rpc = rows;
            double best = -1.0;
            for (long long g = std::max<long long>(1, 4 * slots / per_group); g <= std::max<long long>(1, 9 * slots / per_group); g++) {
                long long c = (rows + g - 1) / g;
                c = (c + kMassBatch - 1) / kMassBatch * kMassBatch;
                if (c < 64) c = 64;
                if (c > rows) c = rows;
                const long long ctas = ((rows + c - 1) / c) * per_group;
                const double eff = (double)ctas / (double)(((ctas + slots - 1) / slots) * slots);
                if (eff > best + 1e-9) { best = eff; rpc = c; }
            }
            long long groups = (rows + rpc - 1) / rpc;
            if (groups > 65535) return fail(ctx, PATCHKV_E_UNSUPPORTED, "select: grid too large");
            mp.rows_per_cta = (int)rpc;
            PKV_CUDA(ctx, launch_pdl(octet ? token_mass_octet_kernel : block_mass_generic_kernel,
                                     dim3(tiles, (unsigned)groups, L), dim3(256), 0, stream, mp));
            }
        }
        mass = m;
    } else if (n > 0 && !mass) {
        return fail(ctx, PATCHKV_E_INVALID, "select: null mass");
    }

    TopkParams tp;
    tp.mass = mass; tp.shared = 0;
    if (shared && n > 0) {
        if (!sum_direct) PKV_CUDA(ctx, launch_pdl(sum_layers_kernel, dim3((n + 255) / 256), dim3(256), 0, stream, mass, L, n, ws_sum));
        tp.mass = ws_sum; tp.shared = 1;
    }
    if (a->score_out && n > 0)
        PKV_CUDA(ctx, launch_pdl(normalise_kernel, dim3(tp.shared ? 1 : L), dim3(256), 0, stream, tp.mass, n, a->score_out));
    tp.NB = n; tp.n_dirty = (int)nd; tp.top_k = a->top_k;     // the "blocks" of this stage are single tokens
    tp.mask = tok_mask; tp.repair_idx = nullptr; tp.repair_cnt = nullptr; tp.reuse_idx = nullptr; tp.reuse_cnt = nullptr;
    // the request-level ranking (layers shared) is one ranking: one CTA, one token mask that every layer rounds to blocks
    int spill_bytes = 0;
    rc = select_spill(ctx, n - (int)nd, &tp.spill_keys, &spill_bytes, coarse ? 1 : kKeysPerThread);
    if (rc != PATCHKV_OK) return rc;
    // the request-level ranking (layers shared) is one ranking: one CTA, one token mask that every layer rounds to blocks
    tp.coarse_hist = coarse ? coarse_hist : nullptr;
    if (coarse) {
        const int rankings = tp.shared ? 1 : L;
        const int slices = std::max(1, std::min(32, (n - (int)nd + kSelThreads - 1) / kSelThreads));
        PKV_CUDA(ctx, launch_pdl(coarse_hist_kernel, dim3(slices, rankings), dim3(kSelThreads), 0, stream, tp.mass, tp.shared, n, (int)nd,
                                 coarse_hist));
        PKV_CUDA(ctx, launch_pdl(select_kernel<true>, dim3(rankings), dim3(kSelThreads), (size_t)spill_bytes, stream, tp));
    } else {
        PKV_CUDA(ctx, launch_pdl(select_kernel<false>, dim3(tp.shared ? 1 : L), dim3(kSelThreads), (size_t)spill_bytes, stream, tp));
    }
    PKV_CUDA(ctx, launch_pdl(block_round_kernel, dim3(L), dim3(kSelThreads), 0, stream, (const uint8_t*)tok_mask,
                             tp.shared ? 0ll : (long long)n, n, B, NB, a->repair_mask, a->repair_idx, a->repair_cnt,
                             a->reuse_idx, a->reuse_cnt));
    PKV_CUDA(ctx, mirror_to_host(a, L, NB, stream));
    return PATCHKV_OK;
}

// ---------------------------------------------------------------- selection without any allocation
// Scratch of patchkv_select_repair_static: block masses, the layer-summed masses of LAYERS_SHARED, and one
// status word behind them.  It lives in the library image, so every GPU that loads the library holds these
// ~2 MiB until the process exits, and every call on a device shares them.
namespace patchkv {

constexpr size_t kStaticMassElems = PATCHKV_STATIC_MAX_MASS_ELEMS;
static __device__ __align__(256) unsigned long long g_static_scratch[kStaticMassElems + 32];

constexpr int kMaxStaticDevices = 64;
static unsigned long long* g_static_ptr[kMaxStaticDevices];   // device address of g_static_scratch, per device
static std::mutex g_static_mu;

// In host code `g_static_scratch` only names the symbol; the address a kernel can use has to be asked for,
// once per device, while that device is current.
static int static_scratch(unsigned long long** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxStaticDevices) return PATCHKV_E_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return PATCHKV_E_CUDA;
        }
        g_static_ptr[dev] = static_cast<unsigned long long*>(ptr);
    }
    *out = g_static_ptr[dev];
    return PATCHKV_OK;
}

}  // namespace patchkv

extern "C" int patchkv_select_repair_static(const patchkv_select_args* a, void* stream_, int32_t* device_status) {
    if (!a || a->struct_size != sizeof(patchkv_select_args)) return PATCHKV_E_INVALID;
    if (a->n_layers <= 0 || a->n_suffix_tokens < 0 || a->block_tokens <= 0 || a->top_k < 0) return PATCHKV_E_INVALID;
    if (a->layer_mode != PATCHKV_LAYERS_INDEPENDENT && a->layer_mode != PATCHKV_LAYERS_SHARED) return PATCHKV_E_INVALID;
    if (a->kind != PATCHKV_SCORE_ATTN_F16 && a->kind != PATCHKV_SCORE_BLOCK_MASS) return PATCHKV_E_INVALID;
    if (!a->repair_mask || !a->repair_idx || !a->repair_cnt || !a->reuse_idx || !a->reuse_cnt) return PATCHKV_E_INVALID;
    const int L = a->n_layers, n = a->n_suffix_tokens, B = a->block_tokens;
    const int NB = (int)(((long long)n + B - 1) / B);
    long long nd = a->dirty_tokens < 0 ? 0 : a->dirty_tokens;
    if (nd > n) nd = n;
    const int n_dirty = (int)((nd + B - 1) / B);
    const bool shared = a->layer_mode == PATCHKV_LAYERS_SHARED && L > 1;
    const bool from_attn = a->kind == PATCHKV_SCORE_ATTN_F16;
    // the fixed scratch must hold the block masses (when they are computed here) and the layer-summed masses
    const unsigned long long need = (from_attn ? (unsigned long long)L * NB : 0ull) + (shared ? (unsigned long long)NB : 0ull);
    if (need > kStaticMassElems) return PATCHKV_E_TOO_LARGE;
    if (L > 65535) return PATCHKV_E_TOO_LARGE;

    unsigned long long* scratch = nullptr;
    int rc = static_scratch(&scratch);
    if (rc != PATCHKV_OK) return rc;
    int32_t* status = device_status ? device_status : reinterpret_cast<int32_t*>(scratch + kStaticMassElems);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    const unsigned long long* mass = reinterpret_cast<const unsigned long long*>(a->mass);
    unsigned long long* ws = scratch;
    if (from_attn) {
        if (a->n_q_heads < 0 || a->n_queries < 0 || (NB > 0 && a->n_q_heads > 0 && a->n_queries > 0 && !a->attn))
            return PATCHKV_E_INVALID;
        unsigned long long* m = ws;
        ws += (size_t)L * NB;
        const long long rows = (long long)a->n_q_heads * a->n_queries;
        if (rows > 0x7fffffffLL) return PATCHKV_E_TOO_LARGE;
        // the array keeps whatever the previous call left: the sums must start from zero
        if (NB > 0 && cudaMemsetAsync(m, 0, (size_t)L * NB * sizeof(unsigned long long), stream) != cudaSuccess)
            return PATCHKV_E_CUDA;
        if (NB > 0 && rows > 0) {
            MassParams mp;
            mp.attn = static_cast<const uint16_t*>(a->attn);
            mp.stride_layer = a->attn_stride_layer; mp.stride_head = a->attn_stride_head; mp.stride_query = a->attn_stride_query;
            mp.Hq = a->n_q_heads; mp.Q = a->n_queries; mp.n = n; mp.B = B; mp.NB = NB;
            mp.mass = m; mp.mass_stride = NB; mp.status = status;
            const bool octet = (B % 8 == 0) && ((reinterpret_cast<uintptr_t>(a->attn) & 15u) == 0) &&
                               ((a->attn_stride_layer | a->attn_stride_head | a->attn_stride_query) & 7) == 0;
            const int cols = octet ? (n + 7) / 8 : n;
            const int tiles = (cols + 255) / 256;
            long long groups = 8192 / ((long long)tiles * L);       // about 8192 CTAs, at least 16 rows each
            if (groups < 1) groups = 1;
            long long rpc = (rows + groups - 1) / groups;
            rpc = (rpc + kMassBatch - 1) / kMassBatch * kMassBatch;     // whole batches of rows per CTA
            if (rpc < 16) rpc = 16;
            if (rpc > rows) rpc = rows;
            groups = (rows + rpc - 1) / rpc;
            if (groups > 65535) return PATCHKV_E_TOO_LARGE;
            mp.rows_per_cta = (int)rpc;
            dim3 grid(tiles, (unsigned)groups, L);
            if (octet) block_mass_octet_kernel<<<grid, 256, 0, stream>>>(mp);
            else block_mass_generic_kernel<<<grid, 256, 0, stream>>>(mp);
            if (cudaGetLastError() != cudaSuccess) return PATCHKV_E_CUDA;
        }
        if (a->mass_out && NB > 0 &&
            cudaMemcpyAsync(a->mass_out, m, (size_t)L * NB * sizeof(unsigned long long), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
            return PATCHKV_E_CUDA;
        mass = m;
    } else if (NB > 0 && !mass) {
        return PATCHKV_E_INVALID;
    }

    TopkParams tp;
    tp.mass = mass; tp.shared = 0;
    if (shared && NB > 0) {
        sum_layers_kernel<<<(NB + 255) / 256, 256, 0, stream>>>(mass, L, NB, ws);
        if (cudaGetLastError() != cudaSuccess) return PATCHKV_E_CUDA;
        tp.mass = ws; tp.shared = 1;
    }
    tp.NB = NB; tp.n_dirty = n_dirty; tp.top_k = a->top_k; tp.spill_keys = 0; tp.coarse_hist = nullptr;
    tp.mask = a->repair_mask; tp.repair_idx = a->repair_idx; tp.repair_cnt = a->repair_cnt;
    tp.reuse_idx = a->reuse_idx; tp.reuse_cnt = a->reuse_cnt;
    if (a->score_out && NB > 0) normalise_kernel<<<tp.shared ? 1 : L, 256, 0, stream>>>(tp.mass, NB, a->score_out);
    select_kernel<false><<<L, kSelThreads, 0, stream>>>(tp);
    if (cudaGetLastError() != cudaSuccess) return PATCHKV_E_CUDA;
    if (mirror_to_host(a, L, NB, stream) != cudaSuccess) { cudaGetLastError(); return PATCHKV_E_CUDA; }
    return PATCHKV_OK;
}
