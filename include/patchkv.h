/*
 * patchkv.h -- C ABI of the PatchKV suffix-restore library for NVIDIA B200 (sm_100a).
 *
 * After a middle edit of an LLM context, C_new = P + M_new + S keeps a token-identical suffix S
 * whose KV cache was offloaded (Section II-A, Eq. 1).  This library runs the two data-parallel
 * steps of resuming that suffix:
 *
 *   1. patchkv_select_repair -- fix the block partition (R, F) of the suffix before any
 *      reconstruction: per-block attention mass from stored attention (Section IV-C, Eq. 10), the
 *      edit-local dirty window (Section IV-B, Eq. 9), the top-k non-local blocks outside it (Eq. 11),
 *      and R = BlockRound(D u H), F = B(S) \ R (Eq. 12).
 *   2. patchkv_restore / patchkv_restore_from_host -- rebuild every block of F in one fused pass:
 *      dequantise it by its frozen per-block precision tag (Section IV-D, Eq. 14 gives the tags),
 *      correct the RoPE phase of K by the position delta, K_corr = R(rho) R(omega)^-1 K_old
 *      (Section II-B, Eq. 3; V gets no rotation, Section IV-C), and write the rows straight
 *      into the request's destination KV pages (Section IV-D, last paragraph).  Blocks of R are
 *      never read and never written: they belong to the recompute path.
 *
 * Conventions
 *   - Every function returns a patchkv_status (0 = ok, < 0 = error); nothing throws or prints.
 *   - "DEVICE" pointers are CUDA device memory of the context's device; "HOST" pointers are host
 *     memory; "PINNED" is page-locked host memory (cudaHostAlloc / cudaHostRegister).
 *   - The caller owns every buffer it passes and keeps it alive and unmodified until the work
 *     enqueued on `stream` has completed.  The library owns only the context's workspace.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls are
 *     asynchronous with respect to the host unless stated otherwise; completion is stream order,
 *     which is how the rule that decoding waits for every restored page (Section IV-C) is kept.
 *   - Device-side faults are never raised.  A work item whose directory entry, record extent or
 *     destination pages are out of range is skipped whole, the first such error is latched in the
 *     context's status word, and the rest of the call proceeds; see patchkv_query_status.
 *   - Every struct starts with struct_size = sizeof(that struct) as compiled by the caller.
 *
 * Checkpoint byte layout ("PKV1"; the paper prescribes none beyond same-representation runs)
 *   - per layer one payload buffer, 16-byte aligned; tags u8 [L][NB] and blk_off u64 [L][NB] give the
 *     tag and the byte offset of each block's record inside its layer payload (a multiple of 16 wherever the
 *     geometry makes records multiples of 16 bytes, i.e. for every geometry the fast kernels take);
 *   - one block record = [K codes][K scales][V codes][V scales]; codes are [token][head][channel]
 *     row-major; bf16 codes 2 bytes; int8 codes 1 byte two's complement; int4 codes pack channel c
 *     (even) in bits 0-3 and channel c+1 in bits 4-7 of one byte, two's-complement nibbles; scales
 *     are fp16 [token][head][channel / group], symmetric (no zero point); a bf16 section has no
 *     scales; a partial last block is zero-padded to block_tokens tokens.
 *   - value = code * scale formed in fp32 (exact), rounded once to bf16 (nearest even); a bf16 code
 *     is copied bit for bit (V always; K when delta == 0).
 *   - K rotation: theta_i = rope_base^(-2i/rotary_dim) (or inv_freq[i]); c_i, s_i = cos, sin of
 *     (double)delta * theta_i evaluated in double on the host and rounded once to fp32; each rotary
 *     pair (a, b) -> (a*c_i - b*s_i, a*s_i + b*c_i) with every fp32 operation rounded on its own (no
 *     FMA contraction), then one rounding to bf16.  delta == 0 skips the rotation.
 *   - destination: suffix token u = j*block_tokens + t + dst_shift goes to slot u % page_tokens of
 *     page block_table[u / page_tokens]; element offset = layer*stride_layer + page*stride_page +
 *     slot*stride_token + head*stride_head + channel from k_base / v_base.
 */
#ifndef PATCHKV_H_
#define PATCHKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define PATCHKV_API __declspec(dllexport)
#else
#define PATCHKV_API __attribute__((visibility("default")))
#endif

typedef struct patchkv_ctx patchkv_ctx; /* opaque: streams, events, staging ring, workspace, status word */

typedef enum {
    PATCHKV_OK = 0,
    PATCHKV_E_INVALID = -1,     /* bad argument (null pointer, inconsistent geometry, misalignment, pageable payload) */
    PATCHKV_E_CUDA = -2,        /* a CUDA runtime call failed; text in patchkv_last_error */
    PATCHKV_E_BOUNDS = -3,      /* device side: an item was out of range and was skipped */
    PATCHKV_E_NOMEM = -4,       /* workspace or staging allocation failed */
    PATCHKV_E_TIMEOUT = -5,     /* device side: a bounded wait inside a kernel gave up; the launch ended early */
    PATCHKV_E_UNSUPPORTED = -6, /* valid but outside the compiled kernels' geometry limits */
    PATCHKV_E_BADINPUT = -7,    /* device side: stored attention held a negative, infinite or NaN entry */
    PATCHKV_E_TOO_LARGE = -8    /* patchkv_select_repair_static: the problem needs more than its fixed scratch */
} patchkv_status;

/* Per-block precision tags (the frozen policy pi_b of Section IV-D: FP16 | K8/V8 | K8/V4). */
enum {
    PATCHKV_TAG_BF16 = 0, /* K bf16, V bf16 (the full-precision tier; this build stores bf16) */
    PATCHKV_TAG_INT8 = 1, /* K int8, V int8 */
    PATCHKV_TAG_INT4 = 2, /* K int8, V int4 -- the low-bit tier of Section IV-D quantises V to 4 bits and leaves K at 8 */
    PATCHKV_TAG_K4V4 = 3  /* K int4, V int4 -- the uniform-INT4 ablation of Section V-C */
};
enum { PATCHKV_ROPE_HALF = 0 /* pairs (i, i + rotary_dim/2) */, PATCHKV_ROPE_INTERLEAVED = 1 /* pairs (2i, 2i+1) */ };
enum { PATCHKV_LAYERS_INDEPENDENT = 0 /* one (R_l, F_l) per layer */, PATCHKV_LAYERS_SHARED = 1 /* rank on the mass summed over layers */ };
enum { PATCHKV_SCORE_ATTN_F16 = 0 /* stored attention */, PATCHKV_SCORE_BLOCK_MASS = 1 /* stored per-block mass */,
       PATCHKV_SCORE_TOKEN_MASS = 2 /* stored per-token mass (patchkv_select_repair_tokens) */ };

enum {
    PATCHKV_FLAG_DIRECT_LOADS = 1, /* restore with the plain-load kernel even where the bulk-copy pipeline applies */
    PATCHKV_FLAG_HOST_DIRECT = 2,  /* restore_from_host: no staging copies; the restore kernel reads the pinned payload
                                      through its device alias, so exactly the reused records cross the link */
    PATCHKV_FLAG_HOST_STAGED = 4   /* restore_from_host: staging copies only (ranges closer than merge_gap_bytes merged);
                                      without either flag long runs are staged and short ones read directly, at once */
};

enum {
    PATCHKV_MAX_SESSIONS = 8,      /* sessions per restore call */
    PATCHKV_MAX_ROTARY_DIM = 256,  /* rotary_dim <= 256 */
    PATCHKV_MAX_BLOCK_VECTORS = 2048, /* block_tokens * n_kv_heads of the fast kernels and of the writer */
    PATCHKV_STATIC_MAX_MASS_ELEMS = 262144 /* u64 entries (2 MiB) of patchkv_select_repair_static's fixed scratch */
};

typedef struct {
    uint32_t struct_size;
    int32_t device;            /* CUDA device ordinal */
    int32_t staging_slots;     /* restore_from_host: depth of the device staging ring (0 = 4) */
    int32_t flags;             /* PATCHKV_FLAG_* */
    uint64_t merge_gap_bytes;  /* restore_from_host with PATCHKV_FLAG_HOST_STAGED: two reused records closer than this
                                  are fetched by one copy (the bytes between them are transferred and ignored);
                                  UINT64_MAX = default 128 KiB */
} patchkv_config;

/* Model / cache geometry shared by all sessions of a call.  The restore entry points take every geometry that the
 * format allows.  The fast kernels need D and G multiples of 8, Dr a multiple of 16 (HALF) or 8 (INTERLEAVED), at most
 * PATCHKV_MAX_BLOCK_VECTORS (token, head) vectors per block, and record sections that are multiples of 16 bytes
 * (B*H*D a multiple of 32, B*H*D/G a multiple of 8); any other geometry is restored by an element-wise kernel with the
 * same results and no claim to speed.  The checkpoint writer takes only the geometries of the fast kernels. */
typedef struct {
    uint32_t struct_size;
    int32_t n_layers;       /* L */
    int32_t n_kv_heads;     /* H */
    int32_t head_dim;       /* D, even */
    int32_t rotary_dim;     /* Dr <= D, even, at most PATCHKV_MAX_ROTARY_DIM; channels >= Dr are not rotated */
    int32_t rope_style;     /* PATCHKV_ROPE_* */
    int32_t block_tokens;   /* B: tokens per checkpoint block */
    int32_t page_tokens;    /* P: tokens per destination page */
    int32_t group;          /* G: channels per fp16 scale, divides D */
    double rope_base;
    const float* inv_freq;  /* HOST, optional [Dr/2]; overrides rope_base (frequency-scaled RoPE variants) */
} patchkv_geom;

/* Destination paged KV pool: two bf16 tensors addressed by element strides. */
typedef struct {
    uint32_t struct_size;
    int32_t n_pages;
    void* k_base;           /* DEVICE bf16, 16-byte aligned */
    void* v_base;           /* DEVICE bf16, 16-byte aligned */
    int64_t stride_layer;   /* elements, non-negative; the channel stride is 1.  The fast kernels need every stride
                               to be a multiple of 8 (16-byte stores); other pools go to the element-wise kernel */
    int64_t stride_page;
    int64_t stride_token;
    int64_t stride_head;
} patchkv_pool;

/* One resumed session whose checkpoint is resident in device memory.  NB = ceil(n_suffix_tokens / B). */
typedef struct {
    uint32_t struct_size;
    int32_t n_suffix_tokens;            /* |S| */
    int32_t delta;                      /* rho_i - omega_i = |M_new| - |M_old|, the same for every suffix token */
    int32_t dst_shift;                  /* 0 .. P-1: slot of the first suffix token in logical page 0 of block_table */
    int32_t n_table;                    /* entries of block_table */
    int32_t reserved;
    const int32_t* block_table;         /* DEVICE i32 [n_table]: logical page -> physical page */
    const uint8_t* tags;                /* DEVICE u8  [L][NB] */
    const uint64_t* blk_off;            /* DEVICE u64 [L][NB] */
    const void* const* layer_payload;   /* DEVICE array of L DEVICE pointers (each 16-byte aligned) */
    const uint64_t* layer_bytes;        /* DEVICE u64 [L]: size of each layer payload */
    const int32_t* reuse_idx;           /* DEVICE i32 [L][NB]: F_l ascending in the first reuse_cnt[l] entries */
    const int32_t* reuse_cnt;           /* DEVICE i32 [L] */
} patchkv_session;

/* The same session with its checkpoint in pinned host memory; every pointer here is a HOST pointer
 * except block_table's target pool.  The planner reads tags, blk_off and the reuse lists on the host. */
typedef struct {
    uint32_t struct_size;
    int32_t n_suffix_tokens;
    int32_t delta;
    int32_t dst_shift;
    int32_t n_table;
    int32_t reserved;
    const int32_t* block_table;         /* HOST i32 [n_table] */
    const uint8_t* tags;                /* HOST u8  [L][NB] */
    const uint64_t* blk_off;            /* HOST u64 [L][NB] */
    const void* const* layer_payload;   /* HOST array of L PINNED pointers (each 16-byte aligned) */
    const uint64_t* layer_bytes;        /* HOST u64 [L] */
    const int32_t* reuse_idx;           /* HOST i32 [L][NB] */
    const int32_t* reuse_cnt;           /* HOST i32 [L] */
} patchkv_session_host;

typedef struct {
    uint32_t struct_size;
    int32_t kind;                /* PATCHKV_SCORE_* */
    int32_t n_layers;            /* L */
    int32_t n_q_heads;           /* Hq (ATTN_F16 only) */
    int32_t n_queries;           /* Q: stored decode query positions (ATTN_F16 only) */
    int32_t n_suffix_tokens;     /* n = |S| */
    int32_t block_tokens;        /* B */
    int32_t dirty_tokens;        /* d-hat of Eq. 9; clamped to [0, n] */
    int32_t top_k;               /* blocks taken outside the dirty window, per layer (or once, LAYERS_SHARED) */
    int32_t layer_mode;          /* PATCHKV_LAYERS_* */
    const void* attn;            /* DEVICE fp16 [L][Hq][Q][n], token stride 1 (ATTN_F16) */
    int64_t attn_stride_layer;   /* elements */
    int64_t attn_stride_head;
    int64_t attn_stride_query;
    const uint64_t* mass;        /* DEVICE u64 [L][NB], units of 2^-24 (BLOCK_MASS) */
    uint64_t* mass_out;          /* DEVICE u64 [L][NB], optional: receives the exact block masses (ATTN_F16);
                                    when NULL the context's workspace holds them */
    uint8_t* repair_mask;        /* DEVICE u8  [L][NB]: 1 = block is in R_l */
    int32_t* repair_idx;         /* DEVICE i32 [L][NB]: R_l ascending, then -1 */
    int32_t* repair_cnt;         /* DEVICE i32 [L] */
    int32_t* reuse_idx;          /* DEVICE i32 [L][NB]: F_l ascending, then -1 */
    int32_t* reuse_cnt;          /* DEVICE i32 [L] */
    float* score_out;            /* DEVICE fp32, optional: Norm of Eq. 10 read as the share of the total, I_j = mass_j /
                                    sum of the row's masses (dirty window included; quotient in double, rounded once to
                                    fp32; an all-zero row gives zeros).  [L][NB] for LAYERS_INDEPENDENT, one row [NB] of
                                    the layer-summed masses for LAYERS_SHARED; the unit is a token ([L][n] / [n]) in
                                    patchkv_select_repair_tokens.  Reported only: ranking uses the exact masses. */
    /* Optional HOST mirrors (pinned memory) of the outputs, for a caller whose next step runs on the host
     * (patchkv_restore_from_host plans its copies from the reuse lists): each non-NULL pointer receives a copy of
     * the device array of the same name, enqueued on `stream` after the selection.  With sync_to_host != 0 the call
     * waits for `stream` before it returns, so the mirrors are valid on return (not inside a stream capture);
     * otherwise they are valid once the caller has synchronised `stream`. */
    uint8_t* host_repair_mask;   /* HOST u8  [L][NB] */
    int32_t* host_repair_idx;    /* HOST i32 [L][NB] */
    int32_t* host_repair_cnt;    /* HOST i32 [L] */
    int32_t* host_reuse_idx;     /* HOST i32 [L][NB] */
    int32_t* host_reuse_cnt;     /* HOST i32 [L] */
    int32_t sync_to_host;
    int32_t reserved;
} patchkv_select_args;

typedef struct {
    uint32_t struct_size;
    uint32_t n_copies;           /* host->device copies issued */
    uint64_t bytes_copied;       /* bytes that crossed the link */
    uint64_t bytes_useful;       /* bytes of reused records among them */
    uint64_t n_block_layers;     /* reused (layer, block) records */
    uint64_t bytes_direct;       /* of bytes_copied: read over the link by the kernel itself (no staging copy) */
} patchkv_restore_stats;

/* Create / destroy a context bound to one device.  Creation allocates two streams, a few events and the
 * 4-byte status word; workspaces grow on first use (a growing call synchronises the device once). */
PATCHKV_API int patchkv_create(patchkv_ctx** out, const patchkv_config* cfg);
PATCHKV_API int patchkv_destroy(patchkv_ctx* ctx);

/* Copies the text of the last host-side error of this context into buf (NUL-terminated, truncated to n). */
PATCHKV_API int patchkv_last_error(patchkv_ctx* ctx, char* buf, size_t n);

/* Section IV-C Eqs. 10-12 with the dirty window of Section IV-B Eq. 9, at block granularity.
 *   mass[l][j] = exact sum over heads, stored query positions and the tokens of block j of attn (each
 *                finite fp16 >= 0 is an integer number of 2^-24 units, so the sum is order-independent);
 *                a negative non-zero, infinite or NaN entry counts as zero and latches PATCHKV_E_BADINPUT.
 *   dirty      = blocks [0, ceil(min(max(dirty_tokens, 0), n) / B)).
 *   H_l        = the min(top_k, #candidates) non-dirty blocks of largest mass; ties go to the lower index.
 *   R_l = dirty u H_l and F_l = the rest, both ascending; unused list entries are set to -1.
 * Asynchronous on `stream`; all outputs are caller-allocated DEVICE arrays. */
/* Workspace: when the masses are computed here and no mass_out is given, or layer_mode is LAYERS_SHARED, the call
 * (and patchkv_select_repair_tokens always) uses ONE workspace owned by the context.  Selection calls on one
 * context must therefore be ordered on the GPU with respect to each other (same stream, or events between
 * streams); two that overlap race on it.  The workspace grows on demand, which synchronises the device and
 * reallocates: the first call, and any call with a larger problem, must not be made inside a stream capture. */
PATCHKV_API int patchkv_select_repair(patchkv_ctx* ctx, const patchkv_select_args* args, void* stream);

/* The selection in the form the paper prints it (Section IV-C, Eqs. 10-12): the importance score is per TOKEN,
 * H_l is the set of the top_k highest-scoring tokens outside the dirty token set D (ties: lower token index; the
 * caller turns the paper's fraction kappa into a count), and D u H_l is rounded to blocks only afterwards:
 * R_l = blocks holding a token of D u H_l.  (patchkv_select_repair ranks whole blocks by their summed mass, which
 * can pick different blocks.)  Same argument struct; differences: kind is PATCHKV_SCORE_ATTN_F16 (token mass is
 * the exact sum over heads and stored query positions) or PATCHKV_SCORE_TOKEN_MASS (`mass` is DEVICE u64 [L][n]);
 * `mass_out`, if given, is DEVICE u64 [L][n]; PATCHKV_LAYERS_SHARED ranks on the mass summed over layers, which
 * is the request-level score of Eq. 10.  Outputs exactly as for patchkv_select_repair. */
PATCHKV_API int patchkv_select_repair_tokens(patchkv_ctx* ctx, const patchkv_select_args* args, void* stream);

/* The selection of patchkv_select_repair for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the same kernels, not another step of the method.)
 *
 * Who needs it: a serving engine that reserves nearly all of HBM for its KV pool at start-up, after which a
 * cudaMalloc may simply fail; and a resume path that runs next to decode streams and cannot afford the
 * device-wide stall that creating a context, or growing its workspace, brings.  This entry point takes no
 * context and calls no cudaMalloc / cudaFree / allocating routine, now or later.  Its scratch -- the exact block
 * masses (L*NB u64 when kind is ATTN_F16) and the layer-summed masses (NB u64 when layer_mode is
 * LAYERS_SHARED) -- is a fixed array of PATCHKV_STATIC_MAX_MASS_ELEMS u64 inside the library image; each GPU
 * that loads the library holds those 2 MiB until the process exits.
 *
 *   - Runs on the CURRENT device; every pointer in `args` is memory of that device.  Inputs and outputs are
 *     the caller's, exactly as for patchkv_select_repair (mass_out, if given, receives a copy of the masses).
 *   - A problem whose scratch need, (ATTN_F16 ? L*NB : 0) + (LAYERS_SHARED ? NB : 0), exceeds
 *     PATCHKV_STATIC_MAX_MASS_ELEMS is refused with PATCHKV_E_TOO_LARGE and nothing is launched.
 *   - The first call on each device looks up the device address of the array (a host-side query, no
 *     allocation); make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the part that must
 *     start at zero is cleared on `stream` at each call.  Two calls whose work overlaps on the GPU (different
 *     streams, or a second call before the first has finished on another stream) race on it: serialise them.
 *   - `device_status` (DEVICE int32, optional, caller-zeroed) receives PATCHKV_E_BADINPUT if the stored
 *     attention held a negative, infinite or NaN entry; with NULL that latch is dropped.
 * Asynchronous on `stream`; results are bit-identical to patchkv_select_repair. */
PATCHKV_API int patchkv_select_repair_static(const patchkv_select_args* args, void* stream, int32_t* device_status);

/* Section IV-D fused restore (dequantise, Eq. 3 RoPE correction of K, page placement) of the reuse sets of
 * up to PATCHKV_MAX_SESSIONS sessions whose payloads are in device memory.  One kernel launch, asynchronous on
 * `stream`, no host synchronisation, no allocation; it can be captured in a CUDA graph.  The kernel is launched with
 * programmatic stream serialisation, so its set-up overlaps the tail of the kernel in front of it in the stream; it
 * touches no memory before that kernel has completed.
 * Launches from one context may overlap on the GPU when they are on different streams: the kernel's work counters
 * live in a slot that belongs to the stream (at most 190 different streams per context over its life), and a launch
 * recorded into a graph gets a slot of its own (at most 320 captured launches per context); beyond either limit the
 * call returns PATCHKV_E_UNSUPPORTED.  The kernel leaves its slot zeroed, so no reset is enqueued. */
PATCHKV_API int patchkv_restore(patchkv_ctx* ctx, const patchkv_geom* geom, const patchkv_pool* pool,
                                const patchkv_session* sessions, int n_sessions, void* stream);

/* The same restore with the payloads in PINNED host memory (the CPU-resident checkpoint of Section II-C /
 * Section V-A).  Only the records of F cross the link, layer by layer, by two routes at once: the long runs of records
 * that lie back to back in a layer payload (same-tag runs are contiguous in the checkpoint) are fetched by the copy
 * engine, one asynchronous copy per run on an internal copy stream into a ring of device staging slots (one layer of
 * one session per slot), and decoded by the restore kernel on an internal decode stream as soon as the layer has
 * landed; the layer's short runs are read over the link by a small side launch of the same kernel, whose bulk copies
 * address the pinned payload through its device alias, while the engine works.  Nothing but reused records is
 * transferred, and transfer and decode overlap.  PATCHKV_FLAG_HOST_STAGED (copy engine only, neighbouring ranges
 * merged across gaps of up to merge_gap_bytes) and PATCHKV_FLAG_HOST_DIRECT (no staging at all: one launch reads every
 * record itself) select the two routes on their own; a payload without a device alias is always staged.
 * The internal streams start after the work already on `stream` and `stream` waits for them before anything enqueued
 * later, so pages are complete for whatever follows on `stream`, also when the call returns an error half-way.
 * The call returns once everything is enqueued; host arrays are consumed before it returns, the pinned payload must
 * stay valid until the stream work completes.  `stats` is optional. */
PATCHKV_API int patchkv_restore_from_host(patchkv_ctx* ctx, const patchkv_geom* geom, const patchkv_pool* pool,
                                          const patchkv_session_host* sessions, int n_sessions, void* stream,
                                          patchkv_restore_stats* stats);

/* ---- precision planner (offload side) -----------------------------------------------------------------------
 * Section IV-D, Eqs. 13-14: for every block b of the suffix, Z_i = sqrt(A_i * e_i) over its tokens (A_i the
 * normalised stored attention mass, e_i the normalised residual of the candidate low-bit value representation),
 * r_b = alpha * max_i Z_i + (1 - alpha) * mean_i Z_i, and the frozen tag
 *     r_b >= tau_H                  -> PATCHKV_TAG_BF16 (full precision)
 *     tau_L <= r_b < tau_H          -> PATCHKV_TAG_INT8 (K8/V8)
 *     r_b < tau_L and G4(b)         -> PATCHKV_TAG_INT4 (K8/V4)
 *     r_b < tau_L and not G4(b)     -> PATCHKV_TAG_INT8
 * The low-bit test G4 is not spelled out in the paper; here G4(b) = (max_i e_i <= eps4).  The calibration that
 * produces alpha, tau_L, tau_H, eps4 and the measurement of e_i are the caller's.  fp32 throughout, tokens in
 * ascending order, every operation rounded on its own.
 *   attn, resid  DEVICE fp32 [n]     tags DEVICE u8 [NB] (out)     risk DEVICE fp32 [NB] (out, optional) */
PATCHKV_API int patchkv_plan_precision(patchkv_ctx* ctx, const float* attn, const float* resid, int n_suffix_tokens,
                                       int block_tokens, float alpha, float tau_L, float tau_H, float eps4,
                                       uint8_t* tags, float* risk, void* stream);

/* ---- checkpoint writer (offload side; not on the resume path) ----------------------------------------------
 * Section IV-D: at offload a fused kernel gathers the rows of each suffix block, computes the scales and packs
 * the payload at the block's calibrated precision; blocks of the same representation form contiguous runs.
 *
 * patchkv_plan_checkpoint fills the directory of that clustered layout from the tags: per layer all BF16-tag
 * records, then INT8, INT4, K4V4, each run in ascending block index.
 *   tags      DEVICE u8  [L][NB]  (in)      blk_off DEVICE u64 [L][NB] (out)     layer_bytes DEVICE u64 [L] (out)
 * An unknown tag gets blk_off = UINT64_MAX (the writer then skips that block) and latches PATCHKV_E_BOUNDS. */
PATCHKV_API int patchkv_plan_checkpoint(patchkv_ctx* ctx, const patchkv_geom* geom, int n_suffix_tokens,
                                        const uint8_t* tags, uint64_t* blk_off, uint64_t* layer_bytes, void* stream);

/* patchkv_quantize_gather writes the record of every block of every layer of one session from the paged pool.
 * `session` is read as for patchkv_restore, with the roles reversed: block_table / dst_shift locate the SOURCE
 * rows in `pool`, tags / blk_off / layer_payload / layer_bytes describe the DESTINATION records (layer_payload
 * buffers are written), delta and the reuse lists are ignored.  Quantiser, per group of `group` channels of one
 * (token, head): s = fp16(amax / qmax) (fp32 division, round to nearest even), code = clamp(rint(x / s), -qmax,
 * qmax) with ties to even, s == 0 -> code 0; qmax = 127 for int8 and 7 for int4; a bf16 section copies the 16
 * bits; tokens past the end of the suffix encode as zeros.  Values must be finite; a group whose amax / qmax
 * exceeds 65504 gets an infinite scale and all-zero codes.
 * Needs group in {8, 16, 32, 64, 128, 256}.  A block whose tag, record extent or source pages are out of range
 * is skipped whole and PATCHKV_E_BOUNDS is latched.  One launch, asynchronous on `stream`, no allocation; it hands
 * out its blocks from the work counters of the stream's slot, as patchkv_restore does (same limits on streams and
 * on launches captured into graphs), and leaves them zeroed. */
PATCHKV_API int patchkv_quantize_gather(patchkv_ctx* ctx, const patchkv_geom* geom, const patchkv_pool* pool,
                                        const patchkv_session* session, void* stream);

/* Offload of one session to a CPU-resident checkpoint: patchkv_plan_checkpoint, then per layer patchkv_quantize_gather
 * into a slot of the device staging ring and an asynchronous device-to-host copy of the finished layer payload into
 * PINNED host memory, so that encoding layer l+1 overlaps copying layer l out.
 *   session              as for patchkv_quantize_gather; its blk_off and layer_bytes (DEVICE, caller-allocated) are
 *                        WRITTEN by the plan step and stay valid as the checkpoint's directory; layer_payload is ignored
 *   host_layer_payload   HOST array of L PINNED destination pointers (16-byte aligned)
 *   host_layer_capacity  HOST u64 [L]: bytes available behind each pointer (B*H*D*4*NB always suffices)
 *   host_layer_bytes     HOST u64 [L] (out): bytes of each layer payload
 * The call synchronises `stream` once, after the plan, to learn the layer sizes; everything else is enqueued on
 * internal streams that `stream` waits for, as in patchkv_restore_from_host. */
PATCHKV_API int patchkv_checkpoint_to_host(patchkv_ctx* ctx, const patchkv_geom* geom, const patchkv_pool* pool,
                                           const patchkv_session* session, void* const* host_layer_payload,
                                           const uint64_t* host_layer_capacity, uint64_t* host_layer_bytes,
                                           void* stream);

/* Synchronises the context's device work and returns in *device_status the first device-side error latched
 * since the last query (PATCHKV_OK, PATCHKV_E_BOUNDS, PATCHKV_E_BADINPUT or PATCHKV_E_TIMEOUT), then clears it. */
PATCHKV_API int patchkv_query_status(patchkv_ctx* ctx, int* device_status);

/* Diagnostic (the paper has no counterpart).  Every barrier wait inside the pipeline kernels is bounded: after a fixed
 * number of polls the waiting role gives up, raises the CTA's abort flag, lets the copies in flight land and the kernel
 * latches PATCHKV_E_TIMEOUT instead of spinning.  This call runs that same wait, in a one-CTA kernel of its own, on a
 * barrier that nothing completes, with a limit of `max_polls` polls (1 .. 2^20; microseconds to a fraction of a
 * second), so that a caller can check that the limit expires, that patchkv_query_status then reports
 * PATCHKV_E_TIMEOUT, and that the context keeps working afterwards.  Asynchronous on `stream`. */
PATCHKV_API int patchkv_selftest_bounded_wait(patchkv_ctx* ctx, uint32_t max_polls, void* stream);

/* Diagnostic (the paper has no counterpart).  Arms the NEXT launch of a bulk-copy pipeline kernel on this context
 * (patchkv_restore, one launch of patchkv_restore_from_host, patchkv_quantize_gather, or the per-token mass kernel of
 * patchkv_select_repair_tokens on a regular attention shape) to run with a wait limit of
 * `max_polls` polls (1 .. 2^20) and to have the consumer warps of every CTA withhold the `empty` arrivals of
 * their unit number `after_units` (0-based), so that the warp that feeds the ring runs out of patience while copies it
 * issued earlier are still landing or have landed.  That launch then takes the path a real timeout would take:
 * the CTA's abort flag is raised, every role leaves its loop, the feeding warp waits (bounded) for its copies in
 * flight so that none of them can write the shared memory of a CTA that has gone, and PATCHKV_E_TIMEOUT is latched.
 * Blocks the launch did not get to are left untouched; no page outside the reuse set is written.  The launch after
 * it runs normally.  Nothing here faults or spins without a limit. */
PATCHKV_API int patchkv_selftest_stall_next_launch(patchkv_ctx* ctx, int32_t after_units, uint32_t max_polls);

/* Bytes of one block record for a tag under a geometry; 0 for an unknown tag. */
PATCHKV_API uint64_t patchkv_record_bytes(int tag, int block_tokens, int n_kv_heads, int head_dim, int group);

#ifdef __cplusplus
}
#endif
#endif /* PATCHKV_H_ */
