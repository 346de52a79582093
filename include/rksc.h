/*
 * rksc.h - C ABI of the B200 (sm_100a) ASKS hot path: the similarity gate and
 * multi-branch decode attention over a paged bf16 KV pool in which every branch
 * mapped onto a shared prefix reads that prefix's pages once.
 *
 * Conventions
 *   - Every call returns an int32_t status: RKSC_OK (0) or a negative RKSC_ERR_*.
 *     Nothing throws, prints or exits.  rksc_strerror() names a status.
 *   - "dev" pointers are device memory owned by the caller; "host" pointers are
 *     host memory owned by the caller.  The library never frees caller memory.
 *     It owns only rksc_plan objects and tables filled by rksc_tables_from_gate
 *     (released with rksc_plan_destroy / rksc_tables_free).
 *   - Device work is enqueued on the caller's stream (a cudaStream_t passed as
 *     void*, NULL = default stream) and is asynchronous.  The compute calls do not
 *     synchronise the host.
 *   - bf16 tensors are passed as const void* (2 bytes per element).
 *   - The device must be compute capability 10.x; other devices give
 *     RKSC_ERR_UNSUPPORTED.
 */
#ifndef RKSC_H_
#define RKSC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RKSC_OK                   0
#define RKSC_ERR_INVALID_ARG     (-1)  /* NULL pointer, non-positive size, misaligned buffer       */
#define RKSC_ERR_UNSUPPORTED     (-2)  /* head_dim not 64/128, block_size not 16, device not sm_100 */
#define RKSC_ERR_BAD_TABLE       (-3)  /* page id out of range, token count inconsistent with pages */
#define RKSC_ERR_WORKSPACE       (-4)  /* workspace too small or misaligned                         */
#define RKSC_ERR_CUDA            (-5)  /* a CUDA runtime/driver call failed (or no device present)  */
#define RKSC_ERR_DEVICE_TIMEOUT  (-6)  /* value a kernel writes to device_status when a wait ran out */
#define RKSC_ERR_NOMEM           (-7)  /* host allocation failed                                    */

#define RKSC_BLOCK_SIZE 16

#if defined(__GNUC__)
#define RKSC_API __attribute__((visibility("default")))
#else
#define RKSC_API
#endif

RKSC_API const char* rksc_strerror(int32_t status);
/* Text of the CUDA error behind the calling thread's most recent RKSC_ERR_CUDA from a launch. */
RKSC_API const char* rksc_last_cuda_error(void);

/* Self-test of the bounded-wait mechanism every kernel of this library uses: launches one small CTA
 * whose warps wait on a shared-memory barrier that nothing ever completes, with a limit of
 * `limit_cycles` SM cycles (the production kernels' limit is 2^32).  When the limit runs out the
 * waiting warps record RKSC_ERR_DEVICE_TIMEOUT in *device_status (dev int32, zeroed by the caller),
 * stop waiting and the kernel returns normally: the context stays usable and nothing traps.
 * limit_cycles in [1, 2^31].  Asynchronous on `stream`. */
RKSC_API int32_t rksc_debug_wait_timeout(int64_t limit_cycles, int32_t* device_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * ASKS similarity gate  (paper Eq. 2 and Algorithm 2)
 *
 *   w_l     = exp(alpha*l/L) / sum_l' exp(alpha*l'/L),  l = 1..L
 *   sigma_b = sum_l w_l * <h_b^l, h_r^l> / (|h_b^l| |h_r^l|),   r = cand_prefix[b]
 *   branch_to_prefix[b] = r if sigma_b >= tau else -1           (">=": Alg. 2 line 6)
 *
 * h_branch  dev [B][L][D] fp32, one vector per (branch, layer)
 * h_root    dev [P][L][D] fp32, raw or already unit-norm (the norm is always divided out)
 * cand_prefix dev [B] int32 in [0,P): the root each branch is compared with
 * branch_to_prefix dev [B] int32 out; sigma dev [B] fp32 out, may be NULL
 * A zero-norm vector contributes 0 for its layer; NaN inputs give -1.  An out-of-range
 * candidate gives -1 and sigma = NaN.  Arithmetic is fp32 (tree reductions): the map is
 * exact whenever |sigma - tau| is above ~1e-5.
 * One kernel launch on `stream`; no workspace.  D and L are arbitrary positive sizes
 * (16-byte loads are used when D % 4 == 0 and both bases are 16-byte aligned).
 * ------------------------------------------------------------------------------------------ */
RKSC_API int32_t rksc_asks_gate(const float* h_branch, const float* h_root, const int32_t* cand_prefix,
                       int32_t B, int32_t P, int32_t L, int32_t D,
                       float alpha, float tau,
                       int32_t* branch_to_prefix, float* sigma, void* stream);

/* ------------------------------------------------------------------------------------------
 * KV pool layout and block tables
 *
 * Pool: K and V are separate dev tensors [num_pool_blocks][num_kv_heads][16][head_dim] bf16,
 * 16-byte aligned.  Query head h reads KV head h / (num_q_heads / num_kv_heads).
 * Token slots of a listed page that lie past its segment's token count are never attended to
 * (their scores are masked and their probabilities are exactly 0), but they are fetched with the
 * page and multiplied by those zeros: they must hold finite values (not NaN / Inf).
 *
 * Tables (segment form): segment s owns pages seg_blocks[seg_block_off[s] .. seg_block_off[s+1])
 * and seg_num_tokens[s] tokens; every page but the last is full, the last holds at least one
 * token (a segment may also be empty: no pages, 0 tokens).  Branch b attends to the segments
 * br_segs[br_seg_off[b] .. br_seg_off[b+1]) in that (root-to-leaf) order; a segment listed by
 * several branches is a shared prefix.  This is what replaces the B physical copies of the
 * prefix cache that the paper's Algorithm 1 (line 3) makes.
 * The "logical block" j of a branch is the j-th page of that concatenation.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim;         /* 64 or 128 */
    int32_t block_size;       /* 16 */
    float   sm_scale;         /* <= 0 selects 1/sqrt(head_dim) */
    int32_t num_pool_blocks;
} rksc_layout;

typedef struct {
    int32_t num_branches;
    int32_t num_segments;
    const int32_t* seg_block_off;   /* host [S+1] */
    const int32_t* seg_blocks;      /* host, physical page ids */
    const int32_t* seg_num_tokens;  /* host [S]   */
    const int32_t* br_seg_off;      /* host [B+1] */
    const int32_t* br_segs;         /* host       */
} rksc_tables;

/* Tables from a gate map for the two-level case (P shared prefixes; per branch a private
 * prefix copy and a suffix).  All arguments are host pointers; *_off are CSR offsets into the
 * page-id arrays, *_ntok the token counts.  Branch b uses shared prefix branch_to_prefix[b]
 * when that is >= 0 and otherwise its private prefix list (the paper's "independent
 * recomputation" for branches below tau, Section 2.2), followed by its suffix.
 * Segment numbering: shared prefixes by ascending id (only those with a sharer), private
 * prefixes of the non-sharing branches by ascending branch, then all suffixes by ascending
 * branch.  `out` is filled with arrays the library allocates; release with rksc_tables_free.
 * Errors: RKSC_ERR_INVALID_ARG (NULL, map entry >= P), RKSC_ERR_NOMEM. */
RKSC_API int32_t rksc_tables_from_gate(int32_t B, int32_t P, const int32_t* branch_to_prefix,
                              const int32_t* shared_off, const int32_t* shared_pages, const int32_t* shared_ntok,
                              const int32_t* priv_off,   const int32_t* priv_pages,   const int32_t* priv_ntok,
                              const int32_t* sfx_off,    const int32_t* sfx_pages,    const int32_t* sfx_ntok,
                              rksc_tables* out);
RKSC_API void rksc_tables_free(rksc_tables* t);

/* ------------------------------------------------------------------------------------------
 * Plan: validated tables turned into device work lists.
 *
 * rksc_plan_create checks the tables (RKSC_ERR_BAD_TABLE), groups each segment with the
 * ascending list of branches that share it, cuts segments into KV chunks sized for the
 * device's SM count, lays out the partial-result workspace and the block-mass output, and
 * uploads its lists to the current device (synchronously, on a stream of the library's own; device
 * and pinned staging memory are taken from a small cache that destroyed plans return theirs to, so
 * creating a plan per decode step does not allocate in the steady state).  A plan may be destroyed
 * while its last launch is still running: its memory is not reused before that launch has finished.
 * Without a CUDA device the plan is host-only: it can be queried but not run.
 * A plan holds a small device-side work counter that a launch uses and rewinds, so a plan may
 * be in flight on one stream at a time (create one plan per concurrent stream).  It does not
 * keep pointers into `tables`.
 * ------------------------------------------------------------------------------------------ */
typedef struct rksc_plan rksc_plan;

typedef struct {
    size_t  workspace_bytes;     /* required size of the attention workspace              */
    int64_t mass_elems;          /* floats in block_mass: num_q_heads * sum_b nblk_b      */
    const int64_t* mass_off;     /* host [B+1], owned by the plan: sum of nblk over b' < b */
    int32_t num_work_items;      /* work items of the segment kernels (their persistent CTAs claim them) */
    int32_t num_partial_rows;    /* (row, chunk) partial results merged at the end        */
    int64_t unique_kv_tokens;    /* valid tokens of the distinct segments referenced       */
    int64_t duplicated_kv_tokens;/* sum over branches of the tokens they attend to        */
    int32_t on_device;           /* 1 when the lists were uploaded                        */
    int64_t num_pages_listed;    /* page ids in the tables (sum of the segments' pages)    */
    int32_t num_kernel_launches; /* kernels one attention call launches with this plan     */
} rksc_plan_info;

RKSC_API int32_t rksc_plan_create(const rksc_layout* layout, const rksc_tables* tables, rksc_plan** out);
/* rksc_tables_from_gate followed by rksc_plan_create, without handing the tables back: the usual
 * per-step call when the tables come from the gate map (arguments as rksc_tables_from_gate). */
RKSC_API int32_t rksc_plan_create_from_gate(const rksc_layout* layout, int32_t B, int32_t P,
                              const int32_t* branch_to_prefix,
                              const int32_t* shared_off, const int32_t* shared_pages, const int32_t* shared_ntok,
                              const int32_t* priv_off,   const int32_t* priv_pages,   const int32_t* priv_ntok,
                              const int32_t* sfx_off,    const int32_t* sfx_pages,    const int32_t* sfx_ntok,
                              rksc_plan** out);
RKSC_API int32_t rksc_plan_query(const rksc_plan* plan, rksc_plan_info* info);
/* Work item i as 10 int32: segment, kv_head, first page (index within the segment), pages,
 * tokens, first sharer (index within the segment's sharer list), sharers, first partial row,
 * kernel class (0 = warp MMA), reserved.  For tests and tools. */
RKSC_API int32_t rksc_plan_get_item(const rksc_plan* plan, int32_t i, int32_t* out10);
RKSC_API void    rksc_plan_destroy(rksc_plan* plan);

/* ------------------------------------------------------------------------------------------
 * Branch-decode attention  (the attention inside the paper's batched decode on the shared
 * cache: Algorithm 1 line 4, Section 2.2 "KV broadcast and batched decode")
 *
 *   out[b][h][:]       = softmax_j(scale * q[b][h] . k_j) V     over all tokens j of branch b
 *   block_mass[b][h][j] = sum of those softmax probabilities over the tokens of logical block j
 *
 * q          dev [B][Hq][d] bf16 (one decode query per branch and head), 16-byte aligned
 * k_pool, v_pool  dev bf16 pools (see above)
 * out        dev [B][Hq][d] fp32
 * block_mass dev fp32 or NULL; entry (b,h,j) at mass_off[b]*Hq + h*nblk_b + j; sums to 1 over
 *            j for every (b,h) with at least one token.  This is the per-block attention score
 *            an attention-weighted eviction policy (the paper's RSBCM, Algorithm 4) consumes.
 * workspace  dev, >= workspace_bytes, 256-byte aligned; contents need not be initialised
 * device_status dev int32 or NULL.  Kernels only ever write a nonzero RKSC_ERR_* there (when a
 *            bounded wait inside a kernel ran out); the caller zeroes it beforehand and reads
 *            it after synchronising.
 * Each prefix page shared by n branches is fetched from HBM once per KV head and serves all
 * n * (Hq/Hkv) stacked query rows.  A branch without tokens gets out = 0.
 * Launches: the segment-attention kernels (tensor-core and / or warp-MMA, as the plan needs) and one
 * merge kernel on `stream`.  Work is handed out dynamically, but every work item's arithmetic and the
 * order of the merge are fixed: the same plan and inputs give the same bits on every call.
 * ------------------------------------------------------------------------------------------ */
RKSC_API int32_t rksc_branch_decode_attention(const rksc_plan* plan, const void* q,
                                     const void* k_pool, const void* v_pool,
                                     float* out, float* block_mass,
                                     void* workspace, size_t workspace_bytes,
                                     int32_t* device_status, void* stream);

/* The same call restricted to some of its launches, so that a profiler or a benchmark can put
 * CUDA events between them: RKSC_PHASE_SEGMENTS runs the segment-attention kernel (partials and
 * log2 masses), RKSC_PHASE_MERGE the merge kernel (out and final masses).  The merge phase must
 * follow the segment phase on the same stream with the same arguments.
 * rksc_branch_decode_attention == phases (RKSC_PHASE_SEGMENTS | RKSC_PHASE_MERGE). */
#define RKSC_PHASE_SEGMENTS 1
#define RKSC_PHASE_MERGE    2
/* Added to RKSC_PHASE_MERGE: the merge kernel is launched as an ordinary successor of the segment
 * kernels instead of with programmatic stream serialisation.  By default its blocks may take their
 * places on the SMs while the segment kernel drains (and wait there); that saves a little when the
 * call runs alone, but where other streams have kernels waiting for those SMs (the gate kernels of
 * later steps in rksc_pipeline) it is better to leave the drain to them: the step pipeline sets this
 * flag (measured: 0.178 instead of 0.185 ms per step on the batched-serving configuration). */
#define RKSC_PHASE_MERGE_LATE 4
RKSC_API int32_t rksc_branch_decode_attention_phases(const rksc_plan* plan, const void* q,
                                     const void* k_pool, const void* v_pool,
                                     float* out, float* block_mass,
                                     void* workspace, size_t workspace_bytes,
                                     int32_t* device_status, void* stream, int32_t phases);

/* ------------------------------------------------------------------------------------------
 * rksc_decode_step_host: the whole path (gate -> tables -> plan -> attention) in one call for a
 * caller whose per-step data lives in host memory (paper Algorithm 1 lines 2-4 restricted to the
 * ASKS gate and the attention of one decode step of one layer).
 *
 * Host inputs (pinned memory makes the copies asynchronous): h_branch [B][L][D], h_root [P][L][D]
 * fp32, cand_prefix [B], the three page-list CSRs of rksc_tables_from_gate, q [B][Hq][d] bf16.
 * Device inputs: the resident KV pool (k_pool, v_pool) - a KV cache is device state written by
 * earlier steps, not a per-step input.
 * Host outputs: branch_to_prefix [B], sigma [B] (may be NULL), out [B][Hq][d] fp32, block_mass
 * (may be NULL; capacity in floats, RKSC_ERR_INVALID_ARG if smaller than the plan's mass_elems),
 * mass_off [B+1] (may be NULL).
 * The call allocates its device scratch stream-ordered (cudaMallocAsync / cudaFreeAsync on
 * `stream`), synchronises the stream twice (after the gate, and at the end), and returns the
 * status of the first failing stage or the device_status word of the attention.
 * ------------------------------------------------------------------------------------------ */
RKSC_API int32_t rksc_decode_step_host(
    const rksc_layout* layout,
    const float* h_branch, const float* h_root, const int32_t* cand_prefix,
    int32_t B, int32_t P, int32_t L, int32_t D, float alpha, float tau,
    const int32_t* shared_off, const int32_t* shared_pages, const int32_t* shared_ntok,
    const int32_t* priv_off,   const int32_t* priv_pages,   const int32_t* priv_ntok,
    const int32_t* sfx_off,    const int32_t* sfx_pages,    const int32_t* sfx_ntok,
    const void* q, const void* k_pool, const void* v_pool,
    int32_t* branch_to_prefix, float* sigma, float* out, float* block_mass,
    int64_t block_mass_capacity, int64_t* mass_off, void* stream);

/* ------------------------------------------------------------------------------------------
 * rksc_branch_decode_attention_static: the same attention for callers that cannot allocate.
 * (No counterpart in the paper: this is a packaging variant of the call above.)
 *
 * Some callers have no way to supply the workspace: a serving process that handed all device
 * memory to its own pool at start-up and must not grow, a plug-in that is forbidden to call
 * the allocating CUDA entry points, or a latency path that cannot afford the device-wide
 * synchronisation an allocation may imply.  For them this entry point takes no workspace: the
 * partial results go to a scratch array that is compiled into the library
 * (RKSC_STATIC_WORKSPACE_BYTES of device memory on every GPU that loads the library, held
 * until the process exits).  The call itself allocates and frees nothing, on the host side too
 * it only launches kernels.  Inputs, outputs and device_status are passed as above; the plan
 * was created beforehand with rksc_plan_create (that call does allocate).
 *
 *   - A plan that needs more than RKSC_STATIC_WORKSPACE_BYTES (see rksc_plan_query) is
 *     refused with RKSC_ERR_WORKSPACE before anything is launched: use the call above.
 *   - The first call on a device looks up the scratch array's device address (once per
 *     device, with that device current) and keeps it.  Make that first call during set-up,
 *     before any stream capture is begun on the device.
 *   - Every call on a device uses the same scratch array.  Nothing in it has to start at
 *     zero (each launch writes every partial row it later reads), so nothing is cleared and
 *     the previous call's partials simply stay there until overwritten.  Two calls that may
 *     overlap on the GPU (different streams, or different plans in flight together) race on
 *     it: keep calls of this entry point ordered on one stream per device.
 * Errors: as rksc_branch_decode_attention, plus RKSC_ERR_WORKSPACE as described.
 * ------------------------------------------------------------------------------------------ */
#define RKSC_STATIC_WORKSPACE_BYTES (16u << 20)
RKSC_API int32_t rksc_branch_decode_attention_static(const rksc_plan* plan, const void* q,
                                     const void* k_pool, const void* v_pool,
                                     float* out, float* block_mass,
                                     int32_t* device_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * RSBCM eviction (paper Section 2.4 "RSBCM" and Algorithm 4), fed by the attention's block
 * masses.  The paper ranks a cached block by omega = score / (depth + 1) and, while more than
 * N_max blocks are cached, evicts the block with the smallest omega.  It does not say how an
 * attention-derived score is formed; here the score of a table entry e = seg_block_off[s] + p
 * (page p of segment s) is the softmax mass that every (branch, query head) attending to the
 * segment put on that page, summed.
 *
 * rksc_rsbcm_page_scores: score[e] for every entry the plan's tables list (device, fp64,
 * [num_pages_listed]).  score[e] = sum over the branches b listing s, in ascending b (a branch
 * listing s twice counts twice), of (sum over heads h = 0..Hq-1 of block_mass[b][h][j]), j the
 * logical block of the page in b.  Each head sum is formed first, in ascending h, then added to
 * the running score, all in fp64 and in exactly this order: the result is defined bit for bit.
 * block_mass is the array rksc_branch_decode_attention wrote for the same plan.
 * Errors: RKSC_ERR_INVALID_ARG (NULL argument, plan without device lists), RKSC_ERR_CUDA.
 * ------------------------------------------------------------------------------------------ */
RKSC_API int32_t rksc_rsbcm_page_scores(const rksc_plan* plan, const float* block_mass, double* score,
                                        void* stream);

/* ------------------------------------------------------------------------------------------
 * rksc_rsbcm_evict: Algorithm 4 on n entries.  omega[i] = score[i] / (depth[i] + 1) as one IEEE
 * fp64 division; with k = max(0, n - capacity) the k entries that are smallest by (omega, i)
 * are marked - the set the paper's loop (evict the arg-min, the first of equal minima, until at
 * most N_max = capacity entries remain) ends with, since evicting an entry changes no other
 * entry's omega.
 *
 * Device arguments: score fp64 [n] (finite), depth int32 [n] (>= 0), evicted uint8 [n] (out,
 * 1 = evict, every element written), num_evicted int32 [1] (out, may be NULL), workspace of at
 * least rksc_rsbcm_workspace_bytes(n) bytes, 256-byte aligned, contents irrelevant before and
 * undefined after.  The selection runs in one thread block (an exact radix select over the
 * 64 bits of omega), so its time grows linearly with n.
 * Errors: RKSC_ERR_INVALID_ARG (NULL argument, n < 0, n >= 2^31), RKSC_ERR_WORKSPACE, RKSC_ERR_CUDA.
 * ------------------------------------------------------------------------------------------ */
RKSC_API size_t rksc_rsbcm_workspace_bytes(int64_t n);
RKSC_API int32_t rksc_rsbcm_evict(const double* score, const int32_t* depth, int64_t n, int64_t capacity,
                                  uint8_t* evicted, int32_t* num_evicted, void* workspace,
                                  size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * rksc_tables_drop_evicted: the tables after eviction (host arrays in, host arrays out).  Each
 * segment keeps its surviving pages in order; a dropped page takes its tokens with it (every
 * page of a segment holds RKSC_BLOCK_SIZE tokens except the last, which holds the remainder); a
 * segment may end up empty.  Branch lists are copied unchanged.  evicted is uint8
 * [seg_block_off[S]].  `out` is allocated by the library: release it with rksc_tables_free.
 * Errors: RKSC_ERR_INVALID_ARG, RKSC_ERR_BAD_TABLE (offsets not ascending, token count that
 * does not fit the page count), RKSC_ERR_NOMEM.
 * ------------------------------------------------------------------------------------------ */
RKSC_API int32_t rksc_tables_drop_evicted(const rksc_tables* in, const uint8_t* evicted, rksc_tables* out);

/* ------------------------------------------------------------------------------------------
 * Suffix prefill on the shared cache (paper Section 2.2, "KV broadcast and batched decode":
 * y_b = f(s_b | C_B); Appendix "Stepwise Batched Decode", step (1)).  The s tokens of every
 * branch's suffix are attended in one pass: query token i of branch b stands at position
 * T_b - s + i of the branch's token sequence (the keys and values of the s tokens are the last s
 * tokens the branch's tables list) and attends to every position up to and including its own.
 *
 * rksc_tables_for_suffix_prefill turns that into a decode attention over B * s virtual branches,
 * which rksc_plan_create / rksc_branch_decode_attention then run on the same kernels: virtual
 * branch b * s + i is query token i of branch b.  It lists every segment of b but the last
 * unchanged (a shared prefix stays shared, now by s times as many rows), then two new segments
 * cut from b's last segment: its pages that lie wholly before the first of the s tokens (shared
 * by the s virtual branches of b; may be empty), and the pages from there up to the one holding
 * token i, with only the tokens up to token i's own counted.  New segments are numbered after the S original ones:
 * the common part of b is S + b * (s + 1), the part of token i is S + b * (s + 1) + 1 + i; a
 * branch without segments gets s + 1 empty segments and s empty virtual branches.  The logical
 * blocks of a virtual branch are the leading blocks of the branch in the same order (blocks that
 * hold only later tokens are not listed), so block_mass of virtual branch b * s + i is the mass
 * query token i puts on the branch's blocks.
 * Call the attention with q [B * s][Hq][d] (token-major within a branch) and out likewise.
 * Host arrays in, host arrays out; `out` is allocated by the library (rksc_tables_free).
 * Errors: RKSC_ERR_INVALID_ARG (NULL, s < 1), RKSC_ERR_BAD_TABLE (inconsistent tables, or the
 * last segment of a branch holds fewer than s tokens), RKSC_ERR_UNSUPPORTED (sizes beyond 2^30),
 * RKSC_ERR_NOMEM.
 * ------------------------------------------------------------------------------------------ */
RKSC_API int32_t rksc_tables_for_suffix_prefill(const rksc_tables* in, int32_t s, rksc_tables* out);

/* ------------------------------------------------------------------------------------------
 * CGEE numerics (paper Section 2.3, "CGEE: Confidence-Gated Early Exit"; Algorithm 3).
 *
 * rksc_cgee_logit_entropy: for every row h_b of h (bf16 [B][D], device) the entropy, in nats, of
 * p = softmax(h_b W_u^T) (Eq. 5) and its largest probability max_v p_v (the summand of the
 * generation confidence, Eq. 3), fused with the unembedding product: W_u (bf16 [V][D], device,
 * row-major) is read once per block of 16 rows of h and no logit is stored.  Products are bf16 x
 * bf16 accumulated in fp32 on the tensor cores; the softmax statistics are fp32.
 * entropy, top1_prob: device fp32 [B], either may be NULL (not both).  workspace: device, at least
 * rksc_cgee_workspace_bytes() bytes, 16-byte aligned.  device_status (may be NULL): a device
 * int32 that receives RKSC_ERR_DEVICE_TIMEOUT if a bounded wait inside the kernel ran out (the
 * caller zeroes it).  Requires D a multiple of 8, D <= 4096 (the 16 rows of h stay in shared
 * memory), h and w_u 16-byte aligned.
 * Errors: RKSC_ERR_INVALID_ARG, RKSC_ERR_UNSUPPORTED (D, V >= 2^31), RKSC_ERR_WORKSPACE,
 * RKSC_ERR_CUDA.
 *
 * rksc_cgee_entropy_exit: Algorithm 3's test for layer `layer`, per row:
 * exit_flags[b] = (layer >= l_min && entropy[b] < theta && |entropy[b] - entropy_prev[b]| < eps),
 * in fp32; entropy_prev = +inf before the first layer.  Device arrays [B].
 *
 * rksc_cgee_verify_skip: the Level-1 gate (Eq. 3 and 4).  top1_per_step is device fp32 [t][B]
 * (the largest softmax probability of every decode step of every branch); confidence[b] (device
 * [B], may be NULL) receives the mean over the t steps (summed in step order, fp32), and skip[0]
 * (device int32) = (max_b p >= tau_conf && (max_b p - second largest) / max_b p >= r_gap), the
 * second largest taken as 0 when B = 1; 0 when B = 0.
 * ------------------------------------------------------------------------------------------ */
RKSC_API size_t rksc_cgee_workspace_bytes(void);
RKSC_API int32_t rksc_cgee_logit_entropy(const void* h, const void* w_u, int32_t B, int32_t D, int64_t V,
                                         float* entropy, float* top1_prob, void* workspace,
                                         size_t workspace_bytes, int32_t* device_status, void* stream);
RKSC_API int32_t rksc_cgee_entropy_exit(const float* entropy, const float* entropy_prev, int32_t B, int32_t layer,
                                        int32_t l_min, float theta, float eps, int32_t* exit_flags, void* stream);
RKSC_API int32_t rksc_cgee_verify_skip(const float* top1_per_step, int32_t t, int32_t B, float tau_conf,
                                       float r_gap, float* confidence, int32_t* skip, void* stream);

/* ------------------------------------------------------------------------------------------
 * Token-by-token decode on the paged cache (paper Appendix "Stepwise Batched Decode", step (2)).
 * One decode step = rksc_tables_append_token (host: where each branch's new token goes, and the
 * tables afterwards), rksc_kv_append (device: the new keys and values into the pool), then a plan
 * from the new tables and rksc_branch_decode_attention as for any step.
 *
 * rksc_tables_append_token: every branch that lists segments gains one token at the end of its
 * last segment, which no other branch (and no other position of that branch) may list - its
 * private suffix.  When that segment's pages are full (or it has none) page new_pages[b] is
 * appended to it first (new_pages may be NULL if no branch needs one).  page[b], slot[b] (host
 * arrays [B], out) say where branch b's token is stored: k_pool[page][kvh][slot][:]; -1, -1 for
 * a branch without segments.  `out` is allocated by the library (rksc_tables_free).
 * Errors: RKSC_ERR_INVALID_ARG (NULL arguments, a needed new page missing or negative),
 * RKSC_ERR_BAD_TABLE (inconsistent tables, a shared last segment), RKSC_ERR_NOMEM.
 *
 * rksc_kv_append: k_pool[page[b]][h][slot[b]][:] = k_new[b][h][:] (v likewise) for every branch
 * with page[b] >= 0; entries outside the pool are skipped.  Device pointers: pools as for the
 * attention, k_new / v_new bf16 [B][Hkv][d], page / slot int32 [B]; all 16-byte aligned.
 * ------------------------------------------------------------------------------------------ */
RKSC_API int32_t rksc_tables_append_token(const rksc_tables* in, const int32_t* new_pages, rksc_tables* out,
                                          int32_t* page, int32_t* slot);
RKSC_API int32_t rksc_kv_append(const rksc_layout* layout, void* k_pool, void* v_pool, const void* k_new,
                                const void* v_new, int32_t B, const int32_t* page, const int32_t* slot, void* stream);

/* ------------------------------------------------------------------------------------------
 * Step pipeline: whole steps of the path (gate -> map to the host -> tables + plan -> attention,
 * paper Algorithm 1 lines 2-4 restricted to ASKS and the decode attention) kept `depth` deep in
 * flight by the library itself, for callers whose steps do not depend on each other's results
 * (independent batches, the layers' gates of later requests, a serving loop).
 *
 * The tables of a step depend on its gate map, which has to come to the host; a caller that runs
 * the four stages one after another leaves the GPU idle while the host builds the plan.  The
 * pipeline owns its streams (gate, attention, status copies) and depth - 2 (at least one) host threads: rksc_pipeline_submit
 * enqueues the step's gate kernel and the copy of its map on the gate stream and returns; a host
 * thread waits for that copy, builds tables and plan, and enqueues the attention on the attention
 * stream - in submission order, so that attention launches run back to back while the gates of
 * later steps run beside them.
 *
 * rksc_pipeline_create: layout, shapes (B branches, P prefixes, L layers, D hidden size), alpha,
 *   tau and the three page-list CSRs as for rksc_tables_from_gate (host arrays, copied: every step
 *   uses the same lists, only its gate map differs); depth in [2, 8]; mass_capacity = floats the
 *   caller's block_mass buffers hold (0 if it passes none); timing = n > 0 makes every n-th step
 *   (ticket % n == 0) record CUDA events around its segment kernels (that step's attention is then
 *   launched in its two phases); 0: no events.
 * rksc_pipeline_submit: device pointers as for rksc_asks_gate (h_branch, h_root, cand_prefix) and
 *   rksc_branch_decode_attention (q, pools, out, block_mass or NULL).  The buffers must stay valid
 *   and unchanged until the step has been waited for; `after_stream` (may be NULL): work already
 *   enqueued on that stream is waited for by the step (its inputs' producers).  Never blocks; at
 *   most `depth` steps may be in flight: RKSC_ERR_INVALID_ARG if step ticket - depth has not been
 *   waited for yet.  *ticket identifies the step (0, 1, 2, ...).  The calling thread's current
 *   device must be the one the pipeline was created on.
 * rksc_pipeline_wait: blocks the calling thread until step `ticket` has finished; tickets must be
 *   waited for in submission order, each once.  Optional outputs (host, may be NULL):
 *   branch_to_prefix [B], sigma [B], mass_off [B+1], info (the step's plan), segment_ms (device
 *   time of the step's segment kernels if the step was timed, else 0).  Returns the first failing stage's status, or
 *   the attention's device status word, or RKSC_ERR_WORKSPACE when the step's masses did not fit
 *   mass_capacity (the attention was not run).
 * rksc_pipeline_destroy: waits for everything in flight, stops the threads, frees the buffers.
 * Thread safety: one submitting / waiting thread per pipeline.
 * ------------------------------------------------------------------------------------------ */
typedef struct rksc_pipeline rksc_pipeline;
RKSC_API int32_t rksc_pipeline_create(const rksc_layout* layout, int32_t B, int32_t P, int32_t L, int32_t D,
                                      float alpha, float tau,
                                      const int32_t* shared_off, const int32_t* shared_pages, const int32_t* shared_ntok,
                                      const int32_t* priv_off, const int32_t* priv_pages, const int32_t* priv_ntok,
                                      const int32_t* sfx_off, const int32_t* sfx_pages, const int32_t* sfx_ntok,
                                      int32_t depth, int64_t mass_capacity, int32_t timing, rksc_pipeline** out);
RKSC_API int32_t rksc_pipeline_submit(rksc_pipeline* pipe, const float* h_branch, const float* h_root,
                                      const int32_t* cand_prefix, const void* q, const void* k_pool, const void* v_pool,
                                      float* out, float* block_mass, void* after_stream, int64_t* ticket);
RKSC_API int32_t rksc_pipeline_wait(rksc_pipeline* pipe, int64_t ticket, int32_t* branch_to_prefix, float* sigma,
                                    int64_t* mass_off, rksc_plan_info* info, float* segment_ms);
RKSC_API void    rksc_pipeline_destroy(rksc_pipeline* pipe);

#ifdef __cplusplus
}
#endif
#endif /* RKSC_H_ */
