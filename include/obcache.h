/*
 * obcache.h - C ABI of the B200 (sm_100a) OBCache score / select / compact library.
 *
 * The library scores every cached token of a KV cache with the closed-form Optimal-Brain-Damage
 * saliency scores of OBCache, keeps the per-head top-budget, and gathers the kept K/V rows into a
 * compacted cache.  All heavy arguments are DEVICE pointers unless a comment says "host".
 *
 * Conventions that hold for every call
 *   ownership  The caller owns every buffer (inputs, outputs, workspace).  The library allocates
 *              no device memory and frees nothing.  Inputs are never written, except the decode
 *              cache which obc_decode_step updates in place by contract.
 *   async      A call validates its arguments on the host, enqueues its kernels on `stream`
 *              (a cudaStream_t passed as void*; NULL = the legacy default stream) and returns
 *              without synchronising.  Outputs are valid once the stream reaches that point.
 *   errors     The return value is an obc_status; negative = nothing useful was launched.  No
 *              exceptions, aborts or traps cross this boundary.  After OBC_ERR_CUDA,
 *              obc_last_cuda_error() returns the cudaError_t value of the failing runtime call.
 *   layout     head_dim (d) is the innermost, contiguous dimension and must be 128.  Strides are
 *              in ELEMENTS.  Base pointers and strides*elem_size must be multiples of 16 bytes.
 *   notation   B batch, Hq query heads, Hkv KV heads, G = Hq/Hkv, W window queries per head,
 *              R = G*W score rows per KV head, N cached tokens.
 */
#ifndef OBCACHE_H_
#define OBCACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    OBC_OK = 0,
    OBC_ERR_NULL = -1,         /* a required pointer is NULL */
    OBC_ERR_SHAPE = -2,        /* inconsistent or out-of-range sizes */
    OBC_ERR_UNSUPPORTED = -3,  /* head_dim != 128, unknown dtype/variant/pool mode */
    OBC_ERR_ALIGN = -4,        /* base pointer or stride not 16-byte aligned */
    OBC_ERR_WORKSPACE = -5,    /* workspace missing or smaller than obc_*_workspace() says */
    OBC_ERR_CUDA = -6,         /* a CUDA runtime/driver call failed; see obc_last_cuda_error() */
    OBC_ERR_TIMEOUT = -7,      /* a bounded device-side wait gave up */
    OBC_ERR_CAPACITY = -8      /* the problem exceeds the fixed capacity of an allocation-free entry point */
} obc_status;

typedef enum { OBC_F32 = 0, OBC_BF16 = 1 } obc_dtype;

/* score variants (bitmask).  The scores buffer holds one [B,Hkv,max_len] fp32 plane per set bit,
 * in ascending bit order (V, K, VK, ATTN, VATP). */
enum {
    OBC_VAR_V = 1,     /* OBCache-V   : Eq. 4  sum_i A_ip^2 ||v_p||^2                           */
    OBC_VAR_K = 2,     /* OBCache-K   : Eq. 5  sum_i (A_ip Z_ip)^2 ||v_p - o_i||^2              */
    OBC_VAR_VK = 4,    /* OBCache-V&K : Eq. 6  value + key + 2 sum_i A_ip^2 Z_ip (|v_p|^2-v_p.o_i) */
    OBC_VAR_ATTN = 8,  /* attention-only score of Sec. 4.3: sum_i |A_ip|                        */
    OBC_VAR_VATP = 16  /* Eq. 4 with l1 norms (remark after Eq. 4; App. C.2): sum_i |A_ip| ||v_p||_1 */
};

enum { OBC_POOL_NONE = 0, OBC_POOL_AVG = 1, OBC_POOL_MAX = 2 };

/* kernel family used by obc_score */
enum {
    OBC_PATH_AUTO = 0,  /* tensor-core kernels when dtype is bf16 and R is a multiple of 16 and >= 64 */
    OBC_PATH_SIMT = 1,  /* CUDA-core fp32-FMA kernels (any dtype, any R) */
    OBC_PATH_TC = 2     /* tcgen05 kernels; OBC_ERR_UNSUPPORTED if the shape does not qualify */
};

/* Device tensor view.  Logical shape [batch, heads, tokens, head_dim]; head_dim contiguous. */
typedef struct {
    void* ptr;            /* device */
    int32_t dtype;        /* obc_dtype */
    int64_t stride_b;     /* elements between batch items */
    int64_t stride_h;     /* elements between heads */
    int64_t stride_t;     /* elements between tokens (>= head_dim) */
} obc_tensor;

/* ------------------------------------------------------------------------------------------
 * obc_score: saliency scores of every cached token (Sec. 4.2, Eq. 4-6; GQA form App. A.5;
 * perturbation window Eq. 9; the window attention is recomputed as App. C describes).
 *
 * For each batch item b and KV head g, with rows r = (query head h in the group of g, window
 * query i = 0..W-1) and query position N_b - W + i:
 *   Z_rp = scale * q_r . k_p;  A_r. = softmax over the visible p (p <= N_b - W + i if causal);
 *   o_r = sum_p A_rp v_p;  then the selected variants summed over all R rows.  Masked pairs add 0.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    size_t struct_size;       /* sizeof(obc_score_params), for ABI growth */
    int32_t batch, n_q_heads, n_kv_heads, head_dim;
    int32_t window;           /* W >= 1: the last W query positions of every sequence */
    int32_t max_len;          /* token extent of k, v and of each scores plane */
    const int32_t* seq_lens;  /* device [batch], W <= seq_lens[b] <= max_len; NULL = all max_len.
                                 Values are read on the device only. */
    float scale;              /* <= 0 selects 1/sqrt(head_dim) */
    int32_t causal;           /* nonzero: window row i sees keys p <= N_b - W + i */
    uint32_t variants;        /* OBC_VAR_* bitmask, at least one bit */
    int32_t path;             /* OBC_PATH_* */
    const int32_t* mask_lens; /* device [batch] or NULL.  For a cache whose tokens are one shard of a longer
                                 sequence (see obc_window_attention): M_b = the sequence's length minus the
                                 position of the shard's first token.  Window row i then sees the shard's tokens
                                 p <= M_b - W + i, and the preconditions become W <= M_b, 1 <= seq_lens[b].
                                 NULL: M_b = N_b (the cache is the whole sequence). */
} obc_score_params;

/* Bytes of device workspace obc_score needs for these parameters (host computation only). */
obc_status obc_score_workspace(const obc_score_params* p, size_t* bytes /* host out */);

/*
 * q [B,Hq,W,d]; k, v [B,Hkv,max_len,d]; all three share one dtype.  scores: fp32
 * [n_variants,B,Hkv,max_len]; entries at p >= seq_lens[b] are written as 0.  workspace: device,
 * 256-byte aligned, at least obc_score_workspace() bytes; contents are scratch.
 */
obc_status obc_score(const obc_score_params* p, obc_tensor q, obc_tensor k, obc_tensor v,
                     float* scores, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same scores from attention outputs the caller already has, instead of recomputing the window
 * attention: the window rows of O = A V and their log-sum-exp, as the model's own (fused)
 * attention kernel returns them.  Eq. 4-6 are evaluated with A_rp = exp(Z_rp - lse_r) and o_r as
 * given; K and V are then read once instead of twice.  (The paper recomputes the window attention,
 * App. C, because its attention kernel does not expose these; this entry point is the integration
 * the recompute stands in for.)
 *   o    [B,Hq,W,d], device, f32 or bf16 (need not match q), strided like any obc_tensor
 *   lse  device fp32 [B,Hq,W] contiguous: natural log of sum_p exp(scale * q_r . k_p) over the
 *        positions row r sees
 * Everything else as obc_score, including the workspace size (obc_score_workspace).
 */
obc_status obc_score_given(const obc_score_params* p, obc_tensor q, obc_tensor k, obc_tensor v,
                           obc_tensor o, const float* lse,
                           float* scores, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Token-sharded caches (a sequence whose K/V is split by token range over several caches, e.g. one per GPU
 * under context parallelism).  The window attention of Sec. 3 is a softmax over ALL cached tokens, so the
 * shards must agree on it before any of them can score; the scores themselves (Eq. 4-6) are then local to
 * a shard's tokens.  Three steps, with one exchange of R x (d + 1) numbers per head between them:
 *   1. obc_window_attention on every shard (params.mask_lens set): the shard's own softmax over its tokens,
 *      o_out fp32 [B,Hq,W,d] contiguous and lse_out fp32 [B,Hq,W] (natural log of the row's sum of
 *      exp(scaled logit) over the shard's visible tokens; -inf and a zero row of o_out where it sees none);
 *   2. the shards' (o, lse) are gathered (by the caller: NCCL all-gather, peer copies, ...) and
 *      obc_merge_attention combines n_parts of them, stored [n_parts][B,Hq,W,(d)] contiguous, into the
 *      attention over the whole sequence:  lse = log sum_s exp(lse_s),  o = sum_s exp(lse_s - lse) o_s;
 *   3. obc_score_given on every shard with the merged (o, lse) and the same mask_lens.
 * obc_window_attention takes the workspace of obc_score_workspace for the same parameters (variants are
 * ignored but must be valid).  obc_merge_attention needs no workspace; rows = B * Hq * W.
 * ------------------------------------------------------------------------------------------ */
obc_status obc_window_attention(const obc_score_params* p, obc_tensor q, obc_tensor k, obc_tensor v,
                                float* o_out, float* lse_out,
                                void* workspace, size_t workspace_bytes, void* stream);
obc_status obc_merge_attention(int32_t n_parts, int64_t rows, int32_t head_dim,
                               const float* o_parts, const float* lse_parts,
                               float* o_out, float* lse_out, void* stream);
/*
 * After the selection over the gathered scores (Algorithm 2; identical on every rank) a shard keeps the rows it
 * owns: obc_shard_indices writes, for every (b, g), the entries of idx [B,Hkv,idx_stride] (ascending, -1 padded,
 * positions in the whole sequence) that lie in [token_offset, token_offset + n_local), relative to the shard, in
 * ascending order into idx_local [B,Hkv,idx_stride] (-1 padded) and their number into counts [B,Hkv].
 * obc_compact with the shard's k, v and idx_local then fills the first counts[b,g] rows of the shard's compacted
 * cache.  idx and idx_local must not be the same buffer.
 */
obc_status obc_shard_indices(int32_t batch, int32_t n_kv_heads, int32_t idx_stride, const int32_t* idx,
                             int32_t token_offset, int32_t n_local, int32_t* idx_local, int32_t* counts, void* stream);

/*
 * Reads the device status word that obc_score keeps in the first bytes of its workspace.  The
 * tensor-core kernels bound every device-side wait; if one gives up, the kernel raises this word
 * and returns early (its scores are then unspecified).  This call synchronises `stream`, copies
 * the word to the host and returns OBC_OK or OBC_ERR_TIMEOUT.  The word itself (the first 4 bytes
 * of the workspace) holds the source line of the wait that gave up first, for bug reports.
 * (No counterpart in the paper.)
 */
obc_status obc_score_status(const void* workspace, void* stream);

/*
 * Device-side extent of the two tensor-core kernels of obc_score, for measurement.  Every CTA of
 * the window-statistics kernel and of the fused score kernel folds its first and its last reading
 * of the GPU's nanosecond timer into four words of the workspace header; this call synchronises
 * `stream`, returns latest end - earliest start of each kernel in microseconds (host pointers;
 * 0 when nothing was recorded, e.g. on the CUDA-core path) and zeroes the words.  The figures
 * cover the launches since the words were last zero, so zero the workspace header (or call this
 * once) before the obc_score call to be measured, and measure one call at a time.  Unlike an event
 * pair around the launch, the span leaves out launch latency and keeps the overlap of consecutive
 * kernels' prologues intact.  (No counterpart in the paper.)
 */
obc_status obc_score_kernel_spans(void* workspace, void* stream, double* pass1_us, double* pass2_us);

/* ------------------------------------------------------------------------------------------
 * obc_select: pooling + per-head top-budget (Algorithm 2's index selection; SnapKV-style 1-D
 * pooling, App. C.2.1).
 *
 * Per (b, g): keeps tokens [0, n_sink) and [N_b - n_recent, N_b); pools the scores over the
 * candidate range [n_sink, N_b - n_recent) (stride 1, same length, odd kernel; max pads with
 * -inf; avg pads with 0, adds taps in ascending index order in fp32 and divides by the kernel
 * size); keeps the budget_b - n_sink - n_recent candidates with the largest pooled score, equal
 * scores keeping the lowest index; writes all kept indices in ascending order.
 * Scores must be finite; -0.0 ranks equal to +0.0.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    size_t struct_size;
    int32_t batch, n_kv_heads, max_len;
    const int32_t* seq_lens;  /* device [batch] or NULL (all max_len) */
    int32_t budget;           /* kept tokens per head when budgets == NULL */
    const int32_t* budgets;   /* device [batch] per-sequence budgets, or NULL */
    int32_t idx_stride;       /* row length of idx (>= every budget) */
    int32_t n_sink, n_recent;
    int32_t pool_mode;        /* OBC_POOL_* */
    int32_t pool_kernel;      /* odd, >= 1 */
} obc_select_params;

obc_status obc_select_workspace(const obc_select_params* p, size_t* bytes /* host out */);

/*
 * scores: fp32 [B,Hkv,max_len] (one plane).  idx: int32 [B,Hkv,idx_stride]; the first budget_b
 * entries ascending, the rest -1.  A per-sequence budget outside
 * [n_sink + n_recent, N_b] (only detectable on the device) yields a row of -1 for that sequence.
 */
obc_status obc_select(const obc_select_params* p, const float* scores, int32_t* idx,
                      void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * obc_select_adaptive: head-adaptive budgets, the AdaKV allocation that the paper pairs its scores
 * with for its strongest results (Sec. 5.1 "Baselines"; App. C.2.1 "AdaKV": the top-k eviction scores
 * are ranked globally across all heads of the layer; safeguard 0.2).  Per batch item, with
 * n_hh = budget - n_sink - n_recent and H = n_kv_heads: every head first keeps its own
 * floor(safeguard * n_hh) best candidates (pooled scores, ties: lowest index); the remaining
 * H * n_hh - H * floor(..) slots go to the best remaining candidates of all heads ranked together
 * (ties: lowest head, then lowest index).  A head keeps its sinks, its chosen tokens in ascending
 * order and its recent tail.
 *   p          as for obc_select; p->budgets must be NULL (one budget per call); p->idx_stride is
 *              the most one head may keep (a head that would keep more gets a row of -1 and
 *              counts = -1, as does a budget that does not fit its sequence)
 *   idx        device int32 [B,Hkv,idx_stride], rows padded with -1 (obc_compact skips those)
 *   counts     device int32 [B,Hkv]: tokens kept per head; they add up to Hkv * budget per batch item
 *   workspace  device, 256-byte aligned, obc_select_adaptive_workspace() bytes
 * ------------------------------------------------------------------------------------------ */
obc_status obc_select_adaptive_workspace(const obc_select_params* p, float safeguard, size_t* bytes /* host out */);
obc_status obc_select_adaptive(const obc_select_params* p, float safeguard, const float* scores,
                               int32_t* idx, int32_t* counts, void* workspace, size_t workspace_bytes,
                               void* stream);

/*
 * obc_select_noalloc: obc_select for callers that have no device memory to give as workspace and
 * may not allocate any.  (The paper has no counterpart: this is a packaging variant of obc_select.)
 *
 * Typical callers: a plug-in inside an inference engine that owns the whole device heap and hands
 * out no allocator; a serving loop whose memory budget was fixed at start-up, where cudaMalloc
 * would also stall every stream of the device; code that runs after start-up under a policy of
 * "no allocation on the hot path".  Such callers still pass the scores and the index buffer; only
 * the scratch memory is the library's own.
 *
 * The scratch (one 32-bit key per score) lives in a fixed array inside the library image,
 * OBC_SELECT_NOALLOC_MAX_KEYS keys = 4 MiB, which every GPU that loads the library holds until the
 * process exits.  Problems with batch * n_kv_heads * max_len > OBC_SELECT_NOALLOC_MAX_KEYS are
 * rejected with OBC_ERR_CAPACITY and nothing is launched; use obc_select with a caller-owned
 * workspace for those.  The call runs the one-CTA-per-head kernels and gives the same idx, bit
 * for bit, as obc_select; it calls neither cudaMalloc nor cudaFree nor any allocating routine.
 *
 * First call on a device: looks up the device address of the scratch array (a host-side runtime
 * query, done once per device with that device current).  Make that first call outside any stream
 * capture.  All calls on one device share the one array and leave their keys in it: no part of it
 * needs to start at zero (every key that is read was written by the same call), but two calls
 * whose kernels may overlap on the GPU (different streams) race on it; serialise them.
 */
#define OBC_SELECT_NOALLOC_MAX_KEYS (1 << 20)
obc_status obc_select_noalloc(const obc_select_params* p, const float* scores, int32_t* idx, void* stream);

/* ------------------------------------------------------------------------------------------
 * obc_compact: gather of the kept rows (Algorithm 2's gather/concatenate):
 *   k_out[b,g,j,:] = k[b,g,idx[b,g,j],:], same for v, for every j with idx[b,g,j] >= 0.
 * Rows whose index is -1 are left untouched.  If scores_in/scores_out are non-NULL the fp32
 * scores [B,Hkv,max_len] are gathered the same way into [B,Hkv,idx_stride] (they seed the decode
 * accumulator).  k, v, k_out, v_out share one dtype.
 * ------------------------------------------------------------------------------------------ */
obc_status obc_compact(int32_t batch, int32_t n_kv_heads, int32_t head_dim, int32_t idx_stride,
                       int32_t max_len, obc_tensor k, obc_tensor v, const int32_t* idx,
                       obc_tensor k_out, obc_tensor v_out,
                       const float* scores_in, float* scores_out, void* stream);

/* ------------------------------------------------------------------------------------------
 * obc_decode_step: one decode-time rescoring + eviction step (Sec. 3 "Decoding" and "Cache
 * Eviction"; Sec. 4.2: scores accumulated over decode steps; App. C.2.2: sinks and a recent
 * window are protected, one eviction per step once over budget).
 *
 * The cache of each (b, g) is a set of `capacity` slots.  pos[slot] is the token position held
 * by the slot (-1 = free); state[b,g] = {live, next_slot, hi, flag}: live slots, the slot the
 * next token goes to, one past the highest slot ever used, and a word the caller zeroes and the
 * step raises: 1 = the step was not applied (no free slot), 2 = a device-side wait for a copy of
 * cache rows gave up after its time limit (the step's results for that (b, g) are undefined).
 * One call:
 *   1. writes (k_t, v_t) into next_slot with pos = step_pos and accumulator 0;
 *   2. with the newest query of each of the G heads, recomputes attention over the live slots
 *      and the chosen variant's score of every live slot (W = 1);
 *   3. s_acc[slot] += score;
 *   4. if live > budget: frees the live slot with the smallest s_acc among tokens with
 *      n_sink <= pos <= step_pos - n_recent (equal values: the highest pos), which becomes
 *      next_slot; otherwise next_slot = hi.
 *
 * Accumulation window (App. B, "Choice of Perturbation Window in Decoding": scores accumulated
 * only within a recent window instead of over the whole history).  With acc_window = w > 0 step 3
 * becomes  s_acc[slot] = sum of the slot's scores of the last w steps (this one included, fewer
 * while the token is younger than w steps).  The per-step scores are kept in the ring s_hist, fp32
 * [B,Hkv,w,capacity], which the caller zero-fills before the first step and then leaves alone; the
 * step with position step_pos uses ring row step_pos mod w, so consecutive steps must advance
 * step_pos by one.  The sum is formed afresh every step, rows 0..w-1 in order; what s_acc held
 * before is not used (a token's column of the ring is cleared when the token enters the cache).
 * acc_window = 0 (s_hist ignored) accumulates over all steps.  acc_window > 4096: OBC_ERR_SHAPE.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    size_t struct_size;
    int32_t batch, n_q_heads, n_kv_heads, head_dim;
    int32_t capacity;         /* slots per (b, g); must exceed budget */
    int32_t budget, n_sink, n_recent;
    uint32_t variant;         /* exactly one OBC_VAR_* bit */
    float scale;              /* <= 0 selects 1/sqrt(head_dim) */
    int32_t acc_window;       /* 0: accumulate over all steps; w > 0: over the last w steps */
    float* s_hist;            /* device, [B,Hkv,acc_window,capacity]; NULL when acc_window == 0 */
} obc_decode_params;

obc_status obc_decode_workspace(const obc_decode_params* p, size_t* bytes /* host out */);

/*
 * q_t [B,Hq,1,d]; k_t, v_t [B,Hkv,1,d]; k_cache, v_cache [B,Hkv,capacity,d] updated in place;
 * s_acc fp32 [B,Hkv,capacity], pos int32 [B,Hkv,capacity], state int32 [B,Hkv,4]: all updated in
 * place.  step_pos: position of the new token.  All tensors bf16.
 */
obc_status obc_decode_step(const obc_decode_params* p, obc_tensor q_t, obc_tensor k_t, obc_tensor v_t,
                           obc_tensor k_cache, obc_tensor v_cache, float* s_acc, int32_t* pos,
                           int32_t* state, int32_t step_pos,
                           void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Optional per-kernel timing, used by the benchmark (no counterpart in the paper).  Between
 * obc_profile_begin() and obc_profile_end() every kernel the library enqueues from any thread
 * is bracketed by a pair of CUDA events on its stream.  obc_profile_end() synchronises those
 * events, sums the elapsed time per kernel name into out[0..*n_out) (host array of max_out
 * entries) and stops recording.  Off by default; costs two event records per kernel when on.
 * ------------------------------------------------------------------------------------------ */
typedef struct { char name[48]; int32_t launches; float ms_total; } obc_kernel_time;
obc_status obc_profile_begin(void);
obc_status obc_profile_end(obc_kernel_time* out /* host */, int32_t max_out, int32_t* n_out /* host */);

/* Host-only helpers. */
const char* obc_status_string(obc_status s);
int obc_last_cuda_error(void);      /* cudaError_t of the last failing CUDA call on this thread */
int obc_version(void);              /* major*10000 + minor*100 + patch */

#ifdef __cplusplus
}
#endif
#endif /* OBCACHE_H_ */
