/*
 * libcott -- cosine attention (Cottention, arXiv 2409.18747) for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Plain pointers and sizes only.  Unless a parameter says "host", every
 * tensor pointer is a DEVICE pointer owned by the caller; the library never
 * allocates, frees or keeps caller memory.  Scratch memory comes from the
 * caller-supplied workspace (size it with cott_workspace_bytes).
 *
 * Symbols: B batch, H heads, N sequence length, d per-head dimension (one d for
 * keys and values).  q,k,v,o,d_o,dq,dk,dv are contiguous row-major [B,H,N,d] in
 * the I/O dtype `dt` (the *_strided entry points take other strides, the *_varlen
 * ones sequences of different lengths packed into [total_tokens,H,d]); decode
 * tensors are [B,H,d]; `m`, `seq_len`, `state`, `dm` are always fp32.
 *
 * What is computed (paper equations):
 *   x^      = x / max(||x||_2, 1e-12)            row normalisation of Q and K (Eq. 2, Eq. 3)
 *   c[b,h]  = s_b ^ (-sigmoid(m_h))              stabilisation factor (Eq. 4); s_b >= 1
 *   bidirectional: O = c * Q^ (K^^T V)           (Eq. 3 re-associated as in Eq. 5)
 *   causal:        o_t = c * sum_{j<=t} (q^_t . k^_j) v_j     (Eq. 6, diagonal kept)
 *                  computed through the running state of Eq. 7 / Eq. 8,
 *                  S_t = S_{t-1} + k^_t (c v_t)^T ,  o_t = S_t^T q^_t
 *   state layout: [B,H,d_key,d_value] fp32, S = sum_j k^_j (c v_j)^T
 *                  (the paper's hidden state H_t transposed, scale included).
 *
 * All calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 * the legacy default stream).  The returned status covers argument validation and
 * launch errors only.  cott_fwd*, cott_bwd* and cott_decode_step* with caller-owned outputs
 * and workspaces put only kernel launches and memsets on the stream (and, where gradient streams
 * run side by side, event-ordered work on the library's streams): once each kernel has been
 * launched at least once on the device, such calls can be captured in a CUDA graph and
 * replayed.  Calls are thread-safe as long as concurrent calls use
 * different workspaces.  Outputs must not share bytes with inputs or with each other:
 * equal pointers, dense tensors whose byte ranges meet, and equally strided tensors
 * (slices of one buffer) whose rows meet are refused with COTT_ERR_INVALID_ARG.
 *
 * State the library keeps (everything else lives in the caller's buffers):
 *   - per host thread and device, three CUDA streams and five events used by cott_bwd
 *     (gradient streams side by side) and cott_fwd_bwd_host (copies in both directions),
 *     created on first use; cott_shutdown() destroys the calling thread's;
 *   - the options of cott_set_option, a launch counter and, while cott_profile_enable is
 *     on, up to 512 timing events (process-wide);
 *   - per (kernel, device), the fact that the shared-memory opt-in has been made;
 *   - the 8 MiB scratch array of cott_fwd_noalloc.
 */
#ifndef COTT_H_
#define COTT_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    COTT_OK = 0,
    COTT_ERR_INVALID_ARG = -1, /* NULL required pointer, non-positive size, s < 1, aliasing      */
    COTT_ERR_UNSUPPORTED = -2, /* head size, dtype or alignment the kernels do not cover         */
    COTT_ERR_WORKSPACE = -3,   /* workspace NULL or smaller than cott_workspace_bytes()          */
    COTT_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed (see cott_last_cuda_error) */
    COTT_ERR_TIMEOUT = -5      /* a bounded device-side wait expired (reported asynchronously)   */
} cott_status;

typedef enum { COTT_F32 = 0, COTT_BF16 = 1 } cott_dtype;

typedef enum { COTT_OP_FWD = 0, COTT_OP_BWD = 1, COTT_OP_DECODE = 2 } cott_op;

/* Parameters of the stabilisation factor of Eq. 4. */
typedef struct {
    const float* m;       /* device [H]: the learned per-head scalar; required                  */
    const float* seq_len; /* device [B]: scaling base s_b per batch item, or NULL                */
    float seq_len_scalar; /* used when seq_len == NULL: fwd/bwd take s_b = N if this is <= 0,    */
                          /* otherwise this value; decode requires it (>= 1) when seq_len==NULL  */
} cott_scale_params;

/* Library version (major*10000 + minor*100 + patch). */
int cott_version(void);

/* Human-readable name of a status code (static string). */
const char* cott_status_string(cott_status st);

/* Text of the last CUDA error seen by this thread inside the library (static storage). */
const char* cott_last_cuda_error(void);

/* Number of kernels this process has launched through the library so far (all threads). */
unsigned long long cott_launch_count(void);

/*
 * Process-wide switches for tests and measurements (none is needed in use).  Each starts from
 * an environment variable that is read once, on first use, and can be changed at any time
 * with cott_set_option (takes effect for calls issued afterwards; not synchronised with calls
 * in flight on other host threads).  Names (environment variable, default):
 *   "force_group"        (COTT_FORCE_GROUP, 0)        tokens per sequence group; 0 = the plan's choice
 *   "force_path"         (COTT_FORCE_PATH, 1)         0 = bf16 d = 64 / 128 through the fp32-accumulating SIMT kernels
 *   "pair"               (COTT_PAIR, 1)               0 = gradient streams one after the other where they would run side by side
 *   "fused_bwd"          (COTT_FUSED_BWD, 1)          0 = d = 64 backward (causal and bidirectional) as three role-swapped walks instead of one fused walk
 *   "fused_bidir"        (COTT_FUSED_BIDIR, 1)        0 = bidirectional d = 64 forward as a state pass and a read-out instead of one launch
 *   "bidir_bwd"          (COTT_BIDIR_BWD, 1)          0 = bidirectional d = 64 backward with one group per (b, h) as a state pass and a walk instead of one launch
 *   "short_fwd"          (COTT_SHORT_FWD, 1)          0 = sequences of at most 128 tokens through the generic walk instead of the stateless kernel
 *   "block_fwd"          (COTT_BLOCK_FWD, 1)          0 = blocks of at most 64 tokens on a state through the generic walk instead of the block kernel
 *   "host_slices"        (COTT_HOST_SLICES, 8)        most slices cott_fwd_bwd_host cuts a batch into (1 .. 16)
 *   "wait_limit_ms"      (COTT_WAIT_LIMIT_MS, 2000)   bound of every device-side wait
 *   "wait_limit_kcycles" (COTT_WAIT_LIMIT_KCYCLES, -1) the same bound in units of 1024 SM cycles; negative = use the millisecond
 *                        value; 0 = every wait that is not met within a few polls gives up (the timeout test)
 * cott_set_option returns COTT_ERR_INVALID_ARG for an unknown name; cott_get_option returns -1.
 * No paper passage: library plumbing.
 */
cott_status cott_set_option(const char* name, long long value);
long long cott_get_option(const char* name);

/*
 * Per-launch timing of the tensor-core walk kernels, for benchmarks.  cott_profile_enable(n)
 * with n > 0 starts recording a pair of library-owned CUDA events around each of the next n
 * (at most 256) walk-kernel launches; n <= 0 stops.  cott_profile_read waits for the recorded
 * launches and writes their durations in milliseconds to ms[] and their kind to kinds[]
 * (0 = partial-state pass, 1 = causal walk, 2 = read-out, 3 = fused backward walk (causal or
 * bidirectional), 4 = one-launch bidirectional forward, 5 = short-sequence forward, 6 = token-block
 * forward on a state, 7 = one-launch bidirectional backward; 17 = a causal walk that ran side by
 * side with a sibling walk of the same size on another stream of the library, in which case
 * its ms is half of the span the pair occupied, first start to last end); both are host
 * arrays of `cap` entries.  Returns the number of entries written, or -1 on a CUDA error.  Not thread-safe
 * against concurrent library calls; leave it off outside measurements.
 */
cott_status cott_profile_enable(int max_launches);
int cott_profile_read(float* ms, int* kinds, int cap);

/*
 * Bytes of device scratch the given call needs (0 is possible).  `op` is a cott_op.
 * The workspace must be 256-byte aligned.  Returns (size_t)-1 for unsupported arguments.
 */
size_t cott_workspace_bytes(int op, cott_dtype dt, int B, int H, int N, int d, int causal);

/*
 * Reports how a call would be executed (for tests and tuning):
 *   *path   0 = fp32 SIMT kernels, 1 = tcgen05 tensor-core kernels
 *   *group  tokens per sequence group (the unit of sequence-level parallelism; the per-group
 *           partial states are combined by an exclusive prefix scan, which is valid because
 *           the cumulative sum of Eq. 7 is associative)
 *   *chunk  tokens per chunk inside a group (tile of the masked Q^K^^T product, Eq. 6)
 * Any output pointer may be NULL.  Host pointers.
 */
cott_status cott_query_plan(int op, cott_dtype dt, int B, int H, int N, int d, int causal,
                            int* path, int* group, int* chunk);

/*
 * Forward pass: Eq. 3/4/5 (causal == 0) or Eq. 6/7/8 (causal != 0).
 *   q,k,v   in : [B,H,N,d] dt
 *   o       out: [B,H,N,d] dt
 *   state_out  : NULL, or fp32 [B,H,d,d] receiving S_N = sum_j k^_j (c v_j)^T over all N tokens
 *                (the state a following cott_decode_step continues from, Eq. 8)
 * Rows of Q or K whose norm is <= 1e-12 normalise to (near) zero: a zero K row contributes
 * nothing, a zero Q row yields a zero output row.  N need not be a multiple of any tile.
 */
cott_status cott_fwd(const void* q, const void* k, const void* v, void* o, float* state_out,
                     int B, int H, int N, int d, int causal, cott_dtype dt,
                     const cott_scale_params* sp, void* workspace, size_t workspace_bytes,
                     void* stream);

/*
 * Element strides of a tensor of logical shape [B,H,N,d] whose rows (the d elements of one
 * token of one head) are contiguous: distance between consecutive batch items, heads and
 * tokens.  Dense [B,H,N,d] is {H*N*d, N*d, d}; [B,N,H,d], the layout a projection GEMM leaves,
 * is {N*H*d, d, H*d}; q inside a fused [B,N,3,H,d] projection output is {N*3*H*d, d, 3*H*d}
 * (k and v start H*d and 2*H*d elements later).  Every stride must be >= d and a multiple of
 * 16 bytes; the tensor's first element must be 16-byte aligned.
 */
typedef struct cott_strides {
    long long batch;
    long long head;
    long long token;
} cott_strides;

/*
 * cott_fwd on tensors that are not dense [B,H,N,d] (no transpose pass before the attention):
 *   qkv_strides : strides shared by q, k and v (NULL: dense)
 *   o_strides   : strides of o (NULL: dense)
 * Everything else as for cott_fwd.  On the tensor-core path (bf16) the strides must
 * also be expressible as a 4-D tiled tensor map (each stride a multiple of the next smaller
 * one, as in the three layouts above); COTT_ERR_UNSUPPORTED or COTT_ERR_CUDA otherwise.
 */
cott_status cott_fwd_strided(const void* q, const void* k, const void* v, void* o, float* state_out,
                             int B, int H, int N, int d, int causal, cott_dtype dt,
                             const cott_strides* qkv_strides, const cott_strides* o_strides,
                             const cott_scale_params* sp, void* workspace, size_t workspace_bytes,
                             void* stream);

/*
 * Causal forward over one SEGMENT of a longer sequence (chunked prefill; blocks of several
 * tokens between decode steps): the running state of Eq. 8 carried across calls.
 *   state_in  : NULL (the sequence starts here) or fp32 [B,H,d,d], the state left by the previous
 *               segment, by cott_fwd (state_out) or by cott_decode_step; it contains c
 *   state_out : NULL or fp32 [B,H,d,d] receiving state_in + sum_j k^_j (c v_j)^T over this segment;
 *               must not be the same buffer as state_in
 *   o         : rows of this segment, o_t = S_t^T q^_t with S_t including state_in
 * The scaling base of Eq. 4 has to be the caller's and the same for every segment of one
 * sequence: sp->seq_len ([B]) or sp->seq_len_scalar (>= 1); with that, the segments together
 * give the rows of one cott_fwd over the whole sequence.  Other arguments as for cott_fwd
 * (workspace: cott_workspace_bytes(COTT_OP_FWD, ..., causal = 1)).
 */
cott_status cott_fwd_stateful(const void* q, const void* k, const void* v, void* o,
                              const float* state_in, float* state_out, int B, int H, int N, int d,
                              cott_dtype dt, const cott_scale_params* sp, void* workspace,
                              size_t workspace_bytes, void* stream);

/* cott_fwd_stateful on tensors that are not dense [B,H,N,d]; strides as for cott_fwd_strided. */
cott_status cott_fwd_stateful_strided(const void* q, const void* k, const void* v, void* o,
                                      const float* state_in, float* state_out, int B, int H, int N,
                                      int d, cott_dtype dt, const cott_strides* qkv_strides,
                                      const cott_strides* o_strides, const cott_scale_params* sp,
                                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of cott_fwd for L = sum(d_o * O): the gradient formulas printed after Eq. 7
 * (dQ^ = (dO V'^T . M) K^, dK^ = (dO V'^T . M)^T Q^, dV' = (Q^ K^^T . M)^T dO; M all-ones when
 * causal == 0), evaluated through a forward running state and a state that accumulates
 * backward in time, followed by the chain rule through the row normalisation (Eq. 2/3) and
 * the stabilisation factor (Eq. 4):
 *   dq,dk,dv out: [B,H,N,d] dt, gradients w.r.t. the RAW q,k,v
 *   dm       out: fp32 [H], gradient w.r.t. m summed over batch and positions; overwritten
 * On a row with norm <= 1e-12 the gradient is that of the clamped formula, d x^ / 1e-12.
 * There is no gradient for the scaling base s.
 * No output tensor may overlap an input tensor.  The call is ordered on `stream` as a whole:
 * work issued to `stream` before it has finished when it starts, and work issued after it
 * sees all its results; inside, the library may run independent gradient streams on two
 * streams of its own (created once per device on first use), forked from and joined back
 * into `stream` with events.
 */
cott_status cott_bwd(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                     void* dk, void* dv, float* dm, int B, int H, int N, int d, int causal,
                     cott_dtype dt, const cott_scale_params* sp, void* workspace,
                     size_t workspace_bytes, void* stream);

/*
 * cott_bwd on tensors that are not dense [B,H,N,d]:
 *   qkv_strides  : strides shared by q, k and v (NULL: dense)
 *   do_strides   : strides of d_o (NULL: dense)
 *   dqkv_strides : strides shared by dq, dk and dv (NULL: dense), e.g. the three slices of a
 *                  fused gradient buffer
 * Everything else, and the conditions on the strides, as for cott_bwd and cott_fwd_strided.
 */
cott_status cott_bwd_strided(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                             void* dk, void* dv, float* dm, int B, int H, int N, int d, int causal,
                             cott_dtype dt, const cott_strides* qkv_strides,
                             const cott_strides* do_strides, const cott_strides* dqkv_strides,
                             const cott_scale_params* sp, void* workspace, size_t workspace_bytes,
                             void* stream);

/*
 * Packed variable-length batches: the rows of B sequences back to back in tensors of shape
 * [total_tokens, H, d] (dense), sequence b occupying rows cu_seqlens[b] .. cu_seqlens[b+1]-1
 * (cu_seqlens: DEVICE array of B + 1 ints, cu_seqlens[0] = 0, cu_seqlens[B] = total_tokens,
 * non-decreasing).  Each sequence is attended on its own, Eq. 5 (causal == 0) or Eq. 6-8
 * (causal != 0), with its own scaling base for Eq. 4: sp->seq_len[b], else sp->seq_len_scalar,
 * else its length.  No padding rows are read as keys or written as outputs.
 *   max_seqlen : an upper bound of the longest sequence (sizes the workspace and the plan)
 *   workspace  : cott_workspace_bytes_varlen(COTT_OP_FWD or COTT_OP_BWD, dt, B, H, total_tokens, max_seqlen, d, causal),
 *                or at least cott_workspace_bytes(op, dt, B, H, max_seqlen, d, causal)
 * bf16 with d a multiple of 8 up to 128, or fp32 with d in {32, 64, 128} (COTT_ERR_UNSUPPORTED otherwise).  On the tensor-core
 * path a sequence is cut into the groups the dense plan for N = max_seqlen uses (group g = its rows g * group .. + group - 1,
 * as far as they exist), so a batch of few long sequences still fills the GPU; the fp32 kernels walk one (sequence, head) per CTA.  A NaN or Inf in the first
 * rows of one sequence can reach the last rows of the sequence stored before it (the tile
 * that holds both is multiplied by zeros, not skipped).  Other arguments, ordering and
 * aliasing rules as for cott_fwd / cott_bwd.
 */
/*
 * Workspace of cott_fwd_varlen / cott_bwd_varlen with room for the finer groups the library uses
 * when the sum of the lengths is well below B * max_seqlen (a few long sequences among short ones:
 * the group size then follows total_tokens, so that all groups of the batch still make about one
 * wave of CTAs).  A workspace of cott_workspace_bytes(op, dt, B, H, max_seqlen, d, causal) bytes
 * works as well: where that is less than the finer groups need, the calls use the groups of the
 * dense plan for max_seqlen tokens.
 */
size_t cott_workspace_bytes_varlen(int op, cott_dtype dt, int B, int H, int total_tokens, int max_seqlen,
                                   int d, int causal);

cott_status cott_fwd_varlen(const void* q, const void* k, const void* v, void* o,
                            const int* cu_seqlens, int B, int H, int total_tokens, int max_seqlen,
                            int d, int causal, cott_dtype dt, const cott_scale_params* sp,
                            void* workspace, size_t workspace_bytes, void* stream);
cott_status cott_bwd_varlen(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                            void* dk, void* dv, float* dm, const int* cu_seqlens, int B, int H,
                            int total_tokens, int max_seqlen, int d, int causal, cott_dtype dt,
                            const cott_scale_params* sp, void* workspace, size_t workspace_bytes,
                            void* stream);

/*
 * One recurrent decode step, Eq. 8:  S <- S + k^ (c v)^T ;  o = S^T q^  (update, then read).
 *   q,k,v  in    : [B,H,d] dt
 *   state  in/out: fp32 [B,H,d,d], updated in place (constant-size inference memory)
 *   o      out   : [B,H,d] dt
 * The scaling base comes from sp->seq_len ([B]) or sp->seq_len_scalar (>= 1); keeping the
 * prefill's value makes prefill + decode equal to one longer causal forward.
 * Needs no workspace.
 */
cott_status cott_decode_step(const void* q, const void* k, const void* v, float* state, void* o,
                             int B, int H, int d, cott_dtype dt, const cott_scale_params* sp,
                             void* stream);

/*
 * cott_bwd_strided for a training step: `fwd_workspace` is the workspace the cott_fwd /
 * cott_fwd_strided call on the SAME q, k, v, scale parameters and options used (with
 * state_out == NULL), not overwritten since.  Where that call left the per-group partial states
 * K^^T V there (the causal tensor-core path at d <= 64 with two to eight groups), the backward
 * reads them instead of streaming k and v once more for its own; everywhere else the pointer is
 * ignored and the call is cott_bwd_strided.  The library cannot check that the workspace belongs
 * to these tensors: passing another one gives wrong gradients, not an error.  NULL is allowed.
 * It must not be the backward's own workspace.
 */
cott_status cott_bwd_after_fwd(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                               void* dk, void* dv, float* dm, int B, int H, int N, int d, int causal,
                               cott_dtype dt, const cott_strides* qkv_strides,
                               const cott_strides* do_strides, const cott_strides* dqkv_strides,
                               const cott_scale_params* sp, const void* fwd_workspace, void* workspace,
                               size_t workspace_bytes, void* stream);

/*
 * Backward of cott_fwd_stateful: the gradients of one SEGMENT of a longer causal sequence (training
 * through chunked prefill).  For L = sum(dO (.) O) + sum(d_state_out (.) state_out) of the segment,
 * the running sums of the backward described after Eq. 7 start from what lies outside it: the
 * forward sum from state_in, the reverse sum from d_state_out,
 *     dq^_t = S_t dO_t ,                      S_t = state_in + sum_{j<=t} k^_j (c v_j)^T
 *     dk^_j = R_j (c v_j) ,  dv'_j = R_j^T k^_j ,  R_j = d_state_out + sum_{t>=j} q^_t dO_t^T
 *     d_state_in = R_1
 * followed by the chain rule through Eq. 2-4 as in cott_bwd.
 *   state_in    : NULL (zero) or fp32 [B,H,d_k,d_v], what cott_fwd_stateful was given
 *   d_state_out : NULL (zero) or fp32 [B,H,d_k,d_v], the gradient of the state the segment handed on
 *                 (the d_state_in of the next segment's backward; NULL for the last one)
 *   d_state_in  : NULL or fp32 [B,H,d_k,d_v], receives the gradient of state_in; not one of the
 *                 other two buffers
 *   dm          : this segment's part of the gradient of m (state_in counts as an input of its
 *                 own: its dependence on m belongs to the segment that produced it, which sees it
 *                 through d_state_in); the parts of all segments add up to the dm of the sequence
 * Run over the segments last to first, with the caller's scaling base (sp->seq_len or
 * sp->seq_len_scalar >= 1, the same for every segment), the calls give the gradients of one
 * cott_bwd over the whole sequence.  bf16 with d_k, d_v multiples of 8 up
 * to 64: the one-walk backward of the tensor-core path.  bf16 with larger sizes (multiples of 8 up
 * to 128): the three tensor-core walks.  fp32 with d_k = d_v in {32, 64, 128}: three running-sum
 * walks of the fp32-accumulating kernels.  COTT_ERR_UNSUPPORTED otherwise.
 * workspace: cott_workspace_bytes_dkdv(COTT_OP_BWD, dt, B, H, N, d_k, d_v, 1).
 */
cott_status cott_bwd_stateful(const void* q, const void* k, const void* v, const void* d_o,
                              const float* state_in, const float* d_state_out, void* dq, void* dk, void* dv,
                              float* d_state_in, float* dm, int B, int H, int N, int d_k, int d_v, cott_dtype dt,
                              const cott_scale_params* sp, void* workspace, size_t workspace_bytes, void* stream);

/* cott_bwd_stateful on tensors that are not dense [B,H,N,d]; strides as for cott_bwd_dkdv (the states stay dense). */
cott_status cott_bwd_stateful_strided(const void* q, const void* k, const void* v, const void* d_o,
                                      const float* state_in, const float* d_state_out, void* dq, void* dk, void* dv,
                                      float* d_state_in, float* dm, int B, int H, int N, int d_k, int d_v, cott_dtype dt,
                                      const cott_strides* qk_strides, const cott_strides* v_strides,
                                      const cott_strides* do_strides, const cott_strides* dqk_strides,
                                      const cott_strides* dv_strides, const cott_scale_params* sp, void* workspace,
                                      size_t workspace_bytes, void* stream);

/*
 * Head sizes.  The paper's section 2.1 gives keys / queries and values sizes of their own
 * (d_H_key, d_H_value); every call above takes one `d` for both.  The *_dkdv calls below take
 * the two separately:
 *   q, k (and dq, dk)     : [B,H,N,d_k]        v, o, dO (and dv) : [B,H,N,d_v]
 *   states                : fp32 [B,H,d_k,d_v]  (S = sum_j k^_j (c v_j)^T)
 * What is supported (either form of call):
 *   bf16: any d_k, d_v that are multiples of 8 up to 128 (rows of 16 bytes) -- tensor-core
 *         kernels of size 64 (both <= 64) or 128, the tiles zero-filled beyond the real
 *         columns, which changes no norm, score or product; a caller's state passes through a
 *         padded copy in the workspace (cott_workspace_bytes_dkdv accounts for it);
 *   fp32: d_k = d_v in {32, 64, 128};
 *   decode step: additionally any d_k, d_v up to 1024 that are multiples of 16 bytes.
 * Packed (varlen) batches take one d (bf16, any multiple of 8 up to 128); cott_fwd_noalloc and
 * cott_fwd_bwd_host take one d as well.
 * Strides: q and k share `qk_strides`, v has `v_strides`, o / dO `o_strides` / `do_strides`,
 * dq and dk share `dqk_strides`, dv has `dv_strides` (NULL: dense for that tensor's own width;
 * with d_k == d_v a NULL v_strides / dv_strides means "as q and k" / "as dq and dk").
 * cott_fwd_dkdv is cott_fwd, cott_fwd_strided and cott_fwd_stateful in one: state_in non-NULL
 * makes it the stateful call (causal only, scaling base required, see cott_fwd_stateful).
 * cott_query_plan_dkdv also reports the size the kernels run at (*kernel_d; NULL allowed).
 */
size_t cott_workspace_bytes_dkdv(int op, cott_dtype dt, int B, int H, int N, int d_k, int d_v, int causal);
cott_status cott_query_plan_dkdv(int op, cott_dtype dt, int B, int H, int N, int d_k, int d_v, int causal,
                                 int* path, int* group, int* chunk, int* kernel_d);
cott_status cott_fwd_dkdv(const void* q, const void* k, const void* v, void* o, const float* state_in,
                          float* state_out, int B, int H, int N, int d_k, int d_v, int causal, cott_dtype dt,
                          const cott_strides* qk_strides, const cott_strides* v_strides,
                          const cott_strides* o_strides, const cott_scale_params* sp, void* workspace,
                          size_t workspace_bytes, void* stream);
cott_status cott_bwd_dkdv(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk,
                          void* dv, float* dm, int B, int H, int N, int d_k, int d_v, int causal, cott_dtype dt,
                          const cott_strides* qk_strides, const cott_strides* v_strides,
                          const cott_strides* do_strides, const cott_strides* dqk_strides,
                          const cott_strides* dv_strides, const cott_scale_params* sp, void* workspace,
                          size_t workspace_bytes, void* stream);
cott_status cott_decode_step_dkdv(const void* q, const void* k, const void* v, float* state, void* o,
                                  int B, int H, int d_k, int d_v, cott_dtype dt, const cott_scale_params* sp,
                                  void* stream);

/*
 * Training step with HOST buffers (end-to-end path): copies q,k,v,d_o from host memory to the
 * device arena, runs cott_fwd then cott_bwd, and copies o,dq,dk,dv,dm back.  The batch goes
 * through in at most 8 slices (option "host_slices") that are contiguous in [B,H,N,d] -- several whole batch items
 * each, or, when the batch is small, a batch item's heads in equal groups
 * (cott_host_step_slicing tells which) --, each a cott_fwd and a cott_bwd call of its own on
 * `stream` with the scaling base s_b = N unless seq_len_host is given: while one slice is computed, the inputs of the next come in and the results
 * of the one before go back on two streams of the library (the link is full duplex), joined
 * into `stream` before the call returns its last copy.  Every row of o, dq, dk, dv equals what
 * the device calls give for its slice; dm (a sum over the batch) is the sum of the slices' dm
 * in slice order.
 *   *_host  : host pointers ([B,H,N,d] dt; dm_host fp32 [H]); pinned memory makes the copies
 *             asynchronous.  m_host fp32 [H], seq_len_host fp32 [B] or NULL (s_b = N).
 *   arena   : device scratch of at least cott_host_step_arena_bytes() bytes, 256-B aligned.
 * The caller synchronises `stream` before reading the host outputs.
 */
size_t cott_host_step_arena_bytes(cott_dtype dt, int B, int H, int N, int d, int causal);
cott_status cott_host_step_slicing(int B, int H, int* items_per_slice, int* heads_per_slice, int* n_slices);
cott_status cott_fwd_bwd_host(const void* q_host, const void* k_host, const void* v_host,
                              const void* d_o_host, void* o_host, void* dq_host, void* dk_host,
                              void* dv_host, float* dm_host, const float* m_host,
                              const float* seq_len_host, int B, int H, int N, int d, int causal,
                              cott_dtype dt, void* arena, size_t arena_bytes, void* stream);

/*
 * cott_fwd without a caller workspace (the paper has no counterpart: this exists for the way
 * the library is embedded, not for the method).  It serves callers that cannot obtain device
 * memory at call time, e.g. a server whose own pool already holds all of HBM, or a loop that
 * cannot afford the device-wide synchronisation of cudaMalloc / cudaFree.  The scratch is a
 * fixed 8 MiB array (cott_fwd_noalloc_max_bytes()) compiled into the library, so every GPU
 * that loads the library gives up that much memory until the process exits.  The call itself
 * allocates and frees nothing.
 *   - Arguments as for cott_fwd (no state export); inputs and outputs are still the caller's.
 *   - Returns COTT_ERR_WORKSPACE when cott_workspace_bytes(COTT_OP_FWD, ...) for this problem
 *     exceeds the 8 MiB; use cott_fwd with your own workspace then.
 *   - The first call on each device looks up the array's device address (a host-side set-up
 *     step); make that first call before starting any stream capture.
 *   - All calls on a device share the one array: two calls whose kernels may overlap on the
 *     GPU (different streams, no ordering) race on it.  Calls ordered on one stream are safe;
 *     nothing needs to be cleared between them.
 */
size_t cott_fwd_noalloc_max_bytes(void);
cott_status cott_fwd_noalloc(const void* q, const void* k, const void* v, void* o, int B, int H,
                             int N, int d, int causal, cott_dtype dt, const cott_scale_params* sp,
                             void* stream);

/*
 * The same for cott_fwd_noalloc, whose scratch (and status word) is inside the library.
 * No paper passage: library plumbing.
 */
cott_status cott_fwd_noalloc_status(void* stream);

/*
 * Destroys the CUDA streams and events the library created for the calling host thread (on
 * every device it used) and the profiling events; they are created again on demand.  Call it
 * when no library call of this thread is in flight.  No paper passage: library plumbing.
 */
cott_status cott_shutdown(void);

/*
 * Synchronises `stream`, then reads the status word the last call using `workspace` left
 * there: COTT_OK, or COTT_ERR_TIMEOUT if a bounded device-side wait gave up, or COTT_ERR_CUDA
 * if the stream reports an error.  After a timeout the next two 32-bit words of the workspace
 * say where the first wait gave up: word 1 = bit 31 set, warp index in bits 16-20, byte offset
 * of the barrier in the kernel's barrier block in bits 4-13, phase parity in bit 0; word 2 =
 * CTA index in bits 0-23, kernel mode in bits 24-27, output stream in bits 28-31.
 */
cott_status cott_last_async_status(const void* workspace, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* COTT_H_ */
