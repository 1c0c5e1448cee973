// Internal declarations shared by the translation units of libcott.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "cott.h"

namespace cott {

constexpr float kEps = 1e-12f;        // denominator floor of the row normalisation (Eq. 2/3)
constexpr int kWsHeaderBytes = 256;   // workspace header: word 0 = asynchronous status

// Row treatment applied to a tile row when it is staged in shared memory.
enum RowMode : int {
    ROW_RAW = 0,    // use as is (dO)
    ROW_NORM = 1,   // x / max(||x||, eps)     (Q and K, Eq. 3)
    ROW_SCALE = 2   // c * x                   (V, Eq. 4)
};

// What happens to the rows a walk produces before they are stored.
enum Epilogue : int {
    EPI_PLAIN = 0,  // store
    EPI_PROJ = 1,   // chain rule through the row normalisation of `proj` (raw q or k)
    EPI_DV = 2      // multiply by c, and accumulate <row, proj row> for dm (proj = raw v)
};

// Where the rows of a [B,H,N,d] tensor sit in memory: element strides of the batch, head and
// token index; the d elements of a row are contiguous.  All zero means dense [B,H,N,d].
struct RowLayout {
    long long sb, sh, sn;
};
inline RowLayout resolve_layout(const RowLayout& l, int H, int N, int d) {
    if (l.sb == 0 && l.sh == 0 && l.sn == 0) return RowLayout{(long long)H * N * d, (long long)N * d, (long long)d};
    return l;
}

// How the scan kernel combines the per-group partial states.
enum ScanMode : int { SCAN_PREFIX = 0, SCAN_SUFFIX = 1, SCAN_TOTAL = 2 };

// One pass of the generic running-sum walk (Eq. 7 / Eq. 8 with operand roles):
//   state[a][b] += A_t[a] * Bv_t[b]   (if update)      out_t[b] = sum_a X_t[a] * state[a][b]
// Forward:  (X,A,Bv) = (q^, k^, c v).      dQ^: (dO, c v, k^)  -> state is S^T.
// dK^: (c v, dO, q^) reversed in time.     dV': (k^, q^, dO) reversed in time.
struct WalkArgs {
    const void* x; const void* a; const void* bv; const void* proj;
    void* out;
    RowLayout lx, la, lbv, lproj, lout;   // layouts of the five tensors (all zero: dense)
    const float* init;   // [BH, n_groups, d*d] or NULL (zero initial state)
    float* final_state;  // NULL, or [BH, n_groups, d*d] (final_grouped) / [BH, d*d] (one group)
    int final_grouped;
    float* dm_partial;   // [BH, n_groups] or NULL
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N; int group; int n_groups;
    int mode_x, mode_a, mode_b;
    int epilogue; int reverse; int update; int write_out;
    // Packed variable-length batch: B + 1 row offsets into tensors of total rows per head
    // (batch stride unused), every sequence cut into groups from its first row on; NULL: dense batch.
    const int* cu_seqlens;
};

cudaError_t launch_walk_simt(const WalkArgs& w, int BH, int d, cott_dtype dt, cudaStream_t st);
// `total_scale_m` non-NULL: the total written to total_out is multiplied by the stabilisation
// factor c[b,h] (the tensor-core path keeps its states unscaled).
cudaError_t launch_scan(float* states, float* total_out, int BH, int n_groups, int d, int mode,
                        cudaStream_t st, const float* total_scale_m = nullptr,
                        const float* seq_len = nullptr, float seq_len_scalar = 0.f, int H = 1,
                        int N = 1, const float* init_in = nullptr);

// Tensor-core running-sum walk (bf16, d in {64,128}) with operand roles (x, a, bv); see
// cott_tc_walk.cu.  mode: 0 partial states of every group, 1 chunk walk from the group's
// prefix / suffix state, 2 read-out Out = X State for a fixed state.
struct TcWalkArgs {
    int mode;
    const void* x; const void* a; const void* bv; const void* proj; void* out;
    RowLayout lx, la, lbv, lproj, lout;   // layouts of the five tensors (all zero: dense)
    // Packed variable-length batch: device array of B + 1 row offsets into tensors that hold
    // total_tokens rows per head (batch stride unused); every sequence cut into groups from its first
    // row on.  NULL: dense batch.
    const int* cu_seqlens; int total_tokens;
    const float* init; float* state_out; float* dm_partial; int* status;
    const float* dm_extra;   // the stream that finalises dm: the [BH, n_groups] part another stream summed, or NULL
    const float* m; const float* seq_len; float seq_len_scalar;
    int group; int n_groups;
    int norm_bv; int x_norm; int epilogue; int reverse;
    int init_sum;   // 1: `init` holds raw partial states; the walk forms its own prefix / suffix / total
    // With init_sum the partial states may come from a finer partition than the walk's groups:
    // init_split consecutive entries of `init` per group (0 or 1: one entry per group).
    int init_split;
    int init_transposed;  // 1: `init` holds the transposes of the states this walk starts from
    // State-only pass: groups first_group .. first_group + grid_groups - 1 are computed
    // (grid_groups == 0 means all of them).  A causal walk never reads the partial state of
    // the group it visits last, so that group is left out unless the total is exported.
    int first_group; int grid_groups;
    // 1: plain stream-ordered launch.  Default (0) is a programmatic dependent launch, whose
    // prologue overlaps the tail of the previous kernel of the same stream; launches that
    // follow a cross-stream event wait are made plain.
    int plain_launch;
    // 1: this is the first kernel of a library call; its first CTA clears the status words of
    // the workspace header (a wait that gives up writes them two seconds later at the earliest),
    // which saves a separate memset in front of every call.
    int clear_status;
    // On the stream that carries the dm sum (dm_partial set: the dQ^ stream of the tensor-core
    // path): when set, the CTA that finishes last turns the
    // [BH, n_groups] partial sums into dm[H] (fixed summation order), so no separate launch
    // is needed.
    float* dm_out;
    // Causal walk of a single group: `init` is a caller's state (it contains c and is divided
    // by c on the way in), and the state after the last token goes to state_final, times c.
    int init_has_scale;
    float* state_final;
    // Columns the tensors really have, when fewer than the kernel's d: x and a have d_xa, bv,
    // the raw rows and out have d_bo (0: d).  The tensor maps get the real extents -- tiles are
    // zero-filled beyond them on the way in and clipped on the way out -- and everything else
    // (states, workspace) keeps the kernel's d.  Zero columns change no norm, score or product.
    int d_xa; int d_bo;
};
cudaError_t launch_tc_walk(const TcWalkArgs& a, int B, int H, int N, int d, cudaStream_t st);

// Fused causal backward at d = 64 (cott_tc_bwd.cu): one walk forward in time over every group
// produces dq, dk, dv and the dm sum.  sq_part / r_part are the partial states of the groups
// (V^T K^ and Q^^T dO), written by launch_tc_bwd_states: a group reads sq_part of the groups
// before it and r_part of itself and the groups after it.
struct TcBwdFusedArgs {
    const void* q; const void* k; const void* v; const void* d_o;
    void* dq; void* dk; void* dv;
    RowLayout l_qkv, l_do, l_dqkv;
    RowLayout l_v, l_dv;      // v and dv (their own when the value size differs from the key size)
    const float* sq_part; const float* r_part;
    float* dm_partial; float* dm_out; int* status;
    const float* m; const float* seq_len; float seq_len_scalar;
    int group; int n_groups;
    int plain_launch;
    // Causal walk: the partial states K^^T V the forward call of the same q, k, v left in its
    // workspace ([BH, n_groups * sq_fwd_split, 64 * 64], unscaled; every group but the last): read
    // transposed instead of sq_part, which the state pass then does not compute.  NULL: none.
    const float* sq_fwd; int sq_fwd_split;
    // Packed variable-length batch: B + 1 row offsets into tensors of total_tokens rows per head, one
    // group per (sequence, head); NULL: dense batch.
    const int* cu_seqlens; int total_tokens;
    // Segment of a longer causal sequence (cott_bwd_stateful; all NULL otherwise): fp32 [BH, 64, 64]
    // in the kernels' size -- the incoming state (it contains c), the gradient of the outgoing
    // state, and where the gradient of the incoming state goes.
    const float* state_in; const float* d_state_out; float* d_state_in;
    int bidir;      // 1: all-ones mask (bidirectional backward): both states are totals over the sequence
    int w_k, w_v;   // real columns of q, k, dq, dk and of v, dO, dv when fewer than 64 (0: 64)
};
cudaError_t launch_tc_bwd_fused(const TcBwdFusedArgs& a, int B, int H, int N, cudaStream_t st);
// Bidirectional backward of one group per (b, h) (or per sequence and head of a packed batch) at
// d <= 64 in one launch (cott_tc_bidir_bwd.cu): uses the tensors, layouts, widths, dm_partial
// ([B * H] floats), dm_out, status (words 0-7 zero at launch), m, seq_len and cu_seqlens of `a`.
cudaError_t launch_tc_bidir_bwd(const TcBwdFusedArgs& a, int B, int H, int N, cudaStream_t st);
// Both partial states of every group in one launch (uses q, k, v, d_o, the layouts, group,
// n_groups and status of `a`); clear_status: this is the first kernel of a library call.
cudaError_t launch_tc_bwd_states(const TcBwdFusedArgs& a, float* sq_out, float* r_out, int clear_status, int B, int H,
                                 int N, cudaStream_t st);

// Partial states A^^T B (A's rows normalised) of the first grid_groups groups of every (b, h) at
// d <= 64, written to out[(bh * n_groups + g) * 64 * 64] (cott_tc_bwd.cu).
cudaError_t launch_tc_pair_states(const void* a_rows, const void* b_rows, const RowLayout& l_a, const RowLayout& l_b,
                                  int w_a, int w_b, float* out, int* status, int clear_status, int B, int H, int N,
                                  int group, int n_groups, int grid_groups, int plain_launch, cudaStream_t st);

// Bidirectional forward at d = 64 in one launch, one CTA per (b, h) (cott_tc_bidir.cu); it is
// the first (and only) kernel of its call and clears the status words itself.
cudaError_t launch_tc_bidir_fwd(const void* q, const void* k, const void* v, void* o, const RowLayout& l_qkv,
                                const RowLayout& l_v, const RowLayout& l_o, float* state_out, int* status, const float* m, const float* seq_len,
                                float seq_len_scalar, int B, int H, int N, cudaStream_t st, int dk = 0, int dv = 0,
                                const int* cu_seqlens = nullptr, int total_tokens = 0);

// Tensor map over a bf16 tensor of logical shape [B,H,N,d] with the given row layout: box of
// 128 tokens x 64 columns of one (b,h), 128-byte swizzle (see cott_tc_walk.cu).
bool make_tile_map(CUtensorMap* map, const void* ptr, int B, int H, int N, int d, const RowLayout& lay,
                   bool* head_first, int box_rows = 128);

bool make_rows_map(CUtensorMap* map, const void* ptr, long long rows, int d, int box_rows);

// Forward for sequences of at most 128 tokens in dense [B,H,N,d] tensors (cott_tc_short.cu): the
// quadratic form, several sequences per 128-row tile, no state; the only kernel of its call.
cudaError_t launch_tc_short_fwd(const void* q, const void* k, const void* v, void* o, int* status, const float* m,
                                const float* seq_len, float seq_len_scalar, int B, int H, int N, int d, int dk, int dv,
                                int causal, cudaStream_t st);

// A block of at most 64 tokens per (b, h) on a caller's state (cott_tc_block.cu): o and the new
// state in one launch, the only kernel of its call.
cudaError_t launch_tc_block_fwd(const void* q, const void* k, const void* v, void* o, const RowLayout& l_qk,
                                const RowLayout& l_v, const RowLayout& l_o, const float* state_in, float* state_out,
                                int* status, const float* m, const float* seq_len, float seq_len_scalar, int B, int H,
                                int N, int d, int dk, int dv, cudaStream_t st);

// Opt-in to `bytes` of dynamic shared memory for a kernel, once per (kernel, device).
cudaError_t configure_smem_once(const void* func, int bytes);

// Library options (cott_set_option; environment variables give the defaults, read once).
int option_force_group();
int option_force_path();
int option_pair();
int option_fused_bwd();
int option_fused_bidir();
int option_bidir_bwd();
int option_short_fwd();
int option_block_fwd();
int wait_limit_kcycles();      // bound of every device-side wait, in units of 1024 SM cycles

cudaError_t launch_dm_finalize(const float* dm_partial, float* dm, const float* m,
                               const float* seq_len, float seq_len_scalar, int B, int H,
                               int n_groups, int N, cudaStream_t st, const int* cu_seqlens = nullptr);
cudaError_t launch_sum_slices(const float* parts, float* out, int n, int H, cudaStream_t st);
// Caller-visible states [BH, dk, dv] <-> the kernels' padded [BH, d, d] (zero outside).
cudaError_t launch_transpose_state(const float* src, float* dst, int BH, int d, cudaStream_t st);
cudaError_t launch_state_prep(const float* src, float* dst, int BH, int d, int transpose, int scale_mode, const float* m,
                              const float* seq_len, float seq_len_scalar, int H, int N, cudaStream_t st);
cudaError_t launch_segment_finish(const float* state_in, const float* d_state_out, const float* tq_total, const float* tk_total,
                                  float* d_state_in, float* dm_partial, const float* fold, int BH, int n_groups, int d,
                                  const float* m, const float* seq_len, float seq_len_scalar, int H, int N, cudaStream_t st);
cudaError_t launch_pad_state(const float* src, float* dst, int BH, int dk, int dv, int d, cudaStream_t st);
cudaError_t launch_unpad_state(const float* src, float* dst, int BH, int dk, int dv, int d, cudaStream_t st);
// Decode step for head sizes the specialised kernel does not cover (any dk, dv multiples of 4 / 8).
cudaError_t launch_decode_generic(const void* q, const void* k, const void* v, float* state, void* o,
                                  int B, int H, int dk, int dv, cott_dtype dt, const float* m,
                                  const float* seq_len, float seq_len_scalar, cudaStream_t st);
cudaError_t launch_decode(const void* q, const void* k, const void* v, float* state, void* o,
                          int B, int H, int d, cott_dtype dt, const float* m,
                          const float* seq_len, float seq_len_scalar, cudaStream_t st);

// Optional per-launch timing of the tensor-core walk kernels (cott_profile_enable): returns
// the index of the event pair to record around the next launch, or -1 when disabled / full.
int profile_begin_launch(int kind, cudaStream_t st);
void profile_end_launch(int idx, cudaStream_t st);

// Counts kernel launches issued by this process (reported by cott_launch_count).
void note_launch(int n = 1);

// Stabilisation factor of Eq. 4 in fp32: c = exp(-sigmoid(m) * ln s).
__device__ __forceinline__ float stab_factor(float m, float s) {
    float sg = 1.0f / (1.0f + expf(-m));
    return expf(-sg * logf(s));
}

}  // namespace cott
