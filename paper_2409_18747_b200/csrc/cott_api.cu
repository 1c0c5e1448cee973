// C-ABI entry points of libcott: argument validation, execution plan, workspace layout and
// the launch sequences.  All arithmetic of the method runs in the kernels.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <atomic>
#include <mutex>
#include <utility>
#include <vector>
#include "cott_internal.h"

namespace cott {

static thread_local char g_cuda_error[256] = "";
static std::atomic<unsigned long long> g_launches{0};
void note_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

// ---- optional per-launch timing (library-owned CUDA events; created on first use)
static constexpr int kProfMax = 256;
static cudaEvent_t g_prof_ev[2 * kProfMax];
static int g_prof_kind[kProfMax];
static int g_prof_tag[kProfMax];        // non-zero: launches with the same tag ran side by side
static thread_local int g_prof_cur_tag = 0;
static std::atomic<int> g_prof_next_tag{1};
static bool g_prof_created = false;
static std::atomic<int> g_prof_n{-1};   // -1: disabled
static int g_prof_cap = 0;

int profile_begin_launch(int kind, cudaStream_t st) {
    int n = g_prof_n.load(std::memory_order_relaxed);
    if (n < 0 || n >= g_prof_cap) return -1;
    n = g_prof_n.fetch_add(1);
    if (n >= g_prof_cap) return -1;
    g_prof_kind[n] = kind;
    g_prof_tag[n] = g_prof_cur_tag;
    cudaEventRecord(g_prof_ev[2 * n], st);
    return n;
}
void profile_end_launch(int idx, cudaStream_t st) {
    if (idx >= 0) cudaEventRecord(g_prof_ev[2 * idx + 1], st);
}

static cott_status cuda_fail(cudaError_t e, const char* where) {
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", where, cudaGetErrorString(e));
    return COTT_ERR_CUDA;
}
#define COTT_CUDA(expr)                                          \
    do {                                                         \
        cudaError_t e__ = (expr);                                \
        if (e__ != cudaSuccess) return cuda_fail(e__, #expr);    \
    } while (0)

// ---- options: process-wide switches for tests and measurements (none is needed in use).
// Each starts from its environment variable, read once on first use, and can be changed with
// cott_set_option.
struct Option {
    const char* name; const char* env; long long dflt;
    std::atomic<long long> value;
    std::once_flag once;
    Option(const char* n, const char* e, long long d) : name(n), env(e), dflt(d), value(d) {}
    long long get() {
        std::call_once(once, [this] {
            const char* v = getenv(env);
            if (v && *v) value.store(atoll(v), std::memory_order_relaxed);
        });
        return value.load(std::memory_order_relaxed);
    }
    void set(long long v) { get(); value.store(v, std::memory_order_relaxed); }
};
static Option g_opt_force_group("force_group", "COTT_FORCE_GROUP", 0);     // tokens per sequence group (0: the plan's)
static Option g_opt_force_path("force_path", "COTT_FORCE_PATH", 1);        // 0: bf16 d=64/128 through the fp32-accumulating SIMT kernels
static Option g_opt_pair("pair", "COTT_PAIR", 1);                          // 0: gradient streams one after the other
static Option g_opt_fused_bwd("fused_bwd", "COTT_FUSED_BWD", 1);           // 0: causal d=64 backward through the three role-swapped walks
static Option g_opt_fused_bidir("fused_bidir", "COTT_FUSED_BIDIR", 1);     // 0: bidirectional d=64 forward as state pass + read-out
static Option g_opt_bidir_bwd("bidir_bwd", "COTT_BIDIR_BWD", 1);           // 0: bidirectional d=64 backward of one group per (b, h) as state pass + walk
static Option g_opt_short_fwd("short_fwd", "COTT_SHORT_FWD", 1);           // 0: sequences of <= 128 tokens through the generic walk
static Option g_opt_block_fwd("block_fwd", "COTT_BLOCK_FWD", 1);           // 0: blocks of <= 64 tokens on a state through the generic walk
static Option g_opt_wait_ms("wait_limit_ms", "COTT_WAIT_LIMIT_MS", 2000);  // bound of every device-side wait
static Option g_opt_wait_kc("wait_limit_kcycles", "COTT_WAIT_LIMIT_KCYCLES", -1);  // the same in units of 1024 SM cycles (< 0: use the ms value)
static Option g_opt_host_slices("host_slices", "COTT_HOST_SLICES", 8);     // slices of the host-buffer step (1 .. 16)
static Option* const g_options[] = {&g_opt_force_group, &g_opt_force_path, &g_opt_pair, &g_opt_fused_bwd,
                                    &g_opt_wait_ms, &g_opt_wait_kc, &g_opt_host_slices, &g_opt_fused_bidir, &g_opt_short_fwd, &g_opt_block_fwd, &g_opt_bidir_bwd};

int option_force_group() { return (int)g_opt_force_group.get(); }
int option_force_path() { return (int)g_opt_force_path.get(); }
int option_pair() { return (int)g_opt_pair.get(); }
int option_fused_bwd() { return (int)g_opt_fused_bwd.get(); }
int option_fused_bidir() { return (int)g_opt_fused_bidir.get(); }
int option_bidir_bwd() { return (int)g_opt_bidir_bwd.get(); }
int option_short_fwd() { return (int)g_opt_short_fwd.get(); }
int option_block_fwd() { return (int)g_opt_block_fwd.get(); }
int wait_limit_kcycles() {
    const long long kc = g_opt_wait_kc.get();
    if (kc >= 0) return (int)(kc > 200000000 ? 200000000 : kc);
    const long long ms = g_opt_wait_ms.get();
    return (int)((ms < 1 ? 1 : (ms > 100000 ? 100000 : ms)) * 2000);   // <= 2 GHz
}

cudaError_t configure_smem_once(const void* func, int bytes) {
    static std::mutex mu;
    static std::vector<std::pair<const void*, int>> done;      // (kernel, device) pairs already configured
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (const auto& it : done)
        if (it.first == func && it.second == dev) return cudaSuccess;
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    done.emplace_back(func, dev);
    return cudaSuccess;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static size_t dtype_size(cott_dtype dt) { return dt == COTT_F32 ? 4 : 2; }

struct Plan {
    int path;      // 0 SIMT, 1 tensor core
    int group;     // tokens per sequence group
    int chunk;     // tokens per chunk inside a group
    int n_groups;
    int split;   // partial-state pass: parts per group when the walk sums the prefix itself
    // Head sizes: dk columns in q, k (and dq, dk), dv in v, o, dO (and dv).  `d` is the size the
    // kernels run at: dk = dv = d on the fp32-accumulating SIMT path; on the tensor-core path
    // the smallest of 64 and 128 that holds both, the tiles zero-filled beyond the real columns
    // (`padded`: a caller's state then goes through a [BH, d, d] copy in the workspace).
    int d, dk, dv;
    bool padded;
};

// Sequence groups give sequence-level parallelism when B*H alone cannot fill the GPU:
// halve the group until there are enough CTAs, but never below a floor that keeps the
// per-group state traffic (d*d fp32) small against the group's own q,k,v,o bytes.
// May every walk CTA sum the partial states it needs itself (no scan launch)?  Only while those
// extra reads (n_groups / 2 states of d x d floats per CTA on average) stay small against the
// group's own rows: measured at B*H = 16, d = 128, dropping the scan launch this way where the
// rule says no cost 14 us at N = 4096 (58.7 against 44.6 us) and at N = 16384 (107 against 94 us).
static bool fused_scan_ok(int n_groups, int d, int group) {
    return (long long)n_groups * d * 8 <= group;
}

static bool make_plan(int op, cott_dtype dt, int B, int H, int N, int dk, int dv, int causal, Plan* p) {
    if (B < 1 || H < 1 || N < 1) return false;
    if (dt != COTT_F32 && dt != COTT_BF16) return false;
    const long BH = (long)B * H;
    const int forced = option_force_group();
    // Tensor cores: bf16, head sizes that are multiples of 8 (16-byte rows) up to 128.
    const bool tc_ok = dt == COTT_BF16 && dk >= 8 && dv >= 8 && dk <= 128 && dv <= 128 && dk % 8 == 0 && dv % 8 == 0;
    const bool simt_ok = dk == dv && (dk == 32 || dk == 64 || dk == 128);
    if (!tc_ok && !simt_ok) return false;
    p->path = (tc_ok && (option_force_path() != 0 || !simt_ok)) ? 1 : 0;
    p->dk = dk; p->dv = dv;
    p->d = p->path == 1 ? ((dk <= 64 && dv <= 64) ? 64 : 128) : dk;
    p->padded = dk != p->d || dv != p->d;
    const int d = p->d;
    int group;
    if (p->path == 1) {
        // One CTA per (b,h) and group, one CTA per SM.  Measured on B200: fewer, longer
        // groups win (per-CTA set-up and the per-group state traffic shrink) as long as
        // about every SM still gets a CTA, and a single group per (b,h) needs no partial-state
        // pass at all.  So: as many groups per (b,h) as fit in ONE wave of CTAs (rounded
        // down), each a multiple of the 128-token chunk.
        p->chunk = 128;
        const long per_head = BH >= 148 ? 1 : 148 / BH;
        long g = (N + per_head - 1) / per_head;
        group = (int)((g + 127) / 128 * 128);
        // Nine groups per (b,h): eight equal ones are faster while a group stays within 32
        // chunks -- the partial-state pass covers 7/8 instead of 8/9 of the sequence and no
        // group is a short straggler (measured at B*H = 16, d = 128: N=16384 96.7 us against
        // 102.5 us, N=32768 160 against 166) -- and slower beyond about N=49152, where 144
        // CTAs instead of 128 matter more.
        if (causal && per_head == 9) {
            const int g8 = (int)((((long)N + 7) / 8 + 127) / 128 * 128);
            if (g8 <= 4096 && (N + g8 - 1) / g8 == 8) group = g8;
        }
    } else {
        p->chunk = 16;
        group = 1024;
        while (group > 128 && BH * ((N + group - 1) / group) < 4 * 148) group >>= 1;
    }
    if (forced > 0) group = (forced + p->chunk - 1) / p->chunk * p->chunk;
    if (group >= N) group = (N + p->chunk - 1) / p->chunk * p->chunk;
    p->group = group;
    p->n_groups = (N + group - 1) / group;
    // With the prefix summed inside the walk (few groups, see run_tc_stream), the state pass
    // may use a finer partition than the walk -- each group cut into `split` equal parts of
    // whole chunks -- when that still fits in one wave of CTAs: its CTAs get shorter, the walk
    // sums `split` times as many states.
    p->split = 1;
    if (p->path == 1 && causal && p->n_groups >= 2 && p->n_groups <= 8 &&
        fused_scan_ok(p->n_groups, d, group) && N % group == 0) {
        const long ctas = BH * (p->n_groups - 1);
        const int chunks = group / p->chunk;
        for (int s2 = 4; s2 >= 2; s2 >>= 1)
            if (ctas * s2 <= 148 && chunks % s2 == 0 && chunks / s2 >= 4) { p->split = s2; break; }
    }
    return true;
}

static size_t states_bytes(const Plan& p, int B, int H, int d) {
    return align_up((size_t)B * H * p.n_groups * p.split * d * d * sizeof(float), 256);
}

// (padded head sizes: room for a caller's initial and final state in the kernels' size)
static size_t padded_state_bytes(const Plan& p, int B, int H) {
    return p.padded ? align_up((size_t)B * H * p.d * p.d * sizeof(float), 256) : 0;
}

// (backward of a segment: the caller's two states and the one it gets back, in the kernels' size)
static size_t segment_state_bytes(int B, int H, int d) { return align_up((size_t)B * H * d * d * sizeof(float), 256); }

static size_t workspace_bytes_impl(int op, const Plan& p, int B, int H, int d) {
    size_t total = kWsHeaderBytes;
    if (op == COTT_OP_FWD) total += states_bytes(p, B, H, d) + 2 * padded_state_bytes(p, B, H);
    else if (op == COTT_OP_BWD)
        total += 3 * states_bytes(p, B, H, d) + 2 * align_up((size_t)B * H * p.n_groups * 4, 256) +
                 (p.padded ? 6 : 3) * segment_state_bytes(B, H, d);
    return total;
}

static cott_status check_scale(const cott_scale_params* sp) {
    if (!sp || !sp->m) return COTT_ERR_INVALID_ARG;
    return COTT_OK;
}

// Layouts of the tensors of one call: q, k, v share one, o (forward) / dO (backward) has one,
// dq, dk, dv share one.  All zero: dense [B,H,N,d].
struct CallLayouts {
    RowLayout qkv, o, dqkv;
    const void* q; const void* k; const void* v; const void* o_or_do;
    // Different key and value sizes: v and dv may have layouts of their own (dense tensors of
    // another width), and every tensor has its own column count.
    RowLayout vl, dvl;
    bool own_v = false;
    const void* dv_ptr = nullptr;
    int dk = 0, dv = 0;
    RowLayout of(const void* ptr) const {
        if (ptr == v && own_v) return vl;
        if (ptr == q || ptr == k || ptr == v) return qkv;
        if (ptr == o_or_do) return o;
        if (ptr == dv_ptr && own_v) return dvl;
        return dqkv;
    }
    int width(const void* ptr) const { return (ptr == v || ptr == o_or_do || ptr == dv_ptr) ? dv : dk; }
    template <class Args> void assign(Args& a) const {
        a.lx = of(a.x); a.la = of(a.a); a.lbv = of(a.bv); a.lproj = of(a.proj);
        a.lout = (a.out == o_or_do) ? o : of(a.out);
    }
    void assign_widths(TcWalkArgs& a) const { a.d_xa = width(a.x ? a.x : a.a); a.d_bo = width(a.bv); }
};
static RowLayout to_layout(const cott_strides* s) {
    return s ? RowLayout{s->batch, s->head, s->token} : RowLayout{0, 0, 0};
}
// Element strides the kernels can address: rows of d contiguous elements, 16-byte aligned.
static bool layout_ok(const cott_strides* s, int d, cott_dtype dt) {
    if (!s) return true;
    const long long q = 16 / (long long)dtype_size(dt);
    return s->batch >= d && s->head >= d && s->token >= d && s->batch % q == 0 && s->head % q == 0 &&
           s->token % q == 0;
}

// Do two tensors of logical shape [B,H,N,d] share bytes?  Each is a set of rows of d elements.
// The test answers "yes" only when it can prove it: (1) equal base addresses; (2) both tensors
// dense in memory (their dimensions merge into one contiguous block): the byte ranges decide;
// (3) both with the same strides, every stride a multiple of the smallest one above the merged
// innermost block (slices of one fused buffer, [B,N,H,d] storage): the rows of both sit on one
// lattice and the offset between the bases decides.  Anything else passes.
struct Extent {
    long long block;     // elements of the contiguous innermost block after merging dimensions
    long long step;      // smallest stride above that block (0: the tensor is one block)
    bool lattice;        // every larger stride is a multiple of `step`
    long long span;      // elements from the first to one past the last
};
static Extent extent_of(const cott_strides* st, int B, int H, int N, int d) {
    long long ext[3] = {B, H, N};
    long long str[3] = {st ? st->batch : (long long)H * N * d, st ? st->head : (long long)N * d, st ? st->token : (long long)d};
    // sort the three outer dimensions by stride (extent-1 dimensions do not matter)
    for (int i = 0; i < 3; ++i)
        for (int j = i + 1; j < 3; ++j)
            if (str[j] < str[i]) { long long t = str[i]; str[i] = str[j]; str[j] = t; t = ext[i]; ext[i] = ext[j]; ext[j] = t; }
    Extent e;
    e.block = d; e.step = 0; e.lattice = true; e.span = d;
    for (int i = 0; i < 3; ++i) {
        if (ext[i] == 1) continue;
        if (e.step == 0 && str[i] == e.block) e.block *= ext[i];          // contiguous with what is below: merge
        else if (e.step == 0) e.step = str[i];
        else if (str[i] % e.step != 0) e.lattice = false;
    }
    e.span = d;
    for (int i = 0; i < 3; ++i) e.span += (ext[i] - 1) * str[i];
    return e;
}
static bool same_strides(const cott_strides* a, const cott_strides* b) {
    if (!a || !b) return a == b;
    return a->batch == b->batch && a->head == b->head && a->token == b->token;
}
static bool tensors_overlap(const void* pa, const cott_strides* sa, const void* pb, const cott_strides* sb2,
                            int B, int H, int N, int d, cott_dtype dt, int d_b = 0) {
    if (pa == pb) return true;
    const long long es = (long long)dtype_size(dt);
    const Extent a = extent_of(sa, B, H, N, d);
    const Extent b = extent_of(sb2, B, H, N, d_b > 0 ? d_b : d);
    const long long a0 = (long long)reinterpret_cast<uintptr_t>(pa), b0 = (long long)reinterpret_cast<uintptr_t>(pb);
    const bool ranges = a0 < b0 + b.span * es && b0 < a0 + a.span * es;
    if (!ranges) return false;
    if (a.step == 0 && b.step == 0) return true;                          // two dense blocks whose ranges meet
    if (same_strides(sa, sb2) && a.lattice && a.step > 0) {
        long long delta = ((b0 - a0) / es) % a.step;                       // (bases are element-aligned)
        if (delta < 0) delta += a.step;
        // rows of a cover [0, a.block) of every period, rows of b [delta, delta + b.block)
        return delta < a.block || a.step - delta < b.block;
    }
    return false;
}

static WalkArgs base_walk(const cott_scale_params* sp, int H, int N, const Plan& p) {
    WalkArgs w;
    memset(&w, 0, sizeof(w));
    w.m = sp->m; w.seq_len = sp->seq_len; w.seq_len_scalar = sp->seq_len_scalar;
    w.H = H; w.N = N; w.group = p.group; w.n_groups = p.n_groups;
    return w;
}

// One gradient / output stream through the generic walk: (optional) per-group partial
// states, their scan, then the walk that produces rows.
static cott_status run_stream(WalkArgs w, const Plan& p, int BH, int d, cott_dtype dt, int causal,
                              float* states, float* total_out, cudaStream_t st,
                              const float* state_in = nullptr) {
    const bool single = causal && p.n_groups == 1 && !state_in;
    if (single) {
        w.init = nullptr; w.update = 1; w.write_out = 1;
        w.final_state = total_out; w.final_grouped = 0;
        COTT_CUDA(launch_walk_simt(w, BH, d, dt, st));
        return COTT_OK;
    }
    WalkArgs a = w;  // phase A: partial state of every group, no rows
    a.init = nullptr; a.update = 1; a.write_out = 0; a.out = nullptr; a.proj = nullptr;
    a.epilogue = EPI_PLAIN; a.dm_partial = nullptr;
    a.final_state = states; a.final_grouped = 1;
    COTT_CUDA(launch_walk_simt(a, BH, d, dt, st));
    const int mode = !causal ? SCAN_TOTAL : (w.reverse ? SCAN_SUFFIX : SCAN_PREFIX);
    // (these states contain c, like a caller's initial state, which the scan starts from)
    COTT_CUDA(launch_scan(states, total_out, BH, p.n_groups, d, mode, st, nullptr, nullptr, 0.f, 1, 1,
                          state_in));
    w.init = states; w.update = causal ? 1 : 0; w.write_out = 1; w.final_state = nullptr;
    COTT_CUDA(launch_walk_simt(w, BH, d, dt, st));
    return COTT_OK;
}

// One output stream through the tensor-core walk: partial states of every group, their
// scan, then the chunk walk (causal) or the read-out against the total (bidirectional).
// A causal call with a single group needs only the walk.
static cott_status run_tc_stream(TcWalkArgs t, const Plan& p, int B, int H, int N, int d,
                                 int causal, const cott_scale_params* sp, int* status,
                                 float* states, float* total_out, cudaStream_t st,
                                 bool reuse_states = false, bool states_only = false,
                                 bool states_transposed = true, const float* state_in = nullptr) {
    const bool reuse_transposed = reuse_states;
    t.status = status; t.m = sp->m; t.seq_len = sp->seq_len; t.seq_len_scalar = sp->seq_len_scalar;
    t.group = p.group; t.n_groups = p.n_groups;
    // t.clear_status (first stream of a call) applies to the first kernel launched here only.
    if (causal && p.n_groups == 1) {
        // One group: the walk alone, starting from the caller's state (if any) and leaving the
        // final state (if asked for).
        t.mode = 1; t.init = state_in; t.init_has_scale = state_in ? 1 : 0; t.state_out = nullptr;
        t.state_final = total_out;
        COTT_CUDA(launch_tc_walk(t, B, H, N, d, st));
        return COTT_OK;
    }
    // Few groups and no state export: every walk CTA sums the partial states it needs itself
    // and the scan launch is dropped -- as long as those extra d x d reads (n_groups / 2 of
    // them on average) stay small against the group's own q, k, v, o bytes.
    // (A caller's initial state enters through the scan kernel.)
    const bool fused_scan = !total_out && !state_in && p.n_groups <= 8 && fused_scan_ok(p.n_groups, d, p.group);
    const int split = (fused_scan && causal) ? p.split : 1;
    if (!reuse_transposed) {
        TcWalkArgs a = t;
        a.group = p.group / split; a.n_groups = p.n_groups * split;
        a.mode = 0; a.x = nullptr; a.proj = nullptr; a.out = nullptr; a.init = nullptr;
        a.state_out = states; a.dm_partial = nullptr; a.dm_out = nullptr; a.epilogue = EPI_PLAIN;
        t.clear_status = 0;              // the state pass, launched first, does it
        a.reverse = t.reverse ? 0 : 1;   // chunk order opposite to the walk's: L2 reuse of its tiles
        if (causal && !total_out) {
            // Nobody reads the partial state of the group the walk visits last.
            a.grid_groups = (p.n_groups - 1) * split;
            a.first_group = t.reverse ? split : 0;
        }
        // The forward's pass at d = 64 (k normalised, v raw, forward in time) has a lighter kernel
        // of its own: stages of two tiles, a ring twice as deep.
        const bool light = d == 64 && !t.cu_seqlens && t.epilogue == EPI_PLAIN && t.x_norm && !t.norm_bv && !t.reverse &&
                           option_fused_bwd() != 0;
        if (light) {
            COTT_CUDA(launch_tc_pair_states(a.a, a.bv, a.la, a.lbv, a.d_xa > 0 ? a.d_xa : d, a.d_bo > 0 ? a.d_bo : d, states,
                                            status, a.clear_status, B, H, N, a.group, a.n_groups,
                                            a.grid_groups > 0 ? a.grid_groups : a.n_groups, a.plain_launch, st));
        } else {
            COTT_CUDA(launch_tc_walk(a, B, H, N, d, st));
        }
        const int mode = !causal ? SCAN_TOTAL : (t.reverse ? SCAN_SUFFIX : SCAN_PREFIX);
        if (!fused_scan)
            COTT_CUDA(launch_scan(states, total_out, B * H, p.n_groups, d, mode, st, sp->m, sp->seq_len,
                                  sp->seq_len_scalar, H, N, state_in));
    }
    // reuse_transposed: `states` already holds, transposed, what this stream needs (raw
    // partials when the scan is fused, scanned states otherwise) from a sibling stream that
    // walks in the same direction.
    if (states_only) return COTT_OK;
    t.init_sum = fused_scan ? 1 : 0;
    t.init_split = split;
    t.init_transposed = (reuse_states && states_transposed) ? 1 : 0;
    t.mode = causal ? 1 : 2; t.init = states; t.state_out = nullptr;
    COTT_CUDA(launch_tc_walk(t, B, H, N, d, st));
    return COTT_OK;
}

// Backward of a segment of a longer causal sequence (cott_bwd_stateful): the caller's fp32
// [B,H,d_k,d_v] states; state_in / d_state_out NULL = zero, d_state_in NULL = not wanted.
struct Segment {
    bool on = false;
    const float* state_in = nullptr;
    const float* d_state_out = nullptr;
    float* d_state_in = nullptr;
};

// Packed variable-length batch (see cott_fwd_varlen): row offsets and total row count.
struct Packed {
    const int* cu_seqlens = nullptr;
    int total_tokens = 0;
};

static cott_status fwd_impl(const void* q, const void* k, const void* v, void* o, float* state_out,
                            int B, int H, int N, int d, int causal, cott_dtype dt,
                            const cott_scale_params* sp, void* ws, const Plan& p,
                            cudaStream_t st, const float* state_in = nullptr,
                            const cott_strides* s_qkv = nullptr, const cott_strides* s_o = nullptr,
                            Packed packed = Packed(), const cott_strides* s_v = nullptr) {
    // (d is the size the kernels run at, p.d; the tensors have p.dk and p.dv columns)
    CallLayouts lay{to_layout(s_qkv), to_layout(s_o), RowLayout{0, 0, 0}, q, k, v, o};
    lay.dk = p.dk; lay.dv = p.dv;
    if (p.dk != p.dv || s_v) { lay.own_v = true; lay.vl = to_layout(s_v); }
    // The tensor-core path clears the status words in its first kernel.
    if (p.path != 1) COTT_CUDA(cudaMemsetAsync(ws, 0, kWsHeaderBytes, st));
    float* states = reinterpret_cast<float*>(static_cast<char*>(ws) + kWsHeaderBytes);
    // Zero-padded head sizes: the kernels read and write states of their own size.
    float* user_state_out = state_out;
    if (p.padded && (state_in || state_out)) {
        char* pad0 = static_cast<char*>(ws) + kWsHeaderBytes + states_bytes(p, B, H, d);
        float* pad_in = reinterpret_cast<float*>(pad0);
        float* pad_out = reinterpret_cast<float*>(pad0 + padded_state_bytes(p, B, H));
        if (state_in) {
            COTT_CUDA(launch_pad_state(state_in, pad_in, B * H, p.dk, p.dv, d, st));
            state_in = pad_in;
        }
        if (state_out) state_out = pad_out;
    }
    auto finish = [&]() -> cott_status {
        if (state_out != user_state_out)
            COTT_CUDA(launch_unpad_state(state_out, user_state_out, B * H, p.dk, p.dv, d, st));
        return COTT_OK;
    };
    if (p.path == 1 && N <= 128 && !packed.cu_seqlens && !state_in && !state_out && !s_qkv && !s_o && !s_v &&
        option_short_fwd() != 0) {
        // Short sequences in dense tensors: the quadratic side of Eq. 5, several sequences per
        // tile, no running state (cott_tc_short.cu).
        COTT_CUDA(launch_tc_short_fwd(q, k, v, o, static_cast<int*>(ws), sp->m, sp->seq_len, sp->seq_len_scalar, B, H, N,
                                      d, p.dk, p.dv, causal, st));
        return COTT_OK;
    }
    if (p.path == 1 && causal && N <= 64 && (state_in || state_out) && !packed.cu_seqlens && option_block_fwd() != 0) {
        // A short block on a caller's state (multi-token decode, short prefill segments): one
        // light kernel, several CTAs per SM (cott_tc_block.cu).
        COTT_CUDA(launch_tc_block_fwd(q, k, v, o, lay.qkv, lay.of(v), lay.o, state_in, state_out, static_cast<int*>(ws),
                                      sp->m, sp->seq_len, sp->seq_len_scalar, B, H, N, d, p.dk, p.dv, st));
        return finish();
    }
    if (p.path == 1 && !causal && d == 64 && p.n_groups == 1 && !(packed.cu_seqlens && state_out) && !state_in &&
        option_fused_bidir() != 0) {
        // One CTA per (b, h) -- or per (sequence, head) of a packed batch -- streams k, v into the
        // d x d state and then q through it: one launch, every tensor touched once.
        COTT_CUDA(launch_tc_bidir_fwd(q, k, v, o, lay.qkv, lay.of(v), lay.o, state_out, static_cast<int*>(ws), sp->m,
                                      sp->seq_len, sp->seq_len_scalar, B, H, N, st, p.dk, p.dv, packed.cu_seqlens,
                                      packed.total_tokens));
        return finish();
    }
    if (p.path == 1) {
        TcWalkArgs t;
        memset(&t, 0, sizeof(t));
        t.x = q; t.a = k; t.bv = v; t.out = o;
        lay.assign(t); lay.assign_widths(t);
        t.cu_seqlens = packed.cu_seqlens; t.total_tokens = packed.total_tokens;
        t.norm_bv = 0; t.x_norm = 1; t.epilogue = EPI_PLAIN; t.reverse = 0;
        // (a padded initial state was staged by a kernel of this call: the walk is not the first)
        t.clear_status = 1;
        cott_status rc = run_tc_stream(t, p, B, H, N, d, causal, sp, static_cast<int*>(ws), states,
                                       state_out, st, false, false, true, state_in);
        return rc != COTT_OK ? rc : finish();
    }
    WalkArgs w = base_walk(sp, H, N, p);
    w.cu_seqlens = packed.cu_seqlens;
    w.x = q; w.a = k; w.bv = v; w.out = o;
    lay.assign(w);
    w.mode_x = ROW_NORM; w.mode_a = ROW_NORM; w.mode_b = ROW_SCALE;
    w.epilogue = EPI_PLAIN; w.reverse = 0;
    return run_stream(w, p, B * H, d, dt, causal, states, state_out, st, state_in);
}

// Side streams and events for launches of one call that run next to each other on the GPU:
// one set per host thread and device (two calls from different threads must not share events),
// created on the first call that needs them and kept until the process ends.
constexpr int kHostSlices = 16;    // the host-buffer step moves and computes the batch in at most this many slices
struct SideStreams {
    bool ready = false;
    cudaStream_t s[3];            // [0], [1]: gradient streams of cott_bwd, copy streams of the host step; [2]: spare
    cudaEvent_t fork, join[3], fork_copy;
    cudaEvent_t slice_in[kHostSlices], slice_out[kHostSlices];   // host step: inputs of a slice landed / its results are ready
};
static SideStreams* side_streams_table() {
    static thread_local SideStreams per_device[64];
    return per_device;
}
static SideStreams* side_streams() {
    SideStreams* per_device = side_streams_table();
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    SideStreams& ss = per_device[dev];
    if (!ss.ready) {
        // s[0] carries a walk that should start together with the one on the caller's stream;
        // it gets the highest priority, so that its CTAs are placed ahead of the state pass on
        // s[1] when both become ready on the same event.
        int prio_lo = 0, prio_hi = 0;
        if (cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) != cudaSuccess) return nullptr;
        for (int i = 0; i < 3; ++i) {
            if (cudaStreamCreateWithPriority(&ss.s[i], cudaStreamNonBlocking, i == 0 ? prio_hi : prio_lo) != cudaSuccess)
                return nullptr;
            if (cudaEventCreateWithFlags(&ss.join[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        }
        if (cudaEventCreateWithFlags(&ss.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&ss.fork_copy, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        for (int i = 0; i < kHostSlices; ++i) {
            if (cudaEventCreateWithFlags(&ss.slice_in[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
            if (cudaEventCreateWithFlags(&ss.slice_out[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        }
        ss.ready = true;
    }
    return &ss;
}

static cott_status bwd_impl(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                            void* dk, void* dv, float* dm, int B, int H, int N, int d, int causal,
                            cott_dtype dt, const cott_scale_params* sp, void* ws, const Plan& p,
                            cudaStream_t st, const cott_strides* s_qkv = nullptr,
                            const cott_strides* s_do = nullptr, const cott_strides* s_dqkv = nullptr,
                            Packed packed = Packed(), const cott_strides* s_v = nullptr,
                            const cott_strides* s_dv = nullptr, const void* fwd_ws = nullptr,
                            Segment seg = Segment()) {
    // (d is the size the kernels run at, p.d; the tensors have p.dk and p.dv columns)
    CallLayouts lay{to_layout(s_qkv), to_layout(s_do), to_layout(s_dqkv), q, k, v, d_o};
    lay.dk = p.dk; lay.dv = p.dv; lay.dv_ptr = dv;
    if (p.dk != p.dv || s_v || s_dv) { lay.own_v = true; lay.vl = to_layout(s_v); lay.dvl = to_layout(s_dv); }
    // The tensor-core path clears the status words in its first kernel.
    if (p.path != 1) COTT_CUDA(cudaMemsetAsync(ws, 0, kWsHeaderBytes, st));
    char* base = static_cast<char*>(ws) + kWsHeaderBytes;
    const size_t sb = states_bytes(p, B, H, d);
    float* st0 = reinterpret_cast<float*>(base);
    float* st1 = reinterpret_cast<float*>(base + sb);
    float* st2 = reinterpret_cast<float*>(base + 2 * sb);
    float* dm_partial = reinterpret_cast<float*>(base + 3 * sb);
    float* dm_partial2 = dm_partial + align_up((size_t)B * H * p.n_groups * 4, 256) / 4;
    const int BH = B * H;
    cott_status rc;
    if (p.path == 1) {
        int* status = static_cast<int*>(ws);
        TcWalkArgs t;
        memset(&t, 0, sizeof(t));
        t.cu_seqlens = packed.cu_seqlens; t.total_tokens = packed.total_tokens;
        // When two walks with one CTA per (b, h) fit on the GPU side by side but not two per
        // (b, h) (74 / 2 < B*H <= 74), the dK^ and dV' streams run next to each other, each
        // over the whole sequence as a single group (no partial-state pass, no scan), with the
        // dQ^ stream's partial-state pass filling the SMs that are left; the dQ^ walk follows on
        // the whole GPU.  Each side stream then carries one tensor-core kernel per call.
        if (d == 64 && option_fused_bwd() != 0) {
            // One walk forward in time gives all three gradients and the dm sum (cott_tc_bwd.cu).
            // It keeps two running states: Sq = V^T K^ over earlier tokens, accumulated chunk by
            // chunk, and R = Q^^T dO over later tokens, which starts at the sum over the group
            // and everything after it and is taken down as the walk passes.  Before it, one
            // state-only launch gives both partial states of every group.
            TcBwdFusedArgs f;
            memset(&f, 0, sizeof(f));
            f.q = q; f.k = k; f.v = v; f.d_o = d_o; f.dq = dq; f.dk = dk; f.dv = dv;
            f.l_qkv = lay.qkv; f.l_do = lay.o; f.l_dqkv = lay.dqkv;
            f.l_v = lay.of(v); f.l_dv = lay.of(dv); f.w_k = p.dk; f.w_v = p.dv;
            f.sq_part = st0; f.r_part = st1;
            f.dm_partial = dm_partial; f.dm_out = dm; f.status = status;
            f.m = sp->m; f.seq_len = sp->seq_len; f.seq_len_scalar = sp->seq_len_scalar;
            f.group = p.group; f.n_groups = p.n_groups;
            f.bidir = causal ? 0 : 1;
            f.cu_seqlens = packed.cu_seqlens; f.total_tokens = packed.total_tokens;
            // The forward call of the same q, k, v (no state in or out) left the partial states
            // K^^T V of every group but the last in its workspace whenever its walk summed them
            // itself: the transposes of what this walk needs, so the state pass skips k and v.
            if (fwd_ws && !packed.cu_seqlens && causal && p.n_groups >= 2 && p.n_groups <= 8 && fused_scan_ok(p.n_groups, d, p.group)) {
                f.sq_fwd = reinterpret_cast<const float*>(static_cast<const char*>(fwd_ws) + kWsHeaderBytes);
                f.sq_fwd_split = p.split;
            }
            if (seg.on) {
                // A segment: the states enter and leave through copies of the kernels' size behind
                // the other regions of the workspace (zero where the caller passed none).
                char* sbase = base + 3 * sb + 2 * align_up((size_t)B * H * p.n_groups * 4, 256);
                const size_t ssb = segment_state_bytes(B, H, d);
                float* s_in = reinterpret_cast<float*>(sbase);
                float* ds_out = reinterpret_cast<float*>(sbase + ssb);
                float* ds_in = reinterpret_cast<float*>(sbase + 2 * ssb);
                if (!p.padded) {
                    // (states of the kernels' own size: read and written where the caller has them)
                    f.state_in = seg.state_in; f.d_state_out = seg.d_state_out; f.d_state_in = seg.d_state_in;
                } else {
                    if (seg.state_in) COTT_CUDA(launch_pad_state(seg.state_in, s_in, BH, p.dk, p.dv, d, st));
                    if (seg.d_state_out) COTT_CUDA(launch_pad_state(seg.d_state_out, ds_out, BH, p.dk, p.dv, d, st));
                    f.state_in = seg.state_in ? s_in : nullptr;
                    f.d_state_out = seg.d_state_out ? ds_out : nullptr;
                    f.d_state_in = seg.d_state_in ? ds_in : nullptr;
                }
                COTT_CUDA(launch_tc_bwd_states(f, st0, st1, 1, B, H, N, st));
                COTT_CUDA(launch_tc_bwd_fused(f, B, H, N, st));
                if (p.padded && seg.d_state_in) COTT_CUDA(launch_unpad_state(ds_in, seg.d_state_in, BH, p.dk, p.dv, d, st));
                return COTT_OK;
            }
            if (causal && !packed.cu_seqlens && p.n_groups == 1 && N <= 128) {
                // One chunk per (b, h): no state is ever read, the walk is the only launch.
                f.sq_part = nullptr; f.r_part = nullptr;
                COTT_CUDA(cudaMemsetAsync(ws, 0, kWsHeaderBytes, st));      // status words and the dm counter
                f.plain_launch = 1;
                COTT_CUDA(launch_tc_bwd_fused(f, B, H, N, st));
                return COTT_OK;
            }
            if (!causal && p.n_groups == 1 && N <= 1024 && option_bidir_bwd() != 0) {
                // One group per (b, h) of at most 1024 tokens: both state totals, the three gradients and
                // dm in one launch (cott_tc_bidir_bwd.cu), nothing but q, k, v, dO read and dq, dk, dv
                // written.  (A CTA walks its sequence twice with two tile pairs in flight: beyond
                // eight chunks the two-launch form with its deeper rings is as fast or faster.)
                COTT_CUDA(cudaMemsetAsync(ws, 0, kWsHeaderBytes, st));      // status words and the dm counter
                COTT_CUDA(launch_tc_bidir_bwd(f, B, H, N, st));
                return COTT_OK;
            }
            COTT_CUDA(launch_tc_bwd_states(f, st0, st1, 1, B, H, N, st));
            COTT_CUDA(launch_tc_bwd_fused(f, B, H, N, st));
            return COTT_OK;
        }
        SideStreams* ss = nullptr;
        Plan pp = p;                       // plan of the two side-by-side streams
        // (d = 64 only: at d = 128 two such walks running at the same time once ended in launch
        // failures -- a transaction barrier of the raw-row tile was re-armed before its phase had
        // completed; it has one barrier per chunk parity since -- and the concurrent form has not
        // been switched on again there.)
        if (causal && !seg.on && d == 64 && p.n_groups >= 2 && 2 * BH <= 148 && 74 / BH == 1 && option_pair() != 0) {
            pp.group = (N + 127) / 128 * 128;
            pp.n_groups = 1; pp.split = 1;
            ss = side_streams();
        }
        // dQ^: forward walk with (dO, V, K^); c multiplies the accumulator; project with raw q
        TcWalkArgs tq = t;
        tq.x = d_o; tq.a = v; tq.bv = k; tq.proj = q; tq.out = dq;
        tq.norm_bv = 1; tq.x_norm = 0; tq.epilogue = EPI_PROJ; tq.reverse = 0;
        tq.clear_status = 1;             // the dQ^ stream is launched first (unless streams run side by side)
        // dK^: backward in time with (V, dO, Q^); project with raw k
        TcWalkArgs tk = t;
        tk.x = v; tk.a = d_o; tk.bv = q; tk.proj = k; tk.out = dk;
        tk.norm_bv = 1; tk.x_norm = 0; tk.epilogue = EPI_PROJ; tk.reverse = 1;
        // dV': backward in time with (K, Q^, dO); rows scale by c / ||k||; <dV', V> for dm
        TcWalkArgs tv = t;
        tv.x = k; tv.a = q; tv.bv = d_o; tv.proj = v; tv.out = dv;
        tv.norm_bv = 0; tv.x_norm = 1; tv.epilogue = EPI_DV; tv.reverse = 1;
        // dm: sum over rows of <dV'_j, v_j>, which equals the sum over rows of <q^_i, dQ^_i>.
        // The dQ^ stream forms the latter in its projection epilogue, so it carries the sum and
        // its last CTA finalises dm.
        tq.dm_partial = dm_partial;
        tq.dm_out = dm;
        lay.assign(tq); lay.assign(tk); lay.assign(tv);
        lay.assign_widths(tq); lay.assign_widths(tk); lay.assign_widths(tv);
        if (seg.on) {
            // A segment at head size 128 (cott_bwd_stateful) through the three walks.  Each stream's
            // running sum starts from what lies outside the segment, in that stream's layout and
            // scale (the walks divide an initial state by c, as they do with a caller's forward
            // state): the dQ^ stream from state_in^T, the dK^ stream from c d_state_out^T; the dV'
            // stream reuses the dK^ stream's scanned states (with one group, where nothing is
            // shared, it starts from c d_state_out).  The totals of the first two give
            // d_state_in and the two terms by which the dm sum over the query rows is off
            // (segment_finish_kernel); dm is finalised after that.
            char* sbase = base + 3 * sb + 2 * align_up((size_t)B * H * p.n_groups * 4, 256);
            const size_t ssb = segment_state_bytes(B, H, d);
            float* b_q = reinterpret_cast<float*>(sbase);
            float* b_k = reinterpret_cast<float*>(sbase + ssb);
            float* tk_tot = reinterpret_cast<float*>(sbase + 2 * ssb);
            float* tq_tot = st2;           // (the third states region is free: dV' has no state pass of its own)
            float* b_v = st0;              // (one group: no stream has a state pass, the regions are free)
            const bool one = p.n_groups == 1;
            // (smaller head sizes: the caller's states enter and leave through zero-padded copies)
            const float* s_in = seg.state_in; const float* ds_out = seg.d_state_out; float* ds_in = seg.d_state_in;
            if (p.padded) {
                float* pad = reinterpret_cast<float*>(sbase + 3 * ssb);
                if (seg.state_in) { COTT_CUDA(launch_pad_state(seg.state_in, pad, BH, p.dk, p.dv, d, st)); s_in = pad; }
                if (seg.d_state_out) { COTT_CUDA(launch_pad_state(seg.d_state_out, pad + ssb / 4, BH, p.dk, p.dv, d, st)); ds_out = pad + ssb / 4; }
                if (seg.d_state_in) ds_in = pad + 2 * (ssb / 4);
            }
            if (s_in)
                COTT_CUDA(launch_state_prep(s_in, b_q, BH, d, 1, 0, sp->m, sp->seq_len, sp->seq_len_scalar, H, N, st));
            if (ds_out) {
                COTT_CUDA(launch_state_prep(ds_out, b_k, BH, d, 1, 1, sp->m, sp->seq_len, sp->seq_len_scalar, H, N, st));
                if (one) COTT_CUDA(launch_state_prep(ds_out, b_v, BH, d, 0, 1, sp->m, sp->seq_len, sp->seq_len_scalar, H, N, st));
            }
            tk.clear_status = 1; tq.clear_status = 0;
            tk.dm_partial = dm_partial2; tk.dm_out = nullptr;
            tq.dm_partial = dm_partial; tq.dm_out = nullptr; tq.dm_extra = nullptr;
            if ((rc = run_tc_stream(tk, p, B, H, N, d, causal, sp, status, st1, tk_tot, st, false, false, true,
                                    seg.d_state_out ? b_k : nullptr)) != COTT_OK) return rc;
            if ((rc = run_tc_stream(tq, p, B, H, N, d, causal, sp, status, one ? st1 : st0, tq_tot, st, false, false, true,
                                    seg.state_in ? b_q : nullptr)) != COTT_OK) return rc;
            if (one) {
                if ((rc = run_tc_stream(tv, p, B, H, N, d, causal, sp, status, st1, nullptr, st, false, false, true,
                                        seg.d_state_out ? b_v : nullptr)) != COTT_OK) return rc;
            } else {
                // (the states were scanned by the dK^ stream's scan launch: the non-null last
                // argument keeps this call from summing them itself)
                if ((rc = run_tc_stream(tv, p, B, H, N, d, causal, sp, status, st1, nullptr, st, true, false, true, b_k)) != COTT_OK)
                    return rc;
            }
            COTT_CUDA(launch_segment_finish(s_in, ds_out, tq_tot, tk_tot, ds_in, dm_partial, dm_partial2,
                                            BH, p.n_groups, d, sp->m, sp->seq_len, sp->seq_len_scalar, H, N, st));
            if (p.padded && seg.d_state_in) COTT_CUDA(launch_unpad_state(ds_in, seg.d_state_in, BH, p.dk, p.dv, d, st));
            COTT_CUDA(launch_dm_finalize(dm_partial, dm, sp->m, sp->seq_len, sp->seq_len_scalar, B, H, p.n_groups, N, st, nullptr));
            return COTT_OK;
        }
        if (ss) {
            struct TagScope { ~TagScope() { g_prof_cur_tag = 0; } } tag_scope;
            // Everything that follows a cross-stream event wait is a plain launch.
            tk.plain_launch = 1; tv.plain_launch = 1;
            // The first kernel of the call is a plain launch too: started early behind the
            // caller's previous kernel it only holds SMs that the side streams could use
            // (measured: 177 us against 194 us per forward+backward step issued back to back).
            tq.plain_launch = 1;
            g_prof_cur_tag = g_prof_next_tag.fetch_add(1);
            COTT_CUDA(cudaEventRecord(ss->fork, st));
            COTT_CUDA(cudaStreamWaitEvent(ss->s[0], ss->fork, 0));
            COTT_CUDA(cudaStreamWaitEvent(ss->s[1], ss->fork, 0));
            // The two streams that run backward in time go side by side: their CTAs of one
            // (b, h) ask for the same q, k, v, dO tiles at about the same time, so the second
            // request is served by L2 (measured: 114 us against 124 us for the dQ^ / dK^ pair).
            // The dQ^ stream (forward in time) keeps its groups: its state pass fills the spare
            // SMs meanwhile, its walk follows on the whole GPU.
            tk.clear_status = 1; tq.clear_status = 0;
            if ((rc = run_tc_stream(tk, pp, B, H, N, d, causal, sp, status, st1, nullptr, st)) != COTT_OK) return rc;
            if ((rc = run_tc_stream(tv, pp, B, H, N, d, causal, sp, status, st2, nullptr, ss->s[0])) != COTT_OK) return rc;
            g_prof_cur_tag = 0;
            if ((rc = run_tc_stream(tq, p, B, H, N, d, causal, sp, status, st0, nullptr, ss->s[1], false, true)) != COTT_OK) return rc;
            COTT_CUDA(cudaEventRecord(ss->join[0], ss->s[0]));
            COTT_CUDA(cudaEventRecord(ss->join[1], ss->s[1]));
            COTT_CUDA(cudaStreamWaitEvent(st, ss->join[0], 0));
            COTT_CUDA(cudaStreamWaitEvent(st, ss->join[1], 0));
            if ((rc = run_tc_stream(tq, p, B, H, N, d, causal, sp, status, st0, nullptr, st, true, false, false)) != COTT_OK) return rc;
        } else {
            // The dK^ stream goes first: it also sums the first-order term by which the dQ^
            // stream's dm sum is off because that stream multiplies by k^ rounded to bf16; the
            // dQ^ stream, second, adds the two parts when it finalises dm.
            tk.clear_status = 1; tq.clear_status = 0;
            tk.dm_partial = dm_partial2; tk.dm_out = nullptr;
            tq.dm_extra = dm_partial2;
            if ((rc = run_tc_stream(tk, p, B, H, N, d, causal, sp, status, st1, nullptr, st)) != COTT_OK) return rc;
            if ((rc = run_tc_stream(tq, p, B, H, N, d, causal, sp, status, st0, nullptr, st)) != COTT_OK) return rc;
            // The dV' state sum_t q^_t dO_t^T is the transpose of the dK^ stream's
            // sum_t dO_t q^_t^T, accumulated in the same direction: reuse those group states
            // instead of a third pass.
            if ((rc = run_tc_stream(tv, p, B, H, N, d, causal, sp, status, st1, nullptr, st, true)) != COTT_OK) return rc;
        }
        return COTT_OK;
    }
    // A segment of a longer sequence (cott_bwd_stateful): every stream's running sum starts from
    // what lies outside the segment.  The dQ^ stream's sum is the caller's state transposed (these
    // states contain c, as the caller's does), the dK^ stream's the transposed gradient of the
    // outgoing state, the dV' stream's that gradient itself -- and its total is the gradient of
    // the incoming state.  dm is summed over the value rows here, which is what a segment needs.
    const float* seg_q = nullptr; const float* seg_k = nullptr; const float* seg_v = nullptr;
    float* seg_total = nullptr;
    if (seg.on) {
        char* sbase = base + 3 * sb + 2 * align_up((size_t)B * H * p.n_groups * 4, 256);
        const size_t ssb = segment_state_bytes(B, H, d);
        if (seg.state_in) {
            float* tbuf = reinterpret_cast<float*>(sbase);
            COTT_CUDA(launch_transpose_state(seg.state_in, tbuf, BH, d, st));
            seg_q = tbuf;
        }
        if (seg.d_state_out) {
            float* tbuf = reinterpret_cast<float*>(sbase + ssb);
            COTT_CUDA(launch_transpose_state(seg.d_state_out, tbuf, BH, d, st));
            seg_k = tbuf;
            seg_v = seg.d_state_out;
        }
        seg_total = seg.d_state_in;
    }
    {   // dQ^_t = S_t dO_t : the forward walk with (dO, V', K^) in the roles of (Q, K, V)
        WalkArgs w = base_walk(sp, H, N, p);
        w.x = d_o; w.a = v; w.bv = k; w.proj = q; w.out = dq;
        w.cu_seqlens = packed.cu_seqlens;
        lay.assign(w);
        w.mode_x = ROW_RAW; w.mode_a = ROW_SCALE; w.mode_b = ROW_NORM;
        w.epilogue = EPI_PROJ; w.reverse = 0;
        if ((rc = run_stream(w, p, BH, d, dt, causal, st0, nullptr, st, seg_q)) != COTT_OK) return rc;
    }
    {   // dK^_j = R_j v'_j : running sum of dO_t q^_t^T accumulated backward in time
        WalkArgs w = base_walk(sp, H, N, p);
        w.x = v; w.a = d_o; w.bv = q; w.proj = k; w.out = dk;
        w.cu_seqlens = packed.cu_seqlens;
        lay.assign(w);
        w.mode_x = ROW_SCALE; w.mode_a = ROW_RAW; w.mode_b = ROW_NORM;
        w.epilogue = EPI_PROJ; w.reverse = 1;
        if ((rc = run_stream(w, p, BH, d, dt, causal, st1, nullptr, st, seg_k)) != COTT_OK) return rc;
    }
    {   // dV'_j = R_j^T k^_j, dV = c dV', and <dV', V> for dm
        WalkArgs w = base_walk(sp, H, N, p);
        w.x = k; w.a = q; w.bv = d_o; w.proj = v; w.out = dv;
        w.cu_seqlens = packed.cu_seqlens;
        lay.assign(w);
        w.mode_x = ROW_NORM; w.mode_a = ROW_NORM; w.mode_b = ROW_RAW;
        w.epilogue = EPI_DV; w.reverse = 1; w.dm_partial = dm_partial;
        if ((rc = run_stream(w, p, BH, d, dt, causal, st2, seg_total, st, seg_v)) != COTT_OK) return rc;
    }
    COTT_CUDA(launch_dm_finalize(dm_partial, dm, sp->m, sp->seq_len, sp->seq_len_scalar, B, H,
                                 p.n_groups, N, st, packed.cu_seqlens));
    return COTT_OK;
}

}  // namespace cott

using namespace cott;

extern "C" {

int cott_version(void) { return 100; }

const char* cott_status_string(cott_status st) {
    switch (st) {
        case COTT_OK: return "ok";
        case COTT_ERR_INVALID_ARG: return "invalid argument";
        case COTT_ERR_UNSUPPORTED: return "unsupported shape, dtype or alignment";
        case COTT_ERR_WORKSPACE: return "workspace missing or too small";
        case COTT_ERR_CUDA: return "CUDA error";
        case COTT_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

const char* cott_last_cuda_error(void) { return g_cuda_error; }

cott_status cott_profile_enable(int max_launches) {
    if (max_launches <= 0) { g_prof_n.store(-1); return COTT_OK; }
    if (!g_prof_created) {
        for (int i = 0; i < 2 * kProfMax; ++i)
            if (cudaEventCreate(&g_prof_ev[i]) != cudaSuccess) return COTT_ERR_CUDA;
        g_prof_created = true;
    }
    g_prof_cap = max_launches < kProfMax ? max_launches : kProfMax;
    g_prof_n.store(0);
    return COTT_OK;
}

int cott_profile_read(float* ms, int* kinds, int cap) {
    int n = g_prof_n.load();
    if (n < 0) return 0;
    if (n > g_prof_cap) n = g_prof_cap;
    if (n > cap) n = cap;
    for (int i = 0; i < n; ++i)
        if (cudaEventSynchronize(g_prof_ev[2 * i + 1]) != cudaSuccess) return -1;
    for (int i = 0; i < n; ++i) {
        if (cudaEventElapsedTime(&ms[i], g_prof_ev[2 * i], g_prof_ev[2 * i + 1]) != cudaSuccess) return -1;
        kinds[i] = g_prof_kind[i];
        if (g_prof_tag[i] == 0 || g_prof_kind[i] != 1) continue;
        // A causal walk that ran side by side with a sibling walk of the same size: report
        // half of the span the pair occupied (first start to last end).
        for (int j = 0; j < n; ++j) {
            if (j == i || g_prof_tag[j] != g_prof_tag[i] || g_prof_kind[j] != 1) continue;
            float span = ms[i], t;
            if (cudaEventElapsedTime(&t, g_prof_ev[2 * j], g_prof_ev[2 * j + 1]) == cudaSuccess && t > span) span = t;
            if (cudaEventElapsedTime(&t, g_prof_ev[2 * i], g_prof_ev[2 * j + 1]) == cudaSuccess && t > span) span = t;
            if (cudaEventElapsedTime(&t, g_prof_ev[2 * j], g_prof_ev[2 * i + 1]) == cudaSuccess && t > span) span = t;
            ms[i] = 0.5f * span;
            kinds[i] = g_prof_kind[i] | 16;
            break;
        }
    }
    return n;
}

cott_status cott_set_option(const char* name, long long value) {
    if (!name) return COTT_ERR_INVALID_ARG;
    for (Option* o : g_options)
        if (strcmp(o->name, name) == 0) { o->set(value); return COTT_OK; }
    return COTT_ERR_INVALID_ARG;
}

long long cott_get_option(const char* name) {
    if (!name) return -1;
    for (Option* o : g_options)
        if (strcmp(o->name, name) == 0) return o->get();
    return -1;
}

unsigned long long cott_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t cott_workspace_bytes_dkdv(int op, cott_dtype dt, int B, int H, int N, int d_k, int d_v, int causal) {
    if (op == COTT_OP_DECODE) return 0;
    if (op != COTT_OP_FWD && op != COTT_OP_BWD) return (size_t)-1;
    Plan p;
    if (!make_plan(op, dt, B, H, N, d_k, d_v, causal, &p)) return (size_t)-1;
    return workspace_bytes_impl(op, p, B, H, p.d);
}

static bool varlen_plan(int op, cott_dtype dt, int B, int H, int total_tokens, int max_seqlen, int d, int causal, Plan* p,
                        size_t room);

size_t cott_workspace_bytes_varlen(int op, cott_dtype dt, int B, int H, int total_tokens, int max_seqlen, int d, int causal) {
    if (op != COTT_OP_FWD && op != COTT_OP_BWD) return (size_t)-1;
    Plan coarse, fine;
    if (!varlen_plan(op, dt, B, H, total_tokens, max_seqlen, d, causal, &coarse, 0)) return (size_t)-1;
    if (!varlen_plan(op, dt, B, H, total_tokens, max_seqlen, d, causal, &fine, (size_t)-1)) return (size_t)-1;
    const size_t a = workspace_bytes_impl(op, coarse, B, H, coarse.d), b = workspace_bytes_impl(op, fine, B, H, fine.d);
    return a > b ? a : b;
}

size_t cott_workspace_bytes(int op, cott_dtype dt, int B, int H, int N, int d, int causal) {
    return cott_workspace_bytes_dkdv(op, dt, B, H, N, d, d, causal);
}

cott_status cott_query_plan_dkdv(int op, cott_dtype dt, int B, int H, int N, int d_k, int d_v, int causal,
                                 int* path, int* group, int* chunk, int* kernel_d) {
    Plan p;
    if (op == COTT_OP_DECODE) { p.path = 0; p.group = 1; p.chunk = 1; p.d = d_k > d_v ? d_k : d_v; }
    else if (!make_plan(op, dt, B, H, N, d_k, d_v, causal, &p)) return COTT_ERR_UNSUPPORTED;
    if (path) *path = p.path;
    if (group) *group = p.group;
    if (chunk) *chunk = p.chunk;
    if (kernel_d) *kernel_d = p.d;
    return COTT_OK;
}

cott_status cott_query_plan(int op, cott_dtype dt, int B, int H, int N, int d, int causal,
                            int* path, int* group, int* chunk) {
    return cott_query_plan_dkdv(op, dt, B, H, N, d, d, causal, path, group, chunk, nullptr);
}

// Validation and dispatch shared by every dense / strided forward entry point.
static cott_status fwd_entry(const void* q, const void* k, const void* v, void* o, const float* state_in,
                             float* state_out, int B, int H, int N, int d_k, int d_v, int causal, bool stateful,
                             cott_dtype dt, const cott_strides* qk_strides, const cott_strides* v_strides,
                             const cott_strides* o_strides, const cott_scale_params* sp, void* workspace,
                             size_t workspace_bytes, void* stream) {
    if (!q || !k || !v || !o || B < 1 || H < 1 || N < 1 || d_k < 1 || d_v < 1) return COTT_ERR_INVALID_ARG;
    const cott_strides* vs = v_strides ? v_strides : (d_k == d_v ? qk_strides : nullptr);
    if (!layout_ok(qk_strides, d_k, dt) || !layout_ok(vs, d_v, dt) || !layout_ok(o_strides, d_v, dt))
        return COTT_ERR_UNSUPPORTED;
    if (check_scale(sp) != COTT_OK) return COTT_ERR_INVALID_ARG;
    if (tensors_overlap(o, o_strides, q, qk_strides, B, H, N, d_v, dt, d_k) ||
        tensors_overlap(o, o_strides, k, qk_strides, B, H, N, d_v, dt, d_k) ||
        tensors_overlap(o, o_strides, v, vs, B, H, N, d_v, dt, d_v))
        return COTT_ERR_INVALID_ARG;
    if (stateful) {
        if (!causal) return COTT_ERR_INVALID_ARG;
        if (state_in && state_in == state_out) return COTT_ERR_INVALID_ARG;
        // the scaling base must be the caller's (the same for every segment of a sequence)
        if (!sp->seq_len && !(sp->seq_len_scalar >= 1.f)) return COTT_ERR_INVALID_ARG;
    } else {
        if (state_in) return COTT_ERR_INVALID_ARG;
        if (!sp->seq_len && sp->seq_len_scalar > 0.f && sp->seq_len_scalar < 1.f) return COTT_ERR_INVALID_ARG;
    }
    Plan p;
    if (!make_plan(COTT_OP_FWD, dt, B, H, N, d_k, d_v, causal, &p)) return COTT_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) ||
        (state_in && !aligned16(state_in)) || (state_out && !aligned16(state_out)))
        return COTT_ERR_UNSUPPORTED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < workspace_bytes_impl(COTT_OP_FWD, p, B, H, p.d))
        return COTT_ERR_WORKSPACE;
    return fwd_impl(q, k, v, o, state_out, B, H, N, p.d, causal, dt, sp, workspace, p,
                    static_cast<cudaStream_t>(stream), state_in, qk_strides, o_strides, Packed(),
                    (d_k != d_v || v_strides) ? vs : nullptr);
}

cott_status cott_fwd(const void* q, const void* k, const void* v, void* o, float* state_out,
                     int B, int H, int N, int d, int causal, cott_dtype dt,
                     const cott_scale_params* sp, void* workspace, size_t workspace_bytes,
                     void* stream) {
    return fwd_entry(q, k, v, o, nullptr, state_out, B, H, N, d, d, causal, false, dt, nullptr, nullptr, nullptr, sp,
                     workspace, workspace_bytes, stream);
}

cott_status cott_fwd_strided(const void* q, const void* k, const void* v, void* o, float* state_out,
                             int B, int H, int N, int d, int causal, cott_dtype dt,
                             const cott_strides* qkv_strides, const cott_strides* o_strides,
                             const cott_scale_params* sp, void* workspace, size_t workspace_bytes,
                             void* stream) {
    return fwd_entry(q, k, v, o, nullptr, state_out, B, H, N, d, d, causal, false, dt, qkv_strides, nullptr, o_strides,
                     sp, workspace, workspace_bytes, stream);
}

cott_status cott_fwd_stateful(const void* q, const void* k, const void* v, void* o,
                              const float* state_in, float* state_out, int B, int H, int N, int d,
                              cott_dtype dt, const cott_scale_params* sp, void* workspace,
                              size_t workspace_bytes, void* stream) {
    return fwd_entry(q, k, v, o, state_in, state_out, B, H, N, d, d, 1, true, dt, nullptr, nullptr, nullptr, sp,
                     workspace, workspace_bytes, stream);
}

cott_status cott_fwd_stateful_strided(const void* q, const void* k, const void* v, void* o,
                                      const float* state_in, float* state_out, int B, int H, int N,
                                      int d, cott_dtype dt, const cott_strides* qkv_strides,
                                      const cott_strides* o_strides, const cott_scale_params* sp,
                                      void* workspace, size_t workspace_bytes, void* stream) {
    return fwd_entry(q, k, v, o, state_in, state_out, B, H, N, d, d, 1, true, dt, qkv_strides, nullptr, o_strides, sp,
                     workspace, workspace_bytes, stream);
}

cott_status cott_fwd_dkdv(const void* q, const void* k, const void* v, void* o, const float* state_in,
                          float* state_out, int B, int H, int N, int d_k, int d_v, int causal, cott_dtype dt,
                          const cott_strides* qk_strides, const cott_strides* v_strides,
                          const cott_strides* o_strides, const cott_scale_params* sp, void* workspace,
                          size_t workspace_bytes, void* stream) {
    return fwd_entry(q, k, v, o, state_in, state_out, B, H, N, d_k, d_v, causal, state_in != nullptr, dt, qk_strides,
                     v_strides, o_strides, sp, workspace, workspace_bytes, stream);
}

// Validation and dispatch shared by every dense / strided backward entry point.
static cott_status bwd_entry(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk,
                             void* dv, float* dm, int B, int H, int N, int d_k, int d_v, int causal, cott_dtype dt,
                             const cott_strides* qk_strides, const cott_strides* v_strides,
                             const cott_strides* do_strides, const cott_strides* dqk_strides,
                             const cott_strides* dv_strides, const cott_scale_params* sp, void* workspace,
                             size_t workspace_bytes, void* stream, const void* fwd_workspace = nullptr,
                             Segment seg = Segment()) {
    if (!q || !k || !v || !d_o || !dq || !dk || !dv || !dm || B < 1 || H < 1 || N < 1 || d_k < 1 || d_v < 1)
        return COTT_ERR_INVALID_ARG;
    if (fwd_workspace && (fwd_workspace == workspace || (reinterpret_cast<uintptr_t>(fwd_workspace) & 255u)))
        return COTT_ERR_INVALID_ARG;
    const bool same = d_k == d_v;
    const cott_strides* vs = v_strides ? v_strides : (same ? qk_strides : nullptr);
    const cott_strides* dvs = dv_strides ? dv_strides : (same ? dqk_strides : nullptr);
    if (!layout_ok(qk_strides, d_k, dt) || !layout_ok(vs, d_v, dt) || !layout_ok(do_strides, d_v, dt) ||
        !layout_ok(dqk_strides, d_k, dt) || !layout_ok(dvs, d_v, dt))
        return COTT_ERR_UNSUPPORTED;
    if (check_scale(sp) != COTT_OK) return COTT_ERR_INVALID_ARG;
    {
        const void* ins[4] = {q, k, v, d_o};
        const cott_strides* in_st[4] = {qk_strides, qk_strides, vs, do_strides};
        const int in_d[4] = {d_k, d_k, d_v, d_v};
        void* outs[3] = {dq, dk, dv};
        const cott_strides* out_st[3] = {dqk_strides, dqk_strides, dvs};
        const int out_d[3] = {d_k, d_k, d_v};
        for (int i = 0; i < 3; ++i) {
            for (int j = 0; j < 4; ++j)
                if (tensors_overlap(outs[i], out_st[i], ins[j], in_st[j], B, H, N, out_d[i], dt, in_d[j])) return COTT_ERR_INVALID_ARG;
            for (int j = i + 1; j < 3; ++j)
                if (tensors_overlap(outs[i], out_st[i], outs[j], out_st[j], B, H, N, out_d[i], dt, out_d[j])) return COTT_ERR_INVALID_ARG;
        }
    }
    if (!sp->seq_len && sp->seq_len_scalar > 0.f && sp->seq_len_scalar < 1.f)
        return COTT_ERR_INVALID_ARG;
    Plan p;
    if (!make_plan(COTT_OP_BWD, dt, B, H, N, d_k, d_v, causal, &p)) return COTT_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(d_o) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return COTT_ERR_UNSUPPORTED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < workspace_bytes_impl(COTT_OP_BWD, p, B, H, p.d))
        return COTT_ERR_WORKSPACE;
    const bool own_v = !same || v_strides || dv_strides;
    if (seg.on) {
        // A segment needs the caller's scaling base (the same for every segment of a sequence), is
        // causal, and runs through the one-walk backward of the tensor-core path at sizes up to 64.
        if (!causal || (!sp->seq_len && !(sp->seq_len_scalar >= 1.f))) return COTT_ERR_INVALID_ARG;
        // Tensor cores: the one-walk backward at sizes up to 64, the three walks at 128.  Everything
        // else the fp32-accumulating kernels cover (equal key and value sizes of 32, 64 or 128) goes
        // through them, with the groups of the plan as it stands (the workspace was sized for it).
        const bool tc_fused = p.path == 1 && p.d == 64 && option_fused_bwd() != 0;
        const bool tc_walks = p.path == 1 && p.d == 128;
        if (p.path == 1 && !tc_fused && !tc_walks) {
            if (!(d_k == d_v && (d_k == 32 || d_k == 64 || d_k == 128))) return COTT_ERR_UNSUPPORTED;
            p.path = 0; p.chunk = 16; p.d = d_k; p.padded = false; p.split = 1;
        }
        if ((seg.state_in && !aligned16(seg.state_in)) || (seg.d_state_out && !aligned16(seg.d_state_out)) ||
            (seg.d_state_in && !aligned16(seg.d_state_in)))
            return COTT_ERR_UNSUPPORTED;
        if (seg.d_state_in && (seg.d_state_in == seg.state_in || seg.d_state_in == seg.d_state_out)) return COTT_ERR_INVALID_ARG;
    }
    return bwd_impl(q, k, v, d_o, dq, dk, dv, dm, B, H, N, p.d, causal, dt, sp, workspace, p,
                    static_cast<cudaStream_t>(stream), qk_strides, do_strides, dqk_strides, Packed(),
                    own_v ? vs : nullptr, own_v ? dvs : nullptr, fwd_workspace, seg);
}

cott_status cott_bwd_stateful_strided(const void* q, const void* k, const void* v, const void* d_o,
                                      const float* state_in, const float* d_state_out, void* dq, void* dk, void* dv,
                                      float* d_state_in, float* dm, int B, int H, int N, int d_k, int d_v, cott_dtype dt,
                                      const cott_strides* qk_strides, const cott_strides* v_strides,
                                      const cott_strides* do_strides, const cott_strides* dqk_strides,
                                      const cott_strides* dv_strides, const cott_scale_params* sp, void* workspace,
                                      size_t workspace_bytes, void* stream) {
    Segment seg;
    seg.on = true; seg.state_in = state_in; seg.d_state_out = d_state_out; seg.d_state_in = d_state_in;
    return bwd_entry(q, k, v, d_o, dq, dk, dv, dm, B, H, N, d_k, d_v, 1, dt, qk_strides, v_strides, do_strides, dqk_strides,
                     dv_strides, sp, workspace, workspace_bytes, stream, nullptr, seg);
}

cott_status cott_bwd_stateful(const void* q, const void* k, const void* v, const void* d_o,
                              const float* state_in, const float* d_state_out, void* dq, void* dk, void* dv,
                              float* d_state_in, float* dm, int B, int H, int N, int d_k, int d_v, cott_dtype dt,
                              const cott_scale_params* sp, void* workspace, size_t workspace_bytes, void* stream) {
    return cott_bwd_stateful_strided(q, k, v, d_o, state_in, d_state_out, dq, dk, dv, d_state_in, dm, B, H, N, d_k, d_v, dt,
                                     nullptr, nullptr, nullptr, nullptr, nullptr, sp, workspace, workspace_bytes, stream);
}

cott_status cott_bwd_after_fwd(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                               void* dk, void* dv, float* dm, int B, int H, int N, int d, int causal,
                               cott_dtype dt, const cott_strides* qkv_strides,
                               const cott_strides* do_strides, const cott_strides* dqkv_strides,
                               const cott_scale_params* sp, const void* fwd_workspace, void* workspace,
                               size_t workspace_bytes, void* stream) {
    return bwd_entry(q, k, v, d_o, dq, dk, dv, dm, B, H, N, d, d, causal, dt, qkv_strides, nullptr, do_strides,
                     dqkv_strides, nullptr, sp, workspace, workspace_bytes, stream, fwd_workspace);
}

cott_status cott_bwd(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                     void* dk, void* dv, float* dm, int B, int H, int N, int d, int causal,
                     cott_dtype dt, const cott_scale_params* sp, void* workspace,
                     size_t workspace_bytes, void* stream) {
    return bwd_entry(q, k, v, d_o, dq, dk, dv, dm, B, H, N, d, d, causal, dt, nullptr, nullptr, nullptr, nullptr,
                     nullptr, sp, workspace, workspace_bytes, stream);
}

cott_status cott_bwd_strided(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                             void* dk, void* dv, float* dm, int B, int H, int N, int d, int causal,
                             cott_dtype dt, const cott_strides* qkv_strides,
                             const cott_strides* do_strides, const cott_strides* dqkv_strides,
                             const cott_scale_params* sp, void* workspace, size_t workspace_bytes,
                             void* stream) {
    return bwd_entry(q, k, v, d_o, dq, dk, dv, dm, B, H, N, d, d, causal, dt, qkv_strides, nullptr, do_strides,
                     dqkv_strides, nullptr, sp, workspace, workspace_bytes, stream);
}

cott_status cott_bwd_dkdv(const void* q, const void* k, const void* v, const void* d_o, void* dq, void* dk,
                          void* dv, float* dm, int B, int H, int N, int d_k, int d_v, int causal, cott_dtype dt,
                          const cott_strides* qk_strides, const cott_strides* v_strides,
                          const cott_strides* do_strides, const cott_strides* dqk_strides,
                          const cott_strides* dv_strides, const cott_scale_params* sp, void* workspace,
                          size_t workspace_bytes, void* stream) {
    return bwd_entry(q, k, v, d_o, dq, dk, dv, dm, B, H, N, d_k, d_v, causal, dt, qk_strides, v_strides, do_strides,
                     dqk_strides, dv_strides, sp, workspace, workspace_bytes, stream);
}

// Plan of a packed batch.
// `room`: bytes of workspace the caller has (0: the plan that the dense workspace query covers).
static bool varlen_plan(int op, cott_dtype dt, int B, int H, int total_tokens, int max_seqlen, int d, int causal, Plan* p,
                        size_t room) {
    if (B < 1 || H < 1 || total_tokens < 1 || max_seqlen < 1 || max_seqlen > total_tokens) return false;
    // bf16, tensor cores: any head size that is a multiple of 8 up to 128 (zero-filled tiles);
    // fp32 (and bf16 with force_path = 0): the fp32-accumulating SIMT kernels at 32, 64, 128
    const bool tc_ok = dt == COTT_BF16 && d >= 8 && d <= 128 && d % 8 == 0;
    const bool simt_ok = (dt == COTT_F32 || dt == COTT_BF16) && (d == 32 || d == 64 || d == 128);
    if (!tc_ok && !simt_ok) return false;
    p->path = (tc_ok && (option_force_path() != 0 || !simt_ok)) ? 1 : 0;
    p->chunk = p->path == 1 ? 128 : 16;
    p->group = (max_seqlen + p->chunk - 1) / p->chunk * p->chunk; p->n_groups = 1; p->split = 1;
    p->dk = p->dv = d; p->d = p->path == 1 ? (d <= 64 ? 64 : 128) : d; p->padded = p->d != d;
    if (p->path == 1) {
        // Tensor cores: the groups of the dense plan for sequences of max_seqlen tokens -- group g
        // of a sequence is its rows g * group .. + group - 1, as far as they exist -- so that a
        // batch of few long sequences still fills the GPU.  (No finer partition for the state pass.)
        Plan dense;
        if (!make_plan(op, dt, B, H, max_seqlen, d, d, causal, &dense) || dense.path != 1) return false;
        p->group = dense.group; p->n_groups = dense.n_groups;
        // That plan sizes the groups as if every sequence had max_seqlen tokens.  The lengths are on
        // the device, but their sum is known: about total / G + B groups per head exist, and one
        // wave holds 148 / H of them -- a smaller G when the batch is skewed (a few long sequences
        // among short ones), as long as the caller's workspace has room for the states of
        // max_seqlen / G groups per sequence (cott_workspace_bytes_varlen asks for it).
        const long per_head = 148 / H - B;
        if (option_force_group() <= 0 && per_head >= 1) {
            long g = ((long)total_tokens + per_head - 1) / per_head;
            g = (g + 127) / 128 * 128;
            if (g < p->group) {
                Plan fine = *p;
                fine.group = (int)g; fine.n_groups = (max_seqlen + fine.group - 1) / fine.group;
                if (room == (size_t)-1 || workspace_bytes_impl(op, fine, B, H, fine.d) <= room) *p = fine;
            }
        }
    }
    return true;
}

cott_status cott_fwd_varlen(const void* q, const void* k, const void* v, void* o,
                            const int* cu_seqlens, int B, int H, int total_tokens, int max_seqlen,
                            int d, int causal, cott_dtype dt, const cott_scale_params* sp,
                            void* workspace, size_t workspace_bytes, void* stream) {
    if (!q || !k || !v || !o || !cu_seqlens) return COTT_ERR_INVALID_ARG;
    if (check_scale(sp) != COTT_OK) return COTT_ERR_INVALID_ARG;
    if (o == q || o == k || o == v) return COTT_ERR_INVALID_ARG;
    if (!sp->seq_len && sp->seq_len_scalar > 0.f && sp->seq_len_scalar < 1.f) return COTT_ERR_INVALID_ARG;
    Plan p;
    if (!varlen_plan(COTT_OP_FWD, dt, B, H, total_tokens, max_seqlen, d, causal, &p, workspace ? workspace_bytes : 0)) return COTT_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return COTT_ERR_UNSUPPORTED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < workspace_bytes_impl(COTT_OP_FWD, p, B, H, p.d))
        return COTT_ERR_WORKSPACE;
    // rows of all sequences back to back, [total_tokens, H, d]
    const cott_strides packed_l = {(long long)total_tokens * H * d, (long long)d, (long long)H * d};
    Packed pk; pk.cu_seqlens = cu_seqlens; pk.total_tokens = total_tokens;
    return fwd_impl(q, k, v, o, nullptr, B, H, max_seqlen, p.d, causal, dt, sp, workspace, p,
                    static_cast<cudaStream_t>(stream), nullptr, &packed_l, &packed_l, pk);
}

cott_status cott_bwd_varlen(const void* q, const void* k, const void* v, const void* d_o, void* dq,
                            void* dk, void* dv, float* dm, const int* cu_seqlens, int B, int H,
                            int total_tokens, int max_seqlen, int d, int causal, cott_dtype dt,
                            const cott_scale_params* sp, void* workspace, size_t workspace_bytes,
                            void* stream) {
    if (!q || !k || !v || !d_o || !dq || !dk || !dv || !dm || !cu_seqlens) return COTT_ERR_INVALID_ARG;
    if (check_scale(sp) != COTT_OK) return COTT_ERR_INVALID_ARG;
    const void* ins[4] = {q, k, v, d_o};
    void* outs[3] = {dq, dk, dv};
    for (int i = 0; i < 3; ++i) {
        for (int j = 0; j < 4; ++j)
            if (outs[i] == ins[j]) return COTT_ERR_INVALID_ARG;
        for (int j = i + 1; j < 3; ++j)
            if (outs[i] == outs[j]) return COTT_ERR_INVALID_ARG;
    }
    if (!sp->seq_len && sp->seq_len_scalar > 0.f && sp->seq_len_scalar < 1.f) return COTT_ERR_INVALID_ARG;
    Plan p;
    if (!varlen_plan(COTT_OP_BWD, dt, B, H, total_tokens, max_seqlen, d, causal, &p, workspace ? workspace_bytes : 0)) return COTT_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(d_o) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return COTT_ERR_UNSUPPORTED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < workspace_bytes_impl(COTT_OP_BWD, p, B, H, p.d))
        return COTT_ERR_WORKSPACE;
    const cott_strides packed_l = {(long long)total_tokens * H * d, (long long)d, (long long)H * d};
    Packed pk; pk.cu_seqlens = cu_seqlens; pk.total_tokens = total_tokens;
    return bwd_impl(q, k, v, d_o, dq, dk, dv, dm, B, H, max_seqlen, p.d, causal, dt, sp, workspace, p,
                    static_cast<cudaStream_t>(stream), &packed_l, &packed_l, &packed_l, pk);
}

cott_status cott_decode_step_dkdv(const void* q, const void* k, const void* v, float* state, void* o,
                                  int B, int H, int d_k, int d_v, cott_dtype dt, const cott_scale_params* sp,
                                  void* stream) {
    if (!q || !k || !v || !state || !o || B < 1 || H < 1 || d_k < 1 || d_v < 1) return COTT_ERR_INVALID_ARG;
    if (check_scale(sp) != COTT_OK) return COTT_ERR_INVALID_ARG;
    if (!sp->seq_len && !(sp->seq_len_scalar >= 1.f)) return COTT_ERR_INVALID_ARG;
    if (dt != COTT_F32 && dt != COTT_BF16) return COTT_ERR_UNSUPPORTED;
    const bool tuned = d_k == d_v && (d_k == 32 || d_k == 64 || d_k == 128);
    // other sizes: rows of 16 bytes at least (as in the forward), at most 1024 columns
    const int q16 = 16 / (int)dtype_size(dt);
    if (!tuned && (d_k % q16 != 0 || d_v % q16 != 0 || d_k > 1024 || d_v > 1024)) return COTT_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(state) || !aligned16(o))
        return COTT_ERR_UNSUPPORTED;
    if (tuned)
        COTT_CUDA(launch_decode(q, k, v, state, o, B, H, d_k, dt, sp->m, sp->seq_len,
                                sp->seq_len_scalar, static_cast<cudaStream_t>(stream)));
    else
        COTT_CUDA(launch_decode_generic(q, k, v, state, o, B, H, d_k, d_v, dt, sp->m, sp->seq_len,
                                        sp->seq_len_scalar, static_cast<cudaStream_t>(stream)));
    return COTT_OK;
}

cott_status cott_decode_step(const void* q, const void* k, const void* v, float* state, void* o,
                             int B, int H, int d, cott_dtype dt, const cott_scale_params* sp,
                             void* stream) {
    return cott_decode_step_dkdv(q, k, v, state, o, B, H, d, d, dt, sp, stream);
}

// The host-buffer training step cuts the batch into at most kHostSlices slices that are
// contiguous in [B,H,N,d]: several whole batch items each, or -- when the batch is small -- a
// batch item's heads in equal groups.
struct HostSlicing {
    int items;     // batch items per slice (head_groups == 1)
    int heads;     // heads per slice
    int n;         // number of slices
};
static HostSlicing host_step_slicing(int B, int H) {
    HostSlicing s;
    long long want = g_opt_host_slices.get();
    const int max_slices = (int)(want < 1 ? 1 : (want > kHostSlices ? kHostSlices : want));
    if (B >= max_slices) {
        s.items = (B + max_slices - 1) / max_slices; s.heads = H; s.n = (B + s.items - 1) / s.items;
        return s;
    }
    int groups = 1;                                   // head groups per batch item: the largest divisor of H that fits
    for (int g = 1; g <= H; ++g)
        if (H % g == 0 && (long long)B * g <= max_slices) groups = g;
    s.items = 1; s.heads = H / groups; s.n = B * groups;
    return s;
}

// Arena layout: 8 tensors, m, seq_len, dm, per-batch-item dm, workspace (for one slice at a time).
static size_t host_step_layout(cott_dtype dt, int B, int H, int N, int d, int causal,
                               size_t* tensor_bytes, size_t* ws_bytes) {
    const size_t tb = align_up((size_t)B * H * N * d * dtype_size(dt), 256);
    const HostSlicing sl = host_step_slicing(B, H);
    const size_t wf = cott_workspace_bytes(COTT_OP_FWD, dt, sl.items, sl.heads, N, d, causal);
    const size_t wb = cott_workspace_bytes(COTT_OP_BWD, dt, sl.items, sl.heads, N, d, causal);
    if (wf == (size_t)-1 || wb == (size_t)-1) return (size_t)-1;
    const size_t wsz = align_up(wf > wb ? wf : wb, 256);
    if (tensor_bytes) *tensor_bytes = tb;
    if (ws_bytes) *ws_bytes = wsz;
    return 8 * tb + 3 * align_up((size_t)(B > H ? B : H) * 4, 256) + align_up((size_t)B * H * 4, 256) + wsz;
}

size_t cott_host_step_arena_bytes(cott_dtype dt, int B, int H, int N, int d, int causal) {
    if (B < 1 || H < 1 || N < 1) return (size_t)-1;
    return host_step_layout(dt, B, H, N, d, causal, nullptr, nullptr);
}

cott_status cott_host_step_slicing(int B, int H, int* items_per_slice, int* heads_per_slice, int* n_slices) {
    if (B < 1 || H < 1) return COTT_ERR_INVALID_ARG;
    const HostSlicing sl = host_step_slicing(B, H);
    if (items_per_slice) *items_per_slice = sl.items;
    if (heads_per_slice) *heads_per_slice = sl.heads;
    if (n_slices) *n_slices = sl.n;
    return COTT_OK;
}

cott_status cott_fwd_bwd_host(const void* q_host, const void* k_host, const void* v_host,
                              const void* d_o_host, void* o_host, void* dq_host, void* dk_host,
                              void* dv_host, float* dm_host, const float* m_host,
                              const float* seq_len_host, int B, int H, int N, int d, int causal,
                              cott_dtype dt, void* arena, size_t arena_bytes, void* stream) {
    if (!q_host || !k_host || !v_host || !d_o_host || !o_host || !dq_host || !dk_host ||
        !dv_host || !dm_host || !m_host || B < 1 || H < 1 || N < 1)
        return COTT_ERR_INVALID_ARG;
    size_t tb = 0, wsz = 0;
    const size_t need = host_step_layout(dt, B, H, N, d, causal, &tb, &wsz);
    if (need == (size_t)-1) return COTT_ERR_UNSUPPORTED;
    if (!arena || (reinterpret_cast<uintptr_t>(arena) & 255u) || arena_bytes < need)
        return COTT_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* p = static_cast<char*>(arena);
    char* dq_ = p;           char* dk_ = p + tb;      char* dv_ = p + 2 * tb;
    char* q_ = p + 3 * tb;   char* k_ = p + 4 * tb;   char* v_ = p + 5 * tb;
    char* do_ = p + 6 * tb;  char* o_ = p + 7 * tb;
    const size_t small = align_up((size_t)(B > H ? B : H) * 4, 256);
    float* m_ = reinterpret_cast<float*>(p + 8 * tb);
    float* sl_ = reinterpret_cast<float*>(p + 8 * tb + small);
    float* dm_ = reinterpret_cast<float*>(p + 8 * tb + 2 * small);
    float* dm_parts = reinterpret_cast<float*>(p + 8 * tb + 3 * small);           // [B or n_slices][H]
    void* ws = p + 8 * tb + 3 * small + align_up((size_t)B * H * 4, 256);
    // While slice i is computed on the caller's stream, the inputs of slice i + 1 come in on one
    // library stream and the results of slice i - 1 go back on another: the link is full
    // duplex, and both directions stay busy.  Each slice is a cott_fwd and a cott_bwd call of
    // its own; dm, a sum over the batch, is summed over the slices in slice order.
    SideStreams* ss = side_streams();
    if (!ss) return COTT_ERR_CUDA;
    const HostSlicing sl = host_step_slicing(B, H);
    const int groups = H / sl.heads;                                // head groups per batch item
    const size_t head_bytes = (size_t)N * d * dtype_size(dt);       // one (b, h) of one tensor
    cudaStream_t s_in = ss->s[0], s_out = ss->s[1];
    COTT_CUDA(cudaEventRecord(ss->fork_copy, st));                  // the arena is free once the caller's earlier work is done
    COTT_CUDA(cudaStreamWaitEvent(s_in, ss->fork_copy, 0));
    COTT_CUDA(cudaStreamWaitEvent(s_out, ss->fork_copy, 0));
    COTT_CUDA(cudaMemcpyAsync(m_, m_host, (size_t)H * 4, cudaMemcpyHostToDevice, s_in));
    if (seq_len_host)
        COTT_CUDA(cudaMemcpyAsync(sl_, seq_len_host, (size_t)B * 4, cudaMemcpyHostToDevice, s_in));
    auto slice_of = [&](int i, int* b0, int* nb, int* h0) {
        if (groups == 1) { *b0 = i * sl.items; *nb = (*b0 + sl.items <= B ? sl.items : B - *b0); *h0 = 0; }
        else { *b0 = i / groups; *nb = 1; *h0 = (i % groups) * sl.heads; }
    };
    for (int i = 0; i < sl.n; ++i) {
        int b0, nb, h0;
        slice_of(i, &b0, &nb, &h0);
        const size_t off = ((size_t)b0 * H + h0) * head_bytes, nbytes = (size_t)nb * sl.heads * head_bytes;
        COTT_CUDA(cudaMemcpyAsync(q_ + off, static_cast<const char*>(q_host) + off, nbytes, cudaMemcpyHostToDevice, s_in));
        COTT_CUDA(cudaMemcpyAsync(k_ + off, static_cast<const char*>(k_host) + off, nbytes, cudaMemcpyHostToDevice, s_in));
        COTT_CUDA(cudaMemcpyAsync(v_ + off, static_cast<const char*>(v_host) + off, nbytes, cudaMemcpyHostToDevice, s_in));
        COTT_CUDA(cudaMemcpyAsync(do_ + off, static_cast<const char*>(d_o_host) + off, nbytes, cudaMemcpyHostToDevice, s_in));
        COTT_CUDA(cudaEventRecord(ss->slice_in[i], s_in));
    }
    for (int i = 0; i < sl.n; ++i) {
        int b0, nb, h0;
        slice_of(i, &b0, &nb, &h0);
        const size_t off = ((size_t)b0 * H + h0) * head_bytes, nbytes = (size_t)nb * sl.heads * head_bytes;
        cott_scale_params sp;
        sp.m = m_ + h0; sp.seq_len = seq_len_host ? sl_ + b0 : nullptr; sp.seq_len_scalar = (float)N;
        // (whole batch items per slice: one dm row per slice; head groups: one row per batch item)
        float* dm_slice = dm_parts + (size_t)(groups == 1 ? i : b0) * H + h0;
        COTT_CUDA(cudaStreamWaitEvent(st, ss->slice_in[i], 0));
        cott_status rc = cott_fwd(q_ + off, k_ + off, v_ + off, o_ + off, nullptr, nb, sl.heads, N, d, causal, dt, &sp, ws, wsz, stream);
        if (rc != COTT_OK) return rc;
        rc = cott_bwd(q_ + off, k_ + off, v_ + off, do_ + off, dq_ + off, dk_ + off, dv_ + off, dm_slice,
                      nb, sl.heads, N, d, causal, dt, &sp, ws, wsz, stream);
        if (rc != COTT_OK) return rc;
        COTT_CUDA(cudaEventRecord(ss->slice_out[i], st));
        COTT_CUDA(cudaStreamWaitEvent(s_out, ss->slice_out[i], 0));
        COTT_CUDA(cudaMemcpyAsync(static_cast<char*>(o_host) + off, o_ + off, nbytes, cudaMemcpyDeviceToHost, s_out));
        COTT_CUDA(cudaMemcpyAsync(static_cast<char*>(dq_host) + off, dq_ + off, nbytes, cudaMemcpyDeviceToHost, s_out));
        COTT_CUDA(cudaMemcpyAsync(static_cast<char*>(dk_host) + off, dk_ + off, nbytes, cudaMemcpyDeviceToHost, s_out));
        COTT_CUDA(cudaMemcpyAsync(static_cast<char*>(dv_host) + off, dv_ + off, nbytes, cudaMemcpyDeviceToHost, s_out));
    }
    COTT_CUDA(launch_sum_slices(dm_parts, dm_, groups == 1 ? sl.n : B, H, st));
    COTT_CUDA(cudaMemcpyAsync(dm_host, dm_, (size_t)H * 4, cudaMemcpyDeviceToHost, st));
    COTT_CUDA(cudaEventRecord(ss->join[2], s_out));
    COTT_CUDA(cudaStreamWaitEvent(st, ss->join[2], 0));
    return COTT_OK;
}

cott_status cott_shutdown(void) {
    // The side streams and events of THIS host thread on every device it used, and the
    // profiling events.  Other threads' sets stay until the process ends.
    int cur = 0;
    cudaGetDevice(&cur);
    SideStreams* all = side_streams_table();
    for (int dev = 0; dev < 64; ++dev) {
        SideStreams& ss = all[dev];
        if (!ss.ready) continue;
        if (cudaSetDevice(dev) != cudaSuccess) continue;
        for (int i = 0; i < 3; ++i) { cudaStreamSynchronize(ss.s[i]); cudaStreamDestroy(ss.s[i]); cudaEventDestroy(ss.join[i]); }
        cudaEventDestroy(ss.fork); cudaEventDestroy(ss.fork_copy);
        for (int i = 0; i < kHostSlices; ++i) { cudaEventDestroy(ss.slice_in[i]); cudaEventDestroy(ss.slice_out[i]); }
        ss.ready = false;
    }
    cudaSetDevice(cur);
    g_prof_n.store(-1);
    if (g_prof_created) {
        for (int i = 0; i < 2 * kProfMax; ++i) cudaEventDestroy(g_prof_ev[i]);
        g_prof_created = false;
    }
    return COTT_OK;
}

cott_status cott_last_async_status(const void* workspace, void* stream) {
    if (!workspace) return COTT_ERR_INVALID_ARG;
    COTT_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    int word = 0;
    COTT_CUDA(cudaMemcpy(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost));
    return word == 0 ? COTT_OK : COTT_ERR_TIMEOUT;
}

}  // extern "C"
