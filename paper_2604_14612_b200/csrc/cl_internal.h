// Internal declarations shared by the CUDA translation units of libconflayers.so.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "conflayers.h"

#ifdef __CUDACC__
// Two stored 16-bit elements in one 32-bit word (the lower address in the low half) widened to fp32.
template <typename ST>
struct ClPair16;
template <>
struct ClPair16<__nv_bfloat16> {
    static __device__ __forceinline__ void get(unsigned u, float &a, float &b) {
        a = __uint_as_float(u << 16);
        b = __uint_as_float(u & 0xffff0000u);
    }
};
template <>
struct ClPair16<__half> {
    static __device__ __forceinline__ void get(unsigned u, float &a, float &b) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&u));
        a = f.x;
        b = f.y;
    }
};
template <>
struct ClPair16<float> {   // never used: fp32 storage has no packed pairs
    static __device__ __forceinline__ void get(unsigned, float &a, float &b) { a = b = 0.f; }
};
#endif

#define CL_MAX_T (CL_MAX_K + 1)   // rows of the widest pass (verify)
#define CL_PREFILL_CHUNK 8        // prompt tokens per prefill pass
#define CL_LOGIT_CLAMP 1.0e4f     // clamp bound applied to fp32 logits (Section 3.1; the paper gives no bound)
#define CL_SLOTS 16

// Device-resident state of one context: everything a cycle needs so that no kernel argument
// depends on values only the device knows (positions, pending tokens, counters).
struct ClDevState {
    int ctx;          // committed KV length; rows of a pass sit at positions ctx + row0 + t
    int done;         // set by accept once max_new tokens are out: later kernels of the batch exit at once
    int n_out;        // tokens written to the output buffer
    int max_new;
    int n_drafted;    // drafts of the current cycle
    int n_acc_last;   // result of the last accept
    int err;          // sticky device-side error flags
    int pad;
    int cyc_tok[CL_SLOTS];    // [0] pending token, [1..K] drafts
    int tgt_tok[CL_SLOTS];    // [t] greedy token after verify row t
    float d_pmax[CL_SLOTS], d_conf[CL_SLOTS];   // per draft step
    float v_pmax[CL_SLOTS], v_conf[CL_SLOTS];   // per verify row
    int emitted[CL_SLOTS];    // tokens emitted by the last accept
    unsigned long long cycles, drafted, accepted, emitted_total;
};

// Partial softmax statistics of a slice of the vocabulary, relative to the slice maximum m:
// z = sum exp(l - m), s = sum (l - m) exp(l - m); idx = position of m (lowest index on ties).
struct ClHeadPartial {
    float m, z, s;
    int idx;
};

#ifdef __CUDACC__
// Merge of two partial softmax statistics (b after a in index order: ties of the maximum keep the lower index).
__device__ __forceinline__ ClHeadPartial cl_hp_merge(const ClHeadPartial &a, const ClHeadPartial &b) {
    if (b.z == 0.f) return a;
    if (a.z == 0.f) return b;
    ClHeadPartial r;
    r.m = fmaxf(a.m, b.m);
    const float ea = expf(a.m - r.m), eb = expf(b.m - r.m);
    r.z = a.z * ea + b.z * eb;
    r.s = ea * (a.s + (a.m - r.m) * a.z) + eb * (b.s + (b.m - r.m) * b.z);
    r.idx = (a.m > b.m) ? a.idx : (b.m > a.m) ? b.idx : min(a.idx, b.idx);
    return r;
}
__device__ __forceinline__ ClHeadPartial cl_hp_shfl_xor(const ClHeadPartial &a, int o) {
    ClHeadPartial r;
    r.m = __shfl_xor_sync(0xffffffffu, a.m, o);
    r.z = __shfl_xor_sync(0xffffffffu, a.z, o);
    r.s = __shfl_xor_sync(0xffffffffu, a.s, o);
    r.idx = __shfl_xor_sync(0xffffffffu, a.idx, o);
    return r;
}
#endif

enum { CL_EPI_STORE = 0, CL_EPI_RESID = 1, CL_EPI_SILU = 2, CL_EPI_HEAD = 3 };

struct ClGemvArgs {
    const void *W;        // [rows, cols] storage type
    int rows, cols;
    const float *xin;     // [T, cols] fp32 activations
    float *out;           // STORE: out[t*ld + r] = y; RESID: out[t*ld + r] += y; SILU: out[t*ld + r/2] = silu(y_r) * y_{r+1}
    int ld;
    const ClDevState *st;
    // HEAD epilogue
    float *logits;              // optional [T, rows]
    ClHeadPartial *partials;    // [grid, T]
    unsigned *ticket;
    int *out_tok;               // [T] device
    float *out_pmax, *out_conf; // [T] device
    float inv_log_v;
};

struct ClAttnArgs {
    const float *q;       // [T, ld_q] rotary-embedded queries (fp32)
    int ld_q;
    const void *kcache;   // this layer's K rows [n_heads, max_seq, head_dim] storage type
    const void *vcache;
    float *part;          // [T, H, nsplit, hd + 2] partial (m, l, o[hd])
    unsigned *tickets;    // [T, H]
    float *out;           // [T, d]
    const ClDevState *st;
    int row0, n_heads, n_kv_heads, head_dim, d_model, nsplit, per_max, max_seq;
};

// Per-layer device pointers as the token-step kernel sees them.
struct ClLayerDev {
    const char *wqkv, *wo, *wgu, *wd;
    const float *n1, *n2;
    char *kc, *vc;
};

enum { CL_STEP_DRAFT = 0, CL_STEP_VANILLA = 1 };

struct ClStepArgs {
    const ClLayerDev *layers;   // device [n_layers]
    const int *kept;            // device [n_kept]: layer index | flags << 16 of the layers that run at least in part
                                // (flag bit 0: attention half skipped, bit 1: FFN half skipped)
    int n_kept;
    const void *embed, *lm_head;
    const float *final_norm;
    int d, F, V, H, Hkv, max_seq;        // Hkv: key/value heads (grouped-query attention), H % Hkv == 0
    int att_parts;                       // S: parts the cached keys of a head are cut into (1 .. 8), one CTA each
    int l2_ahead;                        // bytes per CTA the weight prefetch into L2 runs in front of the ring
    float eps, inv_log_v;
    const float2 *rope_cs;
    ClDevState *st;
    float *x, *qkv, *hff;                // global activation vectors [d] [d + 2 Hkv hd] [F]
    float *att_part;                     // [H, 8, hd + 4] per-part attention records (max, sum, -, -, o[hd])
    ClHeadPartial *head_part;            // [grid]
    unsigned *bar;                       // grid barrier: arrival counter, zero at launch
    const float *cum_w;                  // [grid + 1] cumulative row shares of the CTAs (null: equal shares)
    unsigned long long *busy_ns;         // [grid], calibration launches only: time each CTA spent in the matrix phases
    int n_steps, mode, row0;
    unsigned long long wait_ns;          // bound on any single device-side wait
    unsigned bar_arrivals;               // arrivals that complete a grid barrier (= grid size)
    float stop_p;                        // draft mode: stop after the first step whose top-1 probability is below it (0: never)
    int *out_tokens;                     // vanilla mode: emitted tokens (may be null)
    float *logits;                       // optional [n_steps, V]
};

// Records a message that cl_last_error(NULL) returns (for entry points that have no context).
void cl_set_global_error(const char *fmt, ...) __attribute__((format(printf, 1, 2)));

size_t cl_step_smem_bytes();
int cl_step_max_cols(int wdtype);
cudaError_t cl_launch_token_steps(int wdtype, int head_dim, const ClStepArgs &a, int grid, cudaStream_t s);

// launchers (each returns the CUDA launch status)
cudaError_t cl_launch_gemv(int wdtype, int T, int epi, const ClGemvArgs &a, int grid, cudaStream_t s);
cudaError_t cl_launch_embed(int wdtype, const void *embed, const int *tok, int T, int d, float *x, const ClDevState *st,
                            cudaStream_t s);
cudaError_t cl_launch_rmsnorm(const float *x, const float *g, int T, int d, float eps, float *out, const ClDevState *st,
                              cudaStream_t s);
cudaError_t cl_launch_rmsnorm_rows(int in_dtype, const void *x, const float *g, int T, int d, float eps, float *out,
                                   cudaStream_t s);
cudaError_t cl_launch_rope_append(int wdtype, float *qkv, int T, int row0, int H, int Hkv, int hd, int d, const float2 *rope_cs,
                                  void *kcache, void *vcache, int max_seq, const ClDevState *st, cudaStream_t s);
cudaError_t cl_launch_attn(int wdtype, int T, const ClAttnArgs &a, cudaStream_t s);
cudaError_t cl_launch_tap(int wdtype, const float *x, int T, int row0, int d, void *ring_layer, int P,
                          const ClDevState *st, cudaStream_t s);
cudaError_t cl_launch_accept(ClDevState *st, int K, int *out_tokens, cudaStream_t s);
cudaError_t cl_launch_advance(ClDevState *st, int n, int set_pending_from_tgt, cudaStream_t s);
// epilogues of the tensor-core GEMMs of the T-row pass
enum { CL_VEPI_STORE = 0, CL_VEPI_RESID = 1, CL_VEPI_SILU = 2, CL_VEPI_HEAD = 3 };

struct ClTensorMap {                  // opaque 128-byte TMA descriptor (CUtensorMap)
    alignas(64) unsigned char bytes[128];
};

bool cl_make_tensor_map(ClTensorMap *m, const void *base, int rows, int cols, int box_rows, int f16 = 0);

// ---- persistent tensor-core pass over T <= CL_MAX_T rows (16-bit models): all layers and the LM head in one launch ----
#define CL_ROWS_AROWS 32   // rows per k-block of an activation operand buffer: hi part of token t in row t, lo part in row T + t
struct ClRowsLayer {
    const char *wqkv, *wo, *wgu, *wd;   // copies in the kernel's streaming order (CTA by CTA, [K / 64][block rows][64], 16-byte pieces permuted by row & 7)
    const float *n1, *n2;
    char *kc, *vc;
    void *tap0, *tap1;                  // this layer's hidden-state ring after the attention add / after the FFN add (or null)
};
struct ClRowsArgs {
    const ClRowsLayer *layers;          // device [L]
    int L;
    const char *head;                   // LM head, k-block-major
    const void *embed;                  // [V, d] row-major
    const float *final_norm;
    int d, F, V, H, Hkv, hd, max_seq;
    int T, row0, want_head, f16, att_parts, tap, tap_P;
    int split;                          // CTAs of a group that share the rows of an output / down projection and cut K between them
    int entry;                          // bytes: a ring entry (one group of bulk copies) takes as many k-blocks of a tile as fit in this, at least one
    int chain;                          // k-blocks (64 elements of K) summed in tensor memory before the accumulator is drained into registers
    float eps, inv_d, inv_log_v;
    const float2 *rope_cs;
    ClDevState *st;
    const int *tok;                     // device [T] token ids of the rows
    float *x, *qkv;                     // residual stream [T, d], QKV product [T, d + 2 Hkv hd] (raw: no rotary yet)
    unsigned short *Ax, *Aatt, *Ah;     // activation operands [d / 64 | d / 64 | F / 64][CL_ROWS_AROWS][64]
    float *ws;                          // [grid, CL_MAX_T, 224] raw products of the output / down projections, per CTA (K part)
    float *ssq;                         // [grid, CL_SLOTS] per-CTA sums of squares of the residual rows
    float *att_part;                    // [H, 8, CL_MAX_T, hd + 2] per-part attention records
    unsigned *att_tickets;              // [H], zero between launches
    ClHeadPartial *head_part;           // [grid, CL_SLOTS]
    float *logits;                      // optional [T, V]
    int *out_tok;                       // [T] greedy token after each row
    float *out_pmax, *out_conf;
    unsigned *sync;                     // counters, all zero at launch: [0] the grid barrier, [1 .. 1 + grid / split) the groups' barriers,
                                        // then the completion counters of the buffers that connect the phases, at the offsets below
    int c_ssq, c_ax, c_ah, c_att, c_qkv;   // offsets in sync: 1 | d / 64 | F / 64 | H | (d + 2 Hkv hd) / hd counters
    unsigned bar_arrivals;
    unsigned long long wait_ns;
    unsigned long long *phase_ns;       // diagnostics, optional: [grid, 8] time of each CTA's thread 0 by phase
};
size_t cl_rows_smem_bytes();
int cl_rows_att_part_floats(int H);
// src: row-major [rows, K] 16-bit elements; dst: the same matrix in the streaming order of a grid of `grid` CTAs
// (rows split in units of `unit` rows, exactly as the kernel splits them)
cudaError_t cl_launch_tile_layout(const void *src, void *dst, int rows, int K, int unit, int grid, cudaStream_t s);
cudaError_t cl_launch_rows_pass(int wdtype, int head_dim, const ClRowsArgs &a, int grid, cudaStream_t s);

// ---- wide tensor-core GEMM of the prompt pass (bf16 models): up to CL_WIDE_MAX_M prompt rows at a time ----
#define CL_WIDE_MAX_M 512
struct ClWideArgs {
    int M, rows, KB;                  // token rows of the pass, weight rows, K blocks of 64
    int MT, NT, splits;               // 128-row token tiles, 256-row weight tiles, parts the K range is cut into
    int lo_row0;                      // first row of the lo parts in the activation buffer (hi parts start at row 0)
    float *P;                         // [splits, M, rows] partial products (a later kernel adds the splits in order)
    int *err;
    int f16;                          // the model's 16-bit type: 0 bf16, 1 fp16
};
struct ClWideNormArgs {
    float *x;                         // [M, d] residual stream of the pass
    int M, d, splits;
    const float *P;                   // [splits, M, d] products to add to x, or null
    const void *embed;                // with tok: x = E[tok[t]] instead (start of the pass)
    const int *tok;
    const float *g;                   // gain of the RMSNorm that follows, or null (no normalised rows are written)
    float eps;
    __nv_bfloat16 *A;                 // [2 * lo_row0, d]: normalised rows as bf16 hi (row t) and lo (row lo_row0 + t)
    int lo_row0;
    void *tap;                        // optional: this layer's hidden-state ring [tap_P, d] (bf16)
    int tap_P;
    const ClDevState *st;
    int f16;                          // the model's 16-bit type: 0 bf16, 1 fp16 (embedding, taps, normalised rows)
};
int cl_wide_splits(int M, int rows, int KB, int n_sm, size_t ws_floats);
cudaError_t cl_launch_wide(const ClTensorMap &mapA, const ClTensorMap &mapB, const ClWideArgs &a, cudaStream_t s);
cudaError_t cl_launch_wide_norm(const ClWideNormArgs &a, cudaStream_t s);
cudaError_t cl_launch_wide_rope_append(float *P, int splits, int M, int H, int Hkv, int hd, int d, const float2 *rope_cs,
                                       void *kcache, void *vcache, int max_seq, const ClDevState *st, int f16, cudaStream_t s);
// causal attention of the M rows of the pass (positions ctx ..) over the cache; q: fp32 rows [M, ld_q], rotary applied;
// the output goes out as bf16 hi (row t) and lo (row lo_row0 + t) parts [.., d]
cudaError_t cl_launch_attn_wide(const float *q, int ld_q, const void *kcache, const void *vcache, __nv_bfloat16 *out_b,
                                int lo_row0, int M, int d, int H, int Hkv, int hd, int max_seq, const ClDevState *st,
                                int f16, cudaStream_t s);
cudaError_t cl_launch_wide_silu(const float *P, int splits, int M, int F, __nv_bfloat16 *A, int lo_row0, int f16, cudaStream_t s);

// tensor-core scoring (bf16 / fp16 LM head): normalise to the 16-bit type, contraction fused with the softmax statistics, finalize
int cl_score_tc_ranges(int R, int n_sm);
size_t cl_score_tc_partials(int R, int n_sm);
cudaError_t cl_launch_rmsnorm_bf16(int in_dtype, const void *x, const float *g, int rows, int d, float eps, void *out,
                                   int f16, cudaStream_t s);
cudaError_t cl_launch_score_tc(const void *xn, const void *lm_head, int R, int V, int d, ClHeadPartial *partials, int n_sm,
                               int *err, float *conf, float *pmax, int *arg, int f16, cudaStream_t s);
cudaError_t cl_launch_mean_rows(const float *conf_rows, int rows, int P, float *c_layer, cudaStream_t s);
cudaError_t cl_launch_select(const cl_select_cfg &cfg, int n_layers, const float *c_layer, uint8_t *mask, double *margins,
                             cudaStream_t s);
cudaError_t cl_launch_interleave(int wdtype, const void *wg, const void *wu, void *dst, int F, int d, cudaStream_t s);
