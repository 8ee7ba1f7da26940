// Host side of libconflayers.so: context, weight arena, and the sequencing of the kernels that make
// up a draft step, a verify pass, acceptance and the confidence scoring.  All arithmetic of the
// method runs in the kernels; this file only lays out memory and enqueues launches on one stream.
#include <math.h>
#include <stdarg.h>
#include <stddef.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "cl_internal.h"

struct ClLayer {
    char *wqkv, *wo, *wgu, *wd;   // [3d,d] [d,d] [2F,d] (gate/up rows interleaved) [d,F]
    float *n1, *n2;
    char *kc, *vc;                // this layer's K and V cache [n_heads, max_seq, head_dim]
};

struct cl_ctx {
    cl_model_cfg cfg;
    cudaStream_t stream;
    int device, n_sm;
    char err[512];
    size_t esz;                   // bytes per stored element (weights, KV, taps)
    int taps;                     // hidden states recorded per layer: 1 = after the FFN add, 2 = after the attention add and after the FFN add
    int loaded, head_only, prefilled;
    // device memory
    char *wbuf;                   // all layer matrices, one allocation, in execution order
    char *embed, *lm_head;
    float *final_norm, *norms;
    char *kv;
    float2 *rope_cs;
    float *x, *xn, *qkv, *att, *hff, *att_part, *logits;
    unsigned *tickets;            // [0] LM head ticket, [1 ..] attention tickets
    ClHeadPartial *head_part;
    int head_grid;
    ClDevState *st;
    ClDevState *h_st;             // pinned host mirror
    int *prompt_dev;              // [max_seq]
    int *out_dev;                 // generated tokens
    int out_cap;
    char *ring;                   // [L, P, d] storage type
    // scoring scratch
    float *sc_conf, *sc_pmax, *sc_clayer;
    int *sc_arg;
    size_t sc_cap;                // rows*P capacity
    char *sc_xn;                  // [sc_cap, d] bf16 normalised rows (tensor-core scoring)
    ClHeadPartial *sc_part;       // per-(row, vocabulary range) softmax statistics
    uint8_t *sel_mask;            // device [iters_cap, L]
    double *sel_margins;          // device [L]
    float *sel_clayers;           // device [iters_cap, L]
    int sel_iters_cap;
    // token-step kernel (persistent single-token step)
    float *cum_w_dev;             // [n_sm + 1] cumulative row shares of the token-step kernel's CTAs (null until calibrated)
    unsigned long long *busy_dev; // [n_sm] calibration timings
    ClLayerDev *layers_dev;
    int *kept_dev, *kept_all_dev;
    int n_kept, use_step, max_blk, att_parts, l2_ahead, cum_w_ready, calibrating;
    unsigned *bar_dev;
    float *att_part2;
    ClHeadPartial *head_part2;
    // TMA descriptors of the row-major matrices (B operand of the wide GEMMs of the prompt pass, 16-bit models)
    std::vector<ClTensorMap> map_qkv, map_o, map_gu, map_d;
    // persistent tensor-core pass of the T-row passes (16-bit models): second, k-block-major copy of the matrices
    int use_rows;
    char *wtile, *head_tile;             // per layer [Wqkv | Wo | Wgu | Wd] k-block-major; LM head k-block-major
    ClRowsLayer *rows_layers_dev;
    unsigned short *r_ax, *r_aatt, *r_ah;
    float *r_ssq, *r_att_part, *r_ws;
    unsigned *r_bar;                     // counters of the pass: the grid barrier, one per group of CTAs, the completion counters
    int r_sync_words, r_c_ssq, r_c_ax, r_c_ah, r_c_att, r_c_qkv;
    int rows_entry;                      // bytes per ring entry of the T-row pass (as many k-blocks as fit, at least one)
    int rows_split;                      // CTAs per group that cut the K range of the output / down projections between them
    unsigned *r_tickets;
    ClHeadPartial *r_head_part;
    int rows_chain;                      // k-blocks per accumulation chain in tensor memory
    unsigned long long *r_phase_ns;      // diagnostics (cl_debug_read): per-CTA time by phase of the last pass
    // wide tensor-core GEMM path of the prompt pass (bf16 models)
    int use_wide;
    ClTensorMap map_wx, map_watt, map_wh;  // activation rows as bf16 hi/lo parts, boxes of 128 rows
    __nv_bfloat16 *w_ax, *w_aatt, *w_ah;   // [2 * CL_WIDE_MAX_M, d] [.., d] [.., F]
    float *w_x, *w_P;                      // residual stream [CL_WIDE_MAX_M, d], product parts
    size_t w_P_floats;
    std::vector<ClLayer> layers;
    std::vector<uint8_t> mask;    // host copy of the skip set
    int nsplit, per_max;
    // host view of the device state (exact after every call that synchronises)
    int h_ctx, h_ndraft, tapped;
    int h_filled;                 // positions [0, h_filled) of every layer's cache have been written by full-model passes
    uint64_t launches;
    // diagnostics (cl_debug_set)
    unsigned long long wait_ns;   // bound on any single device-side wait of the step kernel
    int bar_extra;                // extra arrivals the persistent kernels' grid barriers wait for (0: barriers complete)
};

static char g_err[512] = "";

static int fail(cl_ctx *c, int code, const char *fmt, ...) __attribute__((format(printf, 3, 4)));
static int fail(cl_ctx *c, int code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(c ? c->err : g_err, 512, fmt, ap);
    va_end(ap);
    return code;
}

void cl_set_global_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

#define CU(call)                                                                                          \
    do {                                                                                                  \
        cudaError_t e_ = (call);                                                                          \
        if (e_ != cudaSuccess) return fail(c, CL_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

#define KL(call)                                                                                          \
    do {                                                                                                  \
        cudaError_t e_ = (call);                                                                          \
        ++c->launches;                                                                                    \
        if (e_ != cudaSuccess) return fail(c, CL_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

#define ST_FIELD(c, type, field) ((type *)((char *)(c)->st + offsetof(ClDevState, field)))

namespace {

struct ClPoke {
    int ctx, pending, n_drafted, done, n_out, max_new;   // -1 = leave unchanged
    int n_force;
    int force[CL_MAX_K];
};

__global__ void k_poke(ClDevState *st, ClPoke p) {
    if (threadIdx.x != 0) return;
    if (p.ctx >= 0) st->ctx = p.ctx;
    if (p.pending >= 0) st->cyc_tok[0] = p.pending;
    for (int i = 0; i < p.n_force; ++i) st->cyc_tok[1 + i] = p.force[i];
    if (p.n_drafted >= 0) st->n_drafted = p.n_drafted;
    if (p.done >= 0) st->done = p.done;
    if (p.n_out >= 0) st->n_out = p.n_out;
    if (p.max_new >= 0) st->max_new = p.max_new;
}

ClPoke poke_none() {
    ClPoke p;
    p.ctx = p.pending = p.n_drafted = p.done = p.n_out = p.max_new = -1;
    p.n_force = 0;
    return p;
}

}  // namespace

static int poke(cl_ctx *c, const ClPoke &p) {
    k_poke<<<1, 32, 0, c->stream>>>(c->st, p);
    KL(cudaGetLastError());
    return CL_OK;
}

static int sync_state(cl_ctx *c) {
    CU(cudaMemcpyAsync(c->h_st, c->st, sizeof(ClDevState), cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    c->h_ctx = c->h_st->ctx;
    return CL_OK;
}

// ---------------------------------------------------------------------------------------------

extern "C" const char *cl_last_error(cl_ctx *c) { return c ? c->err : g_err; }

extern "C" int cl_create(const cl_model_cfg *cfg, void *cuda_stream, cl_ctx **out) {
    cl_ctx *c = nullptr;
    if (!cfg || !out) return fail(c, CL_EINVAL, "cl_create: null argument");
    *out = nullptr;
    if (cfg->n_layers < 0 || cfg->d_model <= 0 || cfg->n_heads <= 0 || cfg->vocab < 2 || cfg->max_seq <= 0)
        return fail(c, CL_EINVAL, "cl_create: non-positive dimension");
    if (cfg->n_heads * cfg->head_dim != cfg->d_model) return fail(c, CL_EINVAL, "cl_create: d_model != n_heads * head_dim");
    if (cfg->n_kv_heads < 1 || cfg->n_heads % cfg->n_kv_heads)
        return fail(c, CL_EINVAL, "cl_create: n_kv_heads must be at least 1 and divide n_heads");
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return fail(c, CL_EINVAL, "cl_create: head_dim must be 64 or 128");
    if (cfg->d_model % 8 || (cfg->n_layers > 0 && (cfg->d_ffn <= 0 || cfg->d_ffn % 8)))
        return fail(c, CL_EINVAL, "cl_create: d_model and d_ffn must be multiples of 8");
    if (cfg->weight_dtype < 0 || cfg->weight_dtype > 2) return fail(c, CL_EINVAL, "cl_create: weight_dtype must be 0, 1 or 2");
    if (cfg->tap_positions < 0) return fail(c, CL_EINVAL, "cl_create: tap_positions < 0");
    if (cfg->tap_modules < 0 || cfg->tap_modules > 2) return fail(c, CL_EINVAL, "cl_create: tap_modules must be 0, 1 or 2");
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(c, CL_ECUDA, "cl_create: no CUDA device: %s", cudaGetErrorString(e));
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) return fail(c, CL_ECUDA, "cl_create: cudaGetDeviceProperties: %s", cudaGetErrorString(e));
    if (prop.major < 10) return fail(c, CL_ECUDA, "cl_create: compute capability %d.%d, built for sm_100a only", prop.major, prop.minor);
    c = new (std::nothrow) cl_ctx();
    if (!c) return fail(nullptr, CL_ENOMEM, "cl_create: host allocation failed");
    c->cfg = *cfg;
    c->stream = (cudaStream_t)cuda_stream;
    c->device = dev;
    c->n_sm = prop.multiProcessorCount;
    c->esz = cfg->weight_dtype == 0 ? 4 : 2;
    c->taps = cfg->tap_modules == 2 ? 2 : 1;
    c->err[0] = 0;
    c->wait_ns = 2000000000ull;
    c->mask.assign((size_t)cfg->n_layers, 0);
    *out = c;
    return CL_OK;
}

static void free_all(cl_ctx *c) {
    void *ptrs[] = {c->wbuf, c->embed, c->lm_head, c->final_norm, c->norms, c->kv, c->rope_cs, c->x, c->xn, c->qkv,
                    c->att, c->hff, c->att_part, c->logits, c->tickets, c->head_part, c->st, c->prompt_dev, c->out_dev,
                    c->ring, c->sc_conf, c->sc_pmax, c->sc_clayer, c->sc_arg, c->sc_xn, c->sc_part, c->sel_mask, c->sel_margins, c->sel_clayers,
                    c->layers_dev, c->kept_dev, c->kept_all_dev, c->bar_dev, c->att_part2, c->head_part2,
                    c->cum_w_dev, c->busy_dev,
                    c->w_ax, c->w_aatt, c->w_ah, c->w_x, c->w_P, c->wtile, c->head_tile, c->rows_layers_dev, c->r_ax, c->r_aatt,
                    c->r_ah, c->r_ssq, c->r_att_part, c->r_tickets, c->r_head_part, c->r_phase_ns, c->r_ws, c->r_bar};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    if (c->h_st) cudaFreeHost(c->h_st);
}

extern "C" int cl_destroy(cl_ctx *c) {
    if (!c) return CL_OK;
    cudaStreamSynchronize(c->stream);
    free_all(c);
    delete c;
    return CL_OK;
}

template <typename T>
static cudaError_t dmalloc(T **p, size_t bytes) {
    return cudaMalloc((void **)p, bytes ? bytes : 16);
}

#define DM(ptr, bytes)                                                                                          \
    do {                                                                                                        \
        cudaError_t e_ = dmalloc(&(ptr), (bytes));                                                              \
        if (e_ != cudaSuccess) {                                                                                \
            cudaGetLastError();                                                                                 \
            return fail(c, e_ == cudaErrorMemoryAllocation ? CL_ENOMEM : CL_ECUDA, "cudaMalloc(%zu) for %s: %s", \
                        (size_t)(bytes), #ptr, cudaGetErrorString(e_));                                         \
        }                                                                                                       \
    } while (0)

static int calibrate_row_shares(cl_ctx *c);
static char *ring_slot(cl_ctx *c, int l, int which);

extern "C" int cl_load(cl_ctx *c, const cl_weights *w) {
    if (!c || !w) return fail(c, CL_EINVAL, "cl_load: null argument");
    if (c->loaded) return fail(c, CL_ESTATE, "cl_load: weights already loaded");
    const cl_model_cfg &g = c->cfg;
    const size_t d = g.d_model, F = g.d_ffn, V = g.vocab, L = g.n_layers, es = c->esz;
    const size_t kvd = (size_t)g.n_kv_heads * g.head_dim, qkv_rows = d + 2 * kvd;   // [q | k | v] rows of the fused projection
    c->head_only = w->head_only ? 1 : 0;
    if (!w->lm_head || !w->final_norm) return fail(c, CL_EINVAL, "cl_load: lm_head / final_norm missing");
    if (!c->head_only) {
        if (!w->embed || !w->wq || !w->wk || !w->wv || !w->wo || !w->wg || !w->wu || !w->wd || !w->norm1 || !w->norm2)
            return fail(c, CL_EINVAL, "cl_load: null weight array");
        for (size_t l = 0; l < L; ++l)
            if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->wg[l] || !w->wu[l] || !w->wd[l] || !w->norm1[l] ||
                !w->norm2[l])
                return fail(c, CL_EINVAL, "cl_load: null weight pointer in layer %zu", l);
    }
    const cudaMemcpyKind kind = cudaMemcpyDefault;

    // ---- head, norms, state (needed by every context)
    DM(c->lm_head, V * d * es);
    DM(c->final_norm, d * 4);
    CU(cudaMemcpyAsync(c->lm_head, w->lm_head, V * d * es, kind, c->stream));
    CU(cudaMemcpyAsync(c->final_norm, w->final_norm, d * 4, kind, c->stream));
    DM(c->st, sizeof(ClDevState));
    CU(cudaMemsetAsync(c->st, 0, sizeof(ClDevState), c->stream));
    CU(cudaMallocHost((void **)&c->h_st, sizeof(ClDevState)));
    memset(c->h_st, 0, sizeof(ClDevState));
    DM(c->xn, (size_t)CL_MAX_T * d * 4);
    DM(c->logits, (size_t)CL_MAX_T * V * 4);
    c->head_grid = c->n_sm * 4;
    DM(c->head_part, (size_t)c->head_grid * CL_MAX_T * sizeof(ClHeadPartial));
    const size_t n_tickets = 1 + (size_t)CL_MAX_T * g.n_heads;
    DM(c->tickets, n_tickets * 4);
    CU(cudaMemsetAsync(c->tickets, 0, n_tickets * 4, c->stream));
    DM(c->sel_margins, (L ? L : 1) * sizeof(double));
    DM(c->sc_clayer, (L ? L : 1) * 4);

    if (!c->head_only) {
        // ---- weights: per layer [Wqkv | Wo | Wgu | Wd], contiguous in execution order
        const size_t b_qkv = qkv_rows * d * es, b_o = d * d * es, b_gu = 2 * F * d * es, b_d = d * F * es;
        const size_t per_layer = b_qkv + b_o + b_gu + b_d;
        DM(c->wbuf, per_layer * L);
        DM(c->norms, 2 * L * d * 4);
        DM(c->embed, V * d * es);
        CU(cudaMemcpyAsync(c->embed, w->embed, V * d * es, kind, c->stream));
        const size_t kv_layer = (size_t)g.max_seq * kvd * es;
        DM(c->kv, 2 * L * kv_layer);
        CU(cudaMemsetAsync(c->kv, 0, 2 * L * kv_layer, c->stream));
        char *stage_g = nullptr, *stage_u = nullptr;
        if (!w->on_device) {
            DM(stage_g, F * d * es);
            DM(stage_u, F * d * es);
        }
        c->layers.resize(L);
        for (size_t l = 0; l < L; ++l) {
            ClLayer &y = c->layers[l];
            y.wqkv = c->wbuf + l * per_layer;
            y.wo = y.wqkv + b_qkv;
            y.wgu = y.wo + b_o;
            y.wd = y.wgu + b_gu;
            y.n1 = c->norms + (2 * l) * d;
            y.n2 = c->norms + (2 * l + 1) * d;
            y.kc = c->kv + (2 * l) * kv_layer;
            y.vc = c->kv + (2 * l + 1) * kv_layer;
            CU(cudaMemcpyAsync(y.wqkv, w->wq[l], d * d * es, kind, c->stream));
            CU(cudaMemcpyAsync(y.wqkv + d * d * es, w->wk[l], kvd * d * es, kind, c->stream));
            CU(cudaMemcpyAsync(y.wqkv + (d + kvd) * d * es, w->wv[l], kvd * d * es, kind, c->stream));
            CU(cudaMemcpyAsync(y.wo, w->wo[l], b_o, kind, c->stream));
            CU(cudaMemcpyAsync(y.wd, w->wd[l], b_d, kind, c->stream));
            CU(cudaMemcpyAsync(y.n1, w->norm1[l], d * 4, kind, c->stream));
            CU(cudaMemcpyAsync(y.n2, w->norm2[l], d * 4, kind, c->stream));
            const void *sg = w->wg[l], *su = w->wu[l];
            if (!w->on_device) {
                CU(cudaMemcpyAsync(stage_g, sg, F * d * es, kind, c->stream));
                CU(cudaMemcpyAsync(stage_u, su, F * d * es, kind, c->stream));
                sg = stage_g;
                su = stage_u;
            }
            KL(cl_launch_interleave(g.weight_dtype, sg, su, y.wgu, (int)F, (int)d, c->stream));
        }
        // ---- rotary table cos/sin(pos * theta^(-2i/hd)), evaluated in double on the host
        const int half = g.head_dim / 2;
        std::vector<float2> cs((size_t)g.max_seq * half);
        for (int p = 0; p < g.max_seq; ++p)
            for (int i = 0; i < half; ++i) {
                const double ang = (double)p * pow((double)g.rope_theta, -2.0 * i / g.head_dim);
                cs[(size_t)p * half + i] = make_float2((float)cos(ang), (float)sin(ang));
            }
        DM(c->rope_cs, cs.size() * sizeof(float2));
        CU(cudaMemcpyAsync(c->rope_cs, cs.data(), cs.size() * sizeof(float2), cudaMemcpyHostToDevice, c->stream));
        // ---- activations and scratch
        DM(c->x, (size_t)CL_MAX_T * d * 4);
        DM(c->qkv, (size_t)CL_MAX_T * qkv_rows * 4);
        DM(c->att, (size_t)CL_MAX_T * d * 4);
        DM(c->hff, (size_t)CL_MAX_T * F * 4);
        c->nsplit = 4;
        c->per_max = (g.max_seq + c->nsplit - 1) / c->nsplit;
        DM(c->att_part, (size_t)CL_MAX_T * g.n_heads * c->nsplit * (g.head_dim + 2) * 4);
        DM(c->prompt_dev, (size_t)g.max_seq * 4);
        if (g.tap_positions > 0) {
            DM(c->ring, L * (size_t)c->taps * g.tap_positions * d * es);
            CU(cudaMemsetAsync(c->ring, 0, L * (size_t)c->taps * g.tap_positions * d * es, c->stream));
        }
        // ---- token-step kernel: per-layer pointer table, kept-layer lists, barrier, attention / head partials
        {
            std::vector<ClLayerDev> ld(L);
            std::vector<int> all(L);
            for (size_t l = 0; l < L; ++l) {
                const ClLayer &y = c->layers[l];
                ld[l] = ClLayerDev{y.wqkv, y.wo, y.wgu, y.wd, y.n1, y.n2, y.kc, y.vc};
                all[l] = (int)l;
            }
            DM(c->layers_dev, (L ? L : 1) * sizeof(ClLayerDev));
            DM(c->kept_dev, (L ? L : 1) * sizeof(int));
            DM(c->kept_all_dev, (L ? L : 1) * sizeof(int));
            CU(cudaMemcpy(c->layers_dev, ld.data(), L * sizeof(ClLayerDev), cudaMemcpyHostToDevice));
            CU(cudaMemcpy(c->kept_dev, all.data(), L * sizeof(int), cudaMemcpyHostToDevice));
            CU(cudaMemcpy(c->kept_all_dev, all.data(), L * sizeof(int), cudaMemcpyHostToDevice));
            c->n_kept = (int)L;
            c->max_blk = (g.max_seq + 31) / 32;
            DM(c->bar_dev, 2 * sizeof(unsigned));
            CU(cudaMemsetAsync(c->bar_dev, 0, 2 * sizeof(unsigned), c->stream));
            DM(c->att_part2, (size_t)g.n_heads * 8 * (g.head_dim + 4) * 4);
            CU(cudaMemsetAsync(c->att_part2, 0, (size_t)g.n_heads * 8 * (g.head_dim + 4) * 4, c->stream));
            c->att_parts = c->n_sm / g.n_heads;
            if (c->att_parts > 8) c->att_parts = 8;
            if (c->att_parts < 1) c->att_parts = 1;
            const char *ah = getenv("CL_L2_AHEAD_KB");   // tuning knob: L2 run-ahead of the weight stream per SM
            c->l2_ahead = (ah && ah[0]) ? atoi(ah) * 1024 : 0;   // measured on B200: any run-ahead made decoding slower
            if (c->l2_ahead < 0) c->l2_ahead = 0;
            DM(c->head_part2, (size_t)c->n_sm * sizeof(ClHeadPartial));
            const int maxc = cl_step_max_cols(g.weight_dtype);
            int coop = 0;
            cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device);
            const char *off = getenv("CL_DISABLE_STEP_KERNEL");
            c->use_step = coop && d <= (size_t)maxc && F <= (size_t)maxc && !(off && off[0] == '1');
        }
        // ---- wide GEMM path of the prompt pass (16-bit models): tensor maps of every matrix, hi/lo activation rows,
        // residual stream, product parts
        if (g.weight_dtype != 0) {
            const int f16 = g.weight_dtype == 2;
            const char *woff = getenv("CL_DISABLE_WIDE_PREFILL");
            if (!(woff && woff[0] == '1') && g.max_seq > 17) {
                {
                    bool ok = true;
                    c->map_qkv.resize(L); c->map_o.resize(L); c->map_gu.resize(L); c->map_d.resize(L);
                    for (size_t l = 0; l < L && ok; ++l) {
                        const ClLayer &y = c->layers[l];
                        ok = cl_make_tensor_map(&c->map_qkv[l], y.wqkv, (int)qkv_rows, (int)d, 128, f16) &&
                             cl_make_tensor_map(&c->map_o[l], y.wo, (int)d, (int)d, 128, f16) &&
                             cl_make_tensor_map(&c->map_gu[l], y.wgu, (int)(2 * F), (int)d, 128, f16) &&
                             cl_make_tensor_map(&c->map_d[l], y.wd, (int)d, (int)F, 128, f16);
                    }
                    if (!ok) return fail(c, CL_ECUDA, "cl_load: encoding a TMA tensor map failed");
                    const size_t Mw = CL_WIDE_MAX_M, widest = std::max(qkv_rows, 2 * F);
                    DM(c->w_ax, 2 * Mw * d * 2);
                    DM(c->w_aatt, 2 * Mw * d * 2);
                    DM(c->w_ah, 2 * Mw * F * 2);
                    CU(cudaMemsetAsync(c->w_ax, 0, 2 * Mw * d * 2, c->stream));
                    CU(cudaMemsetAsync(c->w_aatt, 0, 2 * Mw * d * 2, c->stream));
                    CU(cudaMemsetAsync(c->w_ah, 0, 2 * Mw * F * 2, c->stream));
                    DM(c->w_x, Mw * d * 4);
                    c->w_P_floats = 2 * Mw * widest;
                    DM(c->w_P, c->w_P_floats * 4);
                    if (!(cl_make_tensor_map(&c->map_wx, c->w_ax, (int)(2 * Mw), (int)d, 128, f16) &&
                          cl_make_tensor_map(&c->map_watt, c->w_aatt, (int)(2 * Mw), (int)d, 128, f16) &&
                          cl_make_tensor_map(&c->map_wh, c->w_ah, (int)(2 * Mw), (int)F, 128, f16)))
                        return fail(c, CL_ECUDA, "cl_load: encoding a TMA tensor map failed");
                    c->use_wide = 1;
                }
            }
        }
        // ---- persistent T-row pass on the tensor cores: k-block-major copies of every matrix, operand buffers, partials
        c->use_rows = 0;
        {
            const char *off = getenv("CL_DISABLE_ROWS_KERNEL");
            int coop = 0;
            cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device);
            const bool shape_ok = d % 64 == 0 && F % 64 == 0 && (d / 8 + c->n_sm - 1) / c->n_sm <= 16 && g.n_heads <= 8 * c->n_sm &&
                                  (d + c->n_sm - 1) / c->n_sm + 8 <= 224;
            if (g.weight_dtype != 0 && coop && shape_ok && L > 0 && !(off && off[0] == '1')) {
                // the output and down projections give each CTA too few rows for an efficient tensor-core tile: groups of
                // CTAs share rows and cut K (a group's partial products meet in a workspace)
                const char *sp = getenv("CL_ROWS_SPLIT");   // tuning knob
                c->rows_split = (sp && sp[0]) ? atoi(sp) : 4;
                if (c->rows_split < 1 || c->rows_split > 8) c->rows_split = 1;
                // (a group's rows must fit one tile of 224 rows: its parts meet in a workspace that holds one tile per CTA)
                while (c->rows_split > 1 && (c->n_sm % c->rows_split || d / 64 < (size_t)c->rows_split || F / 64 < (size_t)c->rows_split ||
                                             (d * c->rows_split + c->n_sm - 1) / c->n_sm + 8 > 224))
                    c->rows_split >>= 1;
                DM(c->wtile, per_layer * L);
                DM(c->head_tile, V * d * es);
                DM(c->r_ws, (size_t)c->n_sm * CL_MAX_T * 224 * 4);
                c->r_c_ssq = 1 + c->n_sm / c->rows_split;
                c->r_c_ax = c->r_c_ssq + 1;
                c->r_c_ah = c->r_c_ax + (int)(d / 64);
                c->r_c_att = c->r_c_ah + (int)(F / 64);
                c->r_c_qkv = c->r_c_att + g.n_heads;
                c->r_sync_words = c->r_c_qkv + (int)(qkv_rows / g.head_dim);
                DM(c->r_bar, (size_t)c->r_sync_words * 4);
                std::vector<ClRowsLayer> rl(L);
                for (size_t l = 0; l < L; ++l) {
                    const ClLayer &y = c->layers[l];
                    char *t0 = c->wtile + l * per_layer;
                    KL(cl_launch_tile_layout(y.wqkv, t0, (int)qkv_rows, (int)d, 1, c->n_sm, c->stream));
                    KL(cl_launch_tile_layout(y.wo, t0 + b_qkv, (int)d, (int)d, 1, c->n_sm / c->rows_split, c->stream));
                    KL(cl_launch_tile_layout(y.wgu, t0 + b_qkv + b_o, (int)(2 * F), (int)d, 2, c->n_sm, c->stream));
                    KL(cl_launch_tile_layout(y.wd, t0 + b_qkv + b_o + b_gu, (int)d, (int)F, 1, c->n_sm / c->rows_split, c->stream));
                    rl[l] = ClRowsLayer{t0, t0 + b_qkv, t0 + b_qkv + b_o, t0 + b_qkv + b_o + b_gu, y.n1, y.n2, y.kc, y.vc,
                                        ring_slot(c, (int)l, 0), ring_slot(c, (int)l, 1)};
                }
                KL(cl_launch_tile_layout(c->lm_head, c->head_tile, (int)V, (int)d, 1, c->n_sm, c->stream));
                DM(c->rows_layers_dev, L * sizeof(ClRowsLayer));
                CU(cudaMemcpyAsync(c->rows_layers_dev, rl.data(), L * sizeof(ClRowsLayer), cudaMemcpyHostToDevice, c->stream));
                CU(cudaStreamSynchronize(c->stream));   // rl goes out of scope
                const size_t a_d = (d / 64) * CL_ROWS_AROWS * 64 * 2, a_f = (F / 64) * CL_ROWS_AROWS * 64 * 2;
                DM(c->r_ax, a_d);
                DM(c->r_aatt, a_d);
                DM(c->r_ah, a_f);
                CU(cudaMemsetAsync(c->r_ax, 0, a_d, c->stream));
                CU(cudaMemsetAsync(c->r_aatt, 0, a_d, c->stream));
                CU(cudaMemsetAsync(c->r_ah, 0, a_f, c->stream));
                DM(c->r_ssq, (size_t)c->n_sm * CL_SLOTS * 4);
                DM(c->r_att_part, (size_t)cl_rows_att_part_floats(g.n_heads) * 4);
                DM(c->r_tickets, (size_t)g.n_heads * 4);
                CU(cudaMemsetAsync(c->r_tickets, 0, (size_t)g.n_heads * 4, c->stream));
                DM(c->r_head_part, (size_t)c->n_sm * CL_SLOTS * sizeof(ClHeadPartial));
                const char *ch = getenv("CL_ROWS_CHAIN");   // tuning knob
                c->rows_chain = (ch && ch[0]) ? atoi(ch) : 8;
                if (c->rows_chain < 1) c->rows_chain = 1;
                const char *en = getenv("CL_ROWS_ENTRY_KB");   // tuning knob
                c->rows_entry = ((en && en[0]) ? atoi(en) : 70) * 1024;   // (a third of the ring)
                if (c->rows_entry < 1024) c->rows_entry = 1024;
                if (c->rows_entry > 96 * 1024) c->rows_entry = 96 * 1024;   // (two entries must fit the ring of 192 KB)
                c->use_rows = 1;
            }
        }
        CU(cudaStreamSynchronize(c->stream));   // host staging vector and borrowed pointers are released after this
        if (stage_g) cudaFree(stage_g);
        if (stage_u) cudaFree(stage_u);
        {
            const char *nb = getenv("CL_DISABLE_ROW_SHARES");
            if (c->use_step && L > 0 && g.max_seq >= 2 && !(nb && nb[0] == '1')) {
                DM(c->cum_w_dev, ((size_t)c->n_sm + 1) * sizeof(float));
                DM(c->busy_dev, (size_t)c->n_sm * sizeof(unsigned long long));
                int rc = calibrate_row_shares(c);
                if (rc) return rc;
            }
        }
    } else {
        CU(cudaStreamSynchronize(c->stream));
    }
    c->loaded = 1;
    return CL_OK;
}

// Ring [L][taps][P][d]: where layer l's tap after the attention add (which = 0) or after the FFN add (which = 1) goes;
// null if that tap is not recorded.
static char *ring_slot(cl_ctx *c, int l, int which) {
    if (!c->ring || (c->taps == 1 && which == 0)) return nullptr;
    const size_t idx = (size_t)l * c->taps + (c->taps == 2 ? which : 0);
    return c->ring + idx * c->cfg.tap_positions * c->cfg.d_model * c->esz;
}

// ---- one pass of T rows through the kept layers ------------------------------------------------

static int gemv(cl_ctx *c, int T, int epi, const void *W, int rows, int cols, const float *xin, float *out, int ld) {
    ClGemvArgs a;
    memset(&a, 0, sizeof(a));
    a.W = W; a.rows = rows; a.cols = cols; a.xin = xin; a.out = out; a.ld = ld; a.st = c->st;
    const int ngroups = (rows + 1) / 2;
    int grid = (ngroups + 7) / 8;
    if (grid > c->n_sm * 4) grid = c->n_sm * 4;
    KL(cl_launch_gemv(c->cfg.weight_dtype, T, epi, a, grid, c->stream));
    return CL_OK;
}

static int head(cl_ctx *c, int T, const float *xin, const ClDevState *st, int *out_tok, float *out_pmax, float *out_conf,
                float *logits) {
    ClGemvArgs a;
    memset(&a, 0, sizeof(a));
    a.W = c->lm_head; a.rows = c->cfg.vocab; a.cols = c->cfg.d_model; a.xin = xin; a.st = st;
    a.logits = logits; a.partials = c->head_part; a.ticket = c->tickets;
    a.out_tok = out_tok; a.out_pmax = out_pmax; a.out_conf = out_conf;
    a.inv_log_v = (float)(1.0 / log((double)c->cfg.vocab));
    const int ngroups = (a.rows + 1) / 2;
    int grid = (ngroups + 7) / 8;
    if (grid > c->head_grid) grid = c->head_grid;
    KL(cl_launch_gemv(c->cfg.weight_dtype, T, CL_EPI_HEAD, a, grid, c->stream));
    return CL_OK;
}

// The same pass as one persistent launch on the tensor cores (16-bit models): all layers and the LM head.
static int forward_rows_persistent(cl_ctx *c, const int *tok, int T, int row0, int tap, int want_head, int *out_tok,
                                   float *out_pmax, float *out_conf, float *logits) {
    const cl_model_cfg &g = c->cfg;
    ClRowsArgs a;
    memset(&a, 0, sizeof(a));
    a.layers = c->rows_layers_dev; a.L = g.n_layers; a.head = c->head_tile; a.embed = c->embed; a.final_norm = c->final_norm;
    a.d = g.d_model; a.F = g.d_ffn; a.V = g.vocab; a.H = g.n_heads; a.Hkv = g.n_kv_heads; a.hd = g.head_dim; a.max_seq = g.max_seq;
    a.T = T; a.row0 = row0; a.want_head = want_head; a.f16 = g.weight_dtype == 2;
    a.att_parts = c->n_sm / g.n_heads;
    if (a.att_parts < 1) a.att_parts = 1;
    if (a.att_parts > 8) a.att_parts = 8;
    a.tap = tap && c->ring; a.tap_P = g.tap_positions;
    a.entry = c->rows_entry; a.chain = c->rows_chain; a.split = c->rows_split; a.ws = c->r_ws;
    a.eps = g.rms_eps; a.inv_d = 1.0f / (float)g.d_model; a.inv_log_v = (float)(1.0 / log((double)g.vocab));
    a.rope_cs = c->rope_cs; a.st = c->st; a.tok = tok;
    a.x = c->x; a.qkv = c->qkv; a.Ax = c->r_ax; a.Aatt = c->r_aatt; a.Ah = c->r_ah;
    a.ssq = c->r_ssq; a.att_part = c->r_att_part; a.att_tickets = c->r_tickets; a.head_part = c->r_head_part;
    a.logits = logits; a.out_tok = out_tok; a.out_pmax = out_pmax; a.out_conf = out_conf;
    a.sync = c->r_bar; a.bar_arrivals = (unsigned)(c->n_sm + c->bar_extra); a.wait_ns = c->wait_ns; a.phase_ns = c->r_phase_ns;
    a.c_ssq = c->r_c_ssq; a.c_ax = c->r_c_ax; a.c_ah = c->r_c_ah; a.c_att = c->r_c_att; a.c_qkv = c->r_c_qkv;
    CU(cudaMemsetAsync(c->r_bar, 0, (size_t)c->r_sync_words * 4, c->stream));   // every counter starts at zero
    KL(cl_launch_rows_pass(g.weight_dtype, g.head_dim, a, c->n_sm, c->stream));
    return CL_OK;
}

// tok: device pointer to the T token ids; rows sit at positions st->ctx + row0 + t.
static int forward_rows(cl_ctx *c, const int *tok, int T, int row0, const uint8_t *mask, int tap, int want_head,
                        int *out_tok, float *out_pmax, float *out_conf, float *logits) {
    const cl_model_cfg &g = c->cfg;
    const int d = g.d_model, F = g.d_ffn, wd = g.weight_dtype, qkv_rows = d + 2 * g.n_kv_heads * g.head_dim;
    int rc;
    if (c->use_rows && !mask) return forward_rows_persistent(c, tok, T, row0, tap, want_head, out_tok, out_pmax, out_conf, logits);
    KL(cl_launch_embed(wd, c->embed, tok, T, d, c->x, c->st, c->stream));
    for (int l = 0; l < g.n_layers; ++l) {
        const int skip_bits = mask ? mask[l] : 0;
        if (skip_bits == 3) continue;
        const ClLayer &y = c->layers[l];
        if (!(skip_bits & 1)) {
        // attention half: RMSNorm -> QKV -> rotary + cache append -> attention over the cache -> output projection + residual
        KL(cl_launch_rmsnorm(c->x, y.n1, T, d, g.rms_eps, c->xn, c->st, c->stream));
        if ((rc = gemv(c, T, CL_EPI_STORE, y.wqkv, qkv_rows, d, c->xn, c->qkv, qkv_rows))) return rc;
        KL(cl_launch_rope_append(wd, c->qkv, T, row0, g.n_heads, g.n_kv_heads, g.head_dim, d, c->rope_cs, y.kc, y.vc, g.max_seq, c->st,
                                 c->stream));
        ClAttnArgs a;
        a.q = c->qkv; a.ld_q = qkv_rows; a.n_kv_heads = g.n_kv_heads; a.kcache = y.kc; a.vcache = y.vc; a.part = c->att_part; a.tickets = c->tickets + 1;
        a.out = c->att; a.st = c->st; a.row0 = row0; a.n_heads = g.n_heads; a.head_dim = g.head_dim; a.d_model = d;
        a.nsplit = c->nsplit; a.per_max = c->per_max; a.max_seq = g.max_seq;
        KL(cl_launch_attn(wd, T, a, c->stream));
        if ((rc = gemv(c, T, CL_EPI_RESID, y.wo, d, d, c->att, c->x, d))) return rc;
        }
        if (tap && ring_slot(c, l, 0))
            KL(cl_launch_tap(wd, c->x, T, row0, d, ring_slot(c, l, 0), g.tap_positions, c->st, c->stream));
        if (!(skip_bits & 2)) {
        // FFN half: RMSNorm -> gate/up + SiLU -> down projection + residual
        KL(cl_launch_rmsnorm(c->x, y.n2, T, d, g.rms_eps, c->xn, c->st, c->stream));
        if ((rc = gemv(c, T, CL_EPI_SILU, y.wgu, 2 * F, d, c->xn, c->hff, F))) return rc;
        if ((rc = gemv(c, T, CL_EPI_RESID, y.wd, d, F, c->hff, c->x, d))) return rc;
        }
        if (tap && ring_slot(c, l, 1))
            KL(cl_launch_tap(wd, c->x, T, row0, d, ring_slot(c, l, 1), g.tap_positions, c->st, c->stream));
    }
    if (want_head) {
        KL(cl_launch_rmsnorm(c->x, c->final_norm, T, d, g.rms_eps, c->xn, c->st, c->stream));
        if ((rc = head(c, T, c->xn, c->st, out_tok, out_pmax, out_conf, logits))) return rc;
    }
    return CL_OK;
}

// The prompt pass over M <= CL_WIDE_MAX_M rows at positions ctx .. ctx + M - 1 (bf16 models): every matrix is one wide
// tensor-core GEMM whose product a small kernel consumes (rotary + cache append, residual add + RMSNorm, SiLU).
// Fills the KV cache and, when asked, the hidden taps; computes no logits (the caller runs the last prompt token
// through the T-row pass for those).
static int forward_wide(cl_ctx *c, const int *tok, int M, int tap) {
    const cl_model_cfg &g = c->cfg;
    const int d = g.d_model, F = g.d_ffn, L = g.n_layers, qkv_rows = d + 2 * g.n_kv_heads * g.head_dim;
    const int KBd = (d + 63) / 64, KBf = (F + 63) / 64, MT = (M + 127) / 128, lo0 = CL_WIDE_MAX_M;
    const int f16 = g.weight_dtype == 2;
    auto gemm = [&](const ClTensorMap &mapA, const ClTensorMap &mapB, int rows, int KB, int *splits) -> int {
        ClWideArgs a;
        a.M = M; a.rows = rows; a.KB = KB; a.MT = MT; a.NT = (rows + 255) / 256;
        a.splits = *splits = cl_wide_splits(M, rows, KB, c->n_sm, c->w_P_floats);
        a.lo_row0 = lo0; a.P = c->w_P; a.err = &c->st->err; a.f16 = f16;
        KL(cl_launch_wide(mapA, mapB, a, c->stream));
        return CL_OK;
    };
    ClWideNormArgs nb;
    memset(&nb, 0, sizeof(nb));
    nb.x = c->w_x; nb.M = M; nb.d = d; nb.eps = g.rms_eps; nb.A = c->w_ax; nb.lo_row0 = lo0; nb.st = c->st;
    nb.tap_P = g.tap_positions; nb.f16 = f16;
    {
        ClWideNormArgs n = nb;
        n.embed = c->embed; n.tok = tok; n.g = L ? c->layers[0].n1 : nullptr;
        KL(cl_launch_wide_norm(n, c->stream));
    }
    int rc, sp;
    for (int l = 0; l < L; ++l) {
        const ClLayer &y = c->layers[l];
        if ((rc = gemm(c->map_wx, c->map_qkv[l], qkv_rows, KBd, &sp))) return rc;
        KL(cl_launch_wide_rope_append(c->w_P, sp, M, g.n_heads, g.n_kv_heads, g.head_dim, d, c->rope_cs, y.kc, y.vc, g.max_seq,
                                      c->st, f16, c->stream));
        KL(cl_launch_attn_wide(c->w_P, qkv_rows, y.kc, y.vc, c->w_aatt, lo0, M, d, g.n_heads, g.n_kv_heads, g.head_dim,
                               g.max_seq, c->st, f16, c->stream));
        if ((rc = gemm(c->map_watt, c->map_o[l], d, KBd, &sp))) return rc;
        ClWideNormArgs n = nb;
        n.P = c->w_P; n.splits = sp; n.g = y.n2;
        if (tap) n.tap = ring_slot(c, l, 0);
        KL(cl_launch_wide_norm(n, c->stream));
        if ((rc = gemm(c->map_wx, c->map_gu[l], 2 * F, KBd, &sp))) return rc;
        KL(cl_launch_wide_silu(c->w_P, sp, M, F, c->w_ah, lo0, f16, c->stream));
        if ((rc = gemm(c->map_wh, c->map_d[l], d, KBf, &sp))) return rc;
        n = nb;
        n.P = c->w_P; n.splits = sp; n.g = (l + 1 < L) ? c->layers[l + 1].n1 : nullptr;
        if (tap) n.tap = ring_slot(c, l, 1);
        KL(cl_launch_wide_norm(n, c->stream));
    }
    return CL_OK;
}

// n_steps consecutive single-token steps in one persistent launch (draft steps with the skip set, or
// vanilla full-model steps that emit and advance on the device).
static int run_steps(cl_ctx *c, int mode, int n_steps, int row0, bool full_model, float *logits, int *out_tokens,
                     float stop_p = 0.f) {
    const cl_model_cfg &g = c->cfg;
    ClStepArgs a;
    memset(&a, 0, sizeof(a));
    a.layers = c->layers_dev;
    a.kept = full_model ? c->kept_all_dev : c->kept_dev;
    a.n_kept = full_model ? g.n_layers : c->n_kept;
    a.embed = c->embed; a.lm_head = c->lm_head; a.final_norm = c->final_norm;
    a.d = g.d_model; a.F = g.d_ffn; a.V = g.vocab; a.H = g.n_heads; a.Hkv = g.n_kv_heads; a.max_seq = g.max_seq;
    a.att_parts = c->att_parts; a.l2_ahead = c->l2_ahead;
    a.eps = g.rms_eps; a.inv_log_v = (float)(1.0 / log((double)g.vocab));
    a.rope_cs = c->rope_cs; a.st = c->st;
    a.x = c->x; a.qkv = c->qkv; a.hff = c->hff;
    a.att_part = c->att_part2; a.head_part = c->head_part2; a.bar = c->bar_dev;
    a.n_steps = n_steps; a.mode = mode; a.row0 = row0; a.out_tokens = out_tokens; a.logits = logits;
    a.wait_ns = c->wait_ns; a.bar_arrivals = (unsigned)(c->n_sm + c->bar_extra); a.stop_p = stop_p;
    a.cum_w = c->cum_w_ready ? c->cum_w_dev : nullptr;
    a.busy_ns = c->calibrating ? c->busy_dev : nullptr;
    CU(cudaMemsetAsync(c->bar_dev, 0, 2 * sizeof(unsigned), c->stream));   // the arrival counter starts at zero
    KL(cl_launch_token_steps(g.weight_dtype, g.head_dim, a, c->n_sm, c->stream));
    return CL_OK;
}

// After a synchronisation: did a bounded device-side wait expire?
static int check_device_err(cl_ctx *c, const char *fn) {
    if (c->h_st->err) {
        const int e = c->h_st->err;
        cudaMemsetAsync(c->bar_dev, 0, 2 * sizeof(unsigned), c->stream);
        cudaMemsetAsync(&c->st->err, 0, sizeof(int), c->stream);
        cudaStreamSynchronize(c->stream);
        return fail(c, CL_ETIMEOUT, "%s: a bounded device-side wait expired (flags %d); results of this call are invalid", fn, e);
    }
    return CL_OK;
}

static int need_model(cl_ctx *c, const char *fn, bool need_prefill) {
    if (!c) return fail(c, CL_EINVAL, "%s: null context", fn);
    if (!c->loaded) return fail(c, CL_ESTATE, "%s: no weights loaded", fn);
    if (c->head_only) return fail(c, CL_ESTATE, "%s: context was loaded head-only", fn);
    if (need_prefill && !c->prefilled) return fail(c, CL_ESTATE, "%s: call cl_prefill first", fn);
    return CL_OK;
}

// One-time measurement of how fast each CTA of the token-step kernel streams (its SM's path to HBM): two full-model
// steps from an empty cache are timed per CTA, the row shares are set in proportion to rows / time, and the measurement
// is repeated once with the new shares.  The shares stay fixed afterwards, so results do not depend on timing.
static int calibrate_row_shares(cl_ctx *c) {
    const int G = c->n_sm;
    std::vector<float> w((size_t)G, 1.0f / (float)G), cum((size_t)G + 1);
    std::vector<unsigned long long> busy((size_t)G);
    auto upload = [&]() -> cudaError_t {
        double acc = 0.0, tot = 0.0;
        for (float v : w) tot += v;
        cum[0] = 0.f;
        for (int b = 0; b < G; ++b) {
            acc += w[b] / tot;
            cum[b + 1] = (float)acc;
        }
        cum[G] = 1.0f;
        return cudaMemcpy(c->cum_w_dev, cum.data(), cum.size() * sizeof(float), cudaMemcpyHostToDevice);
    };
    CU(upload());
    c->cum_w_ready = 1;
    int rc = CL_OK;
    for (int pass = 0; pass < 3 && !rc; ++pass) {
        CU(cudaMemsetAsync(c->st, 0, sizeof(ClDevState), c->stream));
        CU(cudaMemsetAsync(c->busy_dev, 0, (size_t)G * sizeof(unsigned long long), c->stream));
        c->calibrating = pass > 0;   // pass 0 warms up
        rc = run_steps(c, CL_STEP_VANILLA, 2, 0, true, nullptr, nullptr);
        c->calibrating = 0;
        if (rc) break;
        CU(cudaStreamSynchronize(c->stream));
        if (pass == 0) continue;
        CU(cudaMemcpy(busy.data(), c->busy_dev, busy.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
        double mean = 0.0;
        for (unsigned long long t : busy) mean += (double)t;
        mean /= G;
        if (mean <= 0.0) break;
        for (int b = 0; b < G; ++b) {
            double f = busy[b] > 0 ? mean / (double)busy[b] : 1.0;   // faster CTA (less time for its share) -> larger share
            if (f < 0.8) f = 0.8;
            if (f > 1.25) f = 1.25;
            w[b] = (float)(w[b] * f);
        }
        CU(upload());
    }
    CU(cudaMemsetAsync(c->st, 0, sizeof(ClDevState), c->stream));
    CU(cudaStreamSynchronize(c->stream));
    return rc;
}

extern "C" int cl_prefill(cl_ctx *c, const int32_t *tokens, int n, int tap_hidden, int32_t *first_token) {
    int rc = need_model(c, "cl_prefill", false);
    if (rc) return rc;
    if (!tokens || n <= 0) return fail(c, CL_EINVAL, "cl_prefill: empty prompt");
    if (n + 1 > c->cfg.max_seq) return fail(c, CL_ERANGE, "cl_prefill: prompt of %d tokens exceeds max_seq %d", n, c->cfg.max_seq);
    for (int i = 0; i < n; ++i)
        if (tokens[i] < 0 || tokens[i] >= c->cfg.vocab) return fail(c, CL_EINVAL, "cl_prefill: token %d out of range at %d", tokens[i], i);
    CU(cudaMemcpyAsync(c->prompt_dev, tokens, (size_t)n * 4, cudaMemcpyHostToDevice, c->stream));
    if (tap_hidden && c->ring)   // a tapped prefill starts the context window afresh
        CU(cudaMemsetAsync(c->ring, 0, (size_t)c->cfg.n_layers * c->taps * c->cfg.tap_positions * c->cfg.d_model * c->esz, c->stream));
    ClPoke p = poke_none();
    p.ctx = 0; p.n_drafted = 0; p.done = 0;
    if ((rc = poke(c, p))) return rc;
    int c0 = 0;
    if (c->use_wide && n > 2 * CL_PREFILL_CHUNK) {
        // all prompt rows but the last go through the wide GEMMs; the last one takes the T-row pass, which has the LM head
        while (c0 < n - 1) {
            const int M = (n - 1 - c0 < CL_WIDE_MAX_M) ? n - 1 - c0 : CL_WIDE_MAX_M;
            if ((rc = forward_wide(c, c->prompt_dev + c0, M, tap_hidden))) return rc;
            KL(cl_launch_advance(c->st, M, 0, c->stream));
            c0 += M;
        }
    }
    for (; c0 < n; c0 += CL_PREFILL_CHUNK) {
        const int T = (n - c0 < CL_PREFILL_CHUNK) ? n - c0 : CL_PREFILL_CHUNK;
        const bool last = c0 + T >= n;
        rc = forward_rows(c, c->prompt_dev + c0, T, 0, nullptr, tap_hidden, last, ST_FIELD(c, int, tgt_tok),
                          ST_FIELD(c, float, v_pmax), ST_FIELD(c, float, v_conf), nullptr);
        if (rc) return rc;
        KL(cl_launch_advance(c->st, T, last ? 1 : 0, c->stream));
    }
    if ((rc = sync_state(c))) return rc;
    if ((rc = check_device_err(c, "cl_prefill"))) {
        c->prefilled = 0;   // the cache holds rows of an aborted pass
        return rc;
    }
    c->prefilled = 1;
    c->h_ndraft = 0;
    c->h_filled = n;
    c->tapped = tap_hidden ? n : 0;
    if (first_token) *first_token = c->h_st->cyc_tok[0];
    return CL_OK;
}

extern "C" int cl_set_skip_set(cl_ctx *c, const uint8_t *mask) {
    if (!c || !mask) return fail(c, CL_EINVAL, "cl_set_skip_set: null argument");
    for (int l = 0; l < c->cfg.n_layers; ++l)
        if (mask[l] > 3) return fail(c, CL_EINVAL, "cl_set_skip_set: layer %d has mask %d; bits 0 and 1 only", l, mask[l]);
    c->mask.assign(mask, mask + c->cfg.n_layers);
    if (c->kept_dev) {
        std::vector<int> kept;
        for (int l = 0; l < c->cfg.n_layers; ++l)
            if (mask[l] != 3) kept.push_back(l | ((int)mask[l] << 16));
        CU(cudaStreamSynchronize(c->stream));
        if (!kept.empty()) CU(cudaMemcpy(c->kept_dev, kept.data(), kept.size() * sizeof(int), cudaMemcpyHostToDevice));
        c->n_kept = (int)kept.size();
    }
    return CL_OK;
}

extern "C" int cl_get_skip_set(cl_ctx *c, uint8_t *mask) {
    if (!c || !mask) return fail(c, CL_EINVAL, "cl_get_skip_set: null argument");
    memcpy(mask, c->mask.data(), c->mask.size());
    return CL_OK;
}

extern "C" int cl_draft(cl_ctx *c, int K, float stop_p, int32_t *toks, float *p_max, float *conf, float *logits,
                        int *n_drafted) {
    int rc = need_model(c, "cl_draft", true);
    if (rc) return rc;
    if (K < 1 || K > CL_MAX_K) return fail(c, CL_ERANGE, "cl_draft: K = %d outside 1..%d", K, CL_MAX_K);
    if (c->h_ctx + K + 1 > c->cfg.max_seq) return fail(c, CL_ERANGE, "cl_draft: position %d exceeds max_seq", c->h_ctx + K);
    int n = 0;
    if (c->use_step) {
        // one persistent launch; with stop_p > 0 the kernel itself ends the drafting and records how far it got
        if ((rc = run_steps(c, CL_STEP_DRAFT, K, 0, false, logits ? c->logits : nullptr, nullptr, stop_p > 0.f ? stop_p : 0.f)))
            return rc;
        if ((rc = sync_state(c))) return rc;
        n = c->h_st->n_drafted;
    } else {
        for (int i = 0; i < K; ++i) {
            float *lg = logits ? c->logits + (size_t)i * c->cfg.vocab : nullptr;
            rc = forward_rows(c, ST_FIELD(c, int, cyc_tok) + i, 1, i, c->mask.data(), 0, 1,
                              ST_FIELD(c, int, cyc_tok) + i + 1, ST_FIELD(c, float, d_pmax) + i,
                              ST_FIELD(c, float, d_conf) + i, lg);
            if (rc) return rc;
            n = i + 1;
            if (stop_p > 0.f) {   // confidence-aware early stop needs the probability on the host
                if ((rc = sync_state(c))) return rc;
                if (c->h_st->d_pmax[i] < stop_p) break;
            }
        }
        ClPoke p = poke_none();
        p.n_drafted = n;
        if ((rc = poke(c, p))) return rc;
        if ((rc = sync_state(c))) return rc;
    }
    if ((rc = check_device_err(c, "cl_draft"))) return rc;
    if (n < 1 || n > K) return fail(c, CL_ECUDA, "cl_draft: the device reported %d drafted tokens", n);
    c->h_ndraft = n;
    if (logits) CU(cudaMemcpy(logits, c->logits, (size_t)n * c->cfg.vocab * 4, cudaMemcpyDeviceToHost));
    for (int i = 0; i < n; ++i) {
        if (toks) toks[i] = c->h_st->cyc_tok[1 + i];
        if (p_max) p_max[i] = c->h_st->d_pmax[i];
        if (conf) conf[i] = c->h_st->d_conf[i];
    }
    if (n_drafted) *n_drafted = n;
    return CL_OK;
}

extern "C" int cl_force_tokens(cl_ctx *c, const int32_t *toks, int n) {
    int rc = need_model(c, "cl_force_tokens", true);
    if (rc) return rc;
    if (n < 0 || n > CL_MAX_K || (n > 0 && !toks)) return fail(c, CL_ERANGE, "cl_force_tokens: n = %d outside 0..%d", n, CL_MAX_K);
    if (c->h_ctx + n + 1 > c->cfg.max_seq) return fail(c, CL_ERANGE, "cl_force_tokens: position exceeds max_seq");
    ClPoke p = poke_none();
    p.n_drafted = n;
    p.n_force = n;
    for (int i = 0; i < n; ++i) {
        if (toks[i] < 0 || toks[i] >= c->cfg.vocab) return fail(c, CL_EINVAL, "cl_force_tokens: token out of range");
        p.force[i] = toks[i];
    }
    if ((rc = poke(c, p))) return rc;
    c->h_ndraft = n;
    return CL_OK;
}

extern "C" int cl_verify(cl_ctx *c, int tap_hidden, int32_t *target_toks, float *logits) {
    int rc = need_model(c, "cl_verify", true);
    if (rc) return rc;
    const int T = c->h_ndraft + 1;
    if (c->h_ctx + T > c->cfg.max_seq) return fail(c, CL_ERANGE, "cl_verify: position exceeds max_seq");
    rc = forward_rows(c, ST_FIELD(c, int, cyc_tok), T, 0, nullptr, tap_hidden, 1, ST_FIELD(c, int, tgt_tok),
                      ST_FIELD(c, float, v_pmax), ST_FIELD(c, float, v_conf), logits ? c->logits : nullptr);
    if (rc) return rc;
    if ((rc = sync_state(c))) return rc;
    if ((rc = check_device_err(c, "cl_verify"))) return rc;   // target tokens of an aborted pass are never handed out
    if (c->h_ctx + T > c->h_filled) c->h_filled = c->h_ctx + T;
    if (tap_hidden) c->tapped += 1;
    if (logits) CU(cudaMemcpy(logits, c->logits, (size_t)T * c->cfg.vocab * 4, cudaMemcpyDeviceToHost));
    if (target_toks)
        for (int i = 0; i < T; ++i) target_toks[i] = c->h_st->tgt_tok[i];
    return CL_OK;
}

extern "C" int cl_accept(cl_ctx *c, int *n_accepted, int32_t *emitted) {
    int rc = need_model(c, "cl_accept", true);
    if (rc) return rc;
    // an error flag left by an earlier pass means its target tokens are invalid: nothing is committed
    if ((rc = sync_state(c))) return rc;
    if ((rc = check_device_err(c, "cl_accept"))) return rc;
    KL(cl_launch_accept(c->st, -1, nullptr, c->stream));
    if ((rc = sync_state(c))) return rc;
    c->h_ndraft = 0;
    const int n = c->h_st->n_acc_last;
    if (n_accepted) *n_accepted = n;
    if (emitted)
        for (int i = 0; i <= n; ++i) emitted[i] = c->h_st->emitted[i];
    return CL_OK;
}

extern "C" int cl_step_vanilla(cl_ctx *c, int32_t *tok) {
    int rc = need_model(c, "cl_step_vanilla", true);
    if (rc) return rc;
    if (c->h_ctx + 1 > c->cfg.max_seq) return fail(c, CL_ERANGE, "cl_step_vanilla: position exceeds max_seq");
    ClPoke p = poke_none();
    p.n_drafted = 0;
    if ((rc = poke(c, p))) return rc;
    if (c->use_step) {
        if ((rc = run_steps(c, CL_STEP_VANILLA, 1, 0, true, nullptr, nullptr))) return rc;
    } else {
        rc = forward_rows(c, ST_FIELD(c, int, cyc_tok), 1, 0, nullptr, 0, 1, ST_FIELD(c, int, tgt_tok),
                          ST_FIELD(c, float, v_pmax), ST_FIELD(c, float, v_conf), nullptr);
        if (rc) return rc;
        KL(cl_launch_accept(c->st, 0, nullptr, c->stream));
    }
    if ((rc = sync_state(c))) return rc;
    if ((rc = check_device_err(c, "cl_step_vanilla"))) return rc;
    if (c->h_ctx > c->h_filled) c->h_filled = c->h_ctx;
    c->h_ndraft = 0;
    if (tok) *tok = c->h_st->emitted[0];
    return CL_OK;
}

static int enqueue_cycle(cl_ctx *c, int K, int tap = 0) {
    int rc;
    if (c->use_step && K > 0) {
        if ((rc = run_steps(c, CL_STEP_DRAFT, K, 0, false, nullptr, nullptr))) return rc;
    } else {
        for (int i = 0; i < K; ++i) {
            rc = forward_rows(c, ST_FIELD(c, int, cyc_tok) + i, 1, i, c->mask.data(), 0, 1,
                              ST_FIELD(c, int, cyc_tok) + i + 1, ST_FIELD(c, float, d_pmax) + i,
                              ST_FIELD(c, float, d_conf) + i, nullptr);
            if (rc) return rc;
        }
    }
    rc = forward_rows(c, ST_FIELD(c, int, cyc_tok), K + 1, 0, nullptr, tap, 1, ST_FIELD(c, int, tgt_tok),
                      ST_FIELD(c, float, v_pmax), ST_FIELD(c, float, v_conf), nullptr);
    if (rc) return rc;
    KL(cl_launch_accept(c->st, K, c->out_dev, c->stream));
    return CL_OK;
}

extern "C" int cl_generate(cl_ctx *c, int K, int max_new, int32_t *out, int *n_out, cl_stats *stats) {
    int rc = need_model(c, "cl_generate", true);
    if (rc) return rc;
    if (K < 0 || K > CL_MAX_K) return fail(c, CL_ERANGE, "cl_generate: K = %d outside 0..%d", K, CL_MAX_K);
    if (max_new <= 0 || !out) return fail(c, CL_EINVAL, "cl_generate: nothing to generate");
    if (c->h_ctx + max_new + K > c->cfg.max_seq)
        return fail(c, CL_ERANGE, "cl_generate: %d + %d + %d tokens exceed max_seq %d", c->h_ctx, max_new, K, c->cfg.max_seq);
    if (max_new > c->out_cap) {
        if (c->out_dev) cudaFree(c->out_dev);
        c->out_dev = nullptr;
        c->out_cap = 0;
        DM(c->out_dev, (size_t)max_new * 4);
        c->out_cap = max_new;
    }
    ClPoke p = poke_none();
    p.n_out = 0; p.max_new = max_new; p.done = 0; p.n_drafted = 0;
    if ((rc = poke(c, p))) return rc;
    int remaining = max_new;
    if (K == 0 && c->use_step) {
        // vanilla decoding: all max_new steps in one persistent launch, tokens emitted on the device
        if ((rc = run_steps(c, CL_STEP_VANILLA, max_new, 0, true, nullptr, c->out_dev))) return rc;
        if ((rc = sync_state(c))) return rc;
        remaining = 0;
    }
    while (remaining > 0) {
        // the fewest cycles that can finish the job; cycles enqueued past the end exit at once on the device
        const int ncyc = (remaining + K) / (K + 1);
        for (int i = 0; i < ncyc; ++i)
            if ((rc = enqueue_cycle(c, K))) return rc;
        if ((rc = sync_state(c))) return rc;
        remaining = max_new - c->h_st->n_out;
    }
    if ((rc = check_device_err(c, "cl_generate"))) return rc;
    CU(cudaMemcpy(out, c->out_dev, (size_t)max_new * 4, cudaMemcpyDeviceToHost));
    p = poke_none();
    p.done = 0;
    if ((rc = poke(c, p))) return rc;
    if ((rc = sync_state(c))) return rc;
    if (c->h_ctx > c->h_filled) c->h_filled = c->h_ctx;
    c->h_ndraft = 0;
    if (n_out) *n_out = max_new;
    if (stats) cl_get_stats(c, stats);
    return CL_OK;
}

static int check_select(cl_ctx *c, const cl_select_cfg *s);
static int ensure_sel_iters(cl_ctx *c, int iters);
static int score_rows(cl_ctx *c, const void *hidden, int rows, int P, float *c_layer_dev);
static int score_device_err(cl_ctx *c, const char *fn);

// Generation with the interval-based periodic search of Section 3.3.  Host logic only: the cycles of an interval
// are enqueued back to back (no host round trip inside an interval), the search check reads the device counters
// once per interval, and scoring / selection run in the kernels of cl_layer_confidences / cl_select_skip_set.
extern "C" int cl_generate_search(cl_ctx *c, const cl_search_cfg *sc, const cl_select_cfg *sel, int max_new, int32_t *out,
                                  int *n_out, cl_search_report *rep, uint8_t *masks) {
    int rc = need_model(c, "cl_generate_search", true);
    if (rc) return rc;
    if (!sc || !sel || !out || max_new <= 0) return fail(c, CL_EINVAL, "cl_generate_search: null argument or nothing to generate");
    const int K = sc->K, L = c->cfg.n_layers, P = c->cfg.tap_positions;
    if (K < 1 || K > CL_MAX_K) return fail(c, CL_ERANGE, "cl_generate_search: K = %d outside 1..%d", K, CL_MAX_K);
    if (sc->interval < 1 || sc->max_rounds < 0 || sc->max_rounds > CL_MAX_ROUNDS)
        return fail(c, CL_ERANGE, "cl_generate_search: interval >= 1 and 0 <= max_rounds <= %d required", CL_MAX_ROUNDS);
    if (!c->ring) return fail(c, CL_ESTATE, "cl_generate_search: the context has no hidden-state ring (tap_positions = 0)");
    if (c->tapped <= 0)
        return fail(c, CL_ESTATE, "cl_generate_search: the ring holds no rows of this input; call cl_prefill with tap_hidden = 1");
    if (c->h_ctx + max_new + K > c->cfg.max_seq)
        return fail(c, CL_ERANGE, "cl_generate_search: %d + %d + %d tokens exceed max_seq %d", c->h_ctx, max_new, K, c->cfg.max_seq);
    if ((rc = check_select(c, sel))) return rc;
    if ((rc = ensure_sel_iters(c, 1))) return rc;
    if (max_new > c->out_cap) {
        if (c->out_dev) cudaFree(c->out_dev);
        c->out_dev = nullptr;
        c->out_cap = 0;
        DM(c->out_dev, (size_t)max_new * 4);
        c->out_cap = max_new;
    }
    ClPoke p = poke_none();
    p.n_out = 0; p.max_new = max_new; p.done = 0; p.n_drafted = 0;
    if ((rc = poke(c, p))) return rc;
    if ((rc = sync_state(c))) return rc;
    cl_search_report r;
    memset(&r, 0, sizeof(r));
    r.searching = 1;
    std::vector<uint8_t> best(c->mask), cur(c->mask);
    float best_score = -INFINITY;
    int rnd = 0;
    while (c->h_st->n_out < max_new) {
        const int remaining = max_new - c->h_st->n_out;
        const unsigned long long cyc0 = c->h_st->cycles, acc0 = c->h_st->accepted;
        // while searching: one interval; afterwards: the fewest cycles that can finish (cycles past the end exit at once)
        const int ncyc = r.searching ? sc->interval : (remaining + K) / (K + 1);
        // Taps while searching: every cycle advances by at least one position, so the last P cycles of an interval rewrite
        // every slot of the ring (slot = position mod P); what earlier cycles would record is gone by the search check.
        for (int i = 0; i < ncyc; ++i)
            if ((rc = enqueue_cycle(c, K, r.searching && ncyc - i <= P))) return rc;
        const int ctx_before = c->h_ctx;
        if ((rc = sync_state(c))) return rc;
        if ((rc = check_device_err(c, "cl_generate_search"))) return rc;
        if (r.searching) c->tapped += c->h_ctx - ctx_before;   // every verify pass of the interval recorded its rows
        if (!r.searching || (int)(c->h_st->cycles - cyc0) < sc->interval) continue;   // no full interval: nothing to check
        // ---- search check (Section 3.3)
        const float score = (float)((double)(c->h_st->accepted - acc0) / (double)sc->interval);
        r.scores[rnd] = score;
        if (masks) memcpy(masks + (size_t)rnd * L, cur.data(), (size_t)L);
        r.n_scored = rnd + 1;
        if (score > best_score) {
            best_score = score;
            best = cur;
            r.best_round = rnd;
        }
        if (score >= sc->score_goal || rnd >= sc->max_rounds) {
            r.searching = 0;
            cur = best;
        } else {
            if (c->tapped < P)   // slots never written would enter the per-layer mean as zero vectors
                return fail(c, CL_ESTATE, "cl_generate_search: the ring holds %d of %d positions at a search check; use a longer prompt or interval",
                            c->tapped, P);
            if ((rc = score_rows(c, c->ring, L, c->taps * P, c->sc_clayer))) return rc;
            KL(cl_launch_select(*sel, L, c->sc_clayer, c->sel_mask, nullptr, c->stream));
            CU(cudaMemcpyAsync(cur.data(), c->sel_mask, (size_t)L, cudaMemcpyDeviceToHost, c->stream));
            CU(cudaStreamSynchronize(c->stream));
            if ((rc = score_device_err(c, "cl_generate_search"))) return rc;
            ++rnd;
        }
        if ((rc = cl_set_skip_set(c, cur.data()))) return rc;
    }
    CU(cudaMemcpy(out, c->out_dev, (size_t)max_new * 4, cudaMemcpyDeviceToHost));
    p = poke_none();
    p.done = 0;
    if ((rc = poke(c, p))) return rc;
    if ((rc = sync_state(c))) return rc;
    if (c->h_ctx > c->h_filled) c->h_filled = c->h_ctx;
    c->h_ndraft = 0;
    if (n_out) *n_out = max_new;
    if (rep) *rep = r;
    return CL_OK;
}

extern "C" int cl_rollback(cl_ctx *c, int ctx_len, int32_t pending_token) {
    int rc = need_model(c, "cl_rollback", true);
    if (rc) return rc;
    if (ctx_len < 0 || ctx_len > c->cfg.max_seq - 1) return fail(c, CL_ERANGE, "cl_rollback: ctx_len %d out of range", ctx_len);
    if (ctx_len > c->h_filled)   // rolling forward would make later passes attend over cache rows that were never written
        return fail(c, CL_ERANGE, "cl_rollback: ctx_len %d beyond the %d positions the cache holds", ctx_len, c->h_filled);
    if (pending_token < 0 || pending_token >= c->cfg.vocab) return fail(c, CL_EINVAL, "cl_rollback: token out of range");
    ClPoke p = poke_none();
    p.ctx = ctx_len; p.pending = pending_token; p.n_drafted = 0; p.done = 0;
    if ((rc = poke(c, p))) return rc;
    if ((rc = sync_state(c))) return rc;
    c->h_ndraft = 0;
    return CL_OK;
}

// ---- confidence scoring and selection -----------------------------------------------------------

static int ensure_score_cap(cl_ctx *c, size_t n) {
    if (n <= c->sc_cap) return CL_OK;
    void *old[] = {c->sc_conf, c->sc_pmax, c->sc_arg, c->sc_xn, c->sc_part};
    for (void *q : old)
        if (q) cudaFree(q);
    c->sc_conf = c->sc_pmax = nullptr;
    c->sc_arg = nullptr;
    c->sc_xn = nullptr;
    c->sc_part = nullptr;
    c->sc_cap = 0;
    DM(c->sc_conf, n * 4);
    DM(c->sc_pmax, n * 4);
    DM(c->sc_arg, n * 4);
    if (c->cfg.weight_dtype != 0) {
        DM(c->sc_xn, n * (size_t)c->cfg.d_model * 2);
        DM(c->sc_part, cl_score_tc_partials((int)n, c->n_sm) * sizeof(ClHeadPartial));
    }
    c->sc_cap = n;
    return CL_OK;
}

// After a synchronisation: did a bounded wait of the scoring kernel expire?
static int score_device_err(cl_ctx *c, const char *fn) {
    int e = 0;
    if (cudaMemcpy(&e, &c->st->err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return fail(c, CL_ECUDA, "%s: reading the device error flag failed", fn);
    if (e) {
        cudaMemset(&c->st->err, 0, sizeof(int));
        return fail(c, CL_ETIMEOUT, "%s: a bounded device-side wait expired (flags %d); results of this call are invalid", fn, e);
    }
    return CL_OK;
}

// Scores rows*P hidden rows; leaves conf / p_max / argmax in the scoring scratch and the per-layer mean in c_layer_dev.
static int score_rows(cl_ctx *c, const void *hidden, int rows, int P, float *c_layer_dev) {
    const size_t n = (size_t)rows * P, d = c->cfg.d_model;
    int rc = ensure_score_cap(c, n);
    if (rc) return rc;
    if (c->cfg.weight_dtype != 0) {
        // 16-bit head: one dense contraction on the tensor cores with the softmax statistics fused into its epilogue
        if (((uintptr_t)hidden & 15u) != 0 || d % 8 != 0)
            return fail(c, CL_EINVAL, "confidence scoring: hidden rows must be 16-byte aligned and d_model a multiple of 8");
        const int f16 = c->cfg.weight_dtype == 2;
        KL(cl_launch_rmsnorm_bf16(c->cfg.weight_dtype, hidden, c->final_norm, (int)n, (int)d, c->cfg.rms_eps, c->sc_xn, f16, c->stream));
        KL(cl_launch_score_tc(c->sc_xn, c->lm_head, (int)n, c->cfg.vocab, (int)d, c->sc_part, c->n_sm, &c->st->err, c->sc_conf,
                              c->sc_pmax, c->sc_arg, f16, c->stream));
        ++c->launches;
        KL(cl_launch_mean_rows(c->sc_conf, rows, P, c_layer_dev, c->stream));
        return CL_OK;
    }
    for (size_t r0 = 0; r0 < n; r0 += 8) {
        const int T = (n - r0 < 8) ? (int)(n - r0) : 8;
        KL(cl_launch_rmsnorm_rows(c->cfg.weight_dtype, (const char *)hidden + r0 * d * c->esz, c->final_norm, T, (int)d,
                                  c->cfg.rms_eps, c->xn, c->stream));
        if ((rc = head(c, T, c->xn, nullptr, c->sc_arg + r0, c->sc_pmax + r0, c->sc_conf + r0, nullptr))) return rc;
    }
    KL(cl_launch_mean_rows(c->sc_conf, rows, P, c_layer_dev, c->stream));
    return CL_OK;
}

extern "C" int cl_layer_confidences(cl_ctx *c, const void *hidden, int rows, int P, float *conf_rows, float *p_max,
                                    int32_t *argmax, float *c_layer) {
    if (!c) return fail(c, CL_EINVAL, "cl_layer_confidences: null context");
    if (!c->loaded) return fail(c, CL_ESTATE, "cl_layer_confidences: no weights loaded");
    if (!hidden) {
        if (!c->ring) return fail(c, CL_ESTATE, "cl_layer_confidences: no hidden-state ring (tap_positions = 0)");
        if (c->tapped < c->cfg.tap_positions)
            return fail(c, CL_ESTATE, "cl_layer_confidences: ring holds %d of %d positions", c->tapped, c->cfg.tap_positions);
        hidden = c->ring;
        rows = c->cfg.n_layers;
        P = c->taps * c->cfg.tap_positions;   // a layer's taps are contiguous: its confidence is the mean over taps and positions
    }
    if (rows <= 0 || P <= 0) return fail(c, CL_EINVAL, "cl_layer_confidences: rows and P must be positive");
    if (rows > c->cfg.n_layers && c->cfg.n_layers > 0) {
        // c_layer scratch is sized by n_layers; larger row counts use a temporary
    }
    float *cl_dev = c->sc_clayer;
    float *tmp = nullptr;
    if (rows > (c->cfg.n_layers ? c->cfg.n_layers : 1)) {
        DM(tmp, (size_t)rows * 4);
        cl_dev = tmp;
    }
    int rc = score_rows(c, hidden, rows, P, cl_dev);
    if (!rc) {
        const size_t n = (size_t)rows * P;
        cudaError_t e = cudaStreamSynchronize(c->stream);
        if (e == cudaSuccess) rc = score_device_err(c, "cl_layer_confidences");
        if (e == cudaSuccess && conf_rows) e = cudaMemcpy(conf_rows, c->sc_conf, n * 4, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess && p_max) e = cudaMemcpy(p_max, c->sc_pmax, n * 4, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess && argmax) e = cudaMemcpy(argmax, c->sc_arg, n * 4, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess && c_layer) e = cudaMemcpy(c_layer, cl_dev, (size_t)rows * 4, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) rc = fail(c, CL_ECUDA, "cl_layer_confidences: %s", cudaGetErrorString(e));
    }
    if (tmp) cudaFree(tmp);
    return rc;
}

static int check_select(cl_ctx *c, const cl_select_cfg *s) {
    if (!s) return fail(c, CL_EINVAL, "selection config is null");
    if (s->lo < 0 || s->hi >= c->cfg.n_layers || s->hi - s->lo + 1 > 256)
        return fail(c, CL_EINVAL, "selection range %d..%d outside the model's %d layers (or more than 256 eligible)", s->lo, s->hi, c->cfg.n_layers);
    return CL_OK;
}

static int ensure_sel_iters(cl_ctx *c, int iters) {
    if (iters <= c->sel_iters_cap) return CL_OK;
    if (c->sel_mask) cudaFree(c->sel_mask);
    if (c->sel_clayers) cudaFree(c->sel_clayers);
    c->sel_mask = nullptr;
    c->sel_clayers = nullptr;
    c->sel_iters_cap = 0;
    const size_t L = c->cfg.n_layers ? c->cfg.n_layers : 1;
    DM(c->sel_mask, (size_t)iters * L);
    DM(c->sel_clayers, (size_t)iters * L * 4);
    c->sel_iters_cap = iters;
    return CL_OK;
}

extern "C" int cl_select_skip_set(cl_ctx *c, const cl_select_cfg *s, const float *c_layer, uint8_t *mask, double *margins) {
    if (!c || !mask) return fail(c, CL_EINVAL, "cl_select_skip_set: null argument");
    if (!c->loaded) return fail(c, CL_ESTATE, "cl_select_skip_set: no weights loaded");
    int rc = check_select(c, s);
    if (rc) return rc;
    if ((rc = ensure_sel_iters(c, 1))) return rc;
    const int L = c->cfg.n_layers;
    if (c_layer) CU(cudaMemcpyAsync(c->sc_clayer, c_layer, (size_t)L * 4, cudaMemcpyHostToDevice, c->stream));
    KL(cl_launch_select(*s, L, c->sc_clayer, c->sel_mask, c->sel_margins, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    CU(cudaMemcpy(mask, c->sel_mask, (size_t)L, cudaMemcpyDeviceToHost));
    if (margins) CU(cudaMemcpy(margins, c->sel_margins, (size_t)L * sizeof(double), cudaMemcpyDeviceToHost));
    return CL_OK;
}

extern "C" int cl_score_loop(cl_ctx *c, const cl_select_cfg *s, const void *const *hidden_iters, int iters, int P,
                             const float *scores, uint8_t *best_mask, int *best_iter, uint8_t *masks_all,
                             float *c_layers_all) {
    if (!c || !hidden_iters || !scores || iters <= 0 || P <= 0) return fail(c, CL_EINVAL, "cl_score_loop: bad argument");
    if (!c->loaded) return fail(c, CL_ESTATE, "cl_score_loop: no weights loaded");
    int rc = check_select(c, s);
    if (rc) return rc;
    if ((rc = ensure_sel_iters(c, iters))) return rc;
    const int L = c->cfg.n_layers;
    for (int it = 0; it < iters; ++it) {
        if (!hidden_iters[it]) return fail(c, CL_EINVAL, "cl_score_loop: hidden_iters[%d] is null", it);
        float *cl_dev = c->sel_clayers + (size_t)it * L;
        if ((rc = score_rows(c, hidden_iters[it], L, P, cl_dev))) return rc;
        KL(cl_launch_select(*s, L, cl_dev, c->sel_mask + (size_t)it * L, nullptr, c->stream));
    }
    std::vector<uint8_t> all((size_t)iters * L);
    CU(cudaMemcpyAsync(all.data(), c->sel_mask, all.size(), cudaMemcpyDeviceToHost, c->stream));
    CU(cudaStreamSynchronize(c->stream));
    if ((rc = score_device_err(c, "cl_score_loop"))) return rc;
    if (c_layers_all) CU(cudaMemcpy(c_layers_all, c->sel_clayers, (size_t)iters * L * 4, cudaMemcpyDeviceToHost));
    int best = 0;   // round with the highest score; the earliest wins ties
    for (int it = 1; it < iters; ++it)
        if (scores[it] > scores[best]) best = it;
    if (best_iter) *best_iter = best;
    if (best_mask) memcpy(best_mask, all.data() + (size_t)best * L, (size_t)L);
    if (masks_all) memcpy(masks_all, all.data(), all.size());
    return CL_OK;
}

extern "C" int cl_read_hidden_ring(cl_ctx *c, void *out) {
    if (!c || !out) return fail(c, CL_EINVAL, "cl_read_hidden_ring: null argument");
    if (!c->ring) return fail(c, CL_ESTATE, "cl_read_hidden_ring: no ring (tap_positions = 0 or head-only context)");
    CU(cudaStreamSynchronize(c->stream));
    CU(cudaMemcpy(out, c->ring, (size_t)c->cfg.n_layers * c->taps * c->cfg.tap_positions * c->cfg.d_model * c->esz, cudaMemcpyDeviceToHost));
    return CL_OK;
}

extern "C" int cl_debug_set(cl_ctx *c, int what, long long value) {
    if (!c) return fail(c, CL_EINVAL, "cl_debug_set: null context");
    switch (what) {
        case CL_DEBUG_WAIT_LIMIT_US:
            if (value < 1) return fail(c, CL_EINVAL, "cl_debug_set: wait limit must be at least 1 us");
            c->wait_ns = (unsigned long long)value * 1000ull;
            return CL_OK;
        case CL_DEBUG_BARRIER_EXTRA:
            if (value < 0 || value > 1024) return fail(c, CL_EINVAL, "cl_debug_set: extra arrivals outside 0..1024");
            c->bar_extra = (int)value;
            return CL_OK;
        case CL_DEBUG_DEVICE_ERR: {
            if (!c->loaded) return fail(c, CL_ESTATE, "cl_debug_set: no weights loaded");
            const int flags = (int)value;
            CU(cudaMemcpyAsync(&c->st->err, &flags, sizeof(int), cudaMemcpyHostToDevice, c->stream));
            CU(cudaStreamSynchronize(c->stream));
            return CL_OK;
        }
        default:
            return fail(c, CL_EINVAL, "cl_debug_set: unknown setting %d", what);
    }
}

extern "C" int cl_debug_read(cl_ctx *c, int what, void *out, int n) {
    if (!c || !out) return fail(c, CL_EINVAL, "cl_debug_read: null argument");
    if (what == CL_DEBUG_ROWS_PHASE_NS) {
        if (!c->use_rows) return fail(c, CL_ESTATE, "cl_debug_read: this context does not run the persistent T-row pass");
        if (n < c->n_sm * 8) return fail(c, CL_ERANGE, "cl_debug_read: room for %d values needed", c->n_sm * 8);
        if (!c->r_phase_ns) {   // first call: switch the recording on; the next passes fill it
            DM(c->r_phase_ns, (size_t)c->n_sm * 8 * sizeof(unsigned long long));
            CU(cudaMemset(c->r_phase_ns, 0, (size_t)c->n_sm * 8 * sizeof(unsigned long long)));
        }
        CU(cudaStreamSynchronize(c->stream));
        CU(cudaMemcpy(out, c->r_phase_ns, (size_t)c->n_sm * 8 * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
        return CL_OK;
    }
    return fail(c, CL_EINVAL, "cl_debug_read: unknown item %d", what);
}

extern "C" int cl_get_stats(cl_ctx *c, cl_stats *out) {
    if (!c || !out) return fail(c, CL_EINVAL, "cl_get_stats: null argument");
    memset(out, 0, sizeof(*out));
    if (c->loaded && c->h_st) {
        int rc = sync_state(c);
        if (rc) return rc;
        out->cycles = c->h_st->cycles;
        out->drafted = c->h_st->drafted;
        out->accepted = c->h_st->accepted;
        out->emitted = c->h_st->emitted_total;
        out->ctx_len = c->h_st->ctx;
    }
    for (uint8_t m : c->mask) out->n_skipped += (m == 3);   // whole layers (half-skipped layers are not counted)
    out->kernel_launches = c->launches;
    return CL_OK;
}
