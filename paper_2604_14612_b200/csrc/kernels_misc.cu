// Small kernels around the weight-streaming ones: embedding gather, RMSNorm, rotary embedding +
// KV-cache append, KV-cache decode attention (split over the context, warp-shuffle reductions),
// hidden-state taps, greedy acceptance, and the adaptive-window skip-set selection (Eq. 5-10).
#include <math.h>

#include "cl_internal.h"

namespace {

template <typename ST>
__device__ __forceinline__ float to_f32(ST v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <>
__device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }
template <typename ST>
__device__ __forceinline__ ST from_f32(float v);
template <>
__device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }
template <>
__device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float block_sum(float v, float *sm) {
    // fixed-order block reduction (deterministic): warp shuffles, then warp 0 over the warp totals
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    __syncthreads();
    if (lane == 0) sm[warp] = v;
    __syncthreads();
    float r = 0.f;
    for (int w = 0; w < nw; ++w) r += sm[w];
    return r;
}

// ---- embedding gather: x[t] = E[token[t]] -------------------------------------------------
template <typename ST>
__global__ void k_embed(const ST *embed, const int *tok, int d, float *x, const ClDevState *st) {
    if (st->done) return;
    const int t = blockIdx.x;
    const ST *row = embed + (size_t)tok[t] * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) x[(size_t)t * d + i] = to_f32<ST>(row[i]);
}

// ---- RMSNorm: out = x * rsqrt(mean(x^2) + eps) * g ----------------------------------------
template <typename ST>
__global__ void k_rmsnorm(const ST *x, const float *g, int d, float eps, float *out, const ClDevState *st) {
    if (st && st->done) return;
    __shared__ float sm[32];
    const int t = blockIdx.x;
    const ST *xr = x + (size_t)t * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = to_f32<ST>(xr[i]);
        ss = fmaf(v, v, ss);
    }
    ss = block_sum(ss, sm);
    const float sc = 1.0f / sqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x) out[(size_t)t * d + i] = to_f32<ST>(xr[i]) * sc * g[i];
}

// ---- rotary embedding of q and k (pairs (i, i + hd/2)), append k, v to the cache -----------
// qkv: [T, d + 2 kvd] fp32 = [q (H heads) | k (Hkv heads) | v (Hkv heads)]; q is rotated in place; k (rotated) and
// v go to the cache rows of positions ctx + row0 + t, rounded to the storage type.  grid (T, H): block h rotates
// query head h and, if h < Hkv, appends key/value head h.
template <typename ST>
__global__ void k_rope_append(float *qkv, int row0, int hd, int d, int Hkv, const float2 *rope_cs, ST *kcache, ST *vcache,
                              int max_seq, const ClDevState *st) {
    if (st->done) return;
    const int t = blockIdx.x, h = blockIdx.y, i = threadIdx.x, half = hd >> 1;
    const int pos = st->ctx + row0 + t;
    if (pos >= max_seq) return;
    const int kvd = Hkv * hd;
    float *row = qkv + (size_t)t * (d + 2 * kvd);
    float *q = row + h * hd;
    const float2 cs = rope_cs[(size_t)pos * half + i];
    const float qa = q[i], qb = q[i + half];
    q[i] = qa * cs.x - qb * cs.y;
    q[i + half] = qb * cs.x + qa * cs.y;
    if (h >= Hkv) return;
    const float *k = row + d + h * hd, *v = row + d + kvd + h * hd;
    const float ka = k[i], kb = k[i + half];
    ST *kc = kcache + ((size_t)h * max_seq + pos) * hd;   // cache layout [head][position][hd]: a head's rows are contiguous
    ST *vc = vcache + ((size_t)h * max_seq + pos) * hd;
    kc[i] = from_f32<ST>(ka * cs.x - kb * cs.y);
    kc[i + half] = from_f32<ST>(kb * cs.x + ka * cs.y);
    vc[i] = from_f32<ST>(v[i]);
    vc[i + half] = from_f32<ST>(v[i + half]);
}

// ---- decode attention over the KV cache -----------------------------------------------------
// grid (H, T, nsplit); block 128.  Row t attends to cache positions 0 .. ctx + row0 + t; the range
// is cut into nsplit slices; each block produces (max, sum, unnormalised output) of its slice and
// the last block of a (t, h) to finish merges the slices in order.
template <typename ST, int HD>
__global__ void __launch_bounds__(128) k_attn(ClAttnArgs a) {
    if (a.st->done) return;
    extern __shared__ float smem[];
    float *sq = smem;               // [HD]
    float *red = smem + HD;         // [HD * 2] scratch + [32]
    float *sc = smem + 3 * HD + 32; // [per_max]
    __shared__ int is_last;
    const int h = blockIdx.x, t = blockIdx.y, sp = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nkeys = a.st->ctx + a.row0 + t + 1;
    if (nkeys > a.max_seq) return;   // the host rejects such calls; never index past the cache
    const int per = (nkeys + a.nsplit - 1) / a.nsplit;
    const int j0 = min(nkeys, sp * per), j1 = min(nkeys, j0 + per);
    const int n = j1 - j0;
    const int d = a.d_model;
    const int kvh = h / (a.n_heads / a.n_kv_heads);   // grouped-query attention: the key/value head of this query head
    const ST *K = (const ST *)a.kcache + (size_t)kvh * a.max_seq * HD;
    const ST *V = (const ST *)a.vcache + (size_t)kvh * a.max_seq * HD;
    const float scale = rsqrtf((float)HD);

    for (int i = tid; i < HD; i += blockDim.x) sq[i] = a.q[(size_t)t * a.ld_q + h * HD + i];
    __syncthreads();

    // scores: LPK lanes per key, 16 bytes of the key row per lane
    constexpr int EPL = 16 / (int)sizeof(ST);   // elements per lane: 8 (bf16) or 4 (fp32)
    constexpr int LPK = HD / EPL;               // lanes per key: 8/16 (bf16), 16/32 (fp32)
    constexpr int KPW = 32 / LPK;               // keys per warp pass
    const int sub = lane / LPK, li = lane % LPK;
    float qr[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) qr[e] = sq[li * EPL + e];
    float lmax = -INFINITY;
    for (int jb = warp * KPW; jb < n; jb += 4 * KPW) {
        const int j = jb + sub;
        float s = 0.f;
        if (j < n) {
            const uint4 raw = *(const uint4 *)(K + (size_t)(j0 + j) * HD + li * EPL);
            if (sizeof(ST) == 2) {
                const unsigned u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float k0, k1;
                    ClPair16<ST>::get(u[e], k0, k1);
                    s = fmaf(qr[2 * e], k0, s);
                    s = fmaf(qr[2 * e + 1], k1, s);
                }
            } else {
                s = fmaf(qr[0], __uint_as_float(raw.x), s);
                s = fmaf(qr[1], __uint_as_float(raw.y), s);
                s = fmaf(qr[2], __uint_as_float(raw.z), s);
                s = fmaf(qr[3], __uint_as_float(raw.w), s);
            }
        }
#pragma unroll
        for (int o = LPK >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s *= scale;
        if (j < n) {
            if (li == 0) sc[j] = s;
            lmax = fmaxf(lmax, s);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lmax = fmaxf(lmax, __shfl_xor_sync(0xffffffffu, lmax, o));
    if (lane == 0) red[warp] = lmax;
    __syncthreads();
    const float m = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    __syncthreads();
    float ls = 0.f;
    for (int j = tid; j < n; j += blockDim.x) {
        const float p = expf(sc[j] - m);
        sc[j] = p;
        ls += p;
    }
    const float l = block_sum(ls, red + 2 * HD);   // (syncs inside also publish sc[])

    // weighted sum of values: thread (stripe, e) walks keys stripe, stripe + NS, ...
    constexpr int NS = 128 / HD;   // 2 for HD 64, 1 for HD 128
    const int e = tid % HD, stripe = tid / HD;
    float acc = 0.f;
    for (int j = stripe; j < n; j += NS) acc = fmaf(sc[j], to_f32<ST>(V[(size_t)(j0 + j) * HD + e]), acc);
    if (NS > 1) {
        red[tid] = acc;
        __syncthreads();
        if (stripe == 0) acc = red[e] + red[HD + e];
    }
    float *part = a.part + (((size_t)t * a.n_heads + h) * a.nsplit + sp) * (HD + 2);
    if (stripe == 0) part[2 + e] = acc;
    if (tid == 0) {
        part[0] = (n > 0) ? m : -INFINITY;
        part[1] = (n > 0) ? l : 0.f;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = (atomicAdd(a.tickets + t * a.n_heads + h, 1u) == (unsigned)a.nsplit - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    if (tid < HD) {
        const volatile float *p0 = a.part + ((size_t)t * a.n_heads + h) * a.nsplit * (HD + 2);
        float M = -INFINITY;
        for (int s2 = 0; s2 < a.nsplit; ++s2) M = fmaxf(M, p0[s2 * (HD + 2)]);
        float Lsum = 0.f, O = 0.f;
        for (int s2 = 0; s2 < a.nsplit; ++s2) {
            const float ms = p0[s2 * (HD + 2)], lsv = p0[s2 * (HD + 2) + 1];
            if (lsv > 0.f) {
                const float w = expf(ms - M);
                Lsum = fmaf(lsv, w, Lsum);
                O = fmaf(p0[s2 * (HD + 2) + 2 + tid], w, O);
            }
        }
        const float o = O / Lsum;
        a.out[(size_t)t * d + h * HD + tid] = o;
    }
    if (tid == 0) a.tickets[t * a.n_heads + h] = 0u;
}

// ---- hidden-state tap: ring[pos % P] = storage-type(x[t]) ----------------------------------
template <typename ST>
__global__ void k_tap(const float *x, int row0, int d, ST *ring_layer, int P, const ClDevState *st) {
    if (st->done) return;
    const int t = blockIdx.x;
    const int pos = st->ctx + row0 + t;
    ST *dst = ring_layer + (size_t)(pos % P) * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = from_f32<ST>(x[(size_t)t * d + i]);
}

// ---- greedy acceptance (Section 3, Figure 2) ------------------------------------------------
// drafts d_j = cyc_tok[j] (j = 1..K), target g_j = tgt_tok[j-1].  n = longest matching prefix.
__global__ void k_accept(ClDevState *st, int K, int *out_tokens) {
    if (threadIdx.x != 0 || st->done) return;
    const int nd = (K < 0) ? st->n_drafted : K;
    int n = 0;
    while (n < nd && st->cyc_tok[n + 1] == st->tgt_tok[n]) ++n;
    for (int j = 0; j < n; ++j) st->emitted[j] = st->cyc_tok[j + 1];
    st->emitted[n] = st->tgt_tok[n];
    if (out_tokens) {
        for (int j = 0; j <= n; ++j)
            if (st->n_out + j < st->max_new) out_tokens[st->n_out + j] = st->emitted[j];
        st->n_out = min(st->n_out + n + 1, st->max_new);
        if (st->n_out >= st->max_new) st->done = 1;
    }
    st->n_acc_last = n;
    st->ctx += n + 1;
    st->cyc_tok[0] = st->tgt_tok[n];
    st->n_drafted = 0;
    st->cycles += 1ull;
    st->drafted += (unsigned long long)nd;
    st->accepted += (unsigned long long)n;
    st->emitted_total += (unsigned long long)(n + 1);
}

__global__ void k_advance(ClDevState *st, int n, int set_pending_from_tgt) {
    if (threadIdx.x != 0) return;
    st->ctx += n;
    if (set_pending_from_tgt) st->cyc_tok[0] = st->tgt_tok[n - 1];
}

// ---- c_layer[r] = mean over P positions of conf_rows[r, :] (fixed order, double) -------------
__global__ void k_mean_rows(const float *conf_rows, int rows, int P, float *c_layer) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    double s = 0.0;
    for (int p = 0; p < P; ++p) s += (double)conf_rows[(size_t)r * P + p];
    c_layer[r] = (float)(s / (double)P);
}

// ---- gate/up interleave at load: dst[2i] = Wg[i], dst[2i+1] = Wu[i] ---------------------------
template <typename ST>
__global__ void k_interleave(const ST *wg, const ST *wu, ST *dst, int F, int d) {
    const size_t n = (size_t)F * d;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const size_t r = i / d, c = i % d;
        dst[(2 * r) * d + c] = wg[i];
        dst[(2 * r + 1) * d + c] = wu[i];
    }
}

// ---- adaptive-window skip-set selection (Section 3.2, Eq. 5-10) -------------------------------
// One thread, double precision, the operations in the order of the definitions (no fused
// multiply-add: every product and sum is rounded on its own so the result does not depend on
// instruction selection).  At most CL_SEL_MAX eligible layers.
#define CL_SEL_MAX 256
__device__ __forceinline__ double dmul(double a, double b) { return __dmul_rn(a, b); }
__device__ __forceinline__ double dadd(double a, double b) { return __dadd_rn(a, b); }
__device__ __forceinline__ double dsub(double a, double b) { return __dadd_rn(a, -b); }

// One element of the discrete gradient (central differences inside, one-sided at the ends).
__device__ __forceinline__ double sel_gradient_at(const double *x, int i, int n) {
    if (n < 2) return 0.0;
    if (i == 0) return dsub(x[1], x[0]);
    if (i == n - 1) return dsub(x[n - 1], x[n - 2]);
    return dmul(dsub(x[i + 1], x[i - 1]), 0.5);
}

// One warp.  Everything that is a sum over layers in a stated order (Eq. 5, the local statistics of Eq. 8-9) is added
// in that order by one lane, every operation rounded on its own, so the margins are those of a sequential evaluation
// bit for bit; the layers themselves (lane i takes layers i, i + 32, ...) run side by side, and the sequential
// selection of the smallest margins becomes a rank by counting (ties -> lower layer index, as picking minima does).
__global__ void k_select(cl_select_cfg cfg, int L, const float *c_layer, uint8_t *mask, double *margins) {
    if (blockIdx.x != 0 || threadIdx.x >= 32) return;
    __shared__ double c[CL_SEL_MAX], chat[CL_SEL_MAX], g[CL_SEL_MAX], tmp[CL_SEL_MAX], mg[CL_SEL_MAX];
    const int lane = threadIdx.x;
    const int lo = cfg.lo, n = cfg.hi - cfg.lo + 1;
    for (int l = lane; l < L; l += 32) {
        mask[l] = 0;
        if (margins) margins[l] = 0.0;
    }
    if (n <= 0) return;
    for (int i = lane; i < n; i += 32) c[i] = (double)c_layer[lo + i];
    __syncwarp();
    // Eq. 5 (every lane adds up the same sequence: no broadcast needed)
    double s = 0.0;
    for (int i = 0; i < n; ++i) s = dadd(s, c[i]);
    const double mu = s / (double)n;
    s = 0.0;
    for (int i = 0; i < n; ++i) s = dadd(s, dmul(dsub(c[i], mu), dsub(c[i], mu)));
    const double sigma = sqrt(s / (double)n);
    for (int i = lane; i < n; i += 32) chat[i] = dsub(c[i], mu) / dadd(sigma, cfg.eps);
    __syncwarp();
    // Eq. 6
    for (int i = lane; i < n; i += 32) tmp[i] = n >= 3 ? sel_gradient_at(chat, i, n) : 0.0;
    __syncwarp();
    for (int i = lane; i < n; i += 32) g[i] = n >= 3 ? fabs(sel_gradient_at(tmp, i, n)) : 0.0;
    __syncwarp();
    double gmin = g[0], gmax = g[0];   // (minimum and maximum do not depend on the order)
    for (int i = lane; i < n; i += 32) {
        gmin = fmin(gmin, g[i]);
        gmax = fmax(gmax, g[i]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        gmin = fmin(gmin, __shfl_xor_sync(0xffffffffu, gmin, o));
        gmax = fmax(gmax, __shfl_xor_sync(0xffffffffu, gmax, o));
    }
    __syncwarp();
    for (int i = lane; i < n; i += 32) g[i] = dsub(g[i], gmin) / dadd(dsub(gmax, gmin), cfg.eps);
    // w_max
    double w_max = cfg.w_max;
    if (!(w_max > 0.0)) {
        int cnt = 0;
        for (int i = 0; i < n; ++i) {
            if (fabs(dsub(c[i], c[0])) <= cfg.flat_tol) ++cnt;
            else break;
        }
        w_max = (double)(cnt > 1 ? cnt : 1);
    }
    __syncwarp();
    // Eq. 7-10
    for (int i = lane; i < n; i += 32) {
        const double w = dadd(cfg.w_base, dmul(dmul(w_max, g[i]), (double)(lo + i) / (double)L));
        const int W = cfg.fixed_window > 0 ? cfg.fixed_window : (int)floor(dadd(w, 0.5));
        int half = (W + 1) / 2;
        if (half < 1) half = 1;
        const int a = (i - half > 0) ? i - half : 0, b = (i + half < n - 1) ? i + half : n - 1;
        double sum = 0.0;
        int cnt = 0;
        for (int j = a; j <= b; ++j)
            if (j != i) {
                sum = dadd(sum, chat[j]);
                ++cnt;
            }
        double m_i, sd_i;
        if (cnt == 0) {
            m_i = chat[i];
            sd_i = 0.0;
        } else {
            m_i = sum / (double)cnt;
            sum = 0.0;
            for (int j = a; j <= b; ++j)
                if (j != i) sum = dadd(sum, dmul(dsub(chat[j], m_i), dsub(chat[j], m_i)));
            sd_i = sqrt(sum / (double)cnt);
        }
        mg[i] = dsub(chat[i], dsub(m_i, dmul(cfg.lambda, sd_i)));
    }
    __syncwarp();
    // Eq. 10 and the ratio post-step: smallest margins first, ties -> lower layer index
    int n_fixed = 0, need;
    const bool by_sign = cfg.n_skip < 0;   // layers with a negative margin are in; then the smallest others up to the ratio
    if (!by_sign) {
        need = cfg.n_skip < n ? cfg.n_skip : n;
    } else {
        for (int i = 0; i < n; ++i) n_fixed += mg[i] < 0.0 ? 1 : 0;
        need = (int)floor(dadd(dmul(cfg.min_ratio, (double)n), 0.5));
    }
    for (int i = lane; i < n; i += 32) {
        const double m = mg[i];
        bool in = by_sign && m < 0.0;
        if (!in) {
            int rank = 0;   // candidates (layers not in yet) that would be picked before this one
            for (int j = 0; j < n; ++j) {
                const double q = mg[j];
                if (by_sign && q < 0.0) continue;
                rank += (q < m || (j < i && !(m < q))) ? 1 : 0;
            }
            in = n_fixed + rank < need;
        }
        if (in) mask[lo + i] = 3;
        if (margins) margins[lo + i] = m;
    }
}

}  // namespace

// Runs CALL with ST = the storage type that wdtype names (0 fp32, 1 bf16, 2 fp16).
#define CL_DISPATCH_ST(wdtype, CALL)                                \
    do {                                                            \
        if ((wdtype) == 1) { using ST = __nv_bfloat16; CALL; }      \
        else if ((wdtype) == 2) { using ST = __half; CALL; }        \
        else { using ST = float; CALL; }                            \
    } while (0)

cudaError_t cl_launch_embed(int wdtype, const void *embed, const int *tok, int T, int d, float *x, const ClDevState *st,
                            cudaStream_t s) {
    CL_DISPATCH_ST(wdtype, (k_embed<ST><<<T, 256, 0, s>>>((const ST *)embed, tok, d, x, st)));
    return cudaGetLastError();
}

cudaError_t cl_launch_rmsnorm(const float *x, const float *g, int T, int d, float eps, float *out, const ClDevState *st,
                              cudaStream_t s) {
    k_rmsnorm<float><<<T, 256, 0, s>>>(x, g, d, eps, out, st);
    return cudaGetLastError();
}

cudaError_t cl_launch_rmsnorm_rows(int in_dtype, const void *x, const float *g, int T, int d, float eps, float *out,
                                   cudaStream_t s) {
    CL_DISPATCH_ST(in_dtype, (k_rmsnorm<ST><<<T, 256, 0, s>>>((const ST *)x, g, d, eps, out, nullptr)));
    return cudaGetLastError();
}

cudaError_t cl_launch_rope_append(int wdtype, float *qkv, int T, int row0, int H, int Hkv, int hd, int d, const float2 *rope_cs,
                                  void *kcache, void *vcache, int max_seq, const ClDevState *st, cudaStream_t s) {
    dim3 grid(T, H);
    CL_DISPATCH_ST(wdtype, (k_rope_append<ST><<<grid, hd / 2, 0, s>>>(qkv, row0, hd, d, Hkv, rope_cs, (ST *)kcache, (ST *)vcache,
                                                                      max_seq, st)));
    return cudaGetLastError();
}

cudaError_t cl_launch_attn(int wdtype, int T, const ClAttnArgs &a, cudaStream_t s) {
    dim3 grid(a.n_heads, T, a.nsplit);
    const size_t smem = (size_t)(3 * a.head_dim + 32 + a.per_max) * sizeof(float);
    if (a.head_dim == 64) {
        CL_DISPATCH_ST(wdtype, (k_attn<ST, 64><<<grid, 128, smem, s>>>(a)));
    } else if (a.head_dim == 128) {
        CL_DISPATCH_ST(wdtype, (k_attn<ST, 128><<<grid, 128, smem, s>>>(a)));
    } else {
        return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t cl_launch_tap(int wdtype, const float *x, int T, int row0, int d, void *ring_layer, int P,
                          const ClDevState *st, cudaStream_t s) {
    CL_DISPATCH_ST(wdtype, (k_tap<ST><<<T, 256, 0, s>>>(x, row0, d, (ST *)ring_layer, P, st)));
    return cudaGetLastError();
}

cudaError_t cl_launch_accept(ClDevState *st, int K, int *out_tokens, cudaStream_t s) {
    k_accept<<<1, 32, 0, s>>>(st, K, out_tokens);
    return cudaGetLastError();
}

cudaError_t cl_launch_advance(ClDevState *st, int n, int set_pending_from_tgt, cudaStream_t s) {
    k_advance<<<1, 32, 0, s>>>(st, n, set_pending_from_tgt);
    return cudaGetLastError();
}

cudaError_t cl_launch_mean_rows(const float *conf_rows, int rows, int P, float *c_layer, cudaStream_t s) {
    k_mean_rows<<<(rows + 127) / 128, 128, 0, s>>>(conf_rows, rows, P, c_layer);
    return cudaGetLastError();
}

cudaError_t cl_launch_select(const cl_select_cfg &cfg, int n_layers, const float *c_layer, uint8_t *mask, double *margins,
                             cudaStream_t s) {
    if (cfg.hi - cfg.lo + 1 > CL_SEL_MAX) return cudaErrorInvalidValue;
    k_select<<<1, 32, 0, s>>>(cfg, n_layers, c_layer, mask, margins);
    return cudaGetLastError();
}

cudaError_t cl_launch_interleave(int wdtype, const void *wg, const void *wu, void *dst, int F, int d, cudaStream_t s) {
    CL_DISPATCH_ST(wdtype, (k_interleave<ST><<<1184, 256, 0, s>>>((const ST *)wg, (const ST *)wu, (ST *)dst, F, d)));
    return cudaGetLastError();
}
