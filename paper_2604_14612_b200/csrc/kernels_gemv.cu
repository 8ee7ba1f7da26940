// Row-streaming matrix-vector kernels for T <= 9 activation rows on CUDA cores.
//
// y[t][r] = sum_c W[r][c] * x[t][c], W in its storage type (bf16 or fp32), x and the accumulation in fp32.
// Each warp owns pairs of consecutive weight rows and walks them with 16-byte coalesced, streaming
// (L1 no-allocate) loads; the T activation rows are re-read through L1.  The epilogue is one of:
//   STORE  plain store (QKV projection),
//   RESID  residual add in place (attention output and FFN down projections),
//   SILU   gate/up rows are interleaved in memory, so a row pair yields silu(gate) * up directly,
//   HEAD   LM head fused with the clamp, an online softmax / entropy reduction, top-1 probability and
//          argmax (Section 3.1, Eq. 1-4): logits are never written unless asked for.
// This is the general path (any T, fp32 or bf16 weights); it is bound by HBM weight streaming for T = 1.
#include <math.h>
#include <string.h>

#include <mutex>

#include "cl_internal.h"

namespace {

__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <typename WT>
struct W8;
template <>
struct W8<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&w)[8]) {
        uint4 v = ld_stream16(p);
        w[0] = __uint_as_float(v.x << 16); w[1] = __uint_as_float(v.x & 0xffff0000u);
        w[2] = __uint_as_float(v.y << 16); w[3] = __uint_as_float(v.y & 0xffff0000u);
        w[4] = __uint_as_float(v.z << 16); w[5] = __uint_as_float(v.z & 0xffff0000u);
        w[6] = __uint_as_float(v.w << 16); w[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};
template <>
struct W8<__half> {
    static __device__ __forceinline__ void load(const __half *p, float (&w)[8]) {
        uint4 v = ld_stream16(p);
        ClPair16<__half>::get(v.x, w[0], w[1]);
        ClPair16<__half>::get(v.y, w[2], w[3]);
        ClPair16<__half>::get(v.z, w[4], w[5]);
        ClPair16<__half>::get(v.w, w[6], w[7]);
    }
};
template <>
struct W8<float> {
    static __device__ __forceinline__ void load(const float *p, float (&w)[8]) {
        uint4 a = ld_stream16(p), b = ld_stream16(p + 4);
        w[0] = __uint_as_float(a.x); w[1] = __uint_as_float(a.y); w[2] = __uint_as_float(a.z); w[3] = __uint_as_float(a.w);
        w[4] = __uint_as_float(b.x); w[5] = __uint_as_float(b.y); w[6] = __uint_as_float(b.z); w[7] = __uint_as_float(b.w);
    }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Merge two partial softmax statistics (see ClHeadPartial).  Empty partials have z == 0.
__device__ __forceinline__ ClHeadPartial head_merge(const ClHeadPartial &a, const ClHeadPartial &b) {
    if (b.z == 0.f) return a;
    if (a.z == 0.f) return b;
    ClHeadPartial r;
    r.m = fmaxf(a.m, b.m);
    float ea = expf(a.m - r.m), eb = expf(b.m - r.m);
    r.z = a.z * ea + b.z * eb;
    r.s = ea * (a.s + (a.m - r.m) * a.z) + eb * (b.s + (b.m - r.m) * b.z);
    r.idx = (a.m > b.m) ? a.idx : (b.m > a.m) ? b.idx : min(a.idx, b.idx);
    return r;
}

__device__ __forceinline__ float silu_f(float x) { return x / (1.f + expf(-x)); }

template <typename WT, int T, int EPI>
__global__ void __launch_bounds__(256) k_gemv(ClGemvArgs a) {
    if (a.st && a.st->done) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int gw = blockIdx.x * nw + warp, tw = gridDim.x * nw;
    const int ngroups = (a.rows + 1) >> 1;
    const int cols = a.cols;
    const WT *W = (const WT *)a.W;

    ClHeadPartial run[T];
    if (EPI == CL_EPI_HEAD) {
#pragma unroll
        for (int t = 0; t < T; ++t) run[t] = ClHeadPartial{0.f, 0.f, 0.f, 0x7fffffff};
    }

    for (int g = gw; g < ngroups; g += tw) {
        const int r0 = 2 * g;
        const bool has1 = (r0 + 1) < a.rows;
        const WT *w0 = W + (size_t)r0 * cols;
        const WT *w1 = W + (size_t)(has1 ? r0 + 1 : r0) * cols;
        float acc0[T], acc1[T];
#pragma unroll
        for (int t = 0; t < T; ++t) acc0[t] = acc1[t] = 0.f;
#pragma unroll 2
        for (int c = lane * 8; c < cols; c += 256) {
            float wa[8], wb[8];
            W8<WT>::load(w0 + c, wa);
            W8<WT>::load(w1 + c, wb);
#pragma unroll
            for (int t = 0; t < T; ++t) {
                const float4 x0 = __ldg((const float4 *)(a.xin + (size_t)t * cols + c));
                const float4 x1 = __ldg((const float4 *)(a.xin + (size_t)t * cols + c + 4));
                float s0 = acc0[t], s1 = acc1[t];
                s0 = fmaf(wa[0], x0.x, s0); s1 = fmaf(wb[0], x0.x, s1);
                s0 = fmaf(wa[1], x0.y, s0); s1 = fmaf(wb[1], x0.y, s1);
                s0 = fmaf(wa[2], x0.z, s0); s1 = fmaf(wb[2], x0.z, s1);
                s0 = fmaf(wa[3], x0.w, s0); s1 = fmaf(wb[3], x0.w, s1);
                s0 = fmaf(wa[4], x1.x, s0); s1 = fmaf(wb[4], x1.x, s1);
                s0 = fmaf(wa[5], x1.y, s0); s1 = fmaf(wb[5], x1.y, s1);
                s0 = fmaf(wa[6], x1.z, s0); s1 = fmaf(wb[6], x1.z, s1);
                s0 = fmaf(wa[7], x1.w, s0); s1 = fmaf(wb[7], x1.w, s1);
                acc0[t] = s0; acc1[t] = s1;
            }
        }
#pragma unroll
        for (int t = 0; t < T; ++t) {
            acc0[t] = warp_sum(acc0[t]);
            acc1[t] = warp_sum(acc1[t]);
        }
        if (lane == 0) {
#pragma unroll
            for (int t = 0; t < T; ++t) {
                if (EPI == CL_EPI_STORE) {
                    a.out[(size_t)t * a.ld + r0] = acc0[t];
                    if (has1) a.out[(size_t)t * a.ld + r0 + 1] = acc1[t];
                } else if (EPI == CL_EPI_RESID) {
                    a.out[(size_t)t * a.ld + r0] += acc0[t];
                    if (has1) a.out[(size_t)t * a.ld + r0 + 1] += acc1[t];
                } else if (EPI == CL_EPI_SILU) {
                    a.out[(size_t)t * a.ld + g] = silu_f(acc0[t]) * acc1[t];
                } else {
                    float l0 = fminf(fmaxf(acc0[t], -CL_LOGIT_CLAMP), CL_LOGIT_CLAMP);
                    if (a.logits) a.logits[(size_t)t * a.rows + r0] = l0;
                    run[t] = head_merge(run[t], ClHeadPartial{l0, 1.f, 0.f, r0});
                    if (has1) {
                        float l1 = fminf(fmaxf(acc1[t], -CL_LOGIT_CLAMP), CL_LOGIT_CLAMP);
                        if (a.logits) a.logits[(size_t)t * a.rows + r0 + 1] = l1;
                        run[t] = head_merge(run[t], ClHeadPartial{l1, 1.f, 0.f, r0 + 1});
                    }
                }
            }
        }
    }

    if (EPI == CL_EPI_HEAD) {
        __shared__ ClHeadPartial sm[256];
        __shared__ int is_last;
        if (lane == 0) {
#pragma unroll
            for (int t = 0; t < T; ++t) sm[warp * T + t] = run[t];   // nw * T <= 8 * 9 = 72 entries
        }
        __syncthreads();
        if (threadIdx.x < T) {
            ClHeadPartial r = sm[threadIdx.x];
            for (int w = 1; w < nw; ++w) r = head_merge(r, sm[w * T + threadIdx.x]);
            a.partials[(size_t)blockIdx.x * T + threadIdx.x] = r;
            __threadfence();
        }
        __syncthreads();
        if (threadIdx.x == 0) is_last = (atomicAdd(a.ticket, 1u) == gridDim.x - 1);
        __syncthreads();
        if (!is_last) return;
        __threadfence();
        // The last block to finish reduces all blocks' partials in a fixed order (deterministic).
        for (int t = 0; t < T; ++t) {
            ClHeadPartial r{0.f, 0.f, 0.f, 0x7fffffff};
            for (int b = threadIdx.x; b < (int)gridDim.x; b += blockDim.x) {
                const volatile ClHeadPartial *p = a.partials + (size_t)b * T + t;
                ClHeadPartial q;
                q.m = p->m; q.z = p->z; q.s = p->s; q.idx = p->idx;
                r = head_merge(r, q);
            }
            __syncthreads();
            sm[threadIdx.x] = r;
            __syncthreads();
            for (int o = blockDim.x >> 1; o > 0; o >>= 1) {
                if ((int)threadIdx.x < o) sm[threadIdx.x] = head_merge(sm[threadIdx.x], sm[threadIdx.x + o]);
                __syncthreads();
            }
            if (threadIdx.x == 0) {
                ClHeadPartial f = sm[0];
                // H = log Z - S/Z (entropy of the softmax, from sums relative to the maximum);
                // confidence = 1 - H / log V (Eq. 3-4); top-1 probability = 1 / Z.
                float H = logf(f.z) - f.s / f.z;
                if (a.out_tok) a.out_tok[t] = f.idx;
                if (a.out_pmax) a.out_pmax[t] = 1.f / f.z;
                if (a.out_conf) a.out_conf[t] = 1.f - H * a.inv_log_v;
            }
        }
        if (threadIdx.x == 0) *a.ticket = 0u;
    }
}

template <typename WT, int T>
cudaError_t launch_t(int epi, const ClGemvArgs &a, int grid, cudaStream_t s) {
    switch (epi) {
        case CL_EPI_STORE: k_gemv<WT, T, CL_EPI_STORE><<<grid, 256, 0, s>>>(a); break;
        case CL_EPI_RESID: k_gemv<WT, T, CL_EPI_RESID><<<grid, 256, 0, s>>>(a); break;
        case CL_EPI_SILU: k_gemv<WT, T, CL_EPI_SILU><<<grid, 256, 0, s>>>(a); break;
        case CL_EPI_HEAD: k_gemv<WT, T, CL_EPI_HEAD><<<grid, 256, 0, s>>>(a); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

template <typename WT>
cudaError_t launch_w(int T, int epi, const ClGemvArgs &a, int grid, cudaStream_t s) {
    switch (T) {
        case 1: return launch_t<WT, 1>(epi, a, grid, s);
        case 2: return launch_t<WT, 2>(epi, a, grid, s);
        case 3: return launch_t<WT, 3>(epi, a, grid, s);
        case 4: return launch_t<WT, 4>(epi, a, grid, s);
        case 5: return launch_t<WT, 5>(epi, a, grid, s);
        case 6: return launch_t<WT, 6>(epi, a, grid, s);
        case 7: return launch_t<WT, 7>(epi, a, grid, s);
        case 8: return launch_t<WT, 8>(epi, a, grid, s);
        case 9: return launch_t<WT, 9>(epi, a, grid, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t cl_launch_gemv(int wdtype, int T, int epi, const ClGemvArgs &a, int grid, cudaStream_t s) {
    if (wdtype == 1) return launch_w<__nv_bfloat16>(T, epi, a, grid, s);
    if (wdtype == 2) return launch_w<__half>(T, epi, a, grid, s);
    return launch_w<float>(T, epi, a, grid, s);
}

// ---- confidence scoring without any allocation ------------------------------------------------------
// Scratch of cl_layer_confidences_static(): one file-scope array that every GPU loading this library holds until
// the process exits.  Layout (bytes): [0, 256) the LM-head kernel's ticket counter; then the normalised rows
// xn [SC_CHUNK, CL_STATIC_MAX_D] fp32; the per-block softmax partials [SC_MAX_GRID, SC_CHUNK]; and the three
// per-row results (confidence, top-1 probability, greedy token) [CL_STATIC_MAX_ROWS] each.
namespace {

constexpr int SC_MAX_GRID = 1024;
constexpr int SC_CHUNK = 8;   // rows per LM-head pass
constexpr size_t SC_OFF_XN = 256;
constexpr size_t SC_OFF_PART = SC_OFF_XN + (size_t)SC_CHUNK * CL_STATIC_MAX_D * sizeof(float);
constexpr size_t SC_OFF_CONF = SC_OFF_PART + (size_t)SC_MAX_GRID * SC_CHUNK * sizeof(ClHeadPartial);
constexpr size_t SC_OFF_PMAX = SC_OFF_CONF + (size_t)CL_STATIC_MAX_ROWS * sizeof(float);
constexpr size_t SC_OFF_ARG = SC_OFF_PMAX + (size_t)CL_STATIC_MAX_ROWS * sizeof(float);
constexpr size_t SC_BYTES = SC_OFF_ARG + (size_t)CL_STATIC_MAX_ROWS * sizeof(int);

static __device__ __align__(256) unsigned char g_static_scratch[SC_BYTES];

constexpr int SC_MAX_DEVICES = 64;
std::mutex g_sc_mutex;
unsigned char *g_sc_addr[SC_MAX_DEVICES];   // device address of g_static_scratch on each device, once looked up
int g_sc_sms[SC_MAX_DEVICES];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the address a kernel
// may use comes from cudaGetSymbolAddress, asked once per device with that device current.
int static_scratch(unsigned char **addr, int *n_sm) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        cl_set_global_error("cl_layer_confidences_static: no CUDA device: %s", cudaGetErrorString(e));
        return CL_ECUDA;
    }
    if (dev < 0 || dev >= SC_MAX_DEVICES) {
        cl_set_global_error("cl_layer_confidences_static: device ordinal %d not supported (max %d)", dev, SC_MAX_DEVICES - 1);
        return CL_ERANGE;
    }
    std::lock_guard<std::mutex> lock(g_sc_mutex);
    if (!g_sc_addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            cl_set_global_error("cl_layer_confidences_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            return CL_ECUDA;
        }
        int sms = 0, major = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (major < 10 || sms <= 0) {
            cl_set_global_error("cl_layer_confidences_static: compute capability %d.x, built for sm_100a only", major);
            return CL_ECUDA;
        }
        g_sc_sms[dev] = sms;
        g_sc_addr[dev] = (unsigned char *)p;
    }
    *addr = g_sc_addr[dev];
    *n_sm = g_sc_sms[dev];
    return CL_OK;
}

}  // namespace

extern "C" int cl_layer_confidences_static(const void *lm_head, const float *final_norm, int vocab, int d_model,
                                           int weight_dtype, float rms_eps, const void *hidden, int n_rows,
                                           void *cuda_stream, float *conf, float *p_max, int32_t *argmax) {
    if (!lm_head || !final_norm || !hidden) {
        cl_set_global_error("cl_layer_confidences_static: null input pointer");
        return CL_EINVAL;
    }
    if (weight_dtype != 0 && weight_dtype != 1) {
        cl_set_global_error("cl_layer_confidences_static: weight_dtype must be 0 or 1");
        return CL_EINVAL;
    }
    if (vocab < 2 || d_model <= 0 || d_model % 8 || n_rows <= 0) {
        cl_set_global_error("cl_layer_confidences_static: need vocab >= 2, d_model a positive multiple of 8, n_rows > 0");
        return CL_EINVAL;
    }
    if (((uintptr_t)lm_head | (uintptr_t)final_norm | (uintptr_t)hidden) & 15u) {
        // the kernels read these with 16-byte vector loads; a misaligned pointer would trap on the device
        cl_set_global_error("cl_layer_confidences_static: lm_head, final_norm and hidden must be 16-byte aligned");
        return CL_EINVAL;
    }
    if (d_model > CL_STATIC_MAX_D || n_rows > CL_STATIC_MAX_ROWS) {
        cl_set_global_error("cl_layer_confidences_static: d_model %d / n_rows %d beyond the fixed scratch (max %d / %d)", d_model,
                            n_rows, CL_STATIC_MAX_D, CL_STATIC_MAX_ROWS);
        return CL_ERANGE;
    }
    unsigned char *sc = nullptr;
    int n_sm = 0;
    int rc = static_scratch(&sc, &n_sm);
    if (rc) return rc;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    float *xn = (float *)(sc + SC_OFF_XN);
    float *d_conf = (float *)(sc + SC_OFF_CONF), *d_pmax = (float *)(sc + SC_OFF_PMAX);
    int *d_arg = (int *)(sc + SC_OFF_ARG);
    const size_t es = weight_dtype == 1 ? 2 : 4;
    cudaError_t e = cudaMemsetAsync(sc, 0, SC_OFF_XN, s);   // the ticket must start at zero whatever the last call left
    ClGemvArgs a;
    memset(&a, 0, sizeof(a));
    a.W = lm_head; a.rows = vocab; a.cols = d_model; a.xin = xn;
    a.partials = (ClHeadPartial *)(sc + SC_OFF_PART);
    a.ticket = (unsigned *)sc;
    a.inv_log_v = (float)(1.0 / log((double)vocab));
    int grid = ((vocab + 1) / 2 + 7) / 8;
    if (grid > n_sm * 4) grid = n_sm * 4;
    if (grid > SC_MAX_GRID) grid = SC_MAX_GRID;
    for (int r0 = 0; r0 < n_rows && e == cudaSuccess; r0 += SC_CHUNK) {
        const int T = n_rows - r0 < SC_CHUNK ? n_rows - r0 : SC_CHUNK;
        e = cl_launch_rmsnorm_rows(weight_dtype, (const char *)hidden + (size_t)r0 * d_model * es, final_norm, T, d_model, rms_eps,
                                   xn, s);
        if (e != cudaSuccess) break;
        a.out_tok = d_arg + r0; a.out_pmax = d_pmax + r0; a.out_conf = d_conf + r0;
        e = cl_launch_gemv(weight_dtype, T, CL_EPI_HEAD, a, grid, s);
    }
    if (e == cudaSuccess && conf) e = cudaMemcpyAsync(conf, d_conf, (size_t)n_rows * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && p_max) e = cudaMemcpyAsync(p_max, d_pmax, (size_t)n_rows * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && argmax) e = cudaMemcpyAsync(argmax, d_arg, (size_t)n_rows * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        cl_set_global_error("cl_layer_confidences_static: %s", cudaGetErrorString(e));
        return CL_ECUDA;
    }
    return CL_OK;
}
