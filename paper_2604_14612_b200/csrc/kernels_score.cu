// All-layer early-exit confidence scoring as one dense contraction on the 5th-generation tensor cores
// (Section 3.1, Eq. 1-4): logits[r, v] = sum_k xn[r, k] * W_lm[v, k] for every tapped hidden row r, fused with
// the clamp and an online softmax / entropy / top-1 / argmax reduction per row.  Logits never leave the SM.
//
// One persistent CTA per SM, 192 threads:
//   warp 0   TMA producer: 128 x 64 tiles of the normalised hidden rows (A) and 256 x 64 tiles of the LM head (B),
//            128-byte swizzled, into a 4-stage shared-memory ring (48 KB per stage), completion on mbarriers;
//   warp 1   allocates tensor memory and issues tcgen05.mma (M 128, N 256, K 16, bf16 -> fp32) from one thread;
//            the 128 x 256 fp32 accumulator lives in tensor memory, two of them (512 columns) so that the
//            epilogue of one vocabulary tile overlaps the multiply-adds of the next;
//   warps 2-5 epilogue: thread = one hidden row (one tensor-memory lane); it reads its row of the accumulator
//            32 columns at a time (tcgen05.ld) and keeps running softmax statistics relative to the running
//            maximum m: z = sum e^(l-m), s = sum (l-m) e^(l-m), and the argmax (lowest index on ties).
// A CTA owns one block of 128 hidden rows and a contiguous range of vocabulary tiles; CTAs that share the
// vocabulary range run side by side, so a tile of the LM head is fetched from HBM once and served to the other
// row blocks from L2.  Per-(row, vocabulary range) statistics are merged in a fixed order by a second kernel,
// which also evaluates H = log Z - S/Z, the confidence 1 - H / log V (Eq. 3-4) and the top-1 probability 1/Z.
// Every wait is bounded in time; on expiry an error flag is raised and the kernel winds down.
#include <math.h>

#include "tc_common.cuh"

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int NTHREADS = 192;
struct ScoreSmem {
    unsigned long long full[STAGES], empty[STAGES], tfull[2], tempty[2];
    unsigned tmem_base;
    int abort;
};

struct ScoreArgs {
    int R, V, KB, MT, NCG, NT;      // hidden rows, vocabulary, K blocks of 64, row blocks, vocabulary ranges, vocabulary tiles
    ClHeadPartial *partials;        // [MT * BM, NCG]
    int *err;
    int f16;                        // 16-bit type of both operands: 0 bf16, 1 fp16
};


__global__ void __launch_bounds__(NTHREADS, 1)
k_score(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, ScoreArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *tiles = (unsigned char *)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);   // swizzled tiles: 1 KB aligned
    ScoreSmem *sm = (ScoreSmem *)(tiles + (size_t)STAGES * STAGE_BYTES);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    if (cta >= a.MT * a.NCG) return;   // whole CTA leaves before anything is set up
    const int mt = cta % a.MT, cg = cta / a.MT;
    const int nt0 = (int)((long long)a.NT * cg / a.NCG), nt1 = (int)((long long)a.NT * (cg + 1) / a.NCG);
    const int ntiles = nt1 - nt0;

    if (tid == 0) {
        for (int i = 0; i < STAGES; ++i) {
            bar_init(&sm->full[i], 1);
            bar_init(&sm->empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            bar_init(&sm->tfull[i], 1);
            bar_init(&sm->tempty[i], 128);
        }
        sm->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(s_u32(&sm->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem = *(volatile unsigned *)&sm->tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            unsigned stage = 0, par = 0, issued[STAGES];
            for (int i = 0; i < STAGES; ++i) issued[i] = 2u;
            bool ok = true;
            for (int t = 0; t < ntiles && ok; ++t) {
                for (int kb = 0; kb < a.KB; ++kb) {
                    if (!bar_wait(&sm->empty[stage], par ^ 1u, &sm->abort, a.err)) { ok = false; break; }
                    unsigned char *dst = tiles + (size_t)stage * STAGE_BYTES;
                    bar_expect(&sm->full[stage], STAGE_BYTES);
                    tma_load_2d(dst, &mapA, kb * BK, mt * BM, &sm->full[stage]);
                    tma_load_2d(dst + A_BYTES, &mapB, kb * BK, (nt0 + t) * BN, &sm->full[stage]);
                    issued[stage] = par;
                    if (++stage == STAGES) { stage = 0; par ^= 1u; }
                }
            }
            if (!ok) {   // gave up: still let the copies in flight land before the CTA may exit (bounded)
                for (int i = 0; i < STAGES; ++i) {
                    if (issued[i] < 2u) {
                        const unsigned long long t0 = gtime_ns();
                        while (!bar_try(&sm->full[i], issued[i]))
                            if (gtime_ns() - t0 > WAIT_NS) break;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const unsigned idesc = umma_idesc(BM, BN, a.f16);
            unsigned stage = 0, par = 0;
            bool ok = true;
            for (int t = 0; t < ntiles && ok; ++t) {
                const int b = t & 1;
                if (!bar_wait(&sm->tempty[b], (((unsigned)t >> 1) & 1u) ^ 1u, &sm->abort, a.err)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int kb = 0; kb < a.KB; ++kb) {
                    if (!bar_wait(&sm->full[stage], par, &sm->abort, a.err)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned a_addr = s_u32(tiles + (size_t)stage * STAGE_BYTES), b_addr = a_addr + A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_bf16(tmem + (unsigned)b * BN, umma_desc(a_addr + k * 32), umma_desc(b_addr + k * 32), idesc,
                                  (unsigned)(kb | k));
                    umma_commit(&sm->empty[stage]);   // the stage is free once these multiply-adds have read it
                    if (++stage == STAGES) { stage = 0; par ^= 1u; }
                }
                if (ok) umma_commit(&sm->tfull[b]);   // accumulator b is complete
            }
        }
    } else {
        // ---------------- epilogue: one thread per hidden row ----------------
        const int q = warp & 3;                        // the tensor-memory lane quadrant this warp may read
        const int row = q * 32 + lane;
        ClHeadPartial run{0.f, 0.f, 0.f, 0x7fffffff};
        for (int t = 0; t < ntiles; ++t) {
            const int b = t & 1;
            if (!bar_wait(&sm->tfull[b], ((unsigned)t >> 1) & 1u, &sm->abort, a.err)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int n0 = (nt0 + t) * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                float v[32];
                tmem_ld32(tmem + ((unsigned)(q * 32) << 16) + (unsigned)(b * BN + c * 32), v);
                const int col0 = n0 + c * 32;
                const int nvalid = min(32, a.V - col0);   // uniform over the warp
                if (nvalid <= 0) continue;
                float cm = -INFINITY;
                int ci = 0;
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (i < nvalid) {
                        const float l = fminf(fmaxf(v[i], -CL_LOGIT_CLAMP), CL_LOGIT_CLAMP);   // clamp of Section 3.1
                        v[i] = l;
                        if (l > cm) { cm = l; ci = col0 + i; }
                    }
                }
                float m_new = cm;
                if (run.z > 0.f) {
                    m_new = fmaxf(run.m, cm);
                    const float e = expf(run.m - m_new);
                    run.s = e * (run.s + (run.m - m_new) * run.z);
                    run.z *= e;
                    if (cm > run.m) run.idx = ci;   // strictly larger only: the lowest index wins ties
                } else {
                    run.idx = ci;
                }
                run.m = m_new;
                float z = 0.f, s = 0.f;
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (i < nvalid) {
                        const float d = v[i] - m_new;
                        const float e = expf(d);
                        z += e;
                        s = fmaf(d, e, s);
                    }
                }
                run.z += z;
                run.s += s;
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            bar_arrive(&sm->tempty[b]);
        }
        a.partials[(size_t)(mt * BM + row) * a.NCG + cg] = run;
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

// Merge the per-range statistics of every row in a fixed order and evaluate Eq. 2-4.
__global__ void k_score_finalize(const ClHeadPartial *partials, int NCG, int R, float inv_log_v, float *conf, float *pmax,
                                 int *arg) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= R) return;
    ClHeadPartial f{0.f, 0.f, 0.f, 0x7fffffff};
    for (int g = 0; g < NCG; ++g) f = cl_hp_merge(f, partials[(size_t)r * NCG + g]);
    const float H = logf(f.z) - f.s / f.z;   // entropy of the softmax from sums relative to the maximum
    conf[r] = 1.f - H * inv_log_v;
    pmax[r] = 1.f / f.z;
    arg[r] = f.idx;
}

// Final RMSNorm of hidden rows in the storage type -> rows in the 16-bit type of the LM head (the A operand of the
// contraction).
// Eight consecutive elements of a row as floats (one or two 16-byte loads).
template <typename ST>
__device__ __forceinline__ void load8(const ST *p, float (&v)[8]) {
    if (sizeof(ST) == 4) {
        const float4 a = *(const float4 *)p, b = *((const float4 *)p + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
        const uint4 u = *(const uint4 *)p;
        const unsigned w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) ClPair16<ST>::get(w[e], v[2 * e], v[2 * e + 1]);
    }
}

// One CTA per row, 16-byte accesses (d is a multiple of 8).  A thread's first chunks stay in registers between the two
// passes; the sum of squares is added in a fixed order (per thread, shuffle tree, warps in order).
template <typename ST>
__global__ void k_rmsnorm_to_bf16(const ST *x, const float *g, int d, float eps, unsigned short *out, int f16) {
    __shared__ float red[32];
    constexpr int KEEP = 2;
    const ST *xr = x + (size_t)blockIdx.x * d;
    const int nch = d >> 3;
    float keep[KEEP][8];
    float ss = 0.f;
    for (int c = threadIdx.x, k = 0; c < nch; c += blockDim.x, ++k) {
        float v[8];
        load8<ST>(xr + (size_t)c * 8, v);
#pragma unroll
        for (int e = 0; e < 8; ++e) ss = fmaf(v[e], v[e], ss);
        if (k < KEEP) {
#pragma unroll
            for (int e = 0; e < 8; ++e) keep[k < KEEP ? k : 0][e] = v[e];
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += red[w];   // fixed order
    const float sc = 1.0f / sqrtf(tot / (float)d + eps);
    for (int c = threadIdx.x, k = 0; c < nch; c += blockDim.x, ++k) {
        float v[8];
        if (k < KEEP) {
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = keep[k < KEEP ? k : 0][e];
        } else {
            load8<ST>(xr + (size_t)c * 8, v);
        }
        const float4 g0 = *(const float4 *)(g + (size_t)c * 8), g1 = *((const float4 *)(g + (size_t)c * 8) + 1);
        const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        unsigned w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            w[e] = (unsigned)f32_to_b16(v[2 * e] * sc * gg[2 * e], f16) | ((unsigned)f32_to_b16(v[2 * e + 1] * sc * gg[2 * e + 1], f16) << 16);
        *(uint4 *)(out + (size_t)blockIdx.x * d + (size_t)c * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

}  // namespace

int cl_score_tc_ranges(int R, int n_sm) {
    const int MT = (R + BM - 1) / BM;
    int ncg = n_sm / MT;
    return ncg < 1 ? 1 : ncg;
}

size_t cl_score_tc_partials(int R, int n_sm) {
    const int MT = (R + BM - 1) / BM;
    return (size_t)MT * BM * cl_score_tc_ranges(R, n_sm);
}

cudaError_t cl_launch_rmsnorm_bf16(int in_dtype, const void *x, const float *g, int rows, int d, float eps, void *out,
                                   int f16, cudaStream_t s) {
    if (in_dtype == 1)
        k_rmsnorm_to_bf16<__nv_bfloat16><<<rows, 256, 0, s>>>((const __nv_bfloat16 *)x, g, d, eps, (unsigned short *)out, f16);
    else if (in_dtype == 2)
        k_rmsnorm_to_bf16<__half><<<rows, 256, 0, s>>>((const __half *)x, g, d, eps, (unsigned short *)out, f16);
    else
        k_rmsnorm_to_bf16<float><<<rows, 256, 0, s>>>((const float *)x, g, d, eps, (unsigned short *)out, f16);
    return cudaGetLastError();
}

// xn: [R, d] bf16 normalised rows; lm_head: [V, d] bf16.  Needs d % 8 == 0 and 16-byte aligned bases.
cudaError_t cl_launch_score_tc(const void *xn, const void *lm_head, int R, int V, int d, ClHeadPartial *partials, int n_sm,
                               int *err, float *conf, float *pmax, int *arg, int f16, cudaStream_t s) {
    CUtensorMap mapA, mapB;
    if (!make_map(&mapA, xn, R, d, BM, f16) || !make_map(&mapB, lm_head, V, d, BN, f16)) return cudaErrorInvalidValue;
    ScoreArgs a;
    a.f16 = f16;
    a.R = R; a.V = V; a.KB = (d + BK - 1) / BK;
    a.MT = (R + BM - 1) / BM;
    a.NCG = cl_score_tc_ranges(R, n_sm);
    a.NT = (V + BN - 1) / BN;
    if (a.NCG > a.NT) a.NCG = a.NT;
    a.partials = partials; a.err = err;
    const size_t smem = (size_t)STAGES * STAGE_BYTES + sizeof(ScoreSmem) + 1024;
    cudaError_t e = cudaFuncSetAttribute(k_score, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // row blocks beyond n_sm CTAs are handled in waves of whole column ranges
    k_score<<<a.MT * a.NCG, NTHREADS, smem, s>>>(mapA, mapB, a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    k_score_finalize<<<(R + 127) / 128, 128, 0, s>>>(partials, a.NCG, R, (float)(1.0 / log((double)V)), conf, pmax, arg);
    return cudaGetLastError();
}
