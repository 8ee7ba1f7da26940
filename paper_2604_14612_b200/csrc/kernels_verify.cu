// Skinny tensor-core GEMM for passes of T <= 9 token rows through a model stored in a 16-bit type (bf16, or fp16:
// both operands of a tcgen05.mma are of that one type): the (K+1)-row verify pass of Section 3 (and short prompts,
// which are the same pass over chunks of the prompt).
//
//   acc[r, t] = sum_k W[r, k] * b[t, k]        W: [rows, K] 16-bit weights, b: T activation rows
//
// "Swap-AB": the weight rows are the M = 128 operand of tcgen05.mma (they fill the tensor-memory lanes), the token
// rows are N.  Activations are fp32 everywhere else; here each row enters twice, as hi = round16(v) and
// lo = round16(v - hi), in N = 16 (T <= 8) or 32 columns, and the two accumulator columns are added in the epilogue,
// so the product keeps about 16 (bf16) or 22 (fp16) mantissa bits of the activation while the weights stream exactly
// once.
// The pass is bound by HBM weight streaming, so the work is cut for equal bytes per SM ("stream-K"): the units
// (128-row tile, 64-column K block) are numbered tile-major and CTA c takes the contiguous range
// [U c / G, U (c+1) / G).  A CTA that holds only part of a tile's K range writes its 128 x N partial
// accumulator to a workspace and takes a ticket; the last one to arrive for a tile adds the partials in CTA
// order (fixed, so results do not depend on timing) and runs the epilogue for that tile:
//   STORE  qkv[t, r] = s_t * acc                     (s_t = RMSNorm scale of token t, see below)
//   RESID  x[t, r] += acc; next input hi/lo(x * g_next[r]); per-tile sum of x^2 per token; optional hidden tap
//   SILU   rows interleave gate/up: h = silu(s_t g) * (s_t u) -> hi/lo(h), the down projection's input
//   HEAD   logits = clamp(s_t * acc) -> per-tile softmax statistics and argmax per token (Eq. 1-4)
// RMSNorm is split around the GEMM: the input rows hold x * gain (unscaled), the producer of x leaves per-tile
// sums of squares, and s_t = rsqrt(mean x^2 + eps) multiplies the accumulator in the epilogue (a per-token
// scalar commutes with the contraction).
// Warp roles as in the scoring kernel: warp 0 TMA producer (A 128 x 64 and B N x 64 tiles, 128-byte swizzle,
// 4-stage ring, two CTAs per SM), warp 1 tensor-memory allocation and MMA issue, warps 2-5 epilogue (thread = weight row).
// All waits are bounded; nothing waits on another CTA (the ticket is taken, never polled).
#include <math.h>
#include <string.h>

#include "tc_common.cuh"

namespace {

constexpr int VM = 128, VSTAGES = 4;   // 80 KB of tiles per CTA, so that the next launch's CTA fits beside this one
constexpr int VA_BYTES = VM * TC_BK * 2, VB_BYTES = 32 * TC_BK * 2, VSTAGE_BYTES = VA_BYTES + VB_BYTES;   // 20 KB
constexpr int VTHREADS = 192;
constexpr int WS_LD = 32;   // floats per row of a workspace partial

struct VSmem {
    unsigned long long full[VSTAGES], empty[VSTAGES], tfull[2], tempty[2];
    unsigned tmem_base;
    int abort, is_last;
    float scale[CL_SLOTS];
    float red[4][CL_SLOTS];
    ClHeadPartial hp[4][CL_SLOTS];
};

struct Seg {
    int m, kb0, kb1;
};

// CTA c's unit range and its idx-th segment (a maximal run of units inside one tile); false past the end.
__device__ __forceinline__ bool segment_of(long long U, int G, int KB, int c, int idx, Seg &s) {
    if (c >= G) return false;
    long long u = U * c / G;
    const long long u1 = U * (c + 1) / G;
    for (int i = 0; u < u1; ++i) {
        const int m = (int)(u / KB), kb0 = (int)(u % KB);
        const int kb1 = (int)min((long long)KB, kb0 + (u1 - u));
        if (i == idx) {
            s.m = m; s.kb0 = kb0; s.kb1 = kb1;
            return true;
        }
        u += kb1 - kb0;
    }
    return false;
}
__device__ __forceinline__ int cta_of_unit(long long U, int G, long long u) {
    int c = (int)(u * G / U);
    while (c + 1 < G && U * (c + 1) / G <= u) ++c;
    while (c > 0 && U * c / G > u) --c;
    return c;
}

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// Barrier of the 128 epilogue threads that also tells every one of them whether all of them saw ok.
__device__ __forceinline__ bool epi_all(bool ok) {
    int r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.s32 p, %1, 0;\n\tbar.red.and.pred q, 1, 128, p;\n\tselp.s32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((int)ok)
        : "memory");
    return r != 0;
}

__device__ __forceinline__ ClHeadPartial v_merge(const ClHeadPartial &a, const ClHeadPartial &b) {
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
__device__ __forceinline__ ClHeadPartial v_shfl_xor(const ClHeadPartial &a, int o) {
    ClHeadPartial r;
    r.m = __shfl_xor_sync(0xffffffffu, a.m, o);
    r.z = __shfl_xor_sync(0xffffffffu, a.z, o);
    r.s = __shfl_xor_sync(0xffffffffu, a.s, o);
    r.idx = __shfl_xor_sync(0xffffffffu, a.idx, o);
    return r;
}

// Adds the partial accumulators of tile m (from CTAs c_first .. c_last, in that order) into v: PB partials are in
// flight at a time, NQ float4 each (N = 4 NQ columns).  (Eight in flight measured slower: tiles cut over two or three
// CTAs are the common case and the extra requests only load L2.)
template <int NQ, int PB>
__device__ __forceinline__ void add_partials(float (&v)[32], const ClSkinnyArgs &a, long long U, int G, int m, int c_first,
                                             int c_last, int rloc) {
    for (int cc0 = c_first; cc0 <= c_last; cc0 += PB) {
        float4 p[PB][NQ];
#pragma unroll
        for (int j = 0; j < PB; ++j) {
            const int cc = min(cc0 + j, c_last);
            const int seg_idx = m - (int)((U * cc / G) / a.KB);   // tiles CTA cc touches are consecutive
            const float4 *src = (const float4 *)(a.ws + (((size_t)cc * CL_V_MAXSEG + seg_idx) * VM + rloc) * WS_LD);
#pragma unroll
            for (int i = 0; i < NQ; ++i) p[j][i] = __ldcg(src + i);
        }
#pragma unroll
        for (int j = 0; j < PB; ++j) {
            if (cc0 + j <= c_last) {
#pragma unroll
                for (int i = 0; i < NQ; ++i) {
                    v[4 * i] += p[j][i].x; v[4 * i + 1] += p[j][i].y; v[4 * i + 2] += p[j][i].z; v[4 * i + 3] += p[j][i].w;
                }
            }
        }
    }
}

__global__ void __launch_bounds__(VTHREADS, 2)
k_skinny(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, ClSkinnyArgs a) {
    if (a.st && a.st->done) return;   // written only between launches: uniform over the grid
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *tiles = (unsigned char *)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    VSmem *sm = (VSmem *)(tiles + (size_t)VSTAGES * VSTAGE_BYTES);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int MT = (a.rows + VM - 1) / VM;
    const long long U = (long long)MT * a.KB;
    // the split runs over min(grid, U) CTAs so that every CTA of the split owns at least one unit (a tile's
    // partials then come from a gap-free range of CTAs); CTAs beyond it have no segment
    const int c = blockIdx.x, G = (int)min((long long)gridDim.x, U);
    const unsigned b_bytes = (unsigned)a.N * TC_BK * 2;

    if (tid == 0) {
        for (int i = 0; i < VSTAGES; ++i) {
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
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 64;" ::"r"(s_u32(&sm->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem = *(volatile unsigned *)&sm->tmem_base;
    // Programmatic dependent launch: the next launch on the stream may start beside this one as soon as an SM has
    // room, and this one may have started while its predecessor was still finishing.  Weights never change, so the
    // producer fills the ring with weight tiles right away; everything a predecessor writes (activation rows, sums
    // of squares, residual stream, workspace, tickets) is only touched after griddepcontrol.wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            unsigned stage = 0, par = 0, issued[VSTAGES];
            for (int i = 0; i < VSTAGES; ++i) issued[i] = 2u;
            bool ok = true, upstream_done = false;
            int pend_kb[VSTAGES], npend = 0;   // stages whose weight tile is on its way but whose activation tile is not
            Seg sg;
            for (int si = 0; ok && segment_of(U, G, a.KB, c, si, sg); ++si) {
                for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
                    if (!upstream_done && npend == VSTAGES) {
                        asm volatile("griddepcontrol.wait;" ::: "memory");
                        upstream_done = true;
                        for (int i = 0; i < npend; ++i)
                            tma_load_2d(tiles + (size_t)i * VSTAGE_BYTES + VA_BYTES, &mapB, pend_kb[i] * TC_BK, 0, &sm->full[i]);
                    }
                    if (!bar_wait(&sm->empty[stage], par ^ 1u, &sm->abort, a.err)) { ok = false; break; }
                    unsigned char *dst = tiles + (size_t)stage * VSTAGE_BYTES;
                    bar_expect(&sm->full[stage], VA_BYTES + b_bytes);
                    tma_load_2d(dst, &mapA, kb * TC_BK, sg.m * VM, &sm->full[stage]);
                    if (upstream_done) tma_load_2d(dst + VA_BYTES, &mapB, kb * TC_BK, 0, &sm->full[stage]);
                    else pend_kb[npend++] = kb;   // (the first VSTAGES loads use stages 0, 1, ... in order)
                    issued[stage] = par;
                    if (++stage == VSTAGES) { stage = 0; par ^= 1u; }
                }
            }
            if (!upstream_done) {   // fewer than VSTAGES k-blocks in all
                asm volatile("griddepcontrol.wait;" ::: "memory");
                for (int i = 0; i < npend; ++i)
                    tma_load_2d(tiles + (size_t)i * VSTAGE_BYTES + VA_BYTES, &mapB, pend_kb[i] * TC_BK, 0, &sm->full[i]);
            }
            if (!ok) {   // gave up: let the copies in flight land before the CTA may exit (bounded)
                for (int i = 0; i < VSTAGES; ++i) {
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
            const unsigned idesc = umma_idesc(VM, a.N, a.f16);
            unsigned stage = 0, par = 0;
            bool ok = true;
            Seg sg;
            for (int si = 0; ok && segment_of(U, G, a.KB, c, si, sg); ++si) {
                const int b = si & 1;
                if (!bar_wait(&sm->tempty[b], (((unsigned)si >> 1) & 1u) ^ 1u, &sm->abort, a.err)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
                    if (!bar_wait(&sm->full[stage], par, &sm->abort, a.err)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned a_addr = s_u32(tiles + (size_t)stage * VSTAGE_BYTES), b_addr = a_addr + VA_BYTES;
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k)
                        umma_bf16(tmem + (unsigned)b * 32, umma_desc(a_addr + k * 32), umma_desc(b_addr + k * 32), idesc,
                                  (unsigned)((kb - sg.kb0) | k));
                    umma_commit(&sm->empty[stage]);
                    if (++stage == VSTAGES) { stage = 0; par ^= 1u; }
                }
                if (ok) umma_commit(&sm->tfull[b]);
            }
        }
    } else {
        // ---------------- epilogue: thread = one weight row of the tile ----------------
        const int et = tid - 64;                       // 0 .. 127
        const int q = warp & 3, rloc = q * 32 + lane;  // tensor-memory lane = row inside the tile
        const int ew = et >> 5;                        // epilogue warp 0 .. 3 (for shared tables)
        const int T = a.T, nh = a.N >> 1;
        asm volatile("griddepcontrol.wait;" ::: "memory");   // from here on this warp reads what earlier launches wrote
        // RMSNorm scale of every token row: fixed-order sum of the producer's per-tile sums of squares
        if (et < T) {
            float sc = 1.f;
            if (a.ssq_in) {
                float ss = 0.f;
                for (int m = 0; m < a.ssq_tiles; ++m) ss += __ldcg(a.ssq_in + (size_t)m * CL_SLOTS + et);
                sc = 1.0f / sqrtf(ss * a.inv_dim + a.eps);
            }
            sm->scale[et] = sc;
        }
        epi_sync();
        const int pos0 = a.st ? a.st->ctx + a.row0 : a.row0;
        Seg sg;
        for (int si = 0; segment_of(U, G, a.KB, c, si, sg); ++si) {
            const int b = si & 1;
            if (!epi_all(bar_wait(&sm->tfull[b], ((unsigned)si >> 1) & 1u, &sm->abort, a.err))) break;   // uniform
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float v[32];
            tmem_ld32(tmem + ((unsigned)(q * 32) << 16) + (unsigned)(b * 32), v);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            bar_arrive(&sm->tempty[b]);   // the accumulator is in registers: the buffer may be reused
            const int m = sg.m, row = m * VM + rloc;
            if (!(sg.kb0 == 0 && sg.kb1 == a.KB)) {
                // partial K range: publish, take a ticket; the last arrival adds all partials in CTA order
                float4 *dst = (float4 *)(a.ws + (((size_t)c * CL_V_MAXSEG + si) * VM + rloc) * WS_LD);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (4 * i < a.N) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                epi_sync();
                const int c_first = cta_of_unit(U, G, (long long)m * a.KB), c_last = cta_of_unit(U, G, (long long)(m + 1) * a.KB - 1);
                if (et == 0) {
                    const unsigned prev = ticket_acq_rel(a.tickets + m);
                    const int last = (prev == (unsigned)(c_last - c_first));
                    if (last) a.tickets[m] = 0u;
                    sm->is_last = last;
                }
                epi_sync();
                if (!sm->is_last) continue;
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = 0.f;
                if (a.N == 16) add_partials<4, 4>(v, a, U, G, m, c_first, c_last, rloc);
                else add_partials<8, 4>(v, a, U, G, m, c_first, c_last, rloc);
            }
            // ---- epilogue of a complete tile: tot[t] = hi column + lo column (loops unrolled so that the accumulator
            // stays in registers; rows of a pass never exceed CL_MAX_T)
            const bool live = row < a.rows;
            float tot[CL_MAX_T];
#pragma unroll
            for (int t = 0; t < CL_MAX_T; ++t) tot[t] = v[t] + (nh == 8 ? v[(8 + t) & 31] : v[(16 + t) & 31]);
            if (a.epi == CL_VEPI_STORE) {
#pragma unroll
                for (int t = 0; t < CL_MAX_T; ++t)
                    if (live && t < T) a.out[(size_t)t * a.ld + row] = sm->scale[t] * tot[t];
            } else if (a.epi == CL_VEPI_RESID) {
                const float g = live ? a.gnext[row] : 0.f;
                float xo[CL_MAX_T];
#pragma unroll
                for (int t = 0; t < CL_MAX_T; ++t) xo[t] = (live && t < T) ? __ldcg(a.out + (size_t)t * a.ld + row) : 0.f;   // all reads first
#pragma unroll
                for (int t = 0; t < CL_MAX_T; ++t) {
                    if (t < T) {   // uniform
                        const float xn = (live ? xo[t] + tot[t] : 0.f);
                        if (live) {
                            a.out[(size_t)t * a.ld + row] = xn;
                            store_split(a.bnext + (size_t)t * a.bn_ld + row, a.bnext + (size_t)(a.nh + t) * a.bn_ld + row, xn * g, a.f16);
                            if (a.tap) {
                                const size_t o = (size_t)((pos0 + t) % a.tap_P) * a.rows + row;
                                ((unsigned short *)a.tap)[o] = f32_to_b16(xn, a.f16);
                            }
                        }
                        float ss = xn * xn;
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
                        if (lane == 0) sm->red[ew][t] = ss;
                    }
                }
                epi_sync();
                if (et < T) a.ssq_out[(size_t)m * CL_SLOTS + et] = (sm->red[0][et] + sm->red[1][et]) + (sm->red[2][et] + sm->red[3][et]);
                epi_sync();
            } else if (a.epi == CL_VEPI_SILU) {
#pragma unroll
                for (int t = 0; t < CL_MAX_T; ++t) {
                    if (t >= T) break;   // uniform
                    const float mine = sm->scale[t] * tot[t];
                    const float other = __shfl_xor_sync(0xffffffffu, mine, 1);   // gate (even row) / up (odd row) pair
                    if (live && !(lane & 1)) {
                        const float h = mine / (1.f + expf(-mine)) * other;
                        store_split(a.bnext + (size_t)t * a.bn_ld + (row >> 1), a.bnext + (size_t)(a.nh + t) * a.bn_ld + (row >> 1), h, a.f16);
                    }
                }
            } else {
#pragma unroll
                for (int t = 0; t < CL_MAX_T; ++t) {
                    if (t >= T) break;   // uniform
                    ClHeadPartial p{0.f, 0.f, 0.f, 0x7fffffff};
                    if (live) {
                        const float l = fminf(fmaxf(sm->scale[t] * tot[t], -CL_LOGIT_CLAMP), CL_LOGIT_CLAMP);
                        if (a.logits) a.logits[(size_t)t * a.rows + row] = l;
                        p = ClHeadPartial{l, 1.f, 0.f, row};
                    }
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const ClHeadPartial other = v_shfl_xor(p, o);
                        p = ((lane & o) == 0) ? v_merge(p, other) : v_merge(other, p);
                    }
                    if (lane == 0) sm->hp[ew][t] = p;
                }
                epi_sync();
                if (et < T) {
                    // warps hold the tile's rows in tensor-memory quadrant order: combine in row order
                    const int w0 = (0 + 2) & 3, w1 = (1 + 2) & 3, w2 = (2 + 2) & 3, w3 = (3 + 2) & 3;
                    ClHeadPartial r = v_merge(v_merge(sm->hp[w0][et], sm->hp[w1][et]), v_merge(sm->hp[w2][et], sm->hp[w3][et]));
                    a.head_part[(size_t)m * CL_SLOTS + et] = r;
                }
                epi_sync();
            }
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 64;" ::"r"(tmem) : "memory");
    }
}

// Start of a pass: x[t] = E[token t]; the first GEMM's input rows hi/lo(x * g) and the per-tile sums of squares.
__global__ void k_pass_begin(const unsigned short *embed, const int *tok, int T, int d, float *x, __nv_bfloat16 *bnext, int nh,
                             const float *g, float *ssq_out, const ClDevState *st, int f16) {
    if (st->done) return;
    __shared__ float red[4][CL_SLOTS];
    const int row = blockIdx.x * 128 + threadIdx.x, lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int t = 0; t < T; ++t) {
        float v = 0.f;
        if (row < d) {
            v = b16_to_f32(embed[(size_t)tok[t] * d + row], f16);
            x[(size_t)t * d + row] = v;
            store_split(bnext + (size_t)t * d + row, bnext + (size_t)(nh + t) * d + row, v * g[row], f16);
        }
        float ss = v * v;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) red[w][t] = ss;
    }
    __syncthreads();
    if (threadIdx.x < T)
        ssq_out[(size_t)blockIdx.x * CL_SLOTS + threadIdx.x] =
            (red[0][threadIdx.x] + red[1][threadIdx.x]) + (red[2][threadIdx.x] + red[3][threadIdx.x]);
}

// Merge the per-tile LM-head statistics of every token row (one warp per row, fixed order) and evaluate Eq. 2-4.
__global__ void k_head_finalize(const ClHeadPartial *part, int tiles, int T, float inv_log_v, int *out_tok, float *out_pmax,
                                float *out_conf, const ClDevState *st) {
    if (st && st->done) return;
    const int t = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (t >= T) return;
    ClHeadPartial p{0.f, 0.f, 0.f, 0x7fffffff};
    for (int m = lane; m < tiles; m += 32) {
        const ClHeadPartial *src = part + (size_t)m * CL_SLOTS + t;
        ClHeadPartial q;
        q.m = __ldcg(&src->m); q.z = __ldcg(&src->z); q.s = __ldcg(&src->s); q.idx = __ldcg(&src->idx);
        p = v_merge(p, q);
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const ClHeadPartial other = v_shfl_xor(p, o);
        p = ((lane & o) == 0) ? v_merge(p, other) : v_merge(other, p);
    }
    if (lane == 0) {
        const float H = logf(p.z) - p.s / p.z;
        if (out_tok) out_tok[t] = p.idx;
        if (out_pmax) out_pmax[t] = 1.f / p.z;
        if (out_conf) out_conf[t] = 1.f - H * inv_log_v;
    }
}

}  // namespace

bool cl_make_tensor_map(ClTensorMap *m, const void *base, int rows, int cols, int box_rows, int f16) {
    static_assert(sizeof(ClTensorMap) >= sizeof(CUtensorMap), "tensor map storage");
    return make_map((CUtensorMap *)m->bytes, base, rows, cols, box_rows, f16);
}

cudaError_t cl_launch_skinny(const ClTensorMap &mapA, const ClTensorMap &mapB, const ClSkinnyArgs &a, int grid, cudaStream_t s) {
    const size_t smem = (size_t)VSTAGES * VSTAGE_BYTES + sizeof(VSmem) + 1024;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_skinny, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(VTHREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_skinny, *(const CUtensorMap *)mapA.bytes, *(const CUtensorMap *)mapB.bytes, a);
}

cudaError_t cl_launch_pass_begin(const void *embed, const int *tok, int T, int d, float *x, __nv_bfloat16 *bnext, int nh,
                                 const float *g, float *ssq_out, const ClDevState *st, int f16, cudaStream_t s) {
    k_pass_begin<<<(d + 127) / 128, 128, 0, s>>>((const unsigned short *)embed, tok, T, d, x, bnext, nh, g, ssq_out, st, f16);
    return cudaGetLastError();
}

cudaError_t cl_launch_head_finalize(const ClHeadPartial *part, int tiles, int T, float inv_log_v, int *out_tok, float *out_pmax,
                                    float *out_conf, const ClDevState *st, cudaStream_t s) {
    k_head_finalize<<<1, 32 * T, 0, s>>>(part, tiles, T, inv_log_v, out_tok, out_pmax, out_conf, st);
    return cudaGetLastError();
}

// ---- attention of the T rows of a pass over the KV cache ----------------------------------------------------
// grid (H, S): the keys [0, base + T) of a head (base = first row's position; the rows' own keys are already in
// the cache, rotated) are cut into S contiguous parts, a part into 8 warp ranges.  A warp walks its range 32 keys
// at a time: every key row is read once (16 bytes per lane) and scored against all T query rows, row t masking keys
// beyond its own position; per row an online softmax; every value row is read once and accumulated into all rows.
// The CTA merges its warps in shared memory; the last CTA of a head (ticket) merges the S parts in order and
// writes the output rows as fp32 and as bf16 hi/lo parts (the next GEMM's input).
namespace {

constexpr int AR_WARPS = 8;
constexpr int AR_MAXS = 8;   // most parts the keys of a head are cut into

template <typename ST>
__device__ __forceinline__ ST ar_from_f32(float v);
template <>
__device__ __forceinline__ __nv_bfloat16 ar_from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <>
__device__ __forceinline__ __half ar_from_f32<__half>(float v) { return __float2half_rn(v); }
template <typename ST>
__device__ __forceinline__ constexpr int ar_is_f16() { return 0; }
template <>
__device__ __forceinline__ constexpr int ar_is_f16<__half>() { return 1; }

// (Loops over keys stay rolled and the row count is a template parameter: the kernel runs its code once, so its
// time is instruction fetch, and a fully unrolled version measured 55 us against a few us of work.)
template <typename ST, int HD, int T>
__global__ void __launch_bounds__(AR_WARPS * 32) k_attn_rows(ClAttnArgs a, int S) {
    // programmatic dependent launch: the next launch (the output projection) may set itself up beside this one;
    // everything an earlier launch wrote is read after the wait
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int2 ctx_done = *(const int2 *)a.st;   // (ctx, done): one load
    if (ctx_done.y) return;
    constexpr int EPL = 16 / (int)sizeof(ST), LPK = HD / EPL, KPW = 32 / LPK, VPL = HD / 32;
    constexpr int REC = HD + 2;
    extern __shared__ __align__(16) float wrec[];   // [AR_WARPS][T][REC], then per warp 32 key rows and 32 value rows
    __shared__ int is_last;
    constexpr int ROWB = HD * (int)sizeof(ST);                 // bytes of one cached row of a head
    constexpr int CPR = ROWB / 16;                              // 16-byte chunks per row
    constexpr size_t WREC_BYTES = ((size_t)AR_WARPS * T * REC * sizeof(float) + 15) & ~(size_t)15;
    unsigned char *stage_k = (unsigned char *)wrec + WREC_BYTES + (size_t)(threadIdx.x >> 5) * 2 * 32 * ROWB;
    unsigned char *stage_v = stage_k + 32 * ROWB;
    const int h = blockIdx.x, s = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int base = ctx_done.x + a.row0, nkeys = base + T, d = a.d_model;
    if (nkeys > a.max_seq) return;
    const int k0 = (int)((long long)nkeys * s / S), k1 = (int)((long long)nkeys * (s + 1) / S);
    const int kw0 = k0 + (k1 - k0) * warp / AR_WARPS, kw1 = k0 + (k1 - k0) * (warp + 1) / AR_WARPS;
    const int sub = lane / LPK, li = lane % LPK;
    const float scale = rsqrtf((float)HD);
    const int kvh = h / (a.n_heads / a.n_kv_heads);                       // grouped-query attention
    ST *Kc = (ST *)a.kcache + (size_t)kvh * a.max_seq * HD;   // cache layout [kv head][position][hd]
    ST *Vc = (ST *)a.vcache + (size_t)kvh * a.max_seq * HD;

    constexpr int HALF = HD / 2;
    const int kvd = a.n_kv_heads * HD;
    float qr[T][EPL];
    {
        // vector loads, all requested before any is used; rotary embedding at the row's position (pairs i, i + hd / 2)
        const int i0 = li * EPL, ip = (i0 + HALF) % HD;
        float4 own[T][EPL / 4], par[T][EPL / 4], cs[T][EPL / 2];
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const float *qrow = a.q + (size_t)t * a.ld_q + h * HD;
#pragma unroll
            for (int v = 0; v < EPL / 4; ++v) {
                own[t][v] = *(const float4 *)(qrow + i0 + 4 * v);
                if (a.rope_cs) par[t][v] = *(const float4 *)(qrow + ip + 4 * v);
            }
            if (a.rope_cs) {
                const float4 *c4 = (const float4 *)(a.rope_cs + (size_t)(base + t) * HALF + (i0 % HALF));
#pragma unroll
                for (int v = 0; v < EPL / 2; ++v) cs[t][v] = c4[v];
            }
        }
#pragma unroll
        for (int t = 0; t < T; ++t)
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                float v = ((const float *)own[t])[e];
                if (a.rope_cs) {
                    const float p = ((const float *)par[t])[e], c = ((const float *)cs[t])[2 * e], sn = ((const float *)cs[t])[2 * e + 1];
                    v = (i0 < HALF) ? v * c - p * sn : v * c + p * sn;
                }
                qr[t][e] = v * scale;
            }
    }
    float m_run[T], l_run[T], o_run[T][VPL];
#pragma unroll
    for (int t = 0; t < T; ++t) {
        m_run[t] = -INFINITY;
        l_run[t] = 0.f;
#pragma unroll
        for (int e = 0; e < VPL; ++e) o_run[t][e] = 0.f;
    }
    for (int j0 = kw0; j0 < kw1; j0 += 32) {
        const int n = min(32, kw1 - j0);
        const int n_old = a.rope_cs ? max(0, min(n, base - j0)) : n;   // rows of this pass that are in the cache already
        // stage this pass's key and value rows in shared memory: every 16-byte piece is requested before any is used,
        // so the pass costs one memory round trip; the (rolled) loops below then read shared memory
        __syncwarp();
        {
            const uint4 *gk = (const uint4 *)(Kc + (size_t)j0 * HD), *gv = (const uint4 *)(Vc + (size_t)j0 * HD);
            uint4 tk[CPR], tv[CPR];
#pragma unroll
            for (int it = 0; it < CPR; ++it) {
                const int cidx = it * 32 + lane;   // chunk cidx of the pass: row cidx / CPR
                if (cidx < n_old * CPR) {
                    tk[it] = gk[cidx];
                    tv[it] = gv[cidx];
                }
            }
#pragma unroll
            for (int it = 0; it < CPR; ++it) {
                const int cidx = it * 32 + lane;
                if (cidx < n_old * CPR) {
                    ((uint4 *)stage_k)[cidx] = tk[it];
                    ((uint4 *)stage_v)[cidx] = tv[it];
                }
            }
        }
        if (n_old < n && sizeof(ST) == 2) {
            // the pass's own rows: k and v come raw from the projection; rotate k at its position, round both to the
            // storage type, stage them, and (one query head per key/value head) append them to the cache
            const bool writer = h % (a.n_heads / a.n_kv_heads) == 0;
#pragma unroll 4
            for (int idx = lane; idx < (n - n_old) * HALF; idx += 32) {
                const int r = n_old + idx / HALF, i = idx % HALF, j = j0 + r;
                const float *krow = a.q + (size_t)(j - base) * a.ld_q + d + kvh * HD, *vrow = krow + kvd;
                const float2 cs = a.rope_cs[(size_t)j * HALF + i];
                const float ka = krow[i], kb = krow[i + HALF];
                const ST k0 = ar_from_f32<ST>(ka * cs.x - kb * cs.y), k1 = ar_from_f32<ST>(kb * cs.x + ka * cs.y);
                const ST v0 = ar_from_f32<ST>(vrow[i]), v1 = ar_from_f32<ST>(vrow[i + HALF]);
                ST *sk = (ST *)(stage_k + (size_t)r * ROWB), *sv = (ST *)(stage_v + (size_t)r * ROWB);
                sk[i] = k0; sk[i + HALF] = k1; sv[i] = v0; sv[i + HALF] = v1;
                if (writer) {
                    ST *ck = Kc + (size_t)j * HD, *cv = Vc + (size_t)j * HD;
                    ck[i] = k0; ck[i + HALF] = k1; cv[i] = v0; cv[i + HALF] = v1;
                }
            }
        }
        __syncwarp();
        float sc[T];   // lane j: score of key j0 + j against row t
#pragma unroll
        for (int t = 0; t < T; ++t) sc[t] = -INFINITY;
#pragma unroll 1
        for (int jb = 0; jb < n; jb += KPW) {   // (uniform bound: keys past n have no score)
            const int j = jb + sub;
            float kf[EPL];
#pragma unroll
            for (int e = 0; e < EPL; ++e) kf[e] = 0.f;
            if (j < n) {
                const uint4 raw = *(const uint4 *)(stage_k + (size_t)j * ROWB + li * 16);
                if (sizeof(ST) == 2) {
                    const unsigned u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        ClPair16<ST>::get(u[e], kf[(2 * e) % EPL], kf[(2 * e + 1) % EPL]);
                    }
                } else {
                    kf[0] = __uint_as_float(raw.x); kf[1 % EPL] = __uint_as_float(raw.y);
                    kf[2 % EPL] = __uint_as_float(raw.z); kf[3 % EPL] = __uint_as_float(raw.w);
                }
            }
#pragma unroll
            for (int t = 0; t < T; ++t) {
                if (t < T) {   // uniform
                    float v = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) v = fmaf(qr[t][e], kf[e], v);
#pragma unroll
                    for (int o = LPK >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
#pragma unroll
                    for (int k = 0; k < KPW; ++k) {
                        const float w = __shfl_sync(0xffffffffu, v, k * LPK);
                        if (lane == jb + k && jb + k < n && j0 + jb + k <= base + t) sc[t] = w;   // causal mask
                    }
                }
            }
        }
        float p[T];
#pragma unroll
        for (int t = 0; t < T; ++t) {
            p[t] = 0.f;
            if (t < T) {
                float mx = sc[t];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float m_new = fmaxf(mx, m_run[t]);
                if (m_new > -INFINITY) {   // uniform over the warp
                    p[t] = (sc[t] > -INFINITY) ? expf(sc[t] - m_new) : 0.f;
                    const float resc = (l_run[t] > 0.f) ? expf(m_run[t] - m_new) : 0.f;
                    float ps = p[t];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
                    l_run[t] = fmaf(l_run[t], resc, ps);
#pragma unroll
                    for (int e = 0; e < VPL; ++e) o_run[t][e] *= resc;
                    m_run[t] = m_new;
                }
            }
        }
        // value rows: 8 at a time in flight (rows past the end repeat the last one; their weights are 0)
#pragma unroll 1
        for (int jh = 0; jh < 32; jh += 8) {
            if (jh < n) {   // uniform
                float vv[8][VPL];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const ST *vp = (const ST *)(stage_v + (size_t)min(jh + j, n - 1) * ROWB) + lane * VPL;
                    if (sizeof(ST) == 2 && VPL == 4) {
                        const uint2 u = *(const uint2 *)vp;
                        ClPair16<ST>::get(u.x, vv[j][0], vv[j][1 % VPL]);
                        ClPair16<ST>::get(u.y, vv[j][2 % VPL], vv[j][3 % VPL]);
                    } else {
#pragma unroll
                        for (int e = 0; e < VPL; ++e) vv[j][e] = (float)vp[e];
                    }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
#pragma unroll
                    for (int t = 0; t < T; ++t) {
                        if (t < T) {
                            const float pj = __shfl_sync(0xffffffffu, p[t], jh + j);
#pragma unroll
                            for (int e = 0; e < VPL; ++e) o_run[t][e] = fmaf(pj, vv[j][e], o_run[t][e]);
                        }
                    }
                }
            }
        }
    }
    // merge the warps of this CTA (fixed order)
#pragma unroll
    for (int t = 0; t < T; ++t) {
        {
            float *r = wrec + ((size_t)warp * T + t) * REC;
            if (lane == 0) { r[0] = m_run[t]; r[1] = l_run[t]; }
#pragma unroll
            for (int e = 0; e < VPL; ++e) r[2 + lane * VPL + e] = o_run[t][e];
        }
    }
    __syncthreads();
    float *part = a.part + ((size_t)h * S + s) * T * REC;
    for (int i = tid; i < T * HD; i += blockDim.x) {
        const int t = i / HD, e = i % HD;
        float M = -INFINITY;
        for (int w = 0; w < AR_WARPS; ++w) {
            const float *r = wrec + ((size_t)w * T + t) * REC;
            if (r[1] > 0.f) M = fmaxf(M, r[0]);
        }
        float Ls = 0.f, O = 0.f;
        for (int w = 0; w < AR_WARPS; ++w) {
            const float *r = wrec + ((size_t)w * T + t) * REC;
            if (r[1] > 0.f) {
                const float f = expf(r[0] - M);
                Ls = fmaf(r[1], f, Ls);
                O = fmaf(r[2 + e], f, O);
            }
        }
        if (e == 0) { part[(size_t)t * REC] = M; part[(size_t)t * REC + 1] = Ls; }
        part[(size_t)t * REC + 2 + e] = O;
    }
    __syncthreads();
    if (tid == 0) {
        const unsigned prev = ticket_acq_rel(a.tickets + h);
        is_last = (prev == (unsigned)S - 1);
        if (is_last) a.tickets[h] = 0u;
    }
    __syncthreads();
    if (!is_last) return;
    // every part's (max, sum, output element) of every output of this thread is requested before any is used:
    // one round trip in all, not one per part and output
    constexpr int NOUT = (T * HD + AR_WARPS * 32 - 1) / (AR_WARPS * 32);
    float pm[NOUT][AR_MAXS], pl[NOUT][AR_MAXS], po[NOUT][AR_MAXS];
#pragma unroll
    for (int it = 0; it < NOUT; ++it) {
        const int i = min(it * AR_WARPS * 32 + tid, T * HD - 1), t = i / HD, e = i % HD;
        const float *p0 = a.part + (size_t)h * S * T * REC + (size_t)t * REC;
#pragma unroll
        for (int s2 = 0; s2 < AR_MAXS; ++s2) {
            const float *ps = p0 + (size_t)min(s2, S - 1) * T * REC;
            pm[it][s2] = __ldcg(ps);
            pl[it][s2] = (s2 < S) ? __ldcg(ps + 1) : 0.f;
            po[it][s2] = __ldcg(ps + 2 + e);
        }
    }
#pragma unroll
    for (int it = 0; it < NOUT; ++it) {
        const int i = it * AR_WARPS * 32 + tid;
        if (i >= T * HD) break;
        const int t = i / HD, e = i % HD;
        float M = -INFINITY;
#pragma unroll
        for (int s2 = 0; s2 < AR_MAXS; ++s2)
            if (pl[it][s2] > 0.f) M = fmaxf(M, pm[it][s2]);
        float Ls = 0.f, O = 0.f;
#pragma unroll
        for (int s2 = 0; s2 < AR_MAXS; ++s2) {   // part order
            if (pl[it][s2] > 0.f) {
                const float f = expf(pm[it][s2] - M);
                Ls = fmaf(pl[it][s2], f, Ls);
                O = fmaf(po[it][s2], f, O);
            }
        }
        const float o = O / Ls;
        a.out[(size_t)t * d + h * HD + e] = o;
        if (a.out_b) {
            store_split(a.out_b + (size_t)t * d + h * HD + e, a.out_b + (size_t)(a.nh + t) * d + h * HD + e, o, sizeof(ST) == 2 && ar_is_f16<ST>());
        }
    }
}

}  // namespace

size_t cl_attn_rows_part_floats(int H, int S, int T, int hd) { return (size_t)H * S * T * (hd + 2); }

// a.part must hold cl_attn_rows_part_floats(H, S, T, hd) floats, a.tickets H zeroed counters.
cudaError_t cl_launch_attn_rows(int wdtype, int T, int S, const ClAttnArgs &a, cudaStream_t s) {
    if (S < 1 || S > AR_MAXS) return cudaErrorInvalidValue;
    dim3 grid(a.n_heads, S);
    const size_t es = wdtype != 0 ? 2 : 4;
    const size_t smem = (((size_t)AR_WARPS * T * (a.head_dim + 2) * sizeof(float) + 15) & ~(size_t)15) + (size_t)AR_WARPS * 2 * 32 * a.head_dim * es;
#define AR_LAUNCH(STT, HDV, TT)                                                                                          \
    {                                                                                                                 \
        cudaError_t e_ = cudaFuncSetAttribute(k_attn_rows<STT, HDV, TT>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                              (int)smem);                                                             \
        if (e_ != cudaSuccess) return e_;                                                                             \
        cudaLaunchConfig_t cfg_;                                                                                      \
        memset(&cfg_, 0, sizeof(cfg_));                                                                               \
        cfg_.gridDim = grid;                                                                                          \
        cfg_.blockDim = dim3(AR_WARPS * 32);                                                                          \
        cfg_.dynamicSmemBytes = smem;                                                                                 \
        cfg_.stream = s;                                                                                              \
        cudaLaunchAttribute attr_[1];                                                                                 \
        attr_[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                             \
        attr_[0].val.programmaticStreamSerializationAllowed = 1;                                                      \
        cfg_.attrs = attr_;                                                                                           \
        cfg_.numAttrs = 1;                                                                                            \
        return cudaLaunchKernelEx(&cfg_, k_attn_rows<STT, HDV, TT>, a, S);                                  \
    }
#define AR_CASE(TT)                                              \
    case TT:                                                     \
        if (wdtype == 1 && a.head_dim == 128) AR_LAUNCH(__nv_bfloat16, 128, TT) \
        else if (wdtype == 1 && a.head_dim == 64) AR_LAUNCH(__nv_bfloat16, 64, TT) \
        else if (wdtype == 2 && a.head_dim == 128) AR_LAUNCH(__half, 128, TT) \
        else if (wdtype == 2 && a.head_dim == 64) AR_LAUNCH(__half, 64, TT) \
        else return cudaErrorInvalidValue;                       \
        break;
    switch (T) {
        AR_CASE(1) AR_CASE(2) AR_CASE(3) AR_CASE(4) AR_CASE(5) AR_CASE(6) AR_CASE(7) AR_CASE(8) AR_CASE(9)
        default: return cudaErrorInvalidValue;
    }
#undef AR_CASE
#undef AR_LAUNCH
    return cudaGetLastError();
}
