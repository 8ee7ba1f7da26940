// Wide tensor-core GEMM for the prompt pass of a model stored in a 16-bit type (bf16 or fp16): the full-model pass of
// Section 3 over up to 512 prompt rows at a time, so that the weights stream from HBM once per 512 tokens instead
// of once per 8.
//
//   P[ks, t, r] = sum_{k in part ks} a[t, k] * W[r, k]        a: M activation rows, W: [rows, K] 16-bit weights
//
// Here the token rows are the M = 128 operand of tcgen05.mma (one tensor-memory lane per token) and 256 weight rows
// are N.  Activations are fp32 everywhere else; each row enters as hi = round16(v) and lo = round16(v - hi) in the
// weights' type and both products accumulate into the same fp32 accumulator, so the product keeps about 16 (bf16)
// or 22 (fp16) mantissa bits of the activation.
// One CTA computes one (token tile, weight tile, K part): the K range is cut into `splits` parts only to fill the
// 148 SMs when a matrix has few output tiles (4096 outputs are 16 tiles), and the parts are added in a fixed order
// by the small kernel that consumes the product:
//   k_wide_rope_append   q, k, v: rotary embedding at the row's position, cache append, q left in place
//   k_attn_wide          causal attention of the pass's rows over the cache -> hi/lo rows of the output projection
//   k_wide_norm          x += product (or x = E[token]); hidden tap; RMSNorm -> hi/lo rows of the next GEMM
//   k_wide_silu          h = silu(gate) * up on the interleaved gate/up product -> hi/lo rows of the down projection
// Warp roles: warp 0 TMA producer (A hi 128 x 64, A lo 128 x 64, B 256 x 64 as two 128-row boxes, 128-byte swizzle,
// 3-stage ring of 64 KB), warp 1 tensor-memory allocation and MMA issue, warps 2-5 store the accumulator (thread =
// token row, 256 consecutive outputs).  CTAs that share a weight tile are neighbours in the grid, so the tile comes
// from HBM once and from L2 for the other token tiles.  Every wait is bounded in time.
#include <math.h>

#include "tc_common.cuh"

namespace {

constexpr int WM = 128, WN = 256, WSTAGES = 3;
constexpr int WA_BYTES = WM * TC_BK * 2, WB_BYTES = WN * TC_BK * 2, WSTAGE_BYTES = 2 * WA_BYTES + WB_BYTES;   // 64 KB
constexpr int WTHREADS = 192;

struct WSmem {
    unsigned long long full[WSTAGES], empty[WSTAGES], tfull;
    unsigned tmem_base;
    int abort;
};

__global__ void __launch_bounds__(WTHREADS, 1)
k_wide(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, ClWideArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char *tiles = (unsigned char *)(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    WSmem *sm = (WSmem *)(tiles + (size_t)WSTAGES * WSTAGE_BYTES);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    if (cta >= a.MT * a.NT * a.splits) return;   // whole CTA leaves before anything is set up
    const int mt = cta % a.MT, nt = (cta / a.MT) % a.NT, ks = cta / (a.MT * a.NT);
    const int kb0 = (int)((long long)a.KB * ks / a.splits), kb1 = (int)((long long)a.KB * (ks + 1) / a.splits);

    if (tid == 0) {
        for (int i = 0; i < WSTAGES; ++i) {
            bar_init(&sm->full[i], 1);
            bar_init(&sm->empty[i], 1);
        }
        bar_init(&sm->tfull, 1);
        sm->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(s_u32(&sm->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem = *(volatile unsigned *)&sm->tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            unsigned stage = 0, par = 0, issued[WSTAGES];
            for (int i = 0; i < WSTAGES; ++i) issued[i] = 2u;
            bool ok = true;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!bar_wait(&sm->empty[stage], par ^ 1u, &sm->abort, a.err)) { ok = false; break; }
                unsigned char *dst = tiles + (size_t)stage * WSTAGE_BYTES;
                bar_expect(&sm->full[stage], WSTAGE_BYTES);
                tma_load_2d(dst, &mapA, kb * TC_BK, mt * WM, &sm->full[stage]);
                tma_load_2d(dst + WA_BYTES, &mapA, kb * TC_BK, a.lo_row0 + mt * WM, &sm->full[stage]);
                tma_load_2d(dst + 2 * WA_BYTES, &mapB, kb * TC_BK, nt * WN, &sm->full[stage]);
                tma_load_2d(dst + 2 * WA_BYTES + WB_BYTES / 2, &mapB, kb * TC_BK, nt * WN + WN / 2, &sm->full[stage]);
                issued[stage] = par;
                if (++stage == WSTAGES) { stage = 0; par ^= 1u; }
            }
            if (!ok) {   // gave up: still let the copies in flight land before the CTA may exit (bounded)
                for (int i = 0; i < WSTAGES; ++i) {
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
            const unsigned idesc = umma_idesc(WM, WN, a.f16);
            unsigned stage = 0, par = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!bar_wait(&sm->full[stage], par, &sm->abort, a.err)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const unsigned hi_addr = s_u32(tiles + (size_t)stage * WSTAGE_BYTES), lo_addr = hi_addr + WA_BYTES,
                               b_addr = hi_addr + 2 * WA_BYTES;
#pragma unroll
                for (int k = 0; k < TC_BK / 16; ++k) {
                    umma_bf16(tmem, umma_desc(hi_addr + k * 32), umma_desc(b_addr + k * 32), idesc, (unsigned)((kb - kb0) | k));
                    umma_bf16(tmem, umma_desc(lo_addr + k * 32), umma_desc(b_addr + k * 32), idesc, 1u);
                }
                umma_commit(&sm->empty[stage]);   // the stage is free once these multiply-adds have read it
                if (++stage == WSTAGES) { stage = 0; par ^= 1u; }
            }
            if (ok) umma_commit(&sm->tfull);
        }
    } else {
        // ---------------- store: one thread per token row ----------------
        const int q = warp & 3;                        // the tensor-memory lane quadrant this warp may read
        const int t = mt * WM + q * 32 + lane;
        if (bar_wait(&sm->tfull, 0u, &sm->abort, a.err)) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float *dst = a.P + ((size_t)ks * a.M + (size_t)min(t, a.M - 1)) * a.rows;
#pragma unroll 1
            for (int cb = 0; cb < WN / 32; ++cb) {
                float v[32];
                tmem_ld32(tmem + ((unsigned)(q * 32) << 16) + (unsigned)(cb * 32), v);   // (whole warp, also for rows past M)
                const int col0 = nt * WN + cb * 32;
                if (t < a.M) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (col0 + 4 * i + 4 <= a.rows)
                            *(float4 *)(dst + col0 + 4 * i) = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
    }
}

// One CTA per token row: x[t] = E[token] or x[t] += product parts (added in part order); the optional hidden tap;
// then the rows of the next GEMM: hi/lo(x * rsqrt(mean x^2 + eps) * g).
__global__ void __launch_bounds__(256) k_wide_norm(ClWideNormArgs a) {
    __shared__ float red[8];
    const int t = blockIdx.x, tid = threadIdx.x, d = a.d;
    float *xr = a.x + (size_t)t * d;
    const unsigned short *er = a.tok ? (const unsigned short *)a.embed + (size_t)a.tok[t] * d : nullptr;
    // only the last tap_P rows of the pass reach the ring: an earlier row of the same slot would be overwritten anyway
    unsigned short *tap = nullptr;
    if (a.tap && t >= a.M - a.tap_P) tap = (unsigned short *)a.tap + (size_t)((a.st->ctx + t) % a.tap_P) * d;
    float ss = 0.f;
    for (int i = tid * 4; i < d; i += 1024) {
        float4 v;
        if (er) {
            const uint2 u = *(const uint2 *)(er + i);
            pair16_to_f32(u.x, a.f16, v.x, v.y);
            pair16_to_f32(u.y, a.f16, v.z, v.w);
        } else {
            v = *(const float4 *)(xr + i);
            for (int s = 0; s < a.splits; ++s) {
                const float4 p = __ldcg((const float4 *)(a.P + ((size_t)s * a.M + t) * d + i));
                v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
            }
        }
        *(float4 *)(xr + i) = v;
        if (tap) {
            tap[i] = f32_to_b16(v.x, a.f16); tap[i + 1] = f32_to_b16(v.y, a.f16);
            tap[i + 2] = f32_to_b16(v.z, a.f16); tap[i + 3] = f32_to_b16(v.w, a.f16);
        }
        ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
    }
    if (!a.g) return;   // uniform
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += red[w];   // fixed order
    const float sc = 1.0f / sqrtf(tot / (float)d + a.eps);
    __nv_bfloat16 *hi = a.A + (size_t)t * d, *lo = a.A + (size_t)(a.lo_row0 + t) * d;
    for (int i = tid * 4; i < d; i += 1024) {
        const float4 v = *(const float4 *)(xr + i);   // this thread's own writes
        const float4 g = *(const float4 *)(a.g + i);
        store_split(hi + i, lo + i, v.x * sc * g.x, a.f16);
        store_split(hi + i + 1, lo + i + 1, v.y * sc * g.y, a.f16);
        store_split(hi + i + 2, lo + i + 2, v.z * sc * g.z, a.f16);
        store_split(hi + i + 3, lo + i + 3, v.w * sc * g.w, a.f16);
    }
}

// grid (M, H), hd / 2 threads: q, k, v of row t and head h from the QKV product parts; rotary embedding at position
// ctx + t; q goes back in place (part 0), k and v (the first Hkv heads) go to the cache [kv head][position][hd].
__global__ void k_wide_rope_append(float *P, int splits, int M, int hd, int d, int Hkv, const float2 *rope_cs,
                                   unsigned short *kcache, unsigned short *vcache, int max_seq, const ClDevState *st, int f16) {
    const int t = blockIdx.x, h = blockIdx.y, i = threadIdx.x, half = hd >> 1;
    const int pos = st->ctx + t;
    if (pos >= max_seq) return;
    const int kvd = Hkv * hd, ld = d + 2 * kvd;
    const size_t part = (size_t)M * ld;
    float *row = P + (size_t)t * ld;
    auto total = [&](int col) {
        float v = row[col];
        for (int s = 1; s < splits; ++s) v += __ldcg(row + (size_t)s * part + col);
        return v;
    };
    const float2 cs = rope_cs[(size_t)pos * half + i];
    const float qa = total(h * hd + i), qb = total(h * hd + i + half);
    row[h * hd + i] = qa * cs.x - qb * cs.y;
    row[h * hd + i + half] = qb * cs.x + qa * cs.y;
    if (h >= Hkv) return;
    const float ka = total(d + h * hd + i), kb = total(d + h * hd + i + half);
    unsigned short *kc = kcache + ((size_t)h * max_seq + pos) * hd, *vc = vcache + ((size_t)h * max_seq + pos) * hd;
    kc[i] = f32_to_b16(ka * cs.x - kb * cs.y, f16);
    kc[i + half] = f32_to_b16(kb * cs.x + ka * cs.y, f16);
    vc[i] = f32_to_b16(total(d + kvd + h * hd + i), f16);
    vc[i + half] = f32_to_b16(total(d + kvd + h * hd + i + half), f16);
}

// ---- causal attention of the rows of the pass over the cache -------------------------------------------------
// grid (H, blocks of 64 rows), 256 threads.  Row t sits at position ctx + t and attends to the keys 0 .. ctx + t
// (its own key is already in the cache).  The keys are walked 64 at a time; per tile the 64 x 64 scores
// S = Q K^T and the update O += P V are register-tiled fp32 products out of shared memory (thread (ty, tx): rows
// 4 ty .. 4 ty + 3; keys 4 tx .. 4 tx + 3 of S; columns tx * 4 + 64 v .. of O), with the usual running maximum and
// sum per row.  The 16 threads of a row group are half a warp, so row reductions are four shuffles.  Blocks of
// late rows see the most keys and are scheduled first.
constexpr int AQ = 64, AK = 64, APS = 68;   // rows per CTA, keys per tile, row stride of the probability tile

template <int HD>
__global__ void __launch_bounds__(256, 2)
k_attn_wide(const float *q, int ld_q, const unsigned short *kcache, const unsigned short *vcache, __nv_bfloat16 *out_b,
            int lo_row0, int M, int d, int H, int Hkv, int max_seq, const ClDevState *st, int f16) {
    constexpr int NV = HD / 64;                       // float4 column groups of O per thread
    constexpr int KP = (HD * AK > AQ * APS) ? HD * AK : AQ * APS;
    extern __shared__ __align__(16) float asm_[];
    float *Qt = asm_;              // [HD][AQ]   queries, transposed, scaled by 1 / sqrt(hd)
    float *Kt = Qt + HD * AQ;      // [HD][AK]   keys of the tile, transposed; reused as Ps [AQ][APS] (probabilities)
    float *Vs = Kt + KP;           // [AK][HD]   values of the tile
    float *Ps = Kt;
    const int h = blockIdx.x, qb = (int)gridDim.y - 1 - (int)blockIdx.y;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int ctx = st->ctx, r0 = qb * AQ;
    const int rlast = min(r0 + AQ, M) - 1;            // last live row of this block
    const int nkeys = min(ctx + rlast + 1, max_seq);
    const int kvh = h / (H / Hkv);
    const unsigned short *Kc = kcache + (size_t)kvh * max_seq * HD, *Vc = vcache + (size_t)kvh * max_seq * HD;
    const float scale = rsqrtf((float)HD);

    for (int i = tid; i < AQ * HD / 4; i += 256) {
        const int row = i % AQ, c4 = i / AQ;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r0 + row < M) v = *(const float4 *)(q + (size_t)(r0 + row) * ld_q + h * HD + c4 * 4);
        Qt[(c4 * 4 + 0) * AQ + row] = v.x * scale;
        Qt[(c4 * 4 + 1) * AQ + row] = v.y * scale;
        Qt[(c4 * 4 + 2) * AQ + row] = v.z * scale;
        Qt[(c4 * 4 + 3) * AQ + row] = v.w * scale;
    }
    float m_run[4], l_run[4], o[4][NV][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m_run[i] = -INFINITY;
        l_run[i] = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[i][v][e] = 0.f;
    }

    for (int k0 = 0; k0 < nkeys; k0 += AK) {
        __syncthreads();   // the previous tile's reads of Ps and Vs are over (and Qt is written, first time round)
        // keys: thread -> (key, 8 head-dim elements); transposed to Kt.  values: natural layout.
        for (int i = tid; i < AK * HD / 8; i += 256) {
            const int key = i % AK, c8 = i / AK;
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            if (k0 + key < nkeys) raw = *(const uint4 *)(Kc + (size_t)(k0 + key) * HD + c8 * 8);
            const unsigned u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                pair16_to_f32(u[e], f16, Kt[(c8 * 8 + 2 * e) * AK + key], Kt[(c8 * 8 + 2 * e + 1) * AK + key]);
            }
        }
        for (int i = tid; i < AK * HD / 8; i += 256) {
            const int key = i / (HD / 8), c8 = i % (HD / 8);
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            if (k0 + key < nkeys) raw = *(const uint4 *)(Vc + (size_t)(k0 + key) * HD + c8 * 8);
            float4 *dst = (float4 *)(Vs + key * HD + c8 * 8);
            float4 lo4, hi4;
            pair16_to_f32(raw.x, f16, lo4.x, lo4.y);
            pair16_to_f32(raw.y, f16, lo4.z, lo4.w);
            pair16_to_f32(raw.z, f16, hi4.x, hi4.y);
            pair16_to_f32(raw.w, f16, hi4.z, hi4.w);
            dst[0] = lo4;
            dst[1] = hi4;
        }
        __syncthreads();
        float sc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) sc[i][j] = 0.f;
#pragma unroll 8
        for (int k = 0; k < HD; ++k) {
            const float4 qv = *(const float4 *)(Qt + k * AQ + 4 * ty);
            const float4 kv = *(const float4 *)(Kt + k * AK + 4 * tx);
            const float qa[4] = {qv.x, qv.y, qv.z, qv.w}, ka[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) sc[i][j] = fmaf(qa[i], ka[j], sc[i][j]);
        }
        __syncthreads();   // everyone is done with Kt: it becomes Ps
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int pos = ctx + r0 + 4 * ty + i;   // causal limit of this row
            const bool live = r0 + 4 * ty + i < M;
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (!(live && k0 + 4 * tx + j <= pos)) sc[i][j] = -INFINITY;
                mx = fmaxf(mx, sc[i][j]);
            }
#pragma unroll
            for (int w = 8; w > 0; w >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, w));
            const float m_new = fmaxf(m_run[i], mx);
            float p[4] = {0.f, 0.f, 0.f, 0.f}, ps = 0.f, resc = 1.f;
            if (m_new > -INFINITY) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    p[j] = (sc[i][j] > -INFINITY) ? expf(sc[i][j] - m_new) : 0.f;
                    ps += p[j];
                }
                resc = (m_run[i] > -INFINITY) ? expf(m_run[i] - m_new) : 0.f;
                m_run[i] = m_new;
            }
#pragma unroll
            for (int w = 8; w > 0; w >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, w);
            l_run[i] = fmaf(l_run[i], resc, ps);
#pragma unroll
            for (int v = 0; v < NV; ++v)
#pragma unroll
                for (int e = 0; e < 4; ++e) o[i][v][e] *= resc;
            *(float4 *)(Ps + (4 * ty + i) * APS + 4 * tx) = make_float4(p[0], p[1], p[2], p[3]);
        }
        __syncthreads();
#pragma unroll 2
        for (int kk = 0; kk < AK; kk += 4) {
            float pr[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 t4 = *(const float4 *)(Ps + (4 * ty + i) * APS + kk);
                pr[i][0] = t4.x; pr[i][1] = t4.y; pr[i][2] = t4.z; pr[i][3] = t4.w;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    const float4 vv = *(const float4 *)(Vs + (kk + j) * HD + v * 64 + tx * 4);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        o[i][v][0] = fmaf(pr[i][j], vv.x, o[i][v][0]);
                        o[i][v][1] = fmaf(pr[i][j], vv.y, o[i][v][1]);
                        o[i][v][2] = fmaf(pr[i][j], vv.z, o[i][v][2]);
                        o[i][v][3] = fmaf(pr[i][j], vv.w, o[i][v][3]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = r0 + 4 * ty + i;
        if (row >= M || !(l_run[i] > 0.f)) continue;
        const float inv = 1.f / l_run[i];
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const size_t col = (size_t)h * HD + v * 64 + tx * 4;
            unsigned hi[4], lo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                unsigned short bh, bl;
                split_b16(o[i][v][e] * inv, f16, bh, bl);
                hi[e] = bh;
                lo[e] = bl;
            }
            *(uint2 *)(out_b + (size_t)row * d + col) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
            *(uint2 *)(out_b + (size_t)(lo_row0 + row) * d + col) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
        }
    }
}

// grid (M, ceil(F / 256)): the gate/up product has rows interleaved (2 i = gate_i, 2 i + 1 = up_i).
__global__ void __launch_bounds__(256) k_wide_silu(const float *P, int splits, int M, int F, __nv_bfloat16 *A, int lo_row0, int f16) {
    const int t = blockIdx.x, i = blockIdx.y * 256 + threadIdx.x;
    if (i >= F) return;
    float g = 0.f, u = 0.f;
    for (int s = 0; s < splits; ++s) {
        const float2 p = __ldcg((const float2 *)(P + ((size_t)s * M + t) * 2 * F) + i);
        g += p.x;
        u += p.y;
    }
    const float h = g / (1.f + expf(-g)) * u;
    store_split(A + (size_t)t * F + i, A + (size_t)(lo_row0 + t) * F + i, h, f16);
}

}  // namespace

// Parts to cut the K range into: the fewest that fill at least 90 % of the last wave of CTAs (else the best found),
// with at least 8 K blocks per part and the partial products inside the workspace.
int cl_wide_splits(int M, int rows, int KB, int n_sm, size_t ws_floats) {
    const long long tiles = (long long)((M + WM - 1) / WM) * ((rows + WN - 1) / WN);
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= 16; ++s) {
        if (s > 1 && (KB / s < 8 || (size_t)s * M * rows > ws_floats)) break;
        const long long n = tiles * s, waves = (n + n_sm - 1) / n_sm;
        const double eff = (double)n / (double)(waves * n_sm);
        if (eff > best_eff + 1e-9) {
            best_eff = eff;
            best = s;
        }
        if (eff >= 0.9) break;
    }
    return best;
}

cudaError_t cl_launch_wide(const ClTensorMap &mapA, const ClTensorMap &mapB, const ClWideArgs &a, cudaStream_t s) {
    const size_t smem = (size_t)WSTAGES * WSTAGE_BYTES + sizeof(WSmem) + 1024;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_wide, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    if (a.rows % 4 || a.M < 1 || a.M > CL_WIDE_MAX_M) return cudaErrorInvalidValue;
    k_wide<<<a.MT * a.NT * a.splits, WTHREADS, smem, s>>>(*(const CUtensorMap *)mapA.bytes, *(const CUtensorMap *)mapB.bytes, a);
    return cudaGetLastError();
}

cudaError_t cl_launch_wide_norm(const ClWideNormArgs &a, cudaStream_t s) {
    if (a.d % 4) return cudaErrorInvalidValue;
    k_wide_norm<<<a.M, 256, 0, s>>>(a);
    return cudaGetLastError();
}

cudaError_t cl_launch_wide_rope_append(float *P, int splits, int M, int H, int Hkv, int hd, int d, const float2 *rope_cs,
                                       void *kcache, void *vcache, int max_seq, const ClDevState *st, int f16, cudaStream_t s) {
    k_wide_rope_append<<<dim3(M, H), hd / 2, 0, s>>>(P, splits, M, hd, d, Hkv, rope_cs, (unsigned short *)kcache,
                                                     (unsigned short *)vcache, max_seq, st, f16);
    return cudaGetLastError();
}

cudaError_t cl_launch_wide_silu(const float *P, int splits, int M, int F, __nv_bfloat16 *A, int lo_row0, int f16, cudaStream_t s) {
    k_wide_silu<<<dim3(M, (F + 255) / 256), 256, 0, s>>>(P, splits, M, F, A, lo_row0, f16);
    return cudaGetLastError();
}

cudaError_t cl_launch_attn_wide(const float *q, int ld_q, const void *kcache, const void *vcache, __nv_bfloat16 *out_b,
                                int lo_row0, int M, int d, int H, int Hkv, int hd, int max_seq, const ClDevState *st,
                                int f16, cudaStream_t s) {
    const dim3 grid(H, (M + AQ - 1) / AQ);
    const int kp = (hd * AK > AQ * APS) ? hd * AK : AQ * APS;
    const size_t smem = (size_t)(hd * AQ + kp + AK * hd) * sizeof(float);
    if (hd == 128) {
        static bool set128 = false;
        if (!set128) {
            cudaError_t e = cudaFuncSetAttribute(k_attn_wide<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            set128 = true;
        }
        k_attn_wide<128><<<grid, 256, smem, s>>>(q, ld_q, (const unsigned short *)kcache, (const unsigned short *)vcache, out_b,
                                                 lo_row0, M, d, H, Hkv, max_seq, st, f16);
    } else if (hd == 64) {
        static bool set64 = false;
        if (!set64) {
            cudaError_t e = cudaFuncSetAttribute(k_attn_wide<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            set64 = true;
        }
        k_attn_wide<64><<<grid, 256, smem, s>>>(q, ld_q, (const unsigned short *)kcache, (const unsigned short *)vcache, out_b,
                                                lo_row0, M, d, H, Hkv, max_seq, st, f16);
    } else {
        return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

bool cl_make_tensor_map(ClTensorMap *m, const void *base, int rows, int cols, int box_rows, int f16) {
    static_assert(sizeof(ClTensorMap) >= sizeof(CUtensorMap), "tensor map storage");
    return make_map((CUtensorMap *)m->bytes, base, rows, cols, box_rows, f16);
}
