// Building blocks shared by the tensor-core kernels: mbarriers with bounded waits, TMA tile loads, tcgen05
// descriptors / multiply-add / commit / tensor-memory loads, and the host-side tensor-map encoder.
#pragma once
#include <cuda.h>

#include "cl_internal.h"

namespace {

constexpr int TC_BK = 64;   // K extent of one shared-memory tile: 64 16-bit elements = one 128-byte swizzle row
constexpr unsigned long long WAIT_NS = 2000000000ull;

__device__ __forceinline__ unsigned s_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long gtime_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void bar_init(unsigned long long *b, unsigned n) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s_u32(b)), "r"(n));
}
__device__ __forceinline__ void bar_arrive(unsigned long long *b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s_u32(b)) : "memory");
}
__device__ __forceinline__ void bar_expect(unsigned long long *b, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try(unsigned long long *b, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(s_u32(b)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait; false (and the abort flags raised) if it gave up.
__device__ __forceinline__ bool bar_wait(unsigned long long *b, unsigned parity, int *abort_flag, int *err) {
    if (bar_try(b, parity)) return true;
    const unsigned long long t0 = gtime_ns();
    for (unsigned i = 1;; ++i) {
        if (bar_try(b, parity)) return true;
        if ((i & 63u) == 0u) {
            if (*(volatile int *)abort_flag) return false;
            if (gtime_ns() - t0 > WAIT_NS) {
                *(volatile int *)abort_flag = 1;
                atomicOr(err, 4);
                return false;
            }
        }
    }
}

// Non-blocking look at an mbarrier phase.  (mbarrier.try_wait may suspend the thread for a while before it answers
// "not yet"; a loop that serves two queues must not sit in it.)
__device__ __forceinline__ bool bar_test(unsigned long long *b, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(s_u32(b)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bulk asynchronous copy global -> shared (16-byte aligned addresses, size a multiple of 16 bytes; completion counted
// in bytes on an mbarrier).  The _stream form marks the lines evict-first in L2: streamed weights are used once per pass.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, unsigned bytes, unsigned long long *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(s_u32(dst)),
                 "l"(src), "r"(bytes), "r"(s_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void bulk_g2s_stream(void *dst, const void *src, unsigned bytes, unsigned long long *bar,
                                                unsigned long long policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            s_u32(dst)),
        "l"(src), "r"(bytes), "r"(s_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ unsigned long long policy_evict_first() {
    unsigned long long p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// Ticket of a "last arrival finishes the job" protocol, taken by ONE thread after a barrier of the threads that wrote
// the data and before the barrier after which they read other CTAs' data: the release half orders the CTA's earlier
// writes (made visible to this thread by the barrier) before the increment, the acquire half orders the later reads
// after it.  Replaces a __threadfence() by every thread on each side of a plain atomicAdd.
__device__ __forceinline__ unsigned ticket_acq_rel(unsigned *p) {
    unsigned old;
    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(p) : "memory");
    return old;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, unsigned long long *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
            s_u32(dst)),
        "l"(map), "r"(s_u32(bar)), "r"(c0), "r"(c1)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile written by TMA with the 128-byte swizzle: rows of 128
// bytes, groups of 8 rows 1024 bytes apart (stride byte offset), descriptor version 1, layout type 2 (128B swizzle).
__device__ __forceinline__ unsigned long long umma_desc(unsigned smem_addr) {
    unsigned long long d = 0;
    d |= (unsigned long long)((smem_addr & 0x3ffffu) >> 4);   // start address
    d |= (unsigned long long)1 << 16;                          // leading byte offset (unused with swizzle)
    d |= (unsigned long long)(1024 >> 4) << 32;                // stride byte offset
    d |= (unsigned long long)1 << 46;                          // version
    d |= (unsigned long long)2 << 61;                          // 128-byte swizzle
    return d;
}
// Instruction descriptor of kind::f16: fp32 accumulator, A and B of the same 16-bit type (format 1 = bf16, 0 = fp16),
// both K-major, N and M of the tile.
__device__ __forceinline__ unsigned umma_idesc(int m, int n, int f16 = 0) {
    const unsigned fmt = f16 ? 0u : 1u;
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(m >> 4) << 24);
}

// The 16-bit type of a model (storage and tensor-core operands) chosen at run time: f16 != 0 is IEEE binary16,
// else bfloat16.  Values travel as raw 16-bit patterns.
__device__ __forceinline__ unsigned short f32_to_b16(float v, int f16) {
    return f16 ? __half_as_ushort(__float2half_rn(v)) : __bfloat16_as_ushort(__float2bfloat16_rn(v));
}
__device__ __forceinline__ float b16_to_f32(unsigned short b, int f16) {
    return f16 ? __half2float(__ushort_as_half(b)) : __uint_as_float((unsigned)b << 16);
}
__device__ __forceinline__ void pair16_to_f32(unsigned u, int f16, float &a, float &b) {
    if (f16) ClPair16<__half>::get(u, a, b);
    else ClPair16<__nv_bfloat16>::get(u, a, b);
}
// v -> (hi, lo) with hi + lo = v to about 16 (bf16) or 22 (fp16) mantissa bits
__device__ __forceinline__ void split_b16(float v, int f16, unsigned short &hi, unsigned short &lo) {
    hi = f32_to_b16(v, f16);
    lo = f32_to_b16(v - b16_to_f32(hi, f16), f16);
}
__device__ __forceinline__ void store_split(__nv_bfloat16 *hi_p, __nv_bfloat16 *lo_p, float v, int f16) {
    unsigned short hi, lo;
    split_b16(v, f16, hi, lo);
    *reinterpret_cast<unsigned short *>(hi_p) = hi;
    *reinterpret_cast<unsigned short *>(lo_p) = lo;
}
__device__ __forceinline__ void umma_bf16(unsigned tmem_d, unsigned long long adesc, unsigned long long bdesc, unsigned idesc,
                                          unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, float (&v)[32]) {
    unsigned r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// 2-D row-major [rows, cols] tensor of 16-bit elements (bf16, or fp16 with f16 != 0), box = 64 columns x box_rows
// rows, 128-byte swizzle, zero fill outside.
bool make_map(CUtensorMap *m, const void *base, int rows, int cols, int box_rows, int f16 = 0) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void *)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


}  // namespace
