// Persistent single-token decoder step ("token-step kernel"): the skip-masked draft step and the
// vanilla full-model step at batch 1, one cooperative launch for up to CL_MAX_K (draft) or many
// (vanilla) consecutive tokens.
//
// One CTA per SM.  The last warp (one elected thread) is the weight producer: it walks the static schedule
// (steps x kept layers x {QKV, O, gate/up, down} + LM head), and for this CTA's contiguous block of
// rows of each matrix issues bulk asynchronous copies (cp.async.bulk, completion on an mbarrier) into
// a ring of six 32 KB shared-memory slots (whole rows per slot).  It never waits for activations, so the HBM stream runs ahead
// of the grid barriers that separate the phases.  The other 16 warps are consumers: each thread keeps its
// fixed columns of the activation vector in registers for a whole phase, every warp reads its 512-byte
// stripes of each row from the ring (conflict-free 16-byte reads), partial dot products are reduced
// with warp shuffles and a small shared-memory table, and the phase epilogue (store / residual add /
// SiLU*up / LM head with online softmax-entropy-argmax) runs with one thread per row.
// Skipped layers are simply absent from the schedule: they stream nothing and touch no KV entry.
//
// Every wait (mbarrier or grid barrier) is bounded in time; on expiry an error flag is set, every later
// wait falls through, the kernel runs to its end with meaningless data and the host reports CL_ETIMEOUT.
#include "tc_common.cuh"

namespace {

constexpr int NCW = 16;                // consumer warps
constexpr int NCT = NCW * 32;          // consumer threads
constexpr int SLOT_BYTES = 32768;      // ring slot: as many whole weight rows as fit (at least one)
constexpr int NSLOT = 6;               // 192 KB in flight per SM
constexpr int MAXIT = 4;               // 16-byte chunks per thread per row: rows up to 32 KB (C <= 16384 bf16)
constexpr int RB = 256;                // rows per epilogue block
// (every single wait is bounded by ClStepArgs::wait_ns, 2 s unless a diagnostic lowered it)

struct Smem {
    unsigned long long full[NSLOT];
    unsigned long long empty[NSLOT];
    float partial[RB * NCW];
    float red[NCW];
    ClHeadPartial hp[NCT];
    int abort;
    int halt;                     // set by the consumers when drafting stops early: the producer issues no more copies
    unsigned long long wait_ns;   // bound on any single wait (copied from the launch arguments)
};

// Bounded wait.  Returns false (and raises the abort flags) if the phase did not complete in time.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned parity, Smem *sm, ClDevState *st) {
    if (bar_try(bar, parity)) return true;
    if (*(volatile int *)&sm->abort) return false;
    const unsigned long long t0 = gtime_ns();
    for (unsigned i = 1;; ++i) {
        if (bar_try(bar, parity)) return true;
        if ((i & 63u) == 0u) {
            if (*(volatile int *)&sm->abort) return false;
            if (gtime_ns() - t0 > sm->wait_ns) {
                *(volatile int *)&sm->abort = 1;
                atomicOr(&st->err, 1);
                return false;
            }
        }
    }
}


// Ask L2 to fetch a 16-byte-aligned range (multiple of 16 bytes); nothing waits for it.
__device__ __forceinline__ void l2_prefetch_bulk(const void *src, unsigned bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(NCT) : "memory"); }

__device__ __forceinline__ float ldcg_f(const float *p) { return __ldcg(p); }
__device__ __forceinline__ float4 ldcg_f4(const float *p) { return __ldcg((const float4 *)p); }

// Grid barrier on one arrival counter in global memory that only ever grows during a launch (the host zeroes
// it before every launch): barrier number i is passed once the counter reaches i * gridDim.x.  One release
// increment and an acquire poll per CTA; `target` lives in thread 0's registers.  Called by every consumer
// thread of every CTA; bounded in time.
// `bar_arrivals` = arrivals that complete one barrier: the grid size (a diagnostic may ask for more, so that the
// wait provably runs out).
__device__ __forceinline__ void grid_barrier(unsigned *bar, unsigned &target, unsigned bar_arrivals, Smem *sm, ClDevState *st) {
    consumer_sync();
    if (threadIdx.x == 0 && !*(volatile int *)&sm->abort) {
        target += bar_arrivals;
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(bar) : "memory");
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(bar) : "memory");
        if ((int)(v - target) < 0) {
            const unsigned long long t0 = gtime_ns();
            unsigned i = 0;
            do {
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(bar) : "memory");
                if ((++i & 255u) == 0u) {
                    if (*(volatile int *)&st->err || gtime_ns() - t0 > sm->wait_ns) {
                        *(volatile int *)&sm->abort = 1;
                        atomicOr(&st->err, 2);
                        break;
                    }
                }
            } while ((int)(v - target) < 0);
        }
    }
    consumer_sync();
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Fixed-order reduction of one ClHeadPartial per consumer thread; result valid in every thread.
__device__ ClHeadPartial hp_block_reduce(ClHeadPartial v, Smem *sm) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const ClHeadPartial other = cl_hp_shfl_xor(v, o);
        // combine in a lane-independent order so every lane ends with identical bits
        v = ((threadIdx.x & o) == 0) ? cl_hp_merge(v, other) : cl_hp_merge(other, v);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    consumer_sync();
    if (lane == 0) sm->hp[warp] = v;
    consumer_sync();
    ClHeadPartial r = sm->hp[0];
#pragma unroll
    for (int w = 1; w < NCW; ++w) r = cl_hp_merge(r, sm->hp[w]);
    return r;
}

template <typename WT>
struct Chunk;   // one 16-byte chunk of weights against the matching activation registers
template <>
struct Chunk<__nv_bfloat16> {
    static constexpr int EPC = 8;
    static __device__ __forceinline__ float dot(const uint4 &w, const float (&x)[8], float acc) {
        acc = fmaf(__uint_as_float(w.x << 16), x[0], acc);
        acc = fmaf(__uint_as_float(w.x & 0xffff0000u), x[1], acc);
        acc = fmaf(__uint_as_float(w.y << 16), x[2], acc);
        acc = fmaf(__uint_as_float(w.y & 0xffff0000u), x[3], acc);
        acc = fmaf(__uint_as_float(w.z << 16), x[4], acc);
        acc = fmaf(__uint_as_float(w.z & 0xffff0000u), x[5], acc);
        acc = fmaf(__uint_as_float(w.w << 16), x[6], acc);
        acc = fmaf(__uint_as_float(w.w & 0xffff0000u), x[7], acc);
        return acc;
    }
};
template <>
struct Chunk<__half> {
    static constexpr int EPC = 8;
    static __device__ __forceinline__ float dot(const uint4 &w, const float (&x)[8], float acc) {
        const unsigned u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float lo, hi;
            ClPair16<__half>::get(u[e], lo, hi);
            acc = fmaf(lo, x[2 * e], acc);
            acc = fmaf(hi, x[2 * e + 1], acc);
        }
        return acc;
    }
};
template <>
struct Chunk<float> {
    static constexpr int EPC = 4;
    static __device__ __forceinline__ float dot(const uint4 &w, const float (&x)[4], float acc) {
        acc = fmaf(__uint_as_float(w.x), x[0], acc);
        acc = fmaf(__uint_as_float(w.y), x[1], acc);
        acc = fmaf(__uint_as_float(w.z), x[2], acc);
        acc = fmaf(__uint_as_float(w.w), x[3], acc);
        return acc;
    }
};

template <typename ST>
__device__ __forceinline__ float st_to_f32(ST v);
template <>
__device__ __forceinline__ float st_to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float st_to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <>
__device__ __forceinline__ float st_to_f32<__half>(__half v) { return __half2float(v); }
template <typename ST>
__device__ __forceinline__ ST st_from_f32(float v);
template <>
__device__ __forceinline__ __half st_from_f32<__half>(float v) { return __float2half_rn(v); }
template <>
__device__ __forceinline__ float st_from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 st_from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// VPL consecutive stored elements -> fp32, read through L2.
template <typename ST, int VPL>
__device__ __forceinline__ void load_vals(const ST *p, float (&o)[VPL]) {
    constexpr int BYTES = VPL * (int)sizeof(ST);
    if (BYTES == 4) {
        const unsigned u = __ldcg((const unsigned *)p);
        if (sizeof(ST) == 2) {
            ClPair16<ST>::get(u, o[0], o[VPL - 1]);
        } else {
            o[0] = __uint_as_float(u);
        }
    } else if (BYTES == 8) {
        const uint2 u = __ldcg((const uint2 *)p);
        if (sizeof(ST) == 2) {
            ClPair16<ST>::get(u.x, o[0], o[1 % VPL]);
            ClPair16<ST>::get(u.y, o[2 % VPL], o[3 % VPL]);
        } else {
            o[0] = __uint_as_float(u.x);
            o[1 % VPL] = __uint_as_float(u.y);
        }
    } else {
        const uint4 u = __ldcg((const uint4 *)p);
        o[0] = __uint_as_float(u.x);
        o[1 % VPL] = __uint_as_float(u.y);
        o[2 % VPL] = __uint_as_float(u.z);
        o[3 % VPL] = __uint_as_float(u.w);
    }
}

struct Ring {
    unsigned slot, par;   // position in the ring and the parity of the phase to wait for
    __device__ __forceinline__ void advance() {
        if (++slot == NSLOT) {
            slot = 0;
            par ^= 1u;
        }
    }
};

// This CTA's share of `units` row units (a unit is `unit` consecutive rows): an equal share, or -- with a table of
// cumulative shares cum_w[0 .. grid] (0 ... 1), measured once per context -- a share in proportion to the rate at which
// this CTA's SM streams from HBM (SMs differ by several percent; equal rows would make every phase wait for the
// slowest).  Which CTA computes a row never changes the row's arithmetic.
__device__ __forceinline__ void my_rows(int rows, int unit, const float *cum_w, int &r0, int &r1) {
    const long long units = rows / unit;
    if (cum_w) {
        r0 = (int)((double)units * (double)cum_w[blockIdx.x] + 0.5) * unit;
        r1 = (int)((double)units * (double)cum_w[blockIdx.x + 1] + 0.5) * unit;
    } else {
        r0 = (int)(units * blockIdx.x / gridDim.x) * unit;
        r1 = (int)(units * (blockIdx.x + 1) / gridDim.x) * unit;
    }
}

// Rows per ring slot for a matrix with `rowbytes` bytes per row.  Phases whose epilogue pairs rows (unit 2) keep
// pairs inside a slot.  Producer and consumers derive the same slot <-> rows mapping from this.
__device__ __forceinline__ int rows_per_slot(size_t rowbytes, int unit) {
    int rps = (int)((size_t)SLOT_BYTES / rowbytes);
    if (rps < 1) rps = 1;
    if (unit == 2 && (rps & 1) && rps > 1) rps -= 1;
    return rps;
}

// ---- producer -------------------------------------------------------------------------------------
// Walks the static schedule (steps x kept layers x {QKV, O, gate/up, down} + LM head) slot by slot: each call of
// next() yields the next rps rows of this CTA's block of the current matrix, which are contiguous in memory.
template <typename WT>
struct SchedIter {
    const ClStepArgs &a;
    int step, ki, m;        // m: 0..3 = the layer's matrices; ki == n_kept: the LM head (m = 0)
    int r, r1, rps;
    size_t rowbytes;
    const char *W;
    ClLayerDev L;
    int lk;                 // kept-list position L was loaded for (-1: none)
    bool done;
    __device__ SchedIter(const ClStepArgs &args) : a(args), step(0), ki(0), m(0), lk(-1), done(false) {
        if (a.n_steps <= 0) done = true;
        else open();
    }
    __device__ void open() {   // set up (step, ki, m); skips matrices of which this CTA owns no row
        for (;;) {
            int rows, cols, unit = 1;
            if (ki < a.n_kept) {
                const int ent = a.kept[ki], fl = ent >> 16;   // layer | flags << 16: bit 0 no attention half, bit 1 no FFN half
                if ((m < 2 && (fl & 1)) || (m >= 2 && (fl & 2))) {
                    if (!advance()) return;
                    continue;
                }
                if (lk != ki) { L = a.layers[ent & 0xffff]; lk = ki; }
                if (m == 0) { W = L.wqkv; rows = a.d + 2 * a.Hkv * (a.d / a.H); cols = a.d; }
                else if (m == 1) { W = L.wo; rows = a.d; cols = a.d; }
                else if (m == 2) { W = L.wgu; rows = 2 * a.F; cols = a.d; unit = 2; }
                else { W = L.wd; rows = a.d; cols = a.F; }
            } else {
                W = (const char *)a.lm_head; rows = a.V; cols = a.d;
            }
            my_rows(rows, unit, a.cum_w, r, r1);
            rowbytes = (size_t)cols * sizeof(WT);
            rps = rows_per_slot(rowbytes, unit);
            if (r < r1) return;
            if (!advance()) return;
        }
    }
    __device__ bool advance() {   // to the next matrix of the schedule; false at the end
        if (ki < a.n_kept && m < 3) { ++m; return true; }
        m = 0;
        if (ki < a.n_kept) { ++ki; return true; }
        ki = 0;
        if (++step < a.n_steps) return true;
        done = true;
        return false;
    }
    __device__ bool next(const char *&src, unsigned &bytes) {
        if (done) return false;
        const int n = min(rps, r1 - r);
        src = W + (size_t)r * rowbytes;
        bytes = (unsigned)((size_t)n * rowbytes);
        r += n;
        if (r >= r1 && advance()) open();
        return true;
    }
};

// The producer thread.  Two cursors over the same schedule: the fill cursor feeds the shared-memory ring as slots
// come free; the prefetch cursor only asks L2 to fetch, and only moves while the ring is full (the consumers sit in a
// grid barrier or the attention phase), up to l2_ahead bytes in front of the fill cursor, so that HBM keeps streaming
// into L2 during those gaps and the ring is refilled from L2 afterwards.
template <typename WT>
__device__ void producer_loop(const ClStepArgs &a, unsigned char *ring, Smem *sm, ClDevState *st) {
    Ring rg{0u, 0u};
    unsigned last_par[NSLOT];
    for (int i = 0; i < NSLOT; ++i) last_par[i] = 2u;
    const unsigned long long policy = policy_evict_first();
    SchedIter<WT> fill(a), pf(a);
    unsigned long long filled = 0, fetched = 0;
    const unsigned long long ahead = (unsigned long long)a.l2_ahead;
    const char *src;
    unsigned bytes;
    while (fill.next(src, bytes)) {
        if (ahead) {
            const char *psrc;
            unsigned pbytes;
            while (fetched < filled + bytes && pf.next(psrc, pbytes)) fetched += pbytes;   // never behind the fill cursor
            if (!bar_try(&sm->empty[rg.slot], rg.par ^ 1u)) {
                // ring full: the consumers are held up, HBM would go idle; spend the time fetching into L2
                while (fetched < filled + bytes + ahead && !bar_try(&sm->empty[rg.slot], rg.par ^ 1u) && pf.next(psrc, pbytes)) {
                    l2_prefetch_bulk(psrc, pbytes);
                    fetched += pbytes;
                }
            }
        }
        if (!bar_try(&sm->empty[rg.slot], rg.par ^ 1u)) {
            // (a slot stays taken for good once the consumers have stopped early: look at their flag while waiting)
            const unsigned long long t0 = gtime_ns();
            for (unsigned i = 1; !bar_try(&sm->empty[rg.slot], rg.par ^ 1u); ++i) {
                if ((i & 31u) == 0u) {
                    if (*(volatile int *)&sm->halt || *(volatile int *)&sm->abort) break;
                    if (gtime_ns() - t0 > sm->wait_ns) {
                        *(volatile int *)&sm->abort = 1;
                        atomicOr(&st->err, 1);
                        break;
                    }
                }
            }
        }
        if (*(volatile int *)&sm->halt) break;
        if (!*(volatile int *)&sm->abort) {
            bar_expect(&sm->full[rg.slot], bytes);
            bulk_g2s_stream(ring + (size_t)rg.slot * SLOT_BYTES, src, bytes, &sm->full[rg.slot], policy);
            last_par[rg.slot] = rg.par;
        }
        rg.advance();
        filled += bytes;
    }
    // Drain: every copy this thread issued must have landed before the CTA may exit.  In the normal path the
    // consumers have already waited for all of them; after an abort this is the bounded wait for copies in flight.
    for (int i = 0; i < NSLOT; ++i) {
        if (last_par[i] < 2u) {
            const unsigned long long t0 = gtime_ns();
            while (!bar_try(&sm->full[i], last_par[i]))
                if (gtime_ns() - t0 > sm->wait_ns) break;
        }
    }
}

// ---- consumer: one matrix phase ------------------------------------------------------------------------
// Sums R per-thread values across the warp at once ("transposing" butterfly): log2(R) exchange steps halve the
// number of values each lane carries, the remaining steps are plain butterflies.  On return acc[0] holds the
// warp total of row (lane >> (5 - log2 R)) & (R - 1) in every lane; the combine order is fixed.
template <int R>
__device__ __forceinline__ void warp_reduce_rows(float (&acc)[R], int lane) {
    int off = 16;
#pragma unroll
    for (int half = R / 2; half >= 1; half >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            const float send = upper ? acc[i] : acc[i + half];
            const float keep = upper ? acc[i + half] : acc[i];
            acc[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
        off >>= 1;
    }
#pragma unroll
    for (; off >= 1; off >>= 1) acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], off);
}

template <int R>
struct Log2;
template <> struct Log2<1> { static constexpr int v = 0; };
template <> struct Log2<2> { static constexpr int v = 1; };
template <> struct Log2<4> { static constexpr int v = 2; };
template <> struct Log2<8> { static constexpr int v = 3; };

// xr: this thread's activation registers, xr[it][e] = x[(it * NCT + tid) * EPC + e]; NIT = chunks per thread per
// row (rounded up to a supported count).  One wait per slot; inside a slot rows are taken R at a time in
// straight-line code: all of a group's 16-byte reads are issued before the first multiply-add, every row has
// its own accumulation chain, and the R row sums are reduced across the warp together.
// Calls epi(first_row_of_block, rows_in_block) once the partial table of a block of up to RB rows is ready.
__device__ __forceinline__ uint4 lds128(unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

template <typename WT, int NIT, int R, typename Epi>
__device__ __forceinline__ void consume_rows(int r0, int r1, int nchunks, int rps, const float (&xr)[MAXIT][Chunk<WT>::EPC],
                                             Ring &rg, const unsigned char *ring, Smem *sm, ClDevState *st, Epi epi) {
    constexpr int SH = 5 - Log2<R>::v;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned rowbytes = (unsigned)nchunks * 16u;
    const unsigned ring_addr = s_u32(ring);
    // Byte offset of this thread's it-th chunk inside a row.  Chunks past the end of the row are redirected to the
    // row's last chunk: its (finite) weights meet activation registers that hold zeros.
    unsigned coff[NIT];
#pragma unroll
    for (int it = 0; it < NIT; ++it) coff[it] = (unsigned)min(it * NCT + tid, nchunks - 1) * 16u;
    const int blockrows = max(1, RB / rps) * rps;
    for (int rb0 = r0; rb0 < r1; rb0 += blockrows) {
        const int nrb = min(blockrows, r1 - rb0);
        for (int sr = 0; sr < nrb; sr += rps) {
            const int ns = min(rps, nrb - sr);   // rows in this slot
            mbar_wait(&sm->full[rg.slot], rg.par, sm, st);
            const unsigned base = ring_addr + rg.slot * (unsigned)SLOT_BYTES;
            for (int g = 0; g < ns; g += R) {
                uint4 w[R][NIT];
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    // rows past the end of the slot re-read its last row (their sums are dropped below)
                    const unsigned rowp = base + (unsigned)min(g + i, ns - 1) * rowbytes;
#pragma unroll
                    for (int it = 0; it < NIT; ++it) w[i][it] = lds128(rowp + coff[it]);
                }
                float acc[R];
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    float a0 = 0.f, a1 = 0.f;   // two chains per row: even and odd chunks
#pragma unroll
                    for (int it = 0; it < NIT; ++it) {
                        if (it & 1) a1 = Chunk<WT>::dot(w[i][it], xr[it], a1);
                        else a0 = Chunk<WT>::dot(w[i][it], xr[it], a0);
                    }
                    acc[i] = a0 + a1;
                }
                if (g + R >= ns) {   // every read of this slot has returned: hand it back to the producer
                    __syncwarp();
                    if (lane == 0) bar_arrive(&sm->empty[rg.slot]);
                }
                warp_reduce_rows<R>(acc, lane);
                const int row = sr + g + ((lane >> SH) & (R - 1));
                if ((lane & ((1 << SH) - 1)) == 0 && row < sr + ns) sm->partial[row * NCW + warp] = acc[0];
            }
            rg.advance();
        }
        consumer_sync();
        epi(rb0, nrb);
        consumer_sync();
    }
}

template <typename WT, typename Epi>
__device__ __forceinline__ void consume_matrix(int rows, int cols, int unit, const float (&xr)[MAXIT][Chunk<WT>::EPC],
                                               Ring &rg, const unsigned char *ring, Smem *sm, ClDevState *st, Epi epi,
                                               const float *cum_w, unsigned long long *busy) {
    constexpr int EPC = Chunk<WT>::EPC;
    int r0, r1;
    my_rows(rows, unit, cum_w, r0, r1);
    const unsigned long long t_start = busy ? gtime_ns() : 0ull;   // calibration launches only
    const int nchunks = cols / EPC;
    const int rps = rows_per_slot((size_t)nchunks * 16, unit);
    const int nit = (nchunks + NCT - 1) / NCT;   // uniform over the grid
    if (nit <= 1) consume_rows<WT, 1, 4>(r0, r1, nchunks, rps, xr, rg, ring, sm, st, epi);
    else if (nit <= 2) consume_rows<WT, 2, 2>(r0, r1, nchunks, rps, xr, rg, ring, sm, st, epi);
    else consume_rows<WT, 4, 1>(r0, r1, nchunks, rps, xr, rg, ring, sm, st, epi);
    if (busy) *busy += gtime_ns() - t_start;
}

__device__ __forceinline__ float row_sum(const Smem *sm, int r) {
    const float *p = sm->partial + r * NCW;
    float s = p[0];
#pragma unroll
    for (int w = 1; w < NCW; ++w) s += p[w];
    return s;
}

// Load this thread's columns of a global fp32 vector into registers (L2 reads: written by other CTAs).
template <int EPC>
__device__ __forceinline__ void load_x(const float *x, int cols, float (&xr)[MAXIT][EPC]) {
    const int nchunks = cols / EPC;
#pragma unroll
    for (int it = 0; it < MAXIT; ++it) {
        const int ch = it * NCT + threadIdx.x;
        if (ch < nchunks) {
#pragma unroll
            for (int q = 0; q < EPC / 4; ++q) {
                const float4 v = ldcg_f4(x + (size_t)ch * EPC + 4 * q);
                xr[it][4 * q] = v.x; xr[it][4 * q + 1] = v.y; xr[it][4 * q + 2] = v.z; xr[it][4 * q + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < EPC; ++e) xr[it][e] = 0.f;
        }
    }
}

// RMSNorm in registers: xr <- x * rsqrt(mean(x^2) + eps) * g.  The gains are requested together with x so that the
// phase start costs one memory round trip, not two.
template <int EPC, int NI>
__device__ __forceinline__ void load_x_rmsnorm_n(const float *x, const float *g, int cols, float eps, float (&xr)[MAXIT][EPC],
                                                 Smem *sm) {
    const int nchunks = cols / EPC;
    float gr[NI][EPC];
#pragma unroll
    for (int it = 0; it < NI; ++it) {
        const int ch = it * NCT + threadIdx.x;
        if (ch < nchunks) {
#pragma unroll
            for (int q = 0; q < EPC / 4; ++q) {
                const float4 gv = __ldg((const float4 *)(g + (size_t)ch * EPC + 4 * q));
                const float4 xv = ldcg_f4(x + (size_t)ch * EPC + 4 * q);
                gr[it][4 * q] = gv.x; gr[it][4 * q + 1] = gv.y; gr[it][4 * q + 2] = gv.z; gr[it][4 * q + 3] = gv.w;
                xr[it][4 * q] = xv.x; xr[it][4 * q + 1] = xv.y; xr[it][4 * q + 2] = xv.z; xr[it][4 * q + 3] = xv.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < EPC; ++e) gr[it][e] = xr[it][e] = 0.f;
        }
    }
#pragma unroll
    for (int it = NI; it < MAXIT; ++it)
#pragma unroll
        for (int e = 0; e < EPC; ++e) xr[it][e] = 0.f;
    float ss = 0.f;
#pragma unroll
    for (int it = 0; it < NI; ++it)
#pragma unroll
        for (int e = 0; e < EPC; ++e) ss = fmaf(xr[it][e], xr[it][e], ss);
    ss = warp_sum(ss);
    consumer_sync();
    if ((threadIdx.x & 31) == 0) sm->red[threadIdx.x >> 5] = ss;
    consumer_sync();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < NCW; ++w) tot += sm->red[w];
    const float sc = 1.0f / sqrtf(tot / (float)cols + eps);
#pragma unroll
    for (int it = 0; it < NI; ++it)
#pragma unroll
        for (int e = 0; e < EPC; ++e) xr[it][e] *= sc * gr[it][e];
}

// The vector's length decides how many chunks a thread holds (one for d_model = 4096 in 16-bit storage): the short
// cases keep fewer gains in registers.
template <int EPC>
__device__ __forceinline__ void load_x_rmsnorm(const float *x, const float *g, int cols, float eps, float (&xr)[MAXIT][EPC],
                                               Smem *sm) {
    const int nchunks = cols / EPC;
    if (nchunks <= NCT) load_x_rmsnorm_n<EPC, 1>(x, g, cols, eps, xr, sm);
    else if (nchunks <= 2 * NCT) load_x_rmsnorm_n<EPC, 2>(x, g, cols, eps, xr, sm);
    else load_x_rmsnorm_n<EPC, MAXIT>(x, g, cols, eps, xr, sm);
}

// ---- attention phase ---------------------------------------------------------------------------------
// Work split: (head h, part s) -> one CTA; the cached keys [0, pos) of a head are cut into S contiguous parts and a
// part into NCW contiguous warp ranges.  A warp walks its range 32 keys at a time (one score per lane) with an
// online softmax; the new position's key and value (this step's QKV output, rotated, rounded to the storage type
// and appended to the cache) are one more partial, taken by the last warp of the last part.  The CTA merges its
// warps' partials in shared memory and writes one (max, sum, unnormalised output) record per (h, s); the S records
// of a head are merged by whoever reads the attention output (load_att_merged), so no CTA waits on another here.
constexpr int ATT_MAX_PARTS = 8;

template <typename ST, int HD>
struct AttnGeom {
    static constexpr int EPL = 16 / (int)sizeof(ST);   // elements per lane per key
    static constexpr int LPK = HD / EPL;               // lanes per key
    static constexpr int KPW = 32 / LPK;               // keys per warp pass
    static constexpr int VPL = HD / 32;                // value elements per lane
    static constexpr int PSTRIDE = HD + 4;             // (max, sum, pad, pad, o[HD]): o stays 16-byte aligned
};

__device__ __forceinline__ void warp_key_range(int pos, int s, int S, int warp, int &kw0, int &kw1) {
    const int k0 = (int)((unsigned)(pos * s) / (unsigned)S), k1 = (int)((unsigned)(pos * (s + 1)) / (unsigned)S);   // (pos * 8 fits easily)
    // the last warp of the last part takes the new position, so it gets no cached keys (its CTA would otherwise
    // finish last and hold up the barrier that follows)
    const int nw = (s == S - 1) ? NCW - 1 : NCW;
    kw0 = k0 + (k1 - k0) * min(warp, nw) / nw;
    kw1 = k0 + (k1 - k0) * min(warp + 1, nw) / nw;
}

// This CTA's first (usually only) work item of the attention phase: it depends on the position alone, so it is
// worked out once per step, not once per layer (a dozen integer divisions at the head of a latency-bound phase).
struct AttnItem {
    int h, s, kw0, kw1;
};
__device__ __forceinline__ AttnItem attn_item(const ClStepArgs &a, int item, int pos, int warp) {
    AttnItem it;
    it.h = item % a.H;
    it.s = item / a.H;
    warp_key_range(pos, it.s, a.att_parts, warp, it.kw0, it.kw1);
    return it;
}

template <typename ST, int HD>
__device__ void attention_phase(const ClStepArgs &a, const ClLayerDev &L, int pos, Smem *sm, const AttnItem &first) {
    using G = AttnGeom<ST, HD>;
    constexpr int EPL = G::EPL, LPK = G::LPK, KPW = G::KPW, VPL = G::VPL, PSTRIDE = G::PSTRIDE;
    constexpr int WSTRIDE = HD + 2;   // per-warp record in shared memory: (max, sum, o[HD])
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int S = a.att_parts, d = a.d;
    const int sub = lane / LPK, li = lane % LPK;
    const float scale = rsqrtf((float)HD);
    ST *Kc = (ST *)L.kc;
    ST *Vc = (ST *)L.vc;
    const int group = a.H / a.Hkv, kvd = a.Hkv * HD;   // grouped-query attention: `group` query heads share a key/value head
    float *wrec = sm->partial;   // [NCW][WSTRIDE]
    for (int item = blockIdx.x; item < a.H * S; item += gridDim.x) {
        const AttnItem cur = (item == (int)blockIdx.x) ? first : attn_item(a, item, pos, warp);
        const int h = cur.h, s = cur.s, kvh = h / group, kw0 = cur.kw0, kw1 = cur.kw1;
        const float *qraw = a.qkv + h * HD;
        // rotated query, this lane's EPL elements
        float qr[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const int idx = li * EPL + e;
            const int i = idx < HD / 2 ? idx : idx - HD / 2;
            const float2 cs = a.rope_cs[(size_t)pos * (HD / 2) + i];
            const float qa = ldcg_f(qraw + i), qb = ldcg_f(qraw + i + HD / 2);
            qr[e] = idx < HD / 2 ? qa * cs.x - qb * cs.y : qb * cs.x + qa * cs.y;
        }
        float m_run = -INFINITY, l_run = 0.f, o_run[VPL];
#pragma unroll
        for (int e = 0; e < VPL; ++e) o_run[e] = 0.f;
        for (int j0 = kw0; j0 < kw1; j0 += 32) {
            const int n = min(32, kw1 - j0);
            // scores of up to 32 keys; lane j ends up holding the score of key j0 + j
            float my_score = -INFINITY;
            // KPW keys per pass; the key rows of up to PB passes are requested together (one memory round trip), then
            // scored; passes past the last key are skipped (a warp usually holds far fewer than 32 keys)
            constexpr int NPASS = 32 / KPW, PB = NPASS < 8 ? NPASS : 8;
#pragma unroll
            for (int b0 = 0; b0 < NPASS; b0 += PB) {
                if (b0 * KPW >= n) break;   // uniform
                uint4 raw[PB];
#pragma unroll
                for (int p = 0; p < PB; ++p) {
                    const int j = (b0 + p) * KPW + sub;
                    raw[p] = make_uint4(0u, 0u, 0u, 0u);
                    if (j < n) raw[p] = __ldcg((const uint4 *)(Kc + ((size_t)kvh * a.max_seq + j0 + j) * HD + li * EPL));
                }
#pragma unroll
                for (int p = 0; p < PB; ++p) {
                    const int jb = (b0 + p) * KPW;
                    if (jb < n) {   // uniform
                        float sc = 0.f;
                        if (sizeof(ST) == 2) {
                            const unsigned u[4] = {raw[p].x, raw[p].y, raw[p].z, raw[p].w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float k0, k1;
                                ClPair16<ST>::get(u[e], k0, k1);
                                sc = fmaf(qr[(2 * e) % EPL], k0, sc);
                                sc = fmaf(qr[(2 * e + 1) % EPL], k1, sc);
                            }
                        } else {
                            sc = fmaf(qr[0], __uint_as_float(raw[p].x), sc);
                            sc = fmaf(qr[1 % EPL], __uint_as_float(raw[p].y), sc);
                            sc = fmaf(qr[2 % EPL], __uint_as_float(raw[p].z), sc);
                            sc = fmaf(qr[3 % EPL], __uint_as_float(raw[p].w), sc);
                        }
#pragma unroll
                        for (int o = LPK >> 1; o > 0; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
                        sc *= scale;
                        // key jb + k sits in lanes [k * LPK, (k + 1) * LPK): hand it to lane jb + k
#pragma unroll
                        for (int k = 0; k < KPW; ++k) {
                            const float v = __shfl_sync(0xffffffffu, sc, k * LPK);
                            if (lane == jb + k && jb + k < n) my_score = v;
                        }
                    }
                }
            }
            float m_new = my_score;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m_new = fmaxf(m_new, __shfl_xor_sync(0xffffffffu, m_new, o));
            m_new = fmaxf(m_new, m_run);
            const float p = (lane < n) ? expf(my_score - m_new) : 0.f;
            const float resc = (l_run > 0.f) ? expf(m_run - m_new) : 0.f;
            l_run = fmaf(l_run, resc, warp_sum(p));
#pragma unroll
            for (int e = 0; e < VPL; ++e) o_run[e] *= resc;
            m_run = m_new;
            // value rows, eight requested at a time (rows past the end repeat the last one with weight 0); groups past
            // the last key are skipped
#pragma unroll
            for (int jg = 0; jg < 32; jg += 8) {
                if (jg >= n) break;   // uniform
                float vv[8][VPL];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    load_vals<ST, VPL>(Vc + ((size_t)kvh * a.max_seq + j0 + min(jg + j, n - 1)) * HD + lane * VPL, vv[j]);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float pj = __shfl_sync(0xffffffffu, p, jg + j);
#pragma unroll
                    for (int e = 0; e < VPL; ++e) o_run[e] = fmaf(pj, vv[j][e], o_run[e]);
                }
            }
        }
        if (s == S - 1 && warp == NCW - 1) {
            // the new position: rotate this step's key, round key and value to the storage type, append both to the
            // cache and fold them in as one more key
            const float *kraw = a.qkv + d + kvh * HD, *vraw = a.qkv + d + kvd + kvh * HD;
            const bool owner = (h % group) == 0;   // one query head of the group appends the shared key/value head
            float sc = 0.f;
            ST kst[EPL];
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                const int idx = li * EPL + e;
                const int i = idx < HD / 2 ? idx : idx - HD / 2;
                const float2 cs = a.rope_cs[(size_t)pos * (HD / 2) + i];
                const float ka = ldcg_f(kraw + i), kb = ldcg_f(kraw + i + HD / 2);
                kst[e] = st_from_f32<ST>(idx < HD / 2 ? ka * cs.x - kb * cs.y : kb * cs.x + ka * cs.y);
                sc = fmaf(qr[e], st_to_f32<ST>(kst[e]), sc);
            }
#pragma unroll
            for (int o = LPK >> 1; o > 0; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
            sc = __shfl_sync(0xffffffffu, sc, 0) * scale;
            if (sub == 0 && owner) {
#pragma unroll
                for (int e = 0; e < EPL; ++e) Kc[((size_t)kvh * a.max_seq + pos) * HD + li * EPL + e] = kst[e];
            }
            float vn[VPL];
#pragma unroll
            for (int e = 0; e < VPL; ++e) {
                const ST vs = st_from_f32<ST>(ldcg_f(vraw + lane * VPL + e));
                if (owner) Vc[((size_t)kvh * a.max_seq + pos) * HD + lane * VPL + e] = vs;
                vn[e] = st_to_f32<ST>(vs);
            }
            const float m_new = fmaxf(m_run, sc);
            const float resc = (l_run > 0.f) ? expf(m_run - m_new) : 0.f;
            const float pn = expf(sc - m_new);
            l_run = fmaf(l_run, resc, pn);
#pragma unroll
            for (int e = 0; e < VPL; ++e) o_run[e] = fmaf(o_run[e], resc, pn * vn[e]);
            m_run = m_new;
        }
        // merge the warps of this CTA in shared memory (fixed order), one record per (h, s) to global memory
        if (lane == 0) {
            wrec[warp * WSTRIDE] = m_run;
            wrec[warp * WSTRIDE + 1] = l_run;
        }
#pragma unroll
        for (int e = 0; e < VPL; ++e) wrec[warp * WSTRIDE + 2 + lane * VPL + e] = o_run[e];
        consumer_sync();
        if (tid < HD) {
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < NCW; ++w)
                if (wrec[w * WSTRIDE + 1] > 0.f) M = fmaxf(M, wrec[w * WSTRIDE]);
            float Ls = 0.f, O = 0.f;
#pragma unroll
            for (int w = 0; w < NCW; ++w) {
                const float lw = wrec[w * WSTRIDE + 1];
                if (lw > 0.f) {
                    const float f = expf(wrec[w * WSTRIDE] - M);
                    Ls = fmaf(lw, f, Ls);
                    O = fmaf(wrec[w * WSTRIDE + 2 + tid], f, O);
                }
            }
            float *rec = a.att_part + ((size_t)h * ATT_MAX_PARTS + s) * PSTRIDE;
            if (tid == 0) {
                rec[0] = M;     // -inf for an empty part
                rec[1] = Ls;    // 0 for an empty part
            }
            rec[4 + tid] = O;
        }
        consumer_sync();
    }
}

// Attention output as the next projection's input: merges the S part records of each head on the fly.
// xr[it][e] = att[(it * NCT + tid) * EPC + e].
template <int EPC, int HD>
__device__ __forceinline__ void load_att_merged(const ClStepArgs &a, float (&xr)[MAXIT][EPC]) {
    constexpr int PSTRIDE = HD + 4;
    const int nchunks = a.d / EPC, S = a.att_parts;
#pragma unroll
    for (int it = 0; it < MAXIT; ++it) {
        const int ch = it * NCT + threadIdx.x;
#pragma unroll
        for (int e = 0; e < EPC; ++e) xr[it][e] = 0.f;
        if (ch < nchunks) {
            const int h = (ch * EPC) / HD, e0 = (ch * EPC) % HD;
            const float *rec = a.att_part + (size_t)h * ATT_MAX_PARTS * PSTRIDE;
            // (max, sum) of every part and the outputs of the first four parts are requested together: one memory
            // round trip for S <= 4.  (Holding all eight parts' outputs at once spilled registers.)
            float2 ml[ATT_MAX_PARTS];
            float o[4][EPC];
#pragma unroll
            for (int s = 0; s < ATT_MAX_PARTS; ++s) {
                ml[s] = make_float2(0.f, 0.f);
                if (s < S) ml[s] = __ldcg((const float2 *)(rec + (size_t)s * PSTRIDE));   // uniform over the grid
            }
            float M = -INFINITY, Ls = 0.f, f[ATT_MAX_PARTS];
#pragma unroll
            for (int b = 0; b < ATT_MAX_PARTS; b += 4) {
                if (b >= S) break;   // uniform
#pragma unroll
                for (int s = 0; s < 4; ++s) {
#pragma unroll
                    for (int e = 0; e < EPC; ++e) o[s][e] = 0.f;
                    if (b + s < S) {
                        const float *r = rec + (size_t)(b + s) * PSTRIDE;
#pragma unroll
                        for (int q = 0; q < EPC / 4; ++q) {
                            const float4 t = ldcg_f4(r + 4 + e0 + 4 * q);
                            o[s][4 * q] = t.x; o[s][4 * q + 1] = t.y; o[s][4 * q + 2] = t.z; o[s][4 * q + 3] = t.w;
                        }
                    }
                }
                if (b == 0) {
#pragma unroll
                    for (int s = 0; s < ATT_MAX_PARTS; ++s)
                        if (s < S && ml[s].y > 0.f) M = fmaxf(M, ml[s].x);
#pragma unroll
                    for (int s = 0; s < ATT_MAX_PARTS; ++s) {   // part order
                        f[s] = (s < S && ml[s].y > 0.f) ? expf(ml[s].x - M) : 0.f;
                        Ls = fmaf(ml[s].y, f[s], Ls);
                    }
                }
#pragma unroll
                for (int s = 0; s < 4; ++s)
#pragma unroll
                    for (int e = 0; e < EPC; ++e) xr[it][e] = fmaf(o[s][e], f[b + s], xr[it][e]);
            }
            const float inv = 1.f / Ls;
#pragma unroll
            for (int e = 0; e < EPC; ++e) xr[it][e] *= inv;
        }
    }
}

// ---- the kernel ----------------------------------------------------------------------------------------
template <typename WT, int HD>
__global__ void __launch_bounds__(NCT + 32, 1) k_token_steps(ClStepArgs a) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char *ring = smem_raw;
    Smem *sm = (Smem *)(smem_raw + (size_t)NSLOT * SLOT_BYTES);
    ClDevState *st = a.st;
    if (st->done) return;   // written only between launches: uniform over the grid
    constexpr int EPC = Chunk<WT>::EPC;
    const int tid = threadIdx.x;

    if (tid == 0) {
        for (int i = 0; i < NSLOT; ++i) {
            bar_init(&sm->full[i], 1);
            bar_init(&sm->empty[i], NCW);
        }
        sm->abort = 0;
        sm->halt = 0;
        sm->wait_ns = a.wait_ns;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int ctx0 = st->ctx;
    const int d = a.d, F = a.F, V = a.V;

    if (tid >= NCT) {
        // ------------------------------ producer warp ------------------------------
        if (tid == NCT) producer_loop<WT>(a, ring, sm, st);
        return;
    }

    // ------------------------------ consumer warps ------------------------------
    Ring rg{0u, 0u};
    unsigned bar_target = 0u;   // arrivals that complete the next grid barrier (thread 0's copy is the one used)
    unsigned long long busy = 0ull;   // calibration: time this CTA spent in the matrix phases
    unsigned long long *busy_p = (a.busy_ns && tid == 0) ? &busy : nullptr;
    float xr[MAXIT][EPC];
    int tok = st->cyc_tok[a.row0];
    for (int step = 0; step < a.n_steps; ++step) {
        const int pos = ctx0 + a.row0 + step;
        const AttnItem att_first = attn_item(a, blockIdx.x, pos, tid >> 5);
        // phase 0: embedding row -> residual stream (each CTA writes its slice)
        {
            const WT *erow = (const WT *)a.embed + (size_t)tok * d;
            for (int i = blockIdx.x * NCT + tid; i < d; i += gridDim.x * NCT) a.x[i] = st_to_f32<WT>(erow[i]);
        }
        grid_barrier(a.bar, bar_target, a.bar_arrivals, sm, st);
        for (int ki = 0; ki < a.n_kept; ++ki) {
            const int ent = a.kept[ki], fl = ent >> 16;   // bit 0: this layer's attention half is skipped, bit 1: its FFN half
            const ClLayerDev L = a.layers[ent & 0xffff];
            if (!(fl & 1)) {
            // QKV projection of the normalised stream.  (Asking L2 for the attention phase's keys and values from here,
            // a matrix phase early, measured slower: whichever thread issues the request, consumer warp or producer,
            // stalls about 1.5 us on it, more than the attention phase gains.)
            load_x_rmsnorm<EPC>(a.x, L.n1, d, a.eps, xr, sm);
            consume_matrix<WT>(d + 2 * a.Hkv * HD, d, 1, xr, rg, ring, sm, st, [&](int rb0, int nrb) {
                for (int r = tid; r < nrb; r += NCT) a.qkv[rb0 + r] = row_sum(sm, r);
            }, a.cum_w, busy_p);
            grid_barrier(a.bar, bar_target, a.bar_arrivals, sm, st);
            attention_phase<WT, HD>(a, L, pos, sm, att_first);
            grid_barrier(a.bar, bar_target, a.bar_arrivals, sm, st);
            // attention output projection + residual
            load_att_merged<EPC, HD>(a, xr);
            consume_matrix<WT>(d, d, 1, xr, rg, ring, sm, st, [&](int rb0, int nrb) {
                for (int r = tid; r < nrb; r += NCT) a.x[rb0 + r] = ldcg_f(a.x + rb0 + r) + row_sum(sm, r);
            }, a.cum_w, busy_p);
            grid_barrier(a.bar, bar_target, a.bar_arrivals, sm, st);
            }
            if (!(fl & 2)) {
            // gate/up projections (rows interleaved) + SiLU(gate) * up
            load_x_rmsnorm<EPC>(a.x, L.n2, d, a.eps, xr, sm);
            consume_matrix<WT>(2 * F, d, 2, xr, rg, ring, sm, st, [&](int rb0, int nrb) {
                for (int pr = tid; pr < nrb / 2; pr += NCT) {
                    const float gt = row_sum(sm, 2 * pr), up = row_sum(sm, 2 * pr + 1);
                    a.hff[rb0 / 2 + pr] = gt / (1.f + expf(-gt)) * up;
                }
            }, a.cum_w, busy_p);
            grid_barrier(a.bar, bar_target, a.bar_arrivals, sm, st);
            // down projection + residual
            load_x<EPC>(a.hff, F, xr);
            consume_matrix<WT>(d, F, 1, xr, rg, ring, sm, st, [&](int rb0, int nrb) {
                for (int r = tid; r < nrb; r += NCT) a.x[rb0 + r] = ldcg_f(a.x + rb0 + r) + row_sum(sm, r);
            }, a.cum_w, busy_p);
            grid_barrier(a.bar, bar_target, a.bar_arrivals, sm, st);
            }
        }
        // LM head on the normalised stream, fused with clamp + online softmax / entropy / argmax
        load_x_rmsnorm<EPC>(a.x, a.final_norm, d, a.eps, xr, sm);
        ClHeadPartial run{0.f, 0.f, 0.f, 0x7fffffff};
        float *lg = a.logits ? a.logits + (size_t)step * V : nullptr;
        consume_matrix<WT>(V, d, 1, xr, rg, ring, sm, st, [&](int rb0, int nrb) {
            for (int r = tid; r < nrb; r += NCT) {
                const float l = fminf(fmaxf(row_sum(sm, r), -CL_LOGIT_CLAMP), CL_LOGIT_CLAMP);
                if (lg) lg[rb0 + r] = l;
                run = cl_hp_merge(run, ClHeadPartial{l, 1.f, 0.f, rb0 + r});
            }
        }, a.cum_w, busy_p);
        run = hp_block_reduce(run, sm);
        if (tid == 0) a.head_part[blockIdx.x] = run;
        grid_barrier(a.bar, bar_target, a.bar_arrivals, sm, st);
        // every CTA reduces the per-CTA partials itself (same order everywhere), so all know the token
        ClHeadPartial fin{0.f, 0.f, 0.f, 0x7fffffff};
        for (int b = tid; b < (int)gridDim.x; b += NCT) {
            const ClHeadPartial *p = a.head_part + b;
            ClHeadPartial q;
            q.m = ldcg_f(&p->m); q.z = ldcg_f(&p->z); q.s = ldcg_f(&p->s); q.idx = __ldcg(&p->idx);
            fin = cl_hp_merge(fin, q);
        }
        fin = hp_block_reduce(fin, sm);
        tok = min(max(fin.idx, 0), V - 1);   // (only an aborted run can leave the range; keep the next gather in bounds)
        const float pm = 1.f / fin.z;        // top-1 probability: the same bits in every CTA
        // confidence-aware drafting: the candidate whose top-1 probability falls below the threshold is the last one
        const bool stop = a.mode == CL_STEP_DRAFT && a.stop_p > 0.f && pm < a.stop_p;
        if (blockIdx.x == 0 && tid == 0) {
            const float Hh = logf(fin.z) - fin.s / fin.z;   // entropy of the softmax (Eq. 2), from sums relative to the max
            const float conf = 1.f - Hh * a.inv_log_v;      // Eq. 3-4
            if (a.mode == CL_STEP_DRAFT) {
                st->cyc_tok[a.row0 + step + 1] = tok;
                st->d_pmax[a.row0 + step] = pm;
                st->d_conf[a.row0 + step] = conf;
                if (stop || step == a.n_steps - 1) st->n_drafted = a.row0 + step + 1;
            } else {
                // vanilla decoding: the token is emitted at once and becomes the next pending token
                if (a.out_tokens && st->n_out < st->max_new) a.out_tokens[st->n_out] = tok;
                st->n_out = min(st->n_out + 1, st->max_new);
                st->tgt_tok[0] = tok;
                st->emitted[0] = tok;
                st->cyc_tok[0] = tok;
                st->v_pmax[0] = pm;
                st->v_conf[0] = conf;
                st->ctx = pos + 1;
                st->n_acc_last = 0;
                st->cycles += 1ull;
                st->emitted_total += 1ull;
            }
        }
        if (stop) {   // uniform over the grid
            if (tid == 0) *(volatile int *)&sm->halt = 1;
            break;
        }
        // the next step's phase 0 writes x, which nobody reads any more in this step: no barrier needed here,
        // and head_part is rewritten only after the next step's grid barriers
    }
    if (busy_p) a.busy_ns[blockIdx.x] = busy;
}

}  // namespace

size_t cl_step_smem_bytes() { return (size_t)NSLOT * SLOT_BYTES + sizeof(Smem); }

int cl_step_max_cols(int wdtype) { return MAXIT * NCT * (wdtype != 0 ? 8 : 4); }

cudaError_t cl_launch_token_steps(int wdtype, int head_dim, const ClStepArgs &a, int grid, cudaStream_t s) {
    const void *fn = nullptr;
    if (wdtype == 1 && head_dim == 64) fn = (const void *)k_token_steps<__nv_bfloat16, 64>;
    else if (wdtype == 1 && head_dim == 128) fn = (const void *)k_token_steps<__nv_bfloat16, 128>;
    else if (wdtype == 2 && head_dim == 64) fn = (const void *)k_token_steps<__half, 64>;
    else if (wdtype == 2 && head_dim == 128) fn = (const void *)k_token_steps<__half, 128>;
    else if (wdtype == 0 && head_dim == 64) fn = (const void *)k_token_steps<float, 64>;
    else if (wdtype == 0 && head_dim == 128) fn = (const void *)k_token_steps<float, 128>;
    else return cudaErrorInvalidValue;
    const size_t smem = cl_step_smem_bytes();
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    void *params[] = {(void *)&a};
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(NCT + 32), params, smem, s);
}
