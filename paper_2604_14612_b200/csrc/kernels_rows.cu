// Persistent full-model pass over T <= 9 token rows of a model stored in a 16-bit type: the (K+1)-row verify pass of
// Section 3 (Figure 2: the target model checks the K candidates and the pending token in one forward pass), and the
// short prompt chunks, which are the same pass.  One cooperative launch runs every layer and the LM head.
//
// The pass is bound by HBM weight streaming (at most 9 flop per weight byte), so its shape follows the single-token
// step kernel: one CTA per SM, every CTA owns a contiguous block of rows of every matrix (single-row granularity, so
// all SMs stream the same number of bytes), one producer warp walks the static schedule and keeps a 210 KB ring of
// weight tiles filled straight through the phase boundaries, and the phases of a layer (QKV | attention | O |
// gate/up | down) follow one another inside the launch, ordered by completion counters per buffer (below), not by
// launches.  What differs is the arithmetic: 2 T activation
// rows against every weight row is more than the CUDA cores issue at the HBM rate, so the contraction runs on the
// tensor cores:
//
//   D[m, n] = sum_k A[m, k] * B[n, k]      tcgen05.mma, M = 128, N = the CTA's rows (multiple of 16, <= 224), K = 16
//
// A = activation rows: row t holds hi = round16(v), row T + t holds lo = round16(v - hi) of token t, so the product
//     keeps about 16 mantissa bits of the fp32 activations; rows 2 T .. 127 of the operand are whatever the shared
//     memory behind the tile holds -- row m of D depends on row m of A only, and those rows of D are never read.
// B = the CTA's weight rows.  The weights are stored a second time, in the order this kernel streams them: CTA by
//     CTA (each CTA's row block [r0, r1) of a matrix is one contiguous region, so a CTA walks memory sequentially --
//     with a k-block-major order over the whole matrix every copy of a CTA started in another 2 MB page and the
//     stream ran at a third of the HBM rate), inside a block k-block by k-block, [K / 64][r1 - r0][64] elements, with
//     the 16-byte pieces of a row's 128 bytes permuted by (piece ^ (row & 7)): that is the layout the tensor core's
//     128-byte-swizzle shared-memory descriptor expects, so the rows [g0, g1) of one k-block arrive with one bulk
//     copy of exactly the bytes this CTA owns.  The tile in shared memory starts at row g0 & ~7 (keeping row & 7
//     equal on both sides); rows in front of g0 and behind g1 are stale -- column n of D depends on row n of B
//     only, and those columns are never read.
// The accumulator lives in tensor memory (two buffers of 256 columns); it is drained into fp32 registers after
// at most `chain` k-blocks (8 by default: 512 elements of K, more where a ring entry holds more), so a long K is summed
// in fp32 registers in pieces, not in one tensor-core chain: the pieces bound the rounding error of the chain.
// Warp roles: warps 0-13 workers (embedding, attention, epilogues; warps 0, 4, 8, 12 are the four that can read
// tensor-memory lanes 0-31 and drain the accumulator), warp 14 producer, warp 15 MMA issue and tensor-memory owner.
// RMSNorm is split around the GEMM as in the other tensor-core kernels: the activation operand holds x * gain,
// the per-token scale rsqrt(mean x^2 + eps) multiplies the product.
// Every wait is bounded; on expiry an error flag is raised, later waits fall through, copies in flight are waited
// for, tensor memory is released and the host reports CL_ETIMEOUT.
#include <math.h>
#include <stddef.h>
#include <string.h>

#include "tc_common.cuh"

namespace {

constexpr int RW = 14;                 // worker warps (16 warps in all: four per scheduler, 128 registers per thread)
constexpr int RT = RW * 32;            // worker threads
constexpr int R_THREADS = RT + 64;     // + producer warp + MMA warp
constexpr int R_RING = 215040;         // ring of tiles in flight per SM, allocated by the byte (multiples of 1 KB): 210 KB,
                                       // with the control block and the alignment slack all the shared memory a CTA can have
constexpr int R_NE = 16;               // most ring entries (bulk-copy groups with their own pair of mbarriers) in flight
constexpr int R_MAXN = 224;            // most rows of a weight tile (an accumulator buffer has 256 columns)
constexpr int R_CTRL_BYTES = 16384;    // control block behind the ring (at least 16 KB: see the kernel)
constexpr int R_ATT_MAXS = 8;          // most parts the cached keys of a head are cut into

constexpr int R_STAGE_LD = R_MAXN + 1;  // row pitch of the epilogue staging buffer (odd: token rows fall into different banks)
constexpr int R_STAGE_FLOATS = 2032;   // staging buffer: a GEMM tile's raw products of every token row

struct RSmem {
    unsigned long long full[R_NE], empty[R_NE], tfull[2], tempty[2];
    unsigned vstart[R_NE];             // producer: where an entry in flight starts in the ring's running byte count
    unsigned long long wait_ns;
    unsigned tmem_base;
    int abort;
    int is_last;
    float scale[CL_SLOTS];             // RMSNorm scale of every token row for the current phase
    float red[CL_SLOTS];
    float esum[16][CL_SLOTS];          // embedding phase: per-chunk sums of squares
    ClHeadPartial hpw[RW];             // LM head: per-warp statistics
    float wsum[RW];                    // residual phase: per-warp sums of squares
    // one buffer, used in turn by: the GEMM epilogues (raw products of a tile, [T][R_STAGE_LD]); the residual epilogue
    // ([T][64] squares); the attention phase (per-warp (max, sum, o[hd]) records, [RW][hd + 2])
    alignas(16) float stage[R_STAGE_FLOATS];
    alignas(16) unsigned short knew[CL_MAX_T * 128];   // attention: the pass's own keys (rotated) and values in the storage type
    alignas(16) unsigned short vnew[CL_MAX_T * 128];
    unsigned long long t_prev, ph_ns[8];   // diagnostics: time of thread 0 by phase
};

// Diagnostics (a.phase_ns != null): thread 0 adds the time since its last call to phase `idx`
// (0 embedding, 1 QKV, 2 attention, 3 output projection, 4 gate/up, 5 down, 6 LM head, 7 grid barriers).
__device__ __forceinline__ void phase_clock(const ClRowsArgs &a, RSmem *sm, int idx) {
    if (a.phase_ns && threadIdx.x == 0) {
        const unsigned long long now = gtime_ns();
        sm->ph_ns[idx] += now - sm->t_prev;
        sm->t_prev = now;
    }
}

// ---- completion counters -------------------------------------------------------------------------------
// The phases of a layer are not separated by grid barriers.  Every buffer that one phase writes and the next reads has
// counters in global memory that only grow during a launch (the host zeroes them before it): a writer adds, with
// release semantics and after its CTA's stores, how much of a piece it has completed; a reader waits (acquire, bounded)
// until the piece is complete for the pass over the buffer it needs.  a.sync + ...
//   c_ax  + kb   columns [64 kb, 64 kb + 64) of the operand rows Ax, 64 per pass: pass 1 = embedding, 2 l + 2 = layer l's
//                output projection, 2 l + 3 = its down projection (so layer l's QKV needs 64 (2 l + 1), its gate/up 64 (2 l + 2))
//   c_ssq        CTAs that have published their sum of squares of the residual rows, grid size per pass (same passes)
//   c_qkv + b    rows [hd b, hd b + hd) of the QKV product (one head's q, k or v), hd per layer
//   c_att + h    head h's attention output in Aatt, 1 per layer
//   c_ah  + kb   columns [64 kb, 64 kb + 64) of the FFN hidden operand rows Ah, 64 per layer
// A k-block of a GEMM starts as soon as its 64 activation columns are complete, whatever the rest of the grid is
// doing; the weight stream never waits.  Overwriting a buffer needs no counter: every phase needs all of K of the one
// before it to finish, so by the time a CTA can write a buffer again every reader of its previous contents is done.
// One grid barrier remains, in front of the merge of the LM-head statistics.
__device__ __forceinline__ void counter_add(unsigned *c, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(c), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned counter_read(const unsigned *c) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(c) : "memory");
    return v;
}

// ---- schedule ---------------------------------------------------------------------------------------
// GEMM jobs in execution order: job 4 l + m = matrix m of layer l (0 QKV, 1 O, 2 gate/up, 3 down), job 4 L = LM head.
// A CTA's rows [r0, r1) of a job are cut into groups of at most R_MAXN tile rows; a group's K range into ring entries
// of as many k-blocks as fit.  Producer, MMA issuer and drain warps walk the same sequence.
struct Job {
    const char *W;        // k-block-major weights
    const unsigned short *A;
    int rows, KB, unit, epi;
    int dep, dep_shift;   // k-block kb of the activation operand is complete when counter dep + (kb >> dep_shift) ...
    unsigned dep_target;  // ... has reached this value (see "completion counters")
    int split;            // CTAs that share a row block and cut its K range between them (1: every CTA owns rows over all of K)
};

__device__ __forceinline__ Job job_of(const ClRowsArgs &a, int ji) {
    Job j;
    const int L = a.L;
    if (ji < 4 * L) {
        const int l = ji >> 2, m = ji & 3;
        const ClRowsLayer &y = a.layers[l];
        const int hs = a.hd == 128 ? 1 : 0;   // k-blocks per head: 2 (hd 128) or 1 (hd 64)
        if (m == 0) { j.W = y.wqkv; j.A = a.Ax; j.rows = a.d + 2 * a.Hkv * a.hd; j.KB = a.d >> 6; j.unit = 1; j.epi = CL_VEPI_STORE; j.dep = a.c_ax; j.dep_shift = 0; j.dep_target = 64u * (2 * l + 1); j.split = 1; }
        else if (m == 1) { j.W = y.wo; j.A = a.Aatt; j.rows = a.d; j.KB = a.d >> 6; j.unit = 1; j.epi = CL_VEPI_RESID; j.dep = a.c_att; j.dep_shift = hs; j.dep_target = (unsigned)(l + 1); j.split = a.split; }
        else if (m == 2) { j.W = y.wgu; j.A = a.Ax; j.rows = 2 * a.F; j.KB = a.d >> 6; j.unit = 2; j.epi = CL_VEPI_SILU; j.dep = a.c_ax; j.dep_shift = 0; j.dep_target = 64u * (2 * l + 2); j.split = 1; }
        else { j.W = y.wd; j.A = a.Ah; j.rows = a.d; j.KB = a.F >> 6; j.unit = 1; j.epi = CL_VEPI_RESID; j.dep = a.c_ah; j.dep_shift = 0; j.dep_target = 64u * (l + 1); j.split = a.split; }
    } else {
        j.W = a.head; j.A = a.Ax; j.rows = a.V; j.KB = a.d >> 6; j.unit = 1; j.epi = CL_VEPI_HEAD; j.dep = a.c_ax; j.dep_shift = 0; j.dep_target = 64u * (2 * L + 1); j.split = 1;
    }
    return j;
}

// Rows [r0, r1) of a matrix that CTA c of G owns (a unit is `unit` consecutive rows that stay together).
__device__ __forceinline__ void rows_of_cta(int rows, int unit, int c, int G, int &r0, int &r1) {
    const long long units = rows / unit;
    r0 = (int)(units * c / G) * unit;
    r1 = (int)(units * (c + 1) / G) * unit;
}
// Rows of this CTA (split = 1) or of its group of `split` neighbouring CTAs.
__device__ __forceinline__ void rows_of(int rows, int unit, int split, int &r0, int &r1) {
    rows_of_cta(rows, unit, blockIdx.x / split, gridDim.x / split, r0, r1);
}

// Position in the schedule: (job, group of the CTA's rows, ring entry).  advance() is a handful of instructions inside a
// group (the producer, the MMA issuer and the drain warps each run it once per entry, serially, so it has to be);
// everything that costs a division is worked out once per group.
struct Cursor {
    const ClRowsArgs &a;
    int njobs, ars;
    // job
    int ji;
    const char *W;
    const unsigned short *A;
    int rows, KB, unit, epi;
    int dep, dep_shift;
    unsigned dep_target;
    int kb_begin, kb_end;     // the CTA's k-blocks of the job (all of them unless the job is split over K)
    int r0, r1;               // the rows of the CTA (of its group, for a job split over K)
    // group
    int g0, g1, a0, npad;     // weight rows [g0, g1); first tile row g0 & ~7; tile rows (multiple of 16)
    int per;                  // k-blocks per ring entry
    unsigned stride;          // bytes between the k-block tiles of an entry (activation rows + weight rows)
    size_t wbase;             // byte offset in W of (row g0, k-block 0)
    unsigned wstep;           // bytes between k-blocks in W (the CTA's block is [K / 64][r1 - r0][64])
    // ring entry
    int kb0, kbs, in_chain;   // the entry's k-blocks; in_chain: k-blocks of the accumulation chain before this entry
    // the entry's place in the ring: every role computes the same sequence.  Entries are laid end to end; one that would
    // cross the end of the ring starts at its beginning instead.  voff counts all bytes so far, the skipped ones too, so
    // an entry fits once voff + size - (voff of the oldest entry still in use) <= R_RING.
    unsigned e, par;          // entry index (mbarrier pair) and its phase parity
    unsigned poff, voff, size;
    bool done;

    __device__ Cursor(const ClRowsArgs &args) : a(args), ji(-1), in_chain(0), e(R_NE - 1), par(1u), poff(0u), voff(0u), size(0u), done(false) {
        njobs = 4 * a.L + (a.want_head ? 1 : 0);
        ars = (2 * a.T + 7) & ~7;
        next_job();
        place();
    }
    __device__ __forceinline__ bool last() const { return kb0 + kbs >= kb_end; }             // last entry of the group
    __device__ __forceinline__ bool job_last() const { return last() && g1 >= r1; }          // ... of the job, for this CTA
    __device__ __forceinline__ bool chain_first() const { return in_chain == 0; }
    __device__ __forceinline__ bool chain_last() const { return last() || in_chain + kbs >= a.chain; }
    __device__ __forceinline__ void place() {
        if (done) return;
        const unsigned nsize = (unsigned)kbs * stride;
        poff += size;
        voff += size;
        if (poff + nsize > (unsigned)R_RING) {
            voff += (unsigned)R_RING - poff;
            poff = 0u;
        }
        size = nsize;
        if (++e == (unsigned)R_NE) { e = 0u; par ^= 1u; }
    }
    __device__ void open_group(int g) {
        g0 = g;
        a0 = g & ~7;
        g1 = min(r1, a0 + R_MAXN);
        npad = (g1 - a0 + 15) & ~15;
        // a tile takes the rows it is sent, rounded up to 8; the multiply-add reads npad rows, up to 8 more: whatever
        // lies behind the tile (the columns of D they produce are never read)
        stride = (unsigned)(ars + ((g1 - a0 + 7) & ~7)) * 128u;
        per = max(1, min(32, a.entry / (int)stride));
        wbase = ((size_t)r0 * KB + (size_t)(g0 - r0)) * 128;
        wstep = (unsigned)(r1 - r0) * 128u;
        kb0 = kb_begin;
        kbs = min(per, kb_end - kb_begin);
    }
    __device__ void next_job() {
        for (++ji; ji < njobs; ++ji) {
            const Job j = job_of(a, ji);
            W = j.W; A = j.A; rows = j.rows; KB = j.KB; unit = j.unit; epi = j.epi;
            dep = j.dep; dep_shift = j.dep_shift; dep_target = j.dep_target;
            rows_of(rows, unit, j.split, r0, r1);
            const int member = (int)blockIdx.x % j.split;
            kb_begin = KB * member / j.split;
            kb_end = KB * (member + 1) / j.split;
            if (r0 < r1 && kb_begin < kb_end) {
                open_group(r0);
                return;
            }
        }
        done = true;
    }
    __device__ __forceinline__ void advance() {
        in_chain = chain_last() ? 0 : in_chain + kbs;
        kb0 += kbs;
        if (kb0 < kb_end) {
            kbs = min(per, kb_end - kb0);
        } else if (g1 < r1) {
            open_group(g1);
        } else {
            next_job();
        }
        place();
    }
};

// ---- small helpers -------------------------------------------------------------------------------------
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, %0;" ::"n"(RT) : "memory"); }

// Orders this thread's generic-proxy accesses of global memory with async-proxy (bulk copy) accesses.
__device__ __forceinline__ void proxy_fence_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

__device__ __forceinline__ bool r_wait(unsigned long long *b, unsigned parity, RSmem *sm, int *err) {
    if (bar_try(b, parity)) return true;
    if (*(volatile int *)&sm->abort) return false;
    const unsigned long long t0 = gtime_ns();
    for (unsigned i = 1;; ++i) {
        if (bar_try(b, parity)) return true;
        if ((i & 63u) == 0u) {
            if (*(volatile int *)&sm->abort) return false;
            if (gtime_ns() - t0 > sm->wait_ns) {
                *(volatile int *)&sm->abort = 1;
                atomicOr(err, 8);
                return false;
            }
        }
    }
}

// Bounded wait for a completion counter; called by one thread.
__device__ __forceinline__ bool counter_wait(const unsigned *c, unsigned target, RSmem *sm, int *err) {
    if ((int)(counter_read(c) - target) >= 0) return true;
    const unsigned long long t0 = gtime_ns();
    for (unsigned i = 1;; ++i) {
        if ((int)(counter_read(c) - target) >= 0) return true;
        if ((i & 63u) == 0u) {
            if (*(volatile int *)&sm->abort || *(volatile int *)err) return false;
            if (gtime_ns() - t0 > sm->wait_ns) {
                *(volatile int *)&sm->abort = 1;
                atomicOr(err, 16);
                return false;
            }
        }
    }
}

// Grid barrier on one arrival counter that only grows during a launch (the host zeroes it before the launch).
// Called by every worker thread; thread 0 arrives and polls (bounded).
__device__ __forceinline__ void grid_barrier(const ClRowsArgs &a, unsigned &target, RSmem *sm) {
    worker_sync();
    if (threadIdx.x == 0 && !*(volatile int *)&sm->abort) {
        target += a.bar_arrivals;
        counter_add(a.sync, 1u);
        counter_wait(a.sync, target, sm, &a.st->err);
    }
    worker_sync();
    phase_clock(a, sm, 7);
}

__device__ __forceinline__ void tmem_ld16(unsigned taddr, float (&v)[16]) {
    unsigned r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Index (in 16-bit elements) of element k of activation row r in a k-block-major operand buffer [K / 64][R_AROWS][64].
__device__ __forceinline__ size_t a_index(int r, int k) {
    const int kb = k >> 6, c = (k & 63) >> 3, e = k & 7;
    return ((size_t)kb * CL_ROWS_AROWS + r) * 64 + (size_t)(((c ^ (r & 7)) << 3) + e);
}
__device__ __forceinline__ void a_store_split(unsigned short *A, int t, int T, int k, float v, int f16) {
    unsigned short hi, lo;
    split_b16(v, f16, hi, lo);
    A[a_index(t, k)] = hi;
    A[a_index(T + t, k)] = lo;
}

__device__ __forceinline__ ClHeadPartial rp_merge(const ClHeadPartial &a, const ClHeadPartial &b) { return cl_hp_merge(a, b); }

// ---- producer ------------------------------------------------------------------------------------------
// The whole producer warp runs this (uniform control flow; lane j issues the copy of an entry's j-th k-block, so an entry
// costs the same few instructions however many k-blocks it holds).  Weight tiles are requested as soon as the ring
// has room for the entry -- weights never change, so the stream runs ahead of the phases; the activation tiles of an
// entry are requested once the completion counters of their k-blocks say so, both on the entry's one mbarrier.
__device__ void producer(const ClRowsArgs &a, unsigned char *ring, RSmem *sm, int lane) {
    const unsigned long long policy = policy_evict_first();
    Cursor w(a), q(a);                     // weight cursor; head of the queue of entries that still lack their activation tiles
    const unsigned abytes = (unsigned)w.ars * 128u;
    int pn = 0;                            // entries between q and w: weights requested, activation tiles not yet
    int nout = 0;                          // entries between the oldest one still in use and w
    unsigned fe = 0u, fpar = 0u;           // ... that oldest entry: index and parity
    unsigned used = 0;                     // bit i: entry i has copies in flight of phase parity (used_par >> i) & 1
    unsigned used_par = 0;
    bool job_ready = false;                // every k-block of the queue head's job from its current one on is known to be complete
    int known = 0;                         // k-blocks from the queue head's first one that are known to be complete
    unsigned long long t_idle = 0;
    unsigned n_idle = 0;
    while (!w.done || pn > 0) {
        if (__shfl_sync(0xffffffffu, *(volatile int *)&sm->abort, 0)) break;
        bool progress = false;
        // (lane 0's view of a barrier and of the clock is the warp's: control flow stays uniform)
        // the oldest entry in use: have its multiply-adds read it?  Then its bytes are free.
        if (nout > 0 && __shfl_sync(0xffffffffu, (int)bar_test(&sm->empty[fe], fpar), 0)) {
            if (++fe == (unsigned)R_NE) { fe = 0u; fpar ^= 1u; }
            --nout;
            progress = true;
        }
        if (pn > 0) {
            // the head of the queue: are the activation columns of its k-blocks complete?  `known` k-blocks from the head's
            // first one are known to be; when that is not enough, lane j looks at the counter of k-block j from there (one
            // round trip for up to 32 k-blocks: a look per entry would make this loop the bottleneck of the stream)
            if (!job_ready && known < q.kbs) {
                const int kb = q.kb0 + lane;
                const bool ok = kb >= q.kb_end || (int)(counter_read(a.sync + q.dep + (kb >> q.dep_shift)) - q.dep_target) >= 0;
                const unsigned bal = __ballot_sync(0xffffffffu, ok);
                const int nk = bal == 0xffffffffu ? 32 : __ffs(~bal) - 1;
                if (nk > known) {
                    known = nk;
                    proxy_fence_global();   // other CTAs' stores (acquired above) before this warp's bulk-copy reads
                }
                job_ready = q.kb0 + known >= q.kb_end;
            }
            if (job_ready || known >= q.kbs) {
                if (lane < q.kbs)
                    bulk_g2s(ring + q.poff + (size_t)lane * q.stride, q.A + (size_t)(q.kb0 + lane) * (CL_ROWS_AROWS * 64), abytes,
                             &sm->full[q.e]);
                --pn;
                known = max(0, known - q.kbs);
                const int ji_old = q.ji, g0_old = q.g0;
                q.advance();
                if (q.done || q.ji != ji_old) {
                    job_ready = false;
                    known = 0;
                } else if (q.g0 != g0_old) {
                    known = 0;   // the next group of rows starts over at the job's first k-block (job_ready stays)
                }
                progress = true;
            }
        }
        // the next entry's weights, as soon as its bytes and its pair of barriers are free
        if (!w.done && nout < R_NE) {
            const unsigned oldest = nout > 0 ? *(volatile unsigned *)&sm->vstart[fe] : w.voff;
            if (w.voff + w.size - oldest <= (unsigned)R_RING) {
                const unsigned bbytes = (unsigned)(w.g1 - w.g0) * 128u;
                if (lane == 0) {
                    sm->vstart[w.e] = w.voff;
                    bar_expect(&sm->full[w.e], (unsigned)w.kbs * (bbytes + abytes));
                }
                __syncwarp();
                if (lane < w.kbs)
                    bulk_g2s_stream(ring + w.poff + (size_t)lane * w.stride + abytes + (size_t)(w.g0 - w.a0) * 128,
                                    w.W + w.wbase + (size_t)(w.kb0 + lane) * w.wstep, bbytes, &sm->full[w.e], policy);
                used |= 1u << w.e;
                used_par = (used_par & ~(1u << w.e)) | (w.par << w.e);
                ++pn;
                ++nout;
                w.advance();
                progress = true;
            }
        }
        if (progress) {
            t_idle = 0;
            n_idle = 0;
        } else if ((++n_idle & 255u) == 0u) {
            const unsigned long long now = __shfl_sync(0xffffffffu, gtime_ns(), 0);
            if (t_idle == 0) t_idle = now;
            else if (now - t_idle > sm->wait_ns) {
                if (lane == 0) {
                    *(volatile int *)&sm->abort = 1;
                    atomicOr(&a.st->err, 32);
                }
                break;
            }
        }
        __syncwarp();
    }
    // After an abort some entries expect activation bytes that were never requested: their barrier cannot complete, but the
    // weight copies still have to land before the CTA may exit.  A copy takes microseconds; wait a bounded moment.
    if (*(volatile int *)&sm->abort) {
        const unsigned long long t0 = gtime_ns();
        while (gtime_ns() - t0 < 200000ull) {
        }
    } else {
        for (int i = 0; i < R_NE; ++i) {
            if (used & (1u << i)) {
                const unsigned long long t0 = gtime_ns();
                while (!bar_try(&sm->full[i], (used_par >> i) & 1u))
                    if (gtime_ns() - t0 > sm->wait_ns) break;
            }
        }
    }
}

// The four multiply-adds of one 64-element k-block in one block of instructions (the issuing thread is the bottleneck
// when a CTA's tile has few rows: the tensor core needs about 46 cycles for a small tile, a thread that computes
// two descriptors and a predicate per instruction issues one in about 80).  Descriptors advance by 2 units of 16 bytes
// per 16 elements of K; `acc` = 0 makes the first one overwrite the accumulator.
__device__ __forceinline__ void umma_kblock(unsigned tmem_d, unsigned long long adesc, unsigned long long bdesc, unsigned idesc,
                                            unsigned acc) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
        "setp.ne.b32 p, %4, 0;\n\tsetp.eq.b32 q, 0, 0;\n\t"
        "add.u64 a1, %1, 2;\n\tadd.u64 a2, %1, 4;\n\tadd.u64 a3, %1, 6;\n\t"
        "add.u64 b1, %2, 2;\n\tadd.u64 b2, %2, 4;\n\tadd.u64 b3, %2, 6;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a1, b1, %3, q;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a2, b2, %3, q;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a3, b3, %3, q;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}

// ---- MMA issuer ------------------------------------------------------------------------------------------
__device__ void mma_issuer(const ClRowsArgs &a, unsigned char *ring, RSmem *sm, unsigned tmem) {
    Cursor c(a);
    unsigned n = 0;   // accumulation chains so far (buffer n & 1)
    const unsigned long long desc0 = umma_desc(0);
    const unsigned ars16 = (unsigned)c.ars * 8u;   // activation rows of a tile in 16-byte units
    const unsigned ring0 = s_u32(ring);
    while (!c.done) {
        const unsigned buf = n & 1u;
        if (c.chain_first() && !r_wait(&sm->tempty[buf], ((n >> 1) & 1u) ^ 1u, sm, &a.st->err)) return;
        if (!r_wait(&sm->full[c.e], c.par, sm, &a.st->err)) return;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned idesc = umma_idesc(128, c.npad, a.f16);
        const unsigned base = ring0 + c.poff;
        unsigned long long adesc = desc0 + (unsigned long long)((base & 0x3ffffu) >> 4);
        const unsigned stride16 = c.stride >> 4;
        const unsigned d_tmem = tmem + buf * 256u;
        unsigned acc = c.chain_first() ? 0u : 1u;
        for (int j = 0; j < c.kbs; ++j) {
            umma_kblock(d_tmem, adesc, adesc + ars16, idesc, acc);
            acc = 1u;
            adesc += stride16;
        }
        umma_commit(&sm->empty[c.e]);                      // the entry is free once these multiply-adds have read it
        if (c.chain_last()) {
            umma_commit(&sm->tfull[buf]);                  // ... and the accumulator buffer is complete
            ++n;
        }
        c.advance();
    }
}

// ---- GEMM jobs on the worker side: drain the accumulator, epilogue ------------------------------------------------
// Drain warp dw (0..3) takes the 32-column chunks dw and dw + 4 of the tile (N <= 224: seven chunks).  Lane m of the
// warp holds row m of D: lanes t < T the hi product of token t, lanes T + t its lo product.  The sums hi + lo of a
// finished tile go to a staging buffer in shared memory (to the workspace in global memory for an output / down
// projection, whose epilogue follows the group's barrier); then all worker warps apply the epilogue, whole warps per
// token row:
//   STORE  qkv[t, r] = s_t * acc                     (s_t = RMSNorm scale of token t)
//   SILU   rows interleave gate / up: h = silu(s_t g) * (s_t u) -> hi/lo(h), the down projection's operand
//   HEAD   logits = clamp(s_t * acc) -> running softmax statistics and argmax per token (Eq. 1-4)
struct Group {
    int g0, g1, a0, npad;
};

// All worker warps call this with the same cursor state.  `run` carries a thread's LM-head statistics across tiles.
__device__ __forceinline__ void gemm_job(const ClRowsArgs &a, RSmem *sm, unsigned tmem, int ji, Cursor &c, unsigned &n, ClHeadPartial &run) {
    if (c.done || c.ji != ji) return;   // this CTA has no part in the job
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool drains = (warp & 3) == 0;
    const int dw = warp >> 2;
    const int T = a.T, epi = c.epi, rows = c.rows;
    const int wpt = RW / T;                                  // warps per token row in the epilogue
    const int et = warp / wpt, ej = (warp % wpt) * 32 + lane, estride = wpt * 32;
    bool job_done = false;
    while (!job_done) {
        const Group g{c.g0, c.g1, c.a0, c.npad};
        // walk the tile's entries first (an accumulation chain ends after a.chain k-blocks and at the tile's end), so that
        // no schedule arithmetic runs while the accumulator registers are live
        int nchains = 0;
        for (bool group_end = false; !group_end;) {
            nchains += c.chain_last() ? 1 : 0;
            group_end = c.last();
            job_done = c.job_last();
            c.advance();
        }
        float acc[2][32];
        if (drains) {
#pragma unroll
            for (int q = 0; q < 2; ++q)
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[q][i] = 0.f;
            for (int ch = 0; ch < nchains; ++ch) {
                const unsigned buf = (n + ch) & 1u;
                const bool ok = r_wait(&sm->tfull[buf], ((n + ch) >> 1) & 1u, sm, &a.st->err);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (ok) {
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const int chunk = dw + 4 * q;
                        if (chunk * 32 < g.npad) {   // uniform over the warp
#pragma unroll
                            for (int hlf = 0; hlf < 2; ++hlf) {
                                float v[16];
                                tmem_ld16(tmem + buf * 256u + (unsigned)(chunk * 32 + hlf * 16), v);
#pragma unroll
                                for (int i = 0; i < 16; ++i) acc[q][hlf * 16 + i] += v[i];
                            }
                        }
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) bar_arrive(&sm->tempty[buf]);
            }
        }
        n += (unsigned)nchains;
        if (drains) {
            // hi + lo of every token; to the workspace (output / down projection) or to the staging buffer
            float *dst = (epi == CL_VEPI_RESID) ? a.ws + ((size_t)blockIdx.x * CL_MAX_T + lane) * R_MAXN : sm->stage + lane * R_STAGE_LD;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int chunk = dw + 4 * q;
                if (chunk * 32 < g.npad) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float lo = __shfl_down_sync(0xffffffffu, acc[q][i], T);   // all lanes take part
                        if (lane < T && chunk * 32 + i < g.npad) dst[chunk * 32 + i] = acc[q][i] + lo;
                    }
                }
            }
        }
        if (epi == CL_VEPI_RESID) continue;   // resid_phase() follows the job
        worker_sync();
        if (et < T) {
            const float sc = sm->scale[et];
            const float *st = sm->stage + et * R_STAGE_LD - g.a0;   // st[row] = raw product of (token et, weight row)
            if (epi == CL_VEPI_STORE) {
                for (int row = g.g0 + ej; row < g.g1; row += estride) a.qkv[(size_t)et * rows + row] = sc * st[row];
            } else if (epi == CL_VEPI_SILU) {   // rows interleave gate (even) and up (odd); g0 is even
                for (int row = g.g0 + 2 * ej; row < g.g1; row += 2 * estride) {
                    const float gt = sc * st[row], up = sc * st[row + 1];
                    a_store_split(a.Ah, et, T, row >> 1, gt / (1.f + expf(-gt)) * up, a.f16);
                }
                proxy_fence_global();   // these stores are read by other CTAs' bulk copies
            } else {
                for (int row = g.g0 + ej; row < g.g1; row += estride) {
                    const float lg = fminf(fmaxf(sc * st[row], -CL_LOGIT_CLAMP), CL_LOGIT_CLAMP);
                    if (a.logits) a.logits[(size_t)et * a.V + row] = lg;
                    run = rp_merge(run, ClHeadPartial{lg, 1.f, 0.f, row});
                }
            }
        }
        worker_sync();   // the staging buffer is free again; this tile's results are complete
        if (tid == 0) {
            if (epi == CL_VEPI_STORE) {          // rows of the QKV product, counted per head-sized block
                for (int b = g.g0 / a.hd; b * a.hd < g.g1; ++b)
                    counter_add(a.sync + a.c_qkv + b, (unsigned)(min(g.g1, (b + 1) * a.hd) - max(g.g0, b * a.hd)));
            } else if (epi == CL_VEPI_SILU) {    // columns of the FFN hidden operand rows, counted per k-block
                const int j0 = g.g0 >> 1, j1 = g.g1 >> 1;
                for (int kb = j0 >> 6; kb * 64 < j1; ++kb)
                    counter_add(a.sync + a.c_ah + kb, (unsigned)(min(j1, (kb + 1) * 64) - max(j0, kb * 64)));
            }
        }
    }
}

// End of the LM-head job: the statistics of a token row are spread over the threads of its warps; merge them in a
// fixed order (rows ascend with the lane inside a warp pass, so a tree over lanes then warps is a fixed order too).
__device__ void head_finish(const ClRowsArgs &a, RSmem *sm, ClHeadPartial run) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, wpt = RW / a.T;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const ClHeadPartial other = cl_hp_shfl_xor(run, o);
        run = ((lane & o) == 0) ? rp_merge(run, other) : rp_merge(other, run);
    }
    if (lane == 0) sm->hpw[warp] = run;
    worker_sync();
    if (tid < a.T) {
        ClHeadPartial r = sm->hpw[tid * wpt];
        for (int w = 1; w < wpt; ++w) r = rp_merge(r, sm->hpw[tid * wpt + w]);
        a.head_part[(size_t)blockIdx.x * CL_SLOTS + tid] = r;
    }
}

// Second half of an output / down projection: the `split` CTAs of a group hold the products of their K ranges in the
// workspace.  Nobody waits for anybody: each member takes a ticket of its group when its products are stored, and the
// member that draws the last one does the group's rows -- adds the parts in member order (fixed: results do not depend
// on who came last), residual add, the next GEMM's operand rows hi/lo(x * gain), hidden tap, sum of x^2 per token.
// Whole warps per token row (RW / T of them), a thread's rows 32 apart, so a row's sum of squares is a fixed tree.
__device__ void resid_phase(const ClRowsArgs &a, int ji, int pos0, RSmem *sm) {
    const int T = a.T, l = ji >> 2, g = a.split, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Job jb = job_of(a, ji);
    int r0, r1;
    rows_of(jb.rows, jb.unit, g, r0, r1);
    const int first_cta = (int)blockIdx.x - (int)blockIdx.x % g;
    worker_sync();   // the drain warps' stores to the workspace are done
    if (tid == 0) {
        int last = 1;
        if (g > 1) {
            const unsigned prev = ticket_acq_rel(a.sync + 1 + blockIdx.x / g);   // (counts up during a launch: g tickets per job)
            last = (prev % (unsigned)g) == (unsigned)g - 1u;
        }
        sm->is_last = last;
    }
    worker_sync();
    const bool mine = sm->is_last != 0;
    if (mine) {
        const ClRowsLayer &y = a.layers[l];
        const bool attn_half = (ji & 3) == 1;
        const float *gain = attn_half ? y.n2 : ((l + 1 < a.L) ? a.layers[l + 1].n1 : a.final_norm);
        unsigned short *tap = (unsigned short *)(a.tap ? (attn_half ? y.tap0 : y.tap1) : nullptr);
        const int wpt = RW / T, t = warp / wpt, a0 = r0 & ~7;   // (the group's rows are one tile of the GEMM)
        float ss = 0.f;
        if (t < T) {
            for (int row = r0 + (warp % wpt) * 32 + lane; row < r1; row += wpt * 32) {
                float parts[8];
#pragma unroll
                for (int m = 0; m < 8; ++m)
                    parts[m] = m < g ? __ldcg(a.ws + ((size_t)(first_cta + m) * CL_MAX_T + t) * R_MAXN + (row - a0)) : 0.f;
                float sum = parts[0];
#pragma unroll
                for (int m = 1; m < 8; ++m)
                    if (m < g) sum += parts[m];
                float *xp = a.x + (size_t)t * a.d + row;
                const float xn = __ldcg(xp) + sum;
                *xp = xn;
                a_store_split(a.Ax, t, T, row, xn * __ldg(gain + row), a.f16);
                if (tap && t + a.tap_P >= T)   // (slot = position mod P: of rows that share a slot the last one stays)
                    tap[(size_t)((pos0 + t) % a.tap_P) * a.d + row] = f32_to_b16(xn, a.f16);
                ss = fmaf(xn, xn, ss);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) sm->wsum[warp] = ss;
        proxy_fence_global();   // the operand rows written above are read by other CTAs' bulk copies
    }
    if (!mine) return;   // (uniform over the CTA)
    worker_sync();
    // the group's sum of squares goes to its first member's slot and zeros to the others', whoever computed it: the order
    // in which the slots are added up later must not depend on who came last
    if (tid < T) {
        const int wpt = RW / T;
        float ss = 0.f;
        for (int w = 0; w < wpt; ++w) ss += sm->wsum[tid * wpt + w];
        a.ssq[(size_t)first_cta * CL_SLOTS + tid] = ss;
        for (int m = 1; m < g; ++m) a.ssq[(size_t)(first_cta + m) * CL_SLOTS + tid] = 0.f;
    }
    worker_sync();
    if (tid == 0) {
        // the group's columns of the operand rows, counted per k-block; and the sums of squares of its g slots
        for (int kb = r0 >> 6; kb * 64 < r1; ++kb)
            counter_add(a.sync + a.c_ax + kb, (unsigned)(min(r1, (kb + 1) * 64) - max(r0, kb * 64)));
        counter_add(a.sync + a.c_ssq, (unsigned)g);
    }
}

// RMSNorm scale of every token row from the per-CTA sums of squares (fixed order: lane-strided, then a shuffle tree).
// The warps that do not drain the accumulator do this while the GEMM runs (token k <-> the k-th of them); the barrier
// in front of the epilogue, the first reader, orders it.
__device__ void compute_scales(const ClRowsArgs &a, RSmem *sm, int pass) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((warp & 3) == 0) return;
    const int t = warp - 1 - (warp >> 2);
    if (t < a.T) {
        if (lane == 0) counter_wait(a.sync + a.c_ssq, (unsigned)pass * gridDim.x, sm, &a.st->err);   // every CTA's sum is there
        __syncwarp();
        float ss = 0.f;
        for (int c = lane; c < (int)gridDim.x; c += 32) ss += __ldcg(a.ssq + (size_t)c * CL_SLOTS + t);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) sm->scale[t] = 1.0f / sqrtf(ss * a.inv_d + a.eps);
    }
}

// ---- embedding phase: x[t] = E[token t]; first operand hi/lo(x * g); per-CTA sums of squares ---------------------
__device__ void embed_phase(const ClRowsArgs &a, RSmem *sm) {
    const int T = a.T, nch = a.d >> 3, tid = threadIdx.x;
    const float *g = a.L ? a.layers[0].n1 : a.final_norm;
    const int per = (nch + gridDim.x - 1) / gridDim.x;   // chunks of 8 columns per CTA (at most 16)
    for (int idx = tid; idx < 16 * CL_SLOTS; idx += RT) sm->esum[idx / CL_SLOTS][idx % CL_SLOTS] = 0.f;
    worker_sync();
    for (int idx = tid; idx < per * T; idx += RT) {
        const int i = idx / T, t = idx % T, ch = (int)blockIdx.x + i * (int)gridDim.x;
        if (ch < nch) {
            const int tok = a.tok[t];
            const uint4 raw = *(const uint4 *)((const unsigned short *)a.embed + (size_t)tok * a.d + ch * 8);
            const unsigned u[4] = {raw.x, raw.y, raw.z, raw.w};
            float v[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) pair16_to_f32(u[e], a.f16, v[2 * e], v[2 * e + 1]);
            float4 *xp = (float4 *)(a.x + (size_t)t * a.d + ch * 8);
            xp[0] = make_float4(v[0], v[1], v[2], v[3]);
            xp[1] = make_float4(v[4], v[5], v[6], v[7]);
            float ss = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                ss = fmaf(v[e], v[e], ss);
                a_store_split(a.Ax, t, T, ch * 8 + e, v[e] * g[ch * 8 + e], a.f16);
            }
            sm->esum[i][t] = ss;
        }
    }
    proxy_fence_global();   // the operand rows written above are read by other CTAs' bulk copies
    worker_sync();
    if (tid < T) {
        float ss = 0.f;
        for (int i = 0; i < per; ++i) ss += sm->esum[i][tid];
        a.ssq[(size_t)blockIdx.x * CL_SLOTS + tid] = ss;
    }
    worker_sync();
    if (tid < per) {   // 8 operand columns per chunk, counted per k-block
        const int ch = (int)blockIdx.x + tid * (int)gridDim.x;
        if (ch < nch) counter_add(a.sync + a.c_ax + (ch >> 3), 8u);
    }
    if (tid == 0) counter_add(a.sync + a.c_ssq, 1u);
}

// ---- attention of the T rows over the cache ------------------------------------------------------------------
// Work item (head h, part s of the cached keys [0, base)) -> one CTA.  Inside the CTA warp w serves token row
// t = w / nsub and the sub-range sub = w % nsub of the part's keys (nsub = 14 / T warps per row).  A warp walks its
// keys 32 at a time with an online softmax (scores reduced with warp shuffles).  The rows' own keys and values
// (positions base .. base + t, causal) come raw from the QKV product: the CTA of the last part first rotates the
// keys, rounds keys and values to the storage type and keeps them in shared memory (one query head per key/value
// head also appends them to the cache); the last warp of row t folds them in.  The CTA merges its warps per row and writes one
// record per (h, s, t); the last CTA of a head to finish (ticket) merges the parts in order and writes the
// normalised output as the output projection's hi/lo operand rows.
// Ahead of a layer's QKV job: ask for the cached keys and values this CTA's attention item will read, so that they wait
// in L2 when the attention phase starts (the worker warps have nothing else to do while the job's weights stream).
template <int HD>
__device__ __forceinline__ void attention_prefetch(const ClRowsArgs &a, const ClRowsLayer &y, int base) {
    const int S = a.att_parts, item = blockIdx.x;
    if (item >= a.H * S) return;
    const int h = item % a.H, s = item / a.H, kvh = h / (a.H / a.Hkv);
    const int k0 = (int)((long long)base * s / S), k1 = (int)((long long)base * (s + 1) / S);
    const size_t off = ((size_t)kvh * a.max_seq + k0) * HD * 2, bytes = (size_t)(k1 - k0) * HD * 2;
    for (size_t b = (size_t)threadIdx.x * 128; b < bytes; b += (size_t)RT * 128) {
        asm volatile("prefetch.global.L2 [%0];" ::"l"(y.kc + off + b));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(y.vc + off + b));
    }
}

template <typename ST, int HD>
__device__ void attention_phase(const ClRowsArgs &a, const ClRowsLayer &y, int layer, int base, RSmem *sm) {
    constexpr int EPL = 8, LPK = HD / EPL, KPW = 32 / LPK, VPL = HD / 32, WSTRIDE = HD + 2, HALF = HD / 2;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int T = a.T, S = a.att_parts, nsub = RW / T;
    const int t = warp / nsub, sub = warp % nsub;
    const bool active = warp < T * nsub;
    const int li = lane % LPK, ksub = lane / LPK;
    const float scale = rsqrtf((float)HD);
    const int group = a.H / a.Hkv, kvd = a.Hkv * HD, ld = a.d + 2 * kvd;
    ST *Kc = (ST *)y.kc, *Vc = (ST *)y.vc;
    float *wrec = sm->stage;
    for (int item = blockIdx.x; item < a.H * S; item += gridDim.x) {
        const int h = item % a.H, s = item / a.H, kvh = h / group;
        // this head's q rows and its key/value head's k and v rows of the QKV product: complete? (three counters, one
        // lane each)
        if (warp == 0) {
            if (lane < 3) {
                const int b = lane == 0 ? h : (lane == 1 ? a.H + kvh : a.H + a.Hkv + kvh);
                counter_wait(a.sync + a.c_qkv + b, (unsigned)(HD * (layer + 1)), sm, &a.st->err);
            }
            __syncwarp();
        }
        phase_clock(a, sm, 7);
        worker_sync();
        if (s == S - 1) {
            // the pass's own keys and values, raw in the QKV product: rotate the keys, round both to the storage type, keep
            // them for the warps below (one query head per key/value head also appends them to the cache); one thread per
            // (row, pair of elements i, i + hd / 2), so the whole set costs one memory round trip
            const bool writer = (h % group) == 0;
            for (int idx = tid; idx < T * HALF; idx += RT) {
                const int jn = idx / HALF, i = idx % HALF;
                const float *kraw = a.qkv + (size_t)jn * ld + a.d + kvh * HD, *vraw = kraw + kvd;
                const float2 cs = a.rope_cs[(size_t)(base + jn) * HALF + i];
                const float ka = __ldcg(kraw + i), kb = __ldcg(kraw + i + HALF);
                const float va = __ldcg(vraw + i), vb = __ldcg(vraw + i + HALF);
                const unsigned short kk0 = f32_to_b16(ka * cs.x - kb * cs.y, a.f16), kk1 = f32_to_b16(kb * cs.x + ka * cs.y, a.f16);
                const unsigned short v0 = f32_to_b16(va, a.f16), v1 = f32_to_b16(vb, a.f16);
                sm->knew[jn * HD + i] = kk0; sm->knew[jn * HD + i + HALF] = kk1;
                sm->vnew[jn * HD + i] = v0; sm->vnew[jn * HD + i + HALF] = v1;
                if (writer) {
                    unsigned short *ck = (unsigned short *)Kc + ((size_t)kvh * a.max_seq + base + jn) * HD;
                    unsigned short *cv = (unsigned short *)Vc + ((size_t)kvh * a.max_seq + base + jn) * HD;
                    ck[i] = kk0; ck[i + HALF] = kk1; cv[i] = v0; cv[i + HALF] = v1;
                }
            }
            worker_sync();
        }
        float m_run = -INFINITY, l_run = 0.f, o_run[VPL];
#pragma unroll
        for (int e = 0; e < VPL; ++e) o_run[e] = 0.f;
        if (active) {
            const int pos = base + t;
            const float *qraw = a.qkv + (size_t)t * ld + h * HD;
            float qr[EPL];
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                const int idx = li * EPL + e;
                const int i = idx < HALF ? idx : idx - HALF;
                const float2 cs = a.rope_cs[(size_t)pos * HALF + i];
                const float qa = __ldcg(qraw + i), qb = __ldcg(qraw + i + HALF);
                qr[e] = idx < HALF ? qa * cs.x - qb * cs.y : qb * cs.x + qa * cs.y;
            }
            const int k0 = (int)((long long)base * s / S), k1 = (int)((long long)base * (s + 1) / S);
            const int kw0 = k0 + (int)((long long)(k1 - k0) * sub / nsub), kw1 = k0 + (int)((long long)(k1 - k0) * (sub + 1) / nsub);
            const ST *Kh = Kc + (size_t)kvh * a.max_seq * HD, *Vh = Vc + (size_t)kvh * a.max_seq * HD;
            // CH keys per iteration: the key rows and the value rows of the iteration are requested together (the values do
            // not depend on the scores), so an iteration costs one memory round trip; lane j < CH keeps key j's score
            constexpr int CH = 16, NPASS = CH / KPW;
            for (int j0 = kw0; j0 < kw1; j0 += CH) {
                const int n = min(CH, kw1 - j0);
                uint4 raw[NPASS];
#pragma unroll
                for (int p = 0; p < NPASS; ++p) {
                    const int j = p * KPW + ksub;
                    raw[p] = make_uint4(0u, 0u, 0u, 0u);
                    if (j < n) raw[p] = __ldg((const uint4 *)(Kh + (size_t)(j0 + j) * HD + li * EPL));
                }
                uint2 vraw[CH];   // the value rows stay in their storage type until they are used
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    const ST *vp = Vh + (size_t)(j0 + min(j, n - 1)) * HD + lane * VPL;
                    if (VPL == 4) vraw[j] = __ldg((const uint2 *)vp);
                    else vraw[j] = make_uint2(__ldg((const unsigned *)vp), 0u);
                }
                float my_score = -INFINITY;
#pragma unroll
                for (int p = 0; p < NPASS; ++p) {
                    const int jb = p * KPW;
                    if (jb < n) {   // uniform
                        const unsigned u[4] = {raw[p].x, raw[p].y, raw[p].z, raw[p].w};
                        float sc = 0.f;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float ka, kb;
                            ClPair16<ST>::get(u[e], ka, kb);
                            sc = fmaf(qr[2 * e], ka, sc);
                            sc = fmaf(qr[2 * e + 1], kb, sc);
                        }
#pragma unroll
                        for (int o = LPK >> 1; o > 0; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
                        sc *= scale;
#pragma unroll
                        for (int k = 0; k < KPW; ++k) {
                            const float v = __shfl_sync(0xffffffffu, sc, k * LPK);
                            if (lane == jb + k && jb + k < n) my_score = v;
                        }
                    }
                }
                float m_new = my_score;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m_new = fmaxf(m_new, __shfl_xor_sync(0xffffffffu, m_new, o));
                m_new = fmaxf(m_new, m_run);
                const float p = (lane < n) ? expf(my_score - m_new) : 0.f;
                const float resc = (l_run > 0.f) ? expf(m_run - m_new) : 0.f;
                float ps = p;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
                l_run = fmaf(l_run, resc, ps);
#pragma unroll
                for (int e = 0; e < VPL; ++e) o_run[e] *= resc;
                m_run = m_new;
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    const float pj = __shfl_sync(0xffffffffu, p, j);   // (0 for j >= n: the repeated last row adds nothing)
                    float v[4];
                    ClPair16<ST>::get(vraw[j].x, v[0], v[1]);
                    ClPair16<ST>::get(vraw[j].y, v[2], v[3]);
#pragma unroll
                    for (int e = 0; e < VPL; ++e) o_run[e] = fmaf(pj, v[e], o_run[e]);
                }
            }
            if (s == S - 1 && sub == nsub - 1) {
                // the pass's own positions base .. base + t
                for (int jn = 0; jn <= t; ++jn) {
                    float kf[EPL], vn[VPL];
                    const uint4 raw = *(const uint4 *)(sm->knew + jn * HD + li * EPL);
                    const unsigned u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) pair16_to_f32(u[e], a.f16, kf[2 * e], kf[2 * e + 1]);
#pragma unroll
                    for (int e = 0; e < VPL; ++e) vn[e] = b16_to_f32(sm->vnew[jn * HD + lane * VPL + e], a.f16);
                    float sc = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) sc = fmaf(qr[e], kf[e], sc);
#pragma unroll
                    for (int o = LPK >> 1; o > 0; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
                    sc = __shfl_sync(0xffffffffu, sc, 0) * scale;
                    const float m_new = fmaxf(m_run, sc);
                    const float resc = (l_run > 0.f) ? expf(m_run - m_new) : 0.f;
                    const float pn = expf(sc - m_new);
                    l_run = fmaf(l_run, resc, pn);
#pragma unroll
                    for (int e = 0; e < VPL; ++e) o_run[e] = fmaf(o_run[e], resc, pn * vn[e]);
                    m_run = m_new;
                }
            }
        }
        if (lane == 0) {
            wrec[warp * WSTRIDE] = m_run;
            wrec[warp * WSTRIDE + 1] = l_run;
        }
#pragma unroll
        for (int e = 0; e < VPL; ++e) wrec[warp * WSTRIDE + 2 + lane * VPL + e] = o_run[e];
        worker_sync();
        // merge the nsub warps of every row (fixed order); one record per (h, s, t), or the final output if S == 1
        float *part = a.att_part + ((size_t)h * R_ATT_MAXS + s) * CL_MAX_T * WSTRIDE;
        for (int i = tid; i < T * HD; i += RT) {
            const int tt = i / HD, e = i % HD;
            float M = -INFINITY;
            for (int w = 0; w < nsub; ++w) {
                const float *r = wrec + (tt * nsub + w) * WSTRIDE;
                if (r[1] > 0.f) M = fmaxf(M, r[0]);
            }
            float Ls = 0.f, O = 0.f;
            for (int w = 0; w < nsub; ++w) {
                const float *r = wrec + (tt * nsub + w) * WSTRIDE;
                if (r[1] > 0.f) {
                    const float f = expf(r[0] - M);
                    Ls = fmaf(r[1], f, Ls);
                    O = fmaf(r[2 + e], f, O);
                }
            }
            if (S == 1) {
                a_store_split(a.Aatt, tt, T, h * HD + e, O / Ls, a.f16);
            } else {
                float *rec = part + (size_t)tt * WSTRIDE;
                if (e == 0) { rec[0] = M; rec[1] = Ls; }
                rec[2 + e] = O;
            }
        }
        if (S > 1) {
            worker_sync();
            if (tid == 0) {
                const unsigned prev = ticket_acq_rel(a.att_tickets + h);
                const int last = prev == (unsigned)S - 1;
                if (last) a.att_tickets[h] = 0u;
                sm->is_last = last;
            }
            worker_sync();
            if (sm->is_last) {
                const float *p0 = a.att_part + (size_t)h * R_ATT_MAXS * CL_MAX_T * WSTRIDE;
                for (int i = tid; i < T * HD; i += RT) {
                    const int tt = i / HD, e = i % HD;
                    float pm[R_ATT_MAXS], pl[R_ATT_MAXS], po[R_ATT_MAXS];
#pragma unroll
                    for (int s2 = 0; s2 < R_ATT_MAXS; ++s2) {
                        const float *ps = p0 + ((size_t)min(s2, S - 1) * CL_MAX_T + tt) * WSTRIDE;
                        pm[s2] = __ldcg(ps);
                        pl[s2] = (s2 < S) ? __ldcg(ps + 1) : 0.f;
                        po[s2] = __ldcg(ps + 2 + e);
                    }
                    float M = -INFINITY;
#pragma unroll
                    for (int s2 = 0; s2 < R_ATT_MAXS; ++s2)
                        if (pl[s2] > 0.f) M = fmaxf(M, pm[s2]);
                    float Ls = 0.f, O = 0.f;
#pragma unroll
                    for (int s2 = 0; s2 < R_ATT_MAXS; ++s2) {   // part order
                        if (pl[s2] > 0.f) {
                            const float f = expf(pm[s2] - M);
                            Ls = fmaf(pl[s2], f, Ls);
                            O = fmaf(po[s2], f, O);
                        }
                    }
                    a_store_split(a.Aatt, tt, T, h * HD + e, O / Ls, a.f16);
                }
            }
        }
        // the CTA that wrote the head's operand rows says so (its stores are read by other CTAs' bulk copies)
        const bool wrote = S == 1 || sm->is_last;
        if (wrote) proxy_fence_global();
        worker_sync();
        if (wrote && tid == 0) counter_add(a.sync + a.c_att + h, 1u);
    }
}

// ---- the kernel ---------------------------------------------------------------------------------------------
template <typename ST, int HD>
__global__ void __launch_bounds__(R_THREADS, 1) k_rows_pass(const __grid_constant__ ClRowsArgs a) {
    if (a.st->done) return;   // written only between launches: uniform over the grid
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *ring = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    // the control block sits behind the ring: the M = 128 operand descriptor of the last tile reads up to 16 KB past
    // its activation rows, which must stay inside this CTA's shared memory
    RSmem *sm = (RSmem *)(ring + (size_t)R_RING);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < R_NE; ++i) {
            bar_init(&sm->full[i], 1);
            bar_init(&sm->empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            bar_init(&sm->tfull[i], 1);
            bar_init(&sm->tempty[i], 4);
        }
        sm->abort = 0;
        sm->wait_ns = a.wait_ns;
        for (int i = 0; i < 8; ++i) sm->ph_ns[i] = 0ull;
        sm->t_prev = gtime_ns();
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == RW + 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(s_u32(&sm->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem = *(volatile unsigned *)&sm->tmem_base;

    if (warp == RW) {
        producer(a, ring, sm, lane);
    } else if (warp == RW + 1) {
        if (lane == 0) mma_issuer(a, ring, sm, tmem);
    } else {
        const int base = a.st->ctx + a.row0;   // position of row 0
        unsigned bar_target = 0u, n_acc = 0u;
        ClHeadPartial run{0.f, 0.f, 0.f, 0x7fffffff};
        Cursor cur(a);
        embed_phase(a, sm);
        phase_clock(a, sm, 0);
        for (int l = 0; l < a.L; ++l) {
            const ClRowsLayer &y = a.layers[l];
            attention_prefetch<HD>(a, y, base);
            compute_scales(a, sm, 2 * l + 1);
            gemm_job(a, sm, tmem, 4 * l, cur, n_acc, run);
            phase_clock(a, sm, 1);
            attention_phase<ST, HD>(a, y, l, base, sm);
            phase_clock(a, sm, 2);
            gemm_job(a, sm, tmem, 4 * l + 1, cur, n_acc, run);
            resid_phase(a, 4 * l + 1, base, sm);
            phase_clock(a, sm, 3);
            compute_scales(a, sm, 2 * l + 2);
            gemm_job(a, sm, tmem, 4 * l + 2, cur, n_acc, run);
            phase_clock(a, sm, 4);
            gemm_job(a, sm, tmem, 4 * l + 3, cur, n_acc, run);
            resid_phase(a, 4 * l + 3, base, sm);
            phase_clock(a, sm, 5);
        }
        if (a.want_head) {
            compute_scales(a, sm, 2 * a.L + 1);
            gemm_job(a, sm, tmem, 4 * a.L, cur, n_acc, run);
            head_finish(a, sm, run);
            phase_clock(a, sm, 6);
            grid_barrier(a, bar_target, sm);
            // CTA 0 merges the per-CTA statistics of every token row (one warp per row, fixed order): Eq. 1-4
            if (blockIdx.x == 0 && warp < a.T) {
                ClHeadPartial p{0.f, 0.f, 0.f, 0x7fffffff};
                for (int c = lane; c < (int)gridDim.x; c += 32) {
                    const ClHeadPartial *src = a.head_part + (size_t)c * CL_SLOTS + warp;
                    ClHeadPartial q;
                    q.m = __ldcg(&src->m); q.z = __ldcg(&src->z); q.s = __ldcg(&src->s); q.idx = __ldcg(&src->idx);
                    p = rp_merge(p, q);
                }
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const ClHeadPartial other = cl_hp_shfl_xor(p, o);
                    p = ((lane & o) == 0) ? rp_merge(p, other) : rp_merge(other, p);
                }
                if (lane == 0) {
                    const float H = logf(p.z) - p.s / p.z;
                    if (a.out_tok) a.out_tok[warp] = min(max(p.idx, 0), a.V - 1);
                    if (a.out_pmax) a.out_pmax[warp] = 1.f / p.z;
                    if (a.out_conf) a.out_conf[warp] = 1.f - H * a.inv_log_v;
                }
            }
        }
    }
    if (a.phase_ns && tid == 0)
        for (int i = 0; i < 8; ++i) a.phase_ns[(size_t)blockIdx.x * 8 + i] = sm->ph_ns[i];
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == RW + 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

// ---- load-time re-layout: row-major [rows, K] -> the streaming order of this kernel: the row block of CTA 0, of
// CTA 1, ...; inside a block [K / 64][block rows][64] elements with the 16-byte pieces of a row's 128 bytes permuted
// by (piece ^ (row & 7)) -----------------------------------------------------------------------------------------
__global__ void k_tile_layout(const uint4 *src, uint4 *dst, int rows, int KB, int unit, int G) {
    const size_t total = (size_t)rows * KB * 8;
    const long long units = rows / unit;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i & 7);
        const size_t rk = i >> 3;
        const int kb = (int)(rk % KB);
        const int r = (int)(rk / KB);
        int owner = (int)min((long long)G - 1, ((long long)(r / unit) + 1) * G / units);
        int r0, r1;
        rows_of_cta(rows, unit, owner, G, r0, r1);
        while (r < r0) rows_of_cta(rows, unit, --owner, G, r0, r1);
        while (r >= r1) rows_of_cta(rows, unit, ++owner, G, r0, r1);
        dst[((size_t)r0 * KB + (size_t)kb * (r1 - r0) + (r - r0)) * 8 + (size_t)(c ^ (r & 7))] = src[i];
    }
}

}  // namespace

size_t cl_rows_smem_bytes() { return (size_t)R_RING + R_CTRL_BYTES + 1024; }

int cl_rows_att_part_floats(int H) { return H * R_ATT_MAXS * CL_MAX_T * (128 + 2); }

cudaError_t cl_launch_tile_layout(const void *src, void *dst, int rows, int K, int unit, int grid, cudaStream_t s) {
    k_tile_layout<<<1184, 256, 0, s>>>((const uint4 *)src, (uint4 *)dst, rows, K / 64, unit, grid);
    return cudaGetLastError();
}

cudaError_t cl_launch_rows_pass(int wdtype, int head_dim, const ClRowsArgs &a, int grid, cudaStream_t s) {
    static_assert(sizeof(RSmem) <= R_CTRL_BYTES, "control block must fit behind the ring");
    static_assert(R_STAGE_FLOATS >= CL_MAX_T * R_STAGE_LD && R_STAGE_FLOATS % 4 == 0, "staging buffer holds a tile of every token row");
    static_assert(R_STAGE_FLOATS >= RW * (128 + 2), "staging buffer holds the attention records");
    const void *fn = nullptr;
    if (wdtype == 1 && head_dim == 64) fn = (const void *)k_rows_pass<__nv_bfloat16, 64>;
    else if (wdtype == 1 && head_dim == 128) fn = (const void *)k_rows_pass<__nv_bfloat16, 128>;
    else if (wdtype == 2 && head_dim == 64) fn = (const void *)k_rows_pass<__half, 64>;
    else if (wdtype == 2 && head_dim == 128) fn = (const void *)k_rows_pass<__half, 128>;
    else return cudaErrorInvalidValue;
    const size_t smem = cl_rows_smem_bytes();
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    void *params[] = {(void *)&a};
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(R_THREADS), params, smem, s);
}
