// A list of M = 1 decode calls run by persistent launches (elutq_chain_plan / elutq_chain_run).
//
// A decode step is a fixed sequence of linears on one stream.  Launched one by one, every call pays its own
// chain of cross-SM hand-overs (kernel start, activation load, table build, K-split reduction, kernel end), during
// which HBM idles; for the 8B layer shapes that chain is several times longer than the time the call's bytes need.
// Here one grid (one 1024-thread CTA per SM, all resident) walks a run of consecutive calls: calls of G = 128 with
// any mix of bit-widths, or calls that share (q, G) for the other group sizes - normally the whole list is one launch;
// a list that mixes group sizes is cut into one launch per run.  Inside a CTA the warps are specialised (Appendix B's two phases run side by side):
//
//   * 4 builder warps, as two teams of two (team t: the table jobs of parity t, always in table buffer t), load the
//     activations of the CTA's next K chunk and fill the table buffers (fused 8-bit tables, 64 KiB each); before a
//     team builds a job it publishes a small record of it (first item,
//     row-block range, where the partial sums go, tag) in shared memory;
//   * 26 look-up warps follow those records: they stream the packed weights of the job (one warp per 16-row x
//     512-column item, registers refilled one item ahead as in lut_gemv.cu, also across job boundaries) and sum table
//     entries.  Buffers are handed over through shared-memory mbarriers ("full" / "free" per buffer, one arrival per
//     warp, waits suspended in hardware rather than spinning);
//   * K split: every partial sum is stored together with a tag (launch epoch and call number) in one 8-byte
//     word, all sums of a row block side by side ([row block][chunk][16 rows]).  The CTAs that share a row range take
//     its row blocks round robin; each of the CTA's 2 finisher warps brings a block's sums into shared memory with
//     one bulk copy (two copies in flight per warp, completion on an mbarrier), adds the chunks in ascending order -
//     bit-reproducible -, checks the tags, repeats the copy (bounded) while a tag is not this call's yet, writes Y
//     and reports the call's completion on a counter.  No fence, no ticket, no second kernel for the reduction: the
//     copy that finds the tags is the copy that brings the values.  (The last call of a launch that another
//     launch of the chain follows is reduced by that launch's finishers, so that the CTAs leave right after their
//     last look-up.)
//   * Ordering: the result is what the calls give when run one after another.  The plan records, from the buffer
//     addresses, which earlier calls a call really depends on (its X or Y overlaps their Y, or its Y their X);
//     before the builders read X they wait (bounded) for the completion counters of exactly those calls.  Calls
//     without such a dependency overlap freely, so the weight stream does not stop at call boundaries.
//
// Every wait is bounded; when one runs out the CTA raises the plan's status word, stops waiting for the rest of the
// launch (results are then undefined), waits (bounded) for its own bulk copies in flight and returns normally.
#include <cstring>
#include <map>
#include <mutex>
#include <vector>

#include "lut_core.cuh"

namespace elutq {

namespace {

constexpr unsigned kChainMagic = 0x4E494843u;
constexpr int kChainRegions = 6;              // scratch regions for the tagged partial sums, used round-robin: at least
constexpr int kChainRegionsMax = 12;          // this many, more (up to the maximum) while all of them fit kChainScratchBytes
constexpr size_t kChainScratchBytes = 12u << 20;
constexpr int kDescSlots = 4;
constexpr int kLookupWarps = 26;              // (22 or 18 look-up warps with 72 / 80 registers each measured slower)
constexpr int kBuilderWarps = 4;
constexpr int kTeamWarps = 2;                 // builder warps per team; team t builds table buffer t (the jobs of parity t)
constexpr int kBuilderTeams = kBuilderWarps / kTeamWarps;
constexpr int kFinisherWarps = 2;
constexpr int kChainThreads = (kLookupWarps + kBuilderWarps + kFinisherWarps) * 32;
constexpr int kTeamThreads = kTeamWarps * 32;
static_assert(kBuilderTeams == 2, "one builder team per table buffer");
constexpr int kFinisherThreads = kFinisherWarps * 32;
// shared memory: two table buffers, then per buffer 16 group sums, four mbarriers, flags, descriptor ring
constexpr int kOffGsum = 2 * kTableBytes;
constexpr int kOffBar = kOffGsum + 128;
constexpr int kOffShared = kOffBar + 32;
constexpr int kOffRecBar = kOffGsum + 192;                // one "record written" barrier per job record
constexpr int kSlotBytes = 144;                           // descriptor (128) + this CTA's share of the call (16)
constexpr int kOffWarpDesc = kOffGsum + 256;              // a descriptor ring per finisher warp and per builder warp
constexpr int kWarpRings = kFinisherWarps + kBuilderWarps;
constexpr int kOffJobRec = kOffWarpDesc + kWarpRings * kDescSlots * kSlotBytes;   // job records, written by the builders
constexpr int kJobRecs = 4;
static_assert(kOffShared + 32 <= kOffRecBar && kOffRecBar + kJobRecs * 8 <= kOffWarpDesc, "shared-memory layout");
// finisher warps: a ring of buffers per warp that bulk copies fill with the partial sums of one row block
constexpr int kFinSlots = 2;                  // copies in flight per finisher warp (measured, 8B step / 32-layer stack / a
                                              // chain of sixteen 8B gate_up layers: 1: 71.4 / 475 / 122 us, 2: 72.2 / 482 / 107 us,
                                              // 4: 75.6 / 494 us)
constexpr int kFinRingBytes = 8192;           // per warp: one buffer of 32 chunks per slot
constexpr int kOffFinBuf = (kOffJobRec + kJobRecs * 64 + 127) / 128 * 128;
constexpr int kOffFinBar = kOffFinBuf + kFinisherWarps * kFinRingBytes;
constexpr int kChainSmem = kOffFinBar + kFinisherWarps * kFinSlots * 8;
constexpr unsigned kCallTestNoSignal = 0x40000000u;   // test only: the call never reports completion
constexpr int kMaxRuns = 64;                  // launches per chain

struct ChainCtl {                             // first 256 bytes of a plan
    unsigned magic, n_calls, status, epoch;
    unsigned exit_ticket, grid, reserved0, reserved1;
    unsigned long long done_off, calls_off, parts_off, slots_off, region_bytes, total_bytes;
};

struct ChainCall {                            // 128 bytes
    const __half* X;
    const uint8_t* tiles;                     // packed + header
    void* Y;
    unsigned long long* slots;                // [n_rb][n_kc][16] tagged partial sums of this call's scratch region
    int N, K, n_rb, n_kc;
    int q, G;
    unsigned flags;
    int dep_first, dep_last;                  // earlier calls whose completion must precede reading X / writing Y
                                              // (dep_first > dep_last: none)
    int ranges, rb_q, rb_r, cpc;
    int groups, n_ctas;
    int guard_call;                           // call that used this scratch region last (-1: none): it must be complete
    unsigned done_target;                     // completion reports per launch: one per CTA (one per look-up warp of every
                                              // CTA when the call has no K split)
    int release;                              // 1: a later call of the plan waits for this one (see red_release_add)
    unsigned guard_target;                    // done_target of call guard_call
    int pad[5];
};
static_assert(sizeof(ChainCall) == 128, "descriptor size");
static_assert(sizeof(ChainCtl) <= 256, "control block size");

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void bar_team(int team) {      // named barriers 1 and 4: the warps of one builder team
    if (team == 0) asm volatile("bar.sync 1, %0;" ::"n"(kTeamThreads) : "memory");
    else asm volatile("bar.sync 4, %0;" ::"n"(kTeamThreads) : "memory");
}
__device__ __forceinline__ void bar_lookups() {           // named barrier 3: the look-up warps only
    asm volatile("bar.sync 3, %0;" ::"n"(kLookupWarps * 32) : "memory");
}
__device__ __forceinline__ void bar_finishers() {         // named barrier 2: the finisher warps only
    asm volatile("bar.sync 2, %0;" ::"n"(kFinisherThreads) : "memory");
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"((uint32_t)__cvta_generic_to_shared(bar)) : "memory");
}
// One bounded attempt: the thread is suspended by the hardware (it takes no issue slots from the other role's warps,
// unlike a spinning test) until the phase completes or about a microsecond has passed.
__device__ __forceinline__ bool mbar_try(uint64_t* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(parity), "r"(1000u) : "memory");
    return ok != 0;
}

struct ChainShared {
    volatile int abort;                       // a wait ran out: stop waiting
    unsigned epoch;
    volatile int headers_bad;                 // a blob of this launch no longer carries the header it was planned with
};
static_assert(sizeof(ChainShared) <= 32, "shared flags");

// What the look-up warps need to know of one table job (a call's K chunk on this CTA), written by the builders
// before they build the job's tables: the look-up warps follow these records and never touch a descriptor.
struct JobRec {                               // four 16-byte quarters, each read with one shared-memory load
    const uint8_t* tile0;                     // the job's first item (row block rb0 of chunk kc)
    int rb0, rb1;                             //   (a record with rb0 == rb1 has no items: the stop record)
    unsigned long long* out;                  // tagged partial sums of chunk kc (row block 0), or nullptr: no K split, store Y
    void* Y;
    unsigned* done;                           // completion counter of the call (used without a K split)
    int N;
    unsigned flags;
    unsigned tag;
    int last;                                 // bit 0: the call's last job on this CTA; bit 1: the call's report is a release;
                                              // bits 8 and up: the call's bit-width q
    int stop;                                 // bit 0: no more jobs in this launch; bits 8 and up: the look-up warp that
                                              // takes the job's first item
    int out_stride;                           // 64-bit words from one row block's partial sums to the next (16 n_kc)
};
static_assert(sizeof(JobRec) == 64, "job record size");


extern __shared__ __align__(1024) uint8_t chain_smem[];

__device__ __forceinline__ JobRec* job_rec(unsigned job) {
    return reinterpret_cast<JobRec*>(chain_smem + kOffJobRec) + (job & (kJobRecs - 1));
}

__device__ __forceinline__ ChainShared* chain_shared() { return reinterpret_cast<ChainShared*>(chain_smem + kOffShared); }
struct ChainSlot {                            // what a role keeps of a call in shared memory
    ChainCall d;
    int4 part;                                // this CTA's share: rb0, rb1, kc0, nseg | grp << 16
};
static_assert(sizeof(ChainSlot) == kSlotBytes, "slot size");
__device__ __forceinline__ ChainSlot* warp_slot(int fw, int c) {
    return reinterpret_cast<ChainSlot*>(chain_smem + kOffWarpDesc) + fw * kDescSlots + (c & (kDescSlots - 1));
}
// Copies descriptor c and this CTA's share of call c into a slot: nine 16-byte pieces, one per lane.
__device__ __forceinline__ void slot_fetch(ChainSlot* dst, const ChainCall* calls, const int4* parts, int grid, int c, int piece) {
    if (piece < 8) cp_async16(reinterpret_cast<uint8_t*>(dst) + piece * 16, reinterpret_cast<const uint8_t*>(calls + c) + piece * 16);
    else if (piece == 8) cp_async16(&dst->part, parts + (size_t)c * grid + blockIdx.x);
}
__device__ __forceinline__ uint64_t* bar_full(int b) { return reinterpret_cast<uint64_t*>(chain_smem + kOffBar) + b; }
__device__ __forceinline__ uint64_t* bar_free(int b) { return reinterpret_cast<uint64_t*>(chain_smem + kOffBar) + 2 + b; }
// "record of job j is written": one barrier per record slot (the builders are never more than two jobs ahead of the
// slowest look-up warp, so a slot's barrier cannot run a whole phase ahead of a waiter)
__device__ __forceinline__ uint64_t* bar_rec(unsigned job) {
    return reinterpret_cast<uint64_t*>(chain_smem + kOffRecBar) + (job & (kJobRecs - 1));
}

__device__ __forceinline__ void raise_abort(unsigned* status) {
    ChainShared* sh = chain_shared();
    if (!sh->abort) {
        sh->abort = 1;
        atomicExch(status, kStatusWaitExpired);
    }
}
// Bounded wait on a shared-memory barrier phase: at most limit / 64 suspended attempts of about a microsecond.
__device__ __forceinline__ void mbar_wait(uint64_t* bar, unsigned parity, unsigned limit, unsigned* status) {
    ChainShared* sh = chain_shared();
    for (unsigned i = 0; !mbar_try(bar, parity); ++i) {
        if (i >= (limit >> 6) + 16u || sh->abort) {
            raise_abort(status);
            return;
        }
    }
}
// Bounded poll: true once *p has reached `target` (wrap-safe comparison).
__device__ __forceinline__ bool wait_reached(const unsigned* p, unsigned target, unsigned limit) {
    for (unsigned i = 0; i < limit; ++i) {
        if ((int)(ld_acquire_u32(p) - target) >= 0) return true;
        if (i > 64) __nanosleep(64);
    }
    return false;
}

__device__ __forceinline__ void chain_store(void* Y, unsigned flags, size_t idx, float y) {
    if (flags & ELUTQ_FLAG_OUT_F32) {
        float* Yf = reinterpret_cast<float*>(Y);
        Yf[idx] = (flags & ELUTQ_FLAG_ACCUMULATE) ? __ldcg(Yf + idx) + y : y;
    } else {
        __half* Yh = reinterpret_cast<__half*>(Y);
        if (flags & ELUTQ_FLAG_ACCUMULATE) y += __half2float(__ldcg(reinterpret_cast<const __half*>(Yh) + idx));
        Yh[idx] = __float2half_rn(y);
    }
}

// Row range and chunk group of CTA `bid` in call d.
struct ChainPart {
    int rb0, rb1, kc0, nseg, grp;
};
__device__ __forceinline__ ChainPart chain_part(const ChainSlot* s) {
    ChainPart p;
    p.rb0 = s->part.x; p.rb1 = s->part.y; p.kc0 = s->part.z;
    p.nseg = s->part.w & 0xffff; p.grp = s->part.w >> 16;
    return p;
}

// Bulk copy global -> shared memory, completion counted in bytes on a shared-memory barrier (both addresses and
// the size are multiples of 16 bytes).
__device__ __forceinline__ void fin_copy(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(bar);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src), "r"(bytes), "r"(b) : "memory");
}
__device__ __forceinline__ uint64_t* fin_bar(int fw, int slot) {
    return reinterpret_cast<uint64_t*>(chain_smem + kOffFinBar) + fw * kFinSlots + slot;
}
// The completion report of a call nobody in the plan waits for: its count is only a permission (to reuse the
// call's scratch region) and the end of the launch makes the outputs visible, so the report need not hold its thread
// until the outputs have reached memory, which a release does (measured: 3 - 9 us on a sixteen-call chain of one 8B
// layer, since the finisher that reports cannot fetch the next call's sums meanwhile).
__device__ __forceinline__ void red_relaxed_add(unsigned* p, unsigned v) {
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v) {
    // one fire-and-forget instruction: the writes that happen before it (this thread's, and those of the threads it
    // has synchronised with at a barrier) are visible to whoever reads the new count with acquire semantics
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ bool mbar_test(uint64_t* bar, unsigned parity) {     // one look, no suspension
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(parity) : "memory");
    return ok != 0;
}

// K-split reduction of call d by one finisher warp.  The `groups` CTAs of a row range share its row blocks round
// robin (block rb0 + grp, rb0 + grp + groups, ...): the look-up warps produce the blocks of a range in ascending
// order, so every CTA's share becomes ready evenly over the call and its finishers keep pace with the look-ups.
// The CTA's blocks alternate between its finisher warps.  The partial sums of a row block lie together
// ([chunk][16 rows], 128 bytes per chunk), so one bulk copy brings a block's sums (in segments of 32 chunks, when
// there are more) into shared memory without holding a register.  The warp's D = kFinSlots ring slots work on D
// blocks independently (slot k on the warp's blocks k, k + D, ...): when a slot's copy has landed, lane l < 16 adds
// row l's sums in ascending chunk order and checks their tags; if one is not this call's yet, the same copy is issued
// again, otherwise the slot's next copy.  A load issued on an SM whose look-up warps keep ~60 KB of weight loads
// outstanding comes back only after thousands of cycles (measured: ~5000), so what the finishers need is polls in
// flight, not instructions: with per-thread polling loads (8 in flight per thread) the reduction of a call took as
// long as its look-ups on every shape with more than a few row blocks per CTA.  `phases` holds the barrier parities
// of the warp's slots across calls.  Bounded: `limit` sweeps over the ring without a complete copy end the launch
// with the wait-expired status.
// `first_issued`: the warp's first copies of this call (slot k: block k) are in flight already, see chain_reduce_ahead.
__device__ __noinline__ unsigned chain_reduce(const ChainCall* d, const ChainPart p, unsigned tag, unsigned limit,
                                              unsigned* status, int fw, int lane, unsigned phases, bool first_issued) {
    ChainShared* sh = chain_shared();
    const int n_kc = d->n_kc, N = d->N, groups = d->groups;
    constexpr int D = kFinSlots;                               // ring slots in use
    constexpr int seg_chunks = 32, buf_bytes = kFinRingBytes / D;
    const int nseg = (n_kc + seg_chunks - 1) / seg_chunks;
    const int first = p.rb0 + p.grp + fw * groups;             // this warp's first block
    const int nblk = first < p.rb1 ? (p.rb1 - first + kFinisherWarps * groups - 1) / (kFinisherWarps * groups) : 0;
    uint8_t* const ring = chain_smem + kOffFinBuf + fw * kFinRingBytes;
    unsigned pending = 0;                                      // ring slots with a copy in flight
    auto issue = [&](int slot, int j, int sg) {                // segment sg of the warp's block j
        const int rb = first + j * kFinisherWarps * groups;
        const int nch = min(seg_chunks, n_kc - sg * seg_chunks);
        if (lane == 0)
            fin_copy(ring + slot * buf_bytes, d->slots + ((size_t)rb * n_kc + (size_t)sg * seg_chunks) * kTileRows,
                     (unsigned)nch * kTileRows * 8, fin_bar(fw, slot));
        pending |= 1u << slot;
    };
    int blk[kFinSlots], seg[kFinSlots];
    float sums[kFinSlots];
#pragma unroll
    for (int k = 0; k < kFinSlots; ++k) {
        blk[k] = k < D ? k : nblk;                             // (slots beyond D stay idle)
        seg[k] = 0; sums[k] = 0.f;
    }
#pragma unroll
    for (int k = 0; k < kFinSlots; ++k) {
        if (blk[k] < nblk) {
            if (first_issued) pending |= 1u << k;
            else issue(k, blk[k], 0);
        }
    }
    int remaining = nblk;
    unsigned idle = 0;
    while (remaining > 0) {
        bool progress = false, accepted = false;               // a copy has landed; a landed copy was complete
#pragma unroll
        for (int k = 0; k < kFinSlots; ++k) {
            if (blk[k] >= nblk) continue;
            if (!__all_sync(0xffffffffu, mbar_test(fin_bar(fw, k), (phases >> k) & 1u))) continue;
            phases ^= 1u << k;
            pending &= ~(1u << k);
            progress = true;
            const int rb = first + blk[k] * kFinisherWarps * groups;
            const int nch = min(seg_chunks, n_kc - seg[k] * seg_chunks);
            const unsigned long long* buf = reinterpret_cast<const unsigned long long*>(ring + k * buf_bytes);
            bool ok = true;
            float part = 0.f;
            if (lane < kTileRows) {
                for (int c = 0; c < nch; ++c) {
                    const unsigned long long w = buf[c * kTileRows + lane];
                    ok = ok && (unsigned)(w >> 32) == tag;
                    part += __uint_as_float((unsigned)w);
                }
            }
            if (__all_sync(0xffffffffu, ok)) {                  // (also: every lane is done with the buffer)
                sums[k] = seg[k] == 0 ? part : sums[k] + part;
                if (seg[k] + 1 == nseg) {
                    const int row = rb * kTileRows + lane;
                    if (lane < kTileRows && row < N) chain_store(d->Y, d->flags, (size_t)row, sums[k]);
                    blk[k] += D;
                    seg[k] = 0;
                    remaining -= 1;
                } else {
                    seg[k] += 1;
                }
                accepted = true;
            }
            // the slot's next copy, or the same one again when some of its sums were not there yet
            if (blk[k] < nblk) issue(k, blk[k], seg[k]);
        }
        if (accepted) {
            idle = 0;
        } else {
            if (++idle > limit || sh->abort) {
                raise_abort(status);
                break;
            }
            if (!progress) {
                // nothing has landed: wait for one of the copies suspended by the hardware (about a microsecond at
                // most per attempt) instead of sweeping, which would take issue slots from the look-up warps
                const int k0 = __ffs(pending) - 1;
                mbar_try(fin_bar(fw, k0), (phases >> k0) & 1u);
            }
        }
    }
    // a warp that gives up still waits (bounded, without looking at the abort flag) for its copies in flight: the
    // shared memory they write to must not be handed to another CTA before they have landed
#pragma unroll
    for (int k = 0; k < kFinSlots; ++k) {
        if (pending & (1u << k)) {
            bool landed = false;
            for (int tries = 0; tries < 4096 && !landed; ++tries) landed = mbar_try(fin_bar(fw, k), (phases >> k) & 1u);
            phases ^= 1u << k;
        }
    }
    return phases;
}

// The warp's first copies of a call, issued before the call before it is reported complete: the report is a release
// (it holds the reporting thread until the call's outputs have reached memory), and with the next call's first copies
// already under way that round trip and theirs overlap instead of following one another (measured with the release
// taken out: 3 - 9 us on a sixteen-call chain of one 8B layer).  All of the warp's ring slots are free at that point.
__device__ __forceinline__ void chain_reduce_ahead(const ChainCall* d, const ChainPart p, int fw, int lane) {
    const int n_kc = d->n_kc, groups = d->groups;
    constexpr int buf_bytes = kFinRingBytes / kFinSlots;
    const int first = p.rb0 + p.grp + fw * groups;
    const int nblk = first < p.rb1 ? (p.rb1 - first + kFinisherWarps * groups - 1) / (kFinisherWarps * groups) : 0;
    uint8_t* const ring = chain_smem + kOffFinBuf + fw * kFinRingBytes;
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < kFinSlots; ++k) {
            if (k < nblk) {
                const int rb = first + k * kFinisherWarps * groups;
                fin_copy(ring + k * buf_bytes, d->slots + (size_t)rb * n_kc * kTileRows, (unsigned)min(32, n_kc) * kTileRows * 8,
                         fin_bar(fw, k));
            }
        }
    }
}

// The lane's 16 activations of chunk kc (two byte-columns), as (x_i of column 2*lane, x_i of column 2*lane+1).
__device__ __forceinline__ void load_x_pairs(float2 (&x)[8], const __half* __restrict__ X, int kc, int K, int lane) {
    const int k0 = kc * kChunkK + lane * 16;
    if (k0 < K) {
        const uint4 r0 = __ldcg(reinterpret_cast<const uint4*>(X + k0));      // past the incoherent L1: X may have
        const uint4 r1 = __ldcg(reinterpret_cast<const uint4*>(X + k0 + 8));  // been written during this launch
        const uint32_t a[4] = {r0.x, r0.y, r0.z, r0.w}, b[4] = {r1.x, r1.y, r1.z, r1.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 fa = __half22float2(*reinterpret_cast<const __half2*>(&a[i]));
            const float2 fb = __half22float2(*reinterpret_cast<const __half2*>(&b[i]));
            x[2 * i] = make_float2(fa.x, fb.x);
            x[2 * i + 1] = make_float2(fa.y, fb.y);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = make_float2(0.f, 0.f);
    }
}
// Fused tables of a chunk (and its group sums) built by the builder warps from the activations x: lane -> column
// pair (2*lane, 2*lane+1) as in build_tables; builder warp bw takes the (high nibble, low-nibble half) combinations
// vw = bw, bw + 4, ... of the 32 that a full CTA would spread over its warps.
template <int G>
__device__ __forceinline__ void build_tables_bw(uint8_t* tab, float* gsum, const float2 (&x)[8], int bw, int lane) {
    constexpr int W = G / 8;
#pragma unroll
    for (int lh = 0; lh < 2; ++lh) {
        float2 A[8];
        A[0] = lh ? x[3] : make_float2(0.f, 0.f);
        A[1] = fadd2(A[0], x[0]);
        A[2] = fadd2(A[0], x[1]);
        A[3] = fadd2(A[1], x[1]);
        A[4] = fadd2(A[0], x[2]);
        A[5] = fadd2(A[1], x[2]);
        A[6] = fadd2(A[2], x[2]);
        A[7] = fadd2(A[3], x[2]);
#pragma unroll
        for (int s = 0; s < 16 / kTeamWarps; ++s) {
            const int hi = bw + s * kTeamWarps;
            float2 Bv = make_float2(0.f, 0.f);
#pragma unroll
            for (int b = 0; b < 4; ++b)
                if ((hi >> b) & 1) Bv = fadd2(Bv, x[4 + b]);
            float2* row = reinterpret_cast<float2*>(tab) + (size_t)(hi * 16 + lh * 8) * 32 + lane;
#pragma unroll
            for (int t = 0; t < 8; ++t) row[t * 32] = fadd2(A[t], Bv);
            if (lh == 1 && hi == 15) {          // entry 255 = sum of the column's 8 activations -> group sums
                const float2 e = fadd2(A[7], Bv);
                float total = e.x + e.y;
#pragma unroll
                for (int off = W / 4; off >= 1; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
                if ((lane % (W / 2)) == 0) gsum[lane / (W / 2)] = total;
            }
        }
    }
}

// Items of one job on one look-up warp; tables in buffer B.  `buf` holds the warp's first item of the job on entry.
// At its last item of the job the warp looks for the record of the next job (the builders publish it before they
// build that job's tables, normally a whole job ahead): if it is there and gives the warp an item, that item's loads
// ride along with the last item and `buf` holds it on exit (returns true).
// Items are dealt to the look-up warps round robin ACROSS jobs: a job's first item goes to the warp after the one
// that took the last item of the job before (`first`, from the job's record), so that short jobs (fewer items than
// warps: the small layers) alternate between warps, and the latency of a warp's item runs beside the next job's
// instead of in front of it.  The warp's place in a job whose first item goes to warp `first`:
__device__ __forceinline__ int item_slot(int warp, int first) {
    const int s = warp - first;
    return s < 0 ? s + kLookupWarps : s;
}

// Q = 0: the bit-width is the job's (q, from its record; G = 128), and the next job's may differ.
template <int Q, int G>
struct ItemOf { using type = Item<Q, G>; };
template <int G>
struct ItemOf<0, G> { using type = ItemRt; };

template <int Q, int G>
__device__ __forceinline__ int chain_tile_bytes(int q) { return Q ? Cfg<Q ? Q : 1, G>::TILE_BYTES : tile_bytes_g128(q); }

// QC: the job's bit-width as a compile-time value (= Q for a kernel of one bit-width; for Q = 0, the run-time-q kernel,
// the caller switches on the job's q, and only an item whose successor belongs to a job of another q takes a form
// with conditional loads).
template <int Q, int QC, int G, int B>
__device__ __forceinline__ bool chain_items(typename ItemOf<Q, G>::type& buf, const uint32_t (&colp)[4], const int rb0, const int rb1,
                                            unsigned long long* out, void* Y, const int N, const unsigned flags,
                                            const unsigned tag, const int out_stride, const uint8_t* vp, const unsigned job,
                                            const size_t warp_off, const int lw, const int lane, const int b_rt, const int wp) {
    using C = Cfg<QC, G>;
    const int bb = B < 0 ? b_rt : B;
    const uint8_t* const tab = chain_smem + bb * kTableBytes;
    const float* gsum = reinterpret_cast<const float*>(chain_smem + kOffGsum + bb * 64);
    const int h = lane >> 4, l = lane & 15;
    float S[C::GL];
    load_group_sums<G>(S, gsum, h, l, true);
    const unsigned long long tag_hi = (unsigned long long)tag << 32;
    bool carried = false;
    for (int rb = rb0 + lw; rb < rb1; rb += kLookupWarps) {
        const bool in_job = rb + kLookupWarps < rb1;
        const uint8_t* nvp = vp + kLookupWarps * C::TILE_BYTES;
        int nq = QC;
        if (!in_job && __all_sync(0xffffffffu, mbar_test(bar_rec(job + 1), ((job + 1) >> 2) & 1u))) {
            const uint4 n0 = *reinterpret_cast<const uint4*>(job_rec(job + 1));
            const int nlw = item_slot(wp, job_rec(job + 1)->stop >> 8);      // the warp's place in the next job
            if ((int)n0.z + nlw < (int)n0.w) {
                const size_t noff = (size_t)nlw * C::TILE_BYTES + lane * 16;
                if constexpr (Q == 0) nq = job_rec(job + 1)->last >> 8;
                if (nq == QC) {               // (a job of another q: its first item is requested when the job begins)
                    nvp = reinterpret_cast<const uint8_t*>(((unsigned long long)n0.y << 32) | n0.x) + noff;
                    carried = true;
                }
            }
        }
        float y;
        if constexpr (Q == 0) {
            y = item_sum_rt<QC>(buf, tab, colp, S, nvp, (in_job || carried) ? 1u : 0u, lane);
        } else {
            const uint8_t* npp = nvp + (C::PLANE_BYTES - lane * 12);
            if (in_job || carried) y = item_sum<Q, G, kModeFused, true>(buf, tab, colp, S, nvp, npp, true, true);
            else y = item_sum<Q, G, kModeFused, false>(buf, tab, colp, S, nvp, npp, true, true);
        }
        if (h == 0) {
            if (out == nullptr) {
                if (rb * kTileRows + l < N) chain_store(Y, flags, (size_t)(rb * kTileRows + l), y);
            } else {
                st_relaxed_u64(out + (size_t)rb * out_stride + l, tag_hi | __float_as_uint(y));
            }
        }
        vp = nvp;
    }
    return carried;
}

// the job's items, tables in buffer b
template <int Q, int QC, int G>
__device__ __forceinline__ bool chain_items_b(int b, typename ItemOf<Q, G>::type& buf, const uint32_t (&colp)[4], const int rb0,
                                              const int rb1, unsigned long long* out, void* Y, const int N, const unsigned flags,
                                              const unsigned tag, const int out_stride, const uint8_t* vp, const unsigned job,
                                              const size_t warp_off, const int lw, const int lane, const int wp) {
    if (b == 0) return chain_items<Q, QC, G, 0>(buf, colp, rb0, rb1, out, Y, N, flags, tag, out_stride, vp, job, warp_off, lw, lane, 0, wp);
    return chain_items<Q, QC, G, 1>(buf, colp, rb0, rb1, out, Y, N, flags, tag, out_stride, vp, job, warp_off, lw, lane, 1, wp);
}

// What the roles of a launch share.
struct ChainCtx {
    const ChainCall* calls;
    const int4* parts;
    unsigned* done;
    unsigned* status;
    int grid, n_calls, c_begin, c_end;
    unsigned epoch, spin_limit;
};

// Per-warp descriptor copies for the warps that walk the calls on their own (builder and finisher warps): a ring of
// four slots, filled by asynchronous copies two calls ahead, one copy group per call.  Taking call c waits only for
// the groups before the newest one, so the copy of call c + 1 may still be in flight: a walk that waited for it too
// was bound by one global round trip per call (0.9 us, measured on a chain of small calls with everything else off).
__device__ __forceinline__ void desc_fetch(const ChainCtx& x, int slot_warp, int c, int lane) {
    if (lane < 9) {
        if (c < x.c_end) slot_fetch(warp_slot(slot_warp, c), x.calls, x.parts, x.grid, c, lane);
        asm volatile("cp.async.commit_group;" ::: "memory");      // (an empty group past the end keeps the count)
    }
}
__device__ __forceinline__ void desc_begin(const ChainCtx& x, int slot_warp, int c0, int lane) {
    desc_fetch(x, slot_warp, c0, lane);
    desc_fetch(x, slot_warp, c0 + 1, lane);
}
// descriptor of call c for this warp; call c + 1 is on its way or there, call c + 2 is requested
__device__ __forceinline__ const ChainSlot* desc_next(const ChainCtx& x, int slot_warp, int c, int lane) {
    if (lane < 9) asm volatile("cp.async.wait_group 1;" ::: "memory");     // everything but the newest group: call c is there
    __syncwarp();                                 // ... and nobody still reads the slot of call c - 2
    desc_fetch(x, slot_warp, c + 2, lane);
    return warp_slot(slot_warp, c);
}

// Look-up role of one warp: it follows the job records the builders publish.  Q = 0 is the kernel for lists that mix
// bit-widths (G = 128): one register buffer sized for q = 4, and per job a switch to the straight-line code for the
// job's q.  What made that form as fast as a kernel of one q (earlier forms were 1.2 to 3 times slower): the buffer
// is shared by the per-q bodies instead of one buffer type per q (those spilled 0.3-1.5 KB per thread); a body per q
// and table buffer but none per "has a next item" (a predicate on the refill loads instead); the table buffer a
// compile-time constant (a run-time base costs an add per look-up); the unused part of the buffer given a value
// after every job.
template <int Q, int G>
__device__ __forceinline__ void lookup_jobs(const ChainCtx& x) {
    const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    const int h = lane >> 4, l = lane & 15;
    ChainShared* sh = chain_shared();
    uint32_t colp[4];
    make_colp<G>(colp, h, l);
    typename ItemOf<Q, G>::type buf;
    bool carried = false;                     // buf already holds this warp's first item of the job
    for (unsigned job = 0;; ++job) {
        const int b = job & 1;
        // The job's record comes before its tables: the warp requests its first item of the job (unless the item came
        // along with the job before) and only then waits for the tables, so the two latencies overlap.
        mbar_wait(bar_rec(job), (job >> 2) & 1, x.spin_limit, x.status);
        if (sh->abort) break;
        // the record in four loads (one round of shared-memory latency instead of a dependent chain of them)
        const uint4* rq = reinterpret_cast<const uint4*>(job_rec(job));
        const uint4 q0 = rq[0], q1 = rq[1], q2 = rq[2], q3 = rq[3];
        if (q3.z & 1u) break;                                     // stop record
        const int lw = item_slot(wp, (int)(q3.z >> 8));           // this warp's items of the job: lw, lw + 26, ...
        const uint8_t* tile0 = reinterpret_cast<const uint8_t*>(((unsigned long long)q0.y << 32) | q0.x);
        const int rb0 = (int)q0.z, rb1 = (int)q0.w;
        unsigned long long* out = reinterpret_cast<unsigned long long*>(((unsigned long long)q1.y << 32) | q1.x);
        void* Y = reinterpret_cast<void*>(((unsigned long long)q1.w << 32) | q1.z);
        unsigned* done_c = reinterpret_cast<unsigned*>(((unsigned long long)q2.y << 32) | q2.x);
        const int N = (int)q2.z;
        const unsigned flags = q2.w, tag = q3.x;
        const int out_stride = (int)q3.w;
        // (for Q = 0 everything from here on exists once per bit-width, behind a switch on the job's q)
        auto run_job = [&](auto qc) -> bool {
            constexpr int QC = decltype(qc)::value;
            using C = Cfg<QC, G>;
            const size_t warp_off = (size_t)lw * C::TILE_BYTES + lane * 16;
            const uint8_t* vp = tile0 + warp_off;
            if (rb0 + lw < rb1 && !carried) {
                if constexpr (Q == 0) load_item_rt<QC>(buf, vp, lane);
                else load_item<Q, G>(buf, vp, vp + (C::PLANE_BYTES - lane * 12), true);
            }
            mbar_wait(bar_full(b), (job >> 1) & 1, x.spin_limit, x.status);
            if (sh->abort) return false;
            carried = chain_items_b<Q, QC, G>(b, buf, colp, rb0, rb1, out, Y, N, flags, tag, out_stride, vp, job, warp_off, lw, lane, wp);
            if constexpr (Q == 0) {
                // the part of the buffer that items of this q do not use: given a value here, it is known not to carry one
                // through the job, which leaves its registers to the look-ups (without this the bodies for q < 4 ran 8 %
                // slower than a kernel of that q alone)
                static_for<QC, 4>([&](auto j) { buf.v[0][j] = make_uint4(0u, 0u, 0u, 0u); buf.v[1][j] = make_uint4(0u, 0u, 0u, 0u); });
                static_for<QC + 1, 5>([&](auto i) { buf.p[i] = 0u; });
            }
            return true;
        };
        bool went;
        if constexpr (Q == 0) {
            switch (q3.y >> 8) {
                case 1: went = run_job(IntC<1>{}); break;
                case 2: went = run_job(IntC<2>{}); break;
                case 3: went = run_job(IntC<3>{}); break;
                default: went = run_job(IntC<4>{}); break;
            }
        } else {
            went = run_job(IntC<Q>{});
        }
        if (!went) break;
        const bool report = out == nullptr && (q3.y & 1u) != 0u && !(flags & kCallTestNoSignal);
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(bar_free(b));         // this warp no longer reads buffer b (nor the job's record)
            if (report) {                     // no K split: this warp stored its rows of Y itself and reports them
                if (q3.y & 2u) red_release_add(done_c, 1u);
                else red_relaxed_add(done_c, 1u);
            }
        }
    }
}

// Calls [c_begin, c_end) of the plan, all with the kernel's (Q, G).
template <int Q, int G>
__global__ void __launch_bounds__(kChainThreads, 1)
lut_chain_kernel(ChainCtl* ctl, const ChainCall* calls, const int4* parts, unsigned* done, const int n_calls,
                 const int c_begin, const int c_end, const int first_run, const int last_run, const unsigned spin_limit) {
    uint8_t* const smem = chain_smem;
    ChainShared* sh = chain_shared();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // The launches of a chain follow one another by programmatic dependent launch: a CTA of the next launch starts
    // on an SM as soon as this launch's CTA there has left (every launch fills the device, one CTA per SM).  Only the
    // chain's first launch waits for whatever precedes the chain in the stream (and for the previous run of this plan,
    // which advances the epoch at its very end); it releases its successor after that wait, so the guarantee carries
    // over.  Data dependencies between calls of different launches go through the completion counters like those
    // inside a launch.
    if (first_run) grid_dependency_wait();
    grid_launch_dependents();

    // The plan is the one the host launched (its parts are addressed through kernel arguments: no pointer is
    // chased through the control block on the way to the first descriptor).
    const int grid = (int)gridDim.x;
    if (warp >= kLookupWarps && warp < kLookupWarps + kBuilderWarps && lane < 9) {
        // every builder warp keeps its own copies of the descriptors it works through (no barrier between the teams)
        const int ring = kFinisherWarps + (warp - kLookupWarps);
        if (c_begin < c_end) slot_fetch(warp_slot(ring, c_begin), calls, parts, grid, c_begin, lane);
        if (c_begin + 1 < c_end) slot_fetch(warp_slot(ring, c_begin + 1), calls, parts, grid, c_begin + 1, lane);
    }
    // Header check, first part: the look-up threads 64, 65, ... read the header of one call's blob each.  The loads
    // are issued here and looked at after the barrier below, so that they are on their way while the descriptors
    // arrive (the check needs a call's descriptor first: two loads behind one another).
    constexpr int kHdrFirst = 64, kHdrThreads = kLookupWarps * 32 - kHdrFirst;
    uint4 hdr0 = make_uint4(0, 0, 0, 0);
    uint2 hdr1 = make_uint2(0, 0);
    int hdr_q = 0, hdr_g = 0, hdr_n = 0, hdr_k = 0;
    const bool hdr_mine = tid >= kHdrFirst && tid < kLookupWarps * 32 && c_begin + (tid - kHdrFirst) < c_end;
    if (hdr_mine) {
        const ChainCall* d = calls + c_begin + (tid - kHdrFirst);
        hdr_q = d->q; hdr_g = d->G; hdr_n = d->N; hdr_k = d->K;
        blob_header_load(d->tiles, hdr0, hdr1);
    }
    unsigned epoch_now = 0;
    int bad = 0;
    if (tid == 0) {
        bad = (ctl->magic != kChainMagic || ctl->n_calls != (unsigned)n_calls) ? 1 : 0;
        epoch_now = ctl->epoch;
        sh->abort = 0;
        sh->headers_bad = 0;
        sh->epoch = epoch_now;
        // one arrival per warp (its lane 0, after the warp has converged): 32 arrivals of a warp on one barrier word
        // would be 32 serialised shared-memory atomics
        mbar_init(bar_full(0), kTeamWarps);
        mbar_init(bar_full(1), kTeamWarps);
        mbar_init(bar_free(0), kLookupWarps);
        mbar_init(bar_free(1), kLookupWarps);
        for (int j = 0; j < kJobRecs; ++j) mbar_init(bar_rec(j), 1);
        for (int j = 0; j < kFinisherWarps * kFinSlots; ++j) mbar_init(fin_bar(0, j), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    cp_async_wait_all();
    if (__syncthreads_or(bad)) {
        if (tid == 0) atomicExch(&ctl->status, kStatusBlobMismatch);
        return;                               // the same for every CTA: nobody is left waiting
    }
    const unsigned epoch = sh->epoch;
    unsigned* const status = &ctl->status;
    if (tid == 0 && last_run) {
        // The CTA of the chain's last launch that starts last opens the next epoch (completion counters and tags keep
        // counting up across launches of a plan, so nothing has to be cleared).  Every CTA of this launch has read the
        // epoch before it takes its ticket, and when all of them have started every CTA of the launches before has
        // left; the next run of the plan reads the epoch only after this launch has completed (stream order).
        const unsigned t = atomicInc(&ctl->exit_ticket, gridDim.x - 1);
        if (t == gridDim.x - 1) ctl->epoch = epoch + 1u;
    }

    ChainCtx x;
    x.calls = calls; x.parts = parts; x.done = done; x.status = status;
    x.grid = grid; x.n_calls = n_calls; x.c_begin = c_begin; x.c_end = c_end;
    x.epoch = epoch; x.spin_limit = spin_limit;

    if (warp < kLookupWarps) {
        // ---------------------------------------------------------------- look-up warps
        // Before any tile is read: every blob of this launch still carries the header it was planned with.  Only
        // the look-up warps read tiles, so only they wait for the headers; the builders fetch activations and build
        // the first tables meanwhile.
        {
            int hdr_bad = 0;
            if (hdr_mine && ((Q ? hdr_q != Q : (hdr_q < 1 || hdr_q > 4)) || hdr_g != G || !blob_header_ok(hdr0, hdr1, hdr_q, G, hdr_n, hdr_k))) hdr_bad = 1;
            for (int c = c_begin + kHdrThreads + tid; c < c_end; c += kLookupWarps * 32) {      // launches of more calls
                const ChainCall* d = calls + c;
                if ((Q ? d->q != Q : (d->q < 1 || d->q > 4)) || d->G != G || !blob_header_matches(d->tiles, d->q, G, d->N, d->K, nullptr)) hdr_bad = 1;
            }
            if (hdr_bad) sh->headers_bad = 1;
            bar_lookups();
            if (sh->headers_bad) {
                if (tid == 0) {
                    sh->abort = 1;            // the other roles' waits end at their next look at this flag
                    atomicExch(status, kStatusBlobMismatch);
                }
            } else {
                lookup_jobs<Q, G>(x);
            }
        }
    } else if (warp < kLookupWarps + kBuilderWarps) {
        // ---------------------------------------------------------------- builder warps
        // Two teams of two warps; team t builds the jobs of parity t, always into table buffer t, so the per-call
        // latencies of one team's job (descriptor, activation load, record, waits, hand-over) run beside the other
        // team's.  Both teams walk every call to count the jobs; a team works on the segments of its parity.
        const int bw = warp - kLookupWarps, team = bw / kTeamWarps, tw = bw % kTeamWarps;
        const bool lead = tw == 0 && lane == 0;               // the team's thread for records, waits on counters
        const int ring = kFinisherWarps + bw;
        const int b = team;
        unsigned job = 0;                                     // jobs of this CTA before the current call
        unsigned items = 0;                                   // ... and their items, modulo the look-up warps
        for (int c = c_begin; c < c_end; ++c) {
            const ChainSlot* sl = desc_next(x, ring, c, lane);
            const ChainCall* d = &sl->d;
            const ChainPart p = chain_part(sl);
            const int nseg = p.nseg;                          // 0: this CTA has no share of the call
            const int seg0 = ((job & 1u) == (unsigned)team) ? 0 : 1;      // this team's first segment of the call
            if (seg0 < nseg) {
                if (d->dep_first <= d->dep_last) {
                    // as-if-sequential order: every earlier call whose output this call reads or overwrites (or whose
                    // input it overwrites) is complete
                    if (lead && !sh->abort) {
                        bool ok = true;
                        for (int j = d->dep_first; ok && j <= d->dep_last; ++j)
                            ok = wait_reached(done + j, (epoch + 1u) * calls[j].done_target, spin_limit);
                        if (!ok) raise_abort(status);
                    }
                    bar_team(team);
                }
                for (int seg = seg0; seg < nseg; seg += kBuilderTeams) {
                    const unsigned j = job + (unsigned)seg;
                    float2 xv[8];             // requested before the wait for the buffer: the load latency overlaps it
                    load_x_pairs(xv, d->X, p.kc0 + seg, d->K, lane);
                    if (lead) {
                        // the job's record, published before the tables are built: the look-up warps may already request
                        // their first item of this job while they work on the one before (the record's slot was last
                        // read four jobs ago)
                        JobRec* r = job_rec(j);
                        const int kc = p.kc0 + seg;
                        r->tile0 = d->tiles + ((size_t)kc * d->n_rb + p.rb0) * chain_tile_bytes<Q, G>(d->q);
                        r->out = d->n_kc > 1 ? d->slots + (size_t)kc * kTileRows : nullptr;
                        r->out_stride = d->n_kc * kTileRows;
                        r->Y = d->Y;
                        r->done = done + c;
                        r->rb0 = p.rb0; r->rb1 = p.rb1; r->N = d->N;
                        r->flags = d->flags;
                        r->tag = epoch * (unsigned)n_calls + (unsigned)c + 1u;
                        r->last = (seg + 1 == nseg ? 1 : 0) | (d->release ? 2 : 0) | (d->q << 8);
                        r->stop = (int)((items + (unsigned)seg * (unsigned)(p.rb1 - p.rb0)) % kLookupWarps) << 8;
                        __threadfence_block();
                        mbar_arrive(bar_rec(j));
                    }
                    if (j >= 2) mbar_wait(bar_free(b), ((j - 2) >> 1) & 1, spin_limit, status);   // look-ups of job j - 2 are over
                    build_tables_bw<G>(smem + b * kTableBytes, reinterpret_cast<float*>(smem + kOffGsum + b * 64), xv, tw, lane);
                    // the scratch region of this call was last used by call guard_call: its reductions must be over
                    // before the look-up warps store into it; they start when the LAST warp of the team hands the tables
                    // over, so it is enough that the lead waits before its own arrival
                    if (lead && seg == 0 && d->guard_call >= 0 && !sh->abort &&
                        !wait_reached(done + d->guard_call, (epoch + 1u) * d->guard_target, spin_limit))
                        raise_abort(status);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_full(b));
                }
            }
            job += (unsigned)nseg;
            items = (items + (unsigned)nseg * (unsigned)(p.rb1 - p.rb0)) % kLookupWarps;
        }
        if ((job & 1u) == (unsigned)team) {
            // the record that ends the look-up warps' loop, handed over like a job (by the team whose turn it is)
            if (job >= 2) mbar_wait(bar_free(b), ((job - 2) >> 1) & 1, spin_limit, status);
            if (lead) {
                JobRec* r = job_rec(job);
                r->rb0 = 0; r->rb1 = 0;
                r->stop = 1;
                __threadfence_block();
                mbar_arrive(bar_rec(job));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_full(b));
        }
    } else {
        // ---------------------------------------------------------------- finisher warps
        // K-split reduction of every call this CTA works on, then the call's completion report
        const int fw = warp - kLookupWarps - kBuilderWarps, ft = tid - (kLookupWarps + kBuilderWarps) * 32;
        unsigned phases = 0;                  // parities of this warp's copy barriers
        // The reduction of a launch's last call is left to the finishers of the chain's next launch (their CTAs
        // move in as this launch's leave): otherwise every CTA of this launch would stay until its finishers have
        // fetched the last partial sums, a copy round trip after the last look-up, with the rest of the SM idle.
        const int f_begin = first_run ? c_begin : c_begin - 1, f_end = last_run ? c_end : c_end - 1;
        desc_begin(x, fw, f_begin, lane);
        const ChainSlot* sl = f_begin < f_end ? desc_next(x, fw, f_begin, lane) : nullptr;
        bool first_issued = false;            // this call's first copies were issued during the call before
        for (int c = f_begin; c < f_end; ++c) {
            const ChainCall* d = &sl->d;
            const bool mine = chain_part(sl).nseg > 0 && d->n_kc > 1;
            const unsigned flags = d->flags;
            const bool release = d->release != 0;
            if (mine) {
                const unsigned tag = epoch * (unsigned)n_calls + (unsigned)c + 1u;
                phases = chain_reduce(d, chain_part(sl), tag, spin_limit, status, fw, lane, phases, first_issued);
            }
            // the next call's descriptor (requested two calls ago), and its first copies before this call's report
            const ChainSlot* sl_next = c + 1 < f_end ? desc_next(x, fw, c + 1, lane) : nullptr;
            first_issued = false;
            if (sl_next != nullptr && chain_part(sl_next).nseg > 0 && sl_next->d.n_kc > 1 && !sh->abort) {
                chain_reduce_ahead(&sl_next->d, chain_part(sl_next), fw, lane);
                first_issued = true;
            }
            if (mine) {
                bar_finishers();              // every row of this CTA is stored
                if (ft == 0 && !(flags & kCallTestNoSignal)) {
                    if (release) red_release_add(done + c, 1u);
                    else red_relaxed_add(done + c, 1u);
                }
            }
            __syncwarp();
            sl = sl_next;
        }
    }
}

// Activations that lie in page-locked host memory when a chain is launched (elutq_chain_run_host): a small kernel in
// front of the chain reads them across the bus into the device arena, 16 bytes per thread and access, four accesses
// in flight.  A copy operation in the same place costs two hand-overs between copy engine and SMs (measured 11 us per
// step for 160 KB against 5-6 us this way).  (Fetching inside the chain's first launch, with the builders waiting on
// a counter, was built and measured as well: the same end-to-end time, but the extra code cost the device-resident
// step 2 %.)
__global__ void __launch_bounds__(128) chain_fetch_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, unsigned n16) {
    const unsigned stride = gridDim.x * blockDim.x;
    for (unsigned i0 = blockIdx.x * blockDim.x + threadIdx.x; i0 < n16; i0 += 4u * stride) {
        uint4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const unsigned i = i0 + (unsigned)k * stride;
            if (i < n16)
                asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w) : "l"(src + i));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const unsigned i = i0 + (unsigned)k * stride;
            if (i < n16) dst[i] = v[k];
        }
    }
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct ChainLayout {
    size_t done_off, calls_off, parts_off, slots_off, region_bytes, total;
    int regions;
};

ChainLayout chain_layout(const elutq_gemv_call* calls, int n_calls, int sms) {
    ChainLayout L;
    size_t region = 0;
    for (int i = 0; i < n_calls; ++i) {
        const size_t n_rb = ((size_t)calls[i].N + kTileRows - 1) / kTileRows;
        const size_t n_kc = ((size_t)calls[i].K + kChunkK - 1) / kChunkK;
        const size_t b = n_kc > 1 ? n_kc * n_rb * kTileRows * sizeof(unsigned long long) : 0;
        if (b > region) region = b;
    }
    L.region_bytes = round_up(region ? region : 256, 256);
    L.done_off = 256;
    L.calls_off = L.done_off + round_up((size_t)n_calls * sizeof(unsigned), 256);
    L.parts_off = L.calls_off + round_up((size_t)n_calls * sizeof(ChainCall), 256);
    L.slots_off = L.parts_off + round_up((size_t)n_calls * sms * sizeof(int4), 256);
    // Lists of small calls keep more calls in flight (they run side by side on different SMs): more regions, measured
    // on chains of the 8B attention-output layer 1.67 -> 1.54 us per call with ten instead of six.
    size_t regions = kChainScratchBytes / L.region_bytes;
    L.regions = (int)(regions < (size_t)kChainRegions ? (size_t)kChainRegions : regions > (size_t)kChainRegionsMax ? (size_t)kChainRegionsMax : regions);
    L.total = L.slots_off + (size_t)L.regions * L.region_bytes;
    return L;
}

// A call's partition over the CTAs of a launch and every CTA's share of it (host logic only, no CUDA call).
// n_rb row blocks x n_kc chunks are cut into `groups` groups of cpc consecutive chunks times R row ranges, one
// share (a row-block range of one chunk group) per CTA; the shares go to CTAs cta_first, cta_first + 1, ... modulo
// the CTA count.  share[cta] = (first row block, end row block, first chunk, chunks | group << 16); zeros: no share.
// A job with fewer items than look-up warps leaves warps idle while it lasts about as long (an item is mostly a load
// round trip), so a small layer spread over every SM costs every SM a full job cycle.  A small call that is
// independent of its neighbours in the list takes fewer CTAs instead - two rounds of items for every look-up warp of
// a CTA - and consecutive calls start on different CTAs: such calls then run side by side on different SMs.
// (Measured, 8B shapes: chains of attention-output layers 2.16 -> 1.67 us per call at q = 2, 3.50 -> 2.40 at q = 4;
// the 12-call step 63.0 -> 59.2 us; a chain in which every call reads the output of the one before is fastest spread
// over every SM.)
struct CallPartition {
    int cpc, ranges, groups, n_ctas;
};
bool chain_shares(int n_rb, int n_kc, int sms, int cta_first, bool independent, CallPartition* part, int4* share) {
    int cpc = 1, R = 1;
    plan_gemv_partition(n_rb, n_kc, sms, false, &cpc, &R);
    if (cpc == 1 && independent) {
        const int fill = (n_rb + 2 * kLookupWarps - 1) / (2 * kLookupWarps);
        if (R > fill) R = fill;
    }
    part->cpc = cpc; part->ranges = R;
    part->groups = (n_kc + cpc - 1) / cpc;
    part->n_ctas = part->groups * R;
    if (part->n_ctas > sms || part->n_ctas <= 0) return false;
    const int rb_q = n_rb / R, rb_r = n_rb % R;
    for (int cta = 0; cta < sms; ++cta) {
        int4 v = make_int4(0, 0, 0, 0);
        const int b = (cta - cta_first % sms + sms) % sms;
        if (b < part->n_ctas) {
            const int grp = b / R, range = b - grp * R;
            v.x = range * rb_q + (range < rb_r ? range : rb_r);
            v.y = v.x + rb_q + (range < rb_r ? 1 : 0);
            v.z = grp * cpc;
            const int nseg = (cpc < n_kc - v.z) ? cpc : n_kc - v.z;
            v.w = nseg | (grp << 16);
        }
        share[cta] = v;
    }
    return true;
}

int check_call(const elutq_gemv_call& c) {
    if (!c.X || !c.packed || !c.Y) return ELUTQ_ERR_INVALID_ARG;
    if (c.N <= 0 || c.K <= 0) return ELUTQ_ERR_INVALID_ARG;
    const unsigned known = ELUTQ_FLAG_OUT_F32 | ELUTQ_FLAG_ACCUMULATE | kCallTestNoSignal;
    if (c.flags & ~(known | 0x3ffu)) return ELUTQ_ERR_INVALID_ARG;
    if (c.flags & 0x3ffu & ~(ELUTQ_FLAG_OUT_F32 | ELUTQ_FLAG_ACCUMULATE)) return ELUTQ_ERR_UNSUPPORTED;
    auto al = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    if (!al(c.X) || !al(c.packed) || !al(c.Y)) return ELUTQ_ERR_ALIGN;
    return ELUTQ_OK;
}

template <int Q, int G>
cudaError_t launch_run(ChainCtl* ctl, const ChainCall* calls, const int4* parts, unsigned* done, int n_calls, int c0, int c1,
                       int first_run, int last_run, unsigned wait_limit, int sms, cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        e = cudaFuncSetAttribute(lut_chain_kernel<Q, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmem);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)sms);                   // one CTA per SM, all resident (cooperative launch)
    cfg.blockDim = dim3(kChainThreads);
    cfg.dynamicSmemBytes = kChainSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    // The chain's first launch is cooperative (its CTAs wait on one another: the runtime guarantees that all are
    // resident).  Later launches follow by programmatic dependent launch instead, which lets their CTAs move in as
    // the predecessor's leave (the two attributes together were measured to serialise the launches: 109 against 98 us
    // on the twelve calls of three bit-widths); they fill the device in the same way - one CTA per SM, as many CTAs
    // as SMs - so all of them become resident as soon as the predecessor has drained, and every wait is bounded.
    cfg.attrs = first_run ? attr : attr + 1;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, lut_chain_kernel<Q, G>, ctl, calls, parts, done, n_calls, c0, c1, first_run, last_run, wait_limit);
    count_launch(1);
    return e;
}

template <int Q>
cudaError_t launch_run_q(int G, ChainCtl* ctl, const ChainCall* calls, const int4* parts, unsigned* done, int n_calls, int c0,
                         int c1, int first_run, int last_run, unsigned wait_limit, int sms, cudaStream_t stream) {
    switch (G) {
        case 128: return launch_run<Q, 128>(ctl, calls, parts, done, n_calls, c0, c1, first_run, last_run, wait_limit, sms, stream);
        case 64: return launch_run<Q, 64>(ctl, calls, parts, done, n_calls, c0, c1, first_run, last_run, wait_limit, sms, stream);
        case 32: return launch_run<Q, 32>(ctl, calls, parts, done, n_calls, c0, c1, first_run, last_run, wait_limit, sms, stream);
        default: return cudaErrorInvalidValue;
    }
}

// Host-side copy of what elutq_chain_run needs of a plan (its runs: consecutive calls of G = 128, or of equal (q, G)), keyed by the plan's device
// address; written by elutq_chain_plan.
struct PlanRuns {
    int n_calls = 0;
    int n_runs = 0;
    int begin[kMaxRuns + 1] = {};
    int q[kMaxRuns] = {}, G[kMaxRuns] = {};
    size_t calls_off = 0, parts_off = 0, done_off = 0;
};
std::mutex g_plan_mu;
std::map<const void*, PlanRuns> g_plans;

}  // namespace
}  // namespace elutq

using namespace elutq;

extern "C" {

int elutq_chain_plan_bytes(const elutq_gemv_call* calls, int n_calls, size_t* bytes) {
    if (!calls || !bytes || n_calls <= 0 || n_calls > ELUTQ_CHAIN_MAX_CALLS) return ELUTQ_ERR_INVALID_ARG;
    for (int i = 0; i < n_calls; ++i) {
        const int st = check_call(calls[i]);
        if (st != ELUTQ_OK) return st;
    }
    *bytes = chain_layout(calls, n_calls, device_sm_count()).total;
    return ELUTQ_OK;
}

int elutq_chain_plan(const elutq_gemv_call* calls, int n_calls, void* plan, size_t plan_bytes, void* stream) {
    if (!plan) return ELUTQ_ERR_INVALID_ARG;
    size_t need = 0;
    int st = elutq_chain_plan_bytes(calls, n_calls, &need);
    if (st != ELUTQ_OK) return st;
    if ((reinterpret_cast<uintptr_t>(plan) & 255u) != 0) return ELUTQ_ERR_ALIGN;
    if (plan_bytes < need) return ELUTQ_ERR_BUFFER_TOO_SMALL;
    const int sms = device_sm_count();
    const ChainLayout L = chain_layout(calls, n_calls, sms);
    uint8_t* base = reinterpret_cast<uint8_t*>(plan);

    std::vector<uint8_t> host(L.slots_off, 0);
    ChainCtl* ctl = reinterpret_cast<ChainCtl*>(host.data());
    ctl->magic = kChainMagic;
    ctl->n_calls = (unsigned)n_calls;
    ctl->grid = (unsigned)sms;
    ctl->done_off = L.done_off; ctl->calls_off = L.calls_off; ctl->parts_off = L.parts_off; ctl->slots_off = L.slots_off;
    ctl->region_bytes = L.region_bytes; ctl->total_bytes = L.total;
    ChainCall* dc = reinterpret_cast<ChainCall*>(host.data() + L.calls_off);
    PlanRuns runs;
    int cta_first = 0;                        // where the next call's shares begin (round robin over the CTAs)
    runs.n_calls = n_calls;
    runs.calls_off = L.calls_off; runs.parts_off = L.parts_off; runs.done_off = L.done_off;
    for (int i = 0; i < n_calls; ++i) {
        const elutq_gemv_call& c = calls[i];
        int q = 0, G = 0;
        st = blob_meta(c.packed, c.N, c.K, &q, &G);       // reads the blob's header when the address is unknown
        if (st != ELUTQ_OK) return st;
        const Geo g = make_geo(q, G, c.N, c.K);
        ChainCall& d = dc[i];
        d.X = reinterpret_cast<const __half*>(c.X);
        d.tiles = reinterpret_cast<const uint8_t*>(c.packed) + ELUTQ_HEADER_BYTES;
        d.Y = c.Y;
        d.slots = reinterpret_cast<unsigned long long*>(base + L.slots_off + (size_t)(i % L.regions) * L.region_bytes);
        d.N = c.N; d.K = c.K; d.n_rb = g.n_rb; d.n_kc = g.n_kc;
        d.q = q; d.G = G;
        d.flags = c.flags & (ELUTQ_FLAG_OUT_F32 | ELUTQ_FLAG_ACCUMULATE | kCallTestNoSignal);
        // as-if-sequential order: call i must follow every earlier call j whose output it reads (X_i on Y_j) or
        // overwrites (Y_i on Y_j), or whose input it overwrites (Y_i on X_j)
        d.dep_first = i; d.dep_last = -1;
        for (int j = 0; j < i; ++j) {
            const elutq_gemv_call& e = calls[j];
            auto overlap = [](const void* a, size_t na, const void* b, size_t nb) {
                const uintptr_t pa = reinterpret_cast<uintptr_t>(a), pb = reinterpret_cast<uintptr_t>(b);
                return pa < pb + nb && pb < pa + na;
            };
            const size_t xi = (size_t)c.K * 2, yi = (size_t)c.N * ((c.flags & ELUTQ_FLAG_OUT_F32) ? 4 : 2);
            const size_t xj = (size_t)e.K * 2, yj = (size_t)e.N * ((e.flags & ELUTQ_FLAG_OUT_F32) ? 4 : 2);
            if (overlap(c.X, xi, e.Y, yj) || overlap(c.Y, yi, e.Y, yj) || overlap(c.Y, yi, e.X, xj)) {
                if (j < d.dep_first) d.dep_first = j;
                d.dep_last = j;
            }
        }
        for (int j = d.dep_first; j <= d.dep_last; ++j) dc[j].release = 1;   // their reports order their outputs before them
    }
    for (int i = 0; i < n_calls; ++i) {
        const elutq_gemv_call& c = calls[i];
        ChainCall& d = dc[i];
        const int q = d.q, G = d.G;
        const Geo g = make_geo(q, G, c.N, c.K);
        // a call that neither waits for the call before it nor is waited for by the call after it may take fewer CTAs
        const bool waits = d.dep_first <= d.dep_last && d.dep_last == i - 1;
        const bool waited_for = i + 1 < n_calls && dc[i + 1].dep_first <= dc[i + 1].dep_last && dc[i + 1].dep_last == i;
        CallPartition cp;
        int4* pt = reinterpret_cast<int4*>(host.data() + L.parts_off) + (size_t)i * sms;
        if (!chain_shares(g.n_rb, g.n_kc, sms, cta_first, !waits && !waited_for, &cp, pt)) return ELUTQ_ERR_UNSUPPORTED;
        d.cpc = cp.cpc; d.ranges = cp.ranges; d.rb_q = g.n_rb / cp.ranges; d.rb_r = g.n_rb % cp.ranges;
        d.groups = cp.groups;
        d.n_ctas = cp.n_ctas;
        cta_first = (cta_first + d.n_ctas) % sms;
        d.guard_call = i >= L.regions ? i - L.regions : -1;
        d.guard_target = d.guard_call >= 0 ? dc[d.guard_call].done_target : 0u;
        d.done_target = (unsigned)(g.n_kc > 1 ? d.n_ctas : d.n_ctas * kLookupWarps);
        if (runs.n_runs > 0 && G == 128 && runs.G[runs.n_runs - 1] == 128 && runs.q[runs.n_runs - 1] != q) {
            runs.q[runs.n_runs - 1] = 0;      // consecutive calls of G = 128 and different q: one launch of the run-time-q kernel
        } else if (runs.n_runs == 0 || runs.q[runs.n_runs - 1] != q || runs.G[runs.n_runs - 1] != G) {
            if (runs.n_runs == kMaxRuns) return ELUTQ_ERR_UNSUPPORTED;
            runs.begin[runs.n_runs] = i;
            runs.q[runs.n_runs] = q;
            runs.G[runs.n_runs] = G;
            runs.n_runs += 1;
        }
    }
    runs.begin[runs.n_runs] = n_calls;
    cudaError_t e = cudaMemsetAsync(plan, 0, L.total, (cudaStream_t)stream);
    if (e != cudaSuccess) return note_cuda_error((int)e);
    // pageable source: the copy is staged by the runtime before the call returns
    e = cudaMemcpyAsync(plan, host.data(), host.size(), cudaMemcpyHostToDevice, (cudaStream_t)stream);
    if (e != cudaSuccess) return note_cuda_error((int)e);
    e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return note_cuda_error((int)e);
    std::lock_guard<std::mutex> lk(g_plan_mu);
    g_plans[plan] = runs;
    return ELUTQ_OK;
}

int elutq_chain_run_opts(void* plan, int n_calls, unsigned wait_limit, void* stream) {
    if (!plan || n_calls <= 0 || n_calls > ELUTQ_CHAIN_MAX_CALLS) return ELUTQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(plan) & 255u) != 0) return ELUTQ_ERR_ALIGN;
    PlanRuns runs;
    {
        std::lock_guard<std::mutex> lk(g_plan_mu);
        auto it = g_plans.find(plan);
        if (it == g_plans.end() || it->second.n_calls != n_calls) return ELUTQ_ERR_SHAPE;   // not planned by this process
        runs = it->second;
    }
    ChainCtl* ctl = reinterpret_cast<ChainCtl*>(plan);
    const ChainCall* calls = reinterpret_cast<const ChainCall*>(reinterpret_cast<uint8_t*>(plan) + runs.calls_off);
    const int4* parts = reinterpret_cast<const int4*>(reinterpret_cast<uint8_t*>(plan) + runs.parts_off);
    unsigned* done = reinterpret_cast<unsigned*>(reinterpret_cast<uint8_t*>(plan) + runs.done_off);
    if (wait_limit == 0) wait_limit = 1u << 22;
    const int sms = device_sm_count();
    for (int r = 0; r < runs.n_runs; ++r) {
        const int last = r + 1 == runs.n_runs;
        cudaError_t e;
        switch (runs.q[r]) {
            case 0: e = launch_run<0, 128>(ctl, calls, parts, done, n_calls, runs.begin[r], runs.begin[r + 1], r == 0, last, wait_limit, sms, (cudaStream_t)stream); break;
            case 1: e = launch_run_q<1>(runs.G[r], ctl, calls, parts, done, n_calls, runs.begin[r], runs.begin[r + 1], r == 0, last, wait_limit, sms, (cudaStream_t)stream); break;
            case 2: e = launch_run_q<2>(runs.G[r], ctl, calls, parts, done, n_calls, runs.begin[r], runs.begin[r + 1], r == 0, last, wait_limit, sms, (cudaStream_t)stream); break;
            case 3: e = launch_run_q<3>(runs.G[r], ctl, calls, parts, done, n_calls, runs.begin[r], runs.begin[r + 1], r == 0, last, wait_limit, sms, (cudaStream_t)stream); break;
            case 4: e = launch_run_q<4>(runs.G[r], ctl, calls, parts, done, n_calls, runs.begin[r], runs.begin[r + 1], r == 0, last, wait_limit, sms, (cudaStream_t)stream); break;
            default: e = cudaErrorInvalidValue; break;
        }
        if (e != cudaSuccess) return note_cuda_error((int)e);
    }
    return ELUTQ_OK;
}

int elutq_chain_run_host(void* plan, int n_calls, void* x_dev, const void* x_host, size_t x_bytes, const void* y_dev,
                         void* y_host, size_t y_bytes, void* stream) {
    if ((x_bytes && (!x_dev || !x_host)) || (y_bytes && (!y_dev || !y_host))) return ELUTQ_ERR_INVALID_ARG;
    // Page-locked host activations that the device can address are fetched by a small kernel; anything else (pageable
    // memory, odd sizes or alignment, more than 8 MiB) goes through a copy.
    const void* fetch_src = nullptr;
    if (x_bytes && x_bytes <= (8u << 20) && x_bytes % 16 == 0 && (reinterpret_cast<uintptr_t>(x_dev) & 15u) == 0) {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, x_host) == cudaSuccess) {
            if (at.type == cudaMemoryTypeHost && at.devicePointer != nullptr &&
                (reinterpret_cast<uintptr_t>(at.devicePointer) & 15u) == 0)
                fetch_src = at.devicePointer;
        } else {
            cudaGetLastError();               // not an address the runtime knows: plain pageable memory
        }
    }
    if (fetch_src != nullptr) {
        const unsigned n16 = (unsigned)(x_bytes / 16);
        const unsigned blocks = (n16 + 127u) / 128u < (unsigned)device_sm_count() ? (n16 + 127u) / 128u : (unsigned)device_sm_count();
        chain_fetch_kernel<<<blocks, 128, 0, (cudaStream_t)stream>>>(reinterpret_cast<const uint4*>(fetch_src),
                                                                     reinterpret_cast<uint4*>(x_dev), n16);
        count_launch(1);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return note_cuda_error((int)e);
    } else if (x_bytes) {
        const cudaError_t e = cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, (cudaStream_t)stream);
        if (e != cudaSuccess) return note_cuda_error((int)e);
    }
    const int rc = elutq_chain_run_opts(plan, n_calls, 0, stream);
    if (rc != ELUTQ_OK) return rc;
    if (y_bytes) {
        const cudaError_t e = cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
        if (e != cudaSuccess) return note_cuda_error((int)e);
    }
    return ELUTQ_OK;
}

int elutq_chain_run(void* plan, int n_calls, void* stream) {
    return elutq_chain_run_opts(plan, n_calls, 0u, stream);
}

int elutq_chain_status(const void* plan, void* stream, int* status) {
    if (!plan || !status) return ELUTQ_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return note_cuda_error((int)e);
    ChainCtl h;
    e = cudaMemcpy(&h, plan, sizeof(h), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return note_cuda_error((int)e);
    if (h.magic != kChainMagic) return ELUTQ_ERR_SHAPE;
    *status = (int)h.status;
    return ELUTQ_OK;
}


int elutq_chain_shares(int N, int K, int n_ctas_max, int cta_first, int independent, int* shares, int* partition) {
    if (N <= 0 || K <= 0 || n_ctas_max <= 0 || n_ctas_max > 1024 || cta_first < 0 || !shares || !partition) return ELUTQ_ERR_INVALID_ARG;
    const int n_rb = (N + kTileRows - 1) / kTileRows, n_kc = (K + kChunkK - 1) / kChunkK;
    CallPartition cp;
    std::vector<int4> sh((size_t)n_ctas_max);
    if (!chain_shares(n_rb, n_kc, n_ctas_max, cta_first, independent != 0, &cp, sh.data())) return ELUTQ_ERR_UNSUPPORTED;
    for (int i = 0; i < n_ctas_max; ++i) {
        shares[4 * i] = sh[i].x; shares[4 * i + 1] = sh[i].y; shares[4 * i + 2] = sh[i].z; shares[4 * i + 3] = sh[i].w;
    }
    partition[0] = cp.cpc; partition[1] = cp.ranges; partition[2] = cp.groups; partition[3] = cp.n_ctas;
    return ELUTQ_OK;
}

int elutq_chain_forget(const void* plan) {
    if (!plan) return ELUTQ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(g_plan_mu);
    g_plans.erase(plan);
    return ELUTQ_OK;
}

}  // extern "C"
