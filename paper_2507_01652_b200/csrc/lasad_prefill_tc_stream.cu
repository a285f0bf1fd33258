// LASAD chunked prefill on the 5th-generation tensor cores (sm_100a), task-streaming form:
// TMA-fed tcgen05.mma with TMEM accumulators, bf16 I/O, fp32 accumulation, fp32 carried state.
//
// Work decomposition.  The sequence of one (batch, head) -- a chain -- is cut into chunks of
// C = 128 tokens.  One task = one chunk of one chain.  Tasks are numbered chunk-major
// (id = n * X + x for chunk n of chain x, X = B * H chains) and handed out, in increasing order,
// from a launch-wide counter to a grid of persistent CTAs, two per SM (256 TMEM columns and
// ~106 KB of shared memory each): a CTA draws its next task when it has room for the task's tiles,
// two tasks ahead of the one it computes.  Everything in a task except the carried state is
// independent of every other task; the d_k x d_v fp32 state is relayed from the CTA that ran
// chunk n-1 of the chain to the CTA that runs chunk n through a per-chain slot in global memory
// (it stays in L2).  Consecutive tasks of one CTA belong to different chains, so every SM holds
// the same amount of work however B * H relates to the SM count, and consecutive chunks of one
// chain are loaded and multiplied concurrently on different SMs; only the state relay (read 32 KB
// of packets, fp32 update, write 32 KB of packets) is serial along a chain.
// Forward progress: a task waits only for a task with a smaller number; numbers are drawn by CTAs
// that are running, each of which works through what it has drawn in increasing order.  So the
// smallest unfinished number is always held by a running CTA that waits for nothing, whatever
// part of the grid is resident at the time: the grid size (the host's estimate of what fits on
// the device) is a matter of speed, not of correctness.  Every wait is bounded anyway.
//
// Relay packets.  A state value travels as one 64-bit word (tag in the high half, value in the low
// half), two words per 16-byte vector access.  A 64-bit element is read and written as a unit, so
// a word whose tag matches carries its value: the relay needs no fence and no separate flag (release/acquire at GPU scope stalled for
// microseconds while bulk copies were in flight).  The tag is the launch number (folded into
// 1..65535 by the host, which clears the slots before a value comes round again) and the chunk
// index.  Waiting CTAs poll one packet per warp, never the whole slot.
//
// With n_i = number of decaying steps from the chunk start up to and including token i (SAD rule,
// Section 3.4, from the token's grid position), N = n of the chunk's last token and gamma the
// head's decay, the SAD recurrence (Section 3.4) unrolled over one chunk is
//
//     o_i   = scale * ( sum_{j<=i} (q_i.k_j) gamma^(n_i-n_j) v_j  +  gamma^(n_i) q_i^T S_prev )
//     S_new = gamma^N S_prev + sum_j gamma^(N-n_j) k_j v_j^T
//
// Normal path (gamma >= 0.6, so that gamma^-128 stays far inside fp32 range).  Every decay
// factor is moved onto V and onto one per-row factor of the output, so that Q and K feed the
// tensor cores untouched and the scores only need the causal mask:
//
//     V~ = diag(gamma^(N-n_j)) V                       in place in smem
//     dS = K^T V~                        (M2a)         tcgen05.mma 64x64x128
//     S_new = gamma^N S_prev + dS        (E3)          as soon as S_prev has arrived; relayed on at once
//     S  = Q K^T                         (M1)          tcgen05.mma 128x128x64, smem x smem
//     A  = tril(S) -> bf16               (E1)          back into TMEM over S's own columns
//     O' = A V~ + Q (gamma^N S_prev)     (M2b)         tcgen05.mma 128x64x128 (tmem x smem) + 128x64x64
//     o_i = scale * gamma^-(N-n_i) * O'_i   (E2)       -> bf16 -> smem -> TMA store
//
// Exact path (gamma < 0.6, including 0, where gamma^-(N-n_i) would overflow): only factors
// with non-negative exponents are formed, all from a table of gamma^m, m = 0..128:
// P = S o gamma^(n_i-n_j) o [j<=i], Q~ = diag(gamma^(n_i)) Q and K~ = diag(gamma^(N-n_j)) K
// in place, O = P V + Q~ S_prev, dS = K~^T V.  Same MMAs, same barriers, slower element-wise
// stages; it exists for correctness over the whole decay range [0, 1].
//
// Warp roles: warps 0-7 do the element-wise stages; warp w works on TMEM lane quadrant w & 3
// (chunk rows 32(w&3)..+31) and the two warps of a quadrant split its columns.  Warp 8
// allocates TMEM and issues every MMA, warp 9 issues the TMA loads and stores.  All waits are
// bounded: a wait that runs out raises a status word the host can read and the CTA leaves
// through the normal exit (copies in flight are waited for, TMEM is freed).
#include "../../include/lasad.h"
#include "lasad_common.cuh"
#include "lasad_tc_chunk.cuh"
#include "lasad_tc_ptx.cuh"
#include "lasad_tc_tma.cuh"

#include <cmath>
#include <mutex>


namespace lasad {
namespace {

using namespace tcx;

constexpr int kThreads = kEThreads + 64;   // element-wise warps, the MMA warp and the TMA warp
constexpr int kStages = 2;
constexpr int kTmemCols = 256;
constexpr int kHeadCache = 256;

struct __align__(8) Barriers {
    unsigned long long full[kStages];   // TMA loads of a stage have landed
    unsigned long long s_done;     // M1 complete
    unsigned long long x_ready;    // V~ (normal path) or K~ (exact path) written: dS may start (256 arrivals)
    unsigned long long ds_done;    // dS MMAs complete
    unsigned long long p_ready;    // A/P in TMEM (and Q~ in smem) (256 arrivals)
    unsigned long long sb_ready;   // bf16 copy of the incoming state in smem (256 arrivals)
    unsigned long long o_done;     // O MMAs complete (and every MMA issued before them)
    // one per stage: its next phase is the task two further on, whose loads the TMA warp issues only
    // after it has seen this phase, so the one-bit phase parity is never taken for a later phase's
    unsigned long long st_ready[kStages];   // output tile staged in smem (256 arrivals)
    unsigned long long tbl_free;   // exact path: every thread is done with the current table (256)
    unsigned long long tbl_ready;  // exact path: the table of this task's head is written (256)
    unsigned long long drain;      // teardown: all MMAs retired
};

struct Smem {
    // tiles first: each must sit on a 1024-byte boundary (128-byte swizzle atom = 8 rows)
    unsigned char q[kStages][kTileBytes];
    unsigned char k[kStages][kTileBytes];
    unsigned char v[kStages][kTileBytes];
    unsigned char sb[kD * kD * 2];  // bf16 copy of the incoming state, [dk][dv], 128 B rows, swizzled
    float pw[kC + 4];               // gamma^m, m = 0..128 (exact path only, rebuilt per task)
    float gam[kHeadCache];          // the heads' decays and their base-2 logarithms (when H <= kHeadCache)
    float lgam[kHeadCache];
    // the tasks this CTA has drawn, by position in its sequence modulo 4 (n < 0: the work has run out);
    // written by the TMA warp before it issues (or, for the end marker, completes by hand) the `full`
    // barrier of that position's stage, read by the other roles after that wait
    struct Drawn {
        int n, x, b, h;     // chunk, chain, batch, head
        int phase;          // (grid index of the chunk's first token + 1) mod w
    } ring[4];
    Barriers bar;
    uint32_t tmem_base;
    int abort_flag;
};

struct StreamParams {
    int B, T, H;
    int X;                     // chains = B * H
    int n_chunks;              // chunks per chain
    int n_tasks;               // X * n_chunks
    int grid_w, prefix_len;
    long long t0;
    float scale;
    const float* decay;
    const float* state_in;
    float* state_out;
    uint4* relay;              // [X][dk * dv / 2]: two (value, tag) packets per element
    unsigned epoch16;          // launch number folded into 1..65535: high half of the packets' tag
    int* work;                 // [2], zero between launches: tasks drawn so far, CTAs that have left
    int* status;
    unsigned wait_limit;
};

// One task = chunk n of chain x = (b, h).
struct Task {
    int n, x, b, h;
};
__device__ __forceinline__ Task decode_task(int id, int X, int H)
{
    Task t;
    t.n = id / X;
    t.x = id - t.n * X;
    t.b = t.x / H;
    t.h = t.x - t.b * H;
    return t;
}

__global__ void __launch_bounds__(kThreads, 2)
prefill_stream_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                      StreamParams p)
{
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &sm.abort_flag;
    volatile Smem::Drawn* ring = sm.ring;
    const unsigned limit = p.wait_limit;

    // ---- set-up ---------------------------------------------------------------------------
    // A kernel launched behind this one as a programmatic dependent may start to take SMs as they
    // become free; it waits for this kernel's completion before it touches device memory.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&sm.bar.full[s], 1);
        mbar_init(&sm.bar.s_done, 1);
        mbar_init(&sm.bar.x_ready, kEThreads);
        mbar_init(&sm.bar.ds_done, 1);
        mbar_init(&sm.bar.p_ready, kEThreads);
        mbar_init(&sm.bar.sb_ready, kEThreads);
        mbar_init(&sm.bar.o_done, 1);
        for (int s = 0; s < kStages; ++s) mbar_init(&sm.bar.st_ready[s], kEThreads);
        mbar_init(&sm.bar.tbl_free, kEThreads);
        mbar_init(&sm.bar.tbl_ready, kEThreads);
        mbar_init(&sm.bar.drain, 1);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // nothing above reads or writes device memory; everything below may depend on the kernel before
    // this one in the stream
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (p.H <= kHeadCache) {
        for (int hh = tid; hh < p.H; hh += kThreads) {
            const float gm = p.decay[hh];
            sm.gam[hh] = gm;
            sm.lgam[hh] = gm > 0.0f ? log2f(gm) : 0.0f;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 9) {
        // ===================== TMA warp: loads two tasks ahead, stores each output tile ========
        if (elect_one()) {
            // position of the call's first token relative to the grid (SAD rule, Section 3.4)
            int step = 0, phase0 = 0;
            if (p.grid_w > 0) {
                long long ph = (p.t0 - p.prefix_len + 1) % p.grid_w;    // C remainder: may be negative inside the prefix
                if (ph < 0) ph += p.grid_w;
                phase0 = (int)ph;
                step = kC % p.grid_w;
            }
            // Draws the next task from the launch-wide counter for position g of this CTA's sequence,
            // publishes it and issues its loads; at the end of the work it publishes the end marker
            // instead (once) and returns false.  Tasks are numbered chunk-major, so a task only
            // depends on a smaller number, and numbers are handed out in increasing order to CTAs
            // that are running: whoever holds the task another one waits for is making progress,
            // whatever part of the grid is resident.
            auto draw = [&](int g) {
                const int s = g % kStages;
                const int id = atomicAdd(p.work, 1);
                volatile Smem::Drawn& d = ring[g & 3];
                if (id >= p.n_tasks) {
                    d.n = -1;
                    __threadfence_block();
                    mbar_arrive(&sm.bar.full[s]);     // completes the phase: the waiters find the marker
                    return false;
                }
                const Task t = decode_task(id, p.X, p.H);
                d.n = t.n; d.x = t.x; d.b = t.b; d.h = t.h;
                d.phase = p.grid_w > 0 ? (int)(((long long)(t.n % p.grid_w) * step + phase0) % p.grid_w) : 0;
                __threadfence_block();
                mbar_arrive_expect_tx(&sm.bar.full[s], 3 * kTileBytes);
                tma_load_4d(sm.q[s], &tm_q, &sm.bar.full[s], 0, t.h, t.n * kC, t.b);
                tma_load_4d(sm.k[s], &tm_k, &sm.bar.full[s], 0, t.h, t.n * kC, t.b);
                tma_load_4d(sm.v[s], &tm_v, &sm.bar.full[s], 0, t.h, t.n * kC, t.b);
                return true;
            };
            int loads_issued = 0;      // positions whose loads have been issued
            bool more = true;
            for (int g = 0; g < kStages && more; ++g) {
                more = draw(g);
                if (more) loads_issued = g + 1;
            }
            for (int g = 0; g < loads_issued; ++g) {
                const int s = g % kStages;
                // the output tile of task g sits in the Q buffer of its stage; by now every MMA
                // that read this stage has retired (the element-wise warps waited for o_done)
                if (!mbar_wait(&sm.bar.st_ready[s], (g / kStages) & 1, limit, abort_flag, p.status)) break;
                tma_store_4d(&tm_o, sm.q[s], 0, ring[g & 3].h, ring[g & 3].n * kC, ring[g & 3].b);
                tma_store_commit();
                if (more) {
                    tma_store_wait_read();        // the store has finished reading the buffer
                    more = draw(g + kStages);
                    if (more) loads_issued = g + kStages + 1;
                }
            }
            tma_store_wait_all();
            // leave only when every issued load has landed (they write this CTA's shared memory)
            // (once the end marker is out, the task before the last loaded one has been computed, and
            // its stage's barrier has moved on by the marker's phase: only the last one is waited for)
            for (int g = max(0, more ? loads_issued - kStages : loads_issued - 1); g < loads_issued; ++g)
                for (unsigned it = 0; it < kTeardownLimit; ++it)
                    if (mbar_try_wait(&sm.bar.full[g % kStages], (g / kStages) & 1)) break;
        }
        __syncwarp();
    } else if (warp == 8) {
        // ===================== MMA issuer: the whole warp runs the loop, one lane issues =======
        constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);   // Q (K-major) x K (K-major)
        constexpr uint32_t idesc_pv = make_idesc(128, 64, 0, 1);   // A/P (tmem) x V (MN-major)
        constexpr uint32_t idesc_qs = make_idesc(128, 64, 0, 1);   // Q (K-major) x state (MN-major)
        constexpr uint32_t idesc_kv = make_idesc(64, 64, 1, 1);    // K^T (MN-major) x V (MN-major)
        const uint64_t d_sb = make_desc(smem_u32(sm.sb));
        const uint64_t dq0 = make_desc(smem_u32(sm.q[0])), dq1 = make_desc(smem_u32(sm.q[1]));
        const uint64_t dk0 = make_desc(smem_u32(sm.k[0])), dk1 = make_desc(smem_u32(sm.k[1]));
        const uint64_t dv0 = make_desc(smem_u32(sm.v[0])), dv1 = make_desc(smem_u32(sm.v[1]));
        auto issue_m1 = [&](int g) {
            const uint64_t dq = (g & 1) ? dq1 : dq0, dk = (g & 1) ? dk1 : dk0;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)  // 32 bytes along K per step
                    mma_ss(tmem + kColS, dq + 2 * kk, dk + 2 * kk, idesc_s, kk > 0);
                mma_commit(&sm.bar.s_done);
            }
            __syncwarp();
        };
        bool ok = mbar_wait(&sm.bar.full[0], 0, limit, abort_flag, p.status) && ring[0].n >= 0;
        if (ok) issue_m1(0);
        for (int g = 0; ok; ++g) {
            const uint64_t dq = (g & 1) ? dq1 : dq0, dk = (g & 1) ? dk1 : dk0, dv = (g & 1) ? dv1 : dv0;
            if (!mbar_wait(&sm.bar.x_ready, g & 1, limit, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // 16 tokens = 2048 B of K and of V per step
                    mma_ss(tmem + kColDS, dk + 128 * kk, dv + 128 * kk, idesc_kv, kk > 0);
                mma_commit(&sm.bar.ds_done);
            }
            __syncwarp();
            if (!mbar_wait(&sm.bar.p_ready, g & 1, limit, abort_flag, p.status)) { ok = false; break; }
            if (!mbar_wait(&sm.bar.sb_ready, g & 1, limit, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // A/P: 8 TMEM columns per step (tokens 0..63 at columns
                                                      // 0..31, tokens 64..127 at 64..95); V: 2048 B per step
                    mma_ts(tmem + kColO, tmem + kColS + (kk < 4 ? 8 * kk : 64 + 8 * (kk - 4)), dv + 128 * kk,
                           idesc_pv, kk > 0);
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)
                    mma_ss(tmem + kColO, dq + 2 * kk, d_sb + 128 * kk, idesc_qs, 1);
                mma_commit(&sm.bar.o_done);
            }
            __syncwarp();
            // the scores of the next task (they overwrite A's columns: the tensor pipe runs in
            // issue order, so the A V MMAs above read A first)
            if (!mbar_wait(&sm.bar.full[(g + 1) % kStages], ((g + 1) / kStages) & 1, limit, abort_flag, p.status)) {
                ok = false;
                break;
            }
            if (ring[(g + 1) & 3].n < 0) break;      // the work has run out
            issue_m1(g + 1);
        }
        // make sure nothing is still running on the tensor pipe before TMEM is freed
        if (elect_one()) {
            mma_commit(&sm.bar.drain);
            for (unsigned it = 0; it < kTeardownLimit; ++it)
                if (mbar_try_wait(&sm.bar.drain, 0)) break;
        }
        __syncwarp();
    } else {
        // ===================== element-wise warps ==============================================
        const int qd = warp & 3;                 // TMEM lane quadrant
        const int grp = warp >> 2;               // which half of the quadrant's columns
        const int i = qd * 32 + lane;            // chunk row owned by this thread
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        // State ownership.  The dS accumulator (M = 64 layout) keeps state rows 16 qd .. 16 qd + 15 in
        // the first 16 TMEM lanes of quadrant qd; the 16x256b load spreads this warp's 16 rows x 32
        // columns (columns 32 grp ..) over all 32 threads, 16 values each: for column group k,
        // st[4k], st[4k+1] = (row r0, columns c0 + 8k, + 1), st[4k+2], st[4k+3] = (row r0 + 8, same).
        const int r0 = qd * 16 + (lane >> 2);
        const int c0 = 32 * grp + 2 * (lane & 3);

        // position of the call's first token relative to the grid (SAD rule, Section 3.4)
        const GridPos gp = grid_pos_init(p.grid_w, p.prefix_len, p.t0, lane);

        float st[16];
        auto load_state = [&](const float* src_state) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 a = __ldcg(reinterpret_cast<const float2*>(src_state + (size_t)r0 * kD + c0 + 8 * k));
                const float2 b = __ldcg(reinterpret_cast<const float2*>(src_state + (size_t)(r0 + 8) * kD + c0 + 8 * k));
                st[4 * k] = a.x; st[4 * k + 1] = a.y; st[4 * k + 2] = b.x; st[4 * k + 3] = b.y;
            }
        };
        auto store_state = [&](float* dst_state) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                *reinterpret_cast<float2*>(dst_state + (size_t)r0 * kD + c0 + 8 * k) = make_float2(st[4 * k], st[4 * k + 1]);
                *reinterpret_cast<float2*>(dst_state + (size_t)(r0 + 8) * kD + c0 + 8 * k) =
                    make_float2(st[4 * k + 2], st[4 * k + 3]);
            }
        };
        // Relay slot layout: the 16-byte word j (two tagged values) of element-wise thread tid sits
        // at word j * 256 + tid, so that a warp's access covers 512 contiguous bytes; both sides of
        // the relay use the same thread mapping, so the layout never shows outside the slot.
        auto relay_out = [&](uint4* slot, uint32_t tag) {
            uint4* dst = slot + tid;
            const unsigned long long hi = (unsigned long long)tag << 32;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                st_cg_v2u64(dst + j * kEThreads, hi | __float_as_uint(st[2 * j]), hi | __float_as_uint(st[2 * j + 1]));
        };
        // The eight 16-byte words are requested into registers and then accepted (tags checked,
        // values moved into st).
        auto relay_request = [&](const uint4* slot, unsigned long long (&rv)[16]) {
            const uint4* src = slot + tid;
#pragma unroll
            for (int j = 0; j < 8; ++j) ld_cg_v2u64(src + j * kEThreads, rv[2 * j], rv[2 * j + 1]);
        };
        // true when every tag matched (warp-uniform result)
        auto relay_accept = [&](const unsigned long long (&rv)[16], uint32_t tag) {
            bool all = true;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                st[e] = __uint_as_float((uint32_t)rv[e]);
                all = all && (uint32_t)(rv[e] >> 32) == tag;
            }
            return __all_sync(0xffffffffu, all);
        };
        // Cheap look at the relay slot for polling loops: one lane per warp reads the warp's last
        // word (the writer stores its words in ascending order), so that waiting CTAs do not load
        // L2 with 32 KB per poll.
        auto relay_peek = [&](const uint4* slot, uint32_t tag) {
            bool hit = true;
            if (lane == 31) {
                unsigned long long a, b;
                ld_cg_v2u64(slot + 7 * kEThreads + tid, a, b);
                hit = (uint32_t)(a >> 32) == tag && (uint32_t)(b >> 32) == tag;
            }
            return __all_sync(0xffffffffu, hit);
        };
        // bf16 copy of mult * state for the Q x state MMAs: [dk][dv] rows of 128 B, 16-byte pieces
        // swizzled by the row; this thread writes eight bf16 pairs
        auto write_state_bf16 = [&](float mult) {
            unsigned char* row0 = sm.sb + r0 * 128 + 4 * (lane & 3);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int piece = ((4 * grp + k) ^ (r0 & 7)) * 16;    // r0 + 8 has the same low bits
                float a0, a1, b0, b1;
                mul2(st[4 * k], st[4 * k + 1], mult, a0, a1);
                mul2(st[4 * k + 2], st[4 * k + 3], mult, b0, b1);
                *reinterpret_cast<uint32_t*>(row0 + piece) = pack_bf16(a0, a1);
                *reinterpret_cast<uint32_t*>(row0 + 8 * 128 + piece) = pack_bf16(b0, b1);
            }
        };
        // E3: S_new = g * S_prev + dS
        auto update_state = [&](float g) {
            uint32_t dsv[16];
            tmem_ld_16x256b_x4(tmem + lane_base + kColDS + 32 * grp, dsv);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; e += 2)
                fma2(st[e], st[e + 1], g, __uint_as_float(dsv[e]), __uint_as_float(dsv[e + 1]), st[e], st[e + 1]);
        };
        // E2: this thread's 32 columns of output row i -> bf16 -> the stage's Q buffer
        auto stage_output = [&](int s, float f) {
            unsigned char* orow = sm.q[s] + i * 128;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t ov[16];
                tmem_ld16(tmem + lane_base + kColO + 32 * grp + 16 * hh, ov);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float r0, r1;
                        mul2(__uint_as_float(ov[8 * c + 2 * e]), __uint_as_float(ov[8 * c + 2 * e + 1]), f, r0, r1);
                        w[e] = pack_bf16(r0, r1);
                    }
                    reinterpret_cast<uint4*>(orow)[(4 * grp + 2 * hh + c) ^ (i & 7)] = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        };

        bool ok = true;
        unsigned exact_tasks = 0;    // exact-path tasks this CTA has run (phase of the table barriers)
        for (int g = 0; ok; ++g) {
            const int s = g % kStages;
            const unsigned par = g & 1;
            // the task the TMA warp drew for this position (chunk, chain, batch, head, grid phase)
            if (!(ok = mbar_wait(&sm.bar.full[s], (g / kStages) & 1, limit, abort_flag, p.status))) break;
            Task t;
            t.n = ring[g & 3].n;
            if (t.n < 0) break;                      // the work has run out
            t.x = ring[g & 3].x; t.b = ring[g & 3].b; t.h = ring[g & 3].h;
            const int phase = ring[g & 3].phase;
            float gamma, lg;
            if (p.H <= kHeadCache) {
                gamma = sm.gam[t.h];
                lg = sm.lgam[t.h];
            } else {
                gamma = p.decay[t.h];
                lg = gamma > 0.0f ? log2f(gamma) : 0.0f;
            }
            const bool fast = gamma >= kFastPathMinDecay;
            const bool last_chunk = t.n + 1 == p.n_chunks;
            const bool relayed_in = t.n > 0;
            GridPos here = gp;          // the task's chunk: offset and phase within the call
            here.phase = phase;
            const ChunkDecay cd = chunk_decay(here, t.n * kC, min(kC, p.T - t.n * kC), qd, lane);
            uint4* const slot = p.relay ? p.relay + (size_t)t.x * (kD * kD / 2) : nullptr;
            // tag of the state after chunk n - 1 of this launch (what this task consumes): launch
            // number and chunk index; the state this task produces carries the next tag
            const uint32_t tag_in = (p.epoch16 << 16) | ((uint32_t)t.n & 0xffffu);
            const uint32_t tag_out = (p.epoch16 << 16) | ((uint32_t)(t.n + 1) & 0xffffu);

            // gamma^m: normal path straight from ex2.approx (|m log2 gamma| <= 95, relative error ~1e-5);
            // exact path from a table in double precision (0^0 = 1), rebuilt for this task's head
            auto gpow = [&](int m) { return ex2_approx((float)m * lg); };
            if (!fast) {
                // every thread is done with the previous exact task's table before it is rewritten
                if (exact_tasks > 0 &&
                    !(ok = mbar_wait(&sm.bar.tbl_free, (exact_tasks - 1) & 1, limit, abort_flag, p.status))) break;
                if (tid <= kC) {
                    double base = (double)gamma, acc = 1.0;
                    for (int e = tid; e > 0; e >>= 1) {
                        if (e & 1) acc *= base;
                        base *= base;
                    }
                    sm.pw[tid] = (float)acc;
                }
                mbar_arrive(&sm.bar.tbl_ready);
                if (!(ok = mbar_wait(&sm.bar.tbl_ready, exact_tasks & 1, limit, abort_flag, p.status))) break;
            }
            const float g_chunk = fast ? gpow(cd.n_last) : sm.pw[cd.n_last];   // gamma^N

            // ---- operand scaling that the dS MMAs wait for ---------------------------------------
            bool s_seen = false;
            if (fast) {
                // V~ = diag(gamma^(N - n_j)) V, in place
                if (!(ok = mbar_wait(&sm.bar.full[s], (g / kStages) & 1, limit, abort_flag, p.status))) break;
                scale_row_inplace<4>(sm.v[s] + i * 128, gpow(cd.n_last - cd.ni), 4 * grp, i & 7);
            } else {
                // K~ = diag(gamma^(N - n_j)) K, in place, once M1 has read K
                if (!(ok = mbar_wait(&sm.bar.s_done, par, limit, abort_flag, p.status))) break;
                tc_fence_after();
                s_seen = true;
                if (grp == 1) scale_row_inplace<8>(sm.k[s] + i * 128, sm.pw[cd.n_last - cd.ni], 0, i & 7);
            }
            fence_proxy_async();
            mbar_arrive(&sm.bar.x_ready);

            // ---- E1: A = tril(S) (normal) or P = S o gamma^(n_i - n_j) o [j <= i] (exact) -> bf16
            //      over S's own columns, in 16-column pieces.  This warp converts the blocks 2 grp
            //      and 2 grp + 1 of its rows and keeps the result inside its own half of S's columns
            //      (always behind its own reads); the A V MMAs walk the columns in that order.  It
            //      needs no state and fills the time the dS MMAs and the relay take.
            if (!s_seen) {
                if (!(ok = mbar_wait(&sm.bar.s_done, par, limit, abort_flag, p.status))) break;
                tc_fence_after();
            }
            if (fast) {
#pragma unroll
                for (int q16 = 0; q16 < 4; ++q16) {      // 16-column pieces of blocks 2 grp, 2 grp + 1
                    const int pc = 2 * grp + (q16 >> 1);
                    const int c0 = 16 * (q16 & 1);           // first column of the piece inside its block
                    uint32_t pk[8];
                    if (pc <= qd) {
                        uint32_t sv[16];
                        tmem_ld16(tmem + lane_base + kColS + 32 * pc + c0, sv);
                        tmem_wait_ld();
                        if (pc < qd) {
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                pk[c] = pack_bf16(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1]));
                        } else {
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                pk[c] = pack_bf16(c0 + 2 * c <= lane ? __uint_as_float(sv[2 * c]) : 0.0f,
                                                  c0 + 2 * c + 1 <= lane ? __uint_as_float(sv[2 * c + 1]) : 0.0f);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 8; ++c) pk[c] = 0u;
                    }
                    tmem_st8(tmem + lane_base + kColS + 64 * grp + 8 * q16, pk);
                }
            } else {
#pragma unroll 1
                for (int q16 = 0; q16 < 4; ++q16) {
                    const int pc = 2 * grp + (q16 >> 1);
                    const int c0 = 16 * (q16 & 1);
                    uint32_t pk[8];
                    if (pc <= qd) {
                        uint32_t sv[16];
                        tmem_ld16(tmem + lane_base + kColS + 32 * pc + c0, sv);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const int j0 = 32 * pc + c0 + 2 * c;
                            const int d0 = cd.ni - cd.n_of(j0), d1 = cd.ni - cd.n_of(j0 + 1);
                            const float v0 = j0 <= i ? __uint_as_float(sv[2 * c]) * sm.pw[d0 > 0 ? d0 : 0] : 0.0f;
                            const float v1 = j0 + 1 <= i ? __uint_as_float(sv[2 * c + 1]) * sm.pw[d1 > 0 ? d1 : 0] : 0.0f;
                            pk[c] = pack_bf16(v0, v1);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 8; ++c) pk[c] = 0u;
                    }
                    tmem_st8(tmem + lane_base + kColS + 64 * grp + 8 * q16, pk);
                }
                if (grp == 0) scale_row_inplace<8>(sm.q[s] + i * 128, sm.pw[cd.ni], 0, i & 7);   // Q~
            }
            tmem_wait_st();
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&sm.bar.p_ready);
            if (!fast) {
                mbar_arrive(&sm.bar.tbl_free);    // last use of the table in this task
                ++exact_tasks;
            }

            // ---- state section, the only serial link along a chain: take the incoming state
            //      (waiting for it if it is not here yet), copy it for the Q x state MMAs,
            //      E3: S_new = gamma^N S_prev + dS, hand S_new on at once
            if (!(ok = mbar_wait(&sm.bar.ds_done, par, limit, abort_flag, p.status))) break;
            tc_fence_after();
            // (the request is not issued earlier in the task: holding its 32 registers across E1
            // costs more in spills than the exposed trip from L2)
            unsigned long long rv[16];
            if (relayed_in) relay_request(slot, rv);
            if (!relayed_in) {
                if (p.state_in) {
                    load_state(p.state_in + (size_t)t.x * (kD * kD));
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) st[e] = 0.0f;
                }
            } else if (!relay_accept(rv, tag_in)) {
                // not here yet: poll one word per warp, then read the warp's words again
                bool got = false;
                for (unsigned it = 0; it < limit; ++it) {
                    if (relay_peek(slot, tag_in)) {
                        relay_request(slot, rv);
                        if (relay_accept(rv, tag_in)) { got = true; break; }
                    }
                    if ((it & 15u) == 15u && *abort_flag) break;
                    __nanosleep(32);
                }
                if (!got) {
                    if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, 1); }
                    ok = false;
                    break;
                }
            }
            // gamma^N S_prev (normal) / S_prev (exact: Q~ carries gamma^n_i)
            write_state_bf16(fast ? g_chunk : 1.0f);
            fence_proxy_async();
            mbar_arrive(&sm.bar.sb_ready);
            update_state(g_chunk);
            if (!last_chunk) {
                relay_out(slot, tag_out);
            } else if (p.state_out) {
                store_state(p.state_out + (size_t)t.x * (kD * kD));
            }

            // ---- E2: o_i = scale * gamma^-(N - n_i) * O'_i (normal) / scale * O_i (exact) -----------
            const float out_f = fast ? p.scale * gpow(-(cd.n_last - cd.ni)) : p.scale;
            if (!(ok = mbar_wait(&sm.bar.o_done, par, limit, abort_flag, p.status))) break;
            tc_fence_after();
            stage_output(s, out_f);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&sm.bar.st_ready[s]);

        }
    }

    // ---- teardown ---------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    // the last CTA to leave puts the counters back to zero for the next launch
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(p.work + 1, 1) == (int)gridDim.x - 1) {
            p.work[0] = 0;
            p.work[1] = 0;
            __threadfence();
        }
    }
}

}  // namespace

int prefill_stream_chunks(int T) { return (T + kC - 1) / kC; }

// Largest grid whose CTAs are all resident at once on `device`, from the device's shared-memory,
// register and thread limits and the kernel's own needs: the grid size that keeps every SM busy
// without CTAs queueing behind one another (the kernel is correct at any grid size).
int prefill_stream_max_ctas(int device)
{
    static int cached[64] = {0};
    if (device >= 0 && device < 64 && cached[device] > 0) return cached[device];
    const size_t smem = sizeof(Smem) + 1024;
    int sms = 0, smem_sm = 0, smem_reserved = 0, regs_sm = 0, threads_sm = 0;
    cudaFuncAttributes fa;
    if (cudaFuncSetAttribute(prefill_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncGetAttributes(&fa, prefill_stream_kernel) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&smem_reserved, cudaDevAttrReservedSharedMemoryPerBlock, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&regs_sm, cudaDevAttrMaxRegistersPerMultiprocessor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&threads_sm, cudaDevAttrMaxThreadsPerMultiProcessor, device) != cudaSuccess)
        return 0;
    const int by_smem = smem_sm / (int)(smem + fa.sharedSizeBytes + smem_reserved);
    const int regs_block = ((fa.numRegs * 32 + 255) / 256 * 256) * (kThreads / 32);   // allocated per warp in units of 256
    const int by_regs = regs_block > 0 ? regs_sm / regs_block : 0;
    const int by_threads = threads_sm / kThreads;
    // TMEM: 512 columns per SM, kTmemCols per CTA
    int per_sm = min(min(by_smem, by_regs), min(by_threads, 512 / kTmemCols));
    const int n = per_sm * sms;
    if (device >= 0 && device < 64) cached[device] = n;
    return n;
}

cudaError_t launch_prefill_stream(const KernelArgs& a, const TcRelay& r, cudaStream_t st)
{
    CUtensorMap mq, mk, mv, mo;
    if (!encode_chunk_map(&mq, a.q, a.B, a.T, a.H, a.qs) || !encode_chunk_map(&mk, a.k, a.B, a.T, a.H, a.ks) ||
        !encode_chunk_map(&mv, a.v, a.B, a.T, a.H, a.vs) || !encode_chunk_map(&mo, a.o, a.B, a.T, a.H, a.os))
        return cudaErrorInvalidValue;
    StreamParams p;
    p.B = a.B; p.T = a.T; p.H = a.H;
    p.X = a.B * a.H;
    p.n_chunks = prefill_stream_chunks(a.T);
    p.n_tasks = p.X * p.n_chunks;
    p.grid_w = a.grid_w; p.prefix_len = a.prefix_len; p.t0 = a.t0; p.scale = a.scale;
    p.decay = a.decay; p.state_in = a.state_in; p.state_out = a.state_out;
    p.relay = static_cast<uint4*>(r.relay); p.epoch16 = r.epoch16;
    p.work = a.work;
    p.status = a.status; p.wait_limit = a.wait_limit;
    if (r.max_ctas <= 0 || (p.n_chunks > 1 && !p.relay) || !p.work) return cudaErrorInvalidValue;
    const size_t smem = sizeof(Smem) + 1024;
    static bool smem_ok_1[64];
    cudaError_t e = allow_dynamic_smem(prefill_stream_kernel, smem, smem_ok_1);
    if (e != cudaSuccess) return e;
    const int grid = p.n_tasks < r.max_ctas ? p.n_tasks : r.max_ctas;
    // programmatic dependent launch (see the kernel's first lines)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, prefill_stream_kernel, mq, mk, mv, mo, p);
}

}  // namespace lasad

// ---------------------------------------------------------------------------------------------
// Allocation-free prefill entry point (declared in lasad.h)
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticUnits = 256;   // (batch, head) pairs the built-in relay storage covers

// Relay slots for kStaticUnits chains (8 MiB) followed by one 256-byte status block.  It lives in
// the library image: every device that loads the library holds it until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticUnits * lasad::kTcRelaySlotBytes + 256];

struct StaticState {
    void* scratch = nullptr;        // device address of g_static_scratch on this device
    int max_ctas = 0;
    unsigned long long epoch = 0;   // launches through the allocation-free entry point on this device
};
StaticState g_static_state[64];
std::mutex g_static_mutex;

}  // namespace

extern "C" int lasad_forward_static(const lasad_params* p, const void* q, const void* k, const void* v,
                                    const float* decay, const float* state_in, void* o, float* state_out,
                                    int* device_status, void* cuda_stream)
{
    // ---- argument checks (the same rules as lasad_forward, restricted to what this path runs) ----
    if (!p || !q || !k || !v || !o || !decay) return LASAD_ERR_INVALID_ARG;
    if (p->B <= 0 || p->H <= 0 || p->T <= 0 || p->dk <= 0 || p->dv <= 0) return LASAD_ERR_INVALID_ARG;
    if (p->grid_w < 0 || p->prefix_len < 0 || p->t0 < 0 || p->reserved != 0) return LASAD_ERR_INVALID_ARG;
    if (!std::isfinite(p->scale)) return LASAD_ERR_INVALID_ARG;
    if (p->dtype != LASAD_F32 && p->dtype != LASAD_BF16) return LASAD_ERR_INVALID_ARG;
    auto aligned16 = [](const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; };
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return LASAD_ERR_INVALID_ARG;
    if ((state_in && !aligned16(state_in)) || (state_out && !aligned16(state_out))) return LASAD_ERR_INVALID_ARG;
    if (device_status && (reinterpret_cast<uintptr_t>(device_status) & 3u)) return LASAD_ERR_INVALID_ARG;
    const int64_t* strides[4] = {p->q_stride, p->k_stride, p->v_stride, p->o_stride};
    for (int s = 0; s < 4; ++s) {
        for (int d = 0; d < 3; ++d)
            if (strides[s][d] < 0 || (strides[s][d] * 2) % 16 != 0) return LASAD_ERR_INVALID_ARG;
        if (strides[s][2] < 64 && p->H > 1) return LASAD_ERR_INVALID_ARG;
        if ((strides[s][0] == 0 && p->B > 1) || (strides[s][1] == 0 && p->T > 1)) return LASAD_ERR_INVALID_ARG;
    }
    if (p->dtype != LASAD_BF16 || p->dk != 64 || p->dv != 64) return LASAD_ERR_UNSUPPORTED;
    const int64_t units = (int64_t)p->B * p->H;
    if (units > kStaticUnits) return LASAD_ERR_UNSUPPORTED;     // beyond the built-in relay storage
    if (units * lasad::prefill_stream_chunks(p->T) > 0x7fffffffLL) return LASAD_ERR_UNSUPPORTED;

    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return LASAD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticState& st = g_static_state[device];
    if (!st.scratch) {
        // once per device, with that device current: the symbol's name is only a host-side handle;
        // the kernel needs the array's address on this device
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return LASAD_ERR_CUDA;
        const int n = lasad::prefill_stream_max_ctas(device);
        if (n <= 0) return LASAD_ERR_CUDA;
        st.scratch = ptr;
        st.max_ctas = n;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The relay packets are tagged with a call number that this function counts on the host: a
    // call recorded into a CUDA graph would replay with the number it was recorded with and could
    // take the previous replay's packets for its own.  So a stream that is being captured is refused.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) return LASAD_ERR_CUDA;
    if (cap != cudaStreamCaptureStatusNone) return LASAD_ERR_UNSUPPORTED;
    unsigned char* base = static_cast<unsigned char*>(st.scratch);
    const size_t relay_bytes = (size_t)kStaticUnits * lasad::kTcRelaySlotBytes;

    lasad::KernelArgs a{};
    a.B = p->B; a.T = p->T; a.H = p->H;
    a.grid_w = p->grid_w; a.prefix_len = p->prefix_len; a.t0 = p->t0; a.scale = p->scale;
    for (int d = 0; d < 3; ++d) {
        a.qs[d] = p->q_stride[d]; a.ks[d] = p->k_stride[d];
        a.vs[d] = p->v_stride[d]; a.os[d] = p->o_stride[d];
    }
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.decay = decay; a.state_in = state_in; a.state_out = state_out;
    a.status = device_status ? device_status : reinterpret_cast<int*>(base + relay_bytes);
    a.work = reinterpret_cast<int*>(base + relay_bytes) + 16;      // two counters the kernel keeps at zero between launches
    a.wait_limit = 1u << 22;

    lasad::TcRelay r{};
    r.relay = base;
    // The slots keep the packets of earlier calls; their tags carry the call number modulo 65535,
    // so before a number comes round again the slots are cleared (they also start out as zeros,
    // and no tag is ever zero).
    st.epoch += 1;
    r.epoch16 = (unsigned)(st.epoch % 65535u) + 1u;
    if (st.epoch % 65535u == 0 && cudaMemsetAsync(base, 0, relay_bytes, stream) != cudaSuccess) return LASAD_ERR_CUDA;
    r.max_ctas = st.max_ctas;
    return lasad::launch_prefill_stream(a, r, stream) == cudaSuccess ? LASAD_OK : LASAD_ERR_CUDA;
}

