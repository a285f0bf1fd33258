// LASAD chunked prefill on the 5th-generation tensor cores (sm_100a), balanced over the SMs:
// one CTA per SM runs TWO chunk pipelines that take the chunks of ONE chain alternately.
//
// The chunk algebra is that of lasad_prefill_tc.cu (C = 128 tokens; SAD recurrence of Section 3.4
// unrolled over a chunk; all decay on V and one output row factor for gamma >= 0.6, factors with
// non-negative exponents only below that).  What differs is who works on what:
//
//   * Everything in a chunk but the carried state is independent of the other chunks of its
//     chain -- the scores Q K^T, the causal mask, A V~, and also dS = K^T V~.  Only
//     S_n = gamma^N S_{n-1} + dS_n and the term Q (gamma^N S_{n-1}) of the output tie a chunk to
//     its predecessor.  So the two pipelines of a CTA (each: eight element-wise warps, an MMA
//     warp, a TMA warp, 256 TMEM columns, two tile stages) work on chunks n and n+1 of the same
//     chain at the same time, and the fp32 state passes between them through a 16 KiB
//     shared-memory buffer once per chunk (one mbarrier each way).  A single chain then runs at
//     the speed of the whole SM, not at half of it.
//   * With that, the work can be cut evenly without leaving the order in which memory likes to
//     be read.  q, k, v are [B,T,H,d]: the heads of one token lie side by side, so DRAM is read
//     well only while neighbouring heads are worked on at about the same token at about the same
//     time (measured: CTAs that walk unrelated stretches of the sequence lose a quarter of the
//     bandwidth).  So with S CTAs and n = m S + E chains, CTA c takes the chains rho(c), S + rho(c),
//     2 S + rho(c), ... one after the other -- all CTAs move through their chains in step -- and
//     the E chains that are left over are cut into S equal pieces, one per CTA, which the CTA
//     slips into its first chain at the moment the piece's turn comes: piece k of a left-over
//     chain starts at chunk k L, so it is taken up when the CTA's own chain has reached about
//     chunk k L, and it too moves in step with the rest.  The left-over chain's state travels
//     from CTA to CTA through a slot in global memory (see "hand-off" below); the CTA's own
//     chain waits in a slot of its own meanwhile.  rho orders the CTAs by the time at which they
//     take up their piece, so that the chains that have been held up for a piece are neighbours too.
//   * CTAs number themselves in the order they start (an atomic ticket).  CTA c only ever waits
//     for the piece before its own, which is CTA c-1's; that CTA started before it and waits for
//     nothing but the piece before that: progress needs no assumption about which CTAs are
//     resident together.
//
// Hand-off: the 4096 state values travel as 8-byte (value, tag) packets, two per 16-byte access,
// written and read with plain L2 accesses; the tag is the launch's number, counted on the device,
// so a packet of an earlier launch never passes for this one's, also when a captured launch is
// replayed.  An aligned 8-byte access is single-copy atomic, so a packet is either old or new as a
// whole, and the receiver polls its own sixteen packets until all carry the tag: no fence and no
// flag (a membar here stalls for microseconds while the SM's bulk copies are in flight).
//
// All waits are bounded: a wait that runs out raises a status word the host can read and the CTA
// leaves through the normal exit (copies in flight are waited for, TMEM is freed).
#include "lasad_common.cuh"
#include "lasad_tc_chunk.cuh"
#include "lasad_tc_pair_plan.cuh"
#include "lasad_tc_ptx.cuh"
#include "lasad_tc_tma.cuh"

namespace lasad {
namespace {

using namespace tcx;

constexpr int kStages = 2;
constexpr int kPipeThreads = kEThreads + 64;    // element-wise warps, the MMA warp, the TMA warp
constexpr int kPairThreads = 2 * kPipeThreads;
constexpr int kPipeTmemCols = 256;

struct __align__(8) PipeBarriers {
    unsigned long long full[kStages];      // TMA loads of a stage have landed
    unsigned long long s_done;             // M1 complete
    unsigned long long x_ready;            // V~ (normal path) or K~ (exact path) written: dS may start (256 arrivals)
    unsigned long long ds_done;            // dS MMAs complete
    unsigned long long p_ready;            // A/P in TMEM (and Q~ in smem) (256 arrivals)
    unsigned long long sb_ready;           // bf16 copy of the incoming state in smem (256 arrivals)
    unsigned long long o_done[kStages];    // O MMAs complete (and every MMA issued before them)
    unsigned long long st_ready[kStages];  // output tile staged in smem (256 arrivals)
    unsigned long long state_ready;        // this pipeline's chunk has left its state in `sf` (256 arrivals)
    unsigned long long tbl;                // exact path: the decay table may change / has changed (256 arrivals)
    unsigned long long drain;              // teardown: all MMAs retired
};

struct Smem {
    // tiles first: each must sit on a 1024-byte boundary (128-byte swizzle atom = 8 rows)
    unsigned char q[2][kStages][kTileBytes];
    unsigned char k[2][kStages][kTileBytes];
    unsigned char v[2][kStages][kTileBytes];
    unsigned char sb[2][kD * kD * 2];   // per pipeline: bf16 copy of the incoming state, [dk][dv], 128 B rows, swizzled
    float4 sf[4][kEThreads];            // the fp32 state between two chunks: element-wise thread t's 16 values
    float pw[2][kC + 4];                // exact path: gamma^m, m = 0..128, of the pipeline's current head
    PipeBarriers bar[2];
    Plan plan;
    uint32_t tmem_base;
    int abort_flag;
    int cta;                            // this CTA's number in start order
    unsigned tag;                       // this launch's packet tag
};

struct PairParams {
    int B, T, H;
    int grid_w, prefix_len;
    long long t0;
    float scale;
    const float* decay;
    const float* state_in;
    float* state_out;
    int* work;        // [3]: CTAs that have started, CTAs that have left (both zero between launches), launches so far
    unsigned char* slots;   // [2 n_ctas][kSlotBytes], as packets: slot c the state entering CTA c's piece of a
                            // left-over chain, slot n_ctas + c CTA c's own first chain while it works on the piece
    int nc;           // chunks per chain
    int chains;       // B x H
    int* status;
    unsigned wait_limit;
};

__global__ void __launch_bounds__(kPairThreads, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, PairParams p)
{
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    // CTA warps 0-9 are pipeline 0, 10-19 pipeline 1.  A warp reaches the TMEM lanes of quadrant
    // (its index in the CTA) mod 4, so the second pipeline's roles are rotated by two: its MMA and
    // TMA warps are CTA warps 10 and 11 and its element-wise warps 12-19, which again sit on
    // quadrants 0..3 in order.  `warp` is the role: 0-7 element-wise, 8 MMA, 9 TMA.
    const int X = threadIdx.x >= kPipeThreads ? 1 : 0;   // which of the CTA's two pipelines
    const int lane = threadIdx.x & 31;
    const int warp = X ? (int)((threadIdx.x >> 5) - 2) % 10 : (int)(threadIdx.x >> 5);
    const int tid = warp * 32 + lane;                    // element-wise warps: thread 0..255 of the pipeline
    volatile int* abort_flag = &sm.abort_flag;
    const unsigned limit = p.wait_limit;
    PipeBarriers& bar = sm.bar[X];

    // ---- set-up ---------------------------------------------------------------------------
    // A kernel launched behind this one as a programmatic dependent may start to take SMs as they
    // become free; it waits for this kernel's completion before it touches device memory.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) {
        for (int x = 0; x < 2; ++x) {
            PipeBarriers& b = sm.bar[x];
            for (int s = 0; s < kStages; ++s) {
                mbar_init(&b.full[s], 1);
                mbar_init(&b.o_done[s], 1);
                mbar_init(&b.st_ready[s], kEThreads);
            }
            mbar_init(&b.s_done, 1);
            mbar_init(&b.x_ready, kEThreads);
            mbar_init(&b.ds_done, 1);
            mbar_init(&b.p_ready, kEThreads);
            mbar_init(&b.sb_ready, kEThreads);
            mbar_init(&b.state_ready, kEThreads);
            mbar_init(&b.tbl, kEThreads);
            mbar_init(&b.drain, 1);
        }
        // nothing above reads or writes device memory; everything below may depend on the kernel
        // before this one in the stream (its outputs, the work counters it puts back to zero)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        sm.abort_flag = 0;
        sm.cta = atomicAdd(p.work, 1);
        sm.tag = ((unsigned)*reinterpret_cast<volatile int*>(p.work + 2) & 0x3fffffffu) + 1u;   // never 0, the slots' initial content
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9 && lane == 0) {
        // the descriptors' first use then finds them in the descriptor cache
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_q)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_v)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_o)) : "memory");
        // The CTAs' first chains are chains 0 .. gridDim.x - 1 in some order (which CTA takes which
        // is known only after the ticket): ask for the first chunks of chain blockIdx.x to be brought
        // into L2 now, while the launch before this one is still finishing.  A prefetch hands no
        // data to the SM, so it may run ahead of the wait below; whoever takes the chain finds its
        // first tiles in L2.
        if (X == 0) {
            const int pb = (int)blockIdx.x / p.H, ph = (int)blockIdx.x - pb * p.H;
            for (int n = 0; n < min(2 * kStages, p.nc); ++n) {
                tma_prefetch_4d(&tm_k, 0, ph, n * kC, pb);
                tma_prefetch_4d(&tm_v, 0, ph, n * kC, pb);
                tma_prefetch_4d(&tm_q, 0, ph, n * kC, pb);
            }
        }
    }
    if (threadIdx.x >> 5 == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(2 * kPipeTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();
    build_plan(sm.plan, sm.cta, p.chains, p.nc, kPairThreads);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base + (uint32_t)(X * kPipeTmemCols);
    const Plan& plan = sm.plan;
    // this pipeline's chunks are the local chunks g = 2 j + X, j = 0 .. J-1
    const int J = plan.n_local > X ? (plan.n_local - X + 1) / 2 : 0;

    if (warp == 9) {
        // ===================== TMA warp: loads two chunks ahead, stores each output tile =======
        if (elect_one() && J > 0) {
            Unit lu, su;
            lu.g0 = 0; lu.g1 = -1; su.g0 = 0; su.g1 = -1;
            int ld_b = 0, ld_h = 0, ld_tok = 0;
            int issued = 0;
            auto issue_kv = [&](int j) {
                const int s = j % kStages, g = 2 * j + X;
                if (g >= lu.g1) lu = unit_of(plan, g);
                ld_b = lu.chain / p.H;
                ld_h = lu.chain - ld_b * p.H;
                ld_tok = (lu.n0 + g - lu.g0) * kC;
                mbar_arrive_expect_tx(&bar.full[s], 3 * kTileBytes);
                tma_load_4d(sm.k[X][s], &tm_k, &bar.full[s], 0, ld_h, ld_tok, ld_b);
                tma_load_4d(sm.v[X][s], &tm_v, &bar.full[s], 0, ld_h, ld_tok, ld_b);
            };
            auto issue_q = [&](int j) {
                tma_load_4d(sm.q[X][j % kStages], &tm_q, &bar.full[j % kStages], 0, ld_h, ld_tok, ld_b);
                issued = j + 1;
            };
            for (int j = 0; j < min(J, kStages); ++j) {
                issue_kv(j);
                issue_q(j);
            }
            for (int j = 0; j < J; ++j) {
                const int s = j % kStages, g = 2 * j + X;
                const bool refill = j + kStages < J;
                if (!mbar_wait(&bar.o_done[s], (j / kStages) & 1, limit, abort_flag, p.status)) break;
                // K and V of the stage are free once every MMA of the chunk has retired, Q (whose
                // buffer stages the output tile) once the store has read it
                if (refill) issue_kv(j + kStages);
                const bool staged = mbar_wait(&bar.st_ready[s], (j / kStages) & 1, limit, abort_flag, p.status);
                if (staged) {
                    if (g >= su.g1) su = unit_of(plan, g);
                    const int b = su.chain / p.H, h = su.chain - b * p.H;
                    tma_store_4d(&tm_o, sm.q[X][s], 0, h, (su.n0 + g - su.g0) * kC, b);
                    tma_store_commit();
                    if (refill) tma_store_wait_read();    // the store has finished reading the buffer
                }
                if (refill) issue_q(j + kStages);          // (also after a failed wait: the stage's barrier must complete)
                if (!staged) break;
            }
            tma_store_wait_all();
            // leave only when every issued load has landed (they write this CTA's shared memory)
            for (int j = max(0, issued - kStages); j < issued; ++j)
                for (unsigned it = 0; it < kTeardownLimit; ++it)
                    if (mbar_try_wait(&bar.full[j % kStages], (j / kStages) & 1)) break;
        }
        __syncwarp();
    } else if (warp == 8) {
        // ===================== MMA issuer: the whole warp runs the loop, one lane issues =======
        constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);   // Q (K-major) x K (K-major)
        constexpr uint32_t idesc_pv = make_idesc(128, 64, 0, 1);   // A/P (tmem) x V (MN-major)
        constexpr uint32_t idesc_qs = make_idesc(128, 64, 0, 1);   // Q (K-major) x state (MN-major)
        constexpr uint32_t idesc_kv = make_idesc(64, 64, 1, 1);    // K^T (MN-major) x V (MN-major)
        const uint64_t d_sb = make_desc(smem_u32(sm.sb[X]));
        const uint64_t dq0 = make_desc(smem_u32(sm.q[X][0])), dq1 = make_desc(smem_u32(sm.q[X][1]));
        const uint64_t dk0 = make_desc(smem_u32(sm.k[X][0])), dk1 = make_desc(smem_u32(sm.k[X][1]));
        const uint64_t dv0 = make_desc(smem_u32(sm.v[X][0])), dv1 = make_desc(smem_u32(sm.v[X][1]));
        // scores of chunk j as soon as its tiles are in
        auto issue_m1 = [&](int j) {
            const int s = j % kStages;
            const uint64_t dqs = s ? dq1 : dq0, dks = s ? dk1 : dk0;
            if (!mbar_wait(&bar.full[s], (j / kStages) & 1, limit, abort_flag, p.status)) return false;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)  // 32 bytes along K per step
                    mma_ss(tmem + kColS, dqs + 2 * kk, dks + 2 * kk, idesc_s, kk > 0);
                mma_commit(&bar.s_done);
            }
            __syncwarp();
            return true;
        };
        bool ok = J > 0 && issue_m1(0);
        for (int j = 0; ok && j < J; ++j) {
            const int s = j % kStages;
            const uint64_t dqs = s ? dq1 : dq0, dks = s ? dk1 : dk0, dvs = s ? dv1 : dv0;
            if (!mbar_wait(&bar.x_ready, j & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // 16 tokens = 2048 B of K and of V per step
                    mma_ss(tmem + kColDS, dks + 128 * kk, dvs + 128 * kk, idesc_kv, kk > 0);
                mma_commit(&bar.ds_done);
            }
            __syncwarp();
            if (!mbar_wait(&bar.p_ready, j & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // A/P: 8 TMEM columns per step (tokens 0..63 at columns
                                                      // 0..31, tokens 64..127 at 64..95); V: 2048 B per step
                    mma_ts(tmem + kColO, tmem + kColS + (kk < 4 ? 8 * kk : 64 + 8 * (kk - 4)), dvs + 128 * kk,
                           idesc_pv, kk > 0);
            }
            __syncwarp();
            // the carried state's share of O comes last: it is the only part that has to wait for
            // the other pipeline's chunk
            if (!mbar_wait(&bar.sb_ready, j & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)
                    mma_ss(tmem + kColO, dqs + 2 * kk, d_sb + 128 * kk, idesc_qs, 1);
                mma_commit(&bar.o_done[s]);
            }
            __syncwarp();
            if (j + 1 < J) ok = issue_m1(j + 1);
        }
        // make sure nothing is still running on the tensor pipe before TMEM is freed
        if (elect_one()) {
            mma_commit(&bar.drain);
            for (unsigned it = 0; it < kTeardownLimit; ++it)
                if (mbar_try_wait(&bar.drain, 0)) break;
        }
        __syncwarp();
    } else if (J > 0) {
        // ===================== element-wise warps ==============================================
        const int qd = warp & 3;                 // TMEM lane quadrant
        const int grp = warp >> 2;               // which half of the quadrant's columns
        const int i = qd * 32 + lane;            // chunk row owned by this thread
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        // State ownership.  The dS accumulator (M = 64 layout) keeps state rows 16 qd .. 16 qd + 15 in
        // the first 16 TMEM lanes of quadrant qd; the 16x256b load spreads this warp's 16 rows x 32
        // columns (columns 32 grp ..) over all 32 threads, 16 values each: for column group k,
        // st[4k], st[4k+1] = (row r0, columns c0 + 8k, + 1), st[4k+2], st[4k+3] = (row r0 + 8, same).
        // Thread t of either pipeline owns the same 16 elements, so `sf` is private to the pair.
        const int r0 = qd * 16 + (lane >> 2);
        const int c0 = 32 * grp + 2 * (lane & 3);
        float* pw = sm.pw[X];
        PipeBarriers& other = sm.bar[1 - X];

        float st[16];
        // bf16 copy of mult * state for the Q x state MMA: [dk][dv] rows of 128 B, 16-byte pieces
        // swizzled by the row; this thread writes eight bf16 pairs
        auto write_state_bf16 = [&](float mult) {
            unsigned char* row0 = sm.sb[X] + r0 * 128 + 4 * (lane & 3);
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
        // E2: this thread's 32 columns of output row i -> bf16 -> the stage's Q buffer
        auto stage_output = [&](int s, float f) {
            unsigned char* orow = sm.q[X][s] + i * 128;
            uint32_t ov[32];
            tmem_ld32(tmem + lane_base + kColO + 32 * grp, ov);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float x0, x1;
                    mul2(__uint_as_float(ov[8 * c + 2 * e]), __uint_as_float(ov[8 * c + 2 * e + 1]), f, x0, x1);
                    w[e] = pack_bf16(x0, x1);
                }
                reinterpret_cast<uint4*>(orow)[(4 * grp + c) ^ (i & 7)] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        };

        // ---- the chunk this pipeline is working on ------------------------------------------------
        Unit u;
        u.g0 = 0; u.g1 = -1;
        int n = 0;                      // its index within the chain
        int cs = 0;                     // its token offset within the run `gp` was set up for
        float gamma = 1.0f, lg = 0.0f;
        bool fast = true;
        int tbl_head = -1;              // head whose table is in pw
        unsigned tbl_phase = 0;         // completed phases of the table barrier
        GridPos gp = grid_pos_init(0, 0, 0, lane);
        ChunkDecay cd;
        bool ok = true;
        auto gpow = [&](int m) { return ex2_approx((float)m * lg); };
        // makes local chunk g current: unit, decay constants, decay bookkeeping (and, on the exact
        // path, the table of gamma^m by binary exponentiation in double precision, 0^0 = 1)
        auto enter = [&](int g) {
            if (g >= u.g1) {
                u = unit_of(plan, g);
                n = u.n0 + g - u.g0;
                if (u.recv >= (int)gridDim.x) park_prefetch(p.slots + (size_t)u.recv * kSlotBytes, tid);
                else if (u.recv >= 0) slot_prefetch(p.slots + (size_t)u.recv * kSlotBytes, tid);
                const int h = u.chain % p.H;
                gamma = p.decay[h];
                fast = gamma >= kFastPathMinDecay;
                lg = fast ? log2f(gamma) : 0.0f;
                gp = grid_pos_init(p.grid_w, p.prefix_len, p.t0 + (long long)n * kC, lane);
                cs = 0;
                if (!fast && tbl_head != h) {
                    // every thread is done with the previous table before it changes
                    mbar_arrive(&bar.tbl);
                    if (!(ok = mbar_wait(&bar.tbl, tbl_phase & 1, limit, abort_flag, p.status))) return;
                    ++tbl_phase;
                    if (tid <= kC) {
                        double base = (double)gamma, acc = 1.0;
                        for (int e = tid; e > 0; e >>= 1) {
                            if (e & 1) acc *= base;
                            base *= base;
                        }
                        pw[tid] = (float)acc;
                    }
                    mbar_arrive(&bar.tbl);
                    if (!(ok = mbar_wait(&bar.tbl, tbl_phase & 1, limit, abort_flag, p.status))) return;
                    ++tbl_phase;
                    tbl_head = h;
                }
            } else {
                n += 2;
                gp.skip();              // the other pipeline's chunk in between
                cs += 2 * kC;
            }
            cd = chunk_decay(gp, cs, min(kC, p.T - n * kC), qd, lane);
        };
        // normal path: V~ = diag(gamma^(N - n_j)) V of the current chunk, in place, once its tiles are in
        auto scale_v = [&](int j) {
            const int s = j % kStages;
            if (!(ok = mbar_wait(&bar.full[s], (j / kStages) & 1, limit, abort_flag, p.status))) return;
            scale_row_inplace<4>(sm.v[X][s] + i * 128, gpow(cd.n_last - cd.ni), 4 * grp, i & 7);
            fence_proxy_async();
            mbar_arrive(&bar.x_ready);
        };

        enter(X);
        if (ok && fast) scale_v(0);
        for (int j = 0; ok && j < J; ++j) {
            const int s = j % kStages, g = 2 * j + X;
            if (!(ok = mbar_wait(&bar.s_done, j & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
            if (fast) {
                // ---- E1: A = tril(S) -> bf16 over S's own columns.  This warp converts the
                //      32-column blocks 2 grp and 2 grp + 1 of its rows and keeps the result inside
                //      its own half of S's columns (block pc -> columns 64 grp + 16 (pc & 1), always
                //      behind this warp's own reads); the A V~ MMAs walk the columns in that order.
#pragma unroll
                for (int pi = 0; pi < 2; ++pi) {
                    const int pc = 2 * grp + pi;
                    uint32_t pk[16];
                    if (pc <= qd) {
                        uint32_t sv[32];
                        tmem_ld32(tmem + lane_base + kColS + 32 * pc, sv);
                        tmem_wait_ld();
                        if (pc < qd) {
#pragma unroll
                            for (int c = 0; c < 16; ++c)
                                pk[c] = pack_bf16(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1]));
                        } else {
#pragma unroll
                            for (int c = 0; c < 16; ++c)
                                pk[c] = pack_bf16(2 * c <= lane ? __uint_as_float(sv[2 * c]) : 0.0f,
                                                  2 * c + 1 <= lane ? __uint_as_float(sv[2 * c + 1]) : 0.0f);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; ++c) pk[c] = 0u;
                    }
                    tmem_st16(tmem + lane_base + kColS + 64 * grp + 16 * pi, pk);
                }
                tmem_wait_st();
            } else {
                // ---- exact path: K~ = diag(gamma^(N - n_j)) K first (M1 has finished reading K): it
                //      unblocks the dS MMAs; then P = S o gamma^(n_i - n_j) o [j <= i] from the table
                //      and Q~ = diag(gamma^(n_i)) Q in place
                if (grp == 1) scale_row_inplace<8>(sm.k[X][s] + i * 128, pw[cd.n_last - cd.ni], 0, i & 7);
                fence_proxy_async();
                mbar_arrive(&bar.x_ready);
#pragma unroll 1
                for (int pi = 0; pi < 2; ++pi) {
                    const int pc = 2 * grp + pi;
                    uint32_t pk[16];
                    if (pc <= qd) {
                        uint32_t sv[32];
                        tmem_ld32(tmem + lane_base + kColS + 32 * pc, sv);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int j0 = 32 * pc + 2 * c;
                            const int d0 = cd.ni - cd.n_of(j0), d1 = cd.ni - cd.n_of(j0 + 1);
                            const float v0 = j0 <= i ? __uint_as_float(sv[2 * c]) * pw[d0 > 0 ? d0 : 0] : 0.0f;
                            const float v1 = j0 + 1 <= i ? __uint_as_float(sv[2 * c + 1]) * pw[d1 > 0 ? d1 : 0] : 0.0f;
                            pk[c] = pack_bf16(v0, v1);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; ++c) pk[c] = 0u;
                    }
                    tmem_st16(tmem + lane_base + kColS + 64 * grp + 16 * pi, pk);
                }
                if (grp == 0) scale_row_inplace<8>(sm.q[X][s] + i * 128, pw[cd.ni], 0, i & 7);
                tmem_wait_st();
                fence_proxy_async();
            }
            tc_fence_before();
            mbar_arrive(&bar.p_ready);

            // ---- the carried state: in from the other pipeline's chunk (or from where the unit
            //      starts), out to the other pipeline's next chunk (or to where the unit ends) -------
            if (g > 0) {
                // the other pipeline is done with chunk g - 1 (its j index: j for X = 1, j - 1 for X = 0)
                if (!(ok = mbar_wait(&other.state_ready, (j - 1 + X) & 1, limit, abort_flag, p.status))) break;
            }
            const float g_chunk = fast ? gpow(cd.n_last) : pw[cd.n_last];     // gamma^N
            if (g == u.g0) {
                if (u.recv < 0) {
                    // a chain starts: the caller's state or zero
#pragma unroll
                    for (int e = 0; e < 16; ++e) st[e] = 0.0f;
                    if (p.state_in) {
                        const float* sin = p.state_in + (size_t)u.chain * kD * kD;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float2 a = *reinterpret_cast<const float2*>(sin + (size_t)r0 * kD + c0 + 8 * k);
                            const float2 c = *reinterpret_cast<const float2*>(sin + (size_t)(r0 + 8) * kD + c0 + 8 * k);
                            st[4 * k] = a.x; st[4 * k + 1] = a.y; st[4 * k + 2] = c.x; st[4 * k + 3] = c.y;
                        }
                    }
                } else {
                    // the chain was cut here: its state comes from where the part before it was done
                    if (u.recv >= (int)gridDim.x)
                        park_receive(p.slots + (size_t)u.recv * kSlotBytes, tid, st);
                    else if (!(ok = slot_receive(p.slots + (size_t)u.recv * kSlotBytes, tid, st, sm.tag, limit, abort_flag, p.status)))
                        break;
                }
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float4 x = sm.sf[k][tid];
                    st[4 * k] = x.x; st[4 * k + 1] = x.y; st[4 * k + 2] = x.z; st[4 * k + 3] = x.w;
                }
            }
            write_state_bf16(fast ? g_chunk : 1.0f);
            fence_proxy_async();
            mbar_arrive(&bar.sb_ready);
            // S_new = gamma^N S_prev + dS
            if (!(ok = mbar_wait(&bar.ds_done, j & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
            {
                uint32_t dsv[16];
                tmem_ld_16x256b_x4(tmem + lane_base + kColDS + 32 * grp, dsv);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 16; e += 2)
                    fma2(st[e], st[e + 1], g_chunk, __uint_as_float(dsv[e]), __uint_as_float(dsv[e + 1]), st[e], st[e + 1]);
            }
            if (g == u.g1 - 1) {
                if (u.send < 0) {
                    // the chain ends: its final state
                    if (p.state_out) {
                        float* dst = p.state_out + (size_t)u.chain * kD * kD;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            *reinterpret_cast<float2*>(dst + (size_t)r0 * kD + c0 + 8 * k) = make_float2(st[4 * k], st[4 * k + 1]);
                            *reinterpret_cast<float2*>(dst + (size_t)(r0 + 8) * kD + c0 + 8 * k) = make_float2(st[4 * k + 2], st[4 * k + 3]);
                        }
                    }
                } else {
                    // the chain is cut here: the state goes to where its next part will be done
                    if (u.send >= (int)gridDim.x) park_send(p.slots + (size_t)u.send * kSlotBytes, tid, st);
                    else slot_send(p.slots + (size_t)u.send * kSlotBytes, tid, st, sm.tag);
                }
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    sm.sf[k][tid] = make_float4(st[4 * k], st[4 * k + 1], st[4 * k + 2], st[4 * k + 3]);
            }
            tc_fence_before();
            mbar_arrive(&bar.state_ready);

            // ---- E2: o_i = scale * gamma^-(N - n_i) * O'_i (normal path; exact path: scale alone) --
            const float out_f = fast ? p.scale * gpow(-(cd.n_last - cd.ni)) : p.scale;
            const bool more = j + 1 < J;
            if (more) {
                enter(g + 2);
                if (!ok) break;
            }
            if (!(ok = mbar_wait(&bar.o_done[s], (j / kStages) & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
            stage_output(s, out_f);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&bar.st_ready[s]);
            // ---- V~ of this pipeline's next chunk, once its loads have landed.  This stage is
            //      released (st_ready above) before the wait, so the wait never holds a buffer back.
            if (more && fast) scale_v(j + 1);
        }
    }

    // ---- teardown ---------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x >> 5 == 8) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sm.tmem_base), "r"(2 * kPipeTmemCols)
                     : "memory");
    }
    // the last CTA to leave puts the counters back to zero for the next launch and counts this one
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(p.work + 1, 1) == (int)gridDim.x - 1) {
            p.work[0] = 0;
            p.work[1] = 0;
            p.work[2] += 1;
            __threadfence();
        }
    }
}

}  // namespace

size_t prefill_pair_scratch_bytes(int sms)
{
    // two hand-off slots per CTA
    return (size_t)2 * sms * kSlotBytes;
}

cudaError_t launch_prefill_pair(const KernelArgs& a, void* scratch, int sms, cudaStream_t st)
{
    const long long chains = (long long)a.B * a.H;
    const int nc = (a.T + kC - 1) / kC;
    if (chains * nc > 0x7fffffffLL || !scratch || sms <= 0) return cudaErrorInvalidValue;
    CUtensorMap mq, mk, mv, mo;
    if (!encode_chunk_map(&mq, a.q, a.B, a.T, a.H, a.qs) || !encode_chunk_map(&mk, a.k, a.B, a.T, a.H, a.ks) ||
        !encode_chunk_map(&mv, a.v, a.B, a.T, a.H, a.vs) || !encode_chunk_map(&mo, a.o, a.B, a.T, a.H, a.os))
        return cudaErrorInvalidValue;
    PairParams p;
    p.B = a.B; p.T = a.T; p.H = a.H;
    p.grid_w = a.grid_w; p.prefix_len = a.prefix_len; p.t0 = a.t0; p.scale = a.scale;
    p.decay = a.decay; p.state_in = a.state_in; p.state_out = a.state_out;
    p.work = a.work;
    p.slots = static_cast<unsigned char*>(scratch);
    p.nc = nc;
    p.chains = (int)chains;
    p.status = a.status; p.wait_limit = a.wait_limit;
    const size_t smem = sizeof(Smem) + 1024;
    static bool smem_ok_1[64];
    cudaError_t e = allow_dynamic_smem(prefill_pair_kernel, smem, smem_ok_1);
    if (e != cudaSuccess) return e;
    // Fewer chains than SMs: one chain per CTA, nothing is cut.  Otherwise one CTA per SM.
    const unsigned grid = (unsigned)(chains < sms ? chains : sms);
    // Programmatic dependent launch: when the kernel before this one in the stream lets its
    // dependents go early (this kernel does, see its first lines), the CTAs of this launch may take
    // their SMs as soon as that kernel's CTAs leave them and do their set-up there; they read
    // nothing from device memory before griddepcontrol.wait, which returns when the earlier
    // kernel has completed.  After any other kernel the launch behaves like an ordinary one.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, prefill_pair_kernel, mq, mk, mv, mo, p);
}

}  // namespace lasad
