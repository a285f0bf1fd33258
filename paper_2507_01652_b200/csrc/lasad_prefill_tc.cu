// LASAD chunked prefill on the 5th-generation tensor cores (sm_100a): TMA-fed tcgen05.mma with
// TMEM accumulators, bf16 I/O, fp32 accumulation and an fp32 master state.
//
// One CTA owns one (batch, head) at a time and walks its sequence in chunks of C = 128 tokens; two
// CTAs fit on an SM (256 TMEM columns and ~106 KB of shared memory each).  With more chains than
// resident CTAs, a CTA that finishes a chain draws the next one from a device-side work counter;
// its loads run two chunks ahead across the chain boundary.  With n_i = number of
// decaying steps from the chunk start up to and including token i (SAD rule, Section 3.4, from
// the token's grid position), N = n of the chunk's last token and gamma the head's decay, the
// SAD recurrence (Section 3.4) unrolled over one chunk is
//
//     o_i   = scale * ( sum_{j<=i} (q_i.k_j) gamma^(n_i-n_j) v_j  +  gamma^(n_i) q_i^T S_prev )
//     S_new = gamma^N S_prev + sum_j gamma^(N-n_j) k_j v_j^T
//
// Normal path (gamma >= 0.6, so that gamma^-128 stays far inside fp32 range).  Every decay
// factor is moved onto V and onto one per-row factor of the output, so that Q and K feed the
// tensor cores untouched and the scores only need the causal mask:
//
//     V~ = diag(gamma^(N-n_j)) V                       in place in smem, before the scores exist
//     S  = Q K^T                         (M1)          tcgen05.mma 128x128x64, smem x smem
//     A  = tril(S) -> bf16               (E1)          back into TMEM over S's own columns
//     dS = K^T V~                        (M2a)         tcgen05.mma 64x64x128
//     O' = A V~ + Q (gamma^N S_prev)     (M2b)         tcgen05.mma 128x64x128 (tmem x smem) + 128x64x64
//     o_i = scale * gamma^-(N-n_i) * O'_i   (E2)       -> bf16 -> smem -> TMA store
//     S_new = gamma^N S_prev + dS        (E3)          fp32 registers; bf16 copy to smem for M2b
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
#include "lasad_common.cuh"
#include "lasad_tc_chunk.cuh"
#include "lasad_tc_ptx.cuh"
#include "lasad_tc_tma.cuh"

namespace lasad {
namespace {

using namespace tcx;

constexpr int kThreads = kEThreads + 64;   // element-wise warps, the MMA warp and the TMA warp
constexpr int kStages = 2;
constexpr int kTmemCols = 256;

struct __align__(8) Barriers {
    unsigned long long full[kStages];   // TMA loads of a stage have landed
    unsigned long long s_done;     // M1 complete
    unsigned long long x_ready;    // V~ (normal path) or K~ (exact path) written: dS may start (256 arrivals)
    unsigned long long ds_done;    // dS MMAs complete
    unsigned long long p_ready;    // A/P in TMEM, state copy (and Q~) in smem (256 arrivals)
    // The two barriers the TMA warp waits on exist once per stage: a barrier's next phase then
    // belongs to the chunk two further on, whose loads the TMA warp issues only after it has seen
    // this phase, so a one-bit phase parity can never be taken for a later phase's.
    unsigned long long o_done[kStages];    // O MMAs complete (and every MMA issued before them)
    unsigned long long st_ready[kStages];  // output tile staged in smem (256 arrivals)
    unsigned long long tbl;        // exact path: the decay table may change / has changed (256 arrivals)
    unsigned long long drain;      // teardown: all MMAs retired
};

struct Smem {
    // tiles first: each must sit on a 1024-byte boundary (128-byte swizzle atom = 8 rows)
    unsigned char q[kStages][kTileBytes];
    unsigned char k[kStages][kTileBytes];
    unsigned char v[kStages][kTileBytes];
    unsigned char sb[kD * kD * 2];  // bf16 copy of the state, [dk][dv], 128 B rows, swizzled
    float pw[kC + 4];               // exact path: gamma^m, m = 0..128, of the current chain's head
    int ring[4];                    // chain index by ordinal % 4 (-1: no more work)
    Barriers bar;
    uint32_t tmem_base;
    int abort_flag;
};



struct TcParams {
    int B, T, H;
    int grid_w, prefix_len;
    long long t0;
    float scale;
    const float* decay;
    const float* state_in;
    float* state_out;
    int* work;               // [2], zero between launches: chains drawn beyond the grid size, CTAs that have left
    // A chain may be cut into n_segs segments of seg_chunks chunks that are computed independently
    // (work unit = one segment of one chain); a segment then starts from the state
    // seg_state[segment * B * H + chain], which earlier launches have prepared.  n_segs = 1: whole chains.
    int seg_chunks, n_segs;
    const float* seg_state;
    int* status;
    unsigned wait_limit;
};

// kSegments: work units are segments of chains (see TcParams); false: whole chains, and none of
// the unit arithmetic below costs anything.
template <bool kSegments>
__global__ void __launch_bounds__(kThreads, 2)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, TcParams p)
{
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    // work unit u = segment u / (B H) of chain u % (B H): chunks [first, first + count) of the chain
    // (everything from the kernel's parameters each time: nothing of it is worth a register)
    auto unit_chain = [&](int u) { return kSegments ? u % (p.B * p.H) : u; };
    auto unit_seg = [&](int u) { return kSegments ? u / (p.B * p.H) : 0; };
    auto unit_first = [&](int u) { return kSegments ? unit_seg(u) * p.seg_chunks : 0; };
    auto unit_count = [&](int u) {
        return kSegments ? min(p.seg_chunks, (p.T + kC - 1) / kC - unit_first(u)) : (p.T + kC - 1) / kC;
    };
    volatile int* abort_flag = &sm.abort_flag;
    volatile int* ring = sm.ring;
    const unsigned limit = p.wait_limit;

    // ---- set-up ---------------------------------------------------------------------------
    // A kernel launched behind this one as a programmatic dependent may start to take SMs as they
    // become free; it waits for this kernel's completion before it touches device memory.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!kSegments && warp == 9 && lane == 0) {
        // the CTA's first chain is chain blockIdx.x: ask for its first chunks to be brought into L2
        // now, while the launch before this one may still be finishing (a prefetch hands no data to
        // the SM, so it may run ahead of the wait below)
        // (a short chain whole, of a longer one what the stages hold: asking for more than that of
        // long chains measured slower)
        const int pb = (int)blockIdx.x / p.H, ph = (int)blockIdx.x - pb * p.H;
        const int nc = (p.T + kC - 1) / kC;
        for (int n = 0; n < (nc <= 5 ? nc : kStages); ++n) {
            tma_prefetch_4d(&tm_k, 0, ph, n * kC, pb);
            tma_prefetch_4d(&tm_v, 0, ph, n * kC, pb);
            tma_prefetch_4d(&tm_q, 0, ph, n * kC, pb);
        }
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&sm.bar.full[s], 1);
        mbar_init(&sm.bar.s_done, 1);
        mbar_init(&sm.bar.x_ready, kEThreads);
        mbar_init(&sm.bar.ds_done, 1);
        mbar_init(&sm.bar.p_ready, kEThreads);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.bar.o_done[s], 1);
            mbar_init(&sm.bar.st_ready[s], kEThreads);
        }
        mbar_init(&sm.bar.tbl, kEThreads);
        mbar_init(&sm.bar.drain, 1);
        sm.abort_flag = 0;
        sm.ring[0] = (int)blockIdx.x;     // the CTA's first chain; later ones come from the work counter
        // nothing above reads or writes device memory; everything below may depend on the kernel
        // before this one in the stream (its outputs, the work counter it puts back to zero)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    // Every role walks the same sequence of chunks: all chunks of the CTA's first chain, then all
    // chunks of the next chain the TMA warp drew from the work counter, and so on.  g counts the
    // chunks of that sequence (stage g % 2, barrier phases from g); a chain's position in it is
    // its ordinal, and ring[ordinal % 4] holds the chain's index, or -1 when the work has run out.
    // The TMA warp publishes an ordinal's entry before it issues (or, for -1, completes by hand)
    // the `full` barrier of that chain's first chunk, and the other roles read it after that wait.

    if (warp == 9) {
        // ===================== TMA warp: loads two chunks ahead, stores each output tile =======
        if (elect_one()) {
            // load iterator: (chain, chunk, ordinal) of the next chunk to be loaded
            int ld_unit = (int)blockIdx.x, ld_n = 0, ld_ord = 0;
            int ld_b = unit_chain(ld_unit) / p.H, ld_h = unit_chain(ld_unit) - ld_b * p.H;
            int ld_first = unit_first(ld_unit), ld_count = unit_count(ld_unit);
            bool ended = false;            // the end marker has been delivered
            int last_real = -1;            // sequence number of the last chunk whose loads were issued
            auto draw = [&]() {
                const int u = (int)gridDim.x + atomicAdd(p.work, 1);
                return u < p.B * p.H * (kSegments ? p.n_segs : 1) ? u : -1;
            };
            // A stage is refilled in two steps: K and V as soon as every MMA of the chunk that used
            // them has retired, Q (whose buffer stages the output tile) once the store has read it.
            auto issue_kv = [&](int g) {
                const int s = g % kStages;
                if (ld_unit < 0) {
                    if (!ended) {
                        mbar_arrive(&sm.bar.full[s]);     // completes the phase: the waiters find -1 in the ring
                        ended = true;
                    }
                    return;
                }
                mbar_arrive_expect_tx(&sm.bar.full[s], 3 * kTileBytes);
                tma_load_4d(sm.k[s], &tm_k, &sm.bar.full[s], 0, ld_h, (ld_first + ld_n) * kC, ld_b);
                tma_load_4d(sm.v[s], &tm_v, &sm.bar.full[s], 0, ld_h, (ld_first + ld_n) * kC, ld_b);
                last_real = g;
            };
            auto issue_q = [&](int g) {
                if (ld_unit < 0) return;
                const int s = g % kStages;
                tma_load_4d(sm.q[s], &tm_q, &sm.bar.full[s], 0, ld_h, (ld_first + ld_n) * kC, ld_b);
                if (++ld_n == ld_count) {
                    ld_n = 0;
                    ++ld_ord;
                    ld_unit = draw();
                    ring[ld_ord & 3] = ld_unit;
                    if (ld_unit >= 0) {
                        ld_b = unit_chain(ld_unit) / p.H;
                        ld_h = unit_chain(ld_unit) - ld_b * p.H;
                        ld_first = unit_first(ld_unit);
                        ld_count = unit_count(ld_unit);
                    }
                }
            };
            for (int g = 0; g < kStages; ++g) {
                issue_kv(g);
                issue_q(g);
            }
            // store iterator: the chunk whose output tile leaves next
            int st_unit = (int)blockIdx.x, st_n = 0, st_ord = 0;
            int st_b = unit_chain(st_unit) / p.H, st_h = unit_chain(st_unit) - st_b * p.H;
            int st_first = unit_first(st_unit), st_count = unit_count(st_unit);
            for (int g = 0; st_unit >= 0; ++g) {
                const int s = g % kStages;
                if (!mbar_wait(&sm.bar.o_done[s], (g / kStages) & 1, limit, abort_flag, p.status)) break;
                issue_kv(g + kStages);
                // the output tile of chunk g sits in the Q buffer of its stage
                const bool staged = mbar_wait(&sm.bar.st_ready[s], (g / kStages) & 1, limit, abort_flag, p.status);
                if (staged) {
                    tma_store_4d(&tm_o, sm.q[s], 0, st_h, (st_first + st_n) * kC, st_b);
                    tma_store_commit();
                    if (ld_unit >= 0) tma_store_wait_read();   // the store has finished reading the buffer
                }
                issue_q(g + kStages);                          // (also after a failed wait: the stage's barrier must complete)
                if (!staged) break;
                if (++st_n == st_count) {
                    st_n = 0;
                    ++st_ord;
                    st_unit = ring[st_ord & 3];                // published by this thread when the loads reached it
                    if (st_unit >= 0) {
                        st_b = unit_chain(st_unit) / p.H;
                        st_h = unit_chain(st_unit) - st_b * p.H;
                        st_first = unit_first(st_unit);
                        st_count = unit_count(st_unit);
                    }
                }
            }
            tma_store_wait_all();
            // leave only when every issued load has landed (they write this CTA's shared memory)
            // (once the end marker is out, the chunk before the last loaded one has been processed,
            // and its stage's barrier has moved on by the marker's phase: only the last one is waited for)
            for (int g = max(0, ended ? last_real : last_real - kStages + 1); g <= last_real; ++g)
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
        int m_n = 0, m_ord = 0;           // chunk within its unit and unit ordinal of the chunk whose scores come next
        int m_count = 1;                  // chunks of that unit
        bool fast_next = true;            // path of that chunk's chain
        // waits for chunk g's tiles, finds out whose they are and issues its score MMAs;
        // 0 = issued, 1 = the work has run out, -1 = a wait gave up
        auto issue_m1 = [&](int g) {
            const int s = g % kStages;
            const uint64_t dqs = s ? dq1 : dq0, dks = s ? dk1 : dk0;
            if (!mbar_wait(&sm.bar.full[s], (g / kStages) & 1, limit, abort_flag, p.status)) return -1;
            if (m_n == 0) {
                const int u = ring[m_ord & 3];
                if (u < 0) return 1;
                fast_next = p.decay[unit_chain(u) % p.H] >= kFastPathMinDecay;
                m_count = unit_count(u);
            }
            if (++m_n == m_count) {
                m_n = 0;
                ++m_ord;
            }
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)  // 32 bytes along K per step
                    mma_ss(tmem + kColS, dqs + 2 * kk, dks + 2 * kk, idesc_s, kk > 0);
                mma_commit(&sm.bar.s_done);
            }
            __syncwarp();
            return 0;
        };
        int more = issue_m1(0);
        for (int g = 0; more == 0; ++g) {
            const int s = g % kStages;
            const uint64_t dqs = s ? dq1 : dq0, dks = s ? dk1 : dk0, dvs = s ? dv1 : dv0;
            const bool fast = fast_next;
            if (!mbar_wait(&sm.bar.x_ready, g & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // 16 tokens = 2048 B of K and of V per step
                    mma_ss(tmem + kColDS, dks + 128 * kk, dvs + 128 * kk, idesc_kv, kk > 0);
                mma_commit(&sm.bar.ds_done);
                // Normal path: the state's contribution to O needs nothing from E1 (the state copy
                // was written, and the previous O read, before x_ready), so it opens the
                // accumulator now and only the A V~ MMAs remain once A is ready.
                if (fast) {
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk)
                        mma_ss(tmem + kColO, dqs + 2 * kk, d_sb + 128 * kk, idesc_qs, kk > 0);
                }
            }
            __syncwarp();
            if (!mbar_wait(&sm.bar.p_ready, g & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // A/P: 8 TMEM columns per step (tokens 0..63 at columns
                                                      // 0..31, tokens 64..127 at 64..95); V: 2048 B per step
                    mma_ts(tmem + kColO, tmem + kColS + (kk < 4 ? 8 * kk : 64 + 8 * (kk - 4)), dvs + 128 * kk,
                           idesc_pv, fast || kk > 0);
                if (!fast) {
                    // exact path: Q~ is written during E1, so its MMAs come last
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk)
                        mma_ss(tmem + kColO, dqs + 2 * kk, d_sb + 128 * kk, idesc_qs, 1);
                }
                mma_commit(&sm.bar.o_done[s]);
            }
            __syncwarp();
            more = issue_m1(g + 1);
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

        float st[16];                            // fp32 master state, this thread's 16 values
        // bf16 copy of mult * state for the Q x state MMA of the next chunk: [dk][dv] rows of 128 B,
        // 16-byte pieces swizzled by the row; this thread writes eight bf16 pairs
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
            uint32_t ov[32];
            tmem_ld32(tmem + lane_base + kColO + 32 * grp, ov);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float r0, r1;
                    mul2(__uint_as_float(ov[8 * c + 2 * e]), __uint_as_float(ov[8 * c + 2 * e + 1]), f, r0, r1);
                    w[e] = pack_bf16(r0, r1);
                }
                reinterpret_cast<uint4*>(orow)[(4 * grp + c) ^ (i & 7)] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        };

        bool ok = true;
        int g = 0;                      // chunks of this CTA's sequence done so far
        unsigned tbl_phase = 0;         // completed phases of the table barrier
        int cur_unit = (int)blockIdx.x;
        for (int ord = 0; ok; ++ord) {
            // ---- next unit: its index is in the ring once the tiles of its first chunk are in -----
            if (!(ok = mbar_wait(&sm.bar.full[g % kStages], (g / kStages) & 1, limit, abort_flag, p.status))) break;
            if (ord > 0) cur_unit = ring[ord & 3];
            if (cur_unit < 0) break;
            const int chain = unit_chain(cur_unit);
            const int first = unit_first(cur_unit);
            const int T_here = kSegments ? min(unit_count(cur_unit) * kC, p.T - first * kC) : p.T;   // tokens of this unit
            const int n_here = (T_here + kC - 1) / kC;
            const int h = chain % p.H;
            const float gamma = p.decay[h];
            const bool fast = gamma >= kFastPathMinDecay;
            const float lg = fast ? log2f(gamma) : 0.0f;
            // position of the unit's first token relative to the grid (SAD rule, Section 3.4)
            GridPos gp = grid_pos_init(p.grid_w, p.prefix_len, p.t0 + (long long)first * kC, lane);
            {
                // the state the unit starts from: the caller's (or zero) for a whole chain, the prepared
                // one for a segment (also for a chain's first: state_out may alias state_in, and the
                // chain's last segment may be done before its first has started)
                const float* sin = nullptr;
                if (kSegments)
                    sin = p.seg_state + ((size_t)unit_seg(cur_unit) * (p.B * p.H) + chain) * kD * kD;
                else if (p.state_in)
                    sin = p.state_in + (size_t)chain * kD * kD;
#pragma unroll
                for (int e = 0; e < 16; ++e) st[e] = 0.0f;
                if (sin) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float2 a = *reinterpret_cast<const float2*>(sin + (size_t)r0 * kD + c0 + 8 * k);
                        const float2 c = *reinterpret_cast<const float2*>(sin + (size_t)(r0 + 8) * kD + c0 + 8 * k);
                        st[4 * k] = a.x; st[4 * k + 1] = a.y; st[4 * k + 2] = c.x; st[4 * k + 3] = c.y;
                    }
                }
            }
            // the final state leaves with a chain's last segment only
            auto state_leaves = [&]() {
                if (!p.state_out || unit_first(cur_unit) + unit_count(cur_unit) != (p.T + kC - 1) / kC) return;
                float* dst = p.state_out + (size_t)unit_chain(cur_unit) * kD * kD;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    *reinterpret_cast<float2*>(dst + (size_t)r0 * kD + c0 + 8 * k) = make_float2(st[4 * k], st[4 * k + 1]);
                    *reinterpret_cast<float2*>(dst + (size_t)(r0 + 8) * kD + c0 + 8 * k) = make_float2(st[4 * k + 2], st[4 * k + 3]);
                }
            };

            if (fast) {
                // ------------------------------- normal path ---------------------------------------
                // gamma^m straight from ex2.approx: |m log2 gamma| <= 95, relative error ~1e-5, far
                // below what bf16 I/O resolves
                auto gpow = [&](int m) { return ex2_approx((float)m * lg); };
                ChunkDecay cd = chunk_decay(gp, 0, min(kC, T_here), qd, lane);
                write_state_bf16(gpow(cd.n_last));
                scale_row_inplace<4>(sm.v[g % kStages] + i * 128, gpow(cd.n_last - cd.ni), 4 * grp, i & 7);
                fence_proxy_async();
                mbar_arrive(&sm.bar.x_ready);
                for (int n = 0; ok && n < n_here; ++n, ++g) {
                    const int s = g % kStages;
                    if (!(ok = mbar_wait(&sm.bar.s_done, g & 1, limit, abort_flag, p.status))) break;
                    tc_fence_after();
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
                    tc_fence_before();
                    mbar_arrive(&sm.bar.p_ready);

                    // ---- while the O MMAs run: the state recurrence in fp32 registers ----------------
                    const float out_f = p.scale * gpow(-(cd.n_last - cd.ni));   // scale * gamma^-(N - n_i)
                    if (!(ok = mbar_wait(&sm.bar.ds_done, g & 1, limit, abort_flag, p.status))) break;
                    tc_fence_after();
                    update_state(gpow(cd.n_last));
                    const bool more = n + 1 < n_here;
                    if (more) {
                        const int cs1 = (n + 1) * kC;
                        cd = chunk_decay(gp, cs1, min(kC, T_here - cs1), qd, lane);
                    } else {
                        state_leaves();
                    }

                    // ---- E2: o_i = scale * gamma^-(N - n_i) * O'_i ------------------------------------
                    if (!(ok = mbar_wait(&sm.bar.o_done[s], (g / kStages) & 1, limit, abort_flag, p.status))) break;
                    tc_fence_after();
                    stage_output(s, out_f);
                    if (more) write_state_bf16(gpow(cd.n_last));   // gamma^N(next) * S_new
                    fence_proxy_async();
                    tc_fence_before();
                    mbar_arrive(&sm.bar.st_ready[s]);

                    // ---- V~ of the chain's next chunk, once its loads have landed.  This stage is
                    //      released (st_ready above) before the wait, so the wait never holds a buffer
                    //      back.  (The first chunk of the next chain is prepared at the top.)
                    if (more) {
                        const int s1 = (g + 1) % kStages;
                        if (!(ok = mbar_wait(&sm.bar.full[s1], ((g + 1) / kStages) & 1, limit, abort_flag, p.status))) break;
                        scale_row_inplace<4>(sm.v[s1] + i * 128, gpow(cd.n_last - cd.ni), 4 * grp, i & 7);
                        fence_proxy_async();
                        mbar_arrive(&sm.bar.x_ready);
                    }
                }
            } else {
                // ------------------------------- exact path ----------------------------------------
                // table of gamma^m, m = 0..128, by binary exponentiation in double precision
                // (0^0 = 1); every thread is done with the previous chain's table before it changes
                mbar_arrive(&sm.bar.tbl);
                if (!(ok = mbar_wait(&sm.bar.tbl, tbl_phase & 1, limit, abort_flag, p.status))) break;
                ++tbl_phase;
                if (tid <= kC) {
                    double base = (double)gamma, acc = 1.0;
                    for (int e = tid; e > 0; e >>= 1) {
                        if (e & 1) acc *= base;
                        base *= base;
                    }
                    sm.pw[tid] = (float)acc;
                }
                mbar_arrive(&sm.bar.tbl);
                if (!(ok = mbar_wait(&sm.bar.tbl, tbl_phase & 1, limit, abort_flag, p.status))) break;
                ++tbl_phase;
                write_state_bf16(1.0f);
                for (int n = 0; ok && n < n_here; ++n, ++g) {
                    const int s = g % kStages;
                    const int cs = n * kC;
                    const ChunkDecay cd = chunk_decay(gp, cs, min(kC, T_here - cs), qd, lane);
                    if (n > 0 &&
                        !(ok = mbar_wait(&sm.bar.full[s], (g / kStages) & 1, limit, abort_flag, p.status))) break;
                    if (!(ok = mbar_wait(&sm.bar.s_done, g & 1, limit, abort_flag, p.status))) break;
                    tc_fence_after();
                    // K~ first (M1 has finished reading K): it unblocks the dS MMAs
                    if (grp == 1) scale_row_inplace<8>(sm.k[s] + i * 128, sm.pw[cd.n_last - cd.ni], 0, i & 7);
                    fence_proxy_async();
                    mbar_arrive(&sm.bar.x_ready);
                    // P = S o gamma^(n_i - n_j) o [j <= i], weights straight from the table
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
                                const float v0 = j0 <= i ? __uint_as_float(sv[2 * c]) * sm.pw[d0 > 0 ? d0 : 0] : 0.0f;
                                const float v1 = j0 + 1 <= i ? __uint_as_float(sv[2 * c + 1]) * sm.pw[d1 > 0 ? d1 : 0] : 0.0f;
                                pk[c] = pack_bf16(v0, v1);
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 16; ++c) pk[c] = 0u;
                        }
                        tmem_st16(tmem + lane_base + kColS + 64 * grp + 16 * pi, pk);
                    }
                    if (grp == 0) scale_row_inplace<8>(sm.q[s] + i * 128, sm.pw[cd.ni], 0, i & 7);
                    tmem_wait_st();
                    fence_proxy_async();
                    tc_fence_before();
                    mbar_arrive(&sm.bar.p_ready);

                    if (!(ok = mbar_wait(&sm.bar.ds_done, g & 1, limit, abort_flag, p.status))) break;
                    tc_fence_after();
                    update_state(sm.pw[cd.n_last]);
                    if (n + 1 >= n_here) state_leaves();
                    if (!(ok = mbar_wait(&sm.bar.o_done[s], (g / kStages) & 1, limit, abort_flag, p.status))) break;
                    tc_fence_after();
                    stage_output(s, p.scale);
                    if (n + 1 < n_here) write_state_bf16(1.0f);
                    fence_proxy_async();
                    tc_fence_before();
                    mbar_arrive(&sm.bar.st_ready[s]);
                }
            }
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
    // the last CTA to leave puts the work counter back to zero for the next launch
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(p.work + 1, 1) == (int)gridDim.x - 1) {
            p.work[0] = 0;
            p.work[1] = 0;
            __threadfence();
        }
    }
}


// ---------------------------------------------------------------------------------------------
// Few chains, long sequences: the chains are cut into segments that run side by side.
//
// The SAD recurrence (Section 3.4) is linear in the state, so over a segment [a, b) of a chain
//     S_b = gamma^(decaying steps in [a, b)) S_a + L,     L = the state the segment reaches from zero.
// First launch (below): L for every segment but a chain's last, from K and V alone (the dS MMAs
// of the main kernel and nothing else); the CTA that finishes a chain's last L then turns them into
// S_a for every segment, an element-wise scan over the chain's segments.  Second launch: the main
// kernel with one work unit per segment.
// ---------------------------------------------------------------------------------------------
// steps[s] = decaying steps among segment s's tokens (SAD rule, Section 3.4), the same for every
// chain, counted on the host.
constexpr int kMaxSegs = 320;
struct SegSteps {
    int n[kMaxSegs];
};

struct StateSmem {
    unsigned char k[kStages][kTileBytes];
    unsigned char v[kStages][kTileBytes];
    float pw[kC + 4];               // exact path: gamma^m, m = 0..128
    unsigned long long full[kStages];
    unsigned long long x_ready;     // V~ (normal path) or K~ (exact path) written (256 arrivals)
    unsigned long long ds_done[kStages];   // dS MMAs of the stage's chunk complete (per stage: see Barriers)
    unsigned long long drain;
    uint32_t tmem_base;
    int abort_flag;
    int last_of_chain;              // this CTA wrote the chain's last missing segment state: it runs the scan
};
constexpr int kStateTmemCols = 64;

__global__ void __launch_bounds__(kThreads, 2)
prefill_seg_state_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, TcParams p,
                         SegSteps steps, float* seg_state, int* seg_count)
{
    // Launched as a programmatic dependent: the kernel behind this one (the segment pass) may bring
    // its CTAs onto the SMs early; this one waits for the kernel before it to have completed before
    // it touches device memory.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ unsigned char smem_raw[];
    StateSmem& sm = *reinterpret_cast<StateSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int n_chains = p.B * p.H;
    const int seg = blockIdx.x / n_chains, chain = blockIdx.x - seg * n_chains;   // seg < n_segs - 1
    const int b = chain / p.H, h = chain - b * p.H;
    const int first = seg * p.seg_chunks, n_here = p.seg_chunks;                  // only a last segment is shorter
    volatile int* abort_flag = &sm.abort_flag;
    const unsigned limit = p.wait_limit;
    const float gamma = p.decay[h];
    const bool fast = gamma >= kFastPathMinDecay;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&sm.full[s], 1);
        mbar_init(&sm.x_ready, kEThreads);
        for (int s = 0; s < kStages; ++s) mbar_init(&sm.ds_done[s], 1);
        mbar_init(&sm.drain, 1);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(kStateTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (!fast && tid <= kC) {
        double base = (double)gamma, acc = 1.0;
        for (int e = tid; e > 0; e >>= 1) {
            if (e & 1) acc *= base;
            base *= base;
        }
        sm.pw[tid] = (float)acc;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 9) {
        if (elect_one()) {
            auto issue = [&](int n) {
                const int s = n % kStages;
                mbar_arrive_expect_tx(&sm.full[s], 2 * kTileBytes);
                tma_load_4d(sm.k[s], &tm_k, &sm.full[s], 0, h, (first + n) * kC, b);
                tma_load_4d(sm.v[s], &tm_v, &sm.full[s], 0, h, (first + n) * kC, b);
            };
            int issued = min(n_here, kStages);
            for (int n = 0; n < issued; ++n) issue(n);
            for (int n = 0; n + kStages < n_here; ++n) {
                if (!mbar_wait(&sm.ds_done[n % kStages], (n / kStages) & 1, limit, abort_flag, p.status)) break;
                issue(n + kStages);
                issued = n + kStages + 1;
            }
            // leave only when every issued load has landed (they write this CTA's shared memory)
            for (int n = max(0, issued - kStages); n < issued; ++n)
                for (unsigned it = 0; it < kTeardownLimit; ++it)
                    if (mbar_try_wait(&sm.full[n % kStages], (n / kStages) & 1)) break;
        }
        __syncwarp();
    } else if (warp == 8) {
        constexpr uint32_t idesc_kv = make_idesc(64, 64, 1, 1);    // K^T (MN-major) x V (MN-major)
        const uint64_t dk0 = make_desc(smem_u32(sm.k[0])), dk1 = make_desc(smem_u32(sm.k[1]));
        const uint64_t dv0 = make_desc(smem_u32(sm.v[0])), dv1 = make_desc(smem_u32(sm.v[1]));
        for (int n = 0; n < n_here; ++n) {
            const int s = n % kStages;
            const uint64_t dks = s ? dk1 : dk0, dvs = s ? dv1 : dv0;
            if (!mbar_wait(&sm.full[s], (n / kStages) & 1, limit, abort_flag, p.status)) break;
            if (!mbar_wait(&sm.x_ready, n & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // 16 tokens = 2048 B of K and of V per step
                    mma_ss(tmem, dks + 128 * kk, dvs + 128 * kk, idesc_kv, kk > 0);
                mma_commit(&sm.ds_done[s]);
            }
            __syncwarp();
        }
        if (elect_one()) {
            mma_commit(&sm.drain);
            for (unsigned it = 0; it < kTeardownLimit; ++it)
                if (mbar_try_wait(&sm.drain, 0)) break;
        }
        __syncwarp();
    } else {
        const int qd = warp & 3, grp = warp >> 2;
        const int i = qd * 32 + lane;
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        const int r0 = qd * 16 + (lane >> 2);
        const int c0 = 32 * grp + 2 * (lane & 3);
        GridPos gp = grid_pos_init(p.grid_w, p.prefix_len, p.t0 + (long long)first * kC, lane);
        const float lg = fast ? log2f(gamma) : 0.0f;
        float st[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) st[e] = 0.0f;
        bool ok = true;
        // scales chunk n's operand (V~ on the normal path, K~ on the exact one) once its tiles are in;
        // returns gamma^N of the chunk.  (Full chunks: this is never a chain's last segment.)
        auto prepare = [&](int n, float& g_chunk) {
            const int s = n % kStages;
            const ChunkDecay cd = chunk_decay(gp, n * kC, kC, qd, lane);
            if (!mbar_wait(&sm.full[s], (n / kStages) & 1, limit, abort_flag, p.status)) return false;
            if (fast) {
                g_chunk = ex2_approx((float)cd.n_last * lg);
                scale_row_inplace<4>(sm.v[s] + i * 128, ex2_approx((float)(cd.n_last - cd.ni) * lg), 4 * grp, i & 7);
            } else {
                g_chunk = sm.pw[cd.n_last];
                if (grp == 1) scale_row_inplace<8>(sm.k[s] + i * 128, sm.pw[cd.n_last - cd.ni], 0, i & 7);
            }
            fence_proxy_async();
            return true;
        };
        float g_chunk = 1.0f;
        ok = prepare(0, g_chunk);
        if (ok) mbar_arrive(&sm.x_ready);
        for (int n = 0; ok && n < n_here; ++n) {
            const int s = n % kStages;
            // the next chunk's operand is scaled while this chunk's MMAs run (other stage)
            float g_next = 1.0f;
            if (n + 1 < n_here && !(ok = prepare(n + 1, g_next))) break;
            if (!(ok = mbar_wait(&sm.ds_done[s], (n / kStages) & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
            uint32_t dsv[16];
            tmem_ld_16x256b_x4(tmem + lane_base + 32 * grp, dsv);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; e += 2)
                fma2(st[e], st[e + 1], g_chunk, __uint_as_float(dsv[e]), __uint_as_float(dsv[e + 1]), st[e], st[e + 1]);
            tc_fence_before();
            if (n + 1 < n_here) mbar_arrive(&sm.x_ready);     // the accumulator has been read: the next dS may start
            g_chunk = g_next;
        }
        if (ok) {
            float* dst = seg_state + ((size_t)(seg + 1) * n_chains + chain) * kD * kD;    // scanned in place later
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                *reinterpret_cast<float2*>(dst + (size_t)r0 * kD + c0 + 8 * k) = make_float2(st[4 * k], st[4 * k + 1]);
                *reinterpret_cast<float2*>(dst + (size_t)(r0 + 8) * kD + c0 + 8 * k) = make_float2(st[4 * k + 2], st[4 * k + 3]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kStateTmemCols) : "memory");
    }

    // ---- the scan over the chain's segments, by whichever of its CTAs finishes last -------------
    // seg_state[s + 1] holds L of segment s now; afterwards seg_state[s] is the state at the start
    // of segment s (seg_state[0]: the caller's incoming state or zero).  seg_count[chain] counts the
    // CTAs of the chain that are done and goes back to zero with the last one.
    if (tid == 0) {
        __threadfence();           // after the barrier above: covers every thread's stores of L
        const int done = atomicAdd(seg_count + chain, 1);
        sm.last_of_chain = done == p.n_segs - 2;
        if (sm.last_of_chain) seg_count[chain] = 0;
    }
    __syncthreads();
    if (sm.last_of_chain && tid < kEThreads) {
        __threadfence();
        constexpr int kBatch = 4;
        const size_t stride = (size_t)n_chains * kD * kD;          // from one segment's slot to the next
        float4* slot = reinterpret_cast<float4*>(seg_state + (size_t)chain * kD * kD) + tid;   // + j * 256: 16 elements per thread
        const float lg = gamma > 0.0f ? log2f(gamma) : 0.0f;
        float4 carry[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            carry[j] = p.state_in ? reinterpret_cast<const float4*>(p.state_in + (size_t)chain * kD * kD)[tid + j * kEThreads]
                                  : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            slot[j * kEThreads] = carry[j];
        }
        for (int s0 = 0; s0 + 1 < p.n_segs; s0 += kBatch) {
            float4 loc[kBatch][4];
#pragma unroll
            for (int b2 = 0; b2 < kBatch; ++b2)
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    loc[b2][j] = s0 + b2 + 1 < p.n_segs
                                     ? __ldcg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(slot) +
                                                                              (size_t)(s0 + b2 + 1) * stride) + j * kEThreads)
                                     : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
            for (int b2 = 0; b2 < kBatch; ++b2) {
                if (s0 + b2 + 1 < p.n_segs) {
                    const int nst = steps.n[s0 + b2];
                    const float g = nst == 0 ? 1.0f : gamma > 0.0f ? exp2f((float)nst * lg) : 0.0f;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        carry[j].x = fmaf(g, carry[j].x, loc[b2][j].x);
                        carry[j].y = fmaf(g, carry[j].y, loc[b2][j].y);
                        carry[j].z = fmaf(g, carry[j].z, loc[b2][j].z);
                        carry[j].w = fmaf(g, carry[j].w, loc[b2][j].w);
                        *(reinterpret_cast<float4*>(reinterpret_cast<float*>(slot) + (size_t)(s0 + b2 + 1) * stride) +
                          j * kEThreads) = carry[j];
                    }
                }
            }
        }
    }
}

}  // namespace

bool prefill_tc_supported(int dk, int dv, bool bf16) { return bf16 && dk == kD && dv == kD; }

int prefill_tc_segments(int n_chunks, long long chains, int sms)
{
    // as many segments as there are CTA slots per chain, each of at least two chunks
    long long segs = chains > 0 ? 2LL * sms / chains : 1;
    if (segs > n_chunks / 2) segs = n_chunks / 2;
    if (segs > kMaxSegs) segs = kMaxSegs;
    if (segs < 2) return 1;
    const int len = (int)((n_chunks + segs - 1) / segs);
    return (n_chunks + len - 1) / len;
}

cudaError_t launch_prefill_tc(const KernelArgs& a, int sms, cudaStream_t st)
{
    CUtensorMap mq, mk, mv, mo;
    if (!encode_chunk_map(&mq, a.q, a.B, a.T, a.H, a.qs) || !encode_chunk_map(&mk, a.k, a.B, a.T, a.H, a.ks) ||
        !encode_chunk_map(&mv, a.v, a.B, a.T, a.H, a.vs) || !encode_chunk_map(&mo, a.o, a.B, a.T, a.H, a.os))
        return cudaErrorInvalidValue;
    TcParams p;
    p.B = a.B; p.T = a.T; p.H = a.H;
    p.grid_w = a.grid_w; p.prefix_len = a.prefix_len; p.t0 = a.t0; p.scale = a.scale;
    p.decay = a.decay; p.state_in = a.state_in; p.state_out = a.state_out;
    p.work = a.work;
    p.n_segs = 1; p.seg_chunks = (a.T + kC - 1) / kC; p.seg_state = nullptr;
    p.status = a.status; p.wait_limit = a.wait_limit;
    const size_t smem = sizeof(Smem) + 1024;
    static bool smem_ok_1[64], smem_ok_2[64];
    cudaError_t e = allow_dynamic_smem(prefill_tc_kernel<false>, smem, smem_ok_1);
    if (e == cudaSuccess) e = allow_dynamic_smem(prefill_tc_kernel<true>, smem, smem_ok_2);
    if (e != cudaSuccess) return e;
    // Two CTAs fit on an SM; with more chains than that, the CTAs stay and draw further chains
    // from the work counter, so a chain's first loads overlap the previous chain's last chunk.
    if (sms <= 0) return cudaErrorInvalidValue;
    const long long chains = (long long)a.B * a.H;
    if (a.seg_state) {
        // few chains: cut them into segments that run side by side (two launches, see above)
        const int n_chunks = (a.T + kC - 1) / kC;
        const int segs = prefill_tc_segments(n_chunks, chains, sms);
        if (segs > 1) {
            p.seg_chunks = (n_chunks + segs - 1) / segs;
            p.n_segs = segs;
            p.seg_state = a.seg_state;
            const size_t ssmem = sizeof(StateSmem) + 1024;
            static bool smem_ok_3[64];
            e = allow_dynamic_smem(prefill_seg_state_kernel, ssmem, smem_ok_3);
            if (e != cudaSuccess) return e;
            SegSteps steps;
            for (int sg = 0; sg + 1 < segs; ++sg) {
                const long long lo = a.t0 + (long long)sg * p.seg_chunks * kC, hi = lo + (long long)p.seg_chunks * kC;
                steps.n[sg] = (int)(decay_steps_upto(hi - 1, a.grid_w, a.prefix_len) -
                                    decay_steps_upto(lo - 1, a.grid_w, a.prefix_len));
            }
            // the per-chain counters sit behind the 2 x SMs state slots
            int* seg_count = reinterpret_cast<int*>(a.seg_state + (size_t)2 * sms * kD * kD);
            cudaLaunchConfig_t scfg = {};
            scfg.gridDim = dim3((unsigned)(chains * (segs - 1)));
            scfg.blockDim = dim3(kThreads);
            scfg.dynamicSmemBytes = ssmem;
            scfg.stream = st;
            cudaLaunchAttribute sattr[1];
            sattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            sattr[0].val.programmaticStreamSerializationAllowed = 1;
            scfg.attrs = sattr;
            scfg.numAttrs = 1;
            e = cudaLaunchKernelEx(&scfg, prefill_seg_state_kernel, mk, mv, p, steps, a.seg_state, seg_count);
            if (e != cudaSuccess) return e;
        }
    }
    const long long units = chains * p.n_segs;
    const unsigned grid = (unsigned)(units < 2LL * sms ? units : 2LL * sms);
    // A programmatic dependent launch, as for the balanced kernel (its CTAs set up -- and, with whole
    // chains, ask for their first tiles in L2 -- on SMs the launch before has left; they read
    // nothing from device memory before griddepcontrol.wait).  After a kernel that does not let its
    // dependents go early the launch behaves like an ordinary one.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return p.n_segs > 1 ? cudaLaunchKernelEx(&cfg, prefill_tc_kernel<true>, mq, mk, mv, mo, p)
                        : cudaLaunchKernelEx(&cfg, prefill_tc_kernel<false>, mq, mk, mv, mo, p);
}

}  // namespace lasad
