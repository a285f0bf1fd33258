// LASAD prefill with the paper's data-dependent gate on the 5th-generation tensor cores (sm_100a),
// balanced over the SMs: the chunk algebra of lasad_prefill_gated_tc.cu (per-channel decay split
// around a per-chunk reference, see there) in the execution scheme of lasad_prefill_tc_pair.cu
// (one CTA per SM, two chunk pipelines that take the chunks of one chain alternately, the work
// dealt out by the plan of lasad_tc_pair_plan.cuh).
//
// Per 128-token chunk, with b_i[c] = sum_{u <= i in the chunk} log2 Lambda_u[c] and r = b_N / 2:
//
//     Q~ = Q o 2^(b_i - r),   K~ = K o 2^(r - b_j)           (K~ in place over the key tile)
//     S  = Q~ K~^T                          (M1)   tcgen05.mma 128x128x64
//     dS = K~^T V                           (M2a)  tcgen05.mma 64x64x128
//     A  = tril(S) -> bf16                  (E1)   back into TMEM over S's own columns
//     O  = A V + Q~ (diag(2^r) S_prev)      (M2b)  tcgen05.mma 128x64x128 (tmem x smem) + 128x64x64
//     S_new = diag(2^b_N) S_prev + diag(2^(b_N - r)) dS       fp32, through shared memory
//
// Only the last two lines tie a chunk to the one before it, so pipeline X works on chunk n while
// the other works on n + 1; the fp32 state passes between them through a 16 KiB buffer, and the
// Q~ S_prev MMAs are issued last in a chunk (the plain form takes the state in and writes its bf16
// copy while the score MMAs run, the fused form after E1).  Five tiles per pipeline: gate, query (both free for
// the next chunk's loads once Q~ and K~ are written), key (scaled in place; free once the dS MMAs
// have retired), Q~ (free for the next chunk's Q~ when the chunk's MMAs are done) and value, which
// after the chunk's MMAs doubles as the staging buffer of the output tile: the next chunk's
// scaling sweep then does not have to wait for the output store to have read its buffer, only the
// next value tile's load does, and that has the whole sweep to arrive.
//
// A chunk whose decay is too strong for the scaling (|b_N[c]| > 200 for some channel) cannot be
// taken this way.  The kernel then marks the chain in `redo` and lets a flag travel with the
// chain's state (through shared memory, and in the tag of the hand-off packets) so that whoever
// finishes the chain leaves state_out alone; what it computes for that chain in the meantime is
// discarded, because the CUDA-core kernel launched behind this one recomputes the marked chains
// in full (and puts their marks back to zero).
//
// kFused: Algorithm 1's loop body whole -- the gate and the query are pre-activations (the gate
// tile becomes u = Sigmoid(-g~) = 1 - lambda in place, SiLU is applied as Q~ is formed) and the
// output leaves through a weight-free RMS norm over the head's 64 channels.
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

constexpr int kPipeThreads = kEThreads + 64;    // element-wise warps, the MMA warp, the TMA warp
constexpr int kPairThreads = 2 * kPipeThreads;
constexpr int kPipeTmemCols = 256;
constexpr float kSafeRange = 200.0f;   // largest |sum of log2 decays| one chunk may span

struct __align__(8) PipeBarriers {
    unsigned long long full_gq;     // gate and query tiles of the chunk have landed
    unsigned long long full_k;      // key tile has landed (untied keys only)
    unsigned long long full_v;      // value tile has landed
    unsigned long long scan;        // partial sums of the chunk are in shared memory (256 arrivals)
    unsigned long long in_free;     // last read of the gate and query tiles of the chunk (256 arrivals)
    unsigned long long x_ready;     // Q~ and K~ are written (256 arrivals)
    unsigned long long s_done;      // M1 complete
    unsigned long long ds_done;     // dS MMAs complete (and M1): the key tile is free
    unsigned long long p_ready;     // A in TMEM (256 arrivals)
    unsigned long long sb_ready;    // bf16 copy of the incoming state in smem (256 arrivals)
    unsigned long long o_done;      // O MMAs complete (and every MMA issued before them)
    unsigned long long st_ready;    // output tile of the chunk staged in shared memory (256 arrivals)
    unsigned long long state_ready; // this pipeline's chunk has left its state in `sf` (256 arrivals)
    unsigned long long drain;       // teardown: all MMAs retired
};

struct Smem {
    // tiles first: each must sit on a 1024-byte boundary (128-byte swizzle atom = 8 rows)
    unsigned char g[2][kTileBytes];     // gate lambda (fused form: pre-activation, then 1 - lambda)
    unsigned char q[2][kTileBytes];
    unsigned char k[2][kTileBytes];     // keys, scaled in place to K~
    unsigned char v[2][kTileBytes];     // values; after the MMAs the staging buffer of the output tile
    unsigned char qt[2][kTileBytes];    // Q~
    unsigned char sb[2][kD * kD * 2];   // per pipeline: bf16 copy of diag(2^r) state, [dk][dv], 128 B rows, swizzled
    float4 sf[4][kEThreads];            // the fp32 state between two chunks: element-wise thread t's 16 values
    float segsum[2][8][kD];             // log2 of the product of Lambda over rows 16 x .. 16 x + 15, per channel
    float ssq[2][2][kC];                // fused form: sum of squares of each output row's two halves
    PipeBarriers bar[2];
    Plan plan;
    uint32_t tmem_base;
    int abort_flag;
    int cta;                            // this CTA's number in start order
    unsigned tag;                       // this launch's packet tag
    int given_up;                       // chain whose decay was too strong for this kernel (-1: none); see the head of the file
};

struct GatedPairParams {
    int B, T, H;
    int grid_w, prefix_len;
    long long t0;
    float scale;
    const float* state_in;
    float* state_out;
    int* redo;               // [B*H], zero between launches: set to 1 where this kernel gave the chain up
    int* work;               // [3]: CTAs that have started, CTAs that have left (both zero between launches), launches so far
    unsigned char* slots;    // [2 n_ctas][kSlotBytes]: hand-off slots (see lasad_tc_pair_plan.cuh)
    int nc;                  // chunks per chain
    int chains;              // B x H
    int* status;
    unsigned wait_limit;
    float norm_eps;          // fused form: epsilon of the output norm
};

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float tanh_approx(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// packed bf16 multiply, round to nearest
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// kTied: the key is the gate's complement, k = 1 - lambda, and there is no key tensor.
template <bool kFused, bool kTied>
__global__ void __launch_bounds__(kPairThreads, 1)
prefill_gated_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                          const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_g,
                          const __grid_constant__ CUtensorMap tm_o, GatedPairParams p)
{
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    // CTA warps 0-9 are pipeline 0, 10-19 pipeline 1; the second pipeline's roles are rotated by two
    // warps so that its element-wise warps sit on TMEM lane quadrants 0..3 in order (a warp reaches
    // the quadrant (its index in the CTA) mod 4).  `warp` is the role: 0-7 element-wise, 8 MMA, 9 TMA.
    const int X = threadIdx.x >= kPipeThreads ? 1 : 0;
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
            mbar_init(&b.full_gq, 1);
            mbar_init(&b.full_k, 1);
            mbar_init(&b.full_v, 1);
            mbar_init(&b.scan, kEThreads);
            mbar_init(&b.in_free, kEThreads);
            mbar_init(&b.x_ready, kEThreads);
            mbar_init(&b.s_done, 1);
            mbar_init(&b.ds_done, 1);
            mbar_init(&b.p_ready, kEThreads);
            mbar_init(&b.sb_ready, kEThreads);
            mbar_init(&b.o_done, 1);
            mbar_init(&b.st_ready, kEThreads);
            mbar_init(&b.state_ready, kEThreads);
            mbar_init(&b.drain, 1);
        }
        // nothing above reads or writes device memory; everything below may depend on the kernel
        // before this one in the stream (its outputs, the work counters it puts back to zero)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        sm.abort_flag = 0;
        sm.given_up = -1;
        sm.cta = atomicAdd(p.work, 1);
        sm.tag = ((unsigned)*reinterpret_cast<volatile int*>(p.work + 2) & 0x3fffffffu) + 1u;   // never 0, the slots' initial content
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9 && lane == 0) {
        // the descriptors' first use then finds them in the descriptor cache
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_q)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_v)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_g)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_o)) : "memory");
        // The CTAs' first chains are chains 0 .. gridDim.x - 1 in some order: ask for the first
        // chunks of chain blockIdx.x to be brought into L2 now, while the launch before this one is
        // still finishing (a prefetch hands no data to the SM, so it may run ahead of the wait below).
        // (Plain form only: the fused form measured slower with it.)
        if (X == 0 && !kFused) {
            const int pb = (int)blockIdx.x / p.H, ph = (int)blockIdx.x - pb * p.H;
            for (int n = 0; n < min(4, p.nc); ++n) {
                tma_prefetch_4d(&tm_g, 0, ph, n * kC, pb);
                tma_prefetch_4d(&tm_q, 0, ph, n * kC, pb);
                if (!kTied) tma_prefetch_4d(&tm_k, 0, ph, n * kC, pb);
                tma_prefetch_4d(&tm_v, 0, ph, n * kC, pb);
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
        // ===================== TMA warp ========================================================
        // One set of tiles per pipeline; each is refilled for the pipeline's next chunk as soon as its
        // last reader is done.  The output tile leaves from the value buffer.
        if (elect_one() && J > 0) {
            Unit lu;
            lu.g0 = 0; lu.g1 = -1;
            int b = 0, h = 0, tok = 0;      // of the chunk whose loads are being issued
            auto locate = [&](int j) {
                const int g = 2 * j + X;
                if (g >= lu.g1) lu = unit_of(plan, g);
                b = lu.chain / p.H;
                h = lu.chain - b * p.H;
                tok = (lu.n0 + g - lu.g0) * kC;
            };
            auto issue_gq = [&](int j) {
                locate(j);
                mbar_arrive_expect_tx(&bar.full_gq, 2 * kTileBytes);
                tma_load_4d(sm.g[X], &tm_g, &bar.full_gq, 0, h, tok, b);
                tma_load_4d(sm.q[X], &tm_q, &bar.full_gq, 0, h, tok, b);
            };
            auto issue_k = [&]() {     // (after issue_gq of the same chunk)
                mbar_arrive_expect_tx(&bar.full_k, kTileBytes);
                tma_load_4d(sm.k[X], &tm_k, &bar.full_k, 0, h, tok, b);
            };
            auto issue_v = [&]() {
                mbar_arrive_expect_tx(&bar.full_v, kTileBytes);
                tma_load_4d(sm.v[X], &tm_v, &bar.full_v, 0, h, tok, b);
            };
            issue_gq(0);
            if (!kTied) issue_k();
            issue_v();
            int gq_issued = 1, k_issued = kTied ? 0 : 1, v_issued = 1;     // chunks whose loads have been issued
            Unit su;
            su.g0 = 0; su.g1 = -1;
            for (int j = 0; j < J; ++j) {
                const bool more = j + 1 < J;
                if (more) {
                    if (!mbar_wait(&bar.in_free, j & 1, limit, abort_flag, p.status)) break;
                    issue_gq(j + 1);
                    gq_issued = j + 2;
                    if (!kTied) {
                        if (!mbar_wait(&bar.ds_done, j & 1, limit, abort_flag, p.status)) break;
                        issue_k();
                        k_issued = j + 2;
                    }
                }
                if (!mbar_wait(&bar.st_ready, j & 1, limit, abort_flag, p.status)) break;
                {
                    const int g = 2 * j + X;
                    if (g >= su.g1) su = unit_of(plan, g);
                    const int sb_ = su.chain / p.H, sh = su.chain - sb_ * p.H;
                    tma_store_4d(&tm_o, sm.v[X], 0, sh, (su.n0 + g - su.g0) * kC, sb_);
                    tma_store_commit();
                }
                if (more) {
                    tma_store_wait_read();        // the store has finished reading the buffer: the next values may land
                    issue_v();
                    v_issued = j + 2;
                }
            }
            tma_store_wait_all();
            // leave only when every issued load has landed (they write this CTA's shared memory)
            for (unsigned it = 0; it < kTeardownLimit; ++it)
                if (mbar_try_wait(&bar.full_gq, (gq_issued - 1) & 1)) break;
            if (k_issued > 0)
                for (unsigned it = 0; it < kTeardownLimit; ++it)
                    if (mbar_try_wait(&bar.full_k, (k_issued - 1) & 1)) break;
            for (unsigned it = 0; it < kTeardownLimit; ++it)
                if (mbar_try_wait(&bar.full_v, (v_issued - 1) & 1)) break;
        }
        __syncwarp();
    } else if (warp == 8) {
        // ===================== MMA issuer: the whole warp runs the loop, one lane issues =======
        constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);   // Q~ (K-major) x K~ (K-major)
        constexpr uint32_t idesc_pv = make_idesc(128, 64, 0, 1);   // A (tmem) x V (MN-major)
        constexpr uint32_t idesc_qs = make_idesc(128, 64, 0, 1);   // Q~ (K-major) x state (MN-major)
        constexpr uint32_t idesc_kv = make_idesc(64, 64, 1, 1);    // K~^T (MN-major) x V (MN-major)
        const uint64_t d_sb = make_desc(smem_u32(sm.sb[X]));
        const uint64_t d_q = make_desc(smem_u32(sm.qt[X]));
        const uint64_t d_k = make_desc(smem_u32(sm.k[X]));
        const uint64_t d_v = make_desc(smem_u32(sm.v[X]));
        for (int j = 0; j < J; ++j) {
            if (!mbar_wait(&bar.x_ready, j & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)  // 32 bytes along K per step
                    mma_ss(tmem + kColS, d_q + 2 * kk, d_k + 2 * kk, idesc_s, kk > 0);
                mma_commit(&bar.s_done);
            }
            __syncwarp();
            if (!mbar_wait(&bar.full_v, j & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // 16 tokens = 2048 B of K~ and of V per step
                    mma_ss(tmem + kColDS, d_k + 128 * kk, d_v + 128 * kk, idesc_kv, kk > 0);
                mma_commit(&bar.ds_done);
            }
            __syncwarp();
            if (!mbar_wait(&bar.p_ready, j & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // A: 8 TMEM columns per step (tokens 0..63 at columns
                                                      // 0..31, tokens 64..127 at 64..95); V: 2048 B per step
                    mma_ts(tmem + kColO, tmem + kColS + (kk < 4 ? 8 * kk : 64 + 8 * (kk - 4)), d_v + 128 * kk,
                           idesc_pv, kk > 0);
            }
            __syncwarp();
            // the carried state's share of O comes last: the only part that waits for the other pipeline
            if (!mbar_wait(&bar.sb_ready, j & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)
                    mma_ss(tmem + kColO, d_q + 2 * kk, d_sb + 128 * kk, idesc_qs, 1);
                mma_commit(&bar.o_done);
            }
            __syncwarp();
        }
        // make sure nothing is still running on the tensor pipe before TMEM is freed
        if (elect_one()) {
            mma_commit(&bar.drain);
            for (unsigned w = 0; w < kTeardownLimit; ++w)
                if (mbar_try_wait(&bar.drain, 0)) break;
        }
        __syncwarp();
    } else if (J > 0) {
        // ===================== element-wise warps ==============================================
        const int qd = warp & 3;                 // TMEM lane quadrant
        const int grp = warp >> 2;               // which half of the quadrant's columns
        const int i = qd * 32 + lane;            // chunk row owned by this thread in the TMEM stages
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        // State ownership as in the scalar-decay kernels: the 16x256b load of the dS accumulator
        // (M = 64 layout) gives this thread, for column group k, st[4k], st[4k+1] = (row r0,
        // columns c0 + 8k, + 1) and st[4k+2], st[4k+3] = (row r0 + 8, same columns).
        const int r0 = qd * 16 + (lane >> 2);
        const int c0 = 32 * grp + 2 * (lane & 3);
        // Scaling role: rows 16 warp .. 16 warp + 15, channels 2 lane and 2 lane + 1.  Byte offset
        // of that channel pair in row 16 warp + rr of a tile (rows of 128 B, 16-byte pieces
        // swizzled by the row): scale_off + rr * 128 + (((lane >> 2) ^ (rr & 7)) << 4).
        const int scale_off = 16 * warp * 128 + 4 * (lane & 3);
        const int lane_piece = lane >> 2;
        auto row_off = [&](int rr) { return scale_off + rr * 128 + ((lane_piece ^ (rr & 7)) << 4); };
        PipeBarriers& other = sm.bar[1 - X];
        unsigned char* const tg = sm.g[X];
        unsigned char* const tq = sm.q[X];
        unsigned char* const tk = sm.k[X];
        unsigned char* const tqt = sm.qt[X];
        float (*segsum)[kD] = sm.segsum[X];

        float st[16];
        // bf16 copy of diag(mult) state for the Q~ x state MMA: [dk][dv] rows of 128 B, 16-byte
        // pieces swizzled by the row; this thread writes eight bf16 pairs
        auto write_state_bf16 = [&](float mult_a, float mult_b) {
            unsigned char* row0 = sm.sb[X] + r0 * 128 + 4 * (lane & 3);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int piece = ((4 * grp + k) ^ (r0 & 7)) * 16;    // r0 + 8 has the same low bits
                float a0, a1, b0, b1;
                mul2(st[4 * k], st[4 * k + 1], mult_a, a0, a1);
                mul2(st[4 * k + 2], st[4 * k + 3], mult_b, b0, b1);
                *reinterpret_cast<uint32_t*>(row0 + piece) = pack_bf16(a0, a1);
                *reinterpret_cast<uint32_t*>(row0 + 8 * 128 + piece) = pack_bf16(b0, b1);
            }
        };
        // this thread's 32 columns of output row i -> bf16 -> row i of the staging buffer
        auto stage_output = [&](float f) {
            unsigned char* orow = sm.v[X] + i * 128;
            uint32_t ov[32];
            tmem_ld32(tmem + lane_base + kColO + 32 * grp, ov);
            tmem_wait_ld();
            if (kFused) {
                // Norm(o_i): sum of squares of this thread's 32 columns, the other 32 from the thread
                // of warp (warp ^ 4) of this pipeline that holds the same row
                float ss = 0.0f;
#pragma unroll
                for (int c = 0; c < 32; ++c) ss = fmaf(__uint_as_float(ov[c]), __uint_as_float(ov[c]), ss);
                sm.ssq[X][grp][i] = ss;
                asm volatile("bar.sync %0, 64;" ::"r"(1 + 4 * X + qd) : "memory");
                ss += sm.ssq[X][1 - grp][i];
                f *= rsqrtf(f * f * ss * (1.0f / kD) + p.norm_eps);
            }
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

        // ---- where this pipeline's chunks are: `cu` the chunk being worked on, `nx` the one after ----
        struct Where {
            Unit u;
            int n;          // chunk within the chain
            GridPos gp;     // positioned at that chunk
            int cs;         // its token offset within the run gp was set up for
        };
        Where nx;
        nx.u.g0 = 0; nx.u.g1 = -1; nx.n = 0; nx.cs = 0;
        nx.gp = grid_pos_init(0, 0, 0, lane);
        // moves `nx` to local chunk g and returns which of this warp's 16 rows of it are decaying
        // steps (live and not a row boundary, SAD rule of Section 3.4)
        auto advance = [&](int g) -> unsigned {
            if (__builtin_expect(g >= nx.u.g1, 0)) {
                nx.u = unit_of(plan, g);
                nx.n = nx.u.n0 + g - nx.u.g0;
                if (nx.u.recv >= 0) slot_prefetch(p.slots + (size_t)nx.u.recv * kSlotBytes, tid);
                nx.gp = grid_pos_init(p.grid_w, p.prefix_len, p.t0 + (long long)nx.n * kC, lane);
                nx.cs = 0;
            } else {
                nx.n += 2;
                nx.gp.skip();              // the other pipeline's chunk in between
                nx.cs += 2 * kC;
            }
            const ChunkDecay d = chunk_decay(nx.gp, nx.cs, min(kC, p.T - nx.n * kC), 0, lane);
            const int wx = warp >> 1;
            const unsigned own_word = wx == 0 ? d.m0 : wx == 1 ? d.m1 : wx == 2 ? d.m2 : d.m3;
            return (own_word >> (16 * (warp & 1))) & 0xffffu;
        };
        // first sweep over a chunk's gate tile: the product of the decays over this warp's 16 rows,
        // per channel; only its log2 crosses warps (a boundary step or a row past the end multiplies
        // by 1).  It needs nothing but the gate tile, so it runs as early as that tile is in.
        auto first_sweep = [&](unsigned dec) {
            float p0 = 1.0f, p1 = 1.0f;
#pragma unroll
            for (int rr = 0; rr < 16; ++rr) {
                uint32_t g2 = *reinterpret_cast<const uint32_t*>(tg + row_off(rr));
                if (kFused) {
                    // u = Sigmoid(-g~) = 1 / (1 + e^g~) = 1 - lambda, written back in place; lambda = 1 - u
                    // (e^g~ = inf gives u = 0 and e^g~ = 0 gives u = 1: no clamp is needed)
                    const uint32_t u2 = pack_bf16(rcp_approx(1.0f + ex2(1.4426950408889634f * bf16_lo(g2))),
                                                  rcp_approx(1.0f + ex2(1.4426950408889634f * bf16_hi(g2))));
                    *reinterpret_cast<uint32_t*>(tg + row_off(rr)) = u2;
                    const uint32_t us = ((dec >> rr) & 1u) ? u2 : 0u;
                    mul2_pair(p0, p1, 1.0f - bf16_lo(us), 1.0f - bf16_hi(us));
                    continue;
                }
                g2 = ((dec >> rr) & 1u) ? g2 : 0x3f803f80u;
                mul2_pair(p0, p1, bf16_lo(g2), bf16_hi(g2));
            }
            // a product that has left the fp32 range reads as -inf and fails the range check
            *reinterpret_cast<float2*>(&segsum[warp][2 * lane]) = make_float2(lg2(p0), lg2(p1));
            mbar_arrive(&bar.scan);
        };

        bool ok = true;
        unsigned dec16 = advance(X);
        ok = mbar_wait(&bar.full_gq, 0, limit, abort_flag, p.status);
        if (ok) first_sweep(dec16);
        for (int j = 0; ok && j < J; ++j) {
            const int g = 2 * j + X;
            const Unit u = nx.u;                        // the chunk being worked on
            const int n = nx.n;
            const int Lc = min(kC, p.T - n * kC);
            // the decay pair of row rr of this warp in fp32 (fused form: the tile holds u = 1 - lambda);
            // a boundary step or a dead row has decay 1 (one select, on the packed word)
            auto decay_pair = [&](uint32_t g2, int rr, float& l0, float& l1) {
                const uint32_t x = ((dec16 >> rr) & 1u) ? g2 : (kFused ? 0u : 0x3f803f80u);
                l0 = kFused ? 1.0f - bf16_lo(x) : bf16_lo(x);
                l1 = kFused ? 1.0f - bf16_hi(x) : bf16_hi(x);
            };
            if (!(ok = mbar_wait(&bar.scan, j & 1, limit, abort_flag, p.status))) break;

            // ---- this warp's place in the chunk, the chunk's total, the range check ----------------
            float f0, f1;       // 2^(b - r) just before this warp's first row
            float t0, t1;       // 2^(r - b) at this warp's last row
            bool too_strong;
            float tot0 = 0.0f, tot1 = 0.0f;     // log2 of the chunk's total decay, this lane's two channels
            {
                float base0 = 0.0f, base1 = 0.0f;
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const float2 bsx = *reinterpret_cast<const float2*>(&segsum[x][2 * lane]);
                    tot0 += bsx.x; tot1 += bsx.y;
                    if (x < warp) { base0 += bsx.x; base1 += bsx.y; }
                }
                const float2 own = *reinterpret_cast<const float2*>(&segsum[warp][2 * lane]);
                const float h0 = base0 - 0.5f * tot0, h1 = base1 - 0.5f * tot1;
                f0 = ex2(h0); f1 = ex2(h1);
                t0 = ex2(-(h0 + own.x)); t1 = ex2(-(h1 + own.y));
                // (written so that a NaN fails too; a warp's lanes cover all 64 channels, so every
                // warp takes the same decision)
                too_strong = __any_sync(0xffffffffu, !(fabsf(tot0) <= kSafeRange) || !(fabsf(tot1) <= kSafeRange));
            }
            // per-row factors of the state (rows r0 and r0 + 8 are channels): 2^(b_N / 2) = 2^r = 2^(b_N - r)
            // (channel c's total sits in lane c / 2, component c & 1)
            float m_a, m_b;
            {
                const int src = 8 * qd + (lane >> 3);
                const float a0 = __shfl_sync(0xffffffffu, tot0, src), a1 = __shfl_sync(0xffffffffu, tot1, src);
                const float b0 = __shfl_sync(0xffffffffu, tot0, src + 4), b1 = __shfl_sync(0xffffffffu, tot1, src + 4);
                const bool odd = (lane >> 2) & 1;
                m_a = ex2(0.5f * (odd ? a1 : a0));
                m_b = ex2(0.5f * (odd ? b1 : b0));
            }

            // ---- second sweep: Q~ = Q o 2^(b - r) with the factor carried forward down the rows as a
            //      running product of the gates, K~ = K o 2^(r - b) with its factor carried backward
            //      from the warp's last row, so that no factor is ever inverted.  (Rows in groups of
            //      eight: a group's loads are issued before its stores.)  The forward pass keeps the
            //      16 decay pairs in fp32 registers for the backward pass.
            // (the Q~ buffer is free: this thread has waited for the previous chunk's last MMA)
            float ls0[16], ls1[16];
#pragma unroll
            for (int r8 = 0; r8 < 16; r8 += 8) {
                uint32_t g2[8], q2[8];
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    g2[x] = *reinterpret_cast<const uint32_t*>(tg + row_off(r8 + x));
                    q2[x] = *reinterpret_cast<const uint32_t*>(tq + row_off(r8 + x));
                }
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    decay_pair(g2[x], r8 + x, ls0[r8 + x], ls1[r8 + x]);
                    mul2_pair(f0, f1, ls0[r8 + x], ls1[r8 + x]);
                    if (kFused) {
                        // q = SiLU(q~) = q~ (1 + tanh(q~ / 2)) / 2, scaled in the same step
                        const float x0 = bf16_lo(q2[x]), x1 = bf16_hi(q2[x]);
                        *reinterpret_cast<uint32_t*>(tqt + row_off(r8 + x)) =
                            pack_bf16(0.5f * x0 * (1.0f + tanh_approx(0.5f * x0)) * f0,
                                      0.5f * x1 * (1.0f + tanh_approx(0.5f * x1)) * f1);
                    } else {
                        *reinterpret_cast<uint32_t*>(tqt + row_off(r8 + x)) = mul_bf16x2(q2[x], pack_bf16(f0, f1));
                    }
                }
            }
            if (!kTied) {
                if (!(ok = mbar_wait(&bar.full_k, j & 1, limit, abort_flag, p.status))) break;
#pragma unroll
                for (int r8 = 8; r8 >= 0; r8 -= 8) {
                    uint32_t k2[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x) k2[x] = *reinterpret_cast<const uint32_t*>(tk + row_off(r8 + x));
#pragma unroll
                    for (int x = 7; x >= 0; --x) {
                        *reinterpret_cast<uint32_t*>(tk + row_off(r8 + x)) = mul_bf16x2(k2[x], pack_bf16(t0, t1));
                        mul2_pair(t0, t1, ls0[r8 + x], ls1[r8 + x]);
                    }
                }
            } else {
                // key tied to the gate: k = 1 - lambda in fp32 (0 on rows past the end of the sequence)
#pragma unroll
                for (int r8 = 8; r8 >= 0; r8 -= 8) {
                    uint32_t g2[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x) g2[x] = *reinterpret_cast<const uint32_t*>(tg + row_off(r8 + x));
#pragma unroll
                    for (int x = 7; x >= 0; --x) {
                        const float one = 16 * warp + r8 + x < Lc ? 1.0f : 0.0f;
                        if (kFused)     // the tile holds u = 1 - lambda: the tied key itself
                            *reinterpret_cast<uint32_t*>(tk + row_off(r8 + x)) =
                                pack_bf16(one * bf16_lo(g2[x]) * t0, one * bf16_hi(g2[x]) * t1);
                        else
                            *reinterpret_cast<uint32_t*>(tk + row_off(r8 + x)) =
                                pack_bf16((one - bf16_lo(g2[x])) * t0, (one - bf16_hi(g2[x])) * t1);
                        mul2_pair(t0, t1, ls0[r8 + x], ls1[r8 + x]);
                    }
                }
            }
            if (kFused) fence_proxy_async();      // the gate tile was rewritten in place: order that before its refill
            mbar_arrive(&bar.in_free);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&bar.x_ready);

            // ---- the carried state: in from the other pipeline's chunk (or from where the unit
            //      starts), out to the other pipeline's next chunk (or to where the unit ends).  Taking it
            //      in and writing its bf16 copy needs no MMA result, so the plain form does it while
            //      the score MMAs run; the fused form, whose sweeps are longer, runs faster with it
            //      after E1 -------------------------------------------------------------------------
            bool given_up = false;          // this chain has been given up (here or earlier)
            auto take_state = [&]() -> bool {
                if (g > 0) {
                    // the other pipeline is done with chunk g - 1 (its j index: j for X = 1, j - 1 for X = 0)
                    if (!mbar_wait(&other.state_ready, (j - 1 + X) & 1, limit, abort_flag, p.status)) return false;
                }
                if (__builtin_expect(g == u.g0, 0)) {      // (rare: a unit starts)
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
                        // the chain was cut here: its state (and whether it has been given up) comes from
                        // where the part before it was done
                        if (!slot_receive(p.slots + (size_t)u.recv * kSlotBytes, tid, st, sm.tag, limit, abort_flag, p.status, &given_up))
                            return false;
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float4 x = sm.sf[k][tid];
                        st[4 * k] = x.x; st[4 * k + 1] = x.y; st[4 * k + 2] = x.z; st[4 * k + 3] = x.w;
                    }
                    given_up = *reinterpret_cast<volatile int*>(&sm.given_up) == u.chain;
                }
                if (__builtin_expect(too_strong && !given_up, 0)) {
                    given_up = true;
                    if (tid == 0) p.redo[u.chain] = 1;
                }
                write_state_bf16(m_a, m_b);
                fence_proxy_async();
                mbar_arrive(&bar.sb_ready);
                return true;
            };
            if (!kFused && !(ok = take_state())) break;
            // ---- E1: A = tril(S) -> bf16 over S's own columns (blocks 2 grp, 2 grp + 1 of this
            //      thread's row, kept inside this warp's half of S's columns) -------------------------
            if (!(ok = mbar_wait(&bar.s_done, j & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
#pragma unroll 1
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
            mbar_arrive(&bar.p_ready);
            if (kFused && !(ok = take_state())) break;

            // S_new = diag(f) S_prev + diag(m) dS, with f = m * m (rows r0 and r0 + 8)
            if (!(ok = mbar_wait(&bar.ds_done, j & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
            {
                uint32_t dsv[16];
                tmem_ld_16x256b_x4(tmem + lane_base + kColDS + 32 * grp, dsv);
                tmem_wait_ld();
                const float f_a = m_a * m_a, f_b = m_b * m_b;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float x0, x1, y0, y1;
                    mul2(st[4 * k], st[4 * k + 1], f_a, x0, x1);
                    mul2(st[4 * k + 2], st[4 * k + 3], f_b, y0, y1);
                    fma2(__uint_as_float(dsv[4 * k]), __uint_as_float(dsv[4 * k + 1]), m_a, x0, x1, st[4 * k], st[4 * k + 1]);
                    fma2(__uint_as_float(dsv[4 * k + 2]), __uint_as_float(dsv[4 * k + 3]), m_b, y0, y1, st[4 * k + 2],
                         st[4 * k + 3]);
                }
            }
            if (__builtin_expect(g == u.g1 - 1, 0)) {      // (rare: a unit ends)
                if (u.send < 0) {
                    // the chain ends: its final state (a chain that was given up keeps its hands off:
                    // state_out may alias state_in, which the kernel that redoes the chain reads)
                    if (p.state_out && !given_up) {
                        float* dst = p.state_out + (size_t)u.chain * kD * kD;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            *reinterpret_cast<float2*>(dst + (size_t)r0 * kD + c0 + 8 * k) = make_float2(st[4 * k], st[4 * k + 1]);
                            *reinterpret_cast<float2*>(dst + (size_t)(r0 + 8) * kD + c0 + 8 * k) = make_float2(st[4 * k + 2], st[4 * k + 3]);
                        }
                    }
                } else {
                    // the chain is cut here: the state goes to where its next part will be done
                    slot_send(p.slots + (size_t)u.send * kSlotBytes, tid, st, sm.tag, given_up);
                }
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    sm.sf[k][tid] = make_float4(st[4 * k], st[4 * k + 1], st[4 * k + 2], st[4 * k + 3]);
                if (tid == 0) sm.given_up = given_up ? u.chain : -1;
            }
            tc_fence_before();
            mbar_arrive(&bar.state_ready);

            // ---- while the O MMAs run: the first sweep of this pipeline's next chunk, if its gate
            //      tile is in already (it was requested when this chunk's operands were written) ----
            const bool more = j + 1 < J;
            unsigned dec_next = 0;
            bool swept = false;
            if (more) {
                dec_next = advance(g + 2);
                swept = __all_sync(0xffffffffu, mbar_test_wait(&bar.full_gq, (j + 1) & 1));
                if (swept) first_sweep(dec_next);
            }

            // ---- output tile -------------------------------------------------------------------------
            if (!(ok = mbar_wait(&bar.o_done, j & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
            stage_output(p.scale);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&bar.st_ready);
            if (__builtin_expect(more && !swept, 0)) {
                if (!(ok = mbar_wait(&bar.full_gq, (j + 1) & 1, limit, abort_flag, p.status))) break;
                first_sweep(dec_next);
            }
            dec16 = dec_next;
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

cudaError_t launch_prefill_gated_pair(const KernelArgs& a, const void* gate, int* redo, void* scratch, int sms,
                                      cudaStream_t st)
{
    const long long chains = (long long)a.B * a.H;
    const int nc = (a.T + kC - 1) / kC;
    if (chains * nc > 0x7fffffffLL || !scratch || sms <= 0) return cudaErrorInvalidValue;
    CUtensorMap mq, mk, mv, mg, mo;
    // the gate shares the key's strides; without a key tensor its map stands in for the key's
    if (!encode_chunk_map(&mq, a.q, a.B, a.T, a.H, a.qs) || !encode_chunk_map(&mg, gate, a.B, a.T, a.H, a.ks) ||
        !encode_chunk_map(&mk, a.k ? a.k : gate, a.B, a.T, a.H, a.ks) ||
        !encode_chunk_map(&mv, a.v, a.B, a.T, a.H, a.vs) || !encode_chunk_map(&mo, a.o, a.B, a.T, a.H, a.os))
        return cudaErrorInvalidValue;
    GatedPairParams p;
    p.B = a.B; p.T = a.T; p.H = a.H;
    p.grid_w = a.grid_w; p.prefix_len = a.prefix_len; p.t0 = a.t0; p.scale = a.scale;
    p.state_in = a.state_in; p.state_out = a.state_out;
    p.redo = redo;
    p.work = a.work;
    p.slots = static_cast<unsigned char*>(scratch);
    p.nc = nc;
    p.chains = (int)chains;
    p.status = a.status; p.wait_limit = a.wait_limit;
    p.norm_eps = a.norm_eps;
    const size_t smem = sizeof(Smem) + 1024;
    const bool tied = a.k == nullptr;
    auto* kernel = a.fused ? (tied ? prefill_gated_pair_kernel<true, true> : prefill_gated_pair_kernel<true, false>)
                           : (tied ? prefill_gated_pair_kernel<false, true> : prefill_gated_pair_kernel<false, false>);
    static bool smem_ok[4][64];      // one set of flags per kernel variant
    cudaError_t e = allow_dynamic_smem(kernel, smem, smem_ok[(a.fused ? 2 : 0) + (tied ? 1 : 0)]);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)(chains < sms ? chains : sms);
    // programmatic dependent launch, as in launch_prefill_pair
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
    return cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mg, mo, p);
}

}  // namespace lasad
