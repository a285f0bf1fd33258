// LASAD prefill with the paper's data-dependent gate on the 5th-generation tensor cores
// (sm_100a): bf16 I/O, d_k = d_v = 64, fp32 accumulation, fp32 master state.
//
// The operator is Algorithm 1 with a decay vector lambda_t in [0,1]^dk per token and the SAD
// rule of Section 3.4 on top (decay 1 on the step that absorbs the last token of a grid row):
//
//     s_t = diag(Lambda_t) s_{t-1} + k_t v_t^T,    o_t = scale * q_t^T s_t,    k_t = 1 - lambda_t if tied.
//
// One CTA owns one (batch, head) and walks its sequence in chunks of C = 128 tokens; two CTAs fit
// on an SM.  With b_i[c] = sum_{u <= i in the chunk} log2 Lambda_u[c] (non-increasing in i) the
// recurrence unrolled over a chunk is
//
//     o_i   = scale * ( sum_{j<=i} sum_c q_i[c] k_j[c] 2^(b_i[c]-b_j[c]) v_j + sum_c q_i[c] 2^(b_i[c]) S_prev[c,:] )
//     S_new = diag(2^b_N) S_prev + sum_j diag(2^(b_N-b_j)) k_j v_j^T
//
// and the per-channel decay is split around a reference r[c] = b_N[c] / 2 so that each factor
// goes onto one operand and the scores are a plain product of two matrices:
//
//     Q~ = Q o 2^(b_i - r),   K~ = K o 2^(r - b_j)           element-wise, bf16, written to their own tiles
//     S  = Q~ K~^T                          (M1)   tcgen05.mma 128x128x64
//     A  = tril(S) -> bf16                  (E1)   back into TMEM over S's own columns
//     dS = K~^T V                           (M2a)  tcgen05.mma 64x64x128
//     O  = A V + Q~ (diag(2^r) S_prev)      (M2b)  tcgen05.mma 128x64x128 (tmem x smem) + 128x64x64
//     S_new = diag(2^b_N) S_prev + diag(2^(b_N - r)) dS       fp32 registers
//
// Every exponent that is formed lies within +-|b_N|/2.  The kernel takes a chunk this way while
// |b_N[c]| <= 200 for all channels (an average decay above 0.34 per step; gates at or below 0
// count as decay 0); a chain with a chunk beyond that is given up at that chunk and marked in a per-chain
// flag array, and the CUDA-core kernel, launched behind this one on every call, recomputes exactly
// the marked chains (it forms only differences b_i - b_j <= 0 and is safe for every gate in
// [0,1]).  A chain that is given up has not written its final state, so state_out may alias
// state_in.
//
// No exponential or logarithm is taken per element: within a warp's 16 rows the factor 2^(b_i - r)
// is carried forward as a running product of the gates themselves and 2^(r - b_j) backward from
// the warp's last row; log2 and exp2 only appear for the eight partial products per channel that
// cross warps.
//
// Fused form (kFused; Algorithm 1's loop body whole): q and the gate arrive as pre-activations.
// The first sweep turns the gate tile into u = Sigmoid(-g~) = 1 - lambda in place (bf16): the
// complement keeps full relative precision where lambda is close to 1, which is where a rounding
// of lambda itself would be felt over long ranges, and it is the tied key as it stands.  The
// second sweep forms lambda = 1 - u in fp32 for its running products and applies SiLU to the
// query as it scales it; the output tile leaves through a weight-free RMS norm over the head's
// 64 channels (the two threads that hold a row exchange their sums of squares).
//
// Warp roles: warps 0-7 do the element-wise work.  For the scaling they split the chunk by rows
// (warp w: rows 16 w ..), lanes across channel pairs, so the running sum b needs no exchange
// inside a warp and only eight partial sums per channel cross warps through shared memory; for
// the TMEM stages warp w works on lane quadrant w & 3 as in the scalar-decay kernel.  Warp 8
// issues the MMAs, warp 9 the TMA loads and stores.  All waits are bounded: a wait that runs out
// raises a status word the host can read and the CTA leaves through the normal exit.
#include "lasad_common.cuh"
#include "lasad_tc_chunk.cuh"
#include "lasad_tc_ptx.cuh"
#include "lasad_tc_tma.cuh"

namespace lasad {
namespace {

using namespace tcx;

constexpr int kThreads = kEThreads + 64;   // element-wise warps, the MMA warp and the TMA warp
constexpr int kTmemCols = 256;
constexpr float kSafeRange = 200.0f;   // largest |sum of log2 decays| one pass may span

struct __align__(8) Barriers {
    unsigned long long full_in;    // gate, query (and key) tiles of the chunk have landed
    unsigned long long full_v;     // value tile has landed
    unsigned long long scan;       // partial sums of the chunk are in shared memory (256 arrivals)
    unsigned long long in_free;    // last read of the gate, query and key tiles of the chunk (256 arrivals)
    unsigned long long stage_free; // the store of the previous output tile has read its staging buffer
    unsigned long long x_ready;    // Q~ and K~ are written (256 arrivals)
    unsigned long long sb_ready;   // bf16 copy of the scaled state is written (256 arrivals)
    unsigned long long s_done;     // M1 complete
    unsigned long long ds_done;    // dS MMAs complete
    unsigned long long p_ready;    // A in TMEM (256 arrivals)
    unsigned long long o_done;     // O MMAs complete (and every MMA issued before them)
    unsigned long long st_ready;   // output tile of the chunk staged in shared memory (256 arrivals)
    unsigned long long drain;      // teardown: all MMAs retired
};

struct Smem {
    // tiles first: each must sit on a 1024-byte boundary (128-byte swizzle atom = 8 rows)
    unsigned char q[kTileBytes];
    unsigned char k[kTileBytes];    // keys (unused when the key is tied to the gate)
    unsigned char v[kTileBytes];
    unsigned char g[kTileBytes];    // gate lambda
    unsigned char qt[kTileBytes];   // Q~
    unsigned char kt[kTileBytes];   // K~; after the MMAs the staging buffer of the output tile
    unsigned char sb[kD * kD * 2];  // bf16 copy of diag(2^r) state, [dk][dv], 128 B rows, swizzled
    float segsum[8][kD];            // log2 of the product of Lambda over rows 16 x .. 16 x + 15, per channel
    float ssq[2][kC];               // fused form: sum of squares of each output row's two halves
    Barriers bar;
    uint32_t tmem_base;
    int abort_flag;
};

struct GatedParams {
    int B, T, H;
    int grid_w, prefix_len;
    long long t0;
    float scale;
    int tied;                // key tied to the gate: k = 1 - lambda, no key tensor
    const float* state_in;
    float* state_out;
    int* redo;               // [B*H]: 1 where this kernel gave the chain up (decay too strong), else 0
    int* status;
    unsigned wait_limit;
    float norm_eps;          // fused form: epsilon of the output norm
};

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

// packed bf16 multiply, round to nearest
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

template <bool kFused>
__global__ void __launch_bounds__(kThreads, 2)
prefill_gated_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_g,
                        const __grid_constant__ CUtensorMap tm_o, GatedParams p)
{
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int b = blockIdx.x / p.H, h = blockIdx.x % p.H;
    const int n_chunks = (p.T + kC - 1) / kC;
    volatile int* abort_flag = &sm.abort_flag;
    const unsigned limit = p.wait_limit;

    // ---- set-up ---------------------------------------------------------------------------
    // A kernel launched behind this one as a programmatic dependent may start to take SMs as they
    // become free; it waits for this kernel's completion before it touches device memory.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        mbar_init(&sm.bar.full_in, 1);
        mbar_init(&sm.bar.full_v, 1);
        mbar_init(&sm.bar.scan, kEThreads);
        mbar_init(&sm.bar.in_free, kEThreads);
        mbar_init(&sm.bar.stage_free, 1);
        mbar_init(&sm.bar.x_ready, kEThreads);
        mbar_init(&sm.bar.sb_ready, kEThreads);
        mbar_init(&sm.bar.s_done, 1);
        mbar_init(&sm.bar.ds_done, 1);
        mbar_init(&sm.bar.p_ready, kEThreads);
        mbar_init(&sm.bar.o_done, 1);
        mbar_init(&sm.bar.st_ready, kEThreads);
        mbar_init(&sm.bar.drain, 1);
        sm.abort_flag = 0;
        // nothing above reads or writes device memory; everything below may depend on the kernel
        // before this one in the stream
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

    if (warp == 9) {
        // ===================== TMA warp ========================================================
        // One set of tiles; each is refilled for the next chunk as soon as its last reader is done:
        // gate, query and key once the chunk's scaled operands are written, value once the chunk's
        // MMAs have retired.  The output tile leaves from the K~ buffer.
        if (elect_one()) {
            const unsigned in_bytes = (p.tied ? 2 : 3) * kTileBytes;
            auto issue_in = [&](int n) {
                mbar_arrive_expect_tx(&sm.bar.full_in, in_bytes);
                tma_load_4d(sm.g, &tm_g, &sm.bar.full_in, 0, h, n * kC, b);
                tma_load_4d(sm.q, &tm_q, &sm.bar.full_in, 0, h, n * kC, b);
                if (!p.tied) tma_load_4d(sm.k, &tm_k, &sm.bar.full_in, 0, h, n * kC, b);
            };
            auto issue_v = [&](int n) {
                mbar_arrive_expect_tx(&sm.bar.full_v, kTileBytes);
                tma_load_4d(sm.v, &tm_v, &sm.bar.full_v, 0, h, n * kC, b);
            };
            issue_in(0);
            issue_v(0);
            int in_issued = 1, v_issued = 1;     // chunks whose loads have been issued
            for (int n = 0; n < n_chunks; ++n) {
                const bool more = n + 1 < n_chunks;
                if (more) {
                    if (!mbar_wait(&sm.bar.in_free, n & 1, limit, abort_flag, p.status)) break;
                    issue_in(n + 1);
                    in_issued = n + 2;
                    if (!mbar_wait(&sm.bar.o_done, n & 1, limit, abort_flag, p.status)) break;
                    issue_v(n + 1);
                    v_issued = n + 2;
                }
                if (!mbar_wait(&sm.bar.st_ready, n & 1, limit, abort_flag, p.status)) break;
                tma_store_4d(&tm_o, sm.kt, 0, h, n * kC, b);
                tma_store_commit();
                if (more) {
                    tma_store_wait_read();        // the store has finished reading the buffer
                    mbar_arrive(&sm.bar.stage_free);
                }
            }
            tma_store_wait_all();
            // leave only when every issued load has landed (they write this CTA's shared memory)
            for (unsigned it = 0; it < kTeardownLimit; ++it)
                if (mbar_try_wait(&sm.bar.full_in, (in_issued - 1) & 1)) break;
            for (unsigned it = 0; it < kTeardownLimit; ++it)
                if (mbar_try_wait(&sm.bar.full_v, (v_issued - 1) & 1)) break;
        }
        __syncwarp();
    } else if (warp == 8) {
        // ===================== MMA issuer: the whole warp runs the loop, one lane issues =======
        constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);   // Q~ (K-major) x K~ (K-major)
        constexpr uint32_t idesc_pv = make_idesc(128, 64, 0, 1);   // A (tmem) x V (MN-major)
        constexpr uint32_t idesc_qs = make_idesc(128, 64, 0, 1);   // Q~ (K-major) x state (MN-major)
        constexpr uint32_t idesc_kv = make_idesc(64, 64, 1, 1);    // K~^T (MN-major) x V (MN-major)
        const uint64_t d_sb = make_desc(smem_u32(sm.sb));
        const uint64_t d_q = make_desc(smem_u32(sm.qt));
        const uint64_t d_k = make_desc(smem_u32(sm.kt));
        const uint64_t d_v = make_desc(smem_u32(sm.v));
        for (int n = 0; n < n_chunks; ++n) {
            if (!mbar_wait(&sm.bar.x_ready, n & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)  // 32 bytes along K per step
                    mma_ss(tmem + kColS, d_q + 2 * kk, d_k + 2 * kk, idesc_s, kk > 0);
                mma_commit(&sm.bar.s_done);
            }
            __syncwarp();
            if (!mbar_wait(&sm.bar.full_v, n & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // 16 tokens = 2048 B of K~ and of V per step
                    mma_ss(tmem + kColDS, d_k + 128 * kk, d_v + 128 * kk, idesc_kv, kk > 0);
                mma_commit(&sm.bar.ds_done);
            }
            __syncwarp();
            // the state's contribution opens the O accumulator (its bf16 copy is written while the
            // score MMAs run); A V is added once A is ready
            if (!mbar_wait(&sm.bar.sb_ready, n & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)
                    mma_ss(tmem + kColO, d_q + 2 * kk, d_sb + 128 * kk, idesc_qs, kk > 0);
            }
            __syncwarp();
            if (!mbar_wait(&sm.bar.p_ready, n & 1, limit, abort_flag, p.status)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // A: 8 TMEM columns per step (tokens 0..63 at columns
                                                      // 0..31, tokens 64..127 at 64..95); V: 2048 B per step
                    mma_ts(tmem + kColO, tmem + kColS + (kk < 4 ? 8 * kk : 64 + 8 * (kk - 4)), d_v + 128 * kk,
                           idesc_pv, 1);
                mma_commit(&sm.bar.o_done);
            }
            __syncwarp();
        }
        // make sure nothing is still running on the tensor pipe before TMEM is freed
        if (elect_one()) {
            mma_commit(&sm.bar.drain);
            for (unsigned w = 0; w < kTeardownLimit; ++w)
                if (mbar_try_wait(&sm.bar.drain, 0)) break;
        }
        __syncwarp();
    } else {
        // ===================== element-wise warps ==============================================
        const int qd = warp & 3;                 // TMEM lane quadrant
        const int grp = warp >> 2;               // which half of the quadrant's columns
        const int i = qd * 32 + lane;            // chunk row owned by this thread in the TMEM stages
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        // State ownership as in the scalar-decay kernel: the 16x256b load of the dS accumulator
        // (M = 64 layout) gives this thread, for column group k, st[4k], st[4k+1] = (row r0,
        // columns c0 + 8k, + 1) and st[4k+2], st[4k+3] = (row r0 + 8, same columns).
        const int r0 = qd * 16 + (lane >> 2);
        const int c0 = 32 * grp + 2 * (lane & 3);
        const size_t unit = (size_t)blockIdx.x * kD * kD;
        // Scaling role: rows 16 warp .. 16 warp + 15, channels 2 lane and 2 lane + 1.  Byte offset
        // of that channel pair in row 16 warp + rr of a tile (rows of 128 B, 16-byte pieces
        // swizzled by the row): scale_off + rr * 128 + (((lane >> 2) ^ (rr & 7)) << 4).
        const int scale_off = 16 * warp * 128 + 4 * (lane & 3);
        const int lane_piece = lane >> 2;
        auto row_off = [&](int rr) { return scale_off + rr * 128 + ((lane_piece ^ (rr & 7)) << 4); };

        // SAD rule (Section 3.4) without a division per token: token tok of the chunk at call
        // offset cs is a boundary step iff it lies on the grid and phase + (tok mod w) is 0 or w,
        // with phase = (grid index of the chunk's first token + 1) mod w.
        const int grid_w = p.grid_w;
        int pre = 0, phase = 0, phase_step = 0, rmod[4] = {0, 0, 0, 0};
        {
            const long long g0 = p.t0 - p.prefix_len;   // grid index of the call's first token (may be < 0)
            pre = g0 < 0 ? (int)min(-g0, (long long)0x7fffffff) : 0;
            if (grid_w > 0) {
                long long ph = (g0 + 1) % grid_w;
                if (ph < 0) ph += grid_w;
                phase = (int)ph;
                phase_step = kC % grid_w;
#pragma unroll
                for (int x = 0; x < 4; ++x) rmod[x] = (32 * x + lane) % grid_w;
            }
        }

        float st[16];                            // fp32 master state, this thread's 16 values
#pragma unroll
        for (int e = 0; e < 16; ++e) st[e] = 0.0f;
        if (p.state_in) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 a = *reinterpret_cast<const float2*>(p.state_in + unit + (size_t)r0 * kD + c0 + 8 * k);
                const float2 c = *reinterpret_cast<const float2*>(p.state_in + unit + (size_t)(r0 + 8) * kD + c0 + 8 * k);
                st[4 * k] = a.x; st[4 * k + 1] = a.y; st[4 * k + 2] = c.x; st[4 * k + 3] = c.y;
            }
        }
        // bf16 copy of diag(mult) state for the Q~ x state MMA: [dk][dv] rows of 128 B, 16-byte
        // pieces swizzled by the row; this thread writes eight bf16 pairs
        auto write_state_bf16 = [&](float mult_a, float mult_b) {
            unsigned char* row0 = sm.sb + r0 * 128 + 4 * (lane & 3);
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
        // S_new = diag(f) S_prev + diag(m) dS, with f = m * m (rows r0 and r0 + 8)
        auto update_state = [&](float m_a, float m_b) {
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
        };
        // this thread's 32 columns of output row i -> bf16 -> row i of the staging buffer
        auto stage_output = [&](float f) {
            unsigned char* orow = sm.kt + i * 128;
            uint32_t ov[32];
            tmem_ld32(tmem + lane_base + kColO + 32 * grp, ov);
            tmem_wait_ld();
            if (kFused) {
                // Norm(o_i): sum of squares of this thread's 32 columns, the other 32 from the
                // thread of warp (warp ^ 4) that holds the same row
                float ss = 0.0f;
#pragma unroll
                for (int c = 0; c < 32; ++c) ss = fmaf(__uint_as_float(ov[c]), __uint_as_float(ov[c]), ss);
                sm.ssq[grp][i] = ss;
                asm volatile("bar.sync %0, 64;" ::"r"(1 + qd) : "memory");
                ss += sm.ssq[1 - grp][i];
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

        // which of this warp's 16 rows of the next chunk in line are decaying steps (live and not a
        // row boundary); every call moves on by one chunk
        int mask_chunk = 0;
        auto next_mask = [&]() {
            const int cs = mask_chunk * kC;
            const int Lc = min(kC, p.T - cs);
            unsigned mk[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int tok = 32 * x + lane;
                const int m = phase + rmod[x];
                const bool boundary = grid_w > 0 && cs + tok >= pre && (m == 0 || m == grid_w);
                mk[x] = __ballot_sync(0xffffffffu, tok < Lc && !boundary);
            }
            phase += phase_step;
            if (phase >= grid_w) phase -= grid_w;
            ++mask_chunk;
            const int wx = warp >> 1;
            const unsigned own_word = wx == 0 ? mk[0] : wx == 1 ? mk[1] : wx == 2 ? mk[2] : mk[3];
            return (own_word >> (16 * (warp & 1))) & 0xffffu;
        };
        // first sweep over a chunk's gate tile: the product of the decays over this warp's 16 rows,
        // per channel; only its log2 crosses warps (a boundary step or a row past the end multiplies
        // by 1).  It needs nothing but the gate tile, so it runs as early as that tile is in.
        auto first_sweep = [&](unsigned dec) {
            float p0 = 1.0f, p1 = 1.0f;
#pragma unroll
            for (int rr = 0; rr < 16; ++rr) {
                uint32_t g2 = *reinterpret_cast<const uint32_t*>(sm.g + row_off(rr));
                if (kFused) {
                    // u = Sigmoid(-g~) = 1 / (1 + e^g~) = 1 - lambda, written back in place; lambda = 1 - u
                    // (e^g~ = inf gives u = 0 and e^g~ = 0 gives u = 1: no clamp is needed)
                    const uint32_t u2 = pack_bf16(rcp_approx(1.0f + ex2(1.4426950408889634f * bf16_lo(g2))),
                                                  rcp_approx(1.0f + ex2(1.4426950408889634f * bf16_hi(g2))));
                    *reinterpret_cast<uint32_t*>(sm.g + row_off(rr)) = u2;
                    const uint32_t us = ((dec >> rr) & 1u) ? u2 : 0u;
                    mul2_pair(p0, p1, 1.0f - bf16_lo(us), 1.0f - bf16_hi(us));
                    continue;
                }
                g2 = ((dec >> rr) & 1u) ? g2 : 0x3f803f80u;
                mul2_pair(p0, p1, bf16_lo(g2), bf16_hi(g2));
            }
            // a product that has left the fp32 range reads as -inf and fails the range check
            *reinterpret_cast<float2*>(&sm.segsum[warp][2 * lane]) = make_float2(lg2(p0), lg2(p1));
            mbar_arrive(&sm.bar.scan);
        };

        bool ok = true, given_up = false;
        unsigned dec16 = next_mask();
        ok = mbar_wait(&sm.bar.full_in, 0, limit, abort_flag, p.status);
        if (ok) first_sweep(dec16);
        for (int n = 0; ok && n < n_chunks; ++n) {
            const int Lc = min(kC, p.T - n * kC);
            // the gate pair of row rr of this warp, or (1, 1) where the step does not decay
            auto gate_or_one = [&](uint32_t g2, int rr) { return ((dec16 >> rr) & 1u) ? g2 : 0x3f803f80u; };
            // the decay pair of row rr of this warp in fp32 (fused form: the tile holds u = 1 - lambda)
            auto decay_pair = [&](uint32_t g2, int rr, float& l0, float& l1) {
                if (kFused) {
                    const bool dec = (dec16 >> rr) & 1u;
                    l0 = dec ? 1.0f - bf16_lo(g2) : 1.0f;
                    l1 = dec ? 1.0f - bf16_hi(g2) : 1.0f;
                } else {
                    const uint32_t gx = gate_or_one(g2, rr);
                    l0 = bf16_lo(gx);
                    l1 = bf16_hi(gx);
                }
            };
            if (!(ok = mbar_wait(&sm.bar.scan, n & 1, limit, abort_flag, p.status))) break;

            // ---- this warp's place in the chunk, the chunk's total, the range check ----------------
            float f0, f1;       // 2^(b - r) just before this warp's first row
            float t0, t1;       // 2^(r - b) at this warp's last row
            float tot0 = 0.0f, tot1 = 0.0f;     // log2 of the chunk's total decay, this lane's two channels
            {
                float base0 = 0.0f, base1 = 0.0f;
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const float2 bsx = *reinterpret_cast<const float2*>(&sm.segsum[x][2 * lane]);
                    tot0 += bsx.x; tot1 += bsx.y;
                    if (x < warp) { base0 += bsx.x; base1 += bsx.y; }
                }
                const float2 own = *reinterpret_cast<const float2*>(&sm.segsum[warp][2 * lane]);
                const float h0 = base0 - 0.5f * tot0, h1 = base1 - 0.5f * tot1;
                f0 = ex2(h0); f1 = ex2(h1);
                t0 = ex2(-(h0 + own.x)); t1 = ex2(-(h1 + own.y));
                // (written so that a NaN fails too; a warp's lanes cover all 64 channels)
                if (__any_sync(0xffffffffu, !(fabsf(tot0) <= kSafeRange) || !(fabsf(tot1) <= kSafeRange))) {
                    // decay too strong to scale a whole chunk around one reference: leave the chain
                    // to the CUDA-core kernel (every warp takes the same decision)
                    given_up = true;
                    if (tid == 0) *abort_flag = 1;
                    break;
                }
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
            //      from the warp's last row, so that no factor is ever inverted.  The fp32 factors are
            //      rounded to bf16 and applied with packed bf16 multiplies; the forward pass keeps the
            //      16 decay pairs in registers for the backward pass.  (Rows in groups of eight:
            //      a group's loads are issued before its stores, which the compiler must take to
            //      alias later loads.)
            if (n > 0 && !(ok = mbar_wait(&sm.bar.stage_free, (n - 1) & 1, limit, abort_flag, p.status))) break;
            float ls0[16], ls1[16];     // the 16 decay pairs in fp32, kept for the backward pass
#pragma unroll
            for (int r8 = 0; r8 < 16; r8 += 8) {
                uint32_t g2[8], q2[8];
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    g2[x] = *reinterpret_cast<const uint32_t*>(sm.g + row_off(r8 + x));
                    q2[x] = *reinterpret_cast<const uint32_t*>(sm.q + row_off(r8 + x));
                }
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    decay_pair(g2[x], r8 + x, ls0[r8 + x], ls1[r8 + x]);
                    mul2_pair(f0, f1, ls0[r8 + x], ls1[r8 + x]);
                    if (kFused) {
                        // q = SiLU(q~) = q~ (1 + tanh(q~ / 2)) / 2, scaled in the same step
                        const float x0 = bf16_lo(q2[x]), x1 = bf16_hi(q2[x]);
                        *reinterpret_cast<uint32_t*>(sm.qt + row_off(r8 + x)) =
                            pack_bf16(0.5f * x0 * (1.0f + tanh_approx(0.5f * x0)) * f0,
                                      0.5f * x1 * (1.0f + tanh_approx(0.5f * x1)) * f1);
                    } else {
                        *reinterpret_cast<uint32_t*>(sm.qt + row_off(r8 + x)) = mul_bf16x2(q2[x], pack_bf16(f0, f1));
                    }
                }
            }
            if (!p.tied) {
#pragma unroll
                for (int r8 = 8; r8 >= 0; r8 -= 8) {
                    uint32_t k2[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x) k2[x] = *reinterpret_cast<const uint32_t*>(sm.k + row_off(r8 + x));
#pragma unroll
                    for (int x = 7; x >= 0; --x) {
                        *reinterpret_cast<uint32_t*>(sm.kt + row_off(r8 + x)) = mul_bf16x2(k2[x], pack_bf16(t0, t1));
                        mul2_pair(t0, t1, ls0[r8 + x], ls1[r8 + x]);
                    }
                }
            } else {
                // key tied to the gate: k = 1 - lambda in fp32 (0 on rows past the end of the sequence)
#pragma unroll
                for (int r8 = 8; r8 >= 0; r8 -= 8) {
                    uint32_t g2[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x) g2[x] = *reinterpret_cast<const uint32_t*>(sm.g + row_off(r8 + x));
#pragma unroll
                    for (int x = 7; x >= 0; --x) {
                        const float one = 16 * warp + r8 + x < Lc ? 1.0f : 0.0f;
                        if (kFused)     // the tile holds u = 1 - lambda: the tied key itself
                            *reinterpret_cast<uint32_t*>(sm.kt + row_off(r8 + x)) =
                                pack_bf16(one * bf16_lo(g2[x]) * t0, one * bf16_hi(g2[x]) * t1);
                        else
                            *reinterpret_cast<uint32_t*>(sm.kt + row_off(r8 + x)) =
                                pack_bf16((one - bf16_lo(g2[x])) * t0, (one - bf16_hi(g2[x])) * t1);
                        mul2_pair(t0, t1, ls0[r8 + x], ls1[r8 + x]);
                    }
                }
            }
            if (kFused) fence_proxy_async();      // the gate tile was rewritten in place: order that before its refill
            mbar_arrive(&sm.bar.in_free);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&sm.bar.x_ready);
            // the state's bf16 copy, while the score MMAs run (the previous chunk's MMAs, the last
            // readers of the buffer, were waited for at the end of that chunk)
            write_state_bf16(m_a, m_b);
            fence_proxy_async();
            mbar_arrive(&sm.bar.sb_ready);

            // ---- E1: A = tril(S) -> bf16 over S's own columns (blocks 2 grp, 2 grp + 1 of this
            //      thread's row, kept inside this warp's half of S's columns) -------------------------
            if (!(ok = mbar_wait(&sm.bar.s_done, n & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
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

            // ---- while the O MMAs run: the first sweep of the next chunk, if its gate tile is in
            //      already (it was requested when this chunk's operands were written) --------------
            const bool more = n + 1 < n_chunks;
            unsigned dec_next = 0;
            bool swept = false;
            if (more) {
                dec_next = next_mask();
                swept = __all_sync(0xffffffffu, mbar_test_wait(&sm.bar.full_in, (n + 1) & 1));
                if (swept) first_sweep(dec_next);
            }

            // ---- state carry across the chunk, in fp32 registers -----------------------------------
            if (!(ok = mbar_wait(&sm.bar.ds_done, n & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
            update_state(m_a, m_b);

            // ---- output tile -------------------------------------------------------------------------
            if (!(ok = mbar_wait(&sm.bar.o_done, n & 1, limit, abort_flag, p.status))) break;
            tc_fence_after();
            stage_output(p.scale);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&sm.bar.st_ready);
            if (more && !swept) {
                if (!(ok = mbar_wait(&sm.bar.full_in, (n + 1) & 1, limit, abort_flag, p.status))) break;
                first_sweep(dec_next);
            }
            dec16 = dec_next;
        }
        if (tid == 0) p.redo[blockIdx.x] = given_up ? 1 : 0;
        if (ok && !given_up && p.state_out) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                *reinterpret_cast<float2*>(p.state_out + unit + (size_t)r0 * kD + c0 + 8 * k) = make_float2(st[4 * k], st[4 * k + 1]);
                *reinterpret_cast<float2*>(p.state_out + unit + (size_t)(r0 + 8) * kD + c0 + 8 * k) =
                    make_float2(st[4 * k + 2], st[4 * k + 3]);
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
}

}  // namespace

bool prefill_gated_tc_supported(int dk, int dv, bool bf16) { return bf16 && dk == kD && dv == kD; }

cudaError_t launch_prefill_gated_tc(const KernelArgs& a, const void* gate, int* redo, cudaStream_t st)
{
    CUtensorMap mq, mk, mv, mg, mo;
    // the gate shares the key's strides; without a key tensor its map stands in for the key's
    if (!encode_chunk_map(&mq, a.q, a.B, a.T, a.H, a.qs) || !encode_chunk_map(&mg, gate, a.B, a.T, a.H, a.ks) ||
        !encode_chunk_map(&mk, a.k ? a.k : gate, a.B, a.T, a.H, a.ks) ||
        !encode_chunk_map(&mv, a.v, a.B, a.T, a.H, a.vs) || !encode_chunk_map(&mo, a.o, a.B, a.T, a.H, a.os))
        return cudaErrorInvalidValue;
    GatedParams p;
    p.B = a.B; p.T = a.T; p.H = a.H;
    p.grid_w = a.grid_w; p.prefix_len = a.prefix_len; p.t0 = a.t0; p.scale = a.scale;
    p.tied = a.k ? 0 : 1;
    p.state_in = a.state_in; p.state_out = a.state_out;
    p.redo = redo;
    p.status = a.status; p.wait_limit = a.wait_limit;
    p.norm_eps = a.norm_eps;
    const size_t smem = sizeof(Smem) + 1024;
    auto* kernel = a.fused ? prefill_gated_tc_kernel<true> : prefill_gated_tc_kernel<false>;
    static bool smem_ok[2][64];      // one set of flags per kernel variant
    cudaError_t e = allow_dynamic_smem(kernel, smem, smem_ok[a.fused ? 1 : 0]);
    if (e != cudaSuccess) return e;
    // programmatic dependent launch (see the kernel's first lines)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.B * a.H));
    cfg.blockDim = dim3(kThreads);
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
