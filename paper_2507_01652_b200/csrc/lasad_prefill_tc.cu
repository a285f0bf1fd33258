// LASAD chunked prefill on the 5th-generation tensor cores (sm_100a): TMA-fed tcgen05.mma with
// TMEM accumulators, bf16 I/O, fp32 accumulation and an fp32 master state.
//
// One CTA owns one (batch, head) and walks its sequence in chunks of C = 128 tokens; two CTAs
// fit on an SM (256 TMEM columns and ~105 KB of shared memory each) so that one CTA's
// tensor-core and TMA latencies are covered by the other's CUDA-core work.  Per chunk, with
// n_i = number of decaying steps from the chunk start up to token i (SAD rule, Section 3.4,
// from the token's grid position) and gamma the head's decay:
//
//   M1  S  = Q K^T                                  tcgen05.mma  128x128x64   (smem x smem)
//   E1  P  = S o gamma^(n_i - n_j) o [j <= i]  -> bf16 back into TMEM over S's columns;
//       Q~ = diag(gamma^(n_i)) Q,  K~ = diag(gamma^(n_last - n_j)) K   in place in smem
//   M2  O  = P V + Q~ S_prev                        tcgen05.mma  128x64x128 (tmem x smem) + 128x64x64
//       dS = K~^T V                                 tcgen05.mma  64x64x128
//   E2  o  = scale * O -> bf16 -> smem -> TMA store
//   E3  S_new = gamma^(n_last) S_prev + dS          fp32 registers; bf16 copy to smem for M2
//
// which is the SAD recurrence (Section 3.4) unrolled over the chunk.  Every power of gamma has
// an integer exponent in [0, 128] and comes from a per-CTA table, so gamma = 0 is exact.
//
// Warp roles: warps 0-3 do E1/E2/E3 (thread i owns chunk row i = TMEM lane i), warp 4 issues
// the TMA loads, warp 5 allocates TMEM and issues every MMA.  All waits are bounded: a wait that
// runs out raises a status word the host can read and the CTA leaves through the normal exit
// (copies in flight are waited for, TMEM is freed).
#include "lasad_common.cuh"

#include <cuda.h>

namespace lasad {
namespace {

constexpr int kC = 128;            // chunk length (tokens) = MMA M
constexpr int kD = 64;             // d_k = d_v
constexpr int kThreads = 192;
constexpr int kTileBytes = kC * kD * 2;          // 16 KB: one [128 x 64] bf16 tile, 128 B rows
constexpr int kStages = 2;
constexpr int kTmemCols = 256;
constexpr uint32_t kColS = 0;      // S (fp32, 128 columns); P (bf16 pairs) aliases columns 0..63
constexpr uint32_t kColO = 128;    // O accumulator, 64 columns
constexpr uint32_t kColDS = 192;   // dS accumulator (M = 64 layout), 64 columns
constexpr unsigned kTeardownLimit = 1u << 26;

struct __align__(8) Barriers {
    unsigned long long full[kStages];
    unsigned long long empty[kStages];
    unsigned long long s_done;     // M1 complete
    unsigned long long p_ready;    // E1 complete (P in TMEM, Q~/K~/S_bf16 in smem)
    unsigned long long o_done;     // M2 complete
    unsigned long long drain;      // teardown: all MMAs retired
};

struct Smem {
    // tiles first: each must sit on a 1024-byte boundary (128-byte swizzle atom = 8 rows)
    unsigned char q[kStages][kTileBytes];
    unsigned char k[kStages][kTileBytes];
    unsigned char v[kStages][kTileBytes];
    unsigned char sb[kD * kD * 2];  // bf16 copy of the state, [dk][dv], 128 B rows, swizzled
    float pw[kC + 4];               // gamma^m, m = 0..128
    int nj[kC];                     // n_j of the current chunk
    int warp_cnt[4];
    Barriers bar;
    uint32_t tmem_base;
    int abort_flag;
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(void* bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(void* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(void* bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void* bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Gives up after `limit` polls or as soon as another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(void* bar, unsigned parity, unsigned limit, volatile int* abort_flag,
                                          int* status)
{
    for (unsigned it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status, 1);
    return false;
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, void* bar, int c0, int c1, int c2,
                                            int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, const void* src, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// 64-bit shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// kind::f16 instruction descriptor: bf16 x bf16 -> fp32
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int a_mn_major, int b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void mma_commit(void* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(addr)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// AND-reduction of a predicate over the 128 threads of warps 0-3 (named barrier 1).
__device__ __forceinline__ bool wg_all(bool ok)
{
    unsigned r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((unsigned)ok)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ void wg_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);  // .x (low 16 bits) = lo
    return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Multiply the 64 bf16 values of one 128-byte tile row by a scalar, in place (fp32 product,
// one rounding).  The swizzle permutes 16-byte pieces within the row, so a row-uniform factor
// needs no address arithmetic.
__device__ __forceinline__ void scale_row_inplace(unsigned char* row, float f)
{
    uint4* p = reinterpret_cast<uint4*>(row);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint4 x = p[c];
        x.x = pack_bf16(bf16_lo(x.x) * f, bf16_hi(x.x) * f);
        x.y = pack_bf16(bf16_lo(x.y) * f, bf16_hi(x.y) * f);
        x.z = pack_bf16(bf16_lo(x.z) * f, bf16_hi(x.z) * f);
        x.w = pack_bf16(bf16_lo(x.w) * f, bf16_hi(x.w) * f);
        p[c] = x;
    }
}

struct TcParams {
    int B, T, H;
    int grid_w, prefix_len;
    long long t0;
    float scale;
    const float* decay;
    const float* state_in;
    float* state_out;
    int* status;
    unsigned wait_limit;
};

__global__ void __launch_bounds__(kThreads, 2)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, TcParams p)
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
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.bar.full[s], 1);
            mbar_init(&sm.bar.empty[s], 1);
        }
        mbar_init(&sm.bar.s_done, 1);
        mbar_init(&sm.bar.p_ready, 128);
        mbar_init(&sm.bar.o_done, 1);
        mbar_init(&sm.bar.drain, 1);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid < 128) {
        // gamma^m for m = 0..128 in double precision (0^0 = 1)
        const double g = (double)p.decay[h];
        sm.pw[tid] = (float)pow(g, (double)tid);
        if (tid == 0) sm.pw[kC] = (float)pow(g, (double)kC);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 4) {
        // ===================== TMA producer ===============================================
        if (lane == 0) {
            int issued = 0;
            for (int n = 0; n < n_chunks; ++n) {
                const int s = n % kStages;
                if (n >= kStages) {
                    if (!mbar_wait(&sm.bar.empty[s], ((n / kStages) - 1) & 1, limit, abort_flag, p.status)) break;
                }
                mbar_arrive_expect_tx(&sm.bar.full[s], 3 * kTileBytes);
                tma_load_4d(sm.q[s], &tm_q, &sm.bar.full[s], 0, h, n * kC, b);
                tma_load_4d(sm.k[s], &tm_k, &sm.bar.full[s], 0, h, n * kC, b);
                tma_load_4d(sm.v[s], &tm_v, &sm.bar.full[s], 0, h, n * kC, b);
                issued = n + 1;
            }
            // leave only when every issued load has landed (they write this CTA's shared memory)
            for (int n = max(0, issued - kStages); n < issued; ++n) {
                const int s = n % kStages;
                for (unsigned it = 0; it < kTeardownLimit; ++it)
                    if (mbar_try_wait(&sm.bar.full[s], (n / kStages) & 1)) break;
            }
        }
    } else if (warp == 5) {
        // ===================== MMA issuer =================================================
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);   // Q (K-major) x K (K-major)
            constexpr uint32_t idesc_pv = make_idesc(128, 64, 0, 1);   // P (tmem) x V (MN-major)
            constexpr uint32_t idesc_qs = make_idesc(128, 64, 0, 1);   // Q~ (K-major) x S (MN-major)
            constexpr uint32_t idesc_kv = make_idesc(64, 64, 1, 1);    // K~^T (MN-major) x V (MN-major)
            const uint64_t d_sb = make_desc(smem_u32(sm.sb));
            bool ok = true;
            auto issue_m1 = [&](int n) {
                const int s = n % kStages;
                if (!mbar_wait(&sm.bar.full[s], (n / kStages) & 1, limit, abort_flag, p.status)) return false;
                tc_fence_after();
                const uint64_t dq = make_desc(smem_u32(sm.q[s])), dk = make_desc(smem_u32(sm.k[s]));
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)  // 32 bytes along K per step
                    mma_ss(tmem + kColS, dq + 2 * kk, dk + 2 * kk, idesc_s, kk > 0);
                mma_commit(&sm.bar.s_done);
                return true;
            };
            ok = n_chunks > 0 && issue_m1(0);
            for (int n = 0; ok && n < n_chunks; ++n) {
                const int s = n % kStages;
                if (!mbar_wait(&sm.bar.p_ready, n & 1, limit, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint64_t dq = make_desc(smem_u32(sm.q[s])), dk = make_desc(smem_u32(sm.k[s]));
                const uint64_t dv = make_desc(smem_u32(sm.v[s]));
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)  // P: 8 columns per step; V: 16 rows = 2048 B per step
                    mma_ts(tmem + kColO, tmem + kColS + 8 * kk, dv + 128 * kk, idesc_pv, kk > 0);
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)
                    mma_ss(tmem + kColO, dq + 2 * kk, d_sb + 128 * kk, idesc_qs, 1);
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)
                    mma_ss(tmem + kColDS, dk + 128 * kk, dv + 128 * kk, idesc_kv, kk > 0);
                mma_commit(&sm.bar.o_done);
                if (n + 1 < n_chunks) ok = issue_m1(n + 1);
            }
            // make sure nothing is still running on the tensor pipe before TMEM is freed
            mma_commit(&sm.bar.drain);
            for (unsigned it = 0; it < kTeardownLimit; ++it)
                if (mbar_try_wait(&sm.bar.drain, 0)) break;
        }
    } else {
        // ===================== E1 / E2 / E3: thread i owns chunk row i ====================
        const int i = tid;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const int srow = warp * 16 + lane;       // state row held by lanes 0..15 (M = 64 TMEM layout)
        const bool has_state = lane < 16;
        const size_t unit = (size_t)blockIdx.x * kD * kD;
        float st[kD];
#pragma unroll
        for (int e = 0; e < kD; ++e) st[e] = 0.0f;
        if (has_state && p.state_in) {
            const float4* src = reinterpret_cast<const float4*>(p.state_in + unit + (size_t)srow * kD);
#pragma unroll
            for (int e4 = 0; e4 < kD / 4; ++e4) {
                const float4 t = src[e4];
                st[4 * e4] = t.x; st[4 * e4 + 1] = t.y; st[4 * e4 + 2] = t.z; st[4 * e4 + 3] = t.w;
            }
        }
        auto write_state_bf16 = [&]() {
            if (has_state) {
                uint4* row = reinterpret_cast<uint4*>(sm.sb + srow * 128);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint4 x;
                    x.x = pack_bf16(st[8 * c], st[8 * c + 1]);
                    x.y = pack_bf16(st[8 * c + 2], st[8 * c + 3]);
                    x.z = pack_bf16(st[8 * c + 4], st[8 * c + 5]);
                    x.w = pack_bf16(st[8 * c + 6], st[8 * c + 7]);
                    row[c ^ (srow & 7)] = x;
                }
            }
        };
        write_state_bf16();

        bool ok = true;
        for (int n = 0; n < n_chunks; ++n) {
            const int s = n % kStages;
            const int cs = n * kC;
            const int L = min(kC, p.T - cs);

            // ---- decay bookkeeping: n_i by ballot + popcount over the chunk --------------------
            const long long abs_i = p.t0 + cs + i;
            const bool decays = i < L && !is_boundary_step(abs_i, p.grid_w, p.prefix_len);
            const unsigned m = __ballot_sync(0xffffffffu, decays);
            if (lane == 0) sm.warp_cnt[warp] = __popc(m);
            wg_sync();
            int ni = __popc(m & (0xffffffffu >> (31 - lane)));
            int n_last = 0;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const int c = sm.warp_cnt[w];
                if (w < warp) ni += c;
                n_last += c;
            }
            sm.nj[i] = ni;

            ok = wg_all(mbar_wait(&sm.bar.s_done, n & 1, limit, abort_flag, p.status));  // also publishes nj
            if (!ok) break;
            tc_fence_after();

            // ---- E1: P = S o decay o causal, written over S as bf16 pairs -----------------------
#pragma unroll 1
            for (int pc = 0; pc < 4; ++pc) {
                uint32_t pk[16];
                if (pc <= warp) {
                    uint32_t sv[32];
                    tmem_ld32(tmem + lane_base + kColS + 32 * pc, sv);
                    tmem_wait_ld();
                    float val[32];
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        const int j = 32 * pc + jj;
                        const int dn = ni - sm.nj[j];
                        const float w = sm.pw[dn > 0 ? dn : 0];
                        val[jj] = (j <= i) ? __uint_as_float(sv[jj]) * w : 0.0f;
                    }
#pragma unroll
                    for (int c = 0; c < 16; ++c) pk[c] = pack_bf16(val[2 * c], val[2 * c + 1]);
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) pk[c] = 0u;
                }
                tmem_st16(tmem + lane_base + kColS + 16 * pc, pk);
            }
            // Q~ and K~ in place (M1 has finished reading both tiles)
            scale_row_inplace(sm.q[s] + i * 128, sm.pw[ni]);
            scale_row_inplace(sm.k[s] + i * 128, sm.pw[n_last - ni]);
            tmem_wait_st();
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&sm.bar.p_ready);

            // ---- E2: o = scale * O -> bf16 -> smem (the Q tile's buffer) -> TMA store -----------
            ok = wg_all(mbar_wait(&sm.bar.o_done, n & 1, limit, abort_flag, p.status));
            if (!ok) break;
            tc_fence_after();
            {
                unsigned char* orow = sm.q[s] + i * 128;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t ov[32];
                    tmem_ld32(tmem + lane_base + kColO + 32 * half, ov);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 x;
                        x.x = pack_bf16(p.scale * __uint_as_float(ov[8 * c]), p.scale * __uint_as_float(ov[8 * c + 1]));
                        x.y = pack_bf16(p.scale * __uint_as_float(ov[8 * c + 2]), p.scale * __uint_as_float(ov[8 * c + 3]));
                        x.z = pack_bf16(p.scale * __uint_as_float(ov[8 * c + 4]), p.scale * __uint_as_float(ov[8 * c + 5]));
                        x.w = pack_bf16(p.scale * __uint_as_float(ov[8 * c + 6]), p.scale * __uint_as_float(ov[8 * c + 7]));
                        reinterpret_cast<uint4*>(orow)[(4 * half + c) ^ (i & 7)] = x;
                    }
                }
            }
            fence_proxy_async();
            wg_sync();
            if (tid == 0) {
                tma_store_4d(&tm_o, sm.q[s], 0, h, cs, b);
                tma_store_commit();
            }

            // ---- E3: S_new = gamma^(n_last) S_prev + dS (fp32 master in registers) --------------
            {
                const float gl = sm.pw[n_last];
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t dv_[32];
                    tmem_ld32(tmem + lane_base + kColDS + 32 * half, dv_);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        st[32 * half + e] = fmaf(gl, st[32 * half + e], __uint_as_float(dv_[e]));
                }
                write_state_bf16();
            }
            tc_fence_before();
            if (tid == 0) {
                tma_store_wait_read();            // the store has finished reading the Q buffer
                mbar_arrive(&sm.bar.empty[s]);    // stage s may be refilled
            }
        }
        if (ok && has_state && p.state_out) {
            float4* dst = reinterpret_cast<float4*>(p.state_out + unit + (size_t)srow * kD);
#pragma unroll
            for (int e4 = 0; e4 < kD / 4; ++e4)
                dst[e4] = make_float4(st[4 * e4], st[4 * e4 + 1], st[4 * e4 + 2], st[4 * e4 + 3]);
        }
        if (tid == 0) tma_store_wait_all();
    }

    // ---- teardown ---------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// cuTensorMapEncodeTiled, fetched through the runtime so that the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// [B,T,H,64] bf16 with element strides (b,t,h) -> 4-D map (d, h, t, b), box = one chunk of one head.
bool encode_map(CUtensorMap* map, const void* base, int B, int T, int H, const long long* strides)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    auto bytes = [](long long elems) { return (cuuint64_t)(elems > 0 ? elems * 2 : 128); };
    const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B};
    const cuuint64_t gstr[3] = {bytes(strides[2]), bytes(strides[1]), bytes(strides[0])};
    const cuuint32_t box[4] = {(cuuint32_t)kD, 1u, (cuuint32_t)kC, 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, gstr, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool prefill_tc_supported(int dk, int dv, bool bf16) { return bf16 && dk == kD && dv == kD; }

cudaError_t launch_prefill_tc(const KernelArgs& a, cudaStream_t st)
{
    CUtensorMap mq, mk, mv, mo;
    if (!encode_map(&mq, a.q, a.B, a.T, a.H, a.qs) || !encode_map(&mk, a.k, a.B, a.T, a.H, a.ks) ||
        !encode_map(&mv, a.v, a.B, a.T, a.H, a.vs) || !encode_map(&mo, a.o, a.B, a.T, a.H, a.os))
        return cudaErrorInvalidValue;
    TcParams p;
    p.B = a.B; p.T = a.T; p.H = a.H;
    p.grid_w = a.grid_w; p.prefix_len = a.prefix_len; p.t0 = a.t0; p.scale = a.scale;
    p.decay = a.decay; p.state_in = a.state_in; p.state_out = a.state_out;
    p.status = a.status; p.wait_limit = a.wait_limit;
    const size_t smem = sizeof(Smem) + 1024;
    cudaError_t e = cudaFuncSetAttribute(prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    prefill_tc_kernel<<<(unsigned)(a.B * a.H), kThreads, smem, st>>>(mq, mk, mv, mo, p);
    return cudaGetLastError();
}

}  // namespace lasad
