// The work plan of the balanced tensor-core prefill kernels (one CTA per SM, two chunk pipelines
// on one chain): which chunks of which chains a CTA takes, in which order, and how a chain's
// state crosses from one CTA to another.  See lasad_prefill_tc_pair.cu for the reasons.
#pragma once
#include "lasad_tc_chunk.cuh"
#include "lasad_tc_ptx.cuh"

namespace lasad {
namespace tcx {

constexpr int kSlotBytes = kD * kD * 8;          // one hand-off slot: dk x dv (value, tag) packets

// A unit: consecutive chunks of one chain that the CTA works through in one go.  Local chunk
// g = 0 .. n_local-1 counts the CTA's chunks in the order it takes them.
struct Unit {
    int g0, g1;       // local chunks [g0, g1) ...
    int chain, n0;    // ... are chunks n0 .. of `chain`
    int recv;         // slot the unit's starting state comes from; -1: the chain starts here (n0 = 0)
    int send;         // slot the unit's final state goes to; -1: the chain ends here
};

// The CTA's work: up to four units that involve a piece of a left-over chain (the piece, a second
// piece where the CTA's share straddles two left-over chains, and the parts of the CTA's first
// own chain around them), then whole chains.
constexpr int kMaxSpecial = 4;
struct Plan {
    int n_local;      // chunks of this CTA
    int nc;           // chunks per chain
    int n_special;
    int special_len;  // chunks of the special units
    int rho;          // this CTA's place among the chains of a round
    int stride;       // chains per round (= CTAs)
    Unit special[kMaxSpecial];
};
constexpr int kHandoffMargin = 3;   // chunks a CTA stays on its own chain beyond the nominal start of its piece, per hop
constexpr int kMinPiece = 4;        // shortest piece (chunks) a left-over chain is cut into

__device__ __forceinline__ Unit unit_of(const Plan& pl, int g)
{
    if (g < pl.special_len) {
        int i = 0;
        while (i + 1 < pl.n_special && g >= pl.special[i].g1) ++i;
        return pl.special[i];
    }
    Unit u;
    const int r = (g - pl.special_len) / pl.nc;      // whole chains: round r + 1
    u.g0 = pl.special_len + r * pl.nc; u.g1 = u.g0 + pl.nc;
    u.chain = (r + 1) * pl.stride + pl.rho; u.n0 = 0; u.recv = -1; u.send = -1;
    return u;
}

// How the left-over chains (E chains of nc chunks, laid end to end) are shared out: `hosts` CTAs
// take one piece each, CTA c the chunks [c X / hosts, (c + 1) X / hosts) of that sequence.
struct Leftover {
    int E;            // left-over chains
    int hosts;        // CTAs that take a piece (the first `hosts` in start order)
    long long X;      // E * nc
};
__device__ __forceinline__ Leftover leftover_of(int chains, int nc, int n_ctas)
{
    Leftover lo;
    lo.E = chains > n_ctas ? chains % n_ctas : 0;
    lo.X = (long long)lo.E * nc;
    // short chains are not cut at all; long ones into pieces of at least kMinPiece chunks
    if (lo.E == 0) lo.hosts = 0;
    else if (nc < 2 * kMinPiece) lo.hosts = lo.E;
    else lo.hosts = (int)min((long long)n_ctas, max(1LL, lo.X / kMinPiece));
    return lo;
}
// chunk (within its left-over chain) at which CTA c's piece starts; INT_MAX for a CTA without one
__device__ __forceinline__ int piece_start(const Leftover& lo, int nc, int c)
{
    if (c >= lo.hosts) return 0x7fffffff;
    return (int)(((long long)c * lo.X / lo.hosts) % nc);
}

// Hand-off slot layout: element-wise thread t's values 2k, 2k+1 are the two packets of the 16 bytes
// at (k * 256 + t) * 16, so a warp touches 512 contiguous bytes per access.  `tag` is the launch's
// number (below 2^31); bit 31 of the packets' tag is free for one flag that travels with the state.
__device__ __forceinline__ void slot_send(unsigned char* slot, int t, const float (&st)[16], unsigned tag, bool flag = false)
{
    const unsigned long long hi = (unsigned long long)(tag | (flag ? 0x80000000u : 0u)) << 32;
#pragma unroll
    for (int k = 0; k < 8; ++k)
        st_cg_v2u64(slot + ((size_t)k * kEThreads + t) * 16, hi | __float_as_uint(st[2 * k]), hi | __float_as_uint(st[2 * k + 1]));
}
// Asks for this thread's part of a slot to be brought into L2.  A slot that was written tens of
// microseconds ago has been pushed out to DRAM by the kernel's own traffic, and a DRAM read under
// that load takes several microseconds: issued one chunk ahead, it is over by the time the state
// is wanted.
__device__ __forceinline__ void slot_prefetch(const unsigned char* slot, int t)
{
#pragma unroll
    for (int k = 0; k < 8; ++k)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(slot + ((size_t)k * kEThreads + t) * 16));
}
// Bounded: polls until all sixteen packets carry `tag`; `flag` (if given) receives the sender's flag.
__device__ __forceinline__ bool slot_receive(const unsigned char* slot, int t, float (&st)[16], unsigned tag, unsigned limit,
                                             volatile int* abort_flag, int* status, bool* flag = nullptr)
{
    for (unsigned it = 0; it < limit; ++it) {
        unsigned long long a[8], b[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) ld_cg_v2u64(slot + ((size_t)k * kEThreads + t) * 16, a[k], b[k]);
        bool all = true;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            all = all && ((unsigned)(a[k] >> 32) & 0x7fffffffu) == tag && ((unsigned)(b[k] >> 32) & 0x7fffffffu) == tag;
        if (all) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                st[2 * k] = __uint_as_float((unsigned)a[k]);
                st[2 * k + 1] = __uint_as_float((unsigned)b[k]);
            }
            if (flag) *flag = (a[0] >> 63) != 0;
            return true;
        }
        __nanosleep(200);
        if ((it & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status, 1);
    return false;
}

// A CTA's own chain waits in its own slot while the CTA works on a piece.  Nobody else touches
// that slot, so it needs no tags: plain fp32 (the first 16 KiB of the slot, thread t's values
// 4k .. 4k+3 at (k * 256 + t) * 16), ordered between writer and reader by the mbarriers that the
// chunks in between pass through.  Its read is asked for one chunk ahead, into L1: a load issued
// when the state is wanted would queue behind the SM's bulk copies for microseconds.
__device__ __forceinline__ void park_send(unsigned char* slot, int t, const float (&st)[16])
{
#pragma unroll
    for (int k = 0; k < 4; ++k)
        *reinterpret_cast<float4*>(slot + ((size_t)k * kEThreads + t) * 16) = make_float4(st[4 * k], st[4 * k + 1], st[4 * k + 2], st[4 * k + 3]);
}
__device__ __forceinline__ void park_prefetch(const unsigned char* slot, int t)
{
#pragma unroll
    for (int k = 0; k < 4; ++k)
        asm volatile("prefetch.global.L1 [%0];" ::"l"(slot + ((size_t)k * kEThreads + t) * 16));
}
__device__ __forceinline__ void park_receive(const unsigned char* slot, int t, float (&st)[16])
{
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        float4 x;
        asm volatile("ld.global.ca.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w)
                     : "l"(slot + ((size_t)k * kEThreads + t) * 16));
        st[4 * k] = x.x; st[4 * k + 1] = x.y; st[4 * k + 2] = x.z; st[4 * k + 3] = x.w;
    }
}

// Fills `plan` (shared memory) for the CTA with start-order number `cta`; every thread of the CTA
// (n_threads of them) must call it, and a __syncthreads() must follow before the plan is read.
__device__ __forceinline__ void build_plan(Plan& plan, int cta, int chains, int nc, int n_threads)
{
    const int n_ctas = (int)gridDim.x;
    const Leftover lo = leftover_of(chains, nc, n_ctas);
    // rho: this CTA's rank by the chunk at which it takes up its piece (CTAs without one last)
    const int my_start = piece_start(lo, nc, cta);
    int before = 0;
    for (int c0 = 0; c0 < n_ctas; c0 += n_threads) {
        const int c = c0 + (int)threadIdx.x;
        const int st_c = c < n_ctas ? piece_start(lo, nc, c) : 0x7fffffff;
        before += __syncthreads_count(c < n_ctas && (st_c < my_start || (st_c == my_start && c < cta)));
    }
    if (threadIdx.x == 0) {
        Plan pl;
        pl.nc = nc;
        pl.rho = before;
        pl.stride = n_ctas;
        const int rounds = chains > n_ctas ? chains / n_ctas : 1;
        const int own = pl.rho;                      // the CTA's chain of round 0
        const int first_extra = rounds * n_ctas;     // index of the first left-over chain
        int ns = 0, g = 0;
        auto add = [&](int chain, int n0, int len, int recv, int send) {
            Unit& u = pl.special[ns++];
            u.g0 = g; u.g1 = g + len; u.chain = chain; u.n0 = n0; u.recv = recv; u.send = send;
            g += len;
        };
        if (cta < lo.hosts) {
            const long long xlo = (long long)cta * lo.X / lo.hosts, xhi = (long long)(cta + 1) * lo.X / lo.hosts;
            const int e1 = (int)(xlo / nc);
            const int a1 = (int)(xlo - (long long)e1 * nc);
            const int b1 = (int)min((long long)nc, xhi - (long long)e1 * nc);
            const int b2 = (int)(xhi - (long long)(e1 + 1) * nc);      // > 0: the share runs on into the next chain
            if (b2 > 0) add(first_extra + e1 + 1, 0, b2, -1, b2 < nc ? cta + 1 : -1);
            if (a1 == 0) {
                add(first_extra + e1, 0, b1, -1, b1 < nc ? cta + 1 : -1);
                add(own, 0, nc, -1, -1);
            } else {
                // pieces before this one in its chain: each may run late by the margin
                const int hops = cta - (int)((long long)e1 * nc * lo.hosts / lo.X);
                int p1 = a1 + kHandoffMargin * max(hops, 1) - g;
                p1 = max(0, min(nc, p1));
                if (p1 > 0) add(own, 0, p1, -1, p1 < nc ? n_ctas + cta : -1);
                add(first_extra + e1, a1, b1 - a1, cta, b1 < nc ? cta + 1 : -1);
                if (p1 < nc) add(own, p1, nc - p1, p1 > 0 ? n_ctas + cta : -1, -1);
            }
        } else {
            add(own, 0, nc, -1, -1);
        }
        pl.n_special = ns;
        pl.special_len = g;
        pl.n_local = g + (rounds - 1) * nc;
        plan = pl;
    }
}

}  // namespace tcx
}  // namespace lasad
