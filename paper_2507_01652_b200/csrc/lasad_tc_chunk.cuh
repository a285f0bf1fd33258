// What the tensor-core (sm_100a) prefill kernels share about one 128-token chunk: tile and TMEM
// geometry, and the decay bookkeeping of the SAD rule (Section 3.4) from the tokens' positions
// on the grid.
#pragma once
#include <stdint.h>

namespace lasad {
namespace tcx {

constexpr int kC = 128;                    // chunk length (tokens) = MMA M
constexpr int kD = 64;                     // d_k = d_v
constexpr int kEThreads = 256;             // element-wise warps 0-7 of a pipeline
constexpr int kTileBytes = kC * kD * 2;    // 16 KB: one [128 x 64] bf16 tile, 128 B rows
constexpr uint32_t kColS = 0;      // S (fp32, 128 columns); A/P (bf16 pairs) aliases columns 0..31 and 64..95
constexpr uint32_t kColO = 128;    // O accumulator, 64 columns
constexpr uint32_t kColDS = 192;   // dS accumulator (M = 64 layout), 64 columns
constexpr unsigned kTeardownLimit = 1u << 26;
// Scalar-decay kernels: from this decay on every factor gamma^-m, m <= 128, stays far inside fp32
// range and all decay can sit on V and one output row factor; below it only factors with
// non-negative exponents are formed.
constexpr float kFastPathMinDecay = 0.6f;

// Decay bookkeeping of one chunk, computed by every warp on its own with four ballots (one per
// 32-token block): which steps decay, and from their popcounts n_i for the thread's own row.
struct ChunkDecay {
    unsigned m0, m1, m2, m3;   // bit l of m<x>: token 32 x + l of the chunk is a decaying step
    int c0, c1, c2;            // decaying steps up to the end of block 0, 1, 2
    int ni;                    // n of the thread's own row
    int n_last;                // n of the chunk's last token
    // n of chunk column j (warp-uniform j)
    __device__ __forceinline__ int n_of(int j) const
    {
        const int x = j >> 5;
        const unsigned m = x == 0 ? m0 : x == 1 ? m1 : x == 2 ? m2 : m3;
        const int before = x == 0 ? 0 : x == 1 ? c0 : x == 2 ? c1 : c2;
        return before + __popc(m & (0xffffffffu >> (31 - (j & 31))));
    }
};

// Where a run of chunks sits on the token grid, in a form that needs no division inside the
// chunk loop: token `tok` of the chunk that starts at offset cs of the run absorbs the last token
// of a grid row (a boundary step, SAD rule of Section 3.4) iff it lies on the grid
// (cs + tok >= pre) and (phase + r[tok / 32]) is 0 or w, where r = (tok mod w) is fixed per
// thread and phase = (grid column of the chunk's first token + 1) mod w advances by
// (128 mod w) per chunk.
struct GridPos {
    int grid_w;
    int pre;         // tokens of the run that precede the grid (class-token prefix)
    int r[4];        // (32 x + lane) mod w
    int step;        // 128 mod w
    int phase;       // ((grid index of the current chunk's first token) + 1) mod w
    // moves on by one chunk without looking at it
    __device__ __forceinline__ void skip()
    {
        phase += step;
        if (phase >= grid_w) phase -= grid_w;
    }
};

// t_first: absolute index of the run's first token.
__device__ __forceinline__ GridPos grid_pos_init(int grid_w, int prefix_len, long long t_first, int lane)
{
    GridPos g;
    g.grid_w = grid_w;
    const long long g0 = t_first - prefix_len;   // grid index of the run's first token (may be < 0)
    g.pre = g0 < 0 ? (int)min(-g0, (long long)0x7fffffff) : 0;
    g.step = 0; g.phase = 0;
#pragma unroll
    for (int x = 0; x < 4; ++x) g.r[x] = 0;
    if (grid_w > 0) {
        long long ph = (g0 + 1) % grid_w;    // C remainder: may be negative inside the prefix
        if (ph < 0) ph += grid_w;
        g.phase = (int)ph;
        g.step = kC % grid_w;
#pragma unroll
        for (int x = 0; x < 4; ++x) g.r[x] = (32 * x + lane) % grid_w;
    }
    return g;
}

// Decay bookkeeping of the chunk at offset cs of the run (L live tokens); advances g to the next
// chunk.  qd: the 32-token block that holds the thread's own row.
__device__ __forceinline__ ChunkDecay chunk_decay(GridPos& g, int cs, int L, int qd, int lane)
{
    ChunkDecay d;
    unsigned mk[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int tok = 32 * x + lane;
        const int m = g.phase + g.r[x];
        const bool boundary = g.grid_w > 0 && cs + tok >= g.pre && (m == 0 || m == g.grid_w);
        mk[x] = __ballot_sync(0xffffffffu, tok < L && !boundary);
    }
    d.m0 = mk[0]; d.m1 = mk[1]; d.m2 = mk[2]; d.m3 = mk[3];
    d.c0 = __popc(d.m0);
    d.c1 = d.c0 + __popc(d.m1);
    d.c2 = d.c1 + __popc(d.m2);
    d.n_last = d.c2 + __popc(d.m3);
    g.skip();
    const unsigned own = qd == 0 ? d.m0 : qd == 1 ? d.m1 : qd == 2 ? d.m2 : d.m3;
    const int before = qd == 0 ? 0 : qd == 1 ? d.c0 : qd == 2 ? d.c1 : d.c2;
    d.ni = before + __popc(own & (0xffffffffu >> (31 - lane)));
    return d;
}

}  // namespace tcx
}  // namespace lasad
