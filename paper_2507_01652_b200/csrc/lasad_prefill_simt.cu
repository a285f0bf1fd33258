// LASAD chunked prefill on CUDA cores, fp32 arithmetic throughout.
//
// This is the accuracy-first prefill (the fp32-I/O configuration needs max|err|/max|ref| <= 1e-4,
// which single-pass reduced-precision tensor-core inputs do not give) and the reference the
// tensor-core kernel is brought up against.  One CTA owns one (batch, head) and walks the
// sequence in chunks of C tokens.  For a chunk whose first token has absolute index i0, with
// n_i = number of decaying steps in (i0-1, i]  (from the tokens' (row, col) grid positions, SAD
// rule of Section 3.4) and gamma the head's decay:
//
//     P[i][j] = (q_i . k_j) * gamma^(n_i - n_j)            for j <= i, else 0
//     o_i     = scale * ( sum_j P[i][j] v_j  +  gamma^(n_i) * q_i^T S )
//     S      <- gamma^(n_last) * S + sum_j gamma^(n_last - n_j) k_j v_j^T
//
// which is the SAD recurrence (Section 3.4) unrolled over the chunk.  All powers of gamma have
// an integer exponent in [0, C] and come from a per-CTA table computed in double precision, so
// gamma = 0 (0^0 = 1) and long sequences need no special care.
//
// Few chains: one CTA per chain leaves the device idle and a chain's chunks run one after the
// other.  The recurrence is linear in the state: over a segment [a, b) of a chain
//     S_b = gamma^(decaying steps in [a, b)) S_a + L,     L = the state the segment reaches from zero,
// so the chains are cut into segments of whole chunks.  A first launch (kStateOnly) computes L for
// every segment but a chain's last from K and V alone; the second launch runs one CTA per segment,
// which first rebuilds its starting state from the L of the segments before it (a handful of
// 4 - 16 KiB reads) and then walks its chunks as usual.  The caller's incoming state is copied into
// the scratch by the first launch, so state_out may alias state_in.
#include "lasad_common.cuh"
#include "lasad_tc_tma.cuh"

namespace lasad {
namespace {

// How the chains are cut (n_segs = 1: not at all).  scratch: [n_segs][B * H][D * D] floats; slot 0
// of a chain is its incoming state, slot s >= 1 the state segment s - 1 reaches from zero.
struct SimtSegs {
    int n_segs;
    int seg_chunks;      // chunks per segment (the last one may be shorter)
    float* scratch;
};

template <typename T, int D, int C, bool kStateOnly>
__global__ void __launch_bounds__(256) prefill_simt_kernel(KernelArgs a, SimtSegs sg)
{
    constexpr int LD = D + 1;            // padded row length against bank conflicts
    constexpr int RT = C / 16;           // chunk rows per thread (16 row-threads)
    constexpr int CT = D / 16;           // channel columns per thread (16 column-threads)
    constexpr int JT = C / 16;           // score columns per thread
    constexpr int ST = D / 16;           // state rows per thread
    // Launched as a programmatic dependent: the kernel behind this one (the main pass behind the
    // state pass, the next call behind this one) may bring its CTAs onto the SMs early; this one
    // waits for the kernel before it to have completed before it touches device memory.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    extern __shared__ float smem[];
    float* Qs = smem;                    // [C][LD]
    float* Ks = Qs + C * LD;             // [C][LD]
    float* Vs = Ks + C * LD;             // [C][LD]
    float* Ps = Vs + C * LD;             // [C][C+1]
    float* Ss = Ps + C * (C + 1);        // [D][LD]
    float* pw = Ss + D * LD;             // [C+1]  gamma^m
    int* ne = reinterpret_cast<int*>(pw + C + 1);  // [C] n_i

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int n_chains = a.B * a.H;
    const int chain = blockIdx.x % n_chains, seg = blockIdx.x / n_chains;
    const int b = chain / a.H, h = chain % a.H;
    // this CTA's tokens: [t_begin, t_end) of the call
    const int t_begin = sg.n_segs > 1 ? seg * sg.seg_chunks * C : 0;
    const int t_end = sg.n_segs > 1 ? min(a.T, (seg + 1) * sg.seg_chunks * C) : a.T;
    const T* q = static_cast<const T*>(a.q) + b * a.qs[0] + h * a.qs[2];
    const T* k = static_cast<const T*>(a.k) + b * a.ks[0] + h * a.ks[2];
    const T* v = static_cast<const T*>(a.v) + b * a.vs[0] + h * a.vs[2];
    T* o = static_cast<T*>(a.o) + b * a.os[0] + h * a.os[2];
    const size_t unit = (size_t)chain * D * D;
    const size_t slot_stride = (size_t)n_chains * D * D;      // from one segment's slot to the next

    const double gamma = (double)a.decay[h];
    // gamma^m by binary exponentiation in double precision (0^0 = 1)
    auto dpow = [&](long long m) {
        double base = gamma, acc = 1.0;
        for (; m > 0; m >>= 1) {
            if (m & 1) acc *= base;
            base *= base;
        }
        return acc;
    };
    for (int m = tid; m <= C; m += 256) pw[m] = (float)dpow(m);
    if (kStateOnly) {
        // L of this segment, from zero; segment 0's CTA also files the incoming state
        for (int x = tid; x < D * D; x += 256) {
            Ss[(x / D) * LD + (x % D)] = 0.0f;
            if (seg == 0) sg.scratch[unit + x] = a.state_in ? a.state_in[unit + x] : 0.0f;
        }
    } else if (sg.n_segs > 1) {
        // the state at the start of this segment: sum over the slots before it (slot 0: the incoming
        // state, slot s + 1: what segment s reaches from zero), each weighted by gamma^(decaying steps
        // from the end of what the slot stands for to the start of this segment); the weights go
        // through Ps, which nothing else uses yet, and the slots' loads are independent of one another
        const long long seg_tokens = (long long)sg.seg_chunks * C;
        const long long here = decay_steps_upto(a.t0 + seg * seg_tokens - 1, a.grid_w, a.prefix_len);
        for (int s2 = tid; s2 <= seg; s2 += 256) {
            const long long upto = s2 == 0 ? decay_steps_upto(a.t0 - 1, a.grid_w, a.prefix_len)
                                           : decay_steps_upto(a.t0 + s2 * seg_tokens - 1, a.grid_w, a.prefix_len);
            Ps[s2] = (float)dpow(here - upto);
        }
        __syncthreads();
        for (int x = tid; x < D * D; x += 256) {
            float acc = 0.0f;
#pragma unroll 4
            for (int s2 = 0; s2 <= seg; ++s2) acc = fmaf(Ps[s2], sg.scratch[(size_t)s2 * slot_stride + unit + x], acc);
            Ss[(x / D) * LD + (x % D)] = acc;
        }
    } else {
        for (int x = tid; x < D * D; x += 256) {
            const int r = x / D, c = x % D;
            Ss[r * LD + c] = a.state_in ? a.state_in[unit + x] : 0.0f;
        }
    }

    for (int cs = t_begin; cs < t_end; cs += C) {
        const int L = min(C, a.T - cs);
        __syncthreads();  // previous chunk's readers of Q/K/V/n are done; pw/S are visible
        for (int x = tid; x < C * D; x += 256) {
            const int r = x / D, c = x % D;
            const bool in = r < L;
            const long long t = cs + r;
            if (!kStateOnly) Qs[r * LD + c] = in ? io<T>::load(q + t * a.qs[1] + c) : 0.0f;
            Ks[r * LD + c] = in ? io<T>::load(k + t * a.ks[1] + c) : 0.0f;
            Vs[r * LD + c] = in ? io<T>::load(v + t * a.vs[1] + c) : 0.0f;
        }
        if (tid < C) {
            const long long base = decay_steps_upto(a.t0 + cs - 1, a.grid_w, a.prefix_len);
            const long long i = a.t0 + cs + min(tid, L - 1);
            ne[tid] = (int)(decay_steps_upto(i, a.grid_w, a.prefix_len) - base);
        }
        __syncthreads();

        // decayed, causally masked scores
#pragma unroll
        for (int ri = 0; ri < (kStateOnly ? 0 : RT); ++ri) {
            const int i = ty + 16 * ri;
#pragma unroll
            for (int ji = 0; ji < JT; ++ji) {
                const int j = tx + 16 * ji;
                float s = 0.0f;
                if (j <= i) {
#pragma unroll 8
                    for (int c = 0; c < D; ++c) s = fmaf(Qs[i * LD + c], Ks[j * LD + c], s);
                    s *= pw[ne[i] - ne[j]];
                }
                Ps[i * (C + 1) + j] = s;
            }
        }
        if (!kStateOnly) __syncthreads();

        // outputs: intra-chunk part plus the carried state
#pragma unroll
        for (int ri = 0; ri < (kStateOnly ? 0 : RT); ++ri) {
            const int i = ty + 16 * ri;
            float intra[CT], inter[CT];
#pragma unroll
            for (int ci = 0; ci < CT; ++ci) intra[ci] = inter[ci] = 0.0f;
            for (int j = 0; j <= i; ++j) {
                const float p = Ps[i * (C + 1) + j];
#pragma unroll
                for (int ci = 0; ci < CT; ++ci) intra[ci] = fmaf(p, Vs[j * LD + tx + 16 * ci], intra[ci]);
            }
#pragma unroll 8
            for (int c = 0; c < D; ++c) {
                const float qc = Qs[i * LD + c];
#pragma unroll
                for (int ci = 0; ci < CT; ++ci) inter[ci] = fmaf(qc, Ss[c * LD + tx + 16 * ci], inter[ci]);
            }
            if (i < L) {
                const float ri_w = pw[ne[i]];
                const long long t = cs + i;
#pragma unroll
                for (int ci = 0; ci < CT; ++ci)
                    io<T>::store(o + t * a.os[1] + tx + 16 * ci, a.scale * fmaf(ri_w, inter[ci], intra[ci]));
            }
        }
        if (!kStateOnly) __syncthreads();

        // state carry to the end of the chunk (not after the last chunk of a segment whose state nobody wants)
        if (kStateOnly || cs + C < t_end || t_end == a.T) {
            const int nl = ne[L - 1];
            const float gl = pw[nl];
#pragma unroll
            for (int si = 0; si < ST; ++si) {
                const int c = ty + 16 * si;
                float acc[CT];
#pragma unroll
                for (int ci = 0; ci < CT; ++ci) acc[ci] = gl * Ss[c * LD + tx + 16 * ci];
                for (int j = 0; j < L; ++j) {
                    const float kw = Ks[j * LD + c] * pw[nl - ne[j]];
#pragma unroll
                    for (int ci = 0; ci < CT; ++ci) acc[ci] = fmaf(kw, Vs[j * LD + tx + 16 * ci], acc[ci]);
                }
#pragma unroll
                for (int ci = 0; ci < CT; ++ci) Ss[c * LD + tx + 16 * ci] = acc[ci];
            }
        }
    }
    __syncthreads();
    if (kStateOnly) {
        float* dst = sg.scratch + (size_t)(seg + 1) * slot_stride + unit;
        for (int x = tid; x < D * D; x += 256) dst[x] = Ss[(x / D) * LD + (x % D)];
    } else if (a.state_out && t_end == a.T) {
        // the final state leaves with a chain's last segment
        for (int x = tid; x < D * D; x += 256) {
            const int r = x / D, c = x % D;
            a.state_out[unit + x] = Ss[r * LD + c];
        }
    }
}

template <int D, int C> constexpr size_t simt_smem_bytes()
{
    return sizeof(float) * (3 * C * (D + 1) + C * (C + 1) + D * (D + 1) + (C + 1)) + sizeof(int) * C;
}

// Segments per chain: as many as there are CTA slots per chain (two per SM), each of whole chunks.
inline int simt_segments(int n_chunks, long long chains, int sms, size_t scratch_floats, int D)
{
    long long segs = chains > 0 ? 2LL * sms / chains : 1;
    if (segs > n_chunks) segs = n_chunks;
    while (segs > 1 && (size_t)segs * chains * D * D > scratch_floats) --segs;
    if (segs < 2) return 1;
    const int len = (int)((n_chunks + segs - 1) / segs);
    return (n_chunks + len - 1) / len;
}

template <typename T, int D, int C>
cudaError_t launch_simt_t(const KernelArgs& a, float* scratch, size_t scratch_floats, int sms, cudaStream_t st)
{
    constexpr size_t smem = simt_smem_bytes<D, C>();
    static bool ok_main[64], ok_state[64];
    cudaError_t e = tcx::allow_dynamic_smem(prefill_simt_kernel<T, D, C, false>, smem, ok_main);
    if (e == cudaSuccess) e = tcx::allow_dynamic_smem(prefill_simt_kernel<T, D, C, true>, smem, ok_state);
    if (e != cudaSuccess) return e;
    const long long chains = (long long)a.B * a.H;
    const int n_chunks = (a.T + C - 1) / C;
    SimtSegs sg;
    sg.n_segs = scratch ? simt_segments(n_chunks, chains, sms, scratch_floats, D) : 1;
    sg.seg_chunks = sg.n_segs > 1 ? (n_chunks + sg.n_segs - 1) / sg.n_segs : n_chunks;
    sg.scratch = scratch;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (sg.n_segs > 1) {
        cfg.gridDim = dim3((unsigned)(chains * (sg.n_segs - 1)));
        e = cudaLaunchKernelEx(&cfg, prefill_simt_kernel<T, D, C, true>, a, sg);
        if (e != cudaSuccess) return e;
    }
    cfg.gridDim = dim3((unsigned)(chains * sg.n_segs));
    return cudaLaunchKernelEx(&cfg, prefill_simt_kernel<T, D, C, false>, a, sg);
}

template <typename T, int D>
cudaError_t launch_simt_d(const KernelArgs& a, int chunk, float* scratch, size_t scratch_floats, int sms, cudaStream_t st)
{
    switch (chunk) {
        case 16: return launch_simt_t<T, D, 16>(a, scratch, scratch_floats, sms, st);
        case 32: return launch_simt_t<T, D, 32>(a, scratch, scratch_floats, sms, st);
        case 64: return launch_simt_t<T, D, 64>(a, scratch, scratch_floats, sms, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

int prefill_simt_launches(int T, int dk, int chunk, long long chains, int sms, size_t scratch_floats)
{
    return simt_segments((T + chunk - 1) / chunk, chains, sms, scratch_floats, dk) > 1 ? 2 : 1;
}

cudaError_t launch_prefill_simt(const KernelArgs& a, int dk, int dv, bool bf16, int chunk, float* scratch,
                                size_t scratch_floats, int sms, cudaStream_t st)
{
    (void)dv;
    if (dk == 64)
        return bf16 ? launch_simt_d<__nv_bfloat16, 64>(a, chunk, scratch, scratch_floats, sms, st)
                    : launch_simt_d<float, 64>(a, chunk, scratch, scratch_floats, sms, st);
    return bf16 ? launch_simt_d<__nv_bfloat16, 32>(a, chunk, scratch, scratch_floats, sms, st)
                : launch_simt_d<float, 32>(a, chunk, scratch, scratch_floats, sms, st);
}

}  // namespace lasad
