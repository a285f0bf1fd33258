// LASAD prefill with the paper's data-dependent gate: a decay vector lambda_t in R^dk per token
// (Algorithm 1: lambda_t = Sigmoid(Linear(x_t)), optionally k_t = 1 - lambda_t), with the SAD rule
// on top (decay 1 on the step that absorbs the last token of a grid row, Section 3.4).
//
// CUDA cores, fp32 arithmetic, one CTA per (batch, head), chunks of C = 16 tokens.  With
// L_i[c] = sum_{u <= i in the chunk} log2(Lambda_u[c]) (Lambda = 1 on boundary steps), every
// decay product between two tokens of a chunk is exp2 of a difference of two L values with a
// non-positive exponent, so nothing is ever divided and nothing can overflow:
//
//     A[i][j] = sum_c q_i[c] k_j[c] exp2(L_i[c] - L_j[c])                      (j <= i)
//     o_i     = scale * ( sum_j A[i][j] v_j  +  sum_c q_i[c] exp2(L_i[c]) S[c][:] )
//     S[c][:] <- exp2(L_last[c]) S[c][:] + sum_j exp2(L_last[c] - L_j[c]) k_j[c] v_j
//
// which is the SAD recurrence (Section 3.4) unrolled over the chunk.  log2 of a decay is clamped
// at -150, below which exp2 is 0 in fp32 anyway, so a decay of exactly 0 needs no special case.
#include "lasad_common.cuh"

namespace lasad {
namespace {

constexpr int kGC = 16;          // chunk length
constexpr float kMinLog2 = -150.0f;

template <typename T, int D>
__global__ void __launch_bounds__(256) prefill_gated_kernel(KernelArgs a, const void* gate_v, int* only)
{
    // Launched as a programmatic dependent: the kernel behind this one may take SMs early, and this
    // one waits here for the kernel before it (whose marks and outputs it reads) to have completed.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // behind the tensor-core kernel: only the chains it gave up are computed here
    if (only && only[blockIdx.x] == 0) return;
    constexpr int LD = D + 1;
    __shared__ float Qs[kGC][LD], Ks[kGC][LD], Vs[kGC][LD], Ls[kGC][LD];   // Ls: cumulative log2 decay
    __shared__ float Ws[kGC][LD];        // exp2(L_last - L_j) k_j
    __shared__ float As[kGC][kGC + 1];
    extern __shared__ float Ss[];        // [D][LD] state

    const int tid = threadIdx.x;
    const int b = blockIdx.x / a.H, h = blockIdx.x % a.H;
    const T* q = static_cast<const T*>(a.q) + b * a.qs[0] + h * a.qs[2];
    const T* k = a.k ? static_cast<const T*>(a.k) + b * a.ks[0] + h * a.ks[2] : nullptr;
    const T* v = static_cast<const T*>(a.v) + b * a.vs[0] + h * a.vs[2];
    const T* lam = static_cast<const T*>(gate_v) + b * a.ks[0] + h * a.ks[2];   // gate shares k's strides
    T* o = static_cast<T*>(a.o) + b * a.os[0] + h * a.os[2];
    const size_t unit = (size_t)blockIdx.x * D * D;

    for (int x = tid; x < D * D; x += 256) Ss[(x / D) * LD + (x % D)] = a.state_in ? a.state_in[unit + x] : 0.0f;

    for (int cs = 0; cs < a.T; cs += kGC) {
        const int L = min(kGC, a.T - cs);
        __syncthreads();     // the previous chunk's readers are done; the state is visible
        for (int x = tid; x < kGC * D; x += 256) {
            const int r = x / D, c = x % D;
            const bool in = r < L;
            const long long t = cs + r;
            float g = 1.0f, kk = 0.0f, qq = 0.0f;
            if (in) {
                g = io<T>::load(lam + t * a.ks[1] + c);
                qq = io<T>::load(q + t * a.qs[1] + c);
                float tied = 1.0f - g;
                if (a.fused) {
                    // Algorithm 1's activations: lambda = Sigmoid(gate), q = SiLU(q)
                    sigmoid_pair(g, g, tied);
                    qq = silu(qq);
                }
                kk = k ? io<T>::load(k + t * a.ks[1] + c) : tied;          // key tied to the gate
                if (is_boundary_step(a.t0 + t, a.grid_w, a.prefix_len)) g = 1.0f;   // SAD rule
            }
            Qs[r][c] = qq;
            Ks[r][c] = kk;
            Vs[r][c] = in ? io<T>::load(v + t * a.vs[1] + c) : 0.0f;
            Ls[r][c] = g > 0.0f ? fmaxf(log2f(g), kMinLog2) : kMinLog2;   // log2 Lambda for now
        }
        __syncthreads();
        // cumulative log2 decay per channel (rows past the end keep the last value: decay 1)
        if (tid < D) {
            float run = 0.0f;
#pragma unroll
            for (int r = 0; r < kGC; ++r) {
                run += Ls[r][tid];
                Ls[r][tid] = run;
            }
        }
        __syncthreads();
        // decayed scores of the lower triangle, and the keys weighted for the state update
        {
            const int i = tid >> 4, j = tid & 15;
            float s = 0.0f;
            if (j <= i) {
#pragma unroll 8
                for (int c = 0; c < D; ++c) s = fmaf(Qs[i][c] * Ks[j][c], exp2f(Ls[i][c] - Ls[j][c]), s);
            }
            As[i][j] = s;
            for (int x = tid; x < kGC * D; x += 256) {
                const int r = x / D, c = x % D;
                Ws[r][c] = Ks[r][c] * exp2f(Ls[kGC - 1][c] - Ls[r][c]);
            }
        }
        __syncthreads();
        // outputs: each thread owns row i = tid / 16 and the columns e = tid % 16 + 16 m
        {
            const int i = tid >> 4, e0 = tid & 15;
            float acc[D / 16];
#pragma unroll
            for (int m = 0; m < D / 16; ++m) acc[m] = 0.0f;
            for (int j = 0; j <= i; ++j) {
                const float p = As[i][j];
#pragma unroll
                for (int m = 0; m < D / 16; ++m) acc[m] = fmaf(p, Vs[j][e0 + 16 * m], acc[m]);
            }
#pragma unroll 4
            for (int c = 0; c < D; ++c) {
                const float qc = Qs[i][c] * exp2f(Ls[i][c]);
#pragma unroll
                for (int m = 0; m < D / 16; ++m) acc[m] = fmaf(qc, Ss[c * LD + e0 + 16 * m], acc[m]);
            }
            float norm = 1.0f;
            if (a.fused) {
                // Norm(o_t): weight-free RMS over the row's D channels, which sit in 16 adjacent lanes
                float ss = 0.0f;
#pragma unroll
                for (int m = 0; m < D / 16; ++m) ss = fmaf(a.scale * acc[m], a.scale * acc[m], ss);
#pragma unroll
                for (int off = 8; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
                norm = rsqrtf(ss * (1.0f / D) + a.norm_eps);
            }
            if (i < L) {
                const long long t = cs + i;
#pragma unroll
                for (int m = 0; m < D / 16; ++m) io<T>::store(o + t * a.os[1] + e0 + 16 * m, a.scale * acc[m] * norm);
            }
        }
        __syncthreads();
        // state carry to the end of the chunk: thread owns rows c = tid / 16 + 16 n, columns as above
        {
            const int cr = tid >> 4, e0 = tid & 15;
#pragma unroll
            for (int n = 0; n < D / 16; ++n) {
                const int c = cr + 16 * n;
                const float gl = exp2f(Ls[kGC - 1][c]);
                float acc[D / 16];
#pragma unroll
                for (int m = 0; m < D / 16; ++m) acc[m] = gl * Ss[c * LD + e0 + 16 * m];
#pragma unroll
                for (int j = 0; j < kGC; ++j) {
                    const float w = Ws[j][c];
#pragma unroll
                    for (int m = 0; m < D / 16; ++m) acc[m] = fmaf(w, Vs[j][e0 + 16 * m], acc[m]);
                }
#pragma unroll
                for (int m = 0; m < D / 16; ++m) Ss[c * LD + e0 + 16 * m] = acc[m];
            }
        }
    }
    __syncthreads();
    if (a.state_out)
        for (int x = tid; x < D * D; x += 256) a.state_out[unit + x] = Ss[(x / D) * LD + (x % D)];
    if (only && tid == 0) only[blockIdx.x] = 0;      // the mark has been served
}

template <typename T, int D>
cudaError_t launch_gated_t(const KernelArgs& a, const void* gate, int* only, bool early, cudaStream_t st)
{
    const size_t smem = sizeof(float) * D * (D + 1);
    // (`early`: a programmatic dependent launch; behind the CTA-per-chain tensor-core kernel the
    // launch latency then overlaps that kernel's tail)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.B * a.H));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, prefill_gated_kernel<T, D>, a, gate, only);
}

}  // namespace

cudaError_t launch_prefill_gated(const KernelArgs& a, const void* gate, int dk, bool bf16, int* only, bool early,
                                 cudaStream_t st)
{
    if (dk == 64)
        return bf16 ? launch_gated_t<__nv_bfloat16, 64>(a, gate, only, early, st) : launch_gated_t<float, 64>(a, gate, only, early, st);
    return bf16 ? launch_gated_t<__nv_bfloat16, 32>(a, gate, only, early, st) : launch_gated_t<float, 32>(a, gate, only, early, st);
}

}  // namespace lasad
