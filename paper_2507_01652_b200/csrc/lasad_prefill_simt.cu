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
#include "lasad_common.cuh"

namespace lasad {
namespace {

template <typename T, int D, int C>
__global__ void __launch_bounds__(256) prefill_simt_kernel(KernelArgs a)
{
    constexpr int LD = D + 1;            // padded row length against bank conflicts
    constexpr int RT = C / 16;           // chunk rows per thread (16 row-threads)
    constexpr int CT = D / 16;           // channel columns per thread (16 column-threads)
    constexpr int JT = C / 16;           // score columns per thread
    constexpr int ST = D / 16;           // state rows per thread
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
    const int b = blockIdx.x / a.H, h = blockIdx.x % a.H;
    const T* q = static_cast<const T*>(a.q) + b * a.qs[0] + h * a.qs[2];
    const T* k = static_cast<const T*>(a.k) + b * a.ks[0] + h * a.ks[2];
    const T* v = static_cast<const T*>(a.v) + b * a.vs[0] + h * a.vs[2];
    T* o = static_cast<T*>(a.o) + b * a.os[0] + h * a.os[2];
    const size_t unit = (size_t)blockIdx.x * D * D;

    const double gamma = (double)a.decay[h];
    for (int m = tid; m <= C; m += 256) pw[m] = (float)pow(gamma, (double)m);
    for (int x = tid; x < D * D; x += 256) {
        const int r = x / D, c = x % D;
        Ss[r * LD + c] = a.state_in ? a.state_in[unit + x] : 0.0f;
    }

    for (int cs = 0; cs < a.T; cs += C) {
        const int L = min(C, a.T - cs);
        __syncthreads();  // previous chunk's readers of Q/K/V/n are done; pw/S are visible
        for (int x = tid; x < C * D; x += 256) {
            const int r = x / D, c = x % D;
            const bool in = r < L;
            const long long t = cs + r;
            Qs[r * LD + c] = in ? io<T>::load(q + t * a.qs[1] + c) : 0.0f;
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
        for (int ri = 0; ri < RT; ++ri) {
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
        __syncthreads();

        // outputs: intra-chunk part plus the carried state
#pragma unroll
        for (int ri = 0; ri < RT; ++ri) {
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
        __syncthreads();

        // state carry to the end of the chunk
        {
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
    if (a.state_out) {
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

template <typename T, int D, int C>
cudaError_t launch_simt_t(const KernelArgs& a, cudaStream_t st)
{
    constexpr size_t smem = simt_smem_bytes<D, C>();
    cudaError_t e = cudaFuncSetAttribute(prefill_simt_kernel<T, D, C>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    prefill_simt_kernel<T, D, C><<<(unsigned)(a.B * a.H), 256, smem, st>>>(a);
    return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_simt_d(const KernelArgs& a, int chunk, cudaStream_t st)
{
    switch (chunk) {
        case 16: return launch_simt_t<T, D, 16>(a, st);
        case 32: return launch_simt_t<T, D, 32>(a, st);
        case 64: return launch_simt_t<T, D, 64>(a, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_prefill_simt(const KernelArgs& a, int dk, int dv, bool bf16, int chunk,
                                cudaStream_t st)
{
    (void)dv;
    if (dk == 64)
        return bf16 ? launch_simt_d<__nv_bfloat16, 64>(a, chunk, st) : launch_simt_d<float, 64>(a, chunk, st);
    return bf16 ? launch_simt_d<__nv_bfloat16, 32>(a, chunk, st) : launch_simt_d<float, 32>(a, chunk, st);
}

}  // namespace lasad
