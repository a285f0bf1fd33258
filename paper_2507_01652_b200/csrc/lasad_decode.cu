// LASAD decode step (Algorithm 1's loop body for one token): one fused pass over the
// persistent fp32 state per (batch, head):
//     S <- g * S + k v^T   (in place),   o = scale * q^T S
// The kernel is HBM-bound on the state (8*dk*dv bytes per (b,h): one read, one write), so the
// whole design is about streaming it with coalesced 128-bit accesses and enough loads in
// flight; the decay bookkeeping is a warp-shuffle column reduction.
#include "lasad_common.cuh"

namespace lasad {
namespace {

template <typename T> __device__ inline void load4(const T* p, float (&x)[4]);
template <> __device__ inline void load4<float>(const float* p, float (&x)[4])
{
    const float4 t = *reinterpret_cast<const float4*>(p);
    x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
}
template <> __device__ inline void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&x)[4])
{
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    x[0] = __uint_as_float(t.x << 16); x[1] = __uint_as_float(t.x & 0xffff0000u);
    x[2] = __uint_as_float(t.y << 16); x[3] = __uint_as_float(t.y & 0xffff0000u);
}
template <typename T> __device__ inline void store4(T* p, const float (&x)[4]);
template <> __device__ inline void store4<float>(float* p, const float (&x)[4])
{
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
}
template <> __device__ inline void store4<__nv_bfloat16>(__nv_bfloat16* p, const float (&x)[4])
{
    __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(x[2], x[3]);
    uint2 t;
    t.x = *reinterpret_cast<unsigned*>(&a);
    t.y = *reinterpret_cast<unsigned*>(&b);
    *reinterpret_cast<uint2*>(p) = t;
}

// TPU threads cooperate on one (b,h) state of D x D floats.  A state row is D/4 float4s, so
// CG = D/4 adjacent threads cover one row and a warp covers 32/CG consecutive rows: every
// warp-wide load or store is one contiguous 512-byte run.
// POS: every sequence has its own position a.pos[b] (and grid width a.widths[b]).
// GATED: the decay is the paper's data-dependent gate, a value per (batch, head, key channel)
// read from `gate` with q's layout, and the key may be tied to it (k = 1 - lambda when a.k is
// null); otherwise it is the per-head constant a.decay[h].
// FUSED (with GATED): q and the gate are pre-activations (q <- SiLU(q), lambda <- Sigmoid(gate))
// and o leaves through a weight-free RMS norm over its D channels (Algorithm 1's loop body whole).
template <typename T, int D, int TPU, bool GATED, bool POS, bool FUSED = false>
__global__ void __launch_bounds__(256) decode_kernel(KernelArgs a, int decay_on, const void* gate_v)
{
    static_assert(!FUSED || GATED, "the fused form exists for the gated operator");
    constexpr int CG = D / 4;          // threads per state row
    constexpr int RPP = TPU / CG;      // rows covered per pass
    constexpr int PASSES = D / RPP;    // float4s per thread
    constexpr int BATCH = PASSES < 8 ? PASSES : 8;  // loads kept in flight per thread
    constexpr int UPC = 256 / TPU;     // (b,h) units per CTA
    constexpr int WPU = TPU / 32;      // warps per unit
    static_assert(TPU % 32 == 0 && RPP >= 1 && PASSES % BATCH == 0, "bad decode tiling");

    __shared__ float red[UPC][WPU > 1 ? WPU : 1][D];

    // Launched as a programmatic dependent: the kernel behind this one (the next step, as a rule)
    // may bring its CTAs onto the SMs while this one runs, and this one waits here for the kernel
    // before it (whose state it reads) to have completed.  Nothing above touches device memory.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const int tid = threadIdx.x;
    const int lt = tid % TPU;
    const int cg = lt % CG;
    const int r0 = lt / CG;
    const long long n_units = (long long)a.B * a.H;
    const long long unit = (long long)blockIdx.x * UPC + tid / TPU;
    const bool live = unit < n_units;

    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (live) {
        const int b = (int)(unit / a.H), h = (int)(unit % a.H);
        const T* q = static_cast<const T*>(a.q) + b * a.qs[0] + h * a.qs[2];
        const T* k = (!GATED || a.k) ? static_cast<const T*>(a.k) + b * a.ks[0] + h * a.ks[2] : nullptr;
        const T* lam = GATED ? static_cast<const T*>(gate_v) + b * a.ks[0] + h * a.ks[2] : nullptr;
        const T* v = static_cast<const T*>(a.v) + b * a.vs[0] + h * a.vs[2];
        float* S = a.state_out + unit * (D * D) + r0 * D + cg * 4;
        if (POS) {
            // every sequence at its own position (and grid width): the SAD rule per batch element
            const int w = a.widths ? a.widths[b] : a.grid_w;
            decay_on = !is_boundary_step(a.pos[b], w, a.prefix_len);
        }
        const float g = GATED ? 1.0f : (decay_on ? a.decay[h] : 1.0f);
        float vv[4];
        load4<T>(v + cg * 4, vv);

#pragma unroll
        for (int p0 = 0; p0 < PASSES; p0 += BATCH) {
            float4 s[BATCH];
            float qr[BATCH], kr[BATCH];
            float gr[GATED ? BATCH : 1];
#pragma unroll
            for (int u = 0; u < BATCH; ++u)
                s[u] = *reinterpret_cast<const float4*>(S + (size_t)(p0 + u) * RPP * D);
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int row = r0 + (p0 + u) * RPP;
                qr[u] = io<T>::load(q + row);
                if (FUSED) qr[u] = silu(qr[u]);
                if (GATED) {
                    float lr = io<T>::load(lam + row);
                    float tied = 1.0f - lr;
                    if (FUSED) sigmoid_pair(lr, lr, tied);
                    kr[u] = k ? io<T>::load(k + row) : tied;          // key tied to the gate
                    gr[u] = decay_on ? lr : 1.0f;                      // SAD rule: 1 on a boundary step
                } else {
                    kr[u] = io<T>::load(k + row);
                }
            }
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const float gu = GATED ? gr[GATED ? u : 0] : g;
                s[u].x = fmaf(gu, s[u].x, kr[u] * vv[0]);
                s[u].y = fmaf(gu, s[u].y, kr[u] * vv[1]);
                s[u].z = fmaf(gu, s[u].z, kr[u] * vv[2]);
                s[u].w = fmaf(gu, s[u].w, kr[u] * vv[3]);
                acc[0] = fmaf(qr[u], s[u].x, acc[0]);
                acc[1] = fmaf(qr[u], s[u].y, acc[1]);
                acc[2] = fmaf(qr[u], s[u].z, acc[2]);
                acc[3] = fmaf(qr[u], s[u].w, acc[3]);
                *reinterpret_cast<float4*>(S + (size_t)(p0 + u) * RPP * D) = s[u];
            }
        }
    }
    // column sums over the rows held by the lanes of this warp that share a column group
#pragma unroll
    for (int off = CG; off < 32; off <<= 1) {
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], off);
    }
    if (WPU == 1) {
        if (live && (tid & 31) < CG) {
            const int b = (int)(unit / a.H), h = (int)(unit % a.H);
            T* o = static_cast<T*>(a.o) + b * a.os[0] + h * a.os[2];
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[c] *= a.scale;
            if (FUSED) {
                // Norm(o): the D channels sit in lanes 0 .. CG-1, four each
                float ss = acc[0] * acc[0] + acc[1] * acc[1] + acc[2] * acc[2] + acc[3] * acc[3];
#pragma unroll
                for (int off = CG / 2; off >= 1; off >>= 1) ss += __shfl_xor_sync((1u << CG) - 1u, ss, off);
                const float nrm = rsqrtf(ss * (1.0f / D) + a.norm_eps);
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[c] *= nrm;
            }
            store4<T>(o + cg * 4, acc);
        }
    } else {
        const int ul = tid / TPU, wu = lt / 32;
        if ((tid & 31) < CG) {
#pragma unroll
            for (int c = 0; c < 4; ++c) red[ul][wu][cg * 4 + c] = acc[c];
        }
        __syncthreads();
        if (live && lt < CG) {
            float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int w = 0; w < WPU; ++w)
#pragma unroll
                for (int c = 0; c < 4; ++c) sum[c] += red[ul][w][cg * 4 + c];
            const int b = (int)(unit / a.H), h = (int)(unit % a.H);
            T* o = static_cast<T*>(a.o) + b * a.os[0] + h * a.os[2];
#pragma unroll
            for (int c = 0; c < 4; ++c) sum[c] *= a.scale;
            if (FUSED) {
                float ss = sum[0] * sum[0] + sum[1] * sum[1] + sum[2] * sum[2] + sum[3] * sum[3];
#pragma unroll
                for (int off = CG / 2; off >= 1; off >>= 1) ss += __shfl_xor_sync((1u << CG) - 1u, ss, off);
                const float nrm = rsqrtf(ss * (1.0f / D) + a.norm_eps);
#pragma unroll
                for (int c = 0; c < 4; ++c) sum[c] *= nrm;
            }
            store4<T>(o + cg * 4, sum);
        }
    }
}

template <typename T, int D, bool GATED, bool POS, bool FUSED = false>
cudaError_t launch_decode_t(const KernelArgs& a, bool decay_on, int tpu, const void* gate, cudaStream_t st)
{
    const long long n_units = (long long)a.B * a.H;
    const int on = decay_on ? 1 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaSuccess;
#define LASAD_DECODE_CASE(TPU_)                                                               \
    case TPU_: {                                                                              \
        const long long blocks = (n_units + (256 / TPU_) - 1) / (256 / TPU_);                 \
        cfg.gridDim = dim3((unsigned)blocks);                                                 \
        e = cudaLaunchKernelEx(&cfg, decode_kernel<T, D, TPU_, GATED, POS, FUSED>, a, on, gate); \
        break;                                                                                \
    }
    switch (tpu) {
        LASAD_DECODE_CASE(32)
        LASAD_DECODE_CASE(64)
        LASAD_DECODE_CASE(128)
        LASAD_DECODE_CASE(256)
        default: return cudaErrorInvalidValue;
    }
#undef LASAD_DECODE_CASE
    return e;
}

}  // namespace

cudaError_t launch_decode(const KernelArgs& a, int dk, int dv, bool bf16, bool decay_on, int tpu,
                          cudaStream_t st)
{
    (void)dv;
    if (a.pos) {
        if (dk == 64) {
            return bf16 ? launch_decode_t<__nv_bfloat16, 64, false, true>(a, decay_on, tpu, nullptr, st)
                        : launch_decode_t<float, 64, false, true>(a, decay_on, tpu, nullptr, st);
        }
        return bf16 ? launch_decode_t<__nv_bfloat16, 32, false, true>(a, decay_on, tpu, nullptr, st)
                    : launch_decode_t<float, 32, false, true>(a, decay_on, tpu, nullptr, st);
    }
    if (dk == 64) {
        return bf16 ? launch_decode_t<__nv_bfloat16, 64, false, false>(a, decay_on, tpu, nullptr, st)
                    : launch_decode_t<float, 64, false, false>(a, decay_on, tpu, nullptr, st);
    }
    return bf16 ? launch_decode_t<__nv_bfloat16, 32, false, false>(a, decay_on, tpu, nullptr, st)
                : launch_decode_t<float, 32, false, false>(a, decay_on, tpu, nullptr, st);
}

cudaError_t launch_decode_gated(const KernelArgs& a, const void* gate, int dk, bool bf16, bool decay_on, int tpu,
                                cudaStream_t st)
{
    if (a.fused) {
        if (dk == 64) {
            return bf16 ? launch_decode_t<__nv_bfloat16, 64, true, false, true>(a, decay_on, tpu, gate, st)
                        : launch_decode_t<float, 64, true, false, true>(a, decay_on, tpu, gate, st);
        }
        return bf16 ? launch_decode_t<__nv_bfloat16, 32, true, false, true>(a, decay_on, tpu, gate, st)
                    : launch_decode_t<float, 32, true, false, true>(a, decay_on, tpu, gate, st);
    }
    if (dk == 64) {
        return bf16 ? launch_decode_t<__nv_bfloat16, 64, true, false>(a, decay_on, tpu, gate, st)
                    : launch_decode_t<float, 64, true, false>(a, decay_on, tpu, gate, st);
    }
    return bf16 ? launch_decode_t<__nv_bfloat16, 32, true, false>(a, decay_on, tpu, gate, st)
                : launch_decode_t<float, 32, true, false>(a, decay_on, tpu, gate, st);
}

}  // namespace lasad
