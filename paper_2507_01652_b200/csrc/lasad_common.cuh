// Shared device/host helpers of the LASAD CUDA library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lasad {

// What every kernel needs to know about one call (host fills it from lasad_params).
struct KernelArgs {
    int B, T, H;
    int grid_w;      // w; 0 = boundary rule off
    int prefix_len;  // P
    long long t0;    // absolute index of the call's first token
    float scale;
    long long qs[3], ks[3], vs[3], os[3];  // element strides for (b, t, h)
    const void* q;
    const void* k;
    const void* v;
    void* o;
    const float* decay;     // [H]
    const float* state_in;  // [B,H,dk,dv] or nullptr
    float* state_out;       // [B,H,dk,dv] or nullptr
    const int* pos;         // decode only: [B] absolute index of each sequence's token, or nullptr (t0 for all)
    const int* widths;      // decode only: [B] grid width of each sequence, or nullptr (grid_w for all)
    int* status;            // device status word (bounded waits report here)
    int* work;              // device ints: [0], [1] zero between launches (work counters of the persistent
                            // prefill kernels), [2] launches of the balanced prefill so far
    float* seg_state;       // prefill, CTA-per-chain kernel: room for 2 x SMs states, or nullptr (chains are not cut)
    unsigned wait_limit;
    // gated entry points only: q and the gate are pre-activations (q <- SiLU(q), lambda <- Sigmoid(gate))
    // and o leaves through a weight-free RMS norm over its dv channels with this epsilon
    int fused;
    float norm_eps;
};

// The operator's neighbours in Algorithm 1, evaluated in fp32 where the fused entry points need
// them.  sigmoid_pair gives lambda = Sigmoid(x) and its complement 1 - lambda = Sigmoid(-x), each
// to full relative precision (1 - lambda is the tied key, and it must not be formed by a
// subtraction when lambda is close to 1).
__device__ __forceinline__ void sigmoid_pair(float x, float& lam, float& one_minus_lam)
{
    const float t = __expf(-fminf(fmaxf(x, -80.0f), 80.0f));     // e^-x, finite
    const float r = __frcp_rn(1.0f + t);
    lam = r;
    one_minus_lam = t * r;
}
__device__ __forceinline__ float silu(float x)
{
    const float t = __expf(-fminf(fmaxf(x, -80.0f), 80.0f));
    return x * __frcp_rn(1.0f + t);
}

// Number of decaying (non-boundary) steps among absolute indices 0..i, from the token's 2-D
// grid position alone (SAD rule, Section 3.4): a step decays unless it absorbs the last token
// of a grid row.  Prefix tokens always decay.  The decay between tokens s < t of one head is
// gamma^(steps(t) - steps(s)); with (row, col) of each this difference equals
// (row_t-row_s)(w-1) + (col_t-col_s) - [col_t = w-1] + [col_s = w-1].
__host__ __device__ inline long long decay_steps_upto(long long i, int grid_w, int prefix_len)
{
    if (i < 0) return 0;
    if (grid_w <= 0 || i < prefix_len) return i + 1;
    const long long j = i - prefix_len;
    const long long row = j / grid_w;
    const int col = (int)(j - row * grid_w);
    return prefix_len + row * (grid_w - 1) + col + (col == grid_w - 1 ? 0 : 1);
}

__host__ __device__ inline bool is_boundary_step(long long i, int grid_w, int prefix_len)
{
    return grid_w > 0 && i >= prefix_len && ((i - prefix_len + 1) % grid_w) == 0;
}

template <typename T> struct io;
template <> struct io<float> {
    __device__ static float load(const float* p) { return *p; }
    __device__ static void store(float* p, float x) { *p = x; }
};
template <> struct io<__nv_bfloat16> {
    __device__ static float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    __device__ static void store(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};

// Launchers implemented in the kernel files; each returns the cudaError_t of its launch.
cudaError_t launch_decode(const KernelArgs& a, int dk, int dv, bool bf16, bool decay_on, int tpu,
                          cudaStream_t st);
// Data-dependent gate (the paper's own decay): `gate` has q's dtype and k's strides; a.k may be
// null (key tied to the gate, k = 1 - lambda); a.decay is unused.
cudaError_t launch_decode_gated(const KernelArgs& a, const void* gate, int dk, bool bf16, bool decay_on, int tpu,
                                cudaStream_t st);
// `only` (device, [B*H], or null): compute just the chains whose entry is non-zero, and put those
// entries back to zero.  `early`: launch as a programmatic dependent of the kernel before it in the
// stream (the kernel waits for that one's completion before it reads anything).
cudaError_t launch_prefill_gated(const KernelArgs& a, const void* gate, int dk, bool bf16, int* only, bool early,
                                 cudaStream_t st);
// Balanced tensor-core form of the gated prefill (one CTA per SM, two chunk pipelines on one chain;
// bf16, dk = dv = 64).  redo ([B*H], zero on entry): set to 1 for every chain given up; the caller
// launches launch_prefill_gated(..., only = redo, ...) behind it.  scratch as for launch_prefill_pair.
cudaError_t launch_prefill_gated_pair(const KernelArgs& a, const void* gate, int* redo, void* scratch, int sms,
                                      cudaStream_t st);
// Tensor-core form of the gated prefill (bf16, dk = dv = 64).  It writes redo[chain] = 1 for every
// chain it gave up (decay too strong for its scaling) and 0 for the others; the caller launches
// launch_prefill_gated(..., only = redo, ...) behind it.
bool prefill_gated_tc_supported(int dk, int dv, bool bf16);
cudaError_t launch_prefill_gated_tc(const KernelArgs& a, const void* gate, int* redo, cudaStream_t st);
bool prefill_tc_supported(int dk, int dv, bool bf16);
cudaError_t launch_prefill_tc(const KernelArgs& a, int sms, cudaStream_t st);
// Balanced tensor-core prefill: one CTA per SM, two chunk pipelines per CTA on one chain, the flat
// chunk sequence cut into equal runs.  `scratch`: prefill_pair_scratch_bytes(sms) bytes of device
// memory, zero before the first launch (the kernel leaves it zero).
size_t prefill_pair_scratch_bytes(int sms);
cudaError_t launch_prefill_pair(const KernelArgs& a, void* scratch, int sms, cudaStream_t st);
// segments per chain that launch_prefill_tc cuts the chains into when a.seg_state is given (1: not cut)
int prefill_tc_segments(int n_chunks, long long chains, int sms);

// What the task-streaming tensor-core prefill needs beyond the caller's buffers: the per-chain
// relay slots through which the carried state passes from one chunk's CTA to the next chunk's.
struct TcRelay {
    void* relay;                // [B*H] slots of kTcRelaySlotBytes
    unsigned epoch16;           // this launch's number folded into 1..65535: part of the packets' tag
    int max_ctas;               // largest fully resident grid (prefill_stream_max_ctas)
};
constexpr long long kTcRelaySlotBytes = 64 * 64 * 8;   // dk * dv values, each with a 4-byte tag
int prefill_stream_chunks(int T);
int prefill_stream_max_ctas(int device);
cudaError_t launch_prefill_stream(const KernelArgs& a, const TcRelay& r, cudaStream_t st);
// scratch (scratch_floats floats of device memory, or null): room for the states at the cuts when few
// chains are cut into segments that run side by side (two launches then, else one).
cudaError_t launch_prefill_simt(const KernelArgs& a, int dk, int dv, bool bf16, int chunk, float* scratch,
                                size_t scratch_floats, int sms, cudaStream_t st);
int prefill_simt_launches(int T, int dk, int chunk, long long chains, int sms, size_t scratch_floats);

}  // namespace lasad
