// Host side of the LASAD C ABI: argument validation, kernel selection, launches.
#include "../../include/lasad.h"
#include "lasad_common.cuh"

#include <cmath>
#include <new>

struct lasad_ctx {
    int device;
    int* d_status;        // device status word
    int last_cuda_error;
    uint64_t launches;
    int opt_prefill_impl; // LASAD_OPT_PREFILL_IMPL: 0 auto, 1..5 as listed in lasad.h
    int opt_prefill_chunk;
    int opt_decode_tpu;
    unsigned wait_limit;
    int sm_count;
    // state relay of the task-streaming prefill (see lasad_prefill_tc_stream.cu)
    void* d_relay;                // [relay_cap] slots of kTcRelaySlotBytes
    int64_t relay_cap;
    uint64_t epoch;               // launches of the task-streaming prefill so far
    int stream_max_ctas;
    // states at the cuts when the CTA-per-chain prefill splits few, long chains into segments
    float* d_segstate;            // [2 x SMs][dk * dv], then [2 x SMs] counters
    // per-chain flags of the gated tensor-core prefill: chains it left to the CUDA-core kernel
    int* d_redo;                  // [redo_cap]
    int64_t redo_cap;
    // state slots and flags at the cuts of the balanced tensor-core prefill (one per SM)
    void* d_pair;
    // host-buffer pipeline of lasad_forward_host: two staging slots (q | k | v | o of one batch
    // element each), a decay and a state buffer, copy streams and the events that order them
    void* d_stage[2];
    size_t stage_bytes;
    float* d_host_decay;
    int64_t host_decay_cap;
    float* d_host_state;
    size_t host_state_bytes;
    cudaStream_t s_in, s_out;
    cudaEvent_t ev_start, ev_in[2], ev_comp[2], ev_out[2];
    bool pipeline_ready;
};

namespace {

constexpr unsigned kDefaultWaitLimit = 1u << 22;

constexpr int64_t kDefaultRelayUnits = 1024;   // chains covered by the relay storage lasad_create allocates

// Grows the context-owned relay storage to `units` chains.  Allocates (and therefore
// synchronises the device) only when the current storage is too small.
int reserve_units(lasad_ctx* ctx, int64_t units)
{
    if (units <= ctx->relay_cap) return LASAD_OK;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();   // an earlier launch may still use the old slots
    void* nr = nullptr;
    if (e == cudaSuccess) e = cudaMalloc(&nr, (size_t)units * lasad::kTcRelaySlotBytes);
    // stale bytes must never look like a tag of a later launch: start from zero (tags are never 0)
    if (e == cudaSuccess) e = cudaMemset(nr, 0, (size_t)units * lasad::kTcRelaySlotBytes);
    if (e == cudaSuccess) {
        if (ctx->d_relay) cudaFree(ctx->d_relay);
        ctx->d_relay = nr;
        ctx->relay_cap = units;
    } else if (nr) {
        cudaFree(nr);
    }
    cudaSetDevice(prev);
    if (e != cudaSuccess) {
        ctx->last_cuda_error = (int)e;
        return LASAD_ERR_CUDA;
    }
    return LASAD_OK;
}

constexpr int64_t kDefaultRedoUnits = 65536;   // chains covered by the flag array lasad_create allocates

// Grows the per-chain flag array of the gated prefill to `units` chains (same rules as above).
int reserve_redo(lasad_ctx* ctx, int64_t units)
{
    if (units <= ctx->redo_cap) return LASAD_OK;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();   // an earlier launch may still use the old array
    int* nr = nullptr;
    if (e == cudaSuccess) e = cudaMalloc(&nr, (size_t)units * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(nr, 0, (size_t)units * sizeof(int));   // the kernels keep it zero between launches
    if (e == cudaSuccess) {
        if (ctx->d_redo) cudaFree(ctx->d_redo);
        ctx->d_redo = nr;
        ctx->redo_cap = units;
    }
    cudaSetDevice(prev);
    if (e != cudaSuccess) {
        ctx->last_cuda_error = (int)e;
        return LASAD_ERR_CUDA;
    }
    return LASAD_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// What LASAD_OPT_PREFILL_IMPL = 0 stands for on a problem of `batch` sequences.
int auto_prefill_impl(const lasad_ctx* ctx, const lasad_params* p, int64_t batch, bool tc_ok)
{
    if (!tc_ok) return 1;
    // Few chains: one CTA per chain would leave most SMs idle.  Long chains (16 chunks and up to
    // SMs / 3 chains, or 32 chunks and up to SMs / 2) are cut into segments that run side by side;
    // shorter ones (up to SMs / 3) have their chunks streamed over all SMs.  The limits are where
    // the measurements cross.
    const int chunks = lasad::prefill_stream_chunks(p->T);
    const int64_t chains = batch * p->H;
    if ((chains * 3 <= ctx->sm_count && chunks >= 16) || (chains * 2 <= ctx->sm_count && chunks >= 32)) return 4;
    if (chains * 3 <= ctx->sm_count && chunks >= 2 && ctx->stream_max_ctas > 0) return 3;
    // Long chains: the balanced kernel (one chain at a time per SM, left-over chains cut into equal
    // pieces), unless the chains fill the two-per-SM slots of the CTA-per-chain kernel almost exactly.
    if (chunks >= 32) {
        const int64_t slots = 2LL * ctx->sm_count;
        const int64_t waves = (chains + slots - 1) / slots;
        if (chains * 100 < waves * slots * 93) return 5;
    }
    return 2;
}

int fail_cuda(lasad_ctx* ctx, cudaError_t e)
{
    ctx->last_cuda_error = (int)e;
    return LASAD_ERR_CUDA;
}

// Shape / dtype / stride checks shared by both entry points.
int check_common(const lasad_ctx* ctx, const lasad_params* p, bool decode)
{
    if (!ctx || !p) return LASAD_ERR_INVALID_ARG;
    if (p->B <= 0 || p->H <= 0 || p->dk <= 0 || p->dv <= 0) return LASAD_ERR_INVALID_ARG;
    if (!decode && p->T <= 0) return LASAD_ERR_INVALID_ARG;
    if (p->grid_w < 0 || p->prefix_len < 0 || p->t0 < 0 || p->reserved != 0) return LASAD_ERR_INVALID_ARG;
    if (!std::isfinite(p->scale)) return LASAD_ERR_INVALID_ARG;
    if (p->dtype != LASAD_F32 && p->dtype != LASAD_BF16) return LASAD_ERR_INVALID_ARG;
    const int64_t esz = p->dtype == LASAD_F32 ? 4 : 2;
    const int64_t* strides[4] = {p->q_stride, p->k_stride, p->v_stride, p->o_stride};
    for (int s = 0; s < 4; ++s) {
        for (int d = 0; d < 3; ++d) {
            if (decode && d == 1) continue;
            const int64_t st = strides[s][d];
            if (st < 0 || (st * esz) % 16 != 0) return LASAD_ERR_INVALID_ARG;
        }
        // a zero stride would alias the elements of a dimension: allowed only where it has one element
        if ((strides[s][0] == 0 && p->B > 1) || (!decode && strides[s][1] == 0 && p->T > 1)) return LASAD_ERR_INVALID_ARG;
        const int width = (s < 2) ? p->dk : p->dv;
        if (strides[s][2] < width && p->H > 1) return LASAD_ERR_INVALID_ARG;
    }
    if (p->dk != p->dv || (p->dk != 32 && p->dk != 64)) return LASAD_ERR_UNSUPPORTED;
    if ((int64_t)p->B * p->H > 0x7fffffffLL) return LASAD_ERR_UNSUPPORTED;
    // the context's buffers, SM count and kernel attributes belong to its device
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != ctx->device) return LASAD_ERR_INVALID_ARG;
    return LASAD_OK;
}

void fill_args(lasad::KernelArgs& a, const lasad_ctx* ctx, const lasad_params* p)
{
    a.B = p->B; a.T = p->T; a.H = p->H;
    a.grid_w = p->grid_w; a.prefix_len = p->prefix_len; a.t0 = p->t0; a.scale = p->scale;
    for (int d = 0; d < 3; ++d) {
        a.qs[d] = p->q_stride[d]; a.ks[d] = p->k_stride[d];
        a.vs[d] = p->v_stride[d]; a.os[d] = p->o_stride[d];
    }
    a.status = ctx->d_status;
    a.work = ctx->d_status + 16;     // same 256-byte block, zeroed at creation
    a.wait_limit = ctx->wait_limit;
}

}  // namespace

extern "C" {

int lasad_create(lasad_ctx** out, int device)
{
    if (!out) return LASAD_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return LASAD_ERR_CUDA;
    lasad_ctx* ctx = new (std::nothrow) lasad_ctx();
    if (!ctx) return LASAD_ERR_CUDA;
    ctx->device = device;
    ctx->wait_limit = kDefaultWaitLimit;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, 256);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, 256);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) ctx->stream_max_ctas = lasad::prefill_stream_max_ctas(device);
    if (e == cudaSuccess) {
        // 2 x SMs states, then as many counters (zero between launches)
        const size_t bytes = (size_t)2 * ctx->sm_count * (64 * 64 * sizeof(float) + sizeof(int));
        e = cudaMalloc(&ctx->d_segstate, bytes);
        if (e == cudaSuccess) e = cudaMemset(ctx->d_segstate, 0, bytes);
    }
    if (e == cudaSuccess) {
        const size_t bytes = lasad::prefill_pair_scratch_bytes(ctx->sm_count);
        e = cudaMalloc(&ctx->d_pair, bytes);
        if (e == cudaSuccess) e = cudaMemset(ctx->d_pair, 0, bytes);
    }
    cudaSetDevice(prev);
    if (e == cudaSuccess && reserve_units(ctx, kDefaultRelayUnits) != LASAD_OK) e = cudaErrorMemoryAllocation;
    if (e == cudaSuccess && reserve_redo(ctx, kDefaultRedoUnits) != LASAD_OK) e = cudaErrorMemoryAllocation;
    if (e != cudaSuccess) {
        if (ctx->d_status) cudaFree(ctx->d_status);
        if (ctx->d_relay) cudaFree(ctx->d_relay);
        if (ctx->d_redo) cudaFree(ctx->d_redo);
        if (ctx->d_segstate) cudaFree(ctx->d_segstate);
        if (ctx->d_pair) cudaFree(ctx->d_pair);
        delete ctx;
        return LASAD_ERR_CUDA;
    }
    *out = ctx;
    return LASAD_OK;
}

int lasad_destroy(lasad_ctx* ctx)
{
    if (!ctx) return LASAD_ERR_INVALID_ARG;
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->d_relay) cudaFree(ctx->d_relay);
    if (ctx->d_redo) cudaFree(ctx->d_redo);
    if (ctx->d_segstate) cudaFree(ctx->d_segstate);
    if (ctx->d_pair) cudaFree(ctx->d_pair);
    for (int i = 0; i < 2; ++i)
        if (ctx->d_stage[i]) cudaFree(ctx->d_stage[i]);
    if (ctx->d_host_decay) cudaFree(ctx->d_host_decay);
    if (ctx->d_host_state) cudaFree(ctx->d_host_state);
    if (ctx->pipeline_ready) {
        cudaStreamDestroy(ctx->s_in);
        cudaStreamDestroy(ctx->s_out);
        cudaEventDestroy(ctx->ev_start);
        for (int i = 0; i < 2; ++i) {
            cudaEventDestroy(ctx->ev_in[i]);
            cudaEventDestroy(ctx->ev_comp[i]);
            cudaEventDestroy(ctx->ev_out[i]);
        }
    }
    delete ctx;
    return LASAD_OK;
}

int lasad_reserve(lasad_ctx* ctx, int64_t units)
{
    if (!ctx || units <= 0) return LASAD_ERR_INVALID_ARG;
    const int rc = reserve_units(ctx, units);
    return rc != LASAD_OK ? rc : reserve_redo(ctx, units);
}

int lasad_set_option(lasad_ctx* ctx, int option, int value)
{
    if (!ctx) return LASAD_ERR_INVALID_ARG;
    switch (option) {
        case LASAD_OPT_PREFILL_IMPL:
            if (value < 0 || value > 5) return LASAD_ERR_INVALID_ARG;
            ctx->opt_prefill_impl = value;
            return LASAD_OK;
        case LASAD_OPT_PREFILL_CHUNK:
            if (value != 0 && value != 16 && value != 32 && value != 64) return LASAD_ERR_INVALID_ARG;
            ctx->opt_prefill_chunk = value;
            return LASAD_OK;
        case LASAD_OPT_DECODE_TPU:
            if (value != 0 && value != 32 && value != 64 && value != 128 && value != 256)
                return LASAD_ERR_INVALID_ARG;
            ctx->opt_decode_tpu = value;
            return LASAD_OK;
        case LASAD_OPT_WAIT_LIMIT:
            if (value < 0) return LASAD_ERR_INVALID_ARG;
            ctx->wait_limit = value == 0 ? kDefaultWaitLimit : (unsigned)value;
            return LASAD_OK;
        default:
            return LASAD_ERR_INVALID_ARG;
    }
}

int lasad_forward(lasad_ctx* ctx, const lasad_params* p, const void* q, const void* k, const void* v,
                  const float* decay, const float* state_in, void* o, float* state_out,
                  void* cuda_stream)
{
    int rc = check_common(ctx, p, false);
    if (rc != LASAD_OK) return rc;
    if (!q || !k || !v || !o || !decay) return LASAD_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return LASAD_ERR_INVALID_ARG;
    if ((state_in && !aligned16(state_in)) || (state_out && !aligned16(state_out)))
        return LASAD_ERR_INVALID_ARG;

    lasad::KernelArgs a{};
    fill_args(a, ctx, p);
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.decay = decay; a.state_in = state_in; a.state_out = state_out;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const bool bf16 = p->dtype == LASAD_BF16;

    int impl = ctx->opt_prefill_impl;
    const bool tc_ok = lasad::prefill_tc_supported(p->dk, p->dv, bf16);
    const bool chosen = impl == 0;
    if (chosen) impl = auto_prefill_impl(ctx, p, p->B, tc_ok);
    if (impl == 3) {
        // The relay packets of this kernel carry the launch's number, which the host counts: a
        // launch recorded into a CUDA graph would replay with the number it was recorded with and
        // could take an earlier replay's packets for its own.  During a stream capture the default
        // therefore falls back to the CTA-per-chain kernel, and an explicit request is refused.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap != cudaStreamCaptureStatusNone) {
            if (!chosen) return LASAD_ERR_UNSUPPORTED;
            impl = 2;
        }
    }
    if (impl == 3) {
        if (!tc_ok) return LASAD_ERR_UNSUPPORTED;
        const int64_t units = (int64_t)p->B * p->H;
        const int64_t chunks = lasad::prefill_stream_chunks(p->T);
        if (units * chunks > 0x7fffffffLL || ctx->stream_max_ctas <= 0) return LASAD_ERR_UNSUPPORTED;
        // the carried state travels from chunk to chunk through context-owned relay slots
        if (chunks > 1) {
            rc = reserve_units(ctx, units);
            if (rc != LASAD_OK) return rc;
        }
        lasad::TcRelay r{};
        r.relay = ctx->d_relay;
        // The packets' tag holds the launch number modulo 65535; before a value comes round
        // again the slots are cleared, so that no packet of an old launch can pass for a new one.
        ctx->epoch += 1;
        r.epoch16 = (unsigned)(ctx->epoch % 65535u) + 1u;
        if (ctx->epoch % 65535u == 0 && ctx->d_relay) {
            const cudaError_t em =
                cudaMemsetAsync(ctx->d_relay, 0, (size_t)ctx->relay_cap * lasad::kTcRelaySlotBytes, st);
            if (em != cudaSuccess) return fail_cuda(ctx, em);
        }
        r.max_ctas = ctx->stream_max_ctas;
        const cudaError_t e = lasad::launch_prefill_stream(a, r, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ctx->launches += 1;
        return LASAD_OK;
    }
    if (impl == 5) {
        if (!tc_ok || (int64_t)p->B * p->H * lasad::prefill_stream_chunks(p->T) > 0x7fffffffLL) return LASAD_ERR_UNSUPPORTED;
        const cudaError_t e = lasad::launch_prefill_pair(a, ctx->d_pair, ctx->sm_count, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ctx->launches += 1;
        return LASAD_OK;
    }
    if (impl == 2 || impl == 4) {
        if (!tc_ok) return LASAD_ERR_UNSUPPORTED;
        int launches = 1;
        if (impl == 4) {
            a.seg_state = ctx->d_segstate;
            if (lasad::prefill_tc_segments(lasad::prefill_stream_chunks(p->T), (long long)p->B * p->H, ctx->sm_count) > 1)
                launches = 2;
        }
        const cudaError_t e = lasad::launch_prefill_tc(a, ctx->sm_count, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ctx->launches += launches;
        return LASAD_OK;
    }
    int chunk = ctx->opt_prefill_chunk;
    const long long chains = (long long)p->B * p->H;
    // few chains are cut into segments of whole chunks that run side by side: shorter chunks then
    // give more segments (the default chunk is the one that is fastest when every SM has a chain)
    if (chunk == 0) {
        if (chains * 2 <= ctx->sm_count) {
            // the longest chunk that still yields a segment for every CTA slot, else the shortest
            const long long want = 2LL * ctx->sm_count / chains;
            chunk = p->T / 64 >= want ? 64 : p->T / 32 >= want ? 32 : 16;
        } else {
            chunk = p->dk == 64 ? 32 : 64;
        }
    }
    if (p->T <= 16) chunk = 16;
    const size_t scratch_floats = (size_t)2 * ctx->sm_count * 64 * 64;      // the state slots of d_segstate
    const cudaError_t e = lasad::launch_prefill_simt(a, p->dk, p->dv, bf16, chunk, ctx->d_segstate, scratch_floats,
                                                     ctx->sm_count, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->launches += lasad::prefill_simt_launches(p->T, p->dk, chunk, chains, ctx->sm_count, scratch_floats);
    return LASAD_OK;
}

int lasad_decode_step(lasad_ctx* ctx, const lasad_params* p, const void* q, const void* k,
                      const void* v, const float* decay, float* state, void* o, void* cuda_stream)
{
    int rc = check_common(ctx, p, true);
    if (rc != LASAD_OK) return rc;
    if (!q || !k || !v || !o || !decay || !state) return LASAD_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(state))
        return LASAD_ERR_INVALID_ARG;

    lasad::KernelArgs a{};
    fill_args(a, ctx, p);
    a.T = 1;
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.decay = decay; a.state_in = state; a.state_out = state;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // SAD rule (Algorithm 1's if-statement): the decay is 1 on a row-boundary step
    const bool decay_on = !lasad::is_boundary_step(p->t0, p->grid_w, p->prefix_len);
    int tpu = ctx->opt_decode_tpu;
    if (tpu == 0) {
        // few states: spread each over a whole CTA so that all of its loads are in flight at
        // once; many states: fewer threads per state, more states per CTA
        const long long units = (long long)p->B * p->H;
        tpu = units >= 16LL * ctx->sm_count ? 128 : 256;
    }
    const cudaError_t e = lasad::launch_decode(a, p->dk, p->dv, p->dtype == LASAD_BF16, decay_on, tpu, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->launches += 1;
    return LASAD_OK;
}

int lasad_decode_step_pos(lasad_ctx* ctx, const lasad_params* p, const void* q, const void* k, const void* v,
                          const float* decay, float* state, void* o, const int32_t* pos, const int32_t* grid_w,
                          void* cuda_stream)
{
    int rc = check_common(ctx, p, true);
    if (rc != LASAD_OK) return rc;
    if (!q || !k || !v || !o || !decay || !state || !pos) return LASAD_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(state))
        return LASAD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(pos) & 3u) || (reinterpret_cast<uintptr_t>(grid_w) & 3u)) return LASAD_ERR_INVALID_ARG;
    lasad::KernelArgs a{};
    fill_args(a, ctx, p);
    a.T = 1;
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.decay = decay; a.state_in = state; a.state_out = state;
    a.pos = pos; a.widths = grid_w;
    int tpu = ctx->opt_decode_tpu;
    if (tpu == 0) tpu = (long long)p->B * p->H >= 16LL * ctx->sm_count ? 128 : 256;
    const cudaError_t e = lasad::launch_decode(a, p->dk, p->dv, p->dtype == LASAD_BF16, true, tpu,
                                               static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->launches += 1;
    return LASAD_OK;
}

}  // extern "C"

namespace {

// lasad_forward_gated (fused = false) and lasad_forward_fused (fused = true)
int forward_gated(lasad_ctx* ctx, const lasad_params* p, const void* q, const void* k, const void* v,
                  const void* gate, const float* state_in, void* o, float* state_out, bool fused, float norm_eps,
                  void* cuda_stream)
{
    int rc = check_common(ctx, p, false);
    if (rc != LASAD_OK) return rc;
    if (!q || !v || !o || !gate) return LASAD_ERR_INVALID_ARG;
    if (!aligned16(q) || (k && !aligned16(k)) || !aligned16(v) || !aligned16(o) || !aligned16(gate))
        return LASAD_ERR_INVALID_ARG;
    if ((state_in && !aligned16(state_in)) || (state_out && !aligned16(state_out)))
        return LASAD_ERR_INVALID_ARG;
    lasad::KernelArgs a{};
    fill_args(a, ctx, p);
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.decay = nullptr; a.state_in = state_in; a.state_out = state_out;
    a.fused = fused ? 1 : 0; a.norm_eps = norm_eps;
    // tensor cores where the shape allows it, unless the CUDA-core implementation is asked for
    const bool bf16 = p->dtype == LASAD_BF16;
    const bool tc = ctx->opt_prefill_impl != 1 && lasad::prefill_gated_tc_supported(p->dk, p->dv, bf16);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (!tc) {
        const cudaError_t e = lasad::launch_prefill_gated(a, gate, p->dk, bf16, nullptr, false, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        ctx->launches += 1;
        return LASAD_OK;
    }
    // Two launches: the tensor-core kernel marks the chains whose decay is too strong for its
    // scaling, and the CUDA-core kernel behind it computes exactly those (none, as a rule).
    rc = reserve_redo(ctx, (int64_t)p->B * p->H);
    if (rc != LASAD_OK) return rc;
    // which tensor-core kernel: the balanced one (option 5, and the default where the plain prefill
    // would take its counterpart) or the CTA-per-chain one (option 2 and the other defaults)
    bool pair = ctx->opt_prefill_impl == 5;
    if (ctx->opt_prefill_impl == 0) pair = auto_prefill_impl(ctx, p, p->B, true) == 5;
    cudaError_t e = pair ? lasad::launch_prefill_gated_pair(a, gate, ctx->d_redo, ctx->d_pair, ctx->sm_count, st)
                         : lasad::launch_prefill_gated_tc(a, gate, ctx->d_redo, st);
    if (e == cudaSuccess) {
        ctx->launches += 1;
        // (behind the balanced kernel an early launch measured slower, behind the other one faster)
        e = lasad::launch_prefill_gated(a, gate, p->dk, bf16, ctx->d_redo, !pair, st);
    }
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->launches += 1;
    return LASAD_OK;
}

// lasad_decode_step_gated (fused = false) and lasad_decode_step_fused (fused = true)
int decode_step_gated(lasad_ctx* ctx, const lasad_params* p, const void* q, const void* k, const void* v,
                      const void* gate, float* state, void* o, bool fused, float norm_eps, void* cuda_stream)
{
    int rc = check_common(ctx, p, true);
    if (rc != LASAD_OK) return rc;
    if (!q || !v || !o || !gate || !state) return LASAD_ERR_INVALID_ARG;
    if (!aligned16(q) || (k && !aligned16(k)) || !aligned16(v) || !aligned16(o) || !aligned16(gate) ||
        !aligned16(state))
        return LASAD_ERR_INVALID_ARG;
    lasad::KernelArgs a{};
    fill_args(a, ctx, p);
    a.T = 1;
    a.q = q; a.k = k; a.v = v; a.o = o;
    a.decay = nullptr; a.state_in = state; a.state_out = state;
    a.fused = fused ? 1 : 0; a.norm_eps = norm_eps;
    // SAD rule (Algorithm 1's if-statement): the decay is 1 on a row-boundary step
    const bool decay_on = !lasad::is_boundary_step(p->t0, p->grid_w, p->prefix_len);
    int tpu = ctx->opt_decode_tpu;
    if (tpu == 0) tpu = (long long)p->B * p->H >= 16LL * ctx->sm_count ? 128 : 256;
    const cudaError_t e = lasad::launch_decode_gated(a, gate, p->dk, p->dtype == LASAD_BF16, decay_on, tpu,
                                                     static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->launches += 1;
    return LASAD_OK;
}

}  // namespace

extern "C" {

int lasad_forward_gated(lasad_ctx* ctx, const lasad_params* p, const void* q, const void* k, const void* v,
                        const void* gate, const float* state_in, void* o, float* state_out, void* cuda_stream)
{
    return forward_gated(ctx, p, q, k, v, gate, state_in, o, state_out, false, 0.0f, cuda_stream);
}

int lasad_forward_fused(lasad_ctx* ctx, const lasad_params* p, const void* q_pre, const void* k, const void* v,
                        const void* gate_pre, const float* state_in, void* o, float* state_out, float norm_eps,
                        void* cuda_stream)
{
    if (!(norm_eps >= 0.0f) || !std::isfinite(norm_eps)) return LASAD_ERR_INVALID_ARG;
    return forward_gated(ctx, p, q_pre, k, v, gate_pre, state_in, o, state_out, true, norm_eps, cuda_stream);
}

int lasad_decode_step_gated(lasad_ctx* ctx, const lasad_params* p, const void* q, const void* k, const void* v,
                            const void* gate, float* state, void* o, void* cuda_stream)
{
    return decode_step_gated(ctx, p, q, k, v, gate, state, o, false, 0.0f, cuda_stream);
}

int lasad_decode_step_fused(lasad_ctx* ctx, const lasad_params* p, const void* q_pre, const void* k, const void* v,
                            const void* gate_pre, float* state, void* o, float norm_eps, void* cuda_stream)
{
    if (!(norm_eps >= 0.0f) || !std::isfinite(norm_eps)) return LASAD_ERR_INVALID_ARG;
    return decode_step_gated(ctx, p, q_pre, k, v, gate_pre, state, o, true, norm_eps, cuda_stream);
}

int lasad_forward_host(lasad_ctx* ctx, const lasad_params* p, const void* q, const void* k, const void* v,
                       const float* decay, const float* state_in, void* o, float* state_out, void* cuda_stream)
{
    int rc = check_common(ctx, p, false);
    if (rc != LASAD_OK) return rc;
    if (!q || !k || !v || !o || !decay) return LASAD_ERR_INVALID_ARG;
    const size_t esz = p->dtype == LASAD_F32 ? 4 : 2;
    const size_t per_q = (size_t)p->T * p->H * p->dk * esz, per_v = (size_t)p->T * p->H * p->dv * esz;
    const size_t off_k = (per_q + 255) & ~size_t(255), off_v = 2 * off_k;
    const size_t off_o = off_v + ((per_v + 255) & ~size_t(255));
    const size_t slot = off_o + ((per_v + 255) & ~size_t(255));
    const size_t state_bytes = (size_t)p->B * p->H * p->dk * p->dv * sizeof(float);
    const bool use_state = state_in || state_out;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    int prev = 0;
    cudaGetDevice(&prev);
    cudaError_t e = cudaSetDevice(ctx->device);
    // ---- set-up and growth of the context's staging storage (allocates; synchronises) ----
    if (e == cudaSuccess && !ctx->pipeline_ready) {
        e = cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming);
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_comp[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_out[i], cudaEventDisableTiming);
        }
        ctx->pipeline_ready = e == cudaSuccess;
    }
    if (e == cudaSuccess && slot > ctx->stage_bytes) {
        e = cudaDeviceSynchronize();
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            if (ctx->d_stage[i]) cudaFree(ctx->d_stage[i]);
            ctx->d_stage[i] = nullptr;
            e = cudaMalloc(&ctx->d_stage[i], slot);
        }
        ctx->stage_bytes = e == cudaSuccess ? slot : 0;
    }
    if (e == cudaSuccess && p->H > ctx->host_decay_cap) {
        e = cudaDeviceSynchronize();
        if (ctx->d_host_decay) cudaFree(ctx->d_host_decay);
        ctx->d_host_decay = nullptr;
        if (e == cudaSuccess) e = cudaMalloc(&ctx->d_host_decay, (size_t)p->H * sizeof(float));
        ctx->host_decay_cap = e == cudaSuccess ? p->H : 0;
    }
    if (e == cudaSuccess && use_state && state_bytes > ctx->host_state_bytes) {
        e = cudaDeviceSynchronize();
        if (ctx->d_host_state) cudaFree(ctx->d_host_state);
        ctx->d_host_state = nullptr;
        if (e == cudaSuccess) e = cudaMalloc(&ctx->d_host_state, state_bytes);
        ctx->host_state_bytes = e == cudaSuccess ? state_bytes : 0;
    }
    if (e != cudaSuccess) {
        cudaSetDevice(prev);
        return fail_cuda(ctx, e);
    }

    // ---- the pipeline: batch element b is copied in on s_in while b-1 is computed on the
    //      caller's stream and b-2 is copied out on s_out ----
    lasad_params pb = *p;
    pb.B = 1;
    const int64_t row_q = (int64_t)p->H * p->dk, row_v = (int64_t)p->H * p->dv;
    pb.q_stride[0] = pb.k_stride[0] = (int64_t)p->T * row_q;
    pb.q_stride[1] = pb.k_stride[1] = row_q;
    pb.q_stride[2] = pb.k_stride[2] = p->dk;
    pb.v_stride[0] = pb.o_stride[0] = (int64_t)p->T * row_v;
    pb.v_stride[1] = pb.o_stride[1] = row_v;
    pb.v_stride[2] = pb.o_stride[2] = p->dv;
    const size_t unit_floats = (size_t)p->H * p->dk * p->dv;

    e = cudaEventRecord(ctx->ev_start, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_in, ctx->ev_start, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_out, ctx->ev_start, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_host_decay, decay, (size_t)p->H * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && state_in)
        e = cudaMemcpyAsync(ctx->d_host_state, state_in, state_bytes, cudaMemcpyHostToDevice, st);
    for (int b = 0; b < p->B && e == cudaSuccess && rc == LASAD_OK; ++b) {
        const int sl = b & 1;
        unsigned char* base = static_cast<unsigned char*>(ctx->d_stage[sl]);
        const unsigned char* hq = static_cast<const unsigned char*>(q) + (size_t)b * per_q;
        const unsigned char* hk = static_cast<const unsigned char*>(k) + (size_t)b * per_q;
        const unsigned char* hv = static_cast<const unsigned char*>(v) + (size_t)b * per_v;
        unsigned char* ho = static_cast<unsigned char*>(o) + (size_t)b * per_v;
        if (b >= 2) e = cudaStreamWaitEvent(ctx->s_in, ctx->ev_comp[sl], 0);   // the slot's inputs have been consumed
        if (e == cudaSuccess) e = cudaMemcpyAsync(base, hq, per_q, cudaMemcpyHostToDevice, ctx->s_in);
        if (e == cudaSuccess) e = cudaMemcpyAsync(base + off_k, hk, per_q, cudaMemcpyHostToDevice, ctx->s_in);
        if (e == cudaSuccess) e = cudaMemcpyAsync(base + off_v, hv, per_v, cudaMemcpyHostToDevice, ctx->s_in);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_in[sl], ctx->s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, ctx->ev_in[sl], 0);
        if (e == cudaSuccess && b >= 2) e = cudaStreamWaitEvent(st, ctx->ev_out[sl], 0);   // the slot's output has left
        if (e != cudaSuccess) break;
        float* sb = use_state ? ctx->d_host_state + (size_t)b * unit_floats : nullptr;
        // one batch element per launch, but with the kernel the whole batch would get, so that the
        // results equal lasad_forward's on the same data bit for bit
        const int asked = ctx->opt_prefill_impl;
        if (asked == 0)
            ctx->opt_prefill_impl =
                auto_prefill_impl(ctx, p, p->B, lasad::prefill_tc_supported(p->dk, p->dv, p->dtype == LASAD_BF16));
        rc = lasad_forward(ctx, &pb, base, base + off_k, base + off_v, ctx->d_host_decay, state_in ? sb : nullptr,
                           base + off_o, state_out ? sb : nullptr, st);
        ctx->opt_prefill_impl = asked;
        if (rc != LASAD_OK) break;
        e = cudaEventRecord(ctx->ev_comp[sl], st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_out, ctx->ev_comp[sl], 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(ho, base + off_o, per_v, cudaMemcpyDeviceToHost, ctx->s_out);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_out[sl], ctx->s_out);
    }
    // the caller's stream ends the call: it waits for the last copies out
    for (int i = 0; i < 2 && e == cudaSuccess && rc == LASAD_OK; ++i)
        if (i < p->B) e = cudaStreamWaitEvent(st, ctx->ev_out[i], 0);
    if (e == cudaSuccess && rc == LASAD_OK && state_out)
        e = cudaMemcpyAsync(state_out, ctx->d_host_state, state_bytes, cudaMemcpyDeviceToHost, st);
    cudaSetDevice(prev);
    if (rc != LASAD_OK) return rc;
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    return LASAD_OK;
}

int lasad_last_device_status(lasad_ctx* ctx, int* status)
{
    if (!ctx || !status) return LASAD_ERR_INVALID_ARG;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->device);
    int hv = 0;
    cudaError_t e = cudaMemcpy(&hv, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && hv != 0) e = cudaMemset(ctx->d_status, 0, sizeof(int));
    cudaSetDevice(prev);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    *status = hv != 0 ? LASAD_ERR_TIMEOUT : LASAD_OK;
    return LASAD_OK;
}

int lasad_last_cuda_error(const lasad_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

uint64_t lasad_launch_count(const lasad_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* lasad_strerror(int code)
{
    switch (code) {
        case LASAD_OK: return "ok";
        case LASAD_ERR_INVALID_ARG: return "invalid argument (null pointer, size, alignment or stride)";
        case LASAD_ERR_UNSUPPORTED: return "unsupported configuration (need dk == dv in {32, 64}, f32 or bf16)";
        case LASAD_ERR_CUDA: return "CUDA call failed";
        case LASAD_ERR_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown error code";
    }
}

}  // extern "C"
