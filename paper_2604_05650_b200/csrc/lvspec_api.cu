// Host side of liblvspec.so: context, argument validation, scratch memory and
// the launch sequence of each call.  Every step of the verify path itself runs
// in the kernels; nothing here computes on the CPU.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "lvspec_internal.h"

using namespace lvspec;

struct lvspec_ctx {
    int device = 0;
    int n_sm = 0;
    cudaStream_t stream = nullptr;
    uint32_t *status = nullptr;       // device status word
    uint32_t *counters = nullptr;     // [LVSPEC_MAX_BATCH] tickets of the acceptance kernel
    uint32_t *rel_counters = nullptr; // [LVSPEC_MAX_BATCH * LVSPEC_MAX_GAMMA] candidate counts of the relevance score
    void *scratch = nullptr;          // split partials / argmax partials
    size_t scratch_bytes = 0;
    void *staging = nullptr;          // device copies for the *_host calls
    size_t staging_bytes = 0;
    uint64_t launches = 0;
    bool pdl = true;                  // programmatic dependent launch between the attention kernels
    std::string error;
};

namespace {

thread_local std::string g_create_error = "no error";

lvspec_status_t fail(lvspec_ctx *ctx, lvspec_status_t st, const std::string &msg)
{
    if (ctx) ctx->error = msg;
    return st;
}

lvspec_status_t cuda_fail(lvspec_ctx *ctx, const char *what, cudaError_t err)
{
    return fail(ctx, LVSPEC_ERR_CUDA,
                std::string(what) + ": " + cudaGetErrorName(err) + " (" +
                    cudaGetErrorString(err) + ")");
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Is the context's stream being captured into a CUDA graph right now?  (On the legacy
// default stream the query itself fails while another stream captures: that too counts.)
bool stream_is_capturing(lvspec_ctx *ctx)
{
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    const cudaError_t e = cudaStreamIsCapturing(ctx->stream, &cs);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return true;
    }
    return cs != cudaStreamCaptureStatusNone;
}

// Grows *buf to at least `want` bytes.  Growing synchronises the stream, frees and
// allocates: none of that may happen while the stream is being captured, so there the
// call is refused (the capture stays valid) and the caller is told to reserve first.
lvspec_status_t ensure(lvspec_ctx *ctx, void **buf, size_t *have, size_t want, bool zero)
{
    if (want <= *have) return LVSPEC_OK;
    if (stream_is_capturing(ctx))
        return fail(ctx, LVSPEC_ERR_WORKSPACE,
                    "the call needs " + std::to_string(want) + " bytes of scratch memory, the context holds " +
                        std::to_string(*have) + ", and memory cannot be grown while the stream is being "
                        "captured: call lvspec_reserve (or run the call once) before the capture");
    if (*buf) {
        cudaError_t e = cudaStreamSynchronize(ctx->stream);
        if (e != cudaSuccess) return cuda_fail(ctx, "cudaStreamSynchronize", e);
        cudaFree(*buf);
        *buf = nullptr;
        *have = 0;
    }
    size_t bytes = (want + (size_t(1) << 20) - 1) & ~((size_t(1) << 20) - 1);
    cudaError_t e = cudaMalloc(buf, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(ctx, LVSPEC_ERR_WORKSPACE,
                    "scratch allocation of " + std::to_string(bytes) + " bytes failed");
    }
    if (zero) {
        e = cudaMemsetAsync(*buf, 0, bytes, ctx->stream);
        if (e != cudaSuccess) return cuda_fail(ctx, "cudaMemsetAsync", e);
    }
    *have = bytes;
    return LVSPEC_OK;
}

// The tensor-core kernel covers head_dim 64 and 128 with at least one full tile of
// cache; everything else runs on the CUDA-core kernel.
bool tc_shape(const lvspec_attn_shape_t *s)
{
    return (s->head_dim == 128 || s->head_dim == 64) && s->kv_capacity >= 128;
}

int resolve_kernel(const lvspec_attn_shape_t *s)
{
    if (s->kernel == LVSPEC_KERNEL_SIMT || s->kernel == LVSPEC_KERNEL_TCGEN05) return s->kernel;
    return tc_shape(s) ? LVSPEC_KERNEL_TCGEN05 : LVSPEC_KERNEL_SIMT;
}

// KV splits per (sequence, KV head) when the caller leaves the choice to the library.
// The tensor-core kernel runs one CTA per SM.  One CTA works through a tile in a time
// that grows with the query rows it carries (measured: about 2.1 k cycles at 48 padded
// rows, 2.7 k at 80), so with 40 rows about three quarters of the SMs already stream at
// the HBM bandwidth, with 80 rows nearly all are needed, and with an fp8 cache (half the
// bytes per tile for the same work) the device never gets there.  Splits are whole
// 128-position tiles, so a split count that does not divide the tile count leaves a last
// round in which only the CTAs with one tile more are at work, far below the device's
// bandwidth: with 40 rows, 16 splits of 16 tiles beat 18 splits of 14 or 15 on eight
// heads of 256 tiles.  The count is therefore chosen by a small model of the stream, in
// units of the time the whole device takes for one tile: the even rounds at the bandwidth
// their CTA count reaches, the uneven last round at the bandwidth of its few CTAs, and a
// charge per CTA for writing its partial and merging it.  A pure function of the shape:
// results stay reproducible from run to run.
int choose_splits(const lvspec_ctx *ctx, const lvspec_attn_shape_t *s, int max_kv_len, bool fp8 = false)
{
    const int tiles = (max_kv_len + 127) / 128;           // splits never go below 128 positions
    const int units = s->batch * s->n_kv_heads;
    if (resolve_kernel(s) != LVSPEC_KERNEL_TCGEN05) {
        int want = (2 * ctx->n_sm + units - 1) / units;    // about two CTAs per SM
        if (want < 1) want = 1;
        if (want > tiles) want = tiles;
        if (want > 256) want = 256;
        return want;
    }
    int most = ctx->n_sm / units;                          // one CTA per SM, one wave
    if (most < 1) most = 1;
    if (most > tiles) most = tiles;
    if (most > 256) most = 256;
    // CTAs that reach the HBM bandwidth
    const int n_pad = (s->gamma * (s->n_q_heads / s->n_kv_heads) + 15) & ~15;
    double share = 0.73 * (1100.0 + 20.0 * n_pad) / (1100.0 + 20.0 * 48);
    if (share < 0.6) share = 0.6;
    if (fp8) share *= 2.3;
    const double saturating = share * ctx->n_sm;
    auto rate = [&](double ctas) { return ctas >= saturating ? 1.0 : ctas / saturating; };
    int best = most;
    double best_cost = 0.0;
    for (int ns = most; ns >= 1; --ns) {
        const double ctas = (double)ns * units;
        const int t_lo = tiles / ns, rem = tiles - t_lo * ns;
        double cost = t_lo * ctas / rate(ctas) + 0.7 * ctas;
        if (rem > 0) cost += (double)rem * units / rate((double)rem * units);
        if (ns == most || cost < best_cost) {
            best = ns;
            best_cost = cost;
        }
    }
    return best;
}

// Vocabulary slices of the acceptance kernel: enough CTAs for two per SM, at least 4096
// elements each.
int accept_vocab_slices(const lvspec_ctx *ctx, int rows, int vocab)
{
    int vs = (2 * ctx->n_sm + rows - 1) / rows;
    const int max_vs = (vocab + 4095) / 4096;
    if (vs > max_vs) vs = max_vs;
    if (vs < 1) vs = 1;
    return vs;
}

// Scratch bytes of one attention call: the split partials (fp32 rows and their
// statistics) and, for the call with several spans, the log2 denominators.
size_t attention_scratch_bytes(int B, int Hkv, int n_split, int M, int D, int gamma, int Hq, bool with_lse)
{
    const size_t units = (size_t)B * Hkv * n_split;
    return units * M * D * sizeof(float) + units * M * 4 * sizeof(float) +
           (with_lse ? (size_t)B * gamma * Hq * sizeof(float) : 0);
}

// Validation shared by the device and host forms.  On success fills seq.
lvspec_status_t check_attention(lvspec_ctx *ctx, const lvspec_attn_shape_t *s, const void *q,
                                const void *k, const void *v, const int32_t *kv_len,
                                const int32_t *span, const void *out, const float *mass,
                                bool device_ptrs, SeqInfo *seq, int *max_len)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    if (!s || !q || !k || !v || !kv_len || !span || !out || !mass)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "null argument");
    if (s->batch < 1 || s->batch > LVSPEC_MAX_BATCH)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "batch outside 1..LVSPEC_MAX_BATCH");
    if (s->gamma < 1 || s->gamma > LVSPEC_MAX_GAMMA)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "gamma outside 1..LVSPEC_MAX_GAMMA");
    if (s->n_kv_heads < 1 || s->n_q_heads < 1 || s->n_q_heads % s->n_kv_heads != 0)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "n_q_heads must be a positive multiple of n_kv_heads");
    if (s->n_kv_heads > 65535)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "n_kv_heads beyond 65535");
    if (s->kv_capacity < 1) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "kv_capacity < 1");
    if (s->n_split < 0 || s->n_split > 1024)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "n_split outside 0..1024");
    if (s->kernel < 0 || s->kernel > LVSPEC_KERNEL_TCGEN05)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "unknown kernel selector");
    if (s->head_dim != 64 && s->head_dim != 128)
        return fail(ctx, LVSPEC_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
    const int G = s->n_q_heads / s->n_kv_heads;
    if ((long long)s->gamma * G > LVSPEC_MAX_ROWS)
        return fail(ctx, LVSPEC_ERR_UNSUPPORTED,
                    "gamma * (n_q_heads / n_kv_heads) beyond LVSPEC_MAX_ROWS");
    if (device_ptrs && (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) ||
                        (reinterpret_cast<uintptr_t>(mass) & 3u)))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "device tensors must be 16-byte aligned");
    int mx = 0;
    for (int b = 0; b < s->batch; ++b) {
        const int L = kv_len[b], vs = span[2 * b], ve = span[2 * b + 1];
        if (L < s->gamma || L > s->kv_capacity)
            return fail(ctx, LVSPEC_ERR_INVALID_ARG,
                        "kv_len[" + std::to_string(b) + "] outside gamma..kv_capacity");
        if (vs < 0 || vs > ve || ve > L - s->gamma)
            return fail(ctx, LVSPEC_ERR_INVALID_ARG,
                        "visual_span[" + std::to_string(b) + "] outside 0..kv_len-gamma");
        seq->kv_len[b] = L;
        seq->span_start[b] = vs;
        seq->span_end[b] = ve;
        if (L > mx) mx = L;
    }
    *max_len = mx;
    return LVSPEC_OK;
}

struct PagedCache {          // page pools instead of one contiguous cache per sequence
    const int32_t *block_table = nullptr;
    int page_size = 0, pages_per_seq = 0, n_pages = 0;
};

struct Fp8Cache {            // E4M3 codes with one scale per (sequence, KV head)
    const float *k_scale = nullptr, *v_scale = nullptr;
};

lvspec_status_t run_attention(lvspec_ctx *ctx, const lvspec_attn_shape_t *s, const SeqInfo &seq,
                              int max_len, const void *q, const void *k, const void *v, void *out,
                              float *mass, int branch_len = 0, const PagedCache *paged = nullptr,
                              float **lse2 = nullptr, const Fp8Cache *fp8 = nullptr,
                              const lvspec_kv_strides_t *k_strides = nullptr,
                              const lvspec_kv_strides_t *v_strides = nullptr)
{
    AttnParams p;
    std::memset(&p, 0, sizeof p);
    p.q = static_cast<const uint16_t *>(q);
    p.k = static_cast<const uint16_t *>(k);
    p.v = static_cast<const uint16_t *>(v);
    p.out = static_cast<uint16_t *>(out);
    p.mass = mass;
    p.status = ctx->status;
    p.B = s->batch;
    p.gamma = s->gamma;
    p.Hq = s->n_q_heads;
    p.Hkv = s->n_kv_heads;
    p.D = s->head_dim;
    p.Lmax = s->kv_capacity;
    p.G = p.Hq / p.Hkv;
    p.M = p.gamma * p.G;
    p.n_split = s->n_split > 0 ? s->n_split : choose_splits(ctx, s, max_len, fp8 != nullptr);
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)p.D));
    p.pdl = ctx->pdl ? 1 : 0;
    p.branch_len = branch_len > 0 ? branch_len : p.gamma;
    if (fp8) {
        p.fp8 = 1;
        p.k_scale = fp8->k_scale;
        p.v_scale = fp8->v_scale;
    }
    // cache strides: dense [B, Hkv, Lmax, D] unless the caller gave its own
    p.k_sp = p.v_sp = p.D;
    p.k_sh = p.v_sh = (int64_t)p.Lmax * p.D;
    p.k_sb = p.v_sb = (int64_t)p.Hkv * p.Lmax * p.D;
    if (paged) {
        p.block_table = paged->block_table;
        p.page_size = paged->page_size;
        p.pages_per_seq = paged->pages_per_seq;
        p.n_pages = paged->n_pages;
        p.k_sh = p.v_sh = (int64_t)p.page_size * p.D;          // pools [n_pages, Hkv, page_size, D]
        p.k_sb = p.v_sb = (int64_t)p.Hkv * p.page_size * p.D;
    }
    if (k_strides) { p.k_sb = k_strides->batch; p.k_sh = k_strides->head; p.k_sp = k_strides->position; }
    if (v_strides) { p.v_sb = v_strides->batch; p.v_sh = v_strides->head; p.v_sp = v_strides->position; }

    const size_t o_bytes = part_o_elems(p) * sizeof(float);
    const size_t st_bytes = part_stat_elems(p) * sizeof(float);
    lvspec_status_t st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes,
                                attention_scratch_bytes(p.B, p.Hkv, p.n_split, p.M, p.D, p.gamma, p.Hq,
                                                        lse2 != nullptr), false);
    if (st != LVSPEC_OK) return st;
    p.part_o = static_cast<float *>(ctx->scratch);
    p.part_stat = reinterpret_cast<float *>(static_cast<char *>(ctx->scratch) + o_bytes);
    if (lse2) {
        p.lse2 = reinterpret_cast<float *>(static_cast<char *>(ctx->scratch) + o_bytes + st_bytes);
        *lse2 = p.lse2;
    }

    int launches = 0;
    cudaError_t e;
    const int kernel = resolve_kernel(s);
    if (kernel == LVSPEC_KERNEL_TCGEN05) {
        if (!attn_tc_supported(p))
            return fail(ctx, LVSPEC_ERR_UNSUPPORTED,
                        p.fp8 ? "the fp8 cache needs head_dim 128, kv_capacity >= 128 and at most 80 query rows "
                                "per KV head"
                              : "the tcgen05 kernel needs head_dim 64 or 128 and kv_capacity >= 128");
        e = launch_attn_tc(p, seq, ctx->stream, &launches);
    } else {
        e = launch_attn_simt(p, seq, ctx->stream, &launches);
    }
    ctx->launches += launches;
    if (e != cudaSuccess) return cuda_fail(ctx, "attention kernel launch", e);
    // with a single split the tensor-core kernel writes the results itself
    if (kernel == LVSPEC_KERNEL_TCGEN05 && p.n_split == 1) return LVSPEC_OK;
    launches = 0;
    e = launch_attn_combine(p, ctx->stream, &launches);
    ctx->launches += launches;
    if (e != cudaSuccess) return cuda_fail(ctx, "combine kernel launch", e);
    return LVSPEC_OK;
}

lvspec_status_t check_accept(lvspec_ctx *ctx, int batch, int gamma, int vocab, int heads,
                             const void *logits, const void *draft, const void *mass,
                             const lvspec_thresholds_t *th, int window, const void *accept_len,
                             bool device_ptrs, int *n_loose)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    if (!logits || !draft || !mass || !th || !accept_len)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "null argument");
    if (batch < 1 || batch > LVSPEC_MAX_BATCH)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "batch outside 1..LVSPEC_MAX_BATCH");
    if (gamma < 1 || gamma > LVSPEC_MAX_GAMMA)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "gamma outside 1..LVSPEC_MAX_GAMMA");
    if (vocab < 1) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "vocab < 1");
    if (heads < 1) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "n_mass_heads < 1");
    if (window < 0) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "shift_window < 0");
    if (device_ptrs && ((reinterpret_cast<uintptr_t>(logits) & 3u) ||
                        (reinterpret_cast<uintptr_t>(draft) & 3u) ||
                        (reinterpret_cast<uintptr_t>(mass) & 3u) ||
                        (reinterpret_cast<uintptr_t>(accept_len) & 3u)))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "misaligned device pointer");
    int n = th->n_loose;
    if (n < 0) {
        if (!(th->lambda >= 0.0 && th->lambda <= 1.0))
            return fail(ctx, LVSPEC_ERR_INVALID_ARG, "lambda outside [0, 1]");
        n = (int)std::floor(th->lambda * (double)gamma + 1e-9);
    }
    if (n > gamma) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "n_loose > gamma");
    *n_loose = n;
    return LVSPEC_OK;
}

lvspec_status_t run_accept(lvspec_ctx *ctx, int batch, int gamma, int vocab, int heads,
                           const float *logits, const int32_t *draft, const float *mass,
                           int n_loose, int window, int32_t *accept_len, int32_t *target,
                           uint8_t *accepted, const int32_t *kv_len = nullptr, int32_t *emitted = nullptr,
                           int32_t *n_emitted = nullptr, int32_t *new_kv_len = nullptr)
{
    AcceptParams p;
    std::memset(&p, 0, sizeof p);
    p.logits = logits;
    p.draft = draft;
    p.mass = mass;
    p.accept_len = accept_len;
    p.target = target;
    p.accepted = accepted;
    p.kv_len = kv_len;
    p.emitted = emitted;
    p.n_emitted = n_emitted;
    p.new_kv_len = new_kv_len;
    p.counters = ctx->counters;
    p.status = ctx->status;
    p.B = batch;
    p.gamma = gamma;
    p.V = vocab;
    p.Hm = heads;
    p.n_loose = n_loose;
    p.window = window > gamma ? gamma : window;
    const int rows = batch * gamma;
    const int vs = accept_vocab_slices(ctx, rows, vocab);
    p.n_vsplit = vs;
    const size_t n_part = (size_t)rows * vs;
    lvspec_status_t st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes,
                                n_part * (sizeof(float) + sizeof(int32_t)), false);
    if (st != LVSPEC_OK) return st;
    p.part_val = static_cast<float *>(ctx->scratch);
    p.part_idx = reinterpret_cast<int32_t *>(p.part_val + n_part);
    int launches = 0;
    cudaError_t e = launch_loose_accept(p, ctx->stream, &launches);
    ctx->launches += launches;
    if (e != cudaSuccess) return cuda_fail(ctx, "acceptance kernel launch", e);
    return LVSPEC_OK;
}

}  // namespace

extern "C" {

#ifdef LVSPEC_TRACE
// Trace build only (see lvspec_internal.h): where the kernels' time stamps go.
int lvspec_trace_set_buffer(unsigned long long *device_words)
{
    cudaError_t e = trace_set_buffer_attention(device_words);
    if (e == cudaSuccess) e = trace_set_buffer_merge(device_words);
    return (int)e;
}
#endif

lvspec_status_t lvspec_create(lvspec_ctx_t **out, int device)
{
    if (!out) {
        g_create_error = "null context pointer";
        return LVSPEC_ERR_INVALID_ARG;
    }
    *out = nullptr;
    int n_dev = 0;
    cudaError_t e = cudaGetDeviceCount(&n_dev);
    if (e != cudaSuccess || n_dev == 0) {
        cudaGetLastError();
        g_create_error = std::string("no CUDA device: ") + cudaGetErrorString(e);
        return LVSPEC_ERR_CUDA;
    }
    if (device < 0 || device >= n_dev) {
        g_create_error = "device ordinal out of range";
        return LVSPEC_ERR_INVALID_ARG;
    }
    lvspec_ctx *ctx = new (std::nothrow) lvspec_ctx();
    if (!ctx) {
        g_create_error = "out of host memory";
        return LVSPEC_ERR_WORKSPACE;
    }
    ctx->device = device;
    ctx->error = "no error";
    cudaDeviceProp prop;
    if ((e = cudaSetDevice(device)) != cudaSuccess ||
        (e = cudaGetDeviceProperties(&prop, device)) != cudaSuccess) {
        g_create_error = std::string("cudaSetDevice: ") + cudaGetErrorString(e);
        delete ctx;
        return LVSPEC_ERR_CUDA;
    }
    if (prop.major != 10) {
        g_create_error = "this library holds sm_100a code only; device is sm_" +
                         std::to_string(prop.major) + std::to_string(prop.minor);
        delete ctx;
        return LVSPEC_ERR_UNSUPPORTED;
    }
    ctx->n_sm = prop.multiProcessorCount;
    if (const char *e = std::getenv("LVSPEC_NO_PDL")) ctx->pdl = !(e[0] && e[0] != '0');
    const size_t small = sizeof(uint32_t) * (1 + LVSPEC_MAX_BATCH + LVSPEC_MAX_BATCH * LVSPEC_MAX_GAMMA);
    if ((e = cudaMalloc(reinterpret_cast<void **>(&ctx->status), small)) != cudaSuccess ||
        (e = cudaMemset(ctx->status, 0, small)) != cudaSuccess) {
        g_create_error = std::string("status allocation: ") + cudaGetErrorString(e);
        cudaFree(ctx->status);      // null when the allocation itself failed
        cudaGetLastError();
        delete ctx;
        return LVSPEC_ERR_WORKSPACE;
    }
    ctx->counters = ctx->status + 1;
    ctx->rel_counters = ctx->counters + LVSPEC_MAX_BATCH;
    lvspec_status_t st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, size_t(8) << 20, true);
    if (st != LVSPEC_OK) {
        g_create_error = ctx->error;
        cudaFree(ctx->status);
        delete ctx;
        return st;
    }
    cudaDeviceSynchronize();
    *out = ctx;
    return LVSPEC_OK;
}

lvspec_status_t lvspec_destroy(lvspec_ctx_t *ctx)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    cudaFree(ctx->scratch);
    cudaFree(ctx->staging);
    cudaFree(ctx->status);
    delete ctx;
    return LVSPEC_OK;
}

lvspec_status_t lvspec_set_stream(lvspec_ctx_t *ctx, void *cuda_stream)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    return LVSPEC_OK;
}

lvspec_status_t lvspec_device_status(lvspec_ctx_t *ctx, uint32_t *flags)
{
    if (!ctx || !flags) return LVSPEC_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    uint32_t h = 0;
    cudaError_t e = cudaMemcpyAsync(&h, ctx->status, sizeof h, cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->status, 0, sizeof h, ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    if (e != cudaSuccess) return cuda_fail(ctx, "reading the device status", e);
    *flags = h;
    if (h & LVSPEC_DEV_WAIT_EXPIRED)
        return fail(ctx, LVSPEC_ERR_TIMEOUT, "a bounded device-side wait ran out");
    return LVSPEC_OK;
}

const char *lvspec_last_error(const lvspec_ctx_t *ctx)
{
    return ctx ? ctx->error.c_str() : g_create_error.c_str();
}

const char *lvspec_status_string(lvspec_status_t status)
{
    switch (status) {
        case LVSPEC_OK: return "ok";
        case LVSPEC_ERR_INVALID_ARG: return "invalid argument";
        case LVSPEC_ERR_UNSUPPORTED: return "unsupported shape";
        case LVSPEC_ERR_WORKSPACE: return "scratch memory allocation failed";
        case LVSPEC_ERR_CUDA: return "CUDA error";
        case LVSPEC_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

uint64_t lvspec_launch_count(const lvspec_ctx_t *ctx) { return ctx ? ctx->launches : 0; }

int32_t lvspec_attention_splits(const lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                int32_t max_kv_len)
{
    if (!ctx || !shape || shape->batch < 1 || shape->n_kv_heads < 1 || max_kv_len < 1) return 0;
    return shape->n_split > 0 ? shape->n_split : choose_splits(ctx, shape, max_kv_len);
}

int32_t lvspec_attention_splits_fp8(const lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                    int32_t max_kv_len)
{
    if (!ctx || !shape || shape->batch < 1 || shape->n_kv_heads < 1 || max_kv_len < 1) return 0;
    return shape->n_split > 0 ? shape->n_split : choose_splits(ctx, shape, max_kv_len, true);
}

lvspec_status_t lvspec_last_device_status(lvspec_ctx_t *ctx, uint32_t *flags)
{
    return lvspec_device_status(ctx, flags);
}

size_t lvspec_attention_workspace_bytes(const lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                        int32_t max_kv_len)
{
    if (!ctx || !shape || shape->batch < 1 || shape->n_kv_heads < 1 || shape->gamma < 1 ||
        shape->n_q_heads < shape->n_kv_heads || shape->head_dim < 1 || max_kv_len < 1 || shape->n_split < 0)
        return 0;
    // the library's own choice differs between the bf16 and the fp8 cache: the larger of the two
    int n_split = shape->n_split;
    if (n_split == 0) {
        n_split = choose_splits(ctx, shape, max_kv_len);
        const int n8 = choose_splits(ctx, shape, max_kv_len, true);
        if (n8 > n_split) n_split = n8;
    }
    // the call with several spans never runs the tensor-core kernel on a single split
    const int n_eff = n_split < 2 ? 2 : n_split;
    const int M = shape->gamma * (shape->n_q_heads / shape->n_kv_heads);
    return attention_scratch_bytes(shape->batch, shape->n_kv_heads, n_eff, M, shape->head_dim, shape->gamma,
                                   shape->n_q_heads, true);
}

size_t lvspec_accept_workspace_bytes(const lvspec_ctx_t *ctx, int32_t batch, int32_t gamma, int32_t vocab)
{
    if (!ctx || batch < 1 || gamma < 1 || vocab < 1) return 0;
    const int rows = batch * gamma;
    return (size_t)rows * accept_vocab_slices(ctx, rows, vocab) * (sizeof(float) + sizeof(int32_t));
}

size_t lvspec_relevance_workspace_bytes(const lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                        int32_t n_visual, int32_t dim)
{
    if (!ctx || batch < 1 || gamma < 1 || n_visual < 1 || dim < 1) return 0;
    return relevance_scratch_bytes(batch, gamma, n_visual, dim);
}

size_t lvspec_workspace_capacity(const lvspec_ctx_t *ctx) { return ctx ? ctx->scratch_bytes : 0; }

lvspec_status_t lvspec_reserve(lvspec_ctx_t *ctx, size_t workspace_bytes)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    return ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, workspace_bytes, false);
}

lvspec_status_t lvspec_verify_attention(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                        const void *q, const void *k_cache, const void *v_cache,
                                        const int32_t *kv_len, const int32_t *visual_span,
                                        void *out, float *visual_mass)
{
    SeqInfo seq;
    int max_len = 0;
    lvspec_status_t st = check_attention(ctx, shape, q, k_cache, v_cache, kv_len, visual_span, out,
                                         visual_mass, true, &seq, &max_len);
    if (st != LVSPEC_OK) return st;
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    return run_attention(ctx, shape, seq, max_len, q, k_cache, v_cache, out, visual_mass);
}

lvspec_status_t lvspec_verify_attention_strided(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                                const lvspec_kv_strides_t *k_strides,
                                                const lvspec_kv_strides_t *v_strides, const void *q,
                                                const void *k_cache, const void *v_cache,
                                                const int32_t *kv_len, const int32_t *visual_span,
                                                void *out, float *visual_mass)
{
    SeqInfo seq;
    int max_len = 0;
    lvspec_status_t st = check_attention(ctx, shape, q, k_cache, v_cache, kv_len, visual_span, out,
                                         visual_mass, true, &seq, &max_len);
    if (st != LVSPEC_OK) return st;
    if (!k_strides || !v_strides) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "null argument");
    for (const lvspec_kv_strides_t *t : {k_strides, v_strides}) {
        // a position's channels must not overlap the next position's; 16-byte granularity
        if (t->position < shape->head_dim || t->head < 1 || t->batch < 1 || (t->position & 7) || (t->head & 7) ||
            (t->batch & 7) || t->position >= (int64_t(1) << 38) || t->head >= (int64_t(1) << 38) ||
            t->batch >= (int64_t(1) << 38))
            return fail(ctx, LVSPEC_ERR_INVALID_ARG,
                        "cache strides must be positive multiples of 8 elements, the position stride at least head_dim");
    }
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    return run_attention(ctx, shape, seq, max_len, q, k_cache, v_cache, out, visual_mass, 0, nullptr, nullptr,
                         nullptr, k_strides, v_strides);
}

lvspec_status_t lvspec_verify_attention_tree(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                             int32_t n_branches, const void *q, const void *k_cache,
                                             const void *v_cache, const int32_t *kv_len,
                                             const int32_t *visual_span, void *out, float *visual_mass)
{
    SeqInfo seq;
    int max_len = 0;
    lvspec_status_t st = check_attention(ctx, shape, q, k_cache, v_cache, kv_len, visual_span, out,
                                         visual_mass, true, &seq, &max_len);
    if (st != LVSPEC_OK) return st;
    if (n_branches < 1 || shape->gamma % n_branches != 0)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "gamma must be a positive multiple of n_branches");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    return run_attention(ctx, shape, seq, max_len, q, k_cache, v_cache, out, visual_mass,
                         shape->gamma / n_branches);
}

lvspec_status_t lvspec_verify_attention_spans(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                              const void *q, const void *k_cache, const void *v_cache,
                                              const int32_t *kv_len, int32_t n_spans,
                                              const int32_t *visual_spans, void *out, float *visual_mass)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    if (!shape || !visual_spans || !kv_len) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "null argument");
    if (n_spans < 1 || n_spans > kMaxGaps + 1)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "n_spans outside 1.." + std::to_string(kMaxGaps + 1));
    if (shape->batch < 1 || shape->batch > LVSPEC_MAX_BATCH)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "batch outside 1..LVSPEC_MAX_BATCH");
    // per sequence: the hull of the non-empty spans, and the ranges between them
    std::vector<int32_t> hull(2 * (size_t)shape->batch);
    std::vector<std::vector<int32_t>> gaps(shape->batch);
    for (int b = 0; b < shape->batch; ++b) {
        int first = -1, last_end = 0;
        for (int i = 0; i < n_spans; ++i) {
            const int s = visual_spans[((size_t)b * n_spans + i) * 2], e = visual_spans[((size_t)b * n_spans + i) * 2 + 1];
            if (s < 0 || e < s || e > kv_len[b] - shape->gamma)
                return fail(ctx, LVSPEC_ERR_INVALID_ARG, "a visual span lies outside 0..kv_len-gamma");
            if (s == e) continue;                      // padding
            if (first < 0) first = s;
            else {
                if (s < last_end)
                    return fail(ctx, LVSPEC_ERR_INVALID_ARG, "visual spans must be sorted and disjoint");
                if (s > last_end) { gaps[b].push_back(last_end); gaps[b].push_back(s); }
            }
            last_end = e;
        }
        hull[2 * b] = first < 0 ? 0 : first;
        hull[2 * b + 1] = first < 0 ? 0 : last_end;
    }
    SeqInfo seq;
    int max_len = 0;
    lvspec_status_t st = check_attention(ctx, shape, q, k_cache, v_cache, kv_len, hull.data(), out,
                                         visual_mass, true, &seq, &max_len);
    if (st != LVSPEC_OK) return st;
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    // the log2 denominators come from the combine kernel: at least two splits where the
    // tensor-core kernel would otherwise finish alone (the plain kernel always combines)
    lvspec_attn_shape_t s = *shape;
    if (resolve_kernel(&s) == LVSPEC_KERNEL_TCGEN05 && s.n_split == 0 && choose_splits(ctx, &s, max_len) < 2) {
        if (max_len > 128) s.n_split = 2;
        else if (s.kernel == LVSPEC_KERNEL_DEFAULT) s.kernel = LVSPEC_KERNEL_SIMT;
        else
            return fail(ctx, LVSPEC_ERR_UNSUPPORTED,
                        "several spans on a cache of one tile need the plain kernel (two splits cannot be made)");
    }
    if (resolve_kernel(&s) == LVSPEC_KERNEL_TCGEN05 && s.n_split == 1)
        return fail(ctx, LVSPEC_ERR_UNSUPPORTED, "several spans need n_split != 1 with the tcgen05 kernel");
    float *lse2 = nullptr;
    st = run_attention(ctx, &s, seq, max_len, q, k_cache, v_cache, out, visual_mass, 0, nullptr, &lse2);
    if (st != LVSPEC_OK) return st;
    for (int b = 0; b < shape->batch; ++b) {
        if (gaps[b].empty()) continue;
        GapParams g;
        std::memset(&g, 0, sizeof g);
        g.q = static_cast<const uint16_t *>(q);
        g.k = static_cast<const uint16_t *>(k_cache);
        g.lse2 = lse2;
        g.mass = visual_mass;
        g.b = b;
        g.gamma = shape->gamma;
        g.Hq = shape->n_q_heads;
        g.Hkv = shape->n_kv_heads;
        g.D = shape->head_dim;
        g.Lmax = shape->kv_capacity;
        g.G = g.Hq / g.Hkv;
        g.M = g.gamma * g.G;
        g.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)g.D));
        g.n_gaps = (int)gaps[b].size() / 2;
        int flat = 0;
        for (int i = 0; i < g.n_gaps; ++i) {
            g.gap_start[i] = gaps[b][2 * i];
            g.gap_first[i] = flat;
            flat += gaps[b][2 * i + 1] - gaps[b][2 * i];
        }
        g.gap_first[g.n_gaps] = flat;
        int launches = 0;
        e = launch_gap_mass(g, ctx->stream, &launches);
        ctx->launches += launches;
        if (e != cudaSuccess) return cuda_fail(ctx, "gap mass kernel launch", e);
    }
    return LVSPEC_OK;
}

lvspec_status_t lvspec_verify_attention_paged(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                              int32_t page_size, int32_t n_pages, const void *q,
                                              const void *k_pool, const void *v_pool,
                                              const int32_t *block_table, const int32_t *kv_len,
                                              const int32_t *visual_span, void *out, float *visual_mass)
{
    SeqInfo seq;
    int max_len = 0;
    lvspec_status_t st = check_attention(ctx, shape, q, k_pool, v_pool, kv_len, visual_span, out,
                                         visual_mass, true, &seq, &max_len);
    if (st != LVSPEC_OK) return st;
    if (!block_table || (reinterpret_cast<uintptr_t>(block_table) & 3u))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "block_table is null or misaligned");
    if (page_size < 128 || page_size % 128 != 0)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "page_size must be a positive multiple of 128");
    if (n_pages < 1 || (long long)n_pages * shape->n_kv_heads > 2147483647ll)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "n_pages outside 1..2^31 / n_kv_heads");
    if (shape->kv_capacity % page_size != 0)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "kv_capacity must be a whole number of pages");
    if (shape->head_dim != 128 || shape->kernel == LVSPEC_KERNEL_SIMT)
        return fail(ctx, LVSPEC_ERR_UNSUPPORTED, "the paged cache needs the tcgen05 kernel (head_dim 128)");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    PagedCache pc;
    pc.block_table = block_table;
    pc.page_size = page_size;
    pc.pages_per_seq = shape->kv_capacity / page_size;
    pc.n_pages = n_pages;
    lvspec_attn_shape_t s = *shape;
    s.kernel = LVSPEC_KERNEL_TCGEN05;
    return run_attention(ctx, &s, seq, max_len, q, k_pool, v_pool, out, visual_mass, 0, &pc);
}

lvspec_status_t lvspec_verify_attention_fp8(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                            const void *q, const void *k_cache, const void *v_cache,
                                            const float *k_scale, const float *v_scale,
                                            const int32_t *kv_len, const int32_t *visual_span,
                                            void *out, float *visual_mass)
{
    SeqInfo seq;
    int max_len = 0;
    lvspec_status_t st = check_attention(ctx, shape, q, k_cache, v_cache, kv_len, visual_span, out,
                                         visual_mass, true, &seq, &max_len);
    if (st != LVSPEC_OK) return st;
    if (!k_scale || !v_scale || (reinterpret_cast<uintptr_t>(k_scale) & 3u) ||
        (reinterpret_cast<uintptr_t>(v_scale) & 3u))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "k_scale or v_scale is null or misaligned");
    if (shape->head_dim != 128 || shape->kernel == LVSPEC_KERNEL_SIMT || shape->kv_capacity < 128)
        return fail(ctx, LVSPEC_ERR_UNSUPPORTED,
                    "the fp8 cache needs the tcgen05 kernel (head_dim 128, kv_capacity >= 128)");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    Fp8Cache f8;
    f8.k_scale = k_scale;
    f8.v_scale = v_scale;
    lvspec_attn_shape_t s = *shape;
    s.kernel = LVSPEC_KERNEL_TCGEN05;
    return run_attention(ctx, &s, seq, max_len, q, k_cache, v_cache, out, visual_mass, 0, nullptr, nullptr, &f8);
}

lvspec_status_t lvspec_verify_attention_host(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                             const void *q, const void *k_cache,
                                             const void *v_cache, const int32_t *kv_len,
                                             const int32_t *visual_span, void *out,
                                             float *visual_mass)
{
    SeqInfo seq;
    int max_len = 0;
    lvspec_status_t st = check_attention(ctx, shape, q, k_cache, v_cache, kv_len, visual_span, out,
                                         visual_mass, false, &seq, &max_len);
    if (st != LVSPEC_OK) return st;
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
    const size_t q_bytes = (size_t)shape->batch * shape->gamma * shape->n_q_heads * shape->head_dim * 2;
    const size_t kv_bytes = (size_t)shape->batch * shape->n_kv_heads * shape->kv_capacity * shape->head_dim * 2;
    const size_t m_bytes = (size_t)shape->batch * shape->gamma * shape->n_q_heads * sizeof(float);
    const size_t total = 2 * up(q_bytes) + 2 * up(kv_bytes) + up(m_bytes);
    st = ensure(ctx, &ctx->staging, &ctx->staging_bytes, total, false);
    if (st != LVSPEC_OK) return st;
    char *base = static_cast<char *>(ctx->staging);
    char *dq = base, *dk = dq + up(q_bytes), *dv = dk + up(kv_bytes), *dout = dv + up(kv_bytes),
         *dm = dout + up(q_bytes);
    if ((e = cudaMemcpyAsync(dq, q, q_bytes, cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dk, k_cache, kv_bytes, cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dv, v_cache, kv_bytes, cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess)
        return cuda_fail(ctx, "host to device copy", e);
    st = run_attention(ctx, shape, seq, max_len, dq, dk, dv, dout, reinterpret_cast<float *>(dm));
    if (st != LVSPEC_OK) return st;
    if ((e = cudaMemcpyAsync(out, dout, q_bytes, cudaMemcpyDeviceToHost, ctx->stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(visual_mass, dm, m_bytes, cudaMemcpyDeviceToHost, ctx->stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(ctx->stream)) != cudaSuccess)
        return cuda_fail(ctx, "device to host copy", e);
    return LVSPEC_OK;
}

lvspec_status_t lvspec_select_branch(lvspec_ctx_t *ctx, int32_t batch, int32_t n_branches,
                                     const int32_t *accept_len, int32_t *best_branch, int32_t *best_len)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    if (!accept_len || !best_branch || !best_len) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "null argument");
    if (batch < 1 || n_branches < 1 || (long long)batch * n_branches > LVSPEC_MAX_BATCH)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "batch * n_branches outside 1..LVSPEC_MAX_BATCH");
    if ((reinterpret_cast<uintptr_t>(accept_len) & 3u) || (reinterpret_cast<uintptr_t>(best_branch) & 3u) ||
        (reinterpret_cast<uintptr_t>(best_len) & 3u))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "misaligned device pointer");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    int launches = 0;
    e = launch_select_branch(accept_len, batch, n_branches, best_branch, best_len, ctx->stream, &launches);
    ctx->launches += launches;
    if (e != cudaSuccess) return cuda_fail(ctx, "branch selection kernel launch", e);
    return LVSPEC_OK;
}

lvspec_status_t lvspec_selftest_wait_expiry(lvspec_ctx_t *ctx, int32_t limit_ms)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    if (limit_ms < 1 || limit_ms > 2000) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "limit_ms outside 1..2000");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    int launches = 0;
    e = launch_wait_expiry(ctx->status, (unsigned long long)limit_ms * 1000000ull, ctx->stream, &launches);
    ctx->launches += launches;
    if (e != cudaSuccess) return cuda_fail(ctx, "self-test kernel launch", e);
    return LVSPEC_OK;
}

lvspec_status_t lvspec_row_inv_norms(lvspec_ctx_t *ctx, int64_t rows, int32_t dim, const void *x,
                                     float *inv_norm)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    if (!x || !inv_norm) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "null argument");
    if (rows < 1 || rows > (int64_t(1) << 31) * 8 - 8)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "rows out of range");
    if (dim < 8 || dim % 8 != 0) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "dim must be a positive multiple of 8");
    if (!aligned16(x) || (reinterpret_cast<uintptr_t>(inv_norm) & 3u))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "misaligned device pointer");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    int launches = 0;
    e = launch_row_inv_norms(static_cast<const uint16_t *>(x), rows, dim, inv_norm, ctx->stream, &launches);
    ctx->launches += launches;
    if (e != cudaSuccess) return cuda_fail(ctx, "norm kernel launch", e);
    return LVSPEC_OK;
}

lvspec_status_t lvspec_visual_relevance(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                        int32_t n_visual, int32_t dim, const void *h_draft,
                                        const void *h_visual, const float *visual_inv_norm,
                                        int32_t top_n, float *relevance)
{
    if (!ctx) return LVSPEC_ERR_INVALID_ARG;
    if (!h_draft || !h_visual || !visual_inv_norm || !relevance)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "null argument");
    if (batch < 1 || batch > LVSPEC_MAX_BATCH)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "batch outside 1..LVSPEC_MAX_BATCH");
    if (gamma < 1 || gamma > LVSPEC_MAX_GAMMA)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "gamma outside 1..LVSPEC_MAX_GAMMA");
    if (n_visual < 1 || (long long)batch * ((n_visual + 15) / 16) > 0x7fffffffLL)
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "n_visual out of range");
    if (top_n < 1) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "top_n < 1");
    if (dim < 64) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "dim < 64");
    if (dim % 64 != 0) return fail(ctx, LVSPEC_ERR_UNSUPPORTED, "dim must be a multiple of 64");
    if (!aligned16(h_draft) || !aligned16(h_visual) ||
        (reinterpret_cast<uintptr_t>(visual_inv_norm) & 3u) || (reinterpret_cast<uintptr_t>(relevance) & 3u))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "misaligned device pointer");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    lvspec_status_t st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes,
                                relevance_scratch_bytes(batch, gamma, n_visual, dim), false);
    if (st != LVSPEC_OK) return st;
    RelevanceParams p;
    std::memset(&p, 0, sizeof p);
    p.h_draft = static_cast<const uint16_t *>(h_draft);
    p.h_visual = static_cast<const uint16_t *>(h_visual);
    p.v_inv_norm = visual_inv_norm;
    p.cos_t = static_cast<float *>(ctx->scratch);
    p.relevance = relevance;
    p.counters = ctx->rel_counters;
    p.status = ctx->status;
    p.B = batch;
    p.K = gamma;
    p.lv = n_visual;
    p.d = dim;
    p.top_n = top_n;
    p.lv_pad = (n_visual + 3) & ~3;
    p.n_sm = ctx->n_sm;
    int launches = 0;
    e = launch_visual_relevance(p, ctx->stream, &launches);
    ctx->launches += launches;
    if (e != cudaSuccess) return cuda_fail(ctx, "relevance kernel launch", e);
    return LVSPEC_OK;
}

lvspec_status_t lvspec_loose_accept_ex(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                       int32_t vocab, int32_t n_mass_heads,
                                       const float *target_logits, const int32_t *draft_tokens,
                                       const float *visual_mass,
                                       const lvspec_thresholds_t *thresholds,
                                       int32_t shift_window, int32_t *accept_len,
                                       int32_t *target_tokens, uint8_t *accepted)
{
    int n_loose = 0;
    lvspec_status_t st = check_accept(ctx, batch, gamma, vocab, n_mass_heads, target_logits,
                                      draft_tokens, visual_mass, thresholds, shift_window,
                                      accept_len, true, &n_loose);
    if (st != LVSPEC_OK) return st;
    if (target_tokens && (reinterpret_cast<uintptr_t>(target_tokens) & 3u))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "misaligned device pointer");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    return run_accept(ctx, batch, gamma, vocab, n_mass_heads, target_logits, draft_tokens,
                      visual_mass, n_loose, shift_window, accept_len, target_tokens, accepted);
}

lvspec_status_t lvspec_loose_accept_emit(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                         int32_t vocab, int32_t n_mass_heads,
                                         const float *target_logits, const int32_t *draft_tokens,
                                         const float *visual_mass,
                                         const lvspec_thresholds_t *thresholds,
                                         int32_t shift_window, const int32_t *kv_len,
                                         int32_t *accept_len, int32_t *emitted, int32_t *n_emitted,
                                         int32_t *new_kv_len)
{
    int n_loose = 0;
    lvspec_status_t st = check_accept(ctx, batch, gamma, vocab, n_mass_heads, target_logits,
                                      draft_tokens, visual_mass, thresholds, shift_window,
                                      accept_len, true, &n_loose);
    if (st != LVSPEC_OK) return st;
    if (!emitted || !n_emitted) return fail(ctx, LVSPEC_ERR_INVALID_ARG, "null argument");
    if ((kv_len == nullptr) != (new_kv_len == nullptr))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "kv_len and new_kv_len go together");
    if ((reinterpret_cast<uintptr_t>(emitted) & 3u) || (reinterpret_cast<uintptr_t>(n_emitted) & 3u) ||
        (reinterpret_cast<uintptr_t>(kv_len) & 3u) || (reinterpret_cast<uintptr_t>(new_kv_len) & 3u))
        return fail(ctx, LVSPEC_ERR_INVALID_ARG, "misaligned device pointer");
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    return run_accept(ctx, batch, gamma, vocab, n_mass_heads, target_logits, draft_tokens,
                      visual_mass, n_loose, shift_window, accept_len, nullptr, nullptr, kv_len, emitted,
                      n_emitted, new_kv_len);
}

lvspec_status_t lvspec_loose_accept(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                    int32_t vocab, int32_t n_mass_heads,
                                    const float *target_logits, const int32_t *draft_tokens,
                                    const float *visual_mass,
                                    const lvspec_thresholds_t *thresholds, int32_t shift_window,
                                    int32_t *accept_len)
{
    return lvspec_loose_accept_ex(ctx, batch, gamma, vocab, n_mass_heads, target_logits,
                                  draft_tokens, visual_mass, thresholds, shift_window, accept_len,
                                  nullptr, nullptr);
}

lvspec_status_t lvspec_loose_accept_host(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                         int32_t vocab, int32_t n_mass_heads,
                                         const float *target_logits, const int32_t *draft_tokens,
                                         const float *visual_mass,
                                         const lvspec_thresholds_t *thresholds,
                                         int32_t shift_window, int32_t *accept_len)
{
    int n_loose = 0;
    lvspec_status_t st = check_accept(ctx, batch, gamma, vocab, n_mass_heads, target_logits,
                                      draft_tokens, visual_mass, thresholds, shift_window,
                                      accept_len, false, &n_loose);
    if (st != LVSPEC_OK) return st;
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaSetDevice", e);
    auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
    const size_t lg_bytes = (size_t)batch * gamma * vocab * sizeof(float);
    const size_t dr_bytes = (size_t)batch * gamma * sizeof(int32_t);
    const size_t ms_bytes = (size_t)batch * gamma * n_mass_heads * sizeof(float);
    const size_t al_bytes = (size_t)batch * sizeof(int32_t);
    st = ensure(ctx, &ctx->staging, &ctx->staging_bytes,
                up(lg_bytes) + up(dr_bytes) + up(ms_bytes) + up(al_bytes), false);
    if (st != LVSPEC_OK) return st;
    char *dl = static_cast<char *>(ctx->staging), *dd = dl + up(lg_bytes), *dm = dd + up(dr_bytes),
         *da = dm + up(ms_bytes);
    if ((e = cudaMemcpyAsync(dl, target_logits, lg_bytes, cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dd, draft_tokens, dr_bytes, cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(dm, visual_mass, ms_bytes, cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess)
        return cuda_fail(ctx, "host to device copy", e);
    st = run_accept(ctx, batch, gamma, vocab, n_mass_heads, reinterpret_cast<float *>(dl),
                    reinterpret_cast<int32_t *>(dd), reinterpret_cast<float *>(dm), n_loose,
                    shift_window, reinterpret_cast<int32_t *>(da), nullptr, nullptr);
    if (st != LVSPEC_OK) return st;
    if ((e = cudaMemcpyAsync(accept_len, da, al_bytes, cudaMemcpyDeviceToHost, ctx->stream)) != cudaSuccess ||
        (e = cudaStreamSynchronize(ctx->stream)) != cudaSuccess)
        return cuda_fail(ctx, "device to host copy", e);
    return LVSPEC_OK;
}

}  // extern "C"
