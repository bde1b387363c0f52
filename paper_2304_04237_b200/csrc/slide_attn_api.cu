// C-ABI layer of the slide-attention library: argument validation, the context, variant
// selection and the host-buffer entry point.  All arithmetic lives in the kernel files.
#include <new>

#include "common.cuh"

using namespace slide_attn;

struct slide_attn_ctx {
    int B, H, W, heads, head_dim, ksize, has_bias;
    slide_attn_dtype dtype;
    slide_attn_variant variant;      // never AUTO
    bool fixed_shift;                // the caller declared one-hot weights: run the fixed-shift kernel
    int device;
    int num_sms;
    int* d_status;                   // device status word (0 = ok)
    void* workspace;                 // re-laid-out weights for the variants that need them
    size_t workspace_bytes;
    void* strip_ws;                  // transposed weights of the STRIP variant
    void* umma_ws;                   // bf16 B images of the UMMA_TS variant
    void* wide_ws;                   // bf16 B fragments of the MMA_WIDE variant
    void* bwd_ws;                    // attention weights and logit gradients between the two backward kernels (first backward)
    void* block_ws;                  // q, k, v, z of slide_attn_block_forward (first use)
    bool proj_ready;                 // the projection kernel's attributes are set on this device
    // staging buffers for slide_attn_forward_host, allocated on first use
    void* stage;
    size_t stage_bytes;
    // slide_attn_forward_host pipelines batch slices over two copy streams (created on first use)
    cudaStream_t copy_in, copy_out;
    cudaEvent_t host_ev[2 + 2 * 4];  // start, done, then (slice copied in, slice computed) per slice
    bool host_pipe;
    // profiling: ring of event triples (start, before main kernel, end)
    bool profiling;
    int prof_count;                  // forwards recorded since profile_begin
    cudaEvent_t* prof_events;        // kProfRing * 3, created on the first profile_begin
};

namespace {

constexpr int kProfRing = 1024;

size_t elem_size(slide_attn_dtype t) { return t == SLIDE_ATTN_BF16 ? 2 : 4; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The context's workspace, status word and streams belong to the device it was created on; a launch
// with another device current would hand that device foreign pointers.
bool on_ctx_device(const slide_attn_ctx* c) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return false; }
    return dev == c->device;
}

bool variant_supported(const slide_attn_ctx* c, slide_attn_variant v) {
    switch (v) {
        case SLIDE_ATTN_VARIANT_DIRECT: return direct_supports(c->head_dim, c->ksize);
        case SLIDE_ATTN_VARIANT_STRIP: return c->strip_ws && strip_supports(c->head_dim, c->ksize);
        case SLIDE_ATTN_VARIANT_MMA: return c->workspace && mma_supports(c->dtype, c->head_dim, c->ksize);
        case SLIDE_ATTN_VARIANT_UMMA_TS: return c->umma_ws && umma_ts_supports(c->dtype, c->head_dim, c->ksize);
        case SLIDE_ATTN_VARIANT_TILE: return c->strip_ws && tile_supports(c->head_dim, c->ksize);
        case SLIDE_ATTN_VARIANT_MMA_WIDE: return c->wide_ws && mma_wide_supports(c->dtype, c->head_dim, c->ksize);
        default: return false;
    }
}

slide_attn_variant pick_variant(const slide_attn_ctx* c) {
    const slide_attn_variant order[] = {SLIDE_ATTN_VARIANT_UMMA_TS, SLIDE_ATTN_VARIANT_MMA, SLIDE_ATTN_VARIANT_MMA_WIDE, SLIDE_ATTN_VARIANT_TILE,
                                        SLIDE_ATTN_VARIANT_STRIP, SLIDE_ATTN_VARIANT_DIRECT};
    for (slide_attn_variant v : order)
        if (variant_supported(c, v)) return v;
    return SLIDE_ATTN_VARIANT_DIRECT;
}

slide_attn_status validate_shape(int B, int H, int W, int heads, int head_dim, int ksize,
                                 slide_attn_dtype dtype) {
    if (B < 1 || H < 1 || W < 1 || heads < 1 || head_dim < 1 || ksize < 1)
        return SLIDE_ATTN_ERR_INVALID_ARG;
    if (dtype != SLIDE_ATTN_F32 && dtype != SLIDE_ATTN_BF16) return SLIDE_ATTN_ERR_INVALID_ARG;
    if ((ksize & 1) == 0 || ksize > 15) return SLIDE_ATTN_ERR_UNSUPPORTED;
    if (head_dim % 8 != 0 || head_dim > 256) return SLIDE_ATTN_ERR_UNSUPPORTED;
    // element counts must fit the kernels' index arithmetic
    const long long n = (long long)B * H * W;
    if (n > (1LL << 40) / ((long long)heads * head_dim)) return SLIDE_ATTN_ERR_UNSUPPORTED;
    return SLIDE_ATTN_OK;
}

// Launches the context's variant on problem `p` (the context's shape, or a batch slice of it).
slide_attn_status launch_problem(slide_attn_ctx* c, const Problem& p, cudaStream_t stream, bool profile)
{
    cudaEvent_t* ev = nullptr;
    if (profile) {
        ev = c->prof_events + 3 * (c->prof_count % kProfRing);
        cudaEventRecord(ev[0], stream);
    }
    cudaError_t err;
    if (c->fixed_shift) {
        err = launch_shift_check(p, c->d_status, stream);
        if (ev) cudaEventRecord(ev[1], stream);
        if (err == cudaSuccess) err = launch_shift(p, c->d_status, stream);
        if (ev) { cudaEventRecord(ev[2], stream); c->prof_count++; }
        return err == cudaSuccess ? SLIDE_ATTN_OK : SLIDE_ATTN_ERR_CUDA;
    }
    switch (c->variant) {
        case SLIDE_ATTN_VARIANT_DIRECT:
            if (ev) cudaEventRecord(ev[1], stream);
            err = launch_direct(p, stream);
            break;
        case SLIDE_ATTN_VARIANT_STRIP:
            err = launch_strip_prep(p, c->strip_ws, stream);
            if (ev) cudaEventRecord(ev[1], stream);
            if (err == cudaSuccess) err = launch_strip_main(p, c->strip_ws, stream);
            break;
        case SLIDE_ATTN_VARIANT_MMA:
            err = launch_mma_prep(p, c->workspace, stream);
            if (ev) cudaEventRecord(ev[1], stream);
            if (err == cudaSuccess) err = launch_mma_main(p, c->workspace, c->d_status, stream);
            break;
        case SLIDE_ATTN_VARIANT_UMMA_TS:
            err = launch_umma_ts_prep(p, c->umma_ws, stream);
            if (ev) cudaEventRecord(ev[1], stream);
            if (err == cudaSuccess) err = launch_umma_ts(p, c->umma_ws, c->d_status, c->num_sms, stream);
            break;
        case SLIDE_ATTN_VARIANT_MMA_WIDE:
            if (ev) cudaEventRecord(ev[1], stream);          // the prep launch is issued inside launch_mma_wide
            err = launch_mma_wide(p, c->wide_ws, c->d_status, stream);
            break;
        case SLIDE_ATTN_VARIANT_TILE:
            err = launch_strip_prep(p, c->strip_ws, stream);
            if (ev) cudaEventRecord(ev[1], stream);
            if (err == cudaSuccess) err = launch_tile(p, c->strip_ws, c->d_status, stream);
            break;
        default: return SLIDE_ATTN_ERR_UNSUPPORTED;
    }
    if (ev) {
        cudaEventRecord(ev[2], stream);
        c->prof_count++;
    }
    return err == cudaSuccess ? SLIDE_ATTN_OK : SLIDE_ATTN_ERR_CUDA;
}

}  // namespace

extern "C" {

slide_attn_status slide_attn_create(slide_attn_ctx** ctx, int B, int H, int W, int heads,
                                    int head_dim, int ksize, slide_attn_dtype dtype, int has_bias)
{
    if (!ctx) return SLIDE_ATTN_ERR_INVALID_ARG;
    slide_attn_status st = validate_shape(B, H, W, heads, head_dim, ksize, dtype);
    if (st != SLIDE_ATTN_OK) return st;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return SLIDE_ATTN_ERR_CUDA;
    }
    if (major != 10) return SLIDE_ATTN_ERR_ARCH;
    int num_sms = 0;
    if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || num_sms < 1) {
        cudaGetLastError();
        return SLIDE_ATTN_ERR_CUDA;
    }

    slide_attn_ctx* c = new (std::nothrow) slide_attn_ctx();
    if (!c) return SLIDE_ATTN_ERR_ALLOC;
    c->B = B; c->H = H; c->W = W; c->heads = heads; c->head_dim = head_dim; c->ksize = ksize;
    c->has_bias = has_bias ? 1 : 0;
    c->dtype = dtype;
    c->device = dev;
    c->num_sms = num_sms;
    c->d_status = nullptr; c->workspace = nullptr; c->workspace_bytes = 0;
    c->stage = nullptr; c->stage_bytes = 0;
    c->profiling = false; c->prof_count = 0; c->prof_events = nullptr;
    if (cudaMalloc(&c->d_status, sizeof(int)) != cudaSuccess ||
        cudaMemset(c->d_status, 0, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        slide_attn_destroy(c);
        return SLIDE_ATTN_ERR_ALLOC;
    }
    if (mma_supports(dtype, head_dim, ksize)) {
        if (mma_setup() != cudaSuccess || umma_ts_setup() != cudaSuccess) {
            cudaGetLastError();
            slide_attn_destroy(c);
            return SLIDE_ATTN_ERR_CUDA;
        }
        c->workspace_bytes = mma_workspace_bytes(heads);
        if (cudaMalloc(&c->workspace, c->workspace_bytes) != cudaSuccess) {
            cudaGetLastError();
            c->workspace = nullptr;
            slide_attn_destroy(c);
            return SLIDE_ATTN_ERR_ALLOC;
        }
        if (cudaMalloc(&c->umma_ws, umma_ts_workspace_bytes(heads)) != cudaSuccess) {
            cudaGetLastError();
            c->umma_ws = nullptr;
            slide_attn_destroy(c);
            return SLIDE_ATTN_ERR_ALLOC;
        }
    }
    if (mma_wide_supports(dtype, head_dim, ksize) &&
        cudaMalloc(&c->wide_ws, mma_wide_workspace_bytes(heads, ksize)) != cudaSuccess) {
        cudaGetLastError();
        c->wide_ws = nullptr;
        slide_attn_destroy(c);
        return SLIDE_ATTN_ERR_ALLOC;
    }
    if (strip_supports(head_dim, ksize) &&
        cudaMalloc(&c->strip_ws, strip_workspace_bytes(heads, head_dim, ksize)) != cudaSuccess) {
        cudaGetLastError();
        c->strip_ws = nullptr;
        slide_attn_destroy(c);
        return SLIDE_ATTN_ERR_ALLOC;
    }
    c->variant = pick_variant(c);
    *ctx = c;
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_forward(slide_attn_ctx* c, const void* q, const void* k, const void* v,
                                     const float* wk, const float* wv, const float* bias,
                                     void* out, void* cuda_stream)
{
    if (!c || !q || !k || !v || !wk || !wv || !out) return SLIDE_ATTN_ERR_INVALID_ARG;
    if ((c->has_bias != 0) != (bias != nullptr)) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (out == q || out == k || out == v) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!on_ctx_device(c)) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(wk) ||
        !aligned16(wv) || (bias && !aligned16(bias)))
        return SLIDE_ATTN_ERR_ALIGNMENT;

    Problem p;
    p.B = c->B; p.H = c->H; p.W = c->W; p.heads = c->heads; p.head_dim = c->head_dim;
    p.ksize = c->ksize; p.has_bias = c->has_bias; p.dtype = c->dtype;
    p.q = q; p.k = k; p.v = v; p.wk = wk; p.wv = wv; p.bias = bias; p.out = out;
    return launch_problem(c, p, static_cast<cudaStream_t>(cuda_stream), c->profiling);
}

slide_attn_status slide_attn_forward_host(slide_attn_ctx* c, const void* q, const void* k,
                                          const void* v, const float* wk, const float* wv,
                                          const float* bias, void* out, void* cuda_stream)
{
    if (!c || !q || !k || !v || !wk || !wv || !out) return SLIDE_ATTN_ERR_INVALID_ARG;
    if ((c->has_bias != 0) != (bias != nullptr)) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!on_ctx_device(c)) return SLIDE_ATTN_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    const size_t C = (size_t)c->heads * c->head_dim, k2 = (size_t)c->ksize * c->ksize;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t t_raw = (size_t)c->B * c->H * c->W * C * elem_size(c->dtype);
    const size_t w_raw = C * k2 * k2 * sizeof(float);
    const size_t b_raw = (size_t)c->heads * k2 * sizeof(float);
    const size_t t_bytes = up(t_raw), w_bytes = up(w_raw), b_bytes = up(b_raw);
    const size_t total = 4 * t_bytes + 2 * w_bytes + b_bytes;
    if (c->stage_bytes < total) {
        if (c->stage) { cudaFree(c->stage); c->stage = nullptr; c->stage_bytes = 0; }
        if (cudaMalloc(&c->stage, total) != cudaSuccess) { cudaGetLastError(); return SLIDE_ATTN_ERR_ALLOC; }
        c->stage_bytes = total;
    }
    char* base = static_cast<char*>(c->stage);
    void* dq = base;
    void* dk = base + t_bytes;
    void* dv = base + 2 * t_bytes;
    void* dout = base + 3 * t_bytes;
    float* dwk = reinterpret_cast<float*>(base + 4 * t_bytes);
    float* dwv = reinterpret_cast<float*>(base + 4 * t_bytes + w_bytes);
    float* dbias = reinterpret_cast<float*>(base + 4 * t_bytes + 2 * w_bytes);

    // Images are independent, so the batch goes through in slices: slice i+1 is copied in (one copy
    // stream) while slice i is computed (the caller's stream) and slice i-1 is copied out (a second
    // copy stream).  The two directions of the host link then run at the same time.
    if (!c->host_pipe) {
        bool made = cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking) == cudaSuccess;
        for (cudaEvent_t& e : c->host_ev)
            made = made && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
        if (!made) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
        c->host_pipe = true;
    }
    const int nslices = c->B < 4 ? (c->B < 2 || t_raw < (4u << 20) ? 1 : 2) : 4;   // 4 measured best (2: +1 %, 8: +6 %)
    const size_t img = t_raw / (size_t)c->B;                     // bytes of one image (multiple of 16)
    cudaEvent_t e_start = c->host_ev[0], e_done = c->host_ev[1];

    bool ok = cudaEventRecord(e_start, stream) == cudaSuccess &&
              cudaStreamWaitEvent(c->copy_in, e_start, 0) == cudaSuccess &&
              cudaStreamWaitEvent(c->copy_out, e_start, 0) == cudaSuccess &&
              cudaMemcpyAsync(dwk, wk, w_raw, cudaMemcpyHostToDevice, c->copy_in) == cudaSuccess &&
              cudaMemcpyAsync(dwv, wv, w_raw, cudaMemcpyHostToDevice, c->copy_in) == cudaSuccess;
    if (ok && bias)
        ok = cudaMemcpyAsync(dbias, bias, b_raw, cudaMemcpyHostToDevice, c->copy_in) == cudaSuccess;
    slide_attn_status st = SLIDE_ATTN_OK;
    for (int i = 0; ok && st == SLIDE_ATTN_OK && i < nslices; ++i) {
        const int b0 = (int)((long long)c->B * i / nslices), b1 = (int)((long long)c->B * (i + 1) / nslices);
        if (b1 == b0) continue;
        const size_t off = (size_t)b0 * img, bytes = (size_t)(b1 - b0) * img;
        cudaEvent_t e_in = c->host_ev[2 + 2 * i], e_k = c->host_ev[3 + 2 * i];
        ok = cudaMemcpyAsync((char*)dq + off, (const char*)q + off, bytes, cudaMemcpyHostToDevice, c->copy_in) == cudaSuccess &&
             cudaMemcpyAsync((char*)dk + off, (const char*)k + off, bytes, cudaMemcpyHostToDevice, c->copy_in) == cudaSuccess &&
             cudaMemcpyAsync((char*)dv + off, (const char*)v + off, bytes, cudaMemcpyHostToDevice, c->copy_in) == cudaSuccess &&
             cudaEventRecord(e_in, c->copy_in) == cudaSuccess &&
             cudaStreamWaitEvent(stream, e_in, 0) == cudaSuccess;
        if (!ok) break;
        Problem p;
        p.B = b1 - b0; p.H = c->H; p.W = c->W; p.heads = c->heads; p.head_dim = c->head_dim;
        p.ksize = c->ksize; p.has_bias = c->has_bias; p.dtype = c->dtype;
        p.q = (char*)dq + off; p.k = (char*)dk + off; p.v = (char*)dv + off;
        p.wk = dwk; p.wv = dwv; p.bias = bias ? dbias : nullptr; p.out = (char*)dout + off;
        st = launch_problem(c, p, stream, false);
        if (st != SLIDE_ATTN_OK) break;
        ok = cudaEventRecord(e_k, stream) == cudaSuccess &&
             cudaStreamWaitEvent(c->copy_out, e_k, 0) == cudaSuccess &&
             cudaMemcpyAsync((char*)out + off, (char*)dout + off, bytes, cudaMemcpyDeviceToHost, c->copy_out) == cudaSuccess;
    }
    // whatever happened, leave nothing of this call in flight
    const bool joined = cudaEventRecord(e_done, c->copy_out) == cudaSuccess &&
                        cudaStreamWaitEvent(stream, e_done, 0) == cudaSuccess &&
                        cudaStreamSynchronize(c->copy_in) == cudaSuccess &&
                        cudaStreamSynchronize(stream) == cudaSuccess;
    if (st != SLIDE_ATTN_OK) return st;
    if (!ok || !joined) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_backward(slide_attn_ctx* c, const void* q, const void* k, const void* v,
                                      const float* wk, const float* wv, const float* bias, const void* dout,
                                      void* dq, void* dk, void* dv, float* dwk, float* dwv, float* dbias,
                                      void* cuda_stream)
{
    if (!c || !q || !k || !v || !wk || !wv || !dout || !dq || !dk || !dv || !dwk || !dwv) return SLIDE_ATTN_ERR_INVALID_ARG;
    if ((c->has_bias != 0) != (bias != nullptr) || (c->has_bias != 0) != (dbias != nullptr)) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!on_ctx_device(c)) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!backward_supports(c->head_dim, c->ksize) || !c->strip_ws) return SLIDE_ATTN_ERR_UNSUPPORTED;
    const void* ptrs[] = {q, k, v, wk, wv, dout, dq, dk, dv, dwk, dwv};
    for (const void* p : ptrs) if (!aligned16(p)) return SLIDE_ATTN_ERR_ALIGNMENT;
    if ((bias && !aligned16(bias)) || (dbias && !aligned16(dbias))) return SLIDE_ATTN_ERR_ALIGNMENT;
    if (dq == q || dq == k || dq == v || dq == dout || dk == q || dk == k || dk == v || dk == dout ||
        dv == q || dv == k || dv == v || dv == dout || dq == dk || dq == dv || dk == dv)
        return SLIDE_ATTN_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (!c->bwd_ws) {
        if (cudaMalloc(&c->bwd_ws, backward_workspace_bytes(c->B, c->H, c->W, c->heads, c->ksize)) != cudaSuccess) {
            cudaGetLastError();
            c->bwd_ws = nullptr;
            return SLIDE_ATTN_ERR_ALLOC;
        }
    }
    Problem p;
    p.B = c->B; p.H = c->H; p.W = c->W; p.heads = c->heads; p.head_dim = c->head_dim;
    p.ksize = c->ksize; p.has_bias = c->has_bias; p.dtype = c->dtype;
    p.q = q; p.k = k; p.v = v; p.wk = wk; p.wv = wv; p.bias = bias; p.out = nullptr;
    BackwardArgs ga = {dout, dq, dk, dv, dwk, dwv, dbias};
    const size_t k2 = (size_t)c->ksize * c->ksize;
    const size_t wbytes = (size_t)c->heads * c->head_dim * k2 * k2 * sizeof(float);
    bool ok = cudaMemsetAsync(dwk, 0, wbytes, stream) == cudaSuccess && cudaMemsetAsync(dwv, 0, wbytes, stream) == cudaSuccess;
    if (ok && dbias) ok = cudaMemsetAsync(dbias, 0, (size_t)c->heads * k2 * sizeof(float), stream) == cudaSuccess;
    if (ok) ok = launch_strip_prep(p, c->strip_ws, stream) == cudaSuccess;
    if (ok) ok = launch_backward(p, ga, c->strip_ws, c->bwd_ws, c->d_status, c->num_sms, stream) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
    return SLIDE_ATTN_OK;
}

namespace {

size_t block_tensor_bytes(const slide_attn_ctx* c) {
    const size_t raw = (size_t)c->B * c->H * c->W * c->heads * c->head_dim * 2;
    return (raw + 255) & ~(size_t)255;
}

slide_attn_status proj_check(slide_attn_ctx* c) {
    const int C = c->heads * c->head_dim;
    if (c->dtype != SLIDE_ATTN_BF16 || !proj_supports(C, C)) return SLIDE_ATTN_ERR_UNSUPPORTED;
    if ((long long)c->B * c->H * c->W > 0x7fffff00LL) return SLIDE_ATTN_ERR_UNSUPPORTED;
    if (!c->proj_ready) {
        if (proj_setup() != cudaSuccess) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
        c->proj_ready = true;
    }
    return SLIDE_ATTN_OK;
}

// Scratch of the block: four bf16 token tensors (q, k, v, z).
slide_attn_status block_scratch(slide_attn_ctx* c) {
    slide_attn_status st = proj_check(c);
    if (st != SLIDE_ATTN_OK) return st;
    if (c->block_ws) return SLIDE_ATTN_OK;
    const size_t total = 4 * block_tensor_bytes(c);
    if (cudaMalloc(&c->block_ws, total) != cudaSuccess) {
        cudaGetLastError();
        c->block_ws = nullptr;
        return SLIDE_ATTN_ERR_ALLOC;
    }
    return SLIDE_ATTN_OK;
}

}  // namespace

slide_attn_status slide_attn_project(slide_attn_ctx* c, const void* x, const float* w, int nmat,
                                     void* y0, void* y1, void* y2, void* cuda_stream)
{
    if (!c || !x || !w || nmat < 1 || nmat > 3 || !y0 || (nmat > 1 && !y1) || (nmat > 2 && !y2)) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!on_ctx_device(c)) return SLIDE_ATTN_ERR_INVALID_ARG;
    void* y[3] = {y0, nmat > 1 ? y1 : nullptr, nmat > 2 ? y2 : nullptr};
    if (!aligned16(x) || !aligned16(w)) return SLIDE_ATTN_ERR_ALIGNMENT;
    for (int i = 0; i < nmat; ++i) {
        if (!aligned16(y[i])) return SLIDE_ATTN_ERR_ALIGNMENT;
        if (y[i] == x) return SLIDE_ATTN_ERR_INVALID_ARG;
        for (int j = 0; j < i; ++j) if (y[i] == y[j]) return SLIDE_ATTN_ERR_INVALID_ARG;
    }
    slide_attn_status st = proj_check(c);
    if (st != SLIDE_ATTN_OK) return st;
    const int C = c->heads * c->head_dim;
    if (launch_proj(x, (long long)c->B * c->H * c->W, C, w, C, nmat, y, c->d_status, c->num_sms,
                    static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        cudaGetLastError();
        return SLIDE_ATTN_ERR_CUDA;
    }
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_block_forward(slide_attn_ctx* c, const void* x, const float* w_qkv, const float* w_o,
                                           const float* wk, const float* wv, const float* bias, void* out,
                                           void* cuda_stream)
{
    if (!c || !x || !w_qkv || !w_o || !wk || !wv || !out) return SLIDE_ATTN_ERR_INVALID_ARG;
    if ((c->has_bias != 0) != (bias != nullptr)) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (out == x) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!on_ctx_device(c)) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(out) || !aligned16(w_qkv) || !aligned16(w_o) || !aligned16(wk) || !aligned16(wv) ||
        (bias && !aligned16(bias)))
        return SLIDE_ATTN_ERR_ALIGNMENT;
    slide_attn_status st = block_scratch(c);
    if (st != SLIDE_ATTN_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int C = c->heads * c->head_dim;
    const long long rows = (long long)c->B * c->H * c->W;
    const size_t tb = block_tensor_bytes(c);
    unsigned char* base = static_cast<unsigned char*>(c->block_ws);
    void* qkv[3] = {base, base + tb, base + 2 * tb};
    void* z = base + 3 * tb;

    if (launch_proj(x, rows, C, w_qkv, C, 3, qkv, c->d_status, c->num_sms, stream) != cudaSuccess) {
        cudaGetLastError();
        return SLIDE_ATTN_ERR_CUDA;
    }
    Problem p;
    p.B = c->B; p.H = c->H; p.W = c->W; p.heads = c->heads; p.head_dim = c->head_dim;
    p.ksize = c->ksize; p.has_bias = c->has_bias; p.dtype = c->dtype;
    p.q = qkv[0]; p.k = qkv[1]; p.v = qkv[2]; p.wk = wk; p.wv = wv; p.bias = bias; p.out = z;
    st = launch_problem(c, p, stream, false);
    if (st != SLIDE_ATTN_OK) return st;
    void* ys[1] = {out};
    if (launch_proj(z, rows, C, w_o, C, 1, ys, c->d_status, c->num_sms, stream) != cudaSuccess) {
        cudaGetLastError();
        return SLIDE_ATTN_ERR_CUDA;
    }
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_set_variant(slide_attn_ctx* c, slide_attn_variant variant)
{
    if (!c) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (variant == SLIDE_ATTN_VARIANT_AUTO) { c->variant = pick_variant(c); return SLIDE_ATTN_OK; }
    if (variant != SLIDE_ATTN_VARIANT_DIRECT && variant != SLIDE_ATTN_VARIANT_MMA && variant != SLIDE_ATTN_VARIANT_UMMA_TS &&
        variant != SLIDE_ATTN_VARIANT_STRIP && variant != SLIDE_ATTN_VARIANT_TILE && variant != SLIDE_ATTN_VARIANT_MMA_WIDE)
        return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!variant_supported(c, variant)) return SLIDE_ATTN_ERR_UNSUPPORTED;
    c->variant = variant;
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_set_fixed_shift(slide_attn_ctx* c, int enable)
{
    if (!c) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (enable && !shift_supports(c->head_dim, c->ksize)) return SLIDE_ATTN_ERR_UNSUPPORTED;
    c->fixed_shift = enable != 0;
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_detect_fixed_shift(slide_attn_ctx* c, const float* wk, const float* wv,
                                                int* is_fixed, void* cuda_stream)
{
    if (!c || !wk || !wv || !is_fixed) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!on_ctx_device(c)) return SLIDE_ATTN_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // a word of its own is not needed: the context's status word is read, used and restored in
    // stream order, and the call waits for all of it
    int before = 0, after = 0;
    Problem p = {};
    p.heads = c->heads; p.head_dim = c->head_dim; p.ksize = c->ksize; p.wk = wk; p.wv = wv;
    bool ok = cudaMemcpyAsync(&before, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream) == cudaSuccess &&
              cudaMemsetAsync(c->d_status, 0, sizeof(int), stream) == cudaSuccess &&
              launch_shift_check(p, c->d_status, stream) == cudaSuccess &&
              cudaMemcpyAsync(&after, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream) == cudaSuccess &&
              cudaStreamSynchronize(stream) == cudaSuccess;
    if (ok) ok = cudaMemcpyAsync(c->d_status, &before, sizeof(int), cudaMemcpyHostToDevice, stream) == cudaSuccess &&
                 cudaStreamSynchronize(stream) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
    *is_fixed = after == 0 ? 1 : 0;
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_get_variant(const slide_attn_ctx* c, slide_attn_variant* variant)
{
    if (!c || !variant) return SLIDE_ATTN_ERR_INVALID_ARG;
    *variant = c->variant;
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_launches_per_forward(const slide_attn_ctx* c, int* n)
{
    if (!c || !n) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (c->fixed_shift) { *n = 2; return SLIDE_ATTN_OK; }   // weight check + fixed-shift kernel
    switch (c->variant) {
        case SLIDE_ATTN_VARIANT_DIRECT: *n = 1; break;
        case SLIDE_ATTN_VARIANT_MMA: *n = 2; break;      // weight re-layout + fused kernel
        case SLIDE_ATTN_VARIANT_STRIP: *n = 2; break;    // weight transpose + fused kernel
        case SLIDE_ATTN_VARIANT_UMMA_TS: *n = 2; break;  // B-image prep + fused kernel
        case SLIDE_ATTN_VARIANT_TILE: *n = 2; break;     // weight transpose + fused kernel
        case SLIDE_ATTN_VARIANT_MMA_WIDE: *n = 2; break; // weight fragments + fused kernel
        default: *n = 1; break;
    }
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_profile_begin(slide_attn_ctx* c)
{
    if (!c) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!c->prof_events) {
        cudaEvent_t* ev = new (std::nothrow) cudaEvent_t[3 * kProfRing];
        if (!ev) return SLIDE_ATTN_ERR_ALLOC;
        for (int i = 0; i < 3 * kProfRing; ++i) {
            if (cudaEventCreate(&ev[i]) != cudaSuccess) {
                cudaGetLastError();
                for (int j = 0; j < i; ++j) cudaEventDestroy(ev[j]);
                delete[] ev;
                return SLIDE_ATTN_ERR_CUDA;
            }
        }
        c->prof_events = ev;
    }
    c->prof_count = 0;
    c->profiling = true;
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_profile_end(slide_attn_ctx* c, double* forward_ms, double* main_ms, int* n)
{
    if (!c) return SLIDE_ATTN_ERR_INVALID_ARG;
    if (!c->profiling) return SLIDE_ATTN_ERR_INVALID_ARG;
    c->profiling = false;
    const int cnt = c->prof_count < kProfRing ? c->prof_count : kProfRing;
    double fwd = 0.0, mn = 0.0;
    for (int i = 0; i < cnt; ++i) {
        cudaEvent_t* ev = c->prof_events + 3 * i;
        float a = 0.f, b = 0.f;
        if (cudaEventSynchronize(ev[2]) != cudaSuccess ||
            cudaEventElapsedTime(&a, ev[0], ev[2]) != cudaSuccess ||
            cudaEventElapsedTime(&b, ev[1], ev[2]) != cudaSuccess) {
            cudaGetLastError();
            return SLIDE_ATTN_ERR_CUDA;
        }
        fwd += a; mn += b;
    }
    if (forward_ms) *forward_ms = cnt ? fwd / cnt : 0.0;
    if (main_ms) *main_ms = cnt ? mn / cnt : 0.0;
    if (n) *n = cnt;
    return SLIDE_ATTN_OK;
}

slide_attn_status slide_attn_query_status(slide_attn_ctx* c, void* cuda_stream)
{
    if (!c || !on_ctx_device(c)) return SLIDE_ATTN_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaMemsetAsync(c->d_status, 0, sizeof(int), stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return SLIDE_ATTN_ERR_CUDA;
    }
    return word == 0 ? SLIDE_ATTN_OK : (word == 2 ? SLIDE_ATTN_ERR_NOT_FIXED_SHIFT : SLIDE_ATTN_ERR_TIMEOUT);
}

slide_attn_status slide_attn_destroy(slide_attn_ctx* c)
{
    if (!c) return SLIDE_ATTN_OK;
    bool ok = true;
    if (c->d_status) ok &= cudaFree(c->d_status) == cudaSuccess;
    if (c->workspace) ok &= cudaFree(c->workspace) == cudaSuccess;
    if (c->strip_ws) ok &= cudaFree(c->strip_ws) == cudaSuccess;
    if (c->umma_ws) ok &= cudaFree(c->umma_ws) == cudaSuccess;
    if (c->bwd_ws) ok &= cudaFree(c->bwd_ws) == cudaSuccess;
    if (c->wide_ws) ok &= cudaFree(c->wide_ws) == cudaSuccess;
    if (c->block_ws) ok &= cudaFree(c->block_ws) == cudaSuccess;
    if (c->stage) ok &= cudaFree(c->stage) == cudaSuccess;
    if (c->host_pipe) {
        ok &= cudaStreamDestroy(c->copy_in) == cudaSuccess;
        ok &= cudaStreamDestroy(c->copy_out) == cudaSuccess;
        for (cudaEvent_t e : c->host_ev) ok &= cudaEventDestroy(e) == cudaSuccess;
    }
    if (c->prof_events) {
        for (int i = 0; i < 3 * kProfRing; ++i) ok &= cudaEventDestroy(c->prof_events[i]) == cudaSuccess;
        delete[] c->prof_events;
    }
    delete c;
    if (!ok) { cudaGetLastError(); return SLIDE_ATTN_ERR_CUDA; }
    return SLIDE_ATTN_OK;
}

const char* slide_attn_status_string(slide_attn_status status)
{
    switch (status) {
        case SLIDE_ATTN_OK: return "ok";
        case SLIDE_ATTN_ERR_INVALID_ARG: return "invalid argument";
        case SLIDE_ATTN_ERR_UNSUPPORTED: return "unsupported shape, window size or variant";
        case SLIDE_ATTN_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case SLIDE_ATTN_ERR_ALLOC: return "allocation failed";
        case SLIDE_ATTN_ERR_CUDA: return "CUDA call failed";
        case SLIDE_ATTN_ERR_ARCH: return "device is not sm_100 (B200)";
        case SLIDE_ATTN_ERR_TIMEOUT: return "device-side wait timed out";
        case SLIDE_ATTN_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of slide_attn_forward_noalloc (16 heads)";
        case SLIDE_ATTN_ERR_NOT_FIXED_SHIFT: return "fixed-shift mode, but a weight is not the one-hot shift kernel";
        default: return "unknown status";
    }
}

}  // extern "C"
