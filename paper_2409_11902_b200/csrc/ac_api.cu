// C-ABI entry points: argument validation, planning, dispatch. See include/ac.h.
#include "ac_common.h"

namespace ac {

namespace {
thread_local int g_sm_budget = kNumSMs;
}

ac_status launch_relu_mask_backward(const Dims& d, const void* mask, const void* dy, void* dx, cudaStream_t st);   // compress.cu
ac_status launch_compress_mask_y(const Dims& d, const void* a, void* y, void* z, void* mask, cudaStream_t st);      // compress.cu

ac_status make_dims(const ac_conv_desc* d, bool need_conv, Dims* o, int k_h, int k_w) {
    if (!d || !o) return AC_ERR_INVALID_ARG;
    *o = Dims{};   // plans are cached by the bytes of this struct
    const bool rect = k_h != 0 || k_w != 0;
    if (rect && (k_h <= 0 || k_w <= 0)) return AC_ERR_INVALID_ARG;
    if (d->N <= 0 || d->C_in <= 0 || d->H <= 0 || d->W <= 0 || (!rect && d->k <= 0)) return AC_ERR_INVALID_ARG;
    if (d->dtype != AC_F32 && d->dtype != AC_BF16) return AC_ERR_INVALID_ARG;
    if (d->layout != AC_NCHW && d->layout != AC_NHWC) return AC_ERR_INVALID_ARG;
    o->N = d->N; o->Ci = d->C_in; o->H = d->H; o->W = d->W;
    o->kh = rect ? k_h : d->k; o->kw = rect ? k_w : d->k; o->k = o->kh;
    o->dtype = d->dtype; o->layout = d->layout;
    o->elt = d->dtype == AC_F32 ? 4 : 2;
    o->sms = g_sm_budget;
    o->Hp = (d->H + o->kh - 1) / o->kh;
    o->Wp = (d->W + o->kw - 1) / o->kw;
    o->Co = 1; o->R = 1; o->S = 1; o->sh = 1; o->sw = 1; o->ph = 0; o->pw = 0;
    o->Ho = d->H; o->Wo = d->W;
    const long long lim = 1ll << 40;  // elements; far above 180 GB of any dtype
    if ((long long)d->N * d->C_in * d->H * d->W >= lim) return AC_ERR_INVALID_ARG;
    if (!need_conv) return AC_OK;
    if (d->C_out <= 0 || d->R <= 0 || d->S <= 0 || d->stride_h <= 0 || d->stride_w <= 0 ||
        d->pad_h < 0 || d->pad_w < 0)
        return AC_ERR_INVALID_ARG;
    if (d->H + 2 * (long long)d->pad_h < d->R || d->W + 2 * (long long)d->pad_w < d->S)
        return AC_ERR_INVALID_ARG;  // empty output
    o->Co = d->C_out; o->R = d->R; o->S = d->S;
    o->sh = d->stride_h; o->sw = d->stride_w; o->ph = d->pad_h; o->pw = d->pad_w;
    o->Ho = (d->H + 2 * d->pad_h - d->R) / d->stride_h + 1;
    o->Wo = (d->W + 2 * d->pad_w - d->S) / d->stride_w + 1;
    if ((long long)d->N * d->C_out * o->Ho * o->Wo >= lim) return AC_ERR_INVALID_ARG;
    if ((long long)d->C_out * d->C_in * d->R * d->S >= (1ll << 31)) return AC_ERR_INVALID_ARG;
    if ((long long)d->C_in * d->R * d->S >= (1ll << 31)) return AC_ERR_INVALID_ARG;
    return AC_OK;
}

static inline long long ceil_div(long long a, long long b) { return (a + b - 1) / b; }

WgradPlan plan_wgrad_simt(const Dims& d, size_t max_partial_bytes) {
    WgradPlan p{};
    p.path = PATH_SIMT;
    const long long K = d.K();
    const long long J = (long long)d.Ci * d.R * d.S;
    const long long tiles = ceil_div(d.Co, 64) * ceil_div(J, 64);
    // enough blocks to fill the chip four times over, slices of 256..2048
    // positions so that each fp32 running sum stays short
    long long want = ceil_div(4 * kNumSMs, tiles);
    long long kps = ceil_div(ceil_div(K, want), 16) * 16;
    if (kps < 256) kps = 256;
    if (kps > 2048) kps = 2048;
    const long long dw_bytes = d.dw_elems() * 4;
    long long max_splits = (long long)max_partial_bytes / dw_bytes;
    if (max_splits < 1) max_splits = 1;
    if (max_splits > 65535) max_splits = 65535;
    if (ceil_div(K, kps) > max_splits) kps = ceil_div(ceil_div(K, max_splits), 16) * 16;
    p.simt_k_per_split = kps;
    p.splits = (int)ceil_div(K, kps);
    p.bytes = kStatusBlockBytes + (p.splits > 1 ? (size_t)p.splits * dw_bytes : 0);
    return p;
}

namespace {
thread_local cudaEvent_t g_hook_events[2] = {nullptr, nullptr};
}

void record_timing_hook(int which, cudaStream_t stream) {
    cudaEvent_t ev = g_hook_events[which];
    if (!ev) return;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess) return;
    cudaEventRecordWithFlags(ev, stream,
                             cs == cudaStreamCaptureStatusActive ? cudaEventRecordExternal : cudaEventRecordDefault);
}

// The plan for a caller whose workspace has no room for staged operand copies.
WgradPlan plan_wgrad_unstaged(const Dims& d) {
    if (tc2_supported(d, nullptr)) {
        WgradPlan p{};
        plan_tc2(d, &p);
        return p;
    }
    if (tc_supported(d)) {
        WgradPlan p{};
        p.path = PATH_TC;
        plan_tc(d, &p);
        return p;
    }
    return plan_wgrad_simt(d);
}

WgradPlan plan_wgrad(const Dims& d) {
    if (tc2_supported(d, nullptr)) {
        WgradPlan p{};
        if (staged_inflate_preferred(d)) plan_staged(d, &p); else plan_tc2(d, &p);
        return p;
    }
    if (staged_supported(d)) {
        WgradPlan p{};
        plan_staged(d, &p);
        return p;
    }
    if (gather_supported(d)) {
        WgradPlan p{};
        plan_gather(d, &p);
        return p;
    }
    if (tc_supported(d)) {
        WgradPlan p{};
        p.path = PATH_TC;
        plan_tc(d, &p);
        return p;
    }
    return plan_wgrad_simt(d);
}

}  // namespace ac

using namespace ac;

extern "C" {

ac_status ac_set_sm_budget(int32_t sms) {
    if (sms < 0) return AC_ERR_INVALID_ARG;
    g_sm_budget = sms == 0 || sms > kNumSMs ? kNumSMs : sms;
    return AC_OK;
}

int32_t ac_get_sm_budget(void) { return g_sm_budget; }

size_t ac_workspace_bytes(const ac_conv_desc* desc) { return ac_workspace_bytes_rect(desc, 0, 0); }

size_t ac_workspace_bytes_rect(const ac_conv_desc* desc, int32_t k_h, int32_t k_w) {
    Dims d;
    if (make_dims(desc, true, &d, k_h, k_w) != AC_OK) return 0;
    return plan_wgrad(d).bytes;
}

size_t ac_workspace_bytes_min(const ac_conv_desc* desc) {
    Dims d;
    if (make_dims(desc, true, &d) != AC_OK) return 0;
    const WgradPlan p = plan_wgrad(d);
    if (p.path != PATH_STAGED && p.path != PATH_GATHER) return p.bytes;
    const size_t plain = plan_wgrad_unstaged(d).bytes;      // the path on the operands as they are
    return plain < p.bytes ? plain : p.bytes;
}

ac_status ac_compress(const ac_conv_desc* desc, const void* x, void* z, void* y_out, void* stream) {
    return ac_compress_rect(desc, 0, 0, x, z, y_out, stream);
}

ac_status ac_compress_rect(const ac_conv_desc* desc, int32_t k_h, int32_t k_w, const void* x, void* z,
                           void* y_out, void* stream) {
    Dims d;
    ac_status st = make_dims(desc, false, &d, k_h, k_w);
    if (st != AC_OK) return st;
    if (!x || !z) return AC_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(z) || !aligned16(y_out)) return AC_ERR_MISALIGNED;
    return launch_compress(d, x, z, y_out, static_cast<cudaStream_t>(stream));
}

ac_status ac_compress_relu_mask(const ac_conv_desc* desc, const void* a, void* z, void* mask,
                                void* stream) {
    Dims d;
    ac_status st = make_dims(desc, false, &d);
    if (st != AC_OK) return st;
    if (!a || !z || !mask) return AC_ERR_INVALID_ARG;
    if (!aligned16(a) || !aligned16(z) || !aligned16(mask)) return AC_ERR_MISALIGNED;
    return launch_compress_mask(d, a, z, mask, static_cast<cudaStream_t>(stream));
}

ac_status ac_compress_relu_mask_y(const ac_conv_desc* desc, const void* a, void* y_out, void* z, void* mask,
                                  void* stream) {
    Dims d;
    ac_status st = make_dims(desc, false, &d);
    if (st != AC_OK) return st;
    if (!a || !y_out || !z || !mask) return AC_ERR_INVALID_ARG;
    if (!aligned16(a) || !aligned16(y_out) || !aligned16(z) || !aligned16(mask)) return AC_ERR_MISALIGNED;
    return launch_compress_mask_y(d, a, y_out, z, mask, static_cast<cudaStream_t>(stream));
}

ac_status ac_relu_mask_backward(const ac_conv_desc* desc, const void* mask, const void* dy, void* dx,
                                void* stream) {
    Dims d;
    ac_status st = make_dims(desc, false, &d);
    if (st != AC_OK) return st;
    if (!mask || !dy || !dx) return AC_ERR_INVALID_ARG;
    if (!aligned16(mask) || !aligned16(dy) || !aligned16(dx)) return AC_ERR_MISALIGNED;
    return launch_relu_mask_backward(d, mask, dy, dx, static_cast<cudaStream_t>(stream));
}

ac_status ac_conv2d_wgrad_compressed(const ac_conv_desc* desc, const void* z, const void* dy,
                                     float* dw, void* workspace, size_t workspace_bytes,
                                     void* stream) {
    return ac_conv2d_wgrad_compressed_rect(desc, 0, 0, z, dy, dw, workspace, workspace_bytes, stream);
}

ac_status ac_conv2d_wgrad_compressed_rect(const ac_conv_desc* desc, int32_t k_h, int32_t k_w, const void* z,
                                          const void* dy, float* dw, void* workspace,
                                          size_t workspace_bytes, void* stream) {
    Dims d;
    ac_status st = make_dims(desc, true, &d, k_h, k_w);
    if (st != AC_OK) return st;
    if (!z || !dy || !dw || !workspace) return AC_ERR_INVALID_ARG;
    if (!aligned16(z) || !aligned16(dy) || !aligned16(dw) || !aligned16(workspace))
        return AC_ERR_MISALIGNED;
    WgradPlan p = plan_wgrad(d);
    if ((p.path == PATH_STAGED || p.path == PATH_GATHER) && workspace_bytes < p.bytes) p = plan_wgrad_unstaged(d);
    if (workspace_bytes < p.bytes) return AC_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (p.path == PATH_TC2) return launch_wgrad_tc2(d, p, z, dy, dw, workspace, s);   // resets the status itself
    if (p.path == PATH_STAGED) return launch_wgrad_staged(d, p, z, dy, dw, workspace, s);
    if (p.path == PATH_GATHER) return launch_wgrad_gather(d, p, z, dy, dw, workspace, s);
    AC_CUDA_TRY(cudaMemsetAsync(workspace, 0, kStatusBlockBytes, s));
    if (p.path == PATH_TC) return launch_wgrad_tc(d, p, z, dy, dw, workspace, s);
    return launch_wgrad_simt(d, p, z, dy, dw, workspace, s);
}

size_t ac_accumulate_workspace_bytes(const ac_conv_desc* desc) {
    Dims d;
    if (make_dims(desc, true, &d) != AC_OK) return 0;
    return ((plan_wgrad(d).bytes + 255) & ~(size_t)255) + (size_t)d.dw_elems() * 4;
}

ac_status ac_conv2d_wgrad_compressed_accumulate(const ac_conv_desc* desc, const void* z, const void* dy,
                                                float beta, float* dw, void* workspace,
                                                size_t workspace_bytes, void* stream) {
    Dims d;
    ac_status st = make_dims(desc, true, &d);
    if (st != AC_OK) return st;
    if (!dw || !workspace) return AC_ERR_INVALID_ARG;
    if (!aligned16(dw)) return AC_ERR_MISALIGNED;
    if (!(beta == beta) || beta - beta != 0.f) return AC_ERR_INVALID_ARG;   // NaN or infinite
    const size_t dw_bytes = (size_t)d.dw_elems() * 4;
    if (workspace_bytes < dw_bytes + 256) return AC_ERR_WORKSPACE_TOO_SMALL;
    // the gradient's own scratch in front (so that the status block stays where ac_workspace_status
    // looks for it), the new gradient behind it
    const size_t inner = (workspace_bytes - dw_bytes) & ~(size_t)255;
    float* g = reinterpret_cast<float*>(static_cast<char*>(workspace) + inner);
    st = ac_conv2d_wgrad_compressed(desc, z, dy, g, workspace, inner, stream);
    if (st != AC_OK) return st;
    return launch_axpby(g, beta, dw, d.dw_elems(), static_cast<cudaStream_t>(stream));
}

ac_status ac_set_kernel_timing_events(void* before, void* after) {
    const bool on = before && after;
    g_hook_events[0] = on ? static_cast<cudaEvent_t>(before) : nullptr;
    g_hook_events[1] = on ? static_cast<cudaEvent_t>(after) : nullptr;
    return AC_OK;
}

ac_status ac_workspace_status(const void* workspace, void* stream, uint32_t* detail) {
    if (!workspace) return AC_ERR_INVALID_ARG;
    uint32_t word[2] = {0, 0};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    AC_CUDA_TRY(cudaMemcpyAsync(word, workspace, sizeof(word), cudaMemcpyDeviceToHost, s));
    AC_CUDA_TRY(cudaStreamSynchronize(s));
    if (detail) *detail = word[1];
    return word[0] == 0 ? AC_OK : AC_ERR_TIMEOUT;
}

static inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

size_t ac_host_step_arena_bytes(const ac_conv_desc* desc) {
    Dims d;
    if (make_dims(desc, true, &d) != AC_OK) return 0;
    return up256((size_t)d.x_elems() * d.elt) + up256((size_t)d.z_elems() * d.elt) +
           up256((size_t)d.dy_elems() * d.elt) + up256((size_t)d.dw_elems() * 4) +
           up256(plan_wgrad(d).bytes);
}

ac_status ac_backward_step_host(const ac_conv_desc* desc, const void* x_host, const void* dy_host,
                                float* dw_host, void* z_host, void* arena, size_t arena_bytes,
                                void* stream) {
    Dims d;
    ac_status st = make_dims(desc, true, &d);
    if (st != AC_OK) return st;
    if (!x_host || !dy_host || !dw_host || !arena) return AC_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(arena) & 255u) return AC_ERR_MISALIGNED;
    if (arena_bytes < ac_host_step_arena_bytes(desc)) return AC_ERR_WORKSPACE_TOO_SMALL;
    const size_t xb = (size_t)d.x_elems() * d.elt, zb = (size_t)d.z_elems() * d.elt;
    const size_t gb = (size_t)d.dy_elems() * d.elt, wb = (size_t)d.dw_elems() * 4;
    char* base = static_cast<char*>(arena);
    void* x = base;
    void* z = base + up256(xb);
    void* dy = base + up256(xb) + up256(zb);
    float* dw = reinterpret_cast<float*>(base + up256(xb) + up256(zb) + up256(gb));
    void* ws = base + up256(xb) + up256(zb) + up256(gb) + up256(wb);
    const size_t ws_bytes = plan_wgrad(d).bytes;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    AC_CUDA_TRY(cudaMemcpyAsync(x, x_host, xb, cudaMemcpyHostToDevice, s));
    AC_CUDA_TRY(cudaMemcpyAsync(dy, dy_host, gb, cudaMemcpyHostToDevice, s));
    st = ac_compress(desc, x, z, nullptr, stream);
    if (st != AC_OK) return st;
    st = ac_conv2d_wgrad_compressed(desc, z, dy, dw, ws, ws_bytes, stream);
    if (st != AC_OK) return st;
    AC_CUDA_TRY(cudaMemcpyAsync(dw_host, dw, wb, cudaMemcpyDeviceToHost, s));
    if (z_host) AC_CUDA_TRY(cudaMemcpyAsync(z_host, z, zb, cudaMemcpyDeviceToHost, s));
    return AC_OK;
}

ac_status ac_wgrad_plan_info(const ac_conv_desc* desc, ac_plan_info* info) {
    Dims d;
    if (!info) return AC_ERR_INVALID_ARG;
    ac_status st = make_dims(desc, true, &d);
    if (st != AC_OK) return st;
    *info = ac_plan_info{};
    if (tc2_supported(d, nullptr)) {
        if (staged_inflate_preferred(d)) staged_plan_info(d, info); else tc2_plan_info(d, info);
        return AC_OK;
    }
    if (staged_supported(d)) {
        staged_plan_info(d, info);
        return AC_OK;
    }
    if (gather_supported(d)) {
        gather_plan_info(d, info);
        return AC_OK;
    }
    if (tc_supported(d)) {
        tc_plan_info(d, info);
        return AC_OK;
    }
    const WgradPlan p = plan_wgrad_simt(d);
    const long long J = (long long)d.Ci * d.R * d.S;
    info->splits = p.splits;
    info->ctas = (int32_t)(((J + 63) / 64) * ((d.Co + 63) / 64) * p.splits);
    info->smem_bytes = 0;
    return AC_OK;
}

size_t ac_collapsed_workspace_bytes(const ac_conv_desc* desc, int32_t* tiles_collapsed, int32_t* tiles_dense) {
    Dims d;
    if (make_dims(desc, true, &d) != AC_OK) return 0;
    int tc = 0, td = 0;
    const size_t bytes = tc2_collapsed_workspace_bytes(d, &tc, &td);
    if (bytes && tiles_collapsed) *tiles_collapsed = tc;
    if (bytes && tiles_dense) *tiles_dense = td;
    return bytes;
}

ac_status ac_conv2d_wgrad_compressed_collapsed(const ac_conv_desc* desc, const void* z, const void* dy,
                                               float* dw, void* workspace, size_t workspace_bytes,
                                               void* stream) {
    Dims d;
    ac_status st = make_dims(desc, true, &d);
    if (st != AC_OK) return st;
    if (!z || !dy || !dw || !workspace) return AC_ERR_INVALID_ARG;
    if (!aligned16(z) || !aligned16(dy) || !aligned16(dw) || !aligned16(workspace))
        return AC_ERR_MISALIGNED;
    const size_t need = tc2_collapsed_workspace_bytes(d, nullptr, nullptr);
    if (need == 0) return AC_ERR_UNSUPPORTED;
    if (workspace_bytes < need) return AC_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return launch_wgrad_tc2_collapsed(d, z, dy, dw, workspace, s);
}

ac_status ac_selftest_bounded_wait(void* workspace, uint64_t limit_cycles, void* stream) {
    if (!workspace || limit_cycles == 0 || limit_cycles > (1ull << 32)) return AC_ERR_INVALID_ARG;
    if (!aligned16(workspace)) return AC_ERR_MISALIGNED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    AC_CUDA_TRY(cudaMemsetAsync(workspace, 0, kStatusBlockBytes, s));
    return launch_bounded_wait_selftest(workspace, (long long)limit_cycles, s);
}

const char* ac_status_string(ac_status status) {
    switch (status) {
        case AC_OK: return "AC_OK";
        case AC_ERR_INVALID_ARG: return "AC_ERR_INVALID_ARG";
        case AC_ERR_UNSUPPORTED: return "AC_ERR_UNSUPPORTED";
        case AC_ERR_MISALIGNED: return "AC_ERR_MISALIGNED";
        case AC_ERR_WORKSPACE_TOO_SMALL: return "AC_ERR_WORKSPACE_TOO_SMALL";
        case AC_ERR_CUDA: return "AC_ERR_CUDA";
        case AC_ERR_TIMEOUT: return "AC_ERR_TIMEOUT";
    }
    return "AC_ERR_UNKNOWN";
}

}  // extern "C"
