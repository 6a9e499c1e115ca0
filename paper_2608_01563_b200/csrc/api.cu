// C ABI of the attention library: argument validation, workspace layout, dispatch.
#include <math.h>
#include <stdint.h>

#include <mutex>

#include "../../include/mgn_attn.h"
#include "kernels.h"

namespace mgn {
int g_forced_item_order = -1;
}

namespace {

// Device status word set by kernels whose bounded waits ran out.
__device__ unsigned g_mgn_status;

constexpr int kMaxDevices = 64;
unsigned* g_status_ptr[kMaxDevices];
int g_arch_ok[kMaxDevices];   // 0 unknown, 1 ok, -1 wrong arch
std::mutex g_mu;

cudaEvent_t g_ev_before = nullptr, g_ev_after = nullptr;

struct MainKernelTimer {
    cudaStream_t st;
    explicit MainKernelTimer(cudaStream_t s) : st(s) { if (g_ev_before) cudaEventRecord(g_ev_before, st); }
    ~MainKernelTimer() { if (g_ev_after) cudaEventRecord(g_ev_after, st); }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_common(int B, int H, int S, int D, int causal, float scale, int mode)
{
    if (B <= 0 || H <= 0 || S <= 0 || D <= 0) return MGN_ERR_INVALID_ARG;
    if (causal != 0 && causal != 1) return MGN_ERR_INVALID_ARG;
    if (!isfinite(scale)) return MGN_ERR_INVALID_ARG;
    if (mode != MGN_MODE_STRICT_F32 && mode != MGN_MODE_FAST_BF16) return MGN_ERR_INVALID_ARG;
    if (D != 32 && D != 64 && D != 128) return MGN_ERR_UNSUPPORTED;
    const long long bh = static_cast<long long>(B) * H;
    if (bh > 0x7fffffffLL) return MGN_ERR_UNSUPPORTED;
    if (S > (1 << 24)) return MGN_ERR_UNSUPPORTED;
    // grid and byte-offset plan: tiles*BH must fit an int, element counts must fit 2^40
    if (bh * ((S + 63) / 64) > 0x7fffffffLL) return MGN_ERR_UNSUPPORTED;
    if (static_cast<double>(bh) * S * D > 1.0e12) return MGN_ERR_UNSUPPORTED;
    return MGN_OK;
}

// Extended shapes: separate query/key lengths, grouped key/value heads.
int check_ext(int B, int H, int Hkv, int Sq, int Sk, int D, int causal, float scale, int mode)
{
    if (Hkv <= 0 || Sq <= 0 || Sk <= 0) return MGN_ERR_INVALID_ARG;
    if (int r = check_common(B, H, Sq > Sk ? Sq : Sk, D, causal, scale, mode)) return r;
    if (H % Hkv != 0) return MGN_ERR_INVALID_ARG;
    if (causal && Sq > Sk) return MGN_ERR_UNSUPPORTED;   // a query row would see no key
    return MGN_OK;
}

// Per-device set-up: architecture check and the address of the status word.
int device_setup(unsigned** status)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MGN_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return MGN_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_arch_ok[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MGN_ERR_CUDA;
        if (major != 10) { g_arch_ok[dev] = -1; return MGN_ERR_ARCH; }
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_mgn_status) != cudaSuccess) { cudaGetLastError(); return MGN_ERR_CUDA; }
        g_status_ptr[dev] = static_cast<unsigned*>(p);
        g_arch_ok[dev] = 1;
    }
    if (g_arch_ok[dev] < 0) return MGN_ERR_ARCH;
    *status = g_status_ptr[dev];
    return MGN_OK;
}

}  // namespace
namespace mgn {
int device_status_word(unsigned** status) { return device_setup(status); }
}
namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace layout: [delta: BH*S f32][fast mode only: 256 bytes holding the work-item counter of the
// persistent kernel][fast mode only: dQ accumulator BH*S*D f32], 256-byte granules.
size_t ws_delta_bytes(size_t rows) { return align_up(rows * sizeof(float), 256); }
constexpr size_t kSchedBytes = 256;

}  // namespace
extern "C" size_t mgn_attn_bwd_workspace_bytes(int B, int H, int S, int D, int mode);
namespace {

// Argument checks shared by the backward entry points, in the documented order, then the device set-up.
int check_bwd_call(const void* q, const void* k, const void* v, const void* o, const void* d_o, const float* lse,
                   const void* dq, const void* dk, const void* dv, const void* workspace, size_t workspace_bytes,
                   int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                   unsigned** status)
{
    if (!q || !k || !v || !o || !d_o || !lse || !dq || !dk || !dv) return MGN_ERR_INVALID_ARG;
    if (int r = check_ext(B, H, H_kv, S_q, S_k, D, causal, scale, mode)) return r;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(lse) ||
        !aligned16(dq) || !aligned16(dk) || !aligned16(dv))
        return MGN_ERR_MISALIGNED;
    const size_t need = mgn_attn_bwd_workspace_bytes(B, H, S_q, D, mode);
    if (!workspace || workspace_bytes < need) return MGN_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MGN_ERR_WORKSPACE;
    return device_setup(status);
}

}  // namespace

extern "C" {

size_t mgn_attn_bwd_workspace_bytes(int B, int H, int S, int D, int mode)
{
    if (check_common(B, H, S, D, 0, 1.0f, mode) != MGN_OK) return 0;
    const size_t rows = static_cast<size_t>(B) * H * S;
    size_t bytes = ws_delta_bytes(rows);
    if (mode == MGN_MODE_FAST_BF16) bytes += kSchedBytes + align_up(rows * D * sizeof(float), 256);
    return bytes;
}

int mgn_attn_fwd_ext(const void* q, const void* k, const void* v, void* o, float* lse,
                     int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                     void* stream)
{
    if (!q || !k || !v || !o || !lse) return MGN_ERR_INVALID_ARG;
    if (int r = check_ext(B, H, H_kv, S_q, S_k, D, causal, scale, mode)) return r;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(lse)) return MGN_ERR_MISALIGNED;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    const mgn::Problem p{B, H, H_kv, S_q, S_k, D, causal, scale};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    MainKernelTimer timer(st);
    if (mode == MGN_MODE_STRICT_F32)
        e = mgn::launch_strict_fwd(p, static_cast<const float*>(q), static_cast<const float*>(k),
                                   static_cast<const float*>(v), static_cast<float*>(o), lse, status, st);
    else
        e = mgn::launch_fast_fwd(p, q, k, v, o, lse, status, st);
    return e == cudaSuccess ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
                 int B, int H, int S, int D, int causal, float scale, int mode, void* stream)
{
    return mgn_attn_fwd_ext(q, k, v, o, lse, B, H, H, S, S, D, causal, scale, mode, stream);
}

size_t mgn_attn_fwd_accel_workspace_bytes(int B, int H, int H_kv, int S_q, int S_k, int D)
{
    if (D == 32 || check_ext(B, H, H_kv, S_q, S_k, D, 0, 1.0f, MGN_MODE_FAST_BF16) != MGN_OK) return 0;   // f16 forward: D in {64,128}
    const size_t nq = static_cast<size_t>(B) * H * S_q * D, nk = static_cast<size_t>(B) * H_kv * S_k * D;
    return align_up(nq * 2, 256) + 2 * align_up(nk * 2, 256);
}

int mgn_attn_fwd_accel(const float* q, const float* k, const float* v, float* o, float* lse,
                       void* workspace, size_t workspace_bytes,
                       int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, void* stream)
{
    if (!q || !k || !v || !o || !lse) return MGN_ERR_INVALID_ARG;
    if (int r = check_ext(B, H, H_kv, S_q, S_k, D, causal, scale, MGN_MODE_FAST_BF16)) return r;
    if (D == 32) return MGN_ERR_UNSUPPORTED;   // the f16 forward stores f32 rows itself: D in {64,128}
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(lse)) return MGN_ERR_MISALIGNED;
    const size_t need = mgn_attn_fwd_accel_workspace_bytes(B, H, H_kv, S_q, S_k, D);
    if (!workspace || workspace_bytes < need) return MGN_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MGN_ERR_WORKSPACE;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    const mgn::Problem p{B, H, H_kv, S_q, S_k, D, causal, scale};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t nq = static_cast<size_t>(B) * H * S_q * D, nk = static_cast<size_t>(B) * H_kv * S_k * D;
    char* w = static_cast<char*>(workspace);
    void* q16 = w;
    void* k16 = w + align_up(nq * 2, 256);
    void* v16 = static_cast<char*>(k16) + align_up(nk * 2, 256);
    if (mgn::launch_to_f16(q, q16, nq, st) != cudaSuccess || mgn::launch_to_f16(k, k16, nk, st) != cudaSuccess ||
        mgn::launch_to_f16(v, v16, nk, st) != cudaSuccess)
        return MGN_ERR_CUDA;
    MainKernelTimer timer(st);
    return mgn::launch_fast_fwd_f16(p, q16, k16, v16, o, lse, status, st) == cudaSuccess ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_attn_bwd_ext(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                     const float* lse, void* dq, void* dk, void* dv,
                     void* workspace, size_t workspace_bytes,
                     int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                     void* stream)
{
    unsigned* status = nullptr;
    if (int r = check_bwd_call(q, k, v, o, d_o, lse, dq, dk, dv, workspace, workspace_bytes, B, H, H_kv, S_q, S_k, D,
                               causal, scale, mode, &status))
        return r;

    const mgn::Problem p{B, H, H_kv, S_q, S_k, D, causal, scale};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t rows = static_cast<size_t>(B) * H * S_q;
    float* delta = static_cast<float*>(workspace);
    const bool fast = mode == MGN_MODE_FAST_BF16;

    // delta, and the dQ accumulation target cleared in the same pass (dQ is accumulated by
    // floating-point reductions: in place in strict mode, in an f32 workspace tensor in fast mode)
    unsigned* sched = fast ? reinterpret_cast<unsigned*>(static_cast<char*>(workspace) + ws_delta_bytes(rows)) : nullptr;
    float* dq_acc = fast ? reinterpret_cast<float*>(static_cast<char*>(workspace) + ws_delta_bytes(rows) + kSchedBytes)
                         : static_cast<float*>(dq);
    const bool no_acc = fast && mgn::fast_bwd_writes_dq_directly(p);     // single key block: nothing accumulates
    cudaError_t e = mgn::launch_bwd_preprocess(o, d_o, delta, no_acc ? nullptr : dq_acc, sched, rows, D, fast ? 1 : 0, st);
    if (e != cudaSuccess) return MGN_ERR_CUDA;
    MainKernelTimer timer(st);
    if (!fast)
        e = mgn::launch_strict_bwd(p, static_cast<const float*>(q), static_cast<const float*>(k),
                                   static_cast<const float*>(v), static_cast<const float*>(d_o), lse, delta,
                                   static_cast<float*>(dq), static_cast<float*>(dk), static_cast<float*>(dv), status,
                                   st);
    else
        e = mgn::launch_fast_bwd(p, q, k, v, d_o, lse, delta, dq_acc, dq, dk, dv, sched, status, st);
    return e == cudaSuccess ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_attn_bwd_deterministic(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                               const float* lse, void* dq, void* dk, void* dv,
                               void* workspace, size_t workspace_bytes,
                               int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                               void* stream)
{
    unsigned* status = nullptr;
    if (int r = check_bwd_call(q, k, v, o, d_o, lse, dq, dk, dv, workspace, workspace_bytes, B, H, H_kv, S_q, S_k, D,
                               causal, scale, mode, &status))
        return r;

    const mgn::Problem p{B, H, H_kv, S_q, S_k, D, causal, scale};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t rows = static_cast<size_t>(B) * H * S_q;
    float* delta = static_cast<float*>(workspace);
    const bool fast = mode == MGN_MODE_FAST_BF16;
    unsigned* sched = fast ? reinterpret_cast<unsigned*>(static_cast<char*>(workspace) + ws_delta_bytes(rows)) : nullptr;
    cudaError_t e = mgn::launch_bwd_preprocess(o, d_o, delta, nullptr, sched, rows, D, fast ? 1 : 0, st);
    if (e != cudaSuccess) return MGN_ERR_CUDA;
    MainKernelTimer timer(st);
    if (fast) {
        e = mgn::launch_fast_bwd(p, q, k, v, d_o, lse, delta, nullptr, nullptr, dk, dv, sched, status, st);
        if (e != cudaSuccess) return MGN_ERR_CUDA;
        e = mgn::launch_fast_dq(p, q, k, v, d_o, lse, delta, dq, status, st);
        return e == cudaSuccess ? MGN_OK : MGN_ERR_CUDA;
    }
    e = mgn::launch_strict_bwd(p, static_cast<const float*>(q), static_cast<const float*>(k),
                               static_cast<const float*>(v), static_cast<const float*>(d_o), lse, delta, nullptr,
                               static_cast<float*>(dk), static_cast<float*>(dv), status, st);
    if (e != cudaSuccess) return MGN_ERR_CUDA;
    e = mgn::launch_strict_dq(p, static_cast<const float*>(q), static_cast<const float*>(k),
                              static_cast<const float*>(v), static_cast<const float*>(d_o), lse, delta,
                              static_cast<float*>(dq), status, st);
    return e == cudaSuccess ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_attn_bwd_given_delta(const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                             const float* delta, void* dq, void* dk, void* dv,
                             void* workspace, size_t workspace_bytes,
                             int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                             void* stream)
{
    unsigned* status = nullptr;
    // `o` is not an argument here: delta takes its place in the shared null / alignment checks
    if (int r = check_bwd_call(q, k, v, delta, d_o, lse, dq, dk, dv, workspace, workspace_bytes, B, H, H_kv, S_q, S_k, D,
                               causal, scale, mode, &status))
        return r;
    const mgn::Problem p{B, H, H_kv, S_q, S_k, D, causal, scale};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t rows = static_cast<size_t>(B) * H * S_q;
    const bool fast = mode == MGN_MODE_FAST_BF16;
    unsigned* sched = fast ? reinterpret_cast<unsigned*>(static_cast<char*>(workspace) + ws_delta_bytes(rows)) : nullptr;
    float* dq_acc = fast ? reinterpret_cast<float*>(static_cast<char*>(workspace) + ws_delta_bytes(rows) + kSchedBytes)
                         : static_cast<float*>(dq);
    const bool no_acc = fast && mgn::fast_bwd_writes_dq_directly(p);
    cudaError_t e = mgn::launch_bwd_clear(no_acc ? nullptr : dq_acc, rows * D, sched, st);
    if (e != cudaSuccess) return MGN_ERR_CUDA;
    MainKernelTimer timer(st);
    if (!fast)
        e = mgn::launch_strict_bwd(p, static_cast<const float*>(q), static_cast<const float*>(k),
                                   static_cast<const float*>(v), static_cast<const float*>(d_o), lse, delta,
                                   static_cast<float*>(dq), static_cast<float*>(dk), static_cast<float*>(dv), status,
                                   st);
    else
        e = mgn::launch_fast_bwd(p, q, k, v, d_o, lse, delta, dq_acc, dq, dk, dv, sched, status, st);
    return e == cudaSuccess ? MGN_OK : MGN_ERR_CUDA;
}

namespace {
int check_proj(const void* a, const void* b, const void* c, const void* d, int B, int H, int S, int D, int E, int mode)
{
    if (!a || !b || !c || !d) return MGN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || S <= 0 || D <= 0 || E <= 0) return MGN_ERR_INVALID_ARG;
    if (mode != MGN_MODE_STRICT_F32 && mode != MGN_MODE_FAST_BF16) return MGN_ERR_INVALID_ARG;
    if (mode != MGN_MODE_FAST_BF16) return MGN_ERR_UNSUPPORTED;          // tensor-core path only so far
    if (D != 64 && D != 128) return MGN_ERR_UNSUPPORTED;                 // a 64-wide contraction slice stays inside one head
    if (E % 8 != 0) return MGN_ERR_UNSUPPORTED;                          // 16-byte rows for TMA and the vector stores
    if (static_cast<double>(B) * S * (static_cast<double>(H) * D + E) > 1.0e12 || S > (1 << 24)) return MGN_ERR_UNSUPPORTED;
    if (static_cast<long long>(B) * H > 0x7fffffffLL || static_cast<long long>(H) * D > 0x7fffffffLL) return MGN_ERR_UNSUPPORTED;
    if (!aligned16(a) || !aligned16(b) || !aligned16(c) || !aligned16(d)) return MGN_ERR_MISALIGNED;
    return MGN_OK;
}
}  // namespace

int mgn_out_proj_fwd(const void* o, const void* w, void* y, int B, int H, int S, int D, int E, int mode, void* stream)
{
    if (int r = check_proj(o, w, y, y, B, H, S, D, E, mode)) return r;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    return mgn::launch_out_proj_fwd(o, w, y, B, H, S, D, E, status, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_out_proj_bwd_data(const void* d_y, const void* w, const void* o, void* d_o, float* delta,
                          int B, int H, int S, int D, int E, int mode, void* stream)
{
    if (!delta) return MGN_ERR_INVALID_ARG;
    if (int r = check_proj(d_y, w, o, d_o, B, H, S, D, E, mode)) return r;
    if (!aligned16(delta)) return MGN_ERR_MISALIGNED;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    return mgn::launch_out_proj_bwd_data(d_y, w, o, d_o, delta, B, H, S, D, E, status,
                                         static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_out_proj_bwd_weight(const void* o, const void* d_y, void* d_w, int B, int H, int S, int D, int E, int mode,
                            void* stream)
{
    if (int r = check_proj(o, d_y, d_w, d_w, B, H, S, D, E, mode)) return r;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    return mgn::launch_out_proj_bwd_weight(o, d_y, d_w, B, H, S, D, E, status, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess
               ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_qkv_rope_fwd(const void* x, const void* w, const float* cos_t, const float* sin_t, void* q, void* k, void* v,
                     int B, int S, int E, int H, int H_kv, int D, int mode, void* stream)
{
    if (!cos_t || !sin_t || !k || !v || H_kv <= 0) return MGN_ERR_INVALID_ARG;
    if (int r = check_proj(x, w, q, k, B, H, S, D, E, mode)) return r;
    if (static_cast<long long>(H + 2LL * H_kv) * D > 0x7fffffffLL) return MGN_ERR_UNSUPPORTED;
    if (!aligned16(v) || !aligned16(cos_t) || !aligned16(sin_t)) return MGN_ERR_MISALIGNED;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    return mgn::launch_qkv_rope(x, w, cos_t, sin_t, q, k, v, B, S, E, H, H_kv, D, status,
                                static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_rope_bwd_inplace(void* dq, void* dk, const float* cos_t, const float* sin_t, int B, int H, int H_kv, int S,
                         int D, int mode, void* stream)
{
    if (!cos_t || !sin_t || H_kv <= 0) return MGN_ERR_INVALID_ARG;
    if (int r = check_proj(dq, dk, cos_t, sin_t, B, H, S, D, 8, mode)) return r;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    return mgn::launch_rope_bwd(dq, dk, cos_t, sin_t, B, H, H_kv, S, D, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_qkv_bwd_data(const void* gq, const void* gk, const void* gv, const void* w, void* dx, int B, int S, int E, int H,
                     int H_kv, int D, int mode, void* stream)
{
    if (!gv || H_kv <= 0) return MGN_ERR_INVALID_ARG;
    if (int r = check_proj(gq, gk, w, dx, B, H, S, D, E, mode)) return r;
    if (static_cast<long long>(H + 2LL * H_kv) * D > 0x7fffffffLL) return MGN_ERR_UNSUPPORTED;
    if (!aligned16(gv)) return MGN_ERR_MISALIGNED;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    return mgn::launch_qkv_bwd_data(gq, gk, gv, w, dx, B, S, E, H, H_kv, D, status, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess
               ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_qkv_bwd_weight(const void* gq, const void* gk, const void* gv, const void* x, void* dw, int B, int S, int E,
                       int H, int H_kv, int D, int mode, void* stream)
{
    if (!gv || H_kv <= 0) return MGN_ERR_INVALID_ARG;
    if (int r = check_proj(gq, gk, x, dw, B, H, S, D, E, mode)) return r;
    if (static_cast<long long>(H + 2LL * H_kv) * D > 0x7fffffffLL) return MGN_ERR_UNSUPPORTED;
    if (!aligned16(gv)) return MGN_ERR_MISALIGNED;
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    return mgn::launch_qkv_bwd_weight(gq, gk, gv, x, dw, B, S, E, H, H_kv, D, status,
                                      static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MGN_OK : MGN_ERR_CUDA;
}

int mgn_attn_bwd(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                 const float* lse, void* dq, void* dk, void* dv,
                 void* workspace, size_t workspace_bytes,
                 int B, int H, int S, int D, int causal, float scale, int mode, void* stream)
{
    return mgn_attn_bwd_ext(q, k, v, o, d_o, lse, dq, dk, dv, workspace, workspace_bytes, B, H, H, S, S, D, causal,
                            scale, mode, stream);
}

int mgn_attn_check(void* stream)
{
    unsigned* status = nullptr;
    if (int r = device_setup(&status)) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return MGN_ERR_CUDA;
    unsigned h = 0;
    if (cudaMemcpy(&h, status, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return MGN_ERR_CUDA;
    if (h != 0) {
        cudaMemset(status, 0, sizeof(h));
        return h == 8u ? MGN_ERR_CUDA : MGN_ERR_DEVICE_TIMEOUT;   // 8: a kernel found its shared-memory layout short
    }
    return MGN_OK;
}

int mgn_attn_profile_events(void* before_main, void* after_main)
{
    if ((before_main == nullptr) != (after_main == nullptr)) return MGN_ERR_INVALID_ARG;
    g_ev_before = static_cast<cudaEvent_t>(before_main);
    g_ev_after = static_cast<cudaEvent_t>(after_main);
    return MGN_OK;
}

int mgn_attn_fast_item_order(int order)
{
    if (order < -1 || order > 1) return MGN_ERR_INVALID_ARG;
    mgn::g_forced_item_order = order;
    return MGN_OK;
}

int mgn_attn_strict_tiles(int B, int H, int H_kv, int S_q, int S_k, int D, int causal, int* out)
{
    if (out == nullptr || B <= 0 || H <= 0 || H_kv <= 0 || S_q <= 0 || S_k <= 0 || D <= 0) return MGN_ERR_INVALID_ARG;
    if (H % H_kv != 0 || (causal != 0 && causal != 1)) return MGN_ERR_INVALID_ARG;
    if ((D != 32 && D != 64 && D != 128) || (causal && S_q > S_k)) return MGN_ERR_UNSUPPORTED;
    const mgn::Problem p{B, H, H_kv, S_q, S_k, D, causal, 1.0f};
    mgn::strict_fwd_tiles(p, &out[0], &out[1]);
    mgn::strict_bwd_tiles(p, &out[2], &out[3]);
    return MGN_OK;
}

const char* mgn_status_string(int status)
{
    switch (status) {
        case MGN_OK: return "MGN_OK";
        case MGN_ERR_INVALID_ARG: return "MGN_ERR_INVALID_ARG";
        case MGN_ERR_UNSUPPORTED: return "MGN_ERR_UNSUPPORTED";
        case MGN_ERR_MISALIGNED: return "MGN_ERR_MISALIGNED";
        case MGN_ERR_WORKSPACE: return "MGN_ERR_WORKSPACE";
        case MGN_ERR_CUDA: return "MGN_ERR_CUDA";
        case MGN_ERR_ARCH: return "MGN_ERR_ARCH";
        case MGN_ERR_DEVICE_TIMEOUT: return "MGN_ERR_DEVICE_TIMEOUT";
        default: return "MGN_ERR_UNKNOWN";
    }
}

int mgn_version(void) { return 320; }   // 0.3.2: projections either side of attention, forward and backward, rebuilt fast forward; 0.2.1: tile-shape query, low-padding strict tiles, leaner fast forward (0.2.0: extended shapes, deterministic backward, accelerated forward)

}  // extern "C"
