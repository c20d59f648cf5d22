// Shared device/host helpers of the Swimba CUDA library (sm_100a only).
#pragma once
#include <utility>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/swimba.h"

namespace swimba {

struct TmapCache;

// Kernel ids reported by the optional per-kernel timing (swimba_profile_read).
enum Stage {
    STAGE_ROUTER = 1, STAGE_EXPERT_GEMM = 4,
    STAGE_MIX_SLOTS = 5, STAGE_PROJECT_SIMT = 6, STAGE_SSD_SEQUENTIAL = 7, STAGE_DECODE_UPDATE = 8,
    STAGE_SSD_TILES = 9, STAGE_SEGMENT_SCAN = 10, STAGE_SSD_SCALARS = 11, STAGE_SLOT_STREAMS = 12,
    STAGE_SLOT_SUM = 13, STAGE_PROJECT_SMALL = 14, STAGE_CONV = 15, STAGE_GATED_NORM = 16,
    STAGE_DT_COLUMNS = 17, STAGE_SSD_ADJOINT = 18, STAGE_ROUTER_SOFTMAX = 19, STAGE_DPI_DG = 20,
    STAGE_DW_ROUTER = 21, STAGE_DW_EXPERT = 22, STAGE_ADJOINT_PACK = 23, STAGE_SSD_STATE = 24,
};

constexpr int PROF_MAX = 64;
struct Profiler {
    bool on;
    int n;
    cudaEvent_t ev[2 * PROF_MAX];
    int stage[PROF_MAX];
};

struct LaunchCtx {
    cudaStream_t stream;
    int *d_status;   // device status word (0 = ok, else a SWIMBA_ERR_* code)
    int launches;    // kernels enqueued through this context
    Profiler *prof;  // optional CUDA-event bracket around every kernel
    bool check_indices = false;   // SWIMBA_FLAG_CHECK_INDICES: kernels validate indices they read from memory
    struct TmapCache *tmaps = nullptr;   // the handle's tensor-map cache (may be null)
    void begin(int stage) {
        if (prof && prof->on && prof->n < PROF_MAX) {
            prof->stage[prof->n] = stage;
            cudaEventRecord(prof->ev[2 * prof->n], stream);
        }
    }
    void end() {
        if (prof && prof->on && prof->n < PROF_MAX) {
            cudaEventRecord(prof->ev[2 * prof->n + 1], stream);
            prof->n++;
        }
        launches++;
    }
};

// Programmatic dependent launch.
// A kernel launched with programmatic stream serialization may start while the kernel before it
// in the stream still runs; grid_dep_wait() returns once that kernel has completed and its
// writes are visible (a no-op under an ordinary launch).  grid_dep_launch() lets the next such
// kernel be scheduled as soon as every block of this one has called it.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;"); }

// Kernel launch; overlap = true lets the kernel's prologue run under the tail of the kernel before
// it in the stream (the kernel itself calls grid_dep_wait() before it touches that kernel's data).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t stream, bool overlap, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
__host__ __device__ inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
    return __bfloat162float(v);
}
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}

// Eight consecutive elements starting at a 16-byte (bf16) / 32-byte (float) aligned position.
__device__ __forceinline__ void load8(const float *p, float (&v)[8]) {
    const float4 a = *reinterpret_cast<const float4 *>(p);
    const float4 b = *reinterpret_cast<const float4 *>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8]) {
    const uint4 raw = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);            // low half: element 2i
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); // high half: element 2i+1
    }
}

// The same eight elements as raw registers (so that a load can be issued well before its use) and
// their widening to fp32.
struct Raw8f { float4 a, b; };
struct Raw8h { uint4 a; };
__device__ __forceinline__ void load_raw8(const float *p, Raw8f &r) {
    r.a = *reinterpret_cast<const float4 *>(p);
    r.b = *reinterpret_cast<const float4 *>(p + 4);
}
__device__ __forceinline__ void load_raw8(const __nv_bfloat16 *p, Raw8h &r) {
    r.a = *reinterpret_cast<const uint4 *>(p);
}
__device__ __forceinline__ void unpack8(const Raw8f &r, float (&v)[8]) {
    v[0] = r.a.x; v[1] = r.a.y; v[2] = r.a.z; v[3] = r.a.w;
    v[4] = r.b.x; v[5] = r.b.y; v[6] = r.b.z; v[7] = r.b.w;
}
__device__ __forceinline__ void unpack8(const Raw8h &r, float (&v)[8]) {
    const uint32_t w[4] = {r.a.x, r.a.y, r.a.z, r.a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
template <typename T> struct Raw8;
template <> struct Raw8<float> { typedef Raw8f type; };
template <> struct Raw8<__nv_bfloat16> { typedef Raw8h type; };

// Butterfly sum over the 32 lanes; every lane ends with the same bits.
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// softplus(v) = log(1 + e^v) without overflow.
__device__ __forceinline__ float softplus_f(float v) {
    return fmaxf(v, 0.f) + log1pf(expf(-fabsf(v)));
}

}  // namespace swimba
