// httm_global_attention_static: the HTTM path for callers that must not allocate device memory.
//
// All scratch the path needs between its kernels (plan tables, reordered Q/K/V, assignment maps,
// merged tensors, merged attention output) lives in ONE file-scope device array of fixed size.
// The array's name is only a host-side handle; its device address is looked up once per device
// with cudaGetSymbolAddress and that pointer is what the kernels receive.
#include <algorithm>
#include <cmath>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/httm.h"
#include "httm_internal.h"
#include "httm_plan.h"

namespace httm {
void set_global_error(const std::string& msg);   // defined next to httm_last_error
}
using namespace httm;

namespace {

constexpr size_t kStaticScratchBytes = (size_t)HTTM_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready = false;
    unsigned char* base = nullptr;   // device address of g_static_scratch on this device
    int sm_count = 0;
    // the configuration whose plan tables (pi, pi_inv, block table) the array holds on this device: a call that
    // repeats it uploads nothing
    bool tables_resident = false;
    httm_config resident{};
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_mutex;

struct StaticPlan {   // host copy of the plan of the last geometry (rebuilt when the config changes)
    httm_config cfg{};
    bool valid = false;
    HostPlan plan;
};
StaticPlan g_plan;

int fail(int code, const std::string& msg) {
    set_global_error("httm_global_attention_static: " + msg);
    return code;
}

bool same_config(const httm_config& a, const httm_config& b) {
    return a.frames == b.frames && a.n_camera == b.n_camera && a.n_register == b.n_register && a.grid_h == b.grid_h &&
           a.grid_w == b.grid_w && a.heads == b.heads && a.head_dim == b.head_dim && a.blk_frames == b.blk_frames &&
           a.blk_h == b.blk_h && a.blk_w == b.blk_w && a.ratio_q == b.ratio_q && a.ratio_kv == b.ratio_kv;
}

// The array keeps whatever the previous call left in it.  What the kernels do not rewrite on every
// call is reset here: the status word, and the map entries of the special tokens (never merged).
__global__ void static_reset_kernel(int32_t* status, int32_t* assign_q, int32_t* assign_k, int32_t* rank_q, int n_tokens,
                                    int n_special_total, int heads) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) status[0] = kDevOk;
    if (i < heads * n_special_total) {
        const int h = i / n_special_total, p = i - h * n_special_total;
        const int64_t at = (int64_t)h * n_tokens + p;
        assign_q[at] = p;
        assign_k[at] = p;
        rank_q[at] = p;
    }
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

int check_tensor(const httm_tensor& t, int heads, const char* name) {
    std::string why;
    const int rc = check_tensor_layout(t, heads, name, &why);
    return rc == HTTM_OK ? rc : fail(rc, why);
}

}  // namespace

extern "C" int httm_global_attention_static(const httm_config* cfg, httm_tensor q, httm_tensor k, httm_tensor v,
                                            httm_tensor out, void* cuda_stream) {
    if (!cfg) return fail(HTTM_ERR_INVALID_ARG, "null config");
    {
        std::string why;
        const int rc = check_config(*cfg, &why);
        if (rc != HTTM_OK) return fail(rc, why);
    }
    if (cfg->device < 0 || cfg->device >= kMaxDevices) return fail(HTTM_ERR_INVALID_ARG, "device ordinal out of range");
    const int64_t bf = std::min(cfg->blk_frames, cfg->frames), bh = std::min(cfg->blk_h, cfg->grid_h),
                  bw = std::min(cfg->blk_w, cfg->grid_w);
    if (bf * bh * bw > kMaxBlockTokens) return fail(HTTM_ERR_UNSUPPORTED, "a merging block may hold at most 256 tokens");
    if (cfg->anchor_first_frame != 0) return fail(HTTM_ERR_UNSUPPORTED, "first-frame anchoring needs a context (httm_create)");
    // size check BEFORE any plan is built: an upper bound of the scratch need (merged length <= N)
    const int64_t N64 = (int64_t)cfg->frames * ((int64_t)cfg->n_camera + cfg->n_register + (int64_t)cfg->grid_h * cfg->grid_w);
    const int64_t H = cfg->heads;
    if (N64 > (1 << 22) || H > 65535 || H * N64 * kRowBytes * 3 > (int64_t)kStaticScratchBytes)
        return fail(HTTM_ERR_UNSUPPORTED, "problem needs more than the " + std::to_string(kStaticScratchBytes >> 20) +
                                              " MiB static scratch; use httm_create + httm_global_attention");
    int rc;
    if ((rc = check_tensor(q, cfg->heads, "q")) || (rc = check_tensor(k, cfg->heads, "k")) ||
        (rc = check_tensor(v, cfg->heads, "v")) || (rc = check_tensor(out, cfg->heads, "out")))
        return rc;

    std::lock_guard<std::mutex> lock(g_mutex);
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != cfg->device && cudaSetDevice(cfg->device) != cudaSuccess) {
        cudaGetLastError();
        return fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    }
    struct Restore {
        int prev, dev;
        ~Restore() {
            if (prev >= 0 && prev != dev) cudaSetDevice(prev);
        }
    } restore{prev, cfg->device};

    auto cuda_fail = [&](cudaError_t e, const char* what) {
        cudaGetLastError();
        return fail(HTTM_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
    };
    DeviceSetup& ds = g_setup[cfg->device];
    if (!ds.ready) {   // once per device, with that device current
        cudaDeviceProp prop{};
        cudaError_t e = cudaGetDeviceProperties(&prop, cfg->device);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetDeviceProperties");
        if (prop.major != 10) return fail(HTTM_ERR_UNSUPPORTED, "this library is built for sm_100a only");
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        if ((e = configure_kernels()) != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute");
        ds.base = static_cast<unsigned char*>(p);
        ds.sm_count = prop.multiProcessorCount;
        ds.ready = true;
    }
    if (!g_plan.valid || !same_config(g_plan.cfg, *cfg)) {
        g_plan.valid = false;
        build_host_plan(*cfg, &g_plan.plan);
        g_plan.cfg = *cfg;
        g_plan.valid = true;
    }
    const HostPlan& pl = g_plan.plan;
    const int32_t n_special_total = cfg->frames * pl.n_special;
    const size_t N = pl.n_tokens, Hh = cfg->heads;

    // carve the array
    size_t off = 0;
    auto take = [&](size_t bytes) {
        unsigned char* p = ds.base + off;
        off += align256(bytes);
        return p;
    };
    int32_t* d_status = reinterpret_cast<int32_t*>(take(256));
    int32_t* d_pi = reinterpret_cast<int32_t*>(take(N * 4));
    int32_t* d_pi_inv = reinterpret_cast<int32_t*>(take(N * 4));
    BlockInfo* d_blocks = reinterpret_cast<BlockInfo*>(take(pl.blocks.size() * sizeof(BlockInfo)));
    int32_t* d_aq = reinterpret_cast<int32_t*>(take(Hh * N * 4));
    int32_t* d_ak = reinterpret_cast<int32_t*>(take(Hh * N * 4));
    int32_t* d_rq = reinterpret_cast<int32_t*>(take(Hh * N * 4));
    __nv_bfloat16* d_qr = reinterpret_cast<__nv_bfloat16*>(take(Hh * N * kRowBytes));
    __nv_bfloat16* d_kr = reinterpret_cast<__nv_bfloat16*>(take(Hh * N * kRowBytes));
    __nv_bfloat16* d_vr = reinterpret_cast<__nv_bfloat16*>(take(Hh * N * kRowBytes));
    __nv_bfloat16* d_qm = reinterpret_cast<__nv_bfloat16*>(take(Hh * (size_t)pl.m_q * kRowBytes));
    __nv_bfloat16* d_km = reinterpret_cast<__nv_bfloat16*>(take(Hh * (size_t)pl.m_k * kRowBytes));
    __nv_bfloat16* d_vm = reinterpret_cast<__nv_bfloat16*>(take(Hh * (size_t)pl.m_k * kRowBytes));
    __nv_bfloat16* d_om = reinterpret_cast<__nv_bfloat16*>(take(Hh * (size_t)pl.m_q * kRowBytes));
    if (off > kStaticScratchBytes)
        return fail(HTTM_ERR_UNSUPPORTED, "problem needs " + std::to_string(off) + " bytes of scratch, the static array holds " +
                                              std::to_string(kStaticScratchBytes) + "; use httm_create + httm_global_attention");

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaSuccess;
    if (!ds.tables_resident || !same_config(ds.resident, *cfg)) {
        // The plan tables of another configuration (or none) are in the array: upload this one's, in stream order
        // behind whatever earlier calls enqueued on this stream.  Calls that repeat the resident configuration skip
        // this and enqueue kernels only.
        ds.tables_resident = false;
        e = cudaMemcpyAsync(d_pi, pl.pi.data(), N * 4, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_pi_inv, pl.pi_inv.data(), N * 4, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess && !pl.blocks.empty())
            e = cudaMemcpyAsync(d_blocks, pl.blocks.data(), pl.blocks.size() * sizeof(BlockInfo), cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return cuda_fail(e, "plan upload");
        ds.resident = *cfg;
        ds.tables_resident = true;
    }
    {
        const int threads = 256, work = std::max<int>(1, (int)Hh * n_special_total);
        static_reset_kernel<<<(work + threads - 1) / threads, threads, 0, s>>>(d_status, d_aq, d_ak, d_rq, pl.n_tokens,
                                                                             n_special_total, (int)Hh);
        if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "reset launch");
    }
    auto tv = [](const httm_tensor& t) { return TensorView{reinterpret_cast<const __nv_bfloat16*>(t.ptr), t.stride_head, t.stride_token}; };

    ReorderArgs ra{};
    ra.src[0] = tv(q); ra.src[1] = tv(k); ra.src[2] = tv(v);
    ra.dst[0] = d_qr; ra.dst[1] = d_kr; ra.dst[2] = d_vr;
    ra.pi = d_pi; ra.n_tokens = pl.n_tokens; ra.heads = cfg->heads;
    if ((e = launch_reorder(ra, s)) != cudaSuccess) return cuda_fail(e, "reorder launch");

    MatchArgs ma{};
    ma.xr[0] = d_qr; ma.xr[1] = d_kr; ma.assign[0] = d_aq; ma.assign[1] = d_ak;
    ma.blocks = d_blocks; ma.n_blocks = pl.n_blocks; ma.n_tokens = pl.n_tokens; ma.heads = cfg->heads; ma.status = d_status;
    if ((e = launch_match(ma, pl.max_block, ds.sm_count, s)) != cudaSuccess) return cuda_fail(e, "match launch");

    MergeArgs ga{};
    ga.xr[0] = d_qr; ga.xr[1] = d_kr; ga.xr[2] = d_vr; ga.assign[0] = d_aq; ga.assign[1] = d_ak;
    ga.merged[0] = d_qm; ga.merged[1] = d_km; ga.merged[2] = d_vm; ga.rank_q = d_rq;
    ga.blocks = d_blocks; ga.n_blocks = pl.n_blocks; ga.n_tokens = pl.n_tokens; ga.heads = cfg->heads;
    ga.n_special_total = n_special_total; ga.m_q = pl.m_q; ga.m_k = pl.m_k; ga.status = d_status;
    if ((e = launch_merge(ga, pl.max_block, ds.sm_count, s)) != cudaSuccess) return cuda_fail(e, "merge launch");

    AttentionArgs aa{};
    aa.q = TensorView{d_qm, (int64_t)pl.m_q * kHeadDim, kHeadDim};
    aa.k = TensorView{d_km, (int64_t)pl.m_k * kHeadDim, kHeadDim};
    aa.v = TensorView{d_vm, (int64_t)pl.m_k * kHeadDim, kHeadDim};
    aa.out = d_om; aa.out_stride_head = (int64_t)pl.m_q * kHeadDim; aa.out_stride_token = kHeadDim;
    aa.m_q = pl.m_q; aa.m_k = pl.m_k; aa.heads = cfg->heads;
    aa.scale_log2 = 1.4426950408889634f / std::sqrt((float)kHeadDim);
    aa.status = d_status;
    if ((e = launch_attention(aa, ds.sm_count, s)) != cudaSuccess) return cuda_fail(e, "attention launch");

    UnmergeArgs ua{};
    ua.o_m = d_om; ua.rank_q = d_rq; ua.pi_inv = d_pi_inv; ua.out = reinterpret_cast<__nv_bfloat16*>(out.ptr);
    ua.out_stride_head = out.stride_head; ua.out_stride_token = out.stride_token;
    ua.n_tokens = pl.n_tokens; ua.heads = cfg->heads; ua.m_q = pl.m_q; ua.status = d_status;
    if ((e = launch_unmerge(ua, s)) != cudaSuccess) return cuda_fail(e, "unmerge launch");
    return HTTM_OK;
}
