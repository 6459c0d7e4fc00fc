// Host side of the C ABI declared in include/rd.h: model and session objects, the schedule of one
// prefill / AR step / diffusion-forcing step, and the inspection calls.  Every arithmetic step of
// the path runs in the kernels of rd_kernels.cuh and rd_gemm_tc.cuh; this file only launches them.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <deque>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/rd.h"
#include "rd_attn.cuh"
#include "rd_attn_tc.cuh"
#include "rd_gemm_tc.cuh"
#include "rd_kernels.cuh"

using namespace rd;

// ---------------------------------------------------------------------------------------------
// Error plumbing
// ---------------------------------------------------------------------------------------------
static thread_local char g_cuda_err[320] = "no CUDA error recorded";

static int cuda_fail(cudaError_t e, const char* what, int line) {
    snprintf(g_cuda_err, sizeof g_cuda_err, "%s (%s) at rd_lib.cu:%d: %s", cudaGetErrorName(e), what, line,
             cudaGetErrorString(e));
    return e == cudaErrorMemoryAllocation ? RD_E_OOM : RD_E_CUDA;
}
#define CU(expr)                                                        \
    do {                                                                \
        cudaError_t e_ = (expr);                                        \
        if (e_ != cudaSuccess) return cuda_fail(e_, #expr, __LINE__);   \
    } while (0)
#define RD_TRY(expr)                 \
    do {                             \
        int rc_ = (expr);            \
        if (rc_ != RD_OK) return rc_; \
    } while (0)

extern "C" const char* rd_last_cuda_error(void) { return g_cuda_err; }
extern "C" const char* rd_strerror(int code) {
    switch (code) {
        case RD_OK: return "ok";
        case RD_E_INVALID_ARG: return "invalid argument";
        case RD_E_STATE: return "call out of order for the session's state";
        case RD_E_CAPACITY: return "capacity exceeded (context or window)";
        case RD_E_OOM: return "out of device memory";
        case RD_E_CUDA: return "CUDA error";
        case RD_E_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error code";
    }
}

// Device allocations owned by one object; zero-filled; freed together.
struct DevMem {
    std::vector<void*> ptrs;
    template <typename P> int get(P** out, size_t bytes) {
        void* p = nullptr;
        if (bytes == 0) bytes = 16;
        cudaError_t e = cudaMalloc(&p, bytes);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc", __LINE__);
        e = cudaMemset(p, 0, bytes);
        if (e != cudaSuccess) { cudaFree(p); return cuda_fail(e, "cudaMemset", __LINE__); }
        ptrs.push_back(p);
        *out = reinterpret_cast<P*>(p);
        return RD_OK;
    }
    void release(void* p) {
        for (size_t i = 0; i < ptrs.size(); i++)
            if (ptrs[i] == p) { cudaFree(p); ptrs.erase(ptrs.begin() + i); return; }
    }
    ~DevMem() { for (void* p : ptrs) cudaFree(p); }
};

// ---------------------------------------------------------------------------------------------
// Model
// ---------------------------------------------------------------------------------------------
struct LayerW {
    float* g1 = nullptr; void* wqkv = nullptr; void* wo = nullptr;
    float* g2 = nullptr; void* wgu = nullptr; void* wd = nullptr;
    TcWeight t_qkv, t_o, t_gu, t_d;
};

struct rd_model {
    rd_config cfg;
    int device = 0;
    size_t esz = 4;
    DevMem mem;
    void* emb = nullptr; void* head = nullptr; void* adapter = nullptr;
    float* g_core = nullptr; float* g_final = nullptr;
    std::vector<LayerW> layers[3];
    TcWeight t_adapter, t_head;
    bool tc_ok = false;
    bool gu_interleaved = false;   // gate/up matrices stored with rows interleaved (2j: gate j, 2j+1: up j)
    int n_sms = 148;
};

static int n_layers_of(const rd_config& c, int blk) { return blk == 0 ? c.n_prelude : blk == 1 ? c.n_core : c.n_coda; }

// Copy one source tensor (host or device memory) into `dst`, converting float32 -> bf16 on the
// device when the model stores bf16.
static int put_tensor(rd_model* m, void* dst, const void* src, size_t n, int elem_bytes, float** stage,
                      size_t* stage_n) {
    if (m->esz == (size_t)elem_bytes) {
        CU(cudaMemcpy(dst, src, n * m->esz, cudaMemcpyDefault));
        return RD_OK;
    }
    if (*stage_n < n) {
        if (*stage) { cudaFree(*stage); *stage = nullptr; *stage_n = 0; }
        CU(cudaMalloc((void**)stage, n * sizeof(float)));
        *stage_n = n;
    }
    CU(cudaMemcpy(*stage, src, n * sizeof(float), cudaMemcpyDefault));
    convert_kernel<bf16><<<1024, 256>>>(*stage, (bf16*)dst, n);
    CU(cudaGetLastError());
    CU(cudaDeviceSynchronize());
    return RD_OK;
}

static int load_impl(rd_model* m, const void* const* t, int elem_bytes) {
    const rd_config& c = m->cfg;
    const size_t h = c.hidden, I = c.mlp_inner, V = c.vocab, es = m->esz;
    float* stage = nullptr;
    size_t stage_n = 0;
    int rc = RD_OK;
    int idx = 0;
    void* gu_tmp = nullptr;
    // bf16 models that can take the tensor-core path store gate/up interleaved (hidden % 8 == 0 holds)
    m->gu_interleaved = c.dtype == RD_BF16 && tc_init_driver() == RD_OK;

    auto mat = [&](void* dst, size_t n) -> int { return put_tensor(m, dst, t[idx++], n, elem_bytes, &stage, &stage_n); };
    auto gain = [&](float** dst) -> int {
        RD_TRY(m->mem.get(dst, h * sizeof(float)));
        CU(cudaMemcpy(*dst, t[idx++], h * sizeof(float), cudaMemcpyDefault));
        return RD_OK;
    };
    do {
        if ((rc = m->mem.get(&m->emb, V * h * es))) break;
        if ((rc = mat(m->emb, V * h))) break;
        for (int blk = 0; blk < 3 && !rc; blk++) {
            m->layers[blk].resize(n_layers_of(c, blk));
            for (LayerW& L : m->layers[blk]) {
                if ((rc = gain(&L.g1))) break;
                if ((rc = m->mem.get(&L.wqkv, 3 * h * h * es))) break;
                for (int j = 0; j < 3 && !rc; j++) rc = mat((char*)L.wqkv + j * h * h * es, h * h);
                if (rc) break;
                if ((rc = m->mem.get(&L.wo, h * h * es))) break;
                if ((rc = mat(L.wo, h * h))) break;
                if ((rc = gain(&L.g2))) break;
                if ((rc = m->mem.get(&L.wgu, 2 * I * h * es))) break;
                if (m->gu_interleaved) {
                    // gate and up land in a temporary and are woven row by row into the matrix the
                    // fused tensor-core epilogue wants (one tile then holds both halves of a feature)
                    if (!gu_tmp) {
                        cudaError_t et = cudaMalloc(&gu_tmp, 2 * I * h * es);
                        if (et != cudaSuccess) { rc = cuda_fail(et, "cudaMalloc", __LINE__); break; }
                    }
                    if ((rc = mat(gu_tmp, I * h))) break;
                    if ((rc = mat((char*)gu_tmp + I * h * es, I * h))) break;
                    interleave_rows_kernel<bf16><<<2048, 256>>>((const bf16*)gu_tmp, (const bf16*)gu_tmp + I * h, (bf16*)L.wgu, I, h);
                    cudaError_t ek = cudaGetLastError();
                    if (ek == cudaSuccess) ek = cudaDeviceSynchronize();
                    if (ek != cudaSuccess) { rc = cuda_fail(ek, "interleave_rows_kernel", __LINE__); break; }
                } else {
                    if ((rc = mat(L.wgu, I * h))) break;
                    if ((rc = mat((char*)L.wgu + I * h * es, I * h))) break;
                }
                if ((rc = m->mem.get(&L.wd, h * I * es))) break;
                if ((rc = mat(L.wd, h * I))) break;
            }
        }
        if (rc) break;
        if ((rc = m->mem.get(&m->adapter, 2 * h * h * es))) break;
        if ((rc = mat(m->adapter, 2 * h * h))) break;
        if ((rc = gain(&m->g_core))) break;
        if ((rc = gain(&m->g_final))) break;
        if (c.tie_embeddings) {
            m->head = m->emb;
        } else {
            if ((rc = m->mem.get(&m->head, V * h * es))) break;
            if ((rc = mat(m->head, V * h))) break;
        }
    } while (0);
    if (stage) cudaFree(stage);
    if (gu_tmp) cudaFree(gu_tmp);
    if (rc) return rc;
    // Tensor-core path: TMA descriptors over every weight matrix (bf16 only).
    m->tc_ok = false;
    if (c.dtype == RD_BF16 && tc_init_driver() == RD_OK) {
        bool ok = true;
        for (int blk = 0; blk < 3; blk++)
            for (LayerW& L : m->layers[blk]) {
                ok &= tc_make_weight(&L.t_qkv, L.wqkv, 3 * c.hidden, c.hidden) == RD_OK;
                ok &= tc_make_weight(&L.t_o, L.wo, c.hidden, c.hidden) == RD_OK;
                ok &= tc_make_weight(&L.t_gu, L.wgu, 2 * c.mlp_inner, c.hidden) == RD_OK;
                ok &= tc_make_weight(&L.t_d, L.wd, c.hidden, c.mlp_inner) == RD_OK;
            }
        ok &= tc_make_weight(&m->t_adapter, m->adapter, c.hidden, 2 * c.hidden) == RD_OK;
        ok &= tc_make_weight(&m->t_head, m->head, c.vocab, c.hidden) == RD_OK;
        m->tc_ok = ok;
    }
    return RD_OK;
}

extern "C" int rd_load(const rd_config* cfg, const void* const* tensors, int32_t n_tensors, int32_t elem_bytes,
                       rd_model** out) {
    if (!cfg || !tensors || !out) return RD_E_INVALID_ARG;
    const rd_config& c = *cfg;
    if (c.hidden <= 0 || c.n_heads <= 0 || c.head_dim <= 0 || c.mlp_inner <= 0 || c.vocab <= 0) return RD_E_INVALID_ARG;
    if (c.hidden != c.n_heads * c.head_dim || c.hidden % 8 || c.mlp_inner % 8) return RD_E_INVALID_ARG;
    if (c.head_dim % 2 || c.head_dim > 128 || c.hidden > 12288) return RD_E_INVALID_ARG;
    if (c.n_prelude < 0 || c.n_core < 1 || c.n_coda < 0) return RD_E_INVALID_ARG;
    if (c.dtype != RD_F32 && c.dtype != RD_BF16) return RD_E_INVALID_ARG;
    if (elem_bytes != 4 && !(elem_bytes == 2 && c.dtype == RD_BF16)) return RD_E_INVALID_ARG;
    if (!(c.norm_eps >= 0.f) || !(c.rope_base > 0.f) || !(c.init_sigma >= 0.f)) return RD_E_INVALID_ARG;
    const int want = 1 + 9 * (c.n_prelude + c.n_core + c.n_coda) + 3 + (c.tie_embeddings ? 0 : 1);
    if (n_tensors != want) return RD_E_INVALID_ARG;
    for (int i = 0; i < n_tensors; i++)
        if (!tensors[i]) return RD_E_INVALID_ARG;
    rd_model* m = new (std::nothrow) rd_model();
    if (!m) return RD_E_OOM;
    m->cfg = c;
    m->esz = c.dtype == RD_BF16 ? 2 : 4;
    cudaError_t e = cudaGetDevice(&m->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&m->n_sms, cudaDevAttrMultiProcessorCount, m->device);
    if (e != cudaSuccess) { delete m; return cuda_fail(e, "cudaGetDevice", __LINE__); }
    const int rc = load_impl(m, tensors, elem_bytes);
    if (rc) { delete m; return rc; }
    *out = m;
    return RD_OK;
}
extern "C" void rd_free(rd_model* m) { delete m; }

// ---------------------------------------------------------------------------------------------
// Session
// ---------------------------------------------------------------------------------------------
struct rd_session {
    const rd_model* m = nullptr;
    rd_session_config sc;
    cudaStream_t stream = nullptr;
    DevMem mem;
    int n_slots = 0;   // batch * max_window: decode rows
    int R = 0;         // row capacity of the scratch buffers (>= n_slots; prefill chunk size)
    int tok_stride = 0;
    size_t seq_stride = 0;   // elements between sequences in a cache layer
    size_t head_stride = 0;  // elements between heads of a sequence: cache layout [layer][seq][head][pos][head_dim]
    // device state
    int *tokens = nullptr, *n_prompt = nullptr, *n_committed = nullptr, *win_len = nullptr, *done = nullptr;
    int *row_steps = nullptr, *row_iters = nullptr, *row_pos = nullptr, *row_seq = nullptr;
    int *step_first = nullptr, *step_n = nullptr, *draft = nullptr;
    unsigned long long* counters = nullptr;
    int* status = nullptr;   // device word: non-zero when a bounded wait ran out
    size_t poll_ints = 0;    // status[4], n_committed[B], done[B] are one device block ...
    int* mirror = nullptr;   // ... mirrored in pinned host memory by one copy
    uint64_t enqueue_epoch = 1, mirror_epoch = 0;   // mirror is current while the two are equal
    int* poll_mirror[2] = {nullptr, nullptr};       // pinned copies for rd_poll_begin / rd_poll_end
    cudaEvent_t poll_ev[2] = {nullptr, nullptr};
    bool poll_open[2] = {false, false};
    int poll_next = 0;
    float *x = nullptr, *e = nullptr, *z = nullptr, *z_prev = nullptr;
    float *logits = nullptr, *delta = nullptr, *cos_t = nullptr, *sin_t = nullptr;
    float* tc_scratch = nullptr;   // partial sums of tiles whose K range is shared between CTAs
    size_t tc_scratch_elems = 0;
    float* best_val = nullptr;     // per (row, vocabulary chunk): best score and its index
    int* best_idx = nullptr;
    float *pf_e = nullptr, *pf_s = nullptr;   // prefill workspace: e and the latent of every prompt row, [max_context, h]
    static constexpr int PROMPT_STAGES = 4;   // pinned copies of the prompts being uploaded (the caller's buffer is only borrowed)
    int* prompt_stage[PROMPT_STAGES] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t prompt_ev[PROMPT_STAGES] = {nullptr, nullptr, nullptr, nullptr};
    int stage_next = 0;
    struct PrefillJob { int seq, L, r, pass, c0; };
    std::deque<PrefillJob> jobs;              // sliced prefills (rd_prefill_sliced), oldest first
    int units_per_step = 1;                   // prefill units a step works off before its own kernels
    bool expire_next_wait = false;            // test aid: see rd_debug_expire_next_wait
    float* acc = nullptr;          // output of the plain GEMM kernel, [rows, n_out]
    size_t acc_elems = 0;
    bool fuse_swiglu = true;       // gate/up GEMM on whole tiles with the SwiGLU in its epilogue (tensor-core path)
    bool chained = true;           // launch the step's kernels as a programmatic-dependent-launch chain
    bool pooled = false;        // latent slots drawn from a pool smaller than batch * max_window
    SlotPool pool = {nullptr, nullptr, nullptr};
    int* grp_index = nullptr;   // pooled: per sequence, the slots of its in-flight rows (attention groups)
    const int* att_index = nullptr;   // grp_index during a pooled decode step, null otherwise
    int att_groups = 0;         // attention groups of the pass when they are not n_rows / grp_rows
    int att_blk = 0, att_layer = 0;   // block and layer of the attention launch being enqueued
    int grp_rows = 0;           // rows per attention query group in the current pass
    int ctx_max = 0;            // host-side upper bound of the longest context in the current pass
    std::vector<int> grp_ctx;   // the same bound per attention group (sequence in decode, row block in prefill)
    int attn_path = 0;          // 1: windowed tensor-core attention (bf16, head_dim 64/96/128), K/V by cp.async;
                                // 2: the same fed by TMA through an mbarrier ring (needs the tensor maps below)
    bool att_maps_ok = false, attn_capable = false;
    CUtensorMap q_map64, q_map32;   // the query buffer [rows, hidden] in boxes of 128 rows x 64 / 32 columns
    bool q_maps_ok = false;
    AttMaps att_maps[3];        // per block: boxes of 64 and 32 columns over the K and the V cache
    void *act_h = nullptr, *act_2h = nullptr, *act_i = nullptr, *q_t = nullptr;
    void *Kc[3] = {nullptr, nullptr, nullptr}, *Vc[3] = {nullptr, nullptr, nullptr};
    TcAct t_act_h, t_act_2h, t_act_i;
    // host state
    std::vector<char> prefilled, wave_open;
    std::vector<int> host_prompt_len, host_steps;   // host-side view, for byte accounting only
    int gemm_path = 0;
    rd_stats_t stats;
    // measurement aid: event pairs around GEMM (kind 0) and attention (kind 1) launches
    struct Bracket { cudaEvent_t a, b; int kind; uint64_t bytes; };
    bool profiling = false;
    bool bracket_is_open = false;
    std::vector<Bracket> brackets;
    std::vector<cudaEvent_t> event_pool;
    uint64_t ctx_total = 0;   // host-side upper bound of sum over sequences of context length
    ~rd_session() {
        if (mirror) cudaFreeHost(mirror);
        for (int i = 0; i < 2; i++) {
            if (poll_mirror[i]) cudaFreeHost(poll_mirror[i]);
            if (poll_ev[i]) cudaEventDestroy(poll_ev[i]);
        }
        for (int i = 0; i < PROMPT_STAGES; i++) {
            if (prompt_stage[i]) cudaFreeHost(prompt_stage[i]);
            if (prompt_ev[i]) cudaEventDestroy(prompt_ev[i]);
        }
        for (Bracket& b : brackets) { cudaEventDestroy(b.a); cudaEventDestroy(b.b); }
        for (cudaEvent_t e : event_pool) cudaEventDestroy(e);
    }
};

// RAII-free helpers: open a bracket before a launch, close it after.
static int bracket_open(rd_session* s, int kind, uint64_t bytes) {
    if (!s->profiling || s->brackets.size() >= 32768) return -1;
    rd_session::Bracket b;
    b.kind = kind; b.bytes = bytes;
    for (cudaEvent_t* e : {&b.a, &b.b}) {
        if (!s->event_pool.empty()) { *e = s->event_pool.back(); s->event_pool.pop_back(); }
        else if (cudaEventCreate(e) != cudaSuccess) return -1;
    }
    cudaEventRecord(b.a, s->stream);
    s->brackets.push_back(b);
    s->bracket_is_open = true;
    return (int)s->brackets.size() - 1;
}
static void bracket_close(rd_session* s, int idx) {
    if (idx >= 0) { cudaEventRecord(s->brackets[idx].b, s->stream); s->bracket_is_open = false; }
}
// A launch outside a GEMM or attention bracket gets a bracket of its own (kind 2).
static int bracket_other(rd_session* s) { return s->bracket_is_open ? -1 : bracket_open(s, 2, 0); }

// The GEMM kernels need the largest shared-memory carve-out an SM offers.  Every other kernel of a
// step asks for the same carve-out, so that an SM never has to drain and switch its L1 / shared
// split between two kernels of the chain, and a kernel launched early can share an SM with its
// predecessor.
template <typename F> static void want_max_carveout(F* kern) {
    cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
}
template <typename T> static void want_max_carveout_typed() {
    want_max_carveout(embed_kernel<T>);
    want_max_carveout(rmsnorm_kernel<T, 8>);
    want_max_carveout(rmsnorm_kernel<T, 4>);
    want_max_carveout(rmsnorm_kernel<T, 2>);
    want_max_carveout(concat_kernel<T>);
    want_max_carveout(gemm_simt_kernel<T, 1>);
    want_max_carveout(gemm_simt_kernel<T, 4>);
    want_max_carveout(gemm_simt_kernel<T, 8>);
    want_max_carveout(rope_kv_kernel<T, true>);
    want_max_carveout(rope_kv_kernel<T, false>);
    want_max_carveout(attn_row_kernel<T>);
    want_max_carveout(swiglu_kernel<T>);
}
template <int D> static cudaError_t attn_configure_d() {
    cudaError_t e = cudaSuccess;
    auto set = [&](auto* kern, int smem) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        want_max_carveout(kern);
    };
    set(attn_window_kernel<D, 32, 4>, AttCfg<D, 4>::SMEM);
    set(attn_window_kernel<D, 64, 4>, AttCfg<D, 4>::SMEM);
    set(attn_window_kernel<D, 64, 8>, AttCfg<D, 8>::SMEM);
    set(attn_tma_kernel<D, 32, 4>, AttTmaCfg<D, 4>::SMEM);
    set(attn_tma_kernel<D, 64, 4>, AttTmaCfg<D, 4>::SMEM);
    set(attn_tma_kernel<D, 64, 8>, AttTmaCfg<D, 8>::SMEM);
    set(attn_prefill_tc_kernel<D>, AtcCfg<D>::SMEM);
    return e;
}
// Function attributes (shared-memory opt-in, carve-out preference) are kept per device: they are
// set once for every device a session is created on, with that device current.
constexpr int RD_MAX_DEVICES = 64;
constexpr int ATT_TMA_MIN_ROWS = 8;       // attention groups above this many rows take the TMA-fed kernel
static bool g_device_configured[RD_MAX_DEVICES];
static std::mutex g_device_mutex;
static int configure_device_kernels(int device) {
    if (device < 0 || device >= RD_MAX_DEVICES) return RD_E_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_device_mutex);
    if (g_device_configured[device]) return RD_OK;
    want_max_carveout_typed<float>();
    want_max_carveout_typed<bf16>();
    want_max_carveout(plan_rows_kernel);
    want_max_carveout(fill_rows_kernel);
    want_max_carveout(init_state_kernel);
    want_max_carveout(reduce_store_kernel);
    want_max_carveout(sample_scan_kernel);
    want_max_carveout(sample_pick_kernel);
    want_max_carveout(delta_kernel);
    want_max_carveout(advance_kernel);
    cudaGetLastError();   // a preference a kernel does not take is not an error of the session
    if (tc_configure_device() != RD_OK) return cuda_fail(cudaGetLastError(), "shared-memory opt-in of the GEMM kernels", __LINE__);
    cudaError_t e = attn_configure_d<64>();
    if (e == cudaSuccess) e = attn_configure_d<96>();
    if (e == cudaSuccess) e = attn_configure_d<128>();
    if (e != cudaSuccess) return cuda_fail(e, "shared-memory opt-in of the attention kernels", __LINE__);
    g_device_configured[device] = true;
    return RD_OK;
}

// 2-D bf16 tensor [rows, D] over a K or V cache, box {cols, 64 keys}: 128-byte swizzle for boxes of
// 64 columns, 64-byte swizzle for boxes of 32; elements outside the tensor read as zero.
static int attn_encode(CUtensorMap* map, const void* ptr, unsigned long long rows, int D, int cols) {
    if (!g_encode_tiled) return RD_E_STATE;
    if (((uintptr_t)ptr & 15) != 0 || (D * 2) % 16 != 0) return RD_E_INVALID_ARG;
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    const cuuint32_t box[2] = {(cuuint32_t)cols, (cuuint32_t)ATT_KT};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RD_OK : RD_E_CUDA;
}

// The query buffer [rows, hidden] in boxes of 128 rows x `cols` columns (one head's sub-tile of a group).
static int q_encode(CUtensorMap* map, const void* ptr, unsigned long long rows, int hidden, int cols) {
    if (!g_encode_tiled) return RD_E_STATE;
    if (((uintptr_t)ptr & 15) != 0 || (hidden * 2) % 16 != 0) return RD_E_INVALID_ARG;
    const cuuint64_t dims[2] = {(cuuint64_t)hidden, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)hidden * 2};
    const cuuint32_t box[2] = {(cuuint32_t)cols, (cuuint32_t)ATC_Q};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RD_OK : RD_E_CUDA;
}

extern "C" int rd_session_create(const rd_model* m, const rd_session_config* scp, void* cuda_stream,
                                 rd_session** out) {
    if (!m || !scp || !out) return RD_E_INVALID_ARG;
    const rd_session_config& sc = *scp;
    if (sc.batch < 1 || sc.max_context < 2 || sc.max_window < 1 || sc.max_new_tokens < 0) return RD_E_INVALID_ARG;
    if (sc.max_iters_per_pos < 1 || !(sc.temperature >= 0.f)) return RD_E_INVALID_ARG;
    if (!(sc.eta >= 0.f && sc.eta < 1.f) || !(sc.beta >= 0.f && sc.beta <= 1.f)) return RD_E_INVALID_ARG;
    if (!(sc.top_p >= 0.f && sc.top_p <= 1.f)) return RD_E_INVALID_ARG;
    // the top-p kernel keeps a row's logits in the registers of one cluster
    if (sc.temperature > 0.f && sc.top_p > 0.f && sc.top_p < 1.f && m->cfg.vocab > NUC_MAX_VOCAB) return RD_E_INVALID_ARG;
    if ((long long)sc.batch * sc.max_window > 4096) return RD_E_CAPACITY;
    if (sc.latent_slots < 0 || (long long)sc.latent_slots > (long long)sc.batch * sc.max_window) return RD_E_INVALID_ARG;
    const bool pooled = sc.latent_slots > 0 && sc.latent_slots < sc.batch * sc.max_window;
    if (pooled && sc.batch > 1024) return RD_E_CAPACITY;        // one thread per sequence in the pool's bookkeeping kernel
    {
        int dev = -1;
        CU(cudaGetDevice(&dev));
        if (dev != m->device) return RD_E_STATE;      // the model's device must be current
        RD_TRY(configure_device_kernels(dev));
    }
    rd_session* s = new (std::nothrow) rd_session();
    if (!s) return RD_E_OOM;
    s->m = m;
    s->sc = sc;
    s->stream = (cudaStream_t)cuda_stream;
    memset(&s->stats, 0, sizeof s->stats);
    const rd_config& c = m->cfg;
    const size_t h = c.hidden, I = c.mlp_inner, V = c.vocab, es = m->esz;
    s->pooled = pooled;
    s->n_slots = pooled ? sc.latent_slots : sc.batch * sc.max_window;
    s->R = std::max(s->n_slots, 512);   // prefill chunk: rows that share one pass over the weights
    s->R = (s->R + 15) / 16 * 16;
    s->tok_stride = sc.max_context + 1;
    s->seq_stride = (size_t)sc.max_context * h;
    s->head_stride = (size_t)sc.max_context * c.head_dim;
    const size_t R = s->R, B = sc.batch;
    int rc = RD_OK;
    do {
        if ((rc = s->mem.get(&s->tokens, B * s->tok_stride * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->n_prompt, B * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->win_len, B * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->step_first, B * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->step_n, B * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->row_steps, R * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->row_iters, R * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->row_pos, R * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->row_seq, R * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->draft, R * sizeof(int)))) break;
        if ((rc = s->mem.get(&s->counters, RD_COUNTERS * sizeof(unsigned long long)))) break;
        if (pooled) {
            const size_t ring_n = B * sc.max_window;
            if ((rc = s->mem.get(&s->pool.ring, ring_n * sizeof(int)))) break;
            if ((rc = s->mem.get(&s->pool.free_list, (size_t)s->n_slots * sizeof(int)))) break;
            if ((rc = s->mem.get(&s->pool.free_top, sizeof(int)))) break;
            if ((rc = s->mem.get(&s->grp_index, ring_n * sizeof(int)))) break;
            std::vector<int> minus(ring_n, -1), fl(s->n_slots);
            for (int i = 0; i < s->n_slots; i++) fl[i] = s->n_slots - 1 - i;      // slot 0 is handed out first
            const int top = s->n_slots;
            cudaError_t ep = cudaMemcpy(s->pool.ring, minus.data(), ring_n * sizeof(int), cudaMemcpyHostToDevice);
            if (ep == cudaSuccess) ep = cudaMemcpy(s->pool.free_list, fl.data(), fl.size() * sizeof(int), cudaMemcpyHostToDevice);
            if (ep == cudaSuccess) ep = cudaMemcpy(s->pool.free_top, &top, sizeof(int), cudaMemcpyHostToDevice);
            if (ep != cudaSuccess) { rc = cuda_fail(ep, "slot pool init", __LINE__); break; }
        }
        // what the host polls sits in one block (status word, |y_frozen| and done flag per sequence)
        // so that one copy into a pinned mirror brings all of it
        s->poll_ints = 4 + 2 * B;
        if ((rc = s->mem.get(&s->status, s->poll_ints * sizeof(int)))) break;
        s->n_committed = s->status + 4;
        s->done = s->n_committed + B;
        {
            cudaError_t eh = cudaHostAlloc((void**)&s->mirror, s->poll_ints * sizeof(int), cudaHostAllocDefault);
            if (eh != cudaSuccess) { rc = cuda_fail(eh, "cudaHostAlloc", __LINE__); break; }
        }
        {
            cudaError_t eh = cudaSuccess;
            for (int i = 0; i < rd_session::PROMPT_STAGES && eh == cudaSuccess; i++) {
                eh = cudaHostAlloc((void**)&s->prompt_stage[i], (size_t)s->tok_stride * sizeof(int), cudaHostAllocDefault);
                if (eh == cudaSuccess) eh = cudaEventCreateWithFlags(&s->prompt_ev[i], cudaEventDisableTiming);
            }
            if (eh != cudaSuccess) { rc = cuda_fail(eh, "prompt staging", __LINE__); break; }
        }
        {
            cudaError_t eh = cudaSuccess;
            for (int i = 0; i < 2 && eh == cudaSuccess; i++) {
                eh = cudaHostAlloc((void**)&s->poll_mirror[i], s->poll_ints * sizeof(int), cudaHostAllocDefault);
                if (eh == cudaSuccess) eh = cudaEventCreateWithFlags(&s->poll_ev[i], cudaEventDisableTiming);
            }
            if (eh != cudaSuccess) { rc = cuda_fail(eh, "poll mirrors", __LINE__); break; }
        }
        if ((rc = s->mem.get(&s->pf_e, (size_t)sc.max_context * h * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->pf_s, (size_t)sc.max_context * h * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->x, R * h * sizeof(float)))) break;
        s->acc_elems = std::max(R * std::max<size_t>(std::max<size_t>(3 * h, 2 * I), h), (size_t)s->n_slots * V);
        if ((rc = s->mem.get(&s->acc, s->acc_elems * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->e, R * h * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->z, R * h * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->z_prev, R * h * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->logits, (size_t)s->n_slots * V * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->delta, R * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->best_val, R * SAMPLE_CHUNKS * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->best_idx, R * SAMPLE_CHUNKS * sizeof(int)))) break;
        // GEMM-input buffers hold at least 256 rows so that the widest TMA row box stays inside
        const size_t Ra = std::max<size_t>(R, 256);
        if ((rc = s->mem.get(&s->act_h, Ra * h * es))) break;
        if ((rc = s->mem.get(&s->act_2h, Ra * 2 * h * es))) break;
        if ((rc = s->mem.get(&s->act_i, Ra * I * es))) break;
        if ((rc = s->mem.get(&s->q_t, R * h * es))) break;
        for (int blk = 0; blk < 3 && !rc; blk++) {
            const size_t n = (size_t)n_layers_of(c, blk) * B * s->seq_stride * es;
            if ((rc = s->mem.get(&s->Kc[blk], n))) break;
            rc = s->mem.get(&s->Vc[blk], n);
        }
        if (rc) break;
        // Rotary tables: angle pos * base^(-2i/d), evaluated in double, stored as float32.
        const int half = c.head_dim / 2;
        std::vector<float> ct((size_t)sc.max_context * half), st((size_t)sc.max_context * half);
        for (int p = 0; p < sc.max_context; p++)
            for (int i = 0; i < half; i++) {
                const double ang = (double)p * pow((double)c.rope_base, -2.0 * i / c.head_dim);
                ct[(size_t)p * half + i] = (float)cos(ang);
                st[(size_t)p * half + i] = (float)sin(ang);
            }
        if ((rc = s->mem.get(&s->cos_t, ct.size() * sizeof(float)))) break;
        if ((rc = s->mem.get(&s->sin_t, st.size() * sizeof(float)))) break;
        cudaError_t e = cudaMemcpy(s->cos_t, ct.data(), ct.size() * sizeof(float), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(s->sin_t, st.data(), st.size() * sizeof(float), cudaMemcpyHostToDevice);
        // every sequence starts "done" until it is prefilled
        std::vector<int> ones(B, 1);
        if (e == cudaSuccess) e = cudaMemcpy(s->done, ones.data(), B * sizeof(int), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { rc = cuda_fail(e, "session init copies", __LINE__); break; }
        if (c.dtype == RD_BF16 && (c.head_dim == 64 || c.head_dim == 96 || c.head_dim == 128)) {
            s->attn_path = 1;
            s->attn_capable = true;
            // TMA view of each cache: [layers * sequences * heads * max_context, head_dim], row coordinates stay below 2^31
            bool maps_ok = tc_init_driver() == RD_OK;
            for (int blk = 0; blk < 3 && maps_ok; blk++) {
                const unsigned long long rows = (unsigned long long)n_layers_of(c, blk) * B * c.n_heads * sc.max_context;
                if (rows == 0) continue;
                if (rows + ATT_KT >= (1ull << 31)) { maps_ok = false; break; }
                maps_ok &= attn_encode(&s->att_maps[blk].k64, s->Kc[blk], rows, c.head_dim, 64) == RD_OK;
                maps_ok &= attn_encode(&s->att_maps[blk].v64, s->Vc[blk], rows, c.head_dim, 64) == RD_OK;
                maps_ok &= attn_encode(&s->att_maps[blk].k32, s->Kc[blk], rows, c.head_dim, 32) == RD_OK;
                maps_ok &= attn_encode(&s->att_maps[blk].v32, s->Vc[blk], rows, c.head_dim, 32) == RD_OK;
            }
            s->att_maps_ok = maps_ok;
            if (maps_ok) s->attn_path = 2;
            if (maps_ok) {
                s->q_maps_ok = q_encode(&s->q_map64, s->q_t, R, c.hidden, 64) == RD_OK &&
                               q_encode(&s->q_map32, s->q_t, R, c.hidden, 32) == RD_OK;
                if (s->q_maps_ok) s->attn_path = 3;
            }
        }
        if (m->tc_ok) {
            // scratch for the partial sums: the largest need over the model's GEMM shapes and over
            // the row counts a pass can have (one row-tile class each)
            const int shapes[6][2] = {{c.hidden, 3 * c.hidden}, {c.hidden, c.hidden}, {c.hidden, 2 * c.mlp_inner},
                                      {c.mlp_inner, c.hidden}, {2 * c.hidden, c.hidden}, {c.hidden, c.vocab}};
            size_t need = 16;
            for (int nr = 16; ; nr *= 2) {
                const int rows = std::min<int>(nr, (int)R);
                for (auto& sh : shapes)
                    for (int pair = 0; pair < 2; pair++)     // either choice of rd_set_gemm_path
                        need = std::max(need, tc_plan(sh[0], sh[1], rows, m->n_sms, pair != 0).scratch_elems);
                if (nr >= (int)R) break;
            }
            s->tc_scratch_elems = need;
            if ((rc = s->mem.get(&s->tc_scratch, s->tc_scratch_elems * sizeof(float)))) break;
            bool ok = tc_make_act(&s->t_act_h, s->act_h, (int)Ra, c.hidden) == RD_OK;
            ok &= tc_make_act(&s->t_act_2h, s->act_2h, (int)Ra, 2 * c.hidden) == RD_OK;
            ok &= tc_make_act(&s->t_act_i, s->act_i, (int)Ra, c.mlp_inner) == RD_OK;
            s->gemm_path = ok ? 1 : 0;
        }
    } while (0);
    if (rc) { delete s; return rc; }
    s->prefilled.assign(B, 0);
    s->wave_open.assign(B, 0);
    s->host_prompt_len.assign(B, 0);
    s->host_steps.assign(B, 0);
    *out = s;
    return RD_OK;
}
extern "C" void rd_session_destroy(rd_session* s) {
    if (!s) return;
    cudaStreamSynchronize(s->stream);
    delete s;
}
extern "C" int rd_set_gemm_path(rd_session* s, int32_t path) {
    if (!s || path < 0 || path > 2) return RD_E_INVALID_ARG;
    if (path >= 1 && !(s->m->tc_ok && s->tc_scratch)) return RD_E_STATE;
    s->gemm_path = path;
    return RD_OK;
}

extern "C" int rd_set_attention_path(rd_session* s, int32_t path) {
    if (!s || path < 0 || path > 3) return RD_E_INVALID_ARG;
    if (path >= 1 && !s->attn_capable) return RD_E_STATE;             // no tensor-core attention for this model
    if (path >= 2 && !s->att_maps_ok) return RD_E_STATE;
    if (path == 3 && !s->q_maps_ok) return RD_E_STATE;
    s->attn_path = path;
    return RD_OK;
}

extern "C" int rd_set_fused_swiglu(rd_session* s, int32_t on) {
    if (!s || (on != 0 && on != 1)) return RD_E_INVALID_ARG;
    s->fuse_swiglu = on != 0;
    return RD_OK;
}

extern "C" int rd_set_launch_chaining(rd_session* s, int32_t on) {
    if (!s || (on != 0 && on != 1)) return RD_E_INVALID_ARG;
    s->chained = on != 0;
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// The schedule (templated on the storage type T of weights / KV / GEMM inputs)
// ---------------------------------------------------------------------------------------------
// Every kernel of a step is a link of one programmatic-dependent-launch chain (rd_common.cuh).
#define LAUNCH_CLUSTER(s, kern, grid, block, smem, cluster_x, ...)                                 \
    do {                                                                                          \
        const int br_ = bracket_other(s);                                                         \
        cudaError_t e_ = launch_chained_cluster(kern, dim3 grid, dim3(block), smem, (s)->stream, (s)->chained, cluster_x, __VA_ARGS__); \
        if (e_ != cudaSuccess) return cuda_fail(e_, #kern, __LINE__);                             \
        bracket_close(s, br_);                                                                    \
        (s)->stats.kernel_launches++;                                                             \
    } while (0)
#define LAUNCH(s, kern, grid, block, smem, ...)                                                   \
    do {                                                                                          \
        const int br_ = bracket_other(s);                                                         \
        cudaError_t e_ = launch_chained(kern, dim3(grid), dim3(block), smem, (s)->stream, (s)->chained, __VA_ARGS__); \
        if (e_ != cudaSuccess) return cuda_fail(e_, #kern, __LINE__);                             \
        bracket_close(s, br_);                                                                    \
        (s)->stats.kernel_launches++;                                                             \
    } while (0)

// x = src (+ resid): a residual stream whose last GEMM term has not been added yet.  The kernel
// that reads it next adds the term (rd_partial.cuh).
struct Pending {
    RowSource src;
    const float* resid;
};
static Pending plain_rows(const float* x, size_t ld) {
    Pending p = {};
    p.src.plain = x; p.src.ld = ld; p.resid = nullptr;
    return p;
}

// blocks of 128 threads per row of init_state_kernel: one 4-element group per thread, at most 16
static int init_parts(int hidden) { return std::max(1, std::min(16, ((hidden + 3) / 4 + 127) / 128)); }

template <typename T> struct Eng {
    static bool tc_usable(const rd_session* s, const TcAct* ta, const TcWeight* tw) {
        return sizeof(T) == 2 && s->gemm_path >= 1 && ta && tw && ta->valid && tw->valid;
    }

    // acc[r, o] = sum_k A[r, k] W[o, k]; *out tells the consumer where the sums are: partial sums of
    // the tensor-core kernel, or the finished array s->acc of the plain kernel.
    // With swiglu_out (gate/up projection of a model with interleaved gate/up rows) the tensor-core
    // kernel finishes whole tiles and writes silu(gate) * up itself: *fused tells the caller so.
    static int gemm(rd_session* s, const T* A, size_t lda, const TcAct* ta, const T* W, const TcWeight* tw, int K,
                    int n_out, int n_rows, RowSource* out, T* swiglu_out = nullptr, bool* fused = nullptr) {
        const int br = bracket_open(s, 0, (uint64_t)n_out * K * sizeof(T));
        *out = RowSource{};
        if (fused) *fused = false;
        if (tc_usable(s, ta, tw)) {
            TcParamsFuse fz{(bf16*)swiglu_out, n_out / 2, n_rows, n_out / 2};
            const bool fuse = swiglu_out != nullptr && fused != nullptr && s->m->gu_interleaved && s->fuse_swiglu;
            const int rc = tc_gemm(s->stream, *ta, *tw, K, n_out, n_rows, s->tc_scratch, s->tc_scratch_elems, s->m->n_sms,
                                   s->status, s->chained, &out->part, s->gemm_path == 1, &s->expire_next_wait, fuse ? &fz : nullptr);
            if (rc == RD_OK) {
                if (fuse) *fused = true;
                s->stats.tc_gemm_launches++; s->stats.kernel_launches++;
                bracket_close(s, br);
                return RD_OK;
            }
            if (rc == RD_E_CUDA) return cuda_fail(cudaGetLastError(), "tensor-core GEMM launch", __LINE__);
            if (rc != RD_E_INVALID_ARG) return rc;   // INVALID_ARG: shape not taken, fall through
        }
        if ((size_t)n_rows * n_out > s->acc_elems) return RD_E_CAPACITY;
        float* Y = s->acc;
        const size_t ldy = n_out;
        const float* no_resid = nullptr;
        const int warps = 8;
        dim3 grid((n_out + warps - 1) / warps, 1);
        if (n_rows == 1) {
            LAUNCH(s, (gemm_simt_kernel<T, 1>), grid, warps * 32, 0, A, lda, W, K, n_out, Y, ldy, no_resid, ldy, n_rows);
        } else if (n_rows <= 4) {
            LAUNCH(s, (gemm_simt_kernel<T, 4>), grid, warps * 32, 0, A, lda, W, K, n_out, Y, ldy, no_resid, ldy, n_rows);
        } else {
            grid.y = (n_rows + 7) / 8;
            LAUNCH(s, (gemm_simt_kernel<T, 8>), grid, warps * 32, 0, A, lda, W, K, n_out, Y, ldy, no_resid, ldy, n_rows);
        }
        out->plain = Y; out->ld = ldy;
        bracket_close(s, br);
        return RD_OK;
    }

    // out[row] = RMSNorm(x; g) with x = in.src (+ in.resid); x_store (may be null) receives x.
    template <typename TO>
    static int norm(rd_session* s, const Pending& in, float* x_store, const float* g, TO* out, int n_rows) {
        const int h = s->m->cfg.hidden;
        if (n_rows >= 128) return norm_cl<TO, 2>(s, in, x_store, g, out, n_rows);   // (4-block clusters at 256 rows: no difference in an A/B)
        // one wave of blocks: 8 x 64 blocks of 256 threads do not fit the GPU at once
        if (n_rows > 32) return norm_cl<TO, 4>(s, in, x_store, g, out, n_rows);
        return norm_cl<TO, 8>(s, in, x_store, g, out, n_rows);
    }
    template <typename TO, int CL>
    static int norm_cl(rd_session* s, const Pending& in, float* x_store, const float* g, TO* out, int n_rows) {
        const int h = s->m->cfg.hidden;
        const size_t part = (size_t)((h / 4 + CL - 1) / CL) * 4;
        LAUNCH_CLUSTER(s, (rmsnorm_kernel<TO, CL>), (CL, n_rows), 256, part * sizeof(float), CL, in.src, in.resid,
                       (size_t)h, x_store, (size_t)h, g, h, s->m->cfg.norm_eps, out, (size_t)h, s->row_pos);
        return RD_OK;
    }

    // Windowed flash-decode attention (bf16): groups of s->grp_rows rows share their sequence's KV.
    template <int D, int KW, int NW>
    static int attn_windowed_d(rd_session* s, const bf16* Kc, const bf16* Vc, int n_rows) {
        const rd_config& c = s->m->cfg;
        const int groups = s->att_groups > 0 ? s->att_groups : (n_rows + s->grp_rows - 1) / s->grp_rows;
        const int tiles = std::max(1, (s->ctx_max + ATT_KT - 1) / ATT_KT);
        // enough (group, head, split) blocks for two per SM; a split never gets less than one tile
        int ns = (2 * s->m->n_sms + groups * c.n_heads - 1) / (groups * c.n_heads);
        ns = std::max(1, std::min(std::min(ns, 8), tiles));
        const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)c.head_dim));
        // longest contexts first (s->grp_ctx: the host's bound of each group's context)
        GroupOrder order;
        order.n = 0;
        if (groups > 1 && groups <= ATT_MAX_ORDERED && (int)s->grp_ctx.size() >= groups) {
            int ids[ATT_MAX_ORDERED];
            for (int g = 0; g < groups; g++) ids[g] = g;
            std::stable_sort(ids, ids + groups, [&](int a, int b) { return s->grp_ctx[a] > s->grp_ctx[b]; });
            for (int g = 0; g < groups; g++) order.idx[g] = (unsigned char)ids[g];
            order.n = groups;
        }
        // K/V through the TMA ring for groups of more than 8 rows; smaller groups (the sequential decoder's
        // one row per sequence) do so little arithmetic per tile that the copies' latency is exposed, and the
        // cp.async kernel, whose loads every thread issues, is faster there (110.6 against 98.4 tok/s at 8k keys)
        if (s->attn_path >= 2 && s->grp_rows > ATT_TMA_MIN_ROWS) {
            // Kc points at this layer inside block s->att_blk
            const int row_base = s->att_layer * s->sc.batch * c.n_heads * s->sc.max_context;
            LAUNCH_CLUSTER(s, (attn_tma_kernel<D, KW, NW>), (ns, c.n_heads, groups), 32 * NW, (AttTmaCfg<D, NW>::SMEM), ns,
                           s->att_maps[s->att_blk], order, (const bf16*)s->q_t, s->row_pos, s->row_seq, s->att_index, s->grp_rows, n_rows, row_base,
                           c.n_heads, s->sc.max_context, c.hidden, scale_log2, (bf16*)s->act_h, s->status);
            return RD_OK;
        }
        LAUNCH_CLUSTER(s, (attn_window_kernel<D, KW, NW>), (ns, c.n_heads, groups), 32 * NW, (AttCfg<D, NW>::SMEM), ns, order, (const bf16*)s->q_t,
                       s->row_pos, s->row_seq, s->att_index, s->grp_rows, n_rows, Kc, Vc, s->seq_stride, s->head_stride, c.hidden, scale_log2,
                       (bf16*)s->act_h);
        return RD_OK;
    }
    template <int D>
    static int attn_windowed_k(rd_session* s, const bf16* Kc, const bf16* Vc, int n_rows) {
        // groups of at most 32 rows: every warp takes half of a key tile, so all four warps work;
        // up to 64 rows: four warps of 16 queries; up to 128 rows: eight
        if (s->attn_path == 3 && s->grp_rows == ATC_Q && !s->att_index && s->att_groups == 0) {
            // prefill: 128 consecutive prompt rows per group, both products on tcgen05
            const rd_config& c = s->m->cfg;
            AtcMaps maps;
            maps.q64 = s->q_map64; maps.q32 = s->q_map32; maps.kv = s->att_maps[s->att_blk];
            const int row_base = s->att_layer * s->sc.batch * c.n_heads * s->sc.max_context;
            const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)c.head_dim));
            LAUNCH(s, attn_prefill_tc_kernel<D>, dim3(c.n_heads, (n_rows + ATC_Q - 1) / ATC_Q), ATC_THREADS, (AtcCfg<D>::SMEM), maps,
                   s->row_pos, s->row_seq, n_rows, row_base, c.n_heads, s->sc.max_context, c.hidden, scale_log2, (bf16*)s->act_h, s->status);
            return RD_OK;
        }
        if (s->grp_rows <= 32) return attn_windowed_d<D, 32, 4>(s, Kc, Vc, n_rows);
        if (s->grp_rows <= 64) return attn_windowed_d<D, 64, 4>(s, Kc, Vc, n_rows);
        return attn_windowed_d<D, 64, 8>(s, Kc, Vc, n_rows);
    }
    static int attn_windowed(rd_session* s, const void* Kc, const void* Vc, int n_rows) {
        switch (s->m->cfg.head_dim) {
            case 64: return attn_windowed_k<64>(s, (const bf16*)Kc, (const bf16*)Vc, n_rows);
            case 96: return attn_windowed_k<96>(s, (const bf16*)Kc, (const bf16*)Vc, n_rows);
            case 128: return attn_windowed_k<128>(s, (const bf16*)Kc, (const bf16*)Vc, n_rows);
            default: return RD_E_INVALID_ARG;
        }
    }

    // One transformer layer over the rows of the current row table.  Input x = in.src (+ in.resid);
    // the result is returned pending: x_out = s->x + (down-projection sums), added by whoever reads it.
    static int layer(rd_session* s, int blk, int l, const Pending& in, Pending* out, int n_rows) {
        const rd_config& c = s->m->cfg;
        const LayerW& L = s->m->layers[blk][l];
        const int h = c.hidden, I = c.mlp_inner;
        const size_t layer_off = (size_t)l * s->sc.batch * s->seq_stride;
        T* Kc = (T*)s->Kc[blk] + layer_off;
        T* Vc = (T*)s->Vc[blk] + layer_off;
        // x_in is materialised in s->x unless it already is a finished array
        const bool lazy = in.resid != nullptr || in.src.plain == nullptr;
        RD_TRY(norm<T>(s, in, lazy ? s->x : nullptr, L.g1, (T*)s->act_h, n_rows));
        const float* x_in = lazy ? s->x : in.src.plain;
        RowSource acc;
        RD_TRY(gemm(s, (T*)s->act_h, h, &s->t_act_h, (T*)L.wqkv, &L.t_qkv, h, 3 * h, n_rows, &acc));
        if (n_rows >= 128) {
            LAUNCH(s, (rope_kv_kernel<T, false>), dim3(n_rows, 16), 128, 0, acc, s->row_pos, s->row_seq, s->cos_t, s->sin_t, h, c.head_dim,
                   (T*)s->q_t, Kc, Vc, s->seq_stride, s->head_stride);
        } else {
            LAUNCH(s, (rope_kv_kernel<T, true>), dim3(n_rows, 16), 128, 0, acc, s->row_pos, s->row_seq, s->cos_t, s->sin_t, h, c.head_dim,
                   (T*)s->q_t, Kc, Vc, s->seq_stride, s->head_stride);
        }
        const int br = bracket_open(s, 1, s->ctx_total * 2 * h * sizeof(T));
        bool windowed = false;
        if constexpr (sizeof(T) == 2) {
            if (s->attn_path >= 1 && s->grp_rows >= 1 && s->grp_rows <= ATT_QMAX) {
                s->att_blk = blk; s->att_layer = l;
                RD_TRY(attn_windowed(s, Kc, Vc, n_rows));
                windowed = true;
            }
        }
        if (!windowed) {
            LAUNCH(s, attn_row_kernel<T>, dim3(n_rows, c.n_heads), 128, 0, (T*)s->q_t, s->row_pos, s->row_seq, Kc, Vc,
                   s->seq_stride, s->head_stride, h, c.head_dim, (float)(1.0 / sqrt((double)c.head_dim)), (T*)s->act_h);
        }
        bracket_close(s, br);
        RD_TRY(gemm(s, (T*)s->act_h, h, &s->t_act_h, (T*)L.wo, &L.t_o, h, h, n_rows, &acc));
        Pending mid = {acc, x_in};                      // x_mid = x_in + out-projection, stored in s->x
        RD_TRY(norm<T>(s, mid, s->x, L.g2, (T*)s->act_h, n_rows));
        bool fused = false;
        RD_TRY(gemm(s, (T*)s->act_h, h, &s->t_act_h, (T*)L.wgu, &L.t_gu, h, 2 * I, n_rows, &acc, (T*)s->act_i, &fused));
        if (!fused) {
            const size_t n_q = (size_t)n_rows * (I / 4);
            LAUNCH(s, swiglu_kernel<T>, (unsigned)((n_q + 255) / 256), 256, 0, acc, I, (T*)s->act_i, (size_t)I, n_rows, s->row_pos,
                   s->m->gu_interleaved ? 1 : 0);
        }
        RD_TRY(gemm(s, (T*)s->act_i, I, &s->t_act_i, (T*)L.wd, &L.t_d, I, h, n_rows, &out->src));
        out->resid = s->x;
        return RD_OK;
    }

    // dst[row] = x[row] for a pending x; eta > 0: momentum on rows that have taken a step (see the kernel).
    static int materialise(rd_session* s, const Pending& in, float* dst, int n, int n_rows, float eta = 0.f) {
        const size_t items = (size_t)n_rows * ((n + 3) / 4);
        LAUNCH(s, reduce_store_kernel, (unsigned)((items + 255) / 256), 256, 0, in.src, in.resid, (size_t)n, dst, (size_t)n, n,
               n_rows, s->row_pos, s->row_steps, eta);
        return RD_OK;
    }

    // e_out = P(tokens of the rows): embedding + prelude layers (eta: momentum, decode steps only).
    static int prelude(rd_session* s, int n_rows, float* e_out, float eta = 0.f) {
        const rd_config& c = s->m->cfg;
        const bool via_x = c.n_prelude > 0 || eta > 0.f;
        LAUNCH(s, embed_kernel<T>, dim3(n_rows, 4), 128, 0, s->row_pos, s->row_seq, s->tokens, s->tok_stride,
               (const T*)s->m->emb, c.hidden, via_x ? s->x : e_out);
        if (!via_x) return RD_OK;
        Pending x = plain_rows(s->x, c.hidden);
        for (int l = 0; l < c.n_prelude; l++) {
            Pending y;
            RD_TRY(layer(s, 0, l, x, &y, n_rows));
            x = y;
        }
        return materialise(s, x, e_out, c.hidden, n_rows, eta);
    }

    // z_out = R(e, z_in): adapter over concat(e, z), core layers, closing RMSNorm.
    static int core(rd_session* s, const float* e, const float* z_in, float* z_out, int n_rows) {
        const rd_config& c = s->m->cfg;
        const int h = c.hidden;
        LAUNCH(s, concat_kernel<T>, dim3(n_rows, 8), 128, 0, e, (size_t)h, z_in, (size_t)h, h, (T*)s->act_2h, (size_t)2 * h, s->row_pos);
        Pending x = {};
        RD_TRY(gemm(s, (T*)s->act_2h, 2 * h, &s->t_act_2h, (T*)s->m->adapter, &s->m->t_adapter, 2 * h, h, n_rows, &x.src));
        if (x.src.plain) {
            // finished sums sit in the plain kernel's output buffer, which the next GEMM overwrites
            RD_TRY(materialise(s, x, s->x, h, n_rows));
            x = plain_rows(s->x, h);
        }
        for (int l = 0; l < c.n_core; l++) {
            Pending y;
            RD_TRY(layer(s, 1, l, x, &y, n_rows));
            x = y;
        }
        return norm<float>(s, x, nullptr, s->m->g_core, z_out, n_rows);
    }

    // Coda layers on x = z; with `head`: final RMSNorm, LM head, Sample -> drafts.
    static int coda(rd_session* s, const float* z, int n_rows, bool head) {
        const rd_config& c = s->m->cfg;
        const int h = c.hidden;
        Pending x = plain_rows(z, h);
        for (int l = 0; l < c.n_coda; l++) {
            Pending y;
            RD_TRY(layer(s, 2, l, x, &y, n_rows));
            x = y;
        }
        if (!head) return RD_OK;     // (the last layer's pending sums are not needed: only its K/V were)
        RD_TRY(norm<T>(s, x, nullptr, s->m->g_final, (T*)s->act_h, n_rows));
        RowSource lg;
        RD_TRY(gemm(s, (T*)s->act_h, h, &s->t_act_h, (T*)s->m->head, &s->m->t_head, h, c.vocab, n_rows, &lg));
        if (s->sc.temperature > 0.f && s->sc.top_p > 0.f && s->sc.top_p < 1.f) {
            LAUNCH_CLUSTER(s, sample_nucleus_kernel, (NUC_CLUSTER, n_rows), NUC_THREADS, 0, NUC_CLUSTER, lg, c.vocab, s->row_pos,
                           s->row_seq, s->sc.temperature, s->sc.top_p, s->sc.seed, s->sc.keep_logits ? s->logits : (float*)nullptr,
                           s->draft, s->tokens, s->tok_stride);
            return RD_OK;
        }
        // vocabulary split into at most SAMPLE_CHUNKS runs (multiples of 4) per row
        const int chunk = ((c.vocab + SAMPLE_CHUNKS - 1) / SAMPLE_CHUNKS + 3) / 4 * 4;
        const int n_chunks = (c.vocab + chunk - 1) / chunk;
        LAUNCH(s, sample_scan_kernel, dim3(n_rows, n_chunks), 256, 0, lg, c.vocab, chunk, s->row_pos, s->row_seq,
               s->sc.temperature, s->sc.seed, s->sc.keep_logits ? s->logits : (float*)nullptr, s->best_val, s->best_idx);
        LAUNCH(s, sample_pick_kernel, (n_rows + 63) / 64, 64, 0, s->best_val, s->best_idx, n_chunks, n_rows, s->row_pos,
               s->row_seq, s->draft, s->tokens, s->tok_stride);
        return RD_OK;
    }

    // One sampler step over the decode slots (Algorithm 1 / Algorithm 2; AR is window 1).
    static int decode_step(rd_session* s, int window, int inner, float eps, bool stabilise) {
        const rd_config& c = s->m->cfg;
        const int n = s->n_slots, h = c.hidden, B = s->sc.batch;
        // the leading edge of a wavefront advances by at most one position per step
        s->ctx_total = 0;
        s->ctx_max = 1;
        s->grp_rows = s->sc.max_window;
        s->grp_ctx.assign(B, 0);
        for (int b = 0; b < B; b++)
            if (s->prefilled[b]) {
                s->host_steps[b]++;
                const int ctx = std::min(s->host_prompt_len[b] + s->host_steps[b], s->host_prompt_len[b] + s->sc.max_new_tokens);
                s->ctx_total += ctx;
                s->ctx_max = std::max(s->ctx_max, ctx);
                s->grp_ctx[b] = ctx;
            }
        s->att_index = nullptr;
        s->att_groups = 0;
        if (s->pooled) {
            LAUNCH(s, plan_rows_pool_kernel, 1, 1024, 0, s->n_committed, s->win_len, s->done, B, s->sc.max_window, n, s->pool,
                   s->row_pos, s->row_seq, s->grp_index, s->step_first, s->step_n);
            s->att_index = s->grp_index;
            s->att_groups = B;
        } else {
            LAUNCH(s, plan_rows_kernel, (n + 127) / 128, 128, 0, s->n_committed, s->win_len, s->done, B, s->sc.max_window,
                   s->row_pos, s->row_seq, s->step_first, s->step_n);
        }
        // s_0 for the rows appended by the previous step, and the snapshot z_prev <- z
        // (stabilisers of Section 3.4 apply to sampler steps, not to the sequential decoder)
        const float eta = stabilise ? s->sc.eta : 0.f, beta = stabilise ? s->sc.beta : 0.f;
        const int sched = eps <= 0.f ? window : (s->sc.max_iters_per_pos + inner - 1) / inner;
        LAUNCH(s, init_state_kernel, dim3(n, init_parts(h)), 128, 0, s->row_pos, s->row_seq, s->row_steps, 1, h, c.init_sigma, s->sc.seed, s->z,
               (size_t)h, s->z_prev, beta, sched);
        RD_TRY(prelude(s, n, s->e, eta));
        for (int j = 0; j < inner; j++) RD_TRY(core(s, s->e, s->z, s->z, n));
        RD_TRY(coda(s, s->z, n, true));
        LAUNCH(s, delta_kernel, n, DELTA_THREADS, 0, s->z, s->z_prev, h, s->row_pos, s->delta);
        SeqState st{s->n_prompt, s->n_committed, s->win_len, s->done, s->row_steps, s->row_iters, s->counters};
        if (s->pooled) {
            LAUNCH(s, advance_pool_kernel, 1, (B + 31) / 32 * 32, 3 * B * sizeof(int), st, s->delta, B, s->sc.max_window, window, inner, eps,
                   s->sc.max_iters_per_pos, s->sc.max_new_tokens, c.n_prelude + c.n_coda + inner * c.n_core, s->pool);
        } else {
            LAUNCH(s, advance_kernel, (B + 63) / 64, 64, 0, st, s->delta, B, s->sc.max_window, window, inner, eps,
                   s->sc.max_iters_per_pos, s->sc.max_new_tokens, c.n_prelude + c.n_coda + inner * c.n_core);
        }
        s->att_index = nullptr;
        s->att_groups = 0;
        // every weight matrix is streamed once per pass: prelude, coda and head once, core and adapter `inner` times
        const uint64_t per_layer = 4ull * h * h + 3ull * h * c.mlp_inner;
        s->stats.weight_bytes += ((uint64_t)(c.n_prelude + c.n_coda) * per_layer + (uint64_t)c.vocab * h +
                                  (uint64_t)inner * (c.n_core * per_layer + 2ull * h * h)) * s->m->esz;
        return RD_OK;
    }

    // The GEMM launches of one decode step (inner_iters = 1), in the step's order and launch mode, with
    // nothing between them: prelude layers, adapter, core layers, coda layers, head.  Operands are the
    // session's activation buffers as they stand; the results are not used.  Measurement aid.
    static int gemm_sequence(rd_session* s, int n_rows) {
        const rd_config& c = s->m->cfg;
        const int h = c.hidden, I = c.mlp_inner;
        RowSource acc;
        bool fused = false;
        for (int blk = 0; blk < 3; blk++) {
            if (blk == 1) RD_TRY(gemm(s, (T*)s->act_2h, 2 * h, &s->t_act_2h, (T*)s->m->adapter, &s->m->t_adapter, 2 * h, h, n_rows, &acc));
            for (const LayerW& L : s->m->layers[blk]) {
                RD_TRY(gemm(s, (T*)s->act_h, h, &s->t_act_h, (T*)L.wqkv, &L.t_qkv, h, 3 * h, n_rows, &acc));
                RD_TRY(gemm(s, (T*)s->act_h, h, &s->t_act_h, (T*)L.wo, &L.t_o, h, h, n_rows, &acc));
                RD_TRY(gemm(s, (T*)s->act_h, h, &s->t_act_h, (T*)L.wgu, &L.t_gu, h, 2 * I, n_rows, &acc, (T*)s->act_i, &fused));
                RD_TRY(gemm(s, (T*)s->act_i, I, &s->t_act_i, (T*)L.wd, &L.t_d, I, h, n_rows, &acc));
            }
        }
        return gemm(s, (T*)s->act_h, h, &s->t_act_h, (T*)s->m->head, &s->m->t_head, h, c.vocab, n_rows, &acc);
    }

    // One unit of a prefill: pass `pass` of the chunk of prompt rows that starts at c0.
    // pass 0: P and s_0; passes 1..r: one simultaneous application of R; pass r+1: coda layers (fills
    // the coda cache; no head).  Units must run pass by pass, chunk by chunk: pass i of a row attends
    // the pass-i K/V of the rows before it.
    static int prefill_unit(rd_session* s, int seq, int n, int r, int pass, int c0, float* e_all, float* s_all) {
        const rd_config& c = s->m->cfg;
        const int h = c.hidden;
        const int nr = std::min(s->R, n - c0);
        s->grp_rows = ATT_QMAX;
        s->att_index = nullptr;
        s->att_groups = 0;
        s->ctx_max = c0 + nr;
        s->ctx_total = c0 + nr;
        s->grp_ctx.clear();
        for (int g0 = 0; g0 < nr; g0 += ATT_QMAX) s->grp_ctx.push_back(c0 + std::min(nr, g0 + ATT_QMAX));
        LAUNCH(s, fill_rows_kernel, (s->R + 127) / 128, 128, 0, seq, c0, nr, s->R, s->row_pos, s->row_seq);
        float* ec = e_all + (size_t)c0 * h;    // this chunk's rows of e and of the latent
        float* zc = s_all + (size_t)c0 * h;
        if (pass == 0) {
            RD_TRY(prelude(s, nr, ec));
            LAUNCH(s, init_state_kernel, dim3(nr, init_parts(h)), 128, 0, s->row_pos, s->row_seq, s->row_steps, 0, h, c.init_sigma,
                   s->sc.seed, zc, (size_t)h, (float*)nullptr, 0.f, 1);
            return RD_OK;
        }
        if (pass <= r) return core(s, ec, zc, zc, nr);
        return coda(s, zc, nr, false);
    }

    static int prefill_passes(rd_session* s, int seq, int n, int r, float* e_all, float* s_all) {
        for (int pass = 0; pass < r + 2; pass++)
            for (int c0 = 0; c0 < n; c0 += s->R) RD_TRY(prefill_unit(s, seq, n, r, pass, c0, e_all, s_all));
        return RD_OK;
    }

    // Upload of a prompt through one of the session's pinned copies (the caller's buffer is only borrowed).
    static int upload_prompt(rd_session* s, int seq, const int32_t* prompt, int L) {
        const int buf = s->stage_next;
        CU(cudaEventSynchronize(s->prompt_ev[buf]));      // the upload that last used this copy has finished
        memcpy(s->prompt_stage[buf], prompt, (size_t)L * sizeof(int));
        CU(cudaMemcpyAsync(s->tokens + (size_t)seq * s->tok_stride, s->prompt_stage[buf], (size_t)L * sizeof(int),
                           cudaMemcpyHostToDevice, s->stream));
        CU(cudaEventRecord(s->prompt_ev[buf], s->stream));
        s->stage_next = (buf + 1) % rd_session::PROMPT_STAGES;
        return RD_OK;
    }

    // Sequence state behind a prefill: |y_frozen| = L and one fresh in-flight row at position L-1
    // (stop = true: the sequence is taken out of the steps instead, e.g. while its prompt is prefilled in slices).
    static int start_sequence(rd_session* s, int seq, int L, bool stop) {
        SeqState st{s->n_prompt, s->n_committed, s->win_len, s->done, s->row_steps, s->row_iters, s->counters};
        const int is_done = (stop || s->sc.max_new_tokens <= 0) ? 1 : 0;
        if (s->pooled) {
            LAUNCH(s, seq_start_pool_kernel, 1, 32, 0, st, seq, L, s->sc.max_window, is_done, s->pool);
            return RD_OK;
        }
        const int slot = seq * s->sc.max_window + (L - 1) % s->sc.max_window;
        LAUNCH(s, seq_start_kernel, 1, 32, 0, st, seq, L, slot, is_done);
        return RD_OK;
    }

    // Work on the sliced prefills (rd_prefill_sliced): up to `units` units of the oldest job; a job that
    // finishes starts its sequence.
    static int advance_jobs(rd_session* s, int units) {
        while (units > 0 && !s->jobs.empty()) {
            rd_session::PrefillJob& j = s->jobs.front();
            const int n = j.L - 1;
            if (n > 0 && j.pass < j.r + 2) {
                RD_TRY(prefill_unit(s, j.seq, n, j.r, j.pass, j.c0, s->pf_e, s->pf_s));
                units--;
                j.c0 += s->R;
                if (j.c0 >= n) { j.c0 = 0; j.pass++; }
            }
            if (n <= 0 || j.pass >= j.r + 2) {
                RD_TRY(start_sequence(s, j.seq, j.L, false));
                s->prefilled[j.seq] = 1; s->wave_open[j.seq] = 0;
                s->host_prompt_len[j.seq] = j.L; s->host_steps[j.seq] = 0;
                s->jobs.pop_front();
            }
        }
        return RD_OK;
    }

    // Enqueues the whole prefill on the session's stream and returns: the prompt goes through a pinned
    // copy of its own, e and the latents of the prompt rows live in the session's workspace, and the
    // sequence's state is set by a kernel behind the passes.
    static int prefill(rd_session* s, int seq, const int32_t* prompt, int L, int r) {
        RD_TRY(upload_prompt(s, seq, prompt, L));
        const int n = L - 1;   // rows 0..L-2 are prefilled; L-1 is the first in-flight row
        if (n > 0) RD_TRY(prefill_passes(s, seq, n, r, s->pf_e, s->pf_s));
        return start_sequence(s, seq, L, false);
    }

    // rd_prefill_sliced: the prompt is uploaded and the sequence taken out of the steps now; the passes are
    // worked off by the steps that follow.
    static int prefill_sliced(rd_session* s, int seq, const int32_t* prompt, int L, int r) {
        RD_TRY(upload_prompt(s, seq, prompt, L));
        RD_TRY(start_sequence(s, seq, L, true));
        s->jobs.push_back(rd_session::PrefillJob{seq, L, r, 0, 0});
        return RD_OK;
    }
};

// ---------------------------------------------------------------------------------------------
// C ABI: steps and inspection
// ---------------------------------------------------------------------------------------------
static bool any_prefilled(const rd_session* s) {
    for (char c : s->prefilled) if (c) return true;
    return false;
}

static int prefill_args(const rd_session* s, int32_t seq, const int32_t* prompt, int32_t n_prompt, int32_t r) {
    if (!s || !prompt || seq < 0 || seq >= s->sc.batch || n_prompt < 1 || r < 0) return RD_E_INVALID_ARG;
    if ((long long)n_prompt + s->sc.max_new_tokens > s->sc.max_context) return RD_E_CAPACITY;
    for (int i = 0; i < n_prompt; i++)
        if (prompt[i] < 0 || prompt[i] >= s->m->cfg.vocab) return RD_E_INVALID_ARG;
    return RD_OK;
}

extern "C" int rd_prefill(rd_session* s, int32_t seq, const int32_t* prompt, int32_t n_prompt, int32_t r) {
    RD_TRY(prefill_args(s, seq, prompt, n_prompt, r));
    if (!s->jobs.empty()) return RD_E_STATE;     // the prefill workspace belongs to the sliced jobs
    const int rc = s->m->cfg.dtype == RD_BF16 ? Eng<bf16>::prefill(s, seq, prompt, n_prompt, r)
                                              : Eng<float>::prefill(s, seq, prompt, n_prompt, r);
    s->enqueue_epoch++;
    if (rc == RD_OK) {
        s->prefilled[seq] = 1; s->wave_open[seq] = 0;
        s->host_prompt_len[seq] = n_prompt; s->host_steps[seq] = 0;
    }
    return rc;
}

extern "C" int rd_prefill_sliced(rd_session* s, int32_t seq, const int32_t* prompt, int32_t n_prompt, int32_t r) {
    RD_TRY(prefill_args(s, seq, prompt, n_prompt, r));
    for (const rd_session::PrefillJob& j : s->jobs)
        if (j.seq == seq) return RD_E_STATE;
    const int rc = s->m->cfg.dtype == RD_BF16 ? Eng<bf16>::prefill_sliced(s, seq, prompt, n_prompt, r)
                                              : Eng<float>::prefill_sliced(s, seq, prompt, n_prompt, r);
    s->enqueue_epoch++;
    if (rc == RD_OK) { s->prefilled[seq] = 0; s->wave_open[seq] = 0; }
    return rc;
}

extern "C" int rd_prefill_advance(rd_session* s, int32_t units) {
    if (!s || units < 0) return RD_E_INVALID_ARG;
    if (s->jobs.empty() || units == 0) return RD_OK;
    const int rc = s->m->cfg.dtype == RD_BF16 ? Eng<bf16>::advance_jobs(s, units) : Eng<float>::advance_jobs(s, units);
    s->enqueue_epoch++;
    return rc;
}

extern "C" int rd_prefill_pending(const rd_session* s) {
    return s ? (int)s->jobs.size() : RD_E_INVALID_ARG;
}

extern "C" int rd_set_prefill_units(rd_session* s, int32_t units_per_step) {
    if (!s || units_per_step < 0) return RD_E_INVALID_ARG;
    s->units_per_step = units_per_step;
    return RD_OK;
}

extern "C" int rd_ar_step(rd_session* s, int32_t r) {
    if (!s || r < 1) return RD_E_INVALID_ARG;
    if (!any_prefilled(s) && s->jobs.empty()) return RD_E_STATE;
    for (int b = 0; b < s->sc.batch; b++)
        if (s->prefilled[b] && s->wave_open[b]) return RD_E_STATE;
    RD_TRY(rd_prefill_advance(s, s->units_per_step));
    if (!any_prefilled(s)) return RD_OK;         // only prefill work was due
    const int rc = s->m->cfg.dtype == RD_BF16 ? Eng<bf16>::decode_step(s, 1, r, 0.f, false) : Eng<float>::decode_step(s, 1, r, 0.f, false);
    s->enqueue_epoch++;
    if (rc == RD_OK) s->stats.ar_steps++;
    return rc;
}

extern "C" int rd_df_step(rd_session* s, int32_t window, int32_t inner_iters, float exit_threshold) {
    if (!s || window < 1 || inner_iters < 1 || exit_threshold != exit_threshold) return RD_E_INVALID_ARG;
    if (window > s->sc.max_window) return RD_E_CAPACITY;
    if (!any_prefilled(s) && s->jobs.empty()) return RD_E_STATE;
    RD_TRY(rd_prefill_advance(s, s->units_per_step));
    if (!any_prefilled(s)) return RD_OK;         // only prefill work was due
    const int rc = s->m->cfg.dtype == RD_BF16 ? Eng<bf16>::decode_step(s, window, inner_iters, exit_threshold, true)
                                              : Eng<float>::decode_step(s, window, inner_iters, exit_threshold, true);
    s->enqueue_epoch++;
    if (rc == RD_OK) {
        s->stats.df_steps++;
        if (window > 1)
            for (int b = 0; b < s->sc.batch; b++) if (s->prefilled[b]) s->wave_open[b] = 1;
    }
    return rc;
}

extern "C" int rd_sync(rd_session* s) {
    if (!s) return RD_E_INVALID_ARG;
    if (s->mirror_epoch != s->enqueue_epoch) {
        // one copy behind everything enqueued so far, then one wait
        CU(cudaMemcpyAsync(s->mirror, s->status, s->poll_ints * sizeof(int), cudaMemcpyDeviceToHost, s->stream));
        CU(cudaStreamSynchronize(s->stream));
        s->mirror_epoch = s->enqueue_epoch;
    }
    return s->mirror[0] ? RD_E_TIMEOUT : RD_OK;
}

// Pipelined polling: begin enqueues a copy of the polled block (status word, |y_frozen| and done flag of
// every sequence) behind the steps enqueued so far and returns at once; end waits for that copy only,
// so the host can enqueue the next step before it reads the result of this one.
extern "C" int rd_poll_begin(rd_session* s, int32_t* ticket) {
    if (!s || !ticket) return RD_E_INVALID_ARG;
    const int k = s->poll_next;
    if (s->poll_open[k]) return RD_E_STATE;                 // both tickets are out: end one first
    CU(cudaMemcpyAsync(s->poll_mirror[k], s->status, s->poll_ints * sizeof(int), cudaMemcpyDeviceToHost, s->stream));
    CU(cudaEventRecord(s->poll_ev[k], s->stream));
    s->poll_open[k] = true;
    s->poll_next = k ^ 1;
    *ticket = k;
    return RD_OK;
}
extern "C" int rd_poll_end(rd_session* s, int32_t ticket, int32_t seq, int32_t* n_tokens, int32_t* done) {
    if (!s || ticket < 0 || ticket > 1 || seq < -1 || seq >= s->sc.batch) return RD_E_INVALID_ARG;
    if (!s->poll_open[ticket]) return RD_E_STATE;
    CU(cudaEventSynchronize(s->poll_ev[ticket]));
    const int* m = s->poll_mirror[ticket];
    if (seq < 0) {
        // all sequences: *n_tokens = sum of |y_frozen|, *done = 1 when every prefilled sequence is done
        long long tot = 0;
        int all = 1;
        for (int b = 0; b < s->sc.batch; b++)
            if (s->prefilled[b]) { tot += m[4 + b]; all &= m[4 + s->sc.batch + b] != 0; }
        if (n_tokens) *n_tokens = (int32_t)tot;
        if (done) *done = all;
    } else {
        if (n_tokens) *n_tokens = m[4 + seq];
        if (done) *done = s->prefilled[seq] ? m[4 + s->sc.batch + seq] : 0;
    }
    s->poll_open[ticket] = false;
    return m[0] ? RD_E_TIMEOUT : RD_OK;
}

extern "C" int rd_committed(rd_session* s, int32_t seq, int32_t* n_tokens, int32_t* done) {
    if (!s || seq < 0 || seq >= s->sc.batch) return RD_E_INVALID_ARG;
    RD_TRY(rd_sync(s));
    if (n_tokens) *n_tokens = s->mirror[4 + seq];
    if (done) *done = s->prefilled[seq] ? s->mirror[4 + s->sc.batch + seq] : 0;
    return RD_OK;
}

extern "C" int rd_get_tokens(rd_session* s, int32_t seq, int32_t* dst, int32_t cap, int32_t* n_written) {
    if (!s || !dst || cap < 0 || seq < 0 || seq >= s->sc.batch) return RD_E_INVALID_ARG;
    int n = 0;
    RD_TRY(rd_committed(s, seq, &n, nullptr));
    n = std::min(n, cap);
    if (n > 0) CU(cudaMemcpy(dst, s->tokens + (size_t)seq * s->tok_stride, (size_t)n * sizeof(int), cudaMemcpyDeviceToHost));
    if (n_written) *n_written = n;
    return RD_OK;
}

extern "C" int rd_last_step_rows(rd_session* s, int32_t seq, int32_t* first_pos, int32_t* n_rows) {
    if (!s || seq < 0 || seq >= s->sc.batch) return RD_E_INVALID_ARG;
    if (s->stats.df_steps + s->stats.ar_steps == 0) return RD_E_STATE;
    RD_TRY(rd_sync(s));
    int f = 0, n = 0;
    CU(cudaMemcpy(&f, s->step_first + seq, sizeof(int), cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(&n, s->step_n + seq, sizeof(int), cudaMemcpyDeviceToHost));
    if (first_pos) *first_pos = f;
    if (n_rows) *n_rows = n;
    return RD_OK;
}

extern "C" int rd_debug_read(rd_session* s, int32_t what, int32_t seq, void* dst, size_t bytes) {
    if (!s || !dst) return RD_E_INVALID_ARG;
    int f = 0, n = 0;
    RD_TRY(rd_last_step_rows(s, seq, &f, &n));
    const rd_config& c = s->m->cfg;
    size_t row_bytes = 0;
    const char* base = nullptr;
    switch (what) {
        case RD_DBG_LATENTS: row_bytes = (size_t)c.hidden * 4; base = (const char*)s->z; break;
        case RD_DBG_EMBED: row_bytes = (size_t)c.hidden * 4; base = (const char*)s->e; break;
        case RD_DBG_DELTA: row_bytes = 4; base = (const char*)s->delta; break;
        case RD_DBG_DRAFTS: row_bytes = 4; base = (const char*)s->draft; break;
        case RD_DBG_LOGITS:
            if (!s->sc.keep_logits) return RD_E_STATE;
            row_bytes = (size_t)c.vocab * 4; base = (const char*)s->logits; break;
        default: return RD_E_INVALID_ARG;
    }
    if (bytes < row_bytes * n) return RD_E_INVALID_ARG;
    // pooled slots: the slots of the rows the last step processed, oldest first, as that step's row plan listed them
    std::vector<int> plan;
    if (s->pooled) {
        plan.resize(s->sc.max_window);
        CU(cudaMemcpy(plan.data(), s->grp_index + (size_t)seq * s->sc.max_window, plan.size() * sizeof(int), cudaMemcpyDeviceToHost));
    }
    for (int i = 0; i < n; i++) {
        int slot = seq * s->sc.max_window + (f + i) % s->sc.max_window;
        if (s->pooled) {
            slot = plan[i];
            if (slot < 0 || slot >= s->n_slots) return RD_E_STATE;
        }
        CU(cudaMemcpy((char*)dst + (size_t)i * row_bytes, base + (size_t)slot * row_bytes, row_bytes, cudaMemcpyDeviceToHost));
    }
    return RD_OK;
}

extern "C" int rd_debug_force_tokens(rd_session* s, int32_t seq, int32_t first_pos, const int32_t* tokens, int32_t n) {
    if (!s || !tokens || seq < 0 || seq >= s->sc.batch || n < 0 || !s->prefilled[seq]) return RD_E_INVALID_ARG;
    RD_TRY(rd_sync(s));
    int np = 0;
    CU(cudaMemcpy(&np, s->n_prompt + seq, sizeof(int), cudaMemcpyDeviceToHost));
    if (first_pos < np || (long long)first_pos + n > s->tok_stride) return RD_E_INVALID_ARG;
    for (int i = 0; i < n; i++)
        if (tokens[i] < 0 || tokens[i] >= s->m->cfg.vocab) return RD_E_INVALID_ARG;
    if (n) CU(cudaMemcpy(s->tokens + (size_t)seq * s->tok_stride + first_pos, tokens, (size_t)n * sizeof(int), cudaMemcpyHostToDevice));
    return RD_OK;
}

extern "C" int rd_debug_read_kv(rd_session* s, int32_t block, int32_t layer, int32_t which, int32_t seq, int32_t pos0,
                                int32_t n, float* dst) {
    if (!s || !dst || block < 0 || block > 2 || (which != 0 && which != 1) || seq < 0 || seq >= s->sc.batch) return RD_E_INVALID_ARG;
    const rd_config& c = s->m->cfg;
    if (layer < 0 || layer >= n_layers_of(c, block) || pos0 < 0 || n < 0 || pos0 > s->sc.max_context || n > s->sc.max_context - pos0) return RD_E_INVALID_ARG;
    RD_TRY(rd_sync(s));
    if (n == 0) return RD_OK;
    const size_t off = ((size_t)layer * s->sc.batch + seq) * s->seq_stride;
    const size_t cnt = (size_t)n * c.hidden;
    const char* src = (const char*)(which ? s->Vc[block] : s->Kc[block]) + off * s->m->esz;
    float* tmp = nullptr;
    CU(cudaMalloc((void**)&tmp, cnt * 4));
    if (c.dtype == RD_F32)
        kv_gather_kernel<float><<<256, 256, 0, s->stream>>>((const float*)src, s->head_stride, c.head_dim, c.hidden, pos0, n, tmp);
    else
        kv_gather_kernel<bf16><<<256, 256, 0, s->stream>>>((const bf16*)src, s->head_stride, c.head_dim, c.hidden, pos0, n, tmp);
    cudaError_t e = cudaStreamSynchronize(s->stream);
    if (e == cudaSuccess) e = cudaMemcpy(dst, tmp, cnt * 4, cudaMemcpyDeviceToHost);
    cudaFree(tmp);
    if (e != cudaSuccess) return cuda_fail(e, "read_kv", __LINE__);
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// rd_debug_read_kv_noalloc: the K/V read-out without any allocation.
//
// rd_debug_read_kv gathers cache rows into float32 [n, hidden] in a temporary device buffer that it obtains
// from cudaMalloc and returns with cudaFree.  Here the temporary is a fixed array that is part of
// the library image: every device that loads the library holds RD_KV_STAGE_ELEMS floats (4 MiB)
// until the process exits.  In host code `g_kv_stage` is only a handle for the runtime, not an
// address a kernel can use; the address on a given device comes from cudaGetSymbolAddress, asked
// once per device with that device current and remembered in g_kv_stage_dev.
// ---------------------------------------------------------------------------------------------
constexpr size_t RD_KV_STAGE_ELEMS = (size_t)1 << 20;
static __device__ __align__(256) float g_kv_stage[RD_KV_STAGE_ELEMS];
static float* g_kv_stage_dev[RD_MAX_DEVICES];
static std::mutex g_kv_stage_mutex;

// Device address of g_kv_stage on the current device (which must be `device`).
static int kv_stage_address(int device, float** out) {
    if (device < 0 || device >= RD_MAX_DEVICES) return RD_E_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_kv_stage_mutex);
    if (!g_kv_stage_dev[device]) {
        float* p = nullptr;
        CU(cudaGetSymbolAddress((void**)&p, g_kv_stage));
        if (!p) return RD_E_CUDA;
        g_kv_stage_dev[device] = p;
    }
    *out = g_kv_stage_dev[device];
    return RD_OK;
}

extern "C" int rd_debug_read_kv_noalloc(rd_session* s, int32_t block, int32_t layer, int32_t which, int32_t seq,
                                        int32_t pos0, int32_t n, float* dst) {
    if (!s || !dst || block < 0 || block > 2 || (which != 0 && which != 1) || seq < 0 || seq >= s->sc.batch) return RD_E_INVALID_ARG;
    const rd_config& c = s->m->cfg;
    if (layer < 0 || layer >= n_layers_of(c, block) || pos0 < 0 || n < 0 || pos0 > s->sc.max_context || n > s->sc.max_context - pos0) return RD_E_INVALID_ARG;
    const size_t cnt = (size_t)n * c.hidden;
    if (cnt > RD_KV_STAGE_ELEMS) {
        snprintf(g_cuda_err, sizeof g_cuda_err,
                 "rd_debug_read_kv_noalloc: %zu values asked for, the fixed staging array holds %zu (n * hidden too large)",
                 cnt, RD_KV_STAGE_ELEMS);
        return RD_E_CAPACITY;
    }
    int dev = -1;
    CU(cudaGetDevice(&dev));
    if (dev != s->m->device) return RD_E_STATE;   // the session's device must be current
    RD_TRY(rd_sync(s));
    if (n == 0) return RD_OK;
    const size_t off = ((size_t)layer * s->sc.batch + seq) * s->seq_stride;
    const char* src = (const char*)(which ? s->Vc[block] : s->Kc[block]) + off * s->m->esz;
    float* stage = nullptr;
    RD_TRY(kv_stage_address(dev, &stage));
    // every element of stage[0..cnt) is overwritten: nothing of an earlier call can show through
    if (c.dtype == RD_F32)
        kv_gather_kernel<float><<<256, 256, 0, s->stream>>>((const float*)src, s->head_stride, c.head_dim, c.hidden, pos0, n, stage);
    else
        kv_gather_kernel<bf16><<<256, 256, 0, s->stream>>>((const bf16*)src, s->head_stride, c.head_dim, c.hidden, pos0, n, stage);
    CU(cudaGetLastError());
    CU(cudaStreamSynchronize(s->stream));
    CU(cudaMemcpy(dst, stage, cnt * 4, cudaMemcpyDeviceToHost));
    return RD_OK;
}

extern "C" int rd_stats(rd_session* s, rd_stats_t* out) {
    if (!s || !out) return RD_E_INVALID_ARG;
    RD_TRY(rd_sync(s));
    unsigned long long cnt[RD_COUNTERS];
    CU(cudaMemcpy(cnt, s->counters, sizeof cnt, cudaMemcpyDeviceToHost));
    *out = s->stats;
    out->rows_prelude = cnt[0];
    out->rows_core = cnt[1];
    out->rows_coda = cnt[2];
    out->tokens_committed = cnt[3];
    const rd_config& c = s->m->cfg;
    const uint64_t h = c.hidden, per_layer = 4 * h * h + 3 * h * (uint64_t)c.mlp_inner;
    const uint64_t rows_written = cnt[0] * c.n_prelude + cnt[1] * c.n_core + cnt[2] * c.n_coda;
    out->kv_bytes = (cnt[4] + rows_written) * 2 * h * s->m->esz;
    out->flops = 2 * (cnt[0] * c.n_prelude * per_layer + cnt[1] * (c.n_core * per_layer + 2 * h * h) +
                      cnt[2] * (c.n_coda * per_layer + (uint64_t)c.vocab * h)) + 4 * h * cnt[5];
    for (int k = 0; k < RD_HIST_BINS; k++) out->commit_hist[k] = cnt[RD_HIST_AT + k];
    return RD_OK;
}

extern "C" int rd_debug_expire_next_wait(rd_session* s) {
    if (!s) return RD_E_INVALID_ARG;
    if (!(s->gemm_path >= 1 && s->m->tc_ok && s->tc_scratch)) return RD_E_STATE;
    s->expire_next_wait = true;
    return RD_OK;
}

extern "C" int rd_debug_gemm_sequence(rd_session* s, int32_t n_rows, int32_t reps, uint64_t* weight_bytes, int32_t* launches) {
    if (!s || n_rows < 1 || n_rows > s->R || reps < 1) return RD_E_INVALID_ARG;
    if (s->m->cfg.dtype != RD_BF16 || s->gemm_path < 1 || !s->m->tc_ok) return RD_E_STATE;
    const rd_config& c = s->m->cfg;
    const uint64_t h = c.hidden, per_layer = 4 * h * h + 3 * h * (uint64_t)c.mlp_inner;
    const int n_layers = c.n_prelude + c.n_core + c.n_coda;
    for (int i = 0; i < reps; i++) RD_TRY(Eng<bf16>::gemm_sequence(s, n_rows));
    s->enqueue_epoch++;
    if (weight_bytes) *weight_bytes = (uint64_t)reps * (n_layers * per_layer + 2 * h * h + (uint64_t)c.vocab * h) * s->m->esz;
    if (launches) *launches = reps * (4 * n_layers + 2);
    return RD_OK;
}

extern "C" int rd_profile_enable(rd_session* s, int32_t on) {
    if (!s) return RD_E_INVALID_ARG;
    s->profiling = on != 0;
    return RD_OK;
}

extern "C" int rd_profile_read(rd_session* s, rd_profile_t* out) {
    if (!s || !out) return RD_E_INVALID_ARG;
    RD_TRY(rd_sync(s));
    memset(out, 0, sizeof *out);
    for (rd_session::Bracket& b : s->brackets) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, b.a, b.b) == cudaSuccess) {
            if (b.kind == 0) { out->gemm_launches++; out->gemm_ms += ms; out->gemm_weight_bytes += b.bytes; }
            else if (b.kind == 1) { out->attn_launches++; out->attn_ms += ms; out->attn_kv_bytes += b.bytes; }
            else { out->other_launches++; out->other_ms += ms; }
        }
        s->event_pool.push_back(b.a);
        s->event_pool.push_back(b.b);
    }
    s->brackets.clear();
    return RD_OK;
}
