// Host side of the C ABI declared in include/demo.h: context, planner (chunk tables of the blocking
// operator, payload offsets, DCT basis), pointer-table caching and kernel dispatch.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/demo.h"
#include "demo_internal.h"

struct demo_ctx {
    demo_config cfg;
    int device = 0;
    int sm_count = 0;
    int n_tensors = 0;
    int path = DEMO_PATH_AUTO;
    float alpha = 1.0f;  // momentum-subtraction coefficient
    int aggregation = DEMO_AGG_SUM, phi = DEMO_PHI_SIGN;
    long long launches = 0;
    std::vector<demo_tensor_desc> descs;
    std::vector<long long> first_record, n_chunks, n_elems;
    std::vector<int> k_eff;
    long long total_records = 0;

    // work lists
    int n2d = 0, n1d = 0;
    long long chunks2d = 0, chunks1d = 0;
    DemoTensorEntry *d_entries2d = nullptr, *d_entries1d = nullptr;

    float *d_C = nullptr;
    int *d_status = nullptr;

    // contexts made by demo_init_nd: one work list of rectangular chunks of any order, the DCT matrices
    // of every chunk extent in one table; the square-chunk lists above stay empty
    bool nd = false;
    int n_nd = 0, max_M = 0;
    long long chunks_nd = 0;
    DemoNdEntry *d_entries_nd = nullptr;
    float *d_tables = nullptr;

    // caller-supplied orthonormal basis (rows = basis vectors); while `custom_basis` is set every
    // tensor goes through the dense-transform kernels, which read the basis from memory
    float *d_P = nullptr, *d_P_stage = nullptr;  // [s*s], [2*s*s]
    int *d_basis_flag = nullptr;
    bool custom_basis = false;
    bool momentum_dct = false;  // demo_set_momentum_domain(DEMO_MOMENTUM_DCT)

    // device pointer tables and their host mirrors (uploaded only when the caller's pointers change)
    const void **d_g = nullptr;      // [W][T]
    float **d_m = nullptr;           // [W][T]
    float **d_x = nullptr;           // [T]
    const DemoRecord **d_p = nullptr;  // [W]
    signed char **d_s = nullptr;       // [T] sign tensors of the parameter-server form
    std::vector<signed char *> h_s;
    bool s_valid = false;
    DemoFlatEntry *d_flat = nullptr;   // [T] element ranges for demo_apply_signs
    long long n_quads = 0;
    std::vector<const void *> h_g;
    std::vector<float *> h_m, h_x;
    std::vector<const DemoRecord *> h_p;
    std::vector<char> g_valid, m_valid;  // per worker
    bool x_valid = false, p_valid = false;

    // TMA tensor maps for the fast kernels (2-D tensors; box = one s x s tile), rebuilt whenever
    // the caller's pointers change.  NULL when the driver entry point is unavailable.
    PFN_cuTensorMapEncodeTiled encode = nullptr;
    CUtensorMap *d_tm_g = nullptr, *d_tm_m = nullptr;  // [W][T]
    CUtensorMap *d_tm_x = nullptr;                     // [T]
    std::vector<CUtensorMap> h_tm;                     // staging, [T]

    // The small kernel of the 1-D tensors runs on a side stream beside the kernel of the 2-D tensors
    // (fork / join by events; also legal inside a stream capture).  NULL: both on the caller's stream.
    cudaStream_t side_stream = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;

    // demo_step_host: host->device gradient copies run on their own stream so that the copy of worker
    // w+1 overlaps the compress of worker w (created on first use)
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_start = nullptr;
    std::vector<cudaEvent_t> ev_copied;  // [W]
};

static_assert(DEMO_ND_DIMS == DEMO_ND_MAX_DIMS, "public and internal axis limits disagree");

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

// Upload `n` pointers to dev[0..n) if they differ from the mirror.  The mirror is pageable host
// memory: cudaMemcpyAsync stages it before returning, so it may be overwritten by the next call.
template <typename T>
cudaError_t sync_table(T *dev, T *mirror, const T *now, int n, bool *valid, cudaStream_t stream,
                       bool *changed = nullptr)
{
    if (changed) *changed = false;
    if (*valid && std::memcmp(mirror, now, sizeof(T) * (size_t)n) == 0) return cudaSuccess;
    if (changed) *changed = true;
    std::memcpy(mirror, now, sizeof(T) * (size_t)n);
    cudaError_t err = cudaMemcpyAsync(dev, mirror, sizeof(T) * (size_t)n, cudaMemcpyHostToDevice, stream);
    *valid = (err == cudaSuccess);
    return err;
}

// Encode one tensor map per 2-D tensor (box = s x s tile of `elem`-byte elements) for the given base
// pointers and upload them to dev[0..T).  Returns false if the driver rejects a descriptor.
template <typename P>
bool upload_tensor_maps(demo_ctx *c, CUtensorMap *dev, const P *ptrs, bool bf16, cudaStream_t stream)
{
    const int T = c->n_tensors, s = c->cfg.chunk;
    std::memset(c->h_tm.data(), 0, sizeof(CUtensorMap) * (size_t)T);
    for (int t = 0; t < T; ++t) {
        const demo_tensor_desc &d = c->descs[t];
        if (d.ndim != 2) continue;
        const cuuint64_t elem = bf16 ? 2 : 4;
        const cuuint64_t gdim[2] = {(cuuint64_t)d.shape[1], (cuuint64_t)d.shape[0]};
        const cuuint64_t gstride[1] = {(cuuint64_t)d.shape[1] * elem};
        const cuuint32_t box[2] = {(cuuint32_t)s, (cuuint32_t)s};
        const cuuint32_t estr[2] = {1, 1};
        const CUresult r = c->encode(&c->h_tm[t], bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                     2, const_cast<void *>(static_cast<const void *>(ptrs[t])), gdim, gstride, box, estr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return false;
    }
    return cudaMemcpyAsync(dev, c->h_tm.data(), sizeof(CUtensorMap) * (size_t)T, cudaMemcpyHostToDevice, stream) ==
           cudaSuccess;
}

void release(demo_ctx *c)
{
    if (!c) return;
    cudaFree(c->d_entries2d);
    cudaFree(c->d_entries1d);
    cudaFree(c->d_C);
    cudaFree(c->d_entries_nd);
    cudaFree(c->d_tables);
    cudaFree(c->d_P);
    cudaFree(c->d_P_stage);
    cudaFree(c->d_basis_flag);
    cudaFree(c->d_status);
    cudaFree((void *)c->d_g);
    cudaFree((void *)c->d_m);
    cudaFree((void *)c->d_x);
    cudaFree((void *)c->d_p);
    cudaFree((void *)c->d_s);
    cudaFree(c->d_flat);
    cudaFree(c->d_tm_g);
    cudaFree(c->d_tm_m);
    cudaFree(c->d_tm_x);
    for (cudaEvent_t e : c->ev_copied)
        if (e) cudaEventDestroy(e);
    if (c->ev_start) cudaEventDestroy(c->ev_start);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    if (c->side_stream) cudaStreamDestroy(c->side_stream);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    delete c;
}

}  // namespace

extern "C" {

const char *demo_status_string(demo_status status)
{
    switch (status) {
        case DEMO_OK: return "ok";
        case DEMO_ERR_INVALID_ARG: return "invalid argument";
        case DEMO_ERR_SHAPE: return "tensor order not supported or a dimension is not a multiple of its chunk extent";
        case DEMO_ERR_K: return "k out of range (1 <= k <= largest chunk)";
        case DEMO_ERR_UNSUPPORTED: return "unsupported chunk size, dtype or tensor count";
        case DEMO_ERR_ALLOC: return "allocation failed";
        case DEMO_ERR_CUDA: return "CUDA runtime error";
        case DEMO_ERR_TIMEOUT: return "bounded device-side wait expired";
        case DEMO_ERR_PAYLOAD: return "payload record index outside its chunk";
        default: return "unknown status";
    }
}

demo_status demo_init(demo_ctx **out, const demo_config *cfg, const demo_tensor_desc *tensors, int32_t n_tensors,
                      int32_t cuda_device)
{
    if (out) *out = nullptr;
    if (!out || !cfg || !tensors || n_tensors < 1 || cuda_device < 0) return DEMO_ERR_INVALID_ARG;
    if (cfg->num_workers < 1 || cfg->num_workers > 4096) return DEMO_ERR_INVALID_ARG;
    if (!std::isfinite(cfg->beta) || !std::isfinite(cfg->lr) || !std::isfinite(cfg->weight_decay))
        return DEMO_ERR_INVALID_ARG;
    const int s = cfg->chunk;
    if (!(s == 8 || s == 16 || s == 32 || s == 64 || s == 128)) return DEMO_ERR_UNSUPPORTED;
    if (cfg->grad_dtype != DEMO_F32 && cfg->grad_dtype != DEMO_BF16) return DEMO_ERR_UNSUPPORTED;
    if (n_tensors > (1 << 20)) return DEMO_ERR_UNSUPPORTED;
    if (cfg->topk < 1 || (long long)cfg->topk > (long long)s * s) return DEMO_ERR_K;
    for (int t = 0; t < n_tensors; ++t) {
        const demo_tensor_desc &d = tensors[t];
        if (d.ndim != 1 && d.ndim != 2) return DEMO_ERR_SHAPE;
        for (int a = 0; a < d.ndim; ++a)
            if (d.shape[a] < s || d.shape[a] % s != 0 || d.shape[a] > (1LL << 31) - 1) return DEMO_ERR_SHAPE;
        // the kernels index the chunks of one tensor with 31 bits
        const long long n_ch = (d.shape[0] / s) * (d.ndim == 2 ? d.shape[1] / s : 1);
        if (n_ch > (1LL << 31) - 1) return DEMO_ERR_UNSUPPORTED;
    }

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cuda_device >= n_dev) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    DeviceGuard guard(cuda_device);
    if (!guard.ok) return DEMO_ERR_CUDA;

    demo_ctx *c = new (std::nothrow) demo_ctx();
    if (!c) return DEMO_ERR_ALLOC;
    c->cfg = *cfg;
    c->device = cuda_device;
    c->n_tensors = n_tensors;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, cuda_device) != cudaSuccess) {
        release(c);
        return DEMO_ERR_CUDA;
    }

    // planner: payload offsets and the two work lists (2-D tiles, 1-D segments)
    std::vector<DemoTensorEntry> e2d, e1d;
    try {
        c->descs.assign(tensors, tensors + n_tensors);
        c->first_record.resize(n_tensors);
        c->n_chunks.resize(n_tensors);
        c->n_elems.resize(n_tensors);
        c->k_eff.resize(n_tensors);
        long long rec = 0;
        for (int t = 0; t < n_tensors; ++t) {
            const demo_tensor_desc &d = tensors[t];
            const bool two = d.ndim == 2;
            const long long n1 = two ? d.shape[1] : d.shape[0];
            const long long c0 = two ? d.shape[0] / s : 1, c1 = n1 / s;
            const long long M = two ? (long long)s * s : s;
            DemoTensorEntry e;
            e.tensor = t;
            e.n1 = (int)n1;
            e.c1 = (int)c1;
            e.k_eff = (int)(cfg->topk < M ? cfg->topk : M);
            e.rec_begin = rec;
            e.chunk_begin = two ? c->chunks2d : c->chunks1d;
            (two ? c->chunks2d : c->chunks1d) += c0 * c1;
            (two ? e2d : e1d).push_back(e);
            c->first_record[t] = rec;
            c->n_chunks[t] = c0 * c1;
            c->n_elems[t] = two ? d.shape[0] * d.shape[1] : d.shape[0];
            c->k_eff[t] = e.k_eff;
            rec += c0 * c1 * e.k_eff;
        }
        c->total_records = rec;
        const size_t W = (size_t)cfg->num_workers, T = (size_t)n_tensors;
        c->h_g.assign(W * T, nullptr);
        c->h_m.assign(W * T, nullptr);
        c->h_x.assign(T, nullptr);
        c->h_p.assign(W, nullptr);
        c->g_valid.assign(W, 0);
        c->m_valid.assign(W, 0);
    } catch (const std::bad_alloc &) {
        release(c);
        return DEMO_ERR_ALLOC;
    }
    c->n2d = (int)e2d.size();
    c->n1d = (int)e1d.size();

    // orthonormal DCT-II basis, built in fp64 and rounded once to fp32:
    // C[u][n] = a_u cos(pi (2n+1) u / (2s)), a_0 = sqrt(1/s), a_u = sqrt(2/s)
    std::vector<float> C((size_t)s * s);
    {
        const double pi = 3.141592653589793238462643383279502884;
        for (int u = 0; u < s; ++u)
            for (int n = 0; n < s; ++n) {
                const double a = (u == 0) ? std::sqrt(1.0 / s) : std::sqrt(2.0 / s);
                C[(size_t)u * s + n] = (float)(a * std::cos(pi * (2.0 * n + 1.0) * u / (2.0 * s)));
            }
    }

    const size_t W = (size_t)cfg->num_workers, T = (size_t)n_tensors;
    bool ok = true;
    ok = ok && cudaMalloc(&c->d_C, C.size() * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_status, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_P, C.size() * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_P_stage, 2 * C.size() * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_basis_flag, sizeof(int)) == cudaSuccess;
    if (ok && c->n2d) ok = cudaMalloc(&c->d_entries2d, e2d.size() * sizeof(DemoTensorEntry)) == cudaSuccess;
    if (ok && c->n1d) ok = cudaMalloc(&c->d_entries1d, e1d.size() * sizeof(DemoTensorEntry)) == cudaSuccess;
    ok = ok && cudaMalloc((void **)&c->d_g, W * T * sizeof(void *)) == cudaSuccess;
    ok = ok && cudaMalloc((void **)&c->d_m, W * T * sizeof(void *)) == cudaSuccess;
    ok = ok && cudaMalloc((void **)&c->d_x, T * sizeof(void *)) == cudaSuccess;
    ok = ok && cudaMalloc((void **)&c->d_p, W * sizeof(void *)) == cudaSuccess;
    if (ok && c->n2d && demo_fast_supported(s)) {
        // TMA descriptors need the driver's encoder; without it the fast kernels stage row by row
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess && fn) {
            c->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
            try {
                c->h_tm.resize(T);
            } catch (const std::bad_alloc &) {
                ok = false;
            }
            ok = ok && cudaMalloc(&c->d_tm_g, W * T * sizeof(CUtensorMap)) == cudaSuccess;
            ok = ok && cudaMalloc(&c->d_tm_m, W * T * sizeof(CUtensorMap)) == cudaSuccess;
            ok = ok && cudaMalloc(&c->d_tm_x, T * sizeof(CUtensorMap)) == cudaSuccess;
        } else {
            cudaGetLastError();
        }
    }
    if (!ok) {
        cudaGetLastError();
        release(c);
        return DEMO_ERR_ALLOC;
    }
    ok = ok && cudaMemcpy(c->d_C, C.data(), C.size() * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemset(c->d_status, 0, sizeof(int)) == cudaSuccess;
    if (ok && c->n2d && c->n1d) {
        // optional: without them the two kernels of a call simply run one after the other
        if (cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            if (c->side_stream) cudaStreamDestroy(c->side_stream);
            c->side_stream = nullptr;
        }
    }
    if (ok && c->n2d)
        ok = cudaMemcpy(c->d_entries2d, e2d.data(), e2d.size() * sizeof(DemoTensorEntry), cudaMemcpyHostToDevice) ==
             cudaSuccess;
    if (ok && c->n1d)
        ok = cudaMemcpy(c->d_entries1d, e1d.data(), e1d.size() * sizeof(DemoTensorEntry), cudaMemcpyHostToDevice) ==
             cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        release(c);
        return DEMO_ERR_CUDA;
    }
    *out = c;
    return DEMO_OK;
}

demo_status demo_init_nd(demo_ctx **out, const demo_config *cfg, const demo_nd_tensor_desc *tensors, int32_t n_tensors,
                         int32_t cuda_device)
{
    if (out) *out = nullptr;
    if (!out || !cfg || !tensors || n_tensors < 1 || cuda_device < 0) return DEMO_ERR_INVALID_ARG;
    if (cfg->num_workers < 1 || cfg->num_workers > 4096) return DEMO_ERR_INVALID_ARG;
    if (!std::isfinite(cfg->beta) || !std::isfinite(cfg->lr) || !std::isfinite(cfg->weight_decay))
        return DEMO_ERR_INVALID_ARG;
    if (cfg->grad_dtype != DEMO_F32 && cfg->grad_dtype != DEMO_BF16) return DEMO_ERR_UNSUPPORTED;
    if (n_tensors > (1 << 20)) return DEMO_ERR_UNSUPPORTED;
    if (cfg->topk < 1 || cfg->topk > DEMO_ND_MAX_CHUNK_ELEMS) return DEMO_ERR_K;
    for (int t = 0; t < n_tensors; ++t) {
        const demo_nd_tensor_desc &d = tensors[t];
        if (d.ndim < 1 || d.ndim > DEMO_ND_MAX_DIMS) return DEMO_ERR_SHAPE;
        long long M = 1, n_ch = 1, n_el = 1;
        for (int a = 0; a < d.ndim; ++a) {
            if (d.chunk[a] < 1) return DEMO_ERR_SHAPE;
            if (d.chunk[a] > DEMO_ND_MAX_EXTENT) return DEMO_ERR_UNSUPPORTED;
            if (d.shape[a] < d.chunk[a] || d.shape[a] % d.chunk[a] != 0 || d.shape[a] > (1LL << 31) - 1)
                return DEMO_ERR_SHAPE;
            M *= d.chunk[a];
            n_ch *= d.shape[a] / d.chunk[a];
            n_el *= d.shape[a];
            if (M > DEMO_ND_MAX_CHUNK_ELEMS || n_ch > (1LL << 31) - 1 || n_el > (1LL << 40)) return DEMO_ERR_UNSUPPORTED;
        }
    }

    // Square chunks of one size: when every tensor is cut into s x s tiles of its last two axes or into length-s
    // segments of its last axis (all leading chunk extents 1, so the leading axes merely stack rows), for one s
    // that demo_init knows, the layout of chunks and records is that of demo_init on the flattened tensors -- the
    // context is built by it and runs its kernels (fast DCT, tensor maps, side stream).
    {
        int s_common = 0;
        bool regular = true;
        std::vector<demo_tensor_desc> flat;
        try {
            flat.resize((size_t)n_tensors);
        } catch (const std::bad_alloc &) {
            return DEMO_ERR_ALLOC;
        }
        for (int t = 0; t < n_tensors && regular; ++t) {
            const demo_nd_tensor_desc &d = tensors[t];
            int lead = 0;
            while (lead < d.ndim - 1 && d.chunk[lead] == 1) ++lead;
            const int rest = d.ndim - lead;  // axes that are really cut: 1 or 2
            if (rest > 2) {
                regular = false;
                break;
            }
            long long rows = 1;
            for (int a = 0; a < lead; ++a) rows *= d.shape[a];
            for (int a = lead; a < d.ndim; ++a) {
                if (s_common == 0) s_common = d.chunk[a];
                if (d.chunk[a] != s_common) regular = false;
            }
            flat[t].ndim = rest;
            flat[t].shape[0] = rows * d.shape[lead];
            flat[t].shape[1] = rest == 2 ? d.shape[lead + 1] : 0;
            if (flat[t].shape[0] > (1LL << 31) - 1) regular = false;
        }
        if (regular && (s_common == 8 || s_common == 16 || s_common == 32 || s_common == 64 || s_common == 128)) {
            demo_config sq = *cfg;
            sq.chunk = s_common;
            if ((long long)sq.topk > (long long)s_common * s_common) sq.topk = s_common * s_common;  // same k_eff
            return demo_init(out, &sq, flat.data(), n_tensors, cuda_device);
        }
    }

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cuda_device >= n_dev) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    DeviceGuard guard(cuda_device);
    if (!guard.ok) return DEMO_ERR_CUDA;

    demo_ctx *c = new (std::nothrow) demo_ctx();
    if (!c) return DEMO_ERR_ALLOC;
    c->cfg = *cfg;
    c->cfg.chunk = 0;  // chunk shapes are per tensor
    c->device = cuda_device;
    c->n_tensors = n_tensors;
    c->nd = true;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, cuda_device) != cudaSuccess) {
        release(c);
        return DEMO_ERR_CUDA;
    }

    // planner: the work list (axes padded on the left to DEMO_ND_DIMS), payload offsets, and one
    // orthonormal DCT-II matrix per distinct chunk extent
    std::vector<DemoNdEntry> entries;
    std::vector<float> tables;
    try {
        int table_of[DEMO_ND_MAX_EXTENT + 1];
        for (int &v : table_of) v = -1;
        c->first_record.resize(n_tensors);
        c->n_chunks.resize(n_tensors);
        c->n_elems.resize(n_tensors);
        c->k_eff.resize(n_tensors);
        long long rec = 0;
        for (int t = 0; t < n_tensors; ++t) {
            const demo_nd_tensor_desc &d = tensors[t];
            DemoNdEntry e;
            const int pad = DEMO_ND_DIMS - d.ndim;
            long long stride = 1, M = 1, n_ch = 1;
            for (int a = DEMO_ND_DIMS - 1; a >= 0; --a) {
                const bool real = a >= pad;
                const int s = real ? d.chunk[a - pad] : 1;
                const long long n = real ? d.shape[a - pad] : 1;
                e.s[a] = s;
                e.c[a] = (int)(n / s);
                e.stride[a] = stride;
                stride *= n;
                M *= s;
                n_ch *= n / s;
                e.basis[a] = 0;
                e.inv[a] = s > 1 ? (unsigned)(((1ULL << 32) + (unsigned)s - 1) / (unsigned)s) : 0u;
                if (s > 1) {
                    if (table_of[s] < 0) {
                        // C then C^T, each s x s; every table starts on a 16-byte boundary
                        table_of[s] = (int)tables.size();
                        const double pi = 3.141592653589793238462643383279502884;
                        std::vector<float> C((size_t)s * s);
                        for (int u = 0; u < s; ++u)
                            for (int n2 = 0; n2 < s; ++n2) {
                                const double au = (u == 0) ? std::sqrt(1.0 / s) : std::sqrt(2.0 / s);
                                C[(size_t)u * s + n2] = (float)(au * std::cos(pi * (2.0 * n2 + 1.0) * u / (2.0 * s)));
                            }
                        tables.insert(tables.end(), C.begin(), C.end());
                        for (int n2 = 0; n2 < s; ++n2)
                            for (int u = 0; u < s; ++u) tables.push_back(C[(size_t)u * s + n2]);
                        while (tables.size() % 4) tables.push_back(0.f);
                    }
                    e.basis[a] = table_of[s];
                }
            }
            e.tensor = t;
            e.M = (int)M;
            e.k_eff = (int)(cfg->topk < M ? cfg->topk : M);
            e.rec_begin = rec;
            e.chunk_begin = c->chunks_nd;
            c->chunks_nd += n_ch;
            e.chunk_end = c->chunks_nd;
            if (((e.M + 3) & ~3) > c->max_M) c->max_M = (e.M + 3) & ~3;  // buffers stay 16-byte aligned
            entries.push_back(e);
            c->first_record[t] = rec;
            c->n_chunks[t] = n_ch;
            c->n_elems[t] = stride;
            c->k_eff[t] = e.k_eff;
            rec += n_ch * e.k_eff;
        }
        c->total_records = rec;
        if (tables.empty()) tables.push_back(1.0f);  // every extent is 1: no matrix is ever read
        const size_t W = (size_t)cfg->num_workers, T = (size_t)n_tensors;
        c->h_g.assign(W * T, nullptr);
        c->h_m.assign(W * T, nullptr);
        c->h_x.assign(T, nullptr);
        c->h_p.assign(W, nullptr);
        c->g_valid.assign(W, 0);
        c->m_valid.assign(W, 0);
    } catch (const std::bad_alloc &) {
        release(c);
        return DEMO_ERR_ALLOC;
    }
    c->n_nd = n_tensors;

    const size_t W = (size_t)cfg->num_workers, T = (size_t)n_tensors;
    bool ok = true;
    ok = ok && cudaMalloc(&c->d_tables, tables.size() * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_entries_nd, entries.size() * sizeof(DemoNdEntry)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->d_status, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc((void **)&c->d_g, W * T * sizeof(void *)) == cudaSuccess;
    ok = ok && cudaMalloc((void **)&c->d_m, W * T * sizeof(void *)) == cudaSuccess;
    ok = ok && cudaMalloc((void **)&c->d_x, T * sizeof(void *)) == cudaSuccess;
    ok = ok && cudaMalloc((void **)&c->d_p, W * sizeof(void *)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        release(c);
        return DEMO_ERR_ALLOC;
    }
    ok = ok && cudaMemcpy(c->d_tables, tables.data(), tables.size() * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(c->d_entries_nd, entries.data(), entries.size() * sizeof(DemoNdEntry),
                          cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemset(c->d_status, 0, sizeof(int)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        release(c);
        return DEMO_ERR_CUDA;
    }
    *out = c;
    return DEMO_OK;
}

size_t demo_payload_bytes(const demo_ctx *ctx) { return ctx ? (size_t)ctx->total_records * sizeof(DemoRecord) : 0; }

demo_status demo_payload_layout(const demo_ctx *ctx, int32_t tensor, int64_t *first_record, int64_t *n_chunks,
                                int32_t *k_eff)
{
    if (!ctx || tensor < 0 || tensor >= ctx->n_tensors) return DEMO_ERR_INVALID_ARG;
    if (first_record) *first_record = ctx->first_record[tensor];
    if (n_chunks) *n_chunks = ctx->n_chunks[tensor];
    if (k_eff) *k_eff = ctx->k_eff[tensor];
    return DEMO_OK;
}

// The 1-D kernel of a call goes to the side stream: it is ordered after everything already queued on the
// caller's stream (fork) and the caller's stream continues only when it is done (join).
static cudaStream_t fork_side(demo_ctx *ctx, cudaStream_t stream)
{
    if (!ctx->side_stream || !ctx->n2d || !ctx->n1d) return stream;
    if (cudaEventRecord(ctx->ev_fork, stream) != cudaSuccess ||
        cudaStreamWaitEvent(ctx->side_stream, ctx->ev_fork, 0) != cudaSuccess) {
        cudaGetLastError();
        return stream;
    }
    return ctx->side_stream;
}
static cudaError_t join_side(demo_ctx *ctx, cudaStream_t side, cudaStream_t stream)
{
    if (side == stream) return cudaSuccess;
    cudaError_t err = cudaEventRecord(ctx->ev_join, side);
    if (err == cudaSuccess) err = cudaStreamWaitEvent(stream, ctx->ev_join, 0);
    return err;
}

// The fast kernels hard-code the DCT factorisation; any other basis takes the dense-transform kernels.
static bool use_fast_path(const demo_ctx *ctx)
{
    const int s = ctx->cfg.chunk;
    return ctx->path == DEMO_PATH_AUTO && !ctx->custom_basis && demo_fast_supported(s) && (s != 128 || ctx->encode);
}

// A caller-supplied basis has no fast factorisation: its dense transforms run on the tensor cores where
// there is a kernel for the chunk size, else on the CUDA cores.
static bool use_tc_path(const demo_ctx *ctx)
{
    return ctx->path == DEMO_PATH_AUTO && ctx->custom_basis && demo_tc_supported(ctx->cfg.chunk);
}

demo_status demo_compress(demo_ctx *ctx, int32_t worker, const void *const *grads, float *const *momentum,
                          void *payload_out, void *cuda_stream)
{
    if (!ctx || !grads || !momentum || !payload_out) return DEMO_ERR_INVALID_ARG;
    if (worker < 0 || worker >= ctx->cfg.num_workers) return DEMO_ERR_INVALID_ARG;
    if (!aligned16(payload_out)) return DEMO_ERR_INVALID_ARG;
    const int T = ctx->n_tensors;
    for (int t = 0; t < T; ++t)
        if (!grads[t] || !momentum[t] || !aligned16(grads[t]) || !aligned16(momentum[t])) return DEMO_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    const size_t row = (size_t)worker * (size_t)T;
    bool gv = ctx->g_valid[worker] != 0, mv = ctx->m_valid[worker] != 0;
    bool g_changed = false, m_changed = false;
    cudaError_t err =
        sync_table<const void *>(ctx->d_g + row, ctx->h_g.data() + row, grads, T, &gv, stream, &g_changed);
    ctx->g_valid[worker] = gv;
    if (err == cudaSuccess) {
        err = sync_table<float *>(ctx->d_m + row, ctx->h_m.data() + row, const_cast<float *const *>(momentum), T, &mv,
                                  stream, &m_changed);
        ctx->m_valid[worker] = mv;
    }
    if (err == cudaSuccess && ctx->encode) {
        const bool bf16 = ctx->cfg.grad_dtype == DEMO_BF16;
        if (g_changed && !upload_tensor_maps(ctx, ctx->d_tm_g + row, grads, bf16, stream)) err = cudaErrorInvalidValue;
        if (err == cudaSuccess && m_changed && !upload_tensor_maps(ctx, ctx->d_tm_m + row, momentum, false, stream))
            err = cudaErrorInvalidValue;
        if (err != cudaSuccess) ctx->g_valid[worker] = ctx->m_valid[worker] = 0;
    }
    if (err != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }

    if (ctx->momentum_dct && !(use_fast_path(ctx) && ctx->encode && ctx->cfg.chunk == 64 && !ctx->nd))
        return DEMO_ERR_UNSUPPORTED;  // only the s = 64 tile kernel keeps the momentum in the transform domain

    if (ctx->nd) {
        DemoNdCompressArgs n;
        n.entries = ctx->d_entries_nd;
        n.n_entries = ctx->n_nd;
        n.n_chunks = ctx->chunks_nd;
        n.g_ptrs = ctx->d_g + row;
        n.m_ptrs = ctx->d_m + row;
        n.payload = static_cast<DemoRecord *>(payload_out);
        n.tables = ctx->d_tables;
        n.beta = ctx->cfg.beta;
        n.alpha = ctx->alpha;
        n.grad_bf16 = ctx->cfg.grad_dtype == DEMO_BF16;
        n.max_M = ctx->max_M;
        n.status = ctx->d_status;
        if (demo_launch_compress_nd(n, ctx->sm_count, stream) != cudaSuccess) {
            cudaGetLastError();
            return DEMO_ERR_CUDA;
        }
        ctx->launches += 1;
        return DEMO_OK;
    }

    DemoCompressArgs a;
    a.g_ptrs = ctx->d_g + row;
    a.m_ptrs = ctx->d_m + row;
    a.payload = static_cast<DemoRecord *>(payload_out);
    a.C = ctx->custom_basis ? ctx->d_P : ctx->d_C;
    a.beta = ctx->cfg.beta;
    a.alpha = ctx->alpha;
    a.grad_bf16 = ctx->cfg.grad_dtype == DEMO_BF16;
    a.status = ctx->d_status;
    a.tmap_m = ctx->encode ? ctx->d_tm_m + row : nullptr;
    a.tmap_g = ctx->encode ? ctx->d_tm_g + row : nullptr;
    const int s = ctx->cfg.chunk;
    cudaStream_t side = stream;
    if (ctx->n1d) {
        side = fork_side(ctx, stream);
        a.momentum_dct = 0;  // 1-D tensors keep the momentum itself
        a.entries = ctx->d_entries1d;
        a.n_entries = ctx->n1d;
        a.n_chunks = ctx->chunks1d;
        err = demo_launch_compress_generic(s, 0, a, ctx->sm_count, side);
        ctx->launches += 1;
    }
    if (err == cudaSuccess && ctx->n2d) {
        a.entries = ctx->d_entries2d;
        a.n_entries = ctx->n2d;
        a.n_chunks = ctx->chunks2d;
        a.momentum_dct = ctx->momentum_dct ? 1 : 0;
        if (use_fast_path(ctx))
            err = demo_launch_compress_fast(s, a, ctx->sm_count, stream);
        else if (use_tc_path(ctx))
            err = demo_launch_compress_tc(a, ctx->sm_count, stream);
        else
            err = demo_launch_compress_generic(s, 1, a, ctx->sm_count, stream);
        ctx->launches += 1;
    }
    {
        const cudaError_t jerr = join_side(ctx, side, stream);  // always, so that a fork never stays open
        if (err == cudaSuccess) err = jerr;
    }
    if (err != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    return DEMO_OK;
}

// Tables of the parameter-server entry points, built on first use: the device array of sign-tensor
// pointers and the element ranges demo_apply_signs walks.
static demo_status ensure_sign_tables(demo_ctx *ctx)
{
    if (ctx->d_s && ctx->d_flat) return DEMO_OK;
    const int T = ctx->n_tensors;
    std::vector<DemoFlatEntry> flat;
    try {
        ctx->h_s.assign((size_t)T, nullptr);
        flat.resize((size_t)T);
    } catch (const std::bad_alloc &) {
        return DEMO_ERR_ALLOC;
    }
    long long q = 0;
    for (int t = 0; t < T; ++t) {
        flat[t].quad_begin = q;
        flat[t].n = ctx->n_elems[t];
        flat[t].tensor = t;
        flat[t].pad = 0;
        q += (ctx->n_elems[t] + 3) / 4;
    }
    ctx->n_quads = q;
    if (!ctx->d_s && cudaMalloc((void **)&ctx->d_s, (size_t)T * sizeof(void *)) != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_ALLOC;
    }
    if (!ctx->d_flat) {
        if (cudaMalloc(&ctx->d_flat, (size_t)T * sizeof(DemoFlatEntry)) != cudaSuccess) {
            cudaGetLastError();
            return DEMO_ERR_ALLOC;
        }
        if (cudaMemcpy(ctx->d_flat, flat.data(), (size_t)T * sizeof(DemoFlatEntry), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(ctx->d_flat);
            ctx->d_flat = nullptr;
            return DEMO_ERR_CUDA;
        }
    }
    return DEMO_OK;
}

// demo_decode_apply (params != NULL) and demo_decode_signs (signs != NULL) share everything but the last
// step of the kernels.
static demo_status decode_common(demo_ctx *ctx, const void *const *payloads, int32_t n_payloads, float *const *params,
                                 signed char *const *signs, void *cuda_stream)
{
    if (!ctx || !payloads || (!params && !signs)) return DEMO_ERR_INVALID_ARG;
    if (n_payloads != ctx->cfg.num_workers) return DEMO_ERR_INVALID_ARG;
    const int T = ctx->n_tensors, W = n_payloads;
    for (int w = 0; w < W; ++w)
        if (!payloads[w] || !aligned16(payloads[w])) return DEMO_ERR_INVALID_ARG;
    for (int t = 0; t < T; ++t) {
        if (params && (!params[t] || !aligned16(params[t]))) return DEMO_ERR_INVALID_ARG;
        if (signs && (!signs[t] || !aligned16(signs[t]))) return DEMO_ERR_INVALID_ARG;
    }
    if (signs && ctx->phi != DEMO_PHI_SIGN) return DEMO_ERR_INVALID_ARG;  // only the sign is handed out
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (signs) {
        const demo_status st = ensure_sign_tables(ctx);
        if (st != DEMO_OK) return st;
    }

    cudaError_t err = sync_table<const DemoRecord *>(ctx->d_p, ctx->h_p.data(),
                                                     reinterpret_cast<const DemoRecord *const *>(payloads), W,
                                                     &ctx->p_valid, stream);
    bool x_changed = false;
    if (err == cudaSuccess && params)
        err = sync_table<float *>(ctx->d_x, ctx->h_x.data(), const_cast<float *const *>(params), T, &ctx->x_valid,
                                  stream, &x_changed);
    if (err == cudaSuccess && params && ctx->encode && x_changed &&
        !upload_tensor_maps(ctx, ctx->d_tm_x, params, false, stream)) {
        err = cudaErrorInvalidValue;
        ctx->x_valid = false;
    }
    if (err == cudaSuccess && signs)
        err = sync_table<signed char *>(ctx->d_s, ctx->h_s.data(), const_cast<signed char *const *>(signs), T,
                                        &ctx->s_valid, stream);
    if (err != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }

    if (ctx->nd) {
        DemoNdDecodeArgs n;
        n.entries = ctx->d_entries_nd;
        n.n_entries = ctx->n_nd;
        n.n_chunks = ctx->chunks_nd;
        n.payloads = ctx->d_p;
        n.W = W;
        n.x_ptrs = ctx->d_x;
        n.tables = ctx->d_tables;
        n.lr = ctx->cfg.lr;
        n.wd = ctx->cfg.weight_decay;
        n.max_M = ctx->max_M;
        n.status = ctx->d_status;
        n.agg = ctx->aggregation;
        n.phi = ctx->phi;
        n.agg_scale = (ctx->aggregation == DEMO_AGG_MEAN) ? 1.0f / (float)W : 1.0f;
        n.sign_ptrs = signs ? ctx->d_s : nullptr;
        if (demo_launch_decode_nd(n, ctx->sm_count, stream) != cudaSuccess) {
            cudaGetLastError();
            return DEMO_ERR_CUDA;
        }
        ctx->launches += 1;
        return DEMO_OK;
    }

    DemoDecodeArgs a;
    a.payloads = ctx->d_p;
    a.W = W;
    a.x_ptrs = ctx->d_x;
    a.C = ctx->custom_basis ? ctx->d_P : ctx->d_C;
    a.lr = ctx->cfg.lr;
    a.wd = ctx->cfg.weight_decay;
    a.status = ctx->d_status;
    a.tmap_x = (ctx->encode && params) ? ctx->d_tm_x : nullptr;
    a.agg = ctx->aggregation;
    a.phi = ctx->phi;
    a.agg_scale = (ctx->aggregation == DEMO_AGG_MEAN) ? 1.0f / (float)W : 1.0f;
    a.sign_ptrs = signs ? ctx->d_s : nullptr;
    const int s = ctx->cfg.chunk;
    cudaStream_t side = stream;
    if (ctx->n1d) {
        side = fork_side(ctx, stream);
        a.entries = ctx->d_entries1d;
        a.n_entries = ctx->n1d;
        a.n_chunks = ctx->chunks1d;
        err = demo_launch_decode_generic(s, 0, a, ctx->sm_count, side);
        ctx->launches += 1;
    }
    if (err == cudaSuccess && ctx->n2d) {
        a.entries = ctx->d_entries2d;
        a.n_entries = ctx->n2d;
        a.n_chunks = ctx->chunks2d;
        // (a caller-supplied basis: the signs come from the dense kernels, there is no tensor-core variant)
        if (use_fast_path(ctx))
            err = demo_launch_decode_fast(s, a, ctx->sm_count, stream);
        else if (use_tc_path(ctx) && !signs)
            err = demo_launch_decode_tc(a, ctx->sm_count, stream);
        else
            err = demo_launch_decode_generic(s, 1, a, ctx->sm_count, stream);
        ctx->launches += 1;
    }
    {
        const cudaError_t jerr = join_side(ctx, side, stream);
        if (err == cudaSuccess) err = jerr;
    }
    if (err != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    return DEMO_OK;
}

demo_status demo_decode_apply(demo_ctx *ctx, const void *const *payloads, int32_t n_payloads, float *const *params,
                              void *cuda_stream)
{
    if (!params) return DEMO_ERR_INVALID_ARG;
    return decode_common(ctx, payloads, n_payloads, params, nullptr, cuda_stream);
}

demo_status demo_decode_signs(demo_ctx *ctx, const void *const *payloads, int32_t n_payloads, int8_t *const *signs_out,
                              void *cuda_stream)
{
    if (!signs_out) return DEMO_ERR_INVALID_ARG;
    return decode_common(ctx, payloads, n_payloads, nullptr, reinterpret_cast<signed char *const *>(signs_out),
                         cuda_stream);
}

demo_status demo_apply_signs(demo_ctx *ctx, const int8_t *const *signs, float *const *params, void *cuda_stream)
{
    if (!ctx || !signs || !params) return DEMO_ERR_INVALID_ARG;
    const int T = ctx->n_tensors;
    for (int t = 0; t < T; ++t)
        if (!signs[t] || !params[t] || !aligned16(signs[t]) || !aligned16(params[t])) return DEMO_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const demo_status st = ensure_sign_tables(ctx);
    if (st != DEMO_OK) return st;
    bool x_changed = false;
    cudaError_t err = sync_table<float *>(ctx->d_x, ctx->h_x.data(), const_cast<float *const *>(params), T,
                                          &ctx->x_valid, stream, &x_changed);
    if (err == cudaSuccess && ctx->encode && x_changed && !upload_tensor_maps(ctx, ctx->d_tm_x, params, false, stream)) {
        err = cudaErrorInvalidValue;
        ctx->x_valid = false;
    }
    if (err == cudaSuccess)
        err = sync_table<signed char *>(ctx->d_s, ctx->h_s.data(),
                                        const_cast<signed char *const *>(reinterpret_cast<const signed char *const *>(signs)),
                                        T, &ctx->s_valid, stream);
    if (err == cudaSuccess) {
        DemoApplySignsArgs a;
        a.entries = ctx->d_flat;
        a.n_entries = T;
        a.n_quads = ctx->n_quads;
        a.sign_ptrs = ctx->d_s;
        a.x_ptrs = ctx->d_x;
        a.lr = ctx->cfg.lr;
        a.wd = ctx->cfg.weight_decay;
        err = demo_launch_apply_signs(a, ctx->sm_count, stream);
        ctx->launches += 1;
    }
    if (err != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    return DEMO_OK;
}

demo_status demo_step_host(demo_ctx *ctx, const void *const *host_grads, void *const *dev_grads,
                           float *const *momentum, void *const *payloads, float *const *params,
                           void *host_payloads_out, void *cuda_stream)
{
    if (!ctx || !host_grads || !dev_grads || !momentum || !payloads || !params) return DEMO_ERR_INVALID_ARG;
    const int T = ctx->n_tensors, W = ctx->cfg.num_workers;
    const size_t gsize = ctx->cfg.grad_dtype == DEMO_BF16 ? 2 : 4;
    for (size_t i = 0; i < (size_t)W * T; ++i)
        if (!host_grads[i] || !dev_grads[i]) return DEMO_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (!ctx->copy_stream) {
        bool ok = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming) == cudaSuccess;
        try {
            ctx->ev_copied.assign((size_t)W, nullptr);
        } catch (const std::bad_alloc &) {
            ok = false;
        }
        for (int w = 0; ok && w < W; ++w)
            ok = cudaEventCreateWithFlags(&ctx->ev_copied[w], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            return DEMO_ERR_ALLOC;
        }
    }
    // the copies start once everything already queued on the caller's stream (the previous step, which
    // reads the staging tensors) has finished, then run ahead of the compress calls
    bool ok = cudaEventRecord(ctx->ev_start, stream) == cudaSuccess &&
              cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_start, 0) == cudaSuccess;
    for (int w = 0; ok && w < W; ++w) {
        const size_t row = (size_t)w * T;
        for (int t = 0; ok && t < T; ++t)
            ok = cudaMemcpyAsync(dev_grads[row + t], host_grads[row + t], (size_t)ctx->n_elems[t] * gsize,
                                 cudaMemcpyHostToDevice, ctx->copy_stream) == cudaSuccess;
        ok = ok && cudaEventRecord(ctx->ev_copied[w], ctx->copy_stream) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    for (int w = 0; w < W; ++w) {
        const size_t row = (size_t)w * T;
        if (cudaStreamWaitEvent(stream, ctx->ev_copied[w], 0) != cudaSuccess) {
            cudaGetLastError();
            return DEMO_ERR_CUDA;
        }
        demo_status st = demo_compress(ctx, w, const_cast<const void *const *>(dev_grads + row), momentum + row,
                                       payloads[w], cuda_stream);
        if (st != DEMO_OK) return st;
    }
    demo_status st = demo_decode_apply(ctx, const_cast<const void *const *>(payloads), W, params, cuda_stream);
    if (st != DEMO_OK) return st;
    if (host_payloads_out) {
        const size_t pb = demo_payload_bytes(ctx);
        for (int w = 0; w < W; ++w)
            if (cudaMemcpyAsync(static_cast<char *>(host_payloads_out) + (size_t)w * pb, payloads[w], pb,
                                cudaMemcpyDeviceToHost, stream) != cudaSuccess) {
                cudaGetLastError();
                return DEMO_ERR_CUDA;
            }
    }
    return DEMO_OK;
}

demo_status demo_set_lr(demo_ctx *ctx, float lr)
{
    if (!ctx || !std::isfinite(lr)) return DEMO_ERR_INVALID_ARG;
    ctx->cfg.lr = lr;
    return DEMO_OK;
}

demo_status demo_set_alpha(demo_ctx *ctx, float alpha)
{
    if (!ctx || !(alpha >= 0.0f && alpha <= 1.0f)) return DEMO_ERR_INVALID_ARG;
    ctx->alpha = alpha;
    return DEMO_OK;
}

demo_status demo_set_decode_mode(demo_ctx *ctx, int32_t aggregation, int32_t phi)
{
    if (!ctx) return DEMO_ERR_INVALID_ARG;
    if (aggregation != DEMO_AGG_SUM && aggregation != DEMO_AGG_MEAN && aggregation != DEMO_AGG_COUNT_MEAN)
        return DEMO_ERR_INVALID_ARG;
    if (phi != DEMO_PHI_SIGN && phi != DEMO_PHI_IDENTITY) return DEMO_ERR_INVALID_ARG;
    if (aggregation == DEMO_AGG_COUNT_MEAN && ctx->cfg.num_workers > 65535) return DEMO_ERR_UNSUPPORTED;
    ctx->aggregation = aggregation;
    ctx->phi = phi;
    return DEMO_OK;
}

demo_status demo_selftest_bounded_wait(demo_ctx *ctx, int64_t limit_cycles, void *cuda_stream)
{
    if (!ctx || limit_cycles < 1 || limit_cycles > 2000000000LL) return DEMO_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    if (demo_launch_wait_selftest(ctx->d_status, limit_cycles, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    ctx->launches += 1;
    return DEMO_OK;
}

demo_status demo_set_basis(demo_ctx *ctx, const float *basis_host, void *cuda_stream)
{
    if (!ctx) return DEMO_ERR_INVALID_ARG;
    if (ctx->nd) return DEMO_ERR_UNSUPPORTED;  // one basis per chunk extent: only the DCT is built
    if (!basis_host) {
        ctx->custom_basis = false;
        return DEMO_OK;
    }
    const int s = ctx->cfg.chunk;
    // rows must be orthonormal: |<p_u, p_v> - delta_uv| <= 1e-5 (fp32 entries carry ~6e-8 each)
    for (int u = 0; u < s; ++u)
        for (int v = u; v < s; ++v) {
            double dot = 0.0;
            for (int n = 0; n < s; ++n) dot += (double)basis_host[(size_t)u * s + n] * basis_host[(size_t)v * s + n];
            if (!(std::fabs(dot - (u == v ? 1.0 : 0.0)) <= 1e-5)) return DEMO_ERR_INVALID_ARG;
        }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    if (cudaMemcpyAsync(ctx->d_P, basis_host, sizeof(float) * (size_t)s * s, cudaMemcpyHostToDevice,
                        static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    ctx->custom_basis = true;
    return DEMO_OK;
}

demo_status demo_set_basis_gaussian(demo_ctx *ctx, const float *gauss_host, void *cuda_stream)
{
    if (!ctx || !gauss_host) return DEMO_ERR_INVALID_ARG;
    if (ctx->nd) return DEMO_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int s = ctx->cfg.chunk;
    const size_t n = (size_t)s * s;
    // staging = [Gaussian input | orthonormalised output]; the active table is replaced only after the
    // kernel's verdict, so a singular matrix leaves the previous basis in force
    float *gauss = ctx->d_P_stage, *out = ctx->d_P_stage + n;
    int flag = 0;
    bool ok = cudaMemcpyAsync(gauss, gauss_host, n * sizeof(float), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaMemsetAsync(ctx->d_basis_flag, 0, sizeof(int), stream) == cudaSuccess;
    ok = ok && demo_launch_gram_schmidt(gauss, out, ctx->d_basis_flag, s, stream) == cudaSuccess;
    if (ok) ctx->launches += 1;
    ok = ok && cudaMemcpyAsync(&flag, ctx->d_basis_flag, sizeof(int), cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    if (ok && flag) return DEMO_ERR_INVALID_ARG;
    ok = ok && cudaMemcpyAsync(ctx->d_P, out, n * sizeof(float), cudaMemcpyDeviceToDevice, stream) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    ctx->custom_basis = true;
    return DEMO_OK;
}

demo_status demo_get_basis(demo_ctx *ctx, float *basis_host_out, void *cuda_stream)
{
    if (!ctx || !basis_host_out) return DEMO_ERR_INVALID_ARG;
    if (ctx->nd) return DEMO_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t bytes = sizeof(float) * (size_t)ctx->cfg.chunk * ctx->cfg.chunk;
    if (cudaMemcpyAsync(basis_host_out, ctx->custom_basis ? ctx->d_P : ctx->d_C, bytes, cudaMemcpyDeviceToHost,
                        stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    return DEMO_OK;
}

demo_status demo_set_momentum_domain(demo_ctx *ctx, int32_t domain)
{
    if (!ctx || (domain != DEMO_MOMENTUM_SPATIAL && domain != DEMO_MOMENTUM_DCT)) return DEMO_ERR_INVALID_ARG;
    if (domain == DEMO_MOMENTUM_DCT && (ctx->nd || ctx->cfg.chunk != 64 || !ctx->encode)) return DEMO_ERR_UNSUPPORTED;
    ctx->momentum_dct = (domain == DEMO_MOMENTUM_DCT);
    return DEMO_OK;
}

demo_status demo_set_path(demo_ctx *ctx, int32_t path)
{
    if (!ctx || (path != DEMO_PATH_AUTO && path != DEMO_PATH_GENERIC)) return DEMO_ERR_INVALID_ARG;
    ctx->path = path;
    return DEMO_OK;
}

int64_t demo_launch_count(const demo_ctx *ctx) { return ctx ? ctx->launches : 0; }

demo_status demo_device_status(demo_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return DEMO_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DEMO_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    if (word != 0 && (cudaMemsetAsync(ctx->d_status, 0, sizeof(int), stream) != cudaSuccess ||
                      cudaStreamSynchronize(stream) != cudaSuccess)) {
        cudaGetLastError();
        return DEMO_ERR_CUDA;
    }
    if (word == DEMO_DEV_TIMEOUT) return DEMO_ERR_TIMEOUT;
    if (word == DEMO_DEV_PAYLOAD) return DEMO_ERR_PAYLOAD;
    return word == 0 ? DEMO_OK : DEMO_ERR_CUDA;
}

void demo_free(demo_ctx *ctx)
{
    if (!ctx) return;
    DeviceGuard guard(ctx->device);
    release(ctx);
}

}  // extern "C"
