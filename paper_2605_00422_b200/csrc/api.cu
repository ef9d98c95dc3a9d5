// extern "C" boundary: argument validation, workspace carving and per-shape dispatch.  No compute happens here.
#include <cstdlib>
#include <vector>

#include "bwla_common.cuh"

namespace bwla {

thread_local int g_last_cuda_error = 0;
thread_local int g_launch_count = 0;
static thread_local int g_forced_path = BWLA_PATH_AUTO;   // per calling thread, like the other bookkeeping
static thread_local int g_forced_rotation = 0;            // 0: per shape; 1: the FMA / warp-level MMA kernel; 2: tcgen05

// ---- optional kernel timing -------------------------------------------------------------------
struct ProfPair { cudaEvent_t a, b; int kind; };
static thread_local bool g_prof_on = false;
static thread_local std::vector<ProfPair>* g_prof = nullptr;       // pairs recorded since the last collect
static thread_local std::vector<ProfPair>* g_prof_pool = nullptr;  // idle pairs, reused so that recording stays cheap

unsigned launch_overlap_allowed() { return g_prof_on ? 0u : 1u; }

void prof_begin(int kind, cudaStream_t stream) {
    if (!g_prof_on) return;
    if (!g_prof) { g_prof = new std::vector<ProfPair>(); g_prof_pool = new std::vector<ProfPair>(); }
    ProfPair p{nullptr, nullptr, kind};
    if (!g_prof_pool->empty()) {
        p = g_prof_pool->back();
        p.kind = kind;
        g_prof_pool->pop_back();
    } else if (cudaEventCreate(&p.a) != cudaSuccess || cudaEventCreate(&p.b) != cudaSuccess) {
        return;
    }
    cudaEventRecord(p.a, stream);
    g_prof->push_back(p);
}
void prof_end(int kind, cudaStream_t stream) {
    if (!g_prof_on || !g_prof || g_prof->empty() || g_prof->back().kind != kind) return;
    cudaEventRecord(g_prof->back().b, stream);
}

static bool valid_bits(int bits) { return bits == 4 || bits == 6 || bits == 8; }

// The compute entry points need an sm_100 device to be current.
static int check_device() {
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; cudaGetLastError(); return BWLA_ERR_UNSUPPORTED; }
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; cudaGetLastError(); return BWLA_ERR_UNSUPPORTED; }
    return major == 10 ? BWLA_OK : BWLA_ERR_UNSUPPORTED;
}

static bool valid_rotation_dims(int64_t K, int n1, int n2) {
    return K > 0 && K % 32 == 0 && K <= 25600 && n1 > 0 && n2 > 0 && (int64_t)n1 * n2 == K;
}

// Up to how many tokens the bit-plane kernel is chosen over the tcgen05 one (0: never).  Measured per launch with cold
// weights on the Qwen3-32B and LLaMA-2-7B shapes (profiles/contraction_paths_small_m.md): at these sizes both kernels are
// bound by fixed latencies rather than by the stream of sign words, the tensor-core kernel's are the shorter ones
// (21 against 27 microseconds for 5120 -> 25600 at one token), and the bit-plane kernel's time grows with tokens x bits.
// It is therefore only taken where the tensor-core kernel cannot run (K not a multiple of 128, rank above 64).
static int bitplane_max_tokens(int64_t K, int64_t N, int bits) {
    (void)N; (void)bits;
    return (K % 128 != 0) ? 4 : 0;
}

// Which kernel family runs the contraction.  A forced family that cannot take the shape falls back to the simple one.
static int resolve_path(int64_t M, int64_t K, int64_t N, int r, int bits) {
    int path = g_forced_path;
    if (path == BWLA_PATH_AUTO) path = (M <= bitplane_max_tokens(K, N, bits) && bitplane_supports(M, K, N, r, bits)) ? BWLA_PATH_BITPLANE : BWLA_PATH_I8;
    if (path == BWLA_PATH_BITPLANE && !bitplane_supports(M, K, N, r, bits)) path = BWLA_PATH_SIMPLE;
    if (path == BWLA_PATH_I8 && !umma_supports(M, K, N, r, bits)) path = BWLA_PATH_SIMPLE;
    return path;
}

static int run_contraction(int path, GemmArgs& g, const int8_t* codes, cudaStream_t stream) {
    if (path == BWLA_PATH_I8) return launch_gemm_umma(g, codes, stream);
    g.codes = codes;
    if (path == BWLA_PATH_BITPLANE) return launch_gemm_bitplane(g, stream);
    return launch_gemm_simple(g, stream);
}

}  // namespace bwla

using namespace bwla;

// What a prepared layer remembers: the caller's device pointers and the plan of the rotation kernel.
struct bwla_layer {
    int64_t K, N;
    int n1, n2, bits, r;
    const float *P1, *P2, *alpha, *mu;
    const uint32_t* packed;
    const void *U, *V;
    uint8_t* prepared;
    bool okt;                 // the tcgen05 rotation takes these factor sizes
    OktGeom geom;
    int asym;                 // activation quantiser: 0 symmetric, 1 asymmetric (per-token zero point)
    int32_t* rowsum;          // [N] sign sums of the rows, inside `prepared`
};

extern "C" {

int bwla_pack_signs(const void* w, int dtype, int64_t N, int64_t K, int64_t ldw, uint32_t* packed, void* stream) {
    g_launch_count = 0;
    if (N < 0 || K <= 0 || K % 32 != 0 || ldw < K || (dtype != BWLA_DTYPE_F32 && dtype != BWLA_DTYPE_BF16))
        return BWLA_ERR_INVALID_ARG;
    if (N == 0) return BWLA_OK;
    if (!w || !packed) return BWLA_ERR_INVALID_ARG;
    int st = check_device();
    if (st != BWLA_OK) return st;
    return launch_pack_signs(w, dtype, N, K, ldw, packed, (cudaStream_t)stream);
}

size_t bwla_binarize_workspace_bytes(int64_t K) {
    if (K <= 0 || K % 32 != 0 || K > 25600) return 0;
    return binarize_workspace_bytes(K);
}

int bwla_binarize_rows(const void* w_res, int dtype, int64_t N, int64_t K, int64_t ldw, const float* P1, int n1,
                       const float* P2, int n2, uint32_t* packed, float* alpha, float* mu, void* workspace,
                       size_t workspace_bytes, void* stream) {
    g_launch_count = 0;
    if (N < 0 || !valid_rotation_dims(K, n1, n2) || ldw < K || (dtype != BWLA_DTYPE_F32 && dtype != BWLA_DTYPE_BF16))
        return BWLA_ERR_INVALID_ARG;
    if (N == 0) return BWLA_OK;
    if (!w_res || !P1 || !P2 || !packed || !alpha || !mu) return BWLA_ERR_INVALID_ARG;
    if (((uintptr_t)P1 & 15) || ((uintptr_t)P2 & 15)) return BWLA_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < bwla_binarize_workspace_bytes(K)) return BWLA_ERR_WORKSPACE;
    int st = check_device();
    if (st != BWLA_OK) return st;
    return launch_binarize(w_res, dtype, N, K, ldw, P1, n1, P2, n2, packed, alpha, mu, workspace, (cudaStream_t)stream);
}

int bwla_rotate_quant_act(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1,
                          const float* P2, int n2, int bits, int8_t* codes, float* scales, void* stream) {
    g_launch_count = 0;
    if (M < 0 || !valid_rotation_dims(K, n1, n2) || ldx < K || !valid_bits(bits)) return BWLA_ERR_INVALID_ARG;
    if (M == 0) return BWLA_OK;
    if (!x_bf16 || !P1 || !P2 || !codes || !scales) return BWLA_ERR_INVALID_ARG;
    if (((uintptr_t)codes & 15) || ((uintptr_t)P1 & 15) || ((uintptr_t)P2 & 15)) return BWLA_ERR_INVALID_ARG;
    int st = check_device();
    if (st != BWLA_OK) return st;
    return launch_prologue(x_bf16, M, K, ldx, P1, n1, P2, n2, bits, codes, 0, scales, nullptr, nullptr, 0, nullptr, nullptr, nullptr,
                           (cudaStream_t)stream);
}

size_t bwla_workspace_bytes(int64_t M, int64_t K, int64_t N, int r, int bits) {
    if (M < 0 || K <= 0 || K % 32 != 0 || N < 0 || r < 0 || !valid_bits(bits)) return 0;
    return workspace_layout(M, K, N, r, bits).total;
}

static int validate_gemm_tail(int64_t M, int64_t K, int bits, const uint32_t* packed, const float* alpha,
                              const void* U, const void* V, int r, int64_t N, int64_t ldo, const void* workspace,
                              size_t workspace_bytes) {
    if (M < 0 || N < 0 || K <= 0 || K % 32 != 0 || r < 0 || r > 256 || !valid_bits(bits)) return BWLA_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return BWLA_OK;
    if (!packed || !alpha || ldo < N) return BWLA_ERR_INVALID_ARG;
    if (r > 0 && (!U || !V)) return BWLA_ERR_INVALID_ARG;
    if (((uintptr_t)packed & 15)) return BWLA_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < workspace_layout(M, K, N, r, bits).total)
        return BWLA_ERR_WORKSPACE;
    return BWLA_OK;
}

}  // extern "C"

// Every check bwla_w1ax_linear makes before it touches the GPU (also used by the entry point with built-in scratch).
int bwla::validate_linear_call(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1,
                               const float* P2, int n2, int bits, const uint32_t* packed, const float* alpha,
                               const void* U_bf16, const void* V_bf16, int r, const void* out_bf16, int64_t N,
                               int64_t ldo, const void* workspace, size_t workspace_bytes) {
    if (!valid_rotation_dims(K, n1, n2) || ldx < K) return BWLA_ERR_INVALID_ARG;
    int st = validate_gemm_tail(M, K, bits, packed, alpha, U_bf16, V_bf16, r, N, ldo, workspace, workspace_bytes);
    if (st != BWLA_OK) return st;
    if (M == 0 || N == 0) return BWLA_OK;
    if (!x_bf16 || !P1 || !P2 || !out_bf16) return BWLA_ERR_INVALID_ARG;
    if (((uintptr_t)P1 & 15) || ((uintptr_t)P2 & 15)) return BWLA_ERR_INVALID_ARG;
    return check_device();
}

extern "C" {

int bwla_w1ax_linear(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1, const float* P2,
                     int n2, int bits, const uint32_t* packed, const float* alpha, const float* mu, const void* U_bf16,
                     const void* V_bf16, int r, void* out_bf16, int64_t N, int64_t ldo, void* workspace,
                     size_t workspace_bytes, void* stream) {
    g_launch_count = 0;
    int st = validate_linear_call(x_bf16, M, K, ldx, P1, n1, P2, n2, bits, packed, alpha, U_bf16, V_bf16, r, out_bf16, N,
                                  ldo, workspace, workspace_bytes);
    if (st != BWLA_OK) return st;
    if (M == 0 || N == 0) return BWLA_OK;

    cudaStream_t s = (cudaStream_t)stream;
    const Workspace ws = workspace_layout(M, K, N, r, bits);
    char* base = (char*)workspace;
    float* scales = (float*)(base + ws.scales);
    int32_t* qsum = (int32_t*)(base + ws.qsum);
    void* Thl = base + ws.T;
    int8_t* codes = (int8_t*)(base + ws.codes);
    const int path = resolve_path(M, K, N, r, bits);

    OktGeom geom;
    if (g_forced_rotation != 1 && okt_geometry(n1, n2, &geom) && okt_accepts_x(x_bf16, ldx) && okt_prepared_bytes(geom) <= kOktPreparedMax) {
        // the Kronecker factors are handed over raw: their bf16 terms go into the workspace first (a prepared layer
        // does this once instead)
        st = launch_prepare_okt(geom, P1, P2, base + ws.prep, s);
        if (st != BWLA_OK) return st;
        OktProblem pr{(const uint8_t*)(base + ws.prep), codes, path == BWLA_PATH_I8 ? 1 : 0, nullptr, 0, scales, qsum, nullptr};
        OktLowrank lr{V_bf16, r, Thl, r > 0 ? (float*)(base + ws.lr_part) : nullptr, (uint32_t*)(base + ws.status) + kLrCounterWord};
        st = launch_okt(geom, x_bf16, M, ldx, bits, 0, 1, &pr, &lr, (uint32_t*)(base + ws.status), s);
    } else {
        st = launch_prologue(x_bf16, M, K, ldx, P1, n1, P2, n2, bits, codes, path == BWLA_PATH_I8 ? 1 : 0, scales, qsum,
                             V_bf16, r, Thl, r > 0 ? (float*)(base + ws.lr_part) : nullptr, (uint32_t*)(base + ws.status), s);
    }
    if (st != BWLA_OK) return st;
    GemmArgs g{};
    g.scales = scales; g.qsum = qsum; g.M = M; g.K = K; g.N = N; g.bits = bits; g.packed = packed; g.alpha = alpha;
    g.mu = mu; g.Thl = r > 0 ? Thl : nullptr; g.U = U_bf16; g.r = r; g.out = out_bf16; g.ldo = ldo; g.acc_debug = nullptr;
    g.status = (uint32_t*)(base + ws.status);
    return run_contraction(path, g, codes, s);
}

int bwla_w1a_gemm_codes(const int8_t* codes, const float* scales, int64_t M, int64_t K, int bits,
                        const uint32_t* packed, const float* alpha, const float* mu, const void* x_bf16, int64_t ldx,
                        const void* U_bf16, const void* V_bf16, int r, void* out_bf16, int64_t N, int64_t ldo,
                        int32_t* acc_debug, void* workspace, size_t workspace_bytes, void* stream) {
    g_launch_count = 0;
    int st = validate_gemm_tail(M, K, bits, packed, alpha, U_bf16, V_bf16, r, N, ldo, workspace, workspace_bytes);
    if (st != BWLA_OK) return st;
    if (M == 0 || N == 0) return BWLA_OK;
    if (!codes || !scales || (!out_bf16 && !acc_debug)) return BWLA_ERR_INVALID_ARG;
    if (((uintptr_t)codes & 15)) return BWLA_ERR_INVALID_ARG;
    if (r > 0 && (!x_bf16 || ldx < K)) return BWLA_ERR_INVALID_ARG;
    st = check_device();
    if (st != BWLA_OK) return st;

    cudaStream_t s = (cudaStream_t)stream;
    const Workspace ws = workspace_layout(M, K, N, r, bits);
    char* base = (char*)workspace;
    int32_t* qsum = (int32_t*)(base + ws.qsum);
    void* Thl = base + ws.T;
    const int path = resolve_path(M, K, N, r, bits);

    int8_t* inter = (path == BWLA_PATH_I8) ? (int8_t*)(base + ws.codes) : nullptr;
    st = launch_prepare_codes(codes, M, K, inter, qsum, s);
    if (st != BWLA_OK) return st;
    if (r > 0) {
        st = launch_prologue(x_bf16, M, K, ldx, nullptr, 0, nullptr, 0, bits, nullptr, 0, nullptr, nullptr, V_bf16, r, Thl,
                             (float*)(base + ws.lr_part), (uint32_t*)(base + ws.status), s);
        if (st != BWLA_OK) return st;
    }
    GemmArgs g{};
    g.scales = scales; g.qsum = qsum; g.M = M; g.K = K; g.N = N; g.bits = bits; g.packed = packed; g.alpha = alpha;
    g.mu = mu; g.Thl = r > 0 ? Thl : nullptr; g.U = U_bf16; g.r = r; g.out = out_bf16; g.ldo = ldo; g.acc_debug = acc_debug;
    g.status = (uint32_t*)(base + ws.status);
    return run_contraction(path, g, inter ? inter : codes, s);
}

int bwla_workspace_section(int64_t M, int64_t K, int64_t N, int r, int bits, int which, size_t* offset, size_t* bytes) {
    if (!offset || !bytes || M < 0 || K <= 0 || K % 32 != 0 || N < 0 || r < 0 || !valid_bits(bits)) return BWLA_ERR_INVALID_ARG;
    const Workspace w = workspace_layout(M, K, N, r, bits);
    switch (which) {
        case BWLA_WS_SCALES: *offset = w.scales; *bytes = (size_t)M * 4; return BWLA_OK;
        case BWLA_WS_QSUM:   *offset = w.qsum;   *bytes = (size_t)M * 4 * kQsumParts; return BWLA_OK;
        case BWLA_WS_T:      *offset = w.T;      *bytes = (size_t)M * lowrank_cols(r) * 6; return BWLA_OK;
        case BWLA_WS_CODES:  *offset = w.codes;  *bytes = (size_t)M * (size_t)K; return BWLA_OK;
        case BWLA_WS_ZEROS:  *offset = w.zp;     *bytes = (size_t)M * 4; return BWLA_OK;
        default: return BWLA_ERR_INVALID_ARG;
    }
}

// ---- prepared layers -------------------------------------------------------------------------------------------

size_t bwla_layer_prepared_bytes(int64_t K, int64_t N, int n1, int n2, int r) {
    if (!valid_rotation_dims(K, n1, n2) || N < 0 || r < 0 || r > 256) return 0;
    OktGeom g;
    // the terms of the Kronecker factors for the tensor-core rotation, then the sign sums of the rows
    return (okt_geometry(n1, n2, &g) ? align_up(okt_prepared_bytes(g), 256) : 256) + align_up((size_t)N * 4, 256);
}

int bwla_layer_create(bwla_layer** layer, int64_t K, int64_t N, const float* P1, int n1, const float* P2, int n2, int bits,
                      const uint32_t* packed, const float* alpha, const float* mu, const void* U_bf16, const void* V_bf16,
                      int r, void* prepared, size_t prepared_bytes, void* stream) {
    g_launch_count = 0;
    if (!layer) return BWLA_ERR_INVALID_ARG;
    *layer = nullptr;
    if (!valid_rotation_dims(K, n1, n2) || N <= 0 || r < 0 || r > 256 || !valid_bits(bits)) return BWLA_ERR_INVALID_ARG;
    if (!P1 || !P2 || !packed || !alpha || (r > 0 && (!U_bf16 || !V_bf16))) return BWLA_ERR_INVALID_ARG;
    if (((uintptr_t)P1 & 15) || ((uintptr_t)P2 & 15) || ((uintptr_t)packed & 15)) return BWLA_ERR_INVALID_ARG;
    const size_t need = bwla_layer_prepared_bytes(K, N, n1, n2, r);
    if (!prepared || ((uintptr_t)prepared & 255) || prepared_bytes < need) return BWLA_ERR_WORKSPACE;
    int st = check_device();
    if (st != BWLA_OK) return st;
    bwla_layer* L = (bwla_layer*)malloc(sizeof(bwla_layer));
    if (!L) return BWLA_ERR_INVALID_ARG;
    L->K = K; L->N = N; L->n1 = n1; L->n2 = n2; L->bits = bits; L->r = r;
    L->P1 = P1; L->P2 = P2; L->packed = packed; L->alpha = alpha; L->mu = mu; L->U = U_bf16; L->V = V_bf16;
    L->prepared = (uint8_t*)prepared;
    L->okt = okt_geometry(n1, n2, &L->geom);
    L->asym = 0;
    L->rowsum = (int32_t*)((uint8_t*)prepared + (L->okt ? align_up(okt_prepared_bytes(L->geom), 256) : 256));
    if (L->okt) {
        st = launch_prepare_okt(L->geom, P1, P2, prepared, (cudaStream_t)stream);
        if (st != BWLA_OK) { free(L); return st; }
    }
    st = launch_row_sums(packed, N, K, L->rowsum, (cudaStream_t)stream);
    if (st != BWLA_OK) { free(L); return st; }
    *layer = L;
    return BWLA_OK;
}

void bwla_layer_destroy(bwla_layer* layer) { free(layer); }

int bwla_layer_set_activation_quant(bwla_layer* layer, int mode) {
    if (!layer || (mode != BWLA_ACT_SYMMETRIC && mode != BWLA_ACT_ASYMMETRIC)) return BWLA_ERR_INVALID_ARG;
    if (mode == BWLA_ACT_ASYMMETRIC && !layer->okt) return BWLA_ERR_UNSUPPORTED;   // only the tensor-core rotation has it
    layer->asym = mode;
    return BWLA_OK;
}

int bwla_layer_rotate_quant_asym(const bwla_layer* L, const void* x_bf16, int64_t M, int64_t ldx, uint8_t* codes, float* scales,
                                 int32_t* zeros, float* y_f32, void* stream) {
    g_launch_count = 0;
    if (!L || M < 0 || ldx < L->K) return BWLA_ERR_INVALID_ARG;
    if (M == 0) return BWLA_OK;
    if (!x_bf16 || !codes || !scales || !zeros || ((uintptr_t)codes & 15)) return BWLA_ERR_INVALID_ARG;
    int st = check_device();
    if (st != BWLA_OK) return st;
    if (!L->okt || !okt_accepts_x(x_bf16, ldx)) return BWLA_ERR_UNSUPPORTED;
    // the kernel keeps u - 2^(b-1) so that codes fit int8; the bias puts u and the zero point back in [0, 2^b - 1]
    OktProblem pr{L->prepared, (int8_t*)codes, 0, zeros, 1 << (L->bits - 1), scales, nullptr, y_f32};
    return launch_okt(L->geom, x_bf16, M, ldx, L->bits, 1, 1, &pr, nullptr, nullptr, (cudaStream_t)stream);
}

int bwla_layer_rotate_quant(const bwla_layer* L, const void* x_bf16, int64_t M, int64_t ldx, int8_t* codes, float* scales,
                            float* y_f32, void* stream) {
    g_launch_count = 0;
    if (!L || M < 0 || ldx < L->K) return BWLA_ERR_INVALID_ARG;
    if (M == 0) return BWLA_OK;
    if (!x_bf16 || !codes || !scales || ((uintptr_t)codes & 15)) return BWLA_ERR_INVALID_ARG;
    int st = check_device();
    if (st != BWLA_OK) return st;
    if (L->okt && g_forced_rotation != BWLA_ROT_SIMT && okt_accepts_x(x_bf16, ldx)) {
        OktProblem pr{L->prepared, codes, 0, nullptr, 0, scales, nullptr, y_f32};
        return launch_okt(L->geom, x_bf16, M, ldx, L->bits, 0, 1, &pr, nullptr, nullptr, (cudaStream_t)stream);
    }
    if (y_f32) return BWLA_ERR_UNSUPPORTED;      // only the tensor-core kernel can hand out Y
    return launch_prologue(x_bf16, M, L->K, ldx, L->P1, L->n1, L->P2, L->n2, L->bits, codes, 0, scales, nullptr, nullptr, 0,
                           nullptr, nullptr, nullptr, (cudaStream_t)stream);
}

struct A16Workspace { size_t status, Y, yhat, ysum, codes, scales, T, lr_part, total; };
static A16Workspace a16_layout(const bwla_layer* L, int64_t M) {
    A16Workspace w{};
    size_t off = 0;
    w.status = off; off += kStatusBytes;
    w.Y = off;      off += align_up((size_t)M * (size_t)L->K * 4, 256);
    w.yhat = off;   off += align_up((size_t)M * (size_t)L->K * 2, 256);
    w.ysum = off;   off += align_up((size_t)M * 4, 256);
    w.codes = off;  off += align_up((size_t)M * (size_t)L->K, 256);
    w.scales = off; off += align_up((size_t)M * 4, 256);
    const size_t lr_cols = (size_t)lowrank_cols(L->r);
    w.T = off;      off += align_up((size_t)M * lr_cols * 6, 256);
    w.lr_part = off; off += L->r > 0 ? align_up(std::max((size_t)kLrKSplitMax * 16 * lr_cols * 4, lowrank_umma_part_bytes(M, L->K, L->r)), 256) : 0;
    w.total = off;
    return w;
}

size_t bwla_w1a16_workspace_bytes(const bwla_layer* layer, int64_t M) {
    if (!layer || M < 0) return 0;
    return a16_layout(layer, M).total;
}

int bwla_layer_w1a16_linear(const bwla_layer* L, const void* x_bf16, int64_t M, int64_t ldx, void* out_bf16, int64_t ldo,
                            void* workspace, size_t workspace_bytes, void* stream) {
    g_launch_count = 0;
    if (!L || M < 0 || ldx < L->K || ldo < L->N) return BWLA_ERR_INVALID_ARG;
    if (M == 0) return BWLA_OK;
    if (!x_bf16 || !out_bf16) return BWLA_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < bwla_w1a16_workspace_bytes(L, M)) return BWLA_ERR_WORKSPACE;
    int st = check_device();
    if (st != BWLA_OK) return st;
    if (!L->okt || !okt_accepts_x(x_bf16, ldx) || !a16_supports(M, L->K, L->N, L->r)) return BWLA_ERR_UNSUPPORTED;
    cudaStream_t s = (cudaStream_t)stream;
    const A16Workspace w = a16_layout(L, M);
    char* base = (char*)workspace;
    uint32_t* status = (uint32_t*)(base + w.status);
    // the rotation hands out Y in fp32 (its int8 codes, quantised at 8 bits, are a by-product nobody reads here)
    OktProblem pr{L->prepared, (int8_t*)(base + w.codes), 0, nullptr, 0, (float*)(base + w.scales), nullptr, (float*)(base + w.Y)};
    OktLowrank lr{L->V, L->r, base + w.T, L->r > 0 ? (float*)(base + w.lr_part) : nullptr, status + kLrCounterWord};
    st = launch_okt(L->geom, x_bf16, M, ldx, 8, 0, 1, &pr, &lr, status, s);
    if (st != BWLA_OK) return st;
    st = launch_y_to_bf16((const float*)(base + w.Y), M, L->K, base + w.yhat, (float*)(base + w.ysum), s);
    if (st != BWLA_OK) return st;
    return launch_gemm_a16(base + w.yhat, (const float*)(base + w.ysum), M, L->K, L->N, L->packed, L->alpha, L->mu, L->U, L->r,
                           L->r > 0 ? base + w.T : nullptr, out_bf16, ldo, status, s);
}

static bool valid_group(const bwla_layer* const* layers, int count) {
    if (!layers || count < 1 || count > kOktMaxProblems) return false;
    for (int i = 0; i < count; ++i) {
        if (!layers[i]) return false;
        if (layers[i]->K != layers[0]->K || layers[i]->n1 != layers[0]->n1 || layers[i]->n2 != layers[0]->n2 ||
            layers[i]->bits != layers[0]->bits || layers[i]->asym != layers[0]->asym)
            return false;
    }
    return true;
}

size_t bwla_group_workspace_bytes(const bwla_layer* const* layers, int count, int64_t M) {
    if (!valid_group(layers, count) || M < 0) return 0;
    size_t total = 0;
    for (int i = 0; i < count; ++i) total += workspace_layout(M, layers[i]->K, layers[i]->N, layers[i]->r, layers[i]->bits, false).total;
    return total;
}

int bwla_w1ax_linear_group(const bwla_layer* const* layers, int count, const void* x_bf16, int64_t M, int64_t ldx,
                           void* const* outs, const int64_t* ldos, void* workspace, size_t workspace_bytes, void* stream) {
    g_launch_count = 0;
    if (!valid_group(layers, count) || M < 0 || !outs || !ldos || ldx < layers[0]->K) return BWLA_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i)
        if (ldos[i] < layers[i]->N || (M > 0 && !outs[i])) return BWLA_ERR_INVALID_ARG;
    if (M == 0) return BWLA_OK;
    if (!x_bf16) return BWLA_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < bwla_group_workspace_bytes(layers, count, M))
        return BWLA_ERR_WORKSPACE;
    int st = check_device();
    if (st != BWLA_OK) return st;

    cudaStream_t s = (cudaStream_t)stream;
    const bwla_layer* L0 = layers[0];
    char* base = (char*)workspace;
    // The status words of the whole call are the first layer's: only those 256 bytes start at zero.  Layer i keeps its
    // arrival counters for split sums of T in words 4 + 8 i .. 11 + 8 i of them.
    uint32_t* status = (uint32_t*)base;
    Workspace ws[kOktMaxProblems];
    char* wbase[kOktMaxProblems];
    int path[kOktMaxProblems];
    size_t off = 0;
    for (int i = 0; i < count; ++i) {
        ws[i] = workspace_layout(M, layers[i]->K, layers[i]->N, layers[i]->r, layers[i]->bits, false);
        wbase[i] = base + off;
        off += ws[i].total;
        path[i] = resolve_path(M, layers[i]->K, layers[i]->N, layers[i]->r, layers[i]->bits);
    }
    bool okt = g_forced_rotation != BWLA_ROT_SIMT && okt_accepts_x(x_bf16, ldx);
    for (int i = 0; i < count; ++i) okt = okt && layers[i]->okt;
    if (L0->asym && !okt) return BWLA_ERR_UNSUPPORTED;     // the asymmetric quantiser lives in the tensor-core rotation
    if (okt) {
        OktProblem pr[kOktMaxProblems];
        OktLowrank lr[kOktMaxProblems];
        for (int i = 0; i < count; ++i) {
            const bwla_layer* L = layers[i];
            pr[i] = OktProblem{L->prepared, (int8_t*)(wbase[i] + ws[i].codes), path[i] == BWLA_PATH_I8 ? 1 : 0,
                               L->asym ? (int32_t*)(wbase[i] + ws[i].zp) : nullptr, 0,
                               (float*)(wbase[i] + ws[i].scales), (int32_t*)(wbase[i] + ws[i].qsum), nullptr};
            lr[i] = OktLowrank{L->V, L->r, wbase[i] + ws[i].T, L->r > 0 ? (float*)(wbase[i] + ws[i].lr_part) : nullptr,
                               status + 8 * i + kLrCounterWord};
        }
        st = launch_okt(L0->geom, x_bf16, M, ldx, L0->bits, L0->asym, count, pr, lr, status, s);
        if (st != BWLA_OK) return st;
    } else {
        for (int i = 0; i < count; ++i) {
            const bwla_layer* L = layers[i];
            st = launch_prologue(x_bf16, M, L->K, ldx, L->P1, L->n1, L->P2, L->n2, L->bits, (int8_t*)(wbase[i] + ws[i].codes),
                                 path[i] == BWLA_PATH_I8 ? 1 : 0, (float*)(wbase[i] + ws[i].scales),
                                 (int32_t*)(wbase[i] + ws[i].qsum), L->V, L->r, wbase[i] + ws[i].T,
                                 L->r > 0 ? (float*)(wbase[i] + ws[i].lr_part) : nullptr, status + 8 * i, s);
            if (st != BWLA_OK) return st;
        }
    }
    // Several contractions that all go to the small-batch tensor-core kernel run beside one another (GemmArgs::dep_mode).
    bool siblings = count > 1 && M <= 64;
    for (int i = 0; i < count; ++i) siblings = siblings && path[i] == BWLA_PATH_I8;
    // each sibling plans for its share of the SMs (by row tiles) when all of them fit the device at once
    int64_t tiles_total = 0;
    for (int i = 0; i < count; ++i) tiles_total += (layers[i]->N + 127) / 128;
    const int sms_all = sm_count();
    const bool share = siblings && tiles_total <= sms_all;
    for (int i = 0; i < count; ++i) {
        const bwla_layer* L = layers[i];
        GemmArgs g{};
        g.scales = (float*)(wbase[i] + ws[i].scales); g.qsum = (int32_t*)(wbase[i] + ws[i].qsum);
        g.M = M; g.K = L->K; g.N = L->N; g.bits = L->bits; g.packed = L->packed; g.alpha = L->alpha; g.mu = L->mu;
        g.zp = L->asym ? (int32_t*)(wbase[i] + ws[i].zp) : nullptr; g.rowsum = L->rowsum;
        g.Thl = L->r > 0 ? wbase[i] + ws[i].T : nullptr; g.U = L->U; g.r = L->r; g.out = outs[i]; g.ldo = ldos[i];
        g.acc_debug = nullptr; g.status = status;
        g.dep_mode = siblings ? (i == 0 ? kDepHead : kDepSibling) : kDepChain;
        g.sm_budget = share ? (int)(((int64_t)sms_all * ((L->N + 127) / 128)) / tiles_total) : 0;
        st = run_contraction(path[i], g, (int8_t*)(wbase[i] + ws[i].codes), s);
        if (st != BWLA_OK) return st;
    }
    return BWLA_OK;
}

int bwla_check_status(void* workspace, void* stream) {
    if (!workspace) return BWLA_ERR_INVALID_ARG;
    uint32_t host[4] = {0, 0, 0, 0};
    cudaStream_t s = (cudaStream_t)stream;
    BWLA_CUDA_TRY(cudaMemcpyAsync(host, workspace, sizeof(host), cudaMemcpyDeviceToHost, s));
    BWLA_CUDA_TRY(cudaStreamSynchronize(s));
    if (host[0] != 0) {
        BWLA_CUDA_TRY(cudaMemsetAsync(workspace, 0, kStatusBytes, s));
        BWLA_CUDA_TRY(cudaStreamSynchronize(s));
        return BWLA_ERR_DEVICE_TIMEOUT;
    }
    return BWLA_OK;
}

int bwla_force_path(int path) {
    if (path < BWLA_PATH_AUTO || path > BWLA_PATH_I8) return BWLA_ERR_INVALID_ARG;
    g_forced_path = path;
    return BWLA_OK;
}

int bwla_force_rotation(int which) {
    if (which < BWLA_ROT_AUTO || which > BWLA_ROT_UMMA) return BWLA_ERR_INVALID_ARG;
    g_forced_rotation = which;
    return BWLA_OK;
}

int bwla_chosen_path(int64_t M, int64_t K, int64_t N, int r, int bits) { return resolve_path(M, K, N, r, bits); }

int bwla_last_launch_count(void) { return g_launch_count; }

int bwla_profile_enable(int on) {
    g_prof_on = on != 0;
    return BWLA_OK;
}

int bwla_profile_collect(float* ms_by_kind, int* launches_by_kind) {
    if (!ms_by_kind || !launches_by_kind) return BWLA_ERR_INVALID_ARG;
    for (int i = 0; i < kProfKinds; ++i) { ms_by_kind[i] = 0.f; launches_by_kind[i] = 0; }
    if (!g_prof) return BWLA_OK;
    int st = BWLA_OK;
    for (auto& p : *g_prof) {
        float ms = 0.f;
        cudaError_t e = cudaEventSynchronize(p.b);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, p.a, p.b);
        if (e == cudaSuccess && p.kind >= 0 && p.kind < kProfKinds) { ms_by_kind[p.kind] += ms; launches_by_kind[p.kind] += 1; }
        else if (e != cudaSuccess) st = cuda_fail(e);
        g_prof_pool->push_back(p);
    }
    g_prof->clear();
    return st;
}

int bwla_last_cuda_error(void) { return g_last_cuda_error; }

const char* bwla_status_string(int status) {
    switch (status) {
        case BWLA_OK: return "BWLA_OK";
        case BWLA_ERR_INVALID_ARG: return "BWLA_ERR_INVALID_ARG";
        case BWLA_ERR_UNSUPPORTED: return "BWLA_ERR_UNSUPPORTED";
        case BWLA_ERR_WORKSPACE: return "BWLA_ERR_WORKSPACE";
        case BWLA_ERR_CUDA: return "BWLA_ERR_CUDA";
        case BWLA_ERR_DEVICE_TIMEOUT: return "BWLA_ERR_DEVICE_TIMEOUT";
        case BWLA_ERR_STATIC_SCRATCH: return "BWLA_ERR_STATIC_SCRATCH";
        default: return "BWLA_ERR_UNKNOWN";
    }
}

}  // extern "C"
