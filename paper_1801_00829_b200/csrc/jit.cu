// Run-time specialisation of Cell / MAgg chains: the analogue of the paper's
// template expansion to source code, compilation and plan cache (Section 2.1,
// "Codegen Architecture").  A chain that has no built-in specialisation is
// written out as a straight-line C++ functor, placed into the same flat
// streaming kernel the library compiles ahead of time (cell_flat.cuh), compiled
// for the current device with NVRTC and cached by the chain's translated program.
// NVRTC and the driver API are looked up with dlopen at first use; if either is
// missing, or a compilation fails, the caller falls back to the interpreter.
#include <dlfcn.h>
#include <stdio.h>

#include <atomic>
#include <mutex>
#include <string>
#include <unordered_map>
#include <vector>

#include "jit.h"
#include "outer_kernels.cuh"
#include "row_kernels.cuh"

namespace fo {

namespace {

const char kSkeleton[] =
#include "jit_source.inc"
    ;
const char kSkeletonOuter[] =
#include "jit_source_outer.inc"
    ;
const char kSkeletonRow[] =
#include "jit_source_row.inc"
    ;

// ---- the few NVRTC / driver entry points used, declared here so that neither
// library is needed at link time
typedef struct _nvrtcProgram *nvrtcProgram;
typedef int (*nvrtcCreateProgram_t)(nvrtcProgram *, const char *, const char *, int, const char *const *,
                                    const char *const *);
typedef int (*nvrtcCompileProgram_t)(nvrtcProgram, int, const char *const *);
typedef int (*nvrtcGetSize_t)(nvrtcProgram, size_t *);
typedef int (*nvrtcGetData_t)(nvrtcProgram, char *);
typedef int (*nvrtcDestroyProgram_t)(nvrtcProgram *);
typedef struct CUmod_st *CUmodule;
typedef struct CUfunc_st *CUfunction;
typedef int (*cuModuleLoadData_t)(CUmodule *, const void *);
typedef int (*cuModuleGetFunction_t)(CUfunction *, CUmodule, const char *);
typedef int (*cuLaunchKernel_t)(CUfunction, unsigned, unsigned, unsigned, unsigned, unsigned, unsigned,
                                unsigned, void *, void **, void **);
typedef struct CUctx_st *CUcontext;
typedef int (*cuCtxGetCurrent_t)(CUcontext *);
typedef int (*cuOccupancy_t)(int *, CUfunction, int, size_t);
typedef int (*cuFuncSetAttribute_t)(CUfunction, int, int);

struct Api {
    bool nvrtc_ok = false, driver_ok = false;
    nvrtcCreateProgram_t create = nullptr;
    nvrtcCompileProgram_t compile = nullptr;
    nvrtcGetSize_t cubin_size = nullptr, log_size = nullptr;
    nvrtcGetData_t cubin = nullptr, log = nullptr;
    nvrtcDestroyProgram_t destroy = nullptr;
    cuModuleLoadData_t load = nullptr;
    cuModuleGetFunction_t getfn = nullptr;
    cuLaunchKernel_t launch = nullptr;
    cuCtxGetCurrent_t ctx = nullptr;
    cuOccupancy_t occupancy = nullptr;
    cuFuncSetAttribute_t setattr = nullptr;
};

void *open_first(const char *const *names)
{
    for (; *names; ++names) {
        void *h = dlopen(*names, RTLD_NOW | RTLD_GLOBAL);
        if (h) return h;
    }
    return nullptr;
}

Api &api()
{
    static Api a;
    static std::once_flag once;
    std::call_once(once, [] {
        const char *nv[] = {"libnvrtc.so.12", "libnvrtc.so", "/usr/local/cuda/lib64/libnvrtc.so.12",
                            "/usr/local/cuda/lib64/libnvrtc.so", nullptr};
        if (void *h = open_first(nv)) {
            a.create = (nvrtcCreateProgram_t)dlsym(h, "nvrtcCreateProgram");
            a.compile = (nvrtcCompileProgram_t)dlsym(h, "nvrtcCompileProgram");
            a.cubin_size = (nvrtcGetSize_t)dlsym(h, "nvrtcGetCUBINSize");
            a.cubin = (nvrtcGetData_t)dlsym(h, "nvrtcGetCUBIN");
            a.log_size = (nvrtcGetSize_t)dlsym(h, "nvrtcGetProgramLogSize");
            a.log = (nvrtcGetData_t)dlsym(h, "nvrtcGetProgramLog");
            a.destroy = (nvrtcDestroyProgram_t)dlsym(h, "nvrtcDestroyProgram");
            a.nvrtc_ok = a.create && a.compile && a.cubin_size && a.cubin && a.log_size && a.log && a.destroy;
        }
        const char *cu[] = {"libcuda.so.1", "libcuda.so", nullptr};
        if (void *h = open_first(cu)) {
            a.load = (cuModuleLoadData_t)dlsym(h, "cuModuleLoadData");
            a.getfn = (cuModuleGetFunction_t)dlsym(h, "cuModuleGetFunction");
            a.launch = (cuLaunchKernel_t)dlsym(h, "cuLaunchKernel");
            a.ctx = (cuCtxGetCurrent_t)dlsym(h, "cuCtxGetCurrent");
            a.occupancy = (cuOccupancy_t)dlsym(h, "cuOccupancyMaxActiveBlocksPerMultiprocessor");
            a.setattr = (cuFuncSetAttribute_t)dlsym(h, "cuFuncSetAttribute");
            a.driver_ok = a.load && a.getfn && a.launch && a.ctx;
        }
    });
    return a;
}

std::mutex g_mutex;
// key: context + translated program.  A function handle belongs to the context it
// was loaded in, so a new context (after a device reset, say) starts empty.
std::unordered_map<std::string, CUfunction> g_cache;
std::unordered_map<std::string, int> g_load_failures;     // module loads that failed, per key
std::atomic<int> g_mode{1};                               // 0 off, 1 compile at first use, 2 prepared kernels only
int g_compiled = 0, g_launches = 0, g_failures = 0;
constexpr int kLoadRetries = 3;                           // a failed load (out of memory, say) is tried again this often
std::string g_last_log;

// ---- source generation
std::string operand_text(int opnd)
{
    char buf[32];
    if (opnd & 0x80) snprintf(buf, sizeof(buf), "c[%d]", opnd & 0x7f);
    else snprintf(buf, sizeof(buf), "R%d", opnd);
    return buf;
}

std::string op_text(const DevOp &op)
{
    const std::string a = operand_text(op.a), b = operand_text(op.b), c = operand_text(op.c);
    switch (op.opcode) {
        case FO_OP_MOV: return a;
        case FO_OP_NEG: return "-" + a;
        case FO_OP_ABS: return "fabs(" + a + ")";
        case FO_OP_SQRT: return "sqrt(" + a + ")";
        case FO_OP_EXP: return "exp(" + a + ")";
        case FO_OP_LOG: return "log(" + a + ")";
        case FO_OP_SQ: return a + " * " + a;
        case FO_OP_ADD: return a + " + " + b;
        case FO_OP_SUB: return a + " - " + b;
        case FO_OP_MUL: return a + " * " + b;
        case FO_OP_DIV: return a + " / " + b;
        case FO_OP_MIN: return "fmin(" + a + ", " + b + ")";
        case FO_OP_MAX: return "fmax(" + a + ", " + b + ")";
        case FO_OP_POW: return "pow(" + a + ", " + b + ")";
        case FO_OP_EQ: return a + " == " + b + " ? 1.0 : 0.0";
        case FO_OP_NE: return a + " != " + b + " ? 1.0 : 0.0";
        case FO_OP_LT: return a + " < " + b + " ? 1.0 : 0.0";
        case FO_OP_LE: return a + " <= " + b + " ? 1.0 : 0.0";
        case FO_OP_GT: return a + " > " + b + " ? 1.0 : 0.0";
        case FO_OP_GE: return a + " >= " + b + " ? 1.0 : 0.0";
        case FO_OP_SEL: return a + " != 0.0 ? " + b + " : " + c;
        case FO_OP_FMA: return "fma(" + a + ", " + b + ", " + c + ")";
        default: return "0.0";
    }
}

// The wrapper kernel of one kernel instance: which skeleton, with which template arguments.
std::string wrapper_text(const DevChain &ch, const JitSpec &sp)
{
    char buf[512];
    const char *tf[2] = {"false", "true"};
    switch (sp.kind) {
        case kJitFlat:          // a = STORE
            snprintf(buf, sizeof(buf), "fo::cell_flat_body<fo::EvalFn<JitFn>, %d, %s>(ch, p);", ch.n_out, tf[sp.a & 1]);
            break;
        case kJitRows:          // a = AGG, b = ALIGNED
            snprintf(buf, sizeof(buf), "fo::cell_rows_body<fo::EvalFn<JitFn>, %d, %d, %s>(ch, p);", ch.n_out, sp.a,
                     tf[sp.b & 1]);
            break;
        case kJitCols:          // a = ALIGNED
            snprintf(buf, sizeof(buf), "fo::cell_cols_body<fo::EvalFn<JitFn>, %s>(ch, p);", tf[sp.a & 1]);
            break;
        case kJitCsr:           // a = lanes per row
            snprintf(buf, sizeof(buf), "fo::cell_csr_body<fo::EvalFn<JitFn>, %d, %d>(ch, p);", ch.n_out, sp.a);
            break;
        case kJitOuterDirect:   // a = NK2, b = AGG, c = ALIGNED
            snprintf(buf, sizeof(buf), "fo::outer_body<%d, %d, %s>(ch, p);", sp.a, sp.b, tf[sp.c & 1]);
            break;
        case kJitOuterPipe:     // a = NK2, b = AGG
            snprintf(buf, sizeof(buf), "fo::outer_pipe_body<%d, %d, true>(ch, p);", sp.a, sp.b);
            break;
        case kJitOuterBulk:     // a = NK2, b = AGG
            snprintf(buf, sizeof(buf), "fo::outer_bulk_body<%d, %d, 0>(ch, p);", sp.a, sp.b);
            break;
        case kJitOuterDense:    // a = AGG
            snprintf(buf, sizeof(buf), "fo::outer_dense_body<%d>(ch, p, sp);", sp.a);
            break;
        case kJitRowDense:      // a = NCH, b = W, c = R, d = AGG, e = STAGED
            snprintf(buf, sizeof(buf), "fo::row_dense_body<%d, %d, %d, %d, %s>(ch, p);", sp.a, sp.b, sp.c, sp.d,
                     tf[sp.e & 1]);
            break;
        case kJitRowNarrow:     // a = NC, b = AGG, c = VEC
            snprintf(buf, sizeof(buf), "fo::row_narrow_body<%d, %d, %s>(ch, p);", sp.a, sp.b, tf[sp.c & 1]);
            break;
        case kJitRowCsr:        // a = G
            snprintf(buf, sizeof(buf), "fo::row_csr_body<%d, true>(ch, p);", sp.a);
            break;
        default:                // kJitRowCsrReg: a = AGG, b = G
            snprintf(buf, sizeof(buf), "fo::row_csr_reg_body<%d, %d, true>(ch, p);", sp.a, sp.b);
            break;
    }
    return buf;
}

bool is_outer(const JitSpec &sp) { return (sp.kind >= kJitOuterDirect && sp.kind <= kJitOuterDense) || sp.kind == kJitOuterBulk; }
bool is_row(const JitSpec &sp) { return sp.kind >= kJitRowDense && sp.kind <= kJitRowCsrReg; }

// The chain as a straight-line functor: in[] holds the input registers (Cell: a, sides;
// Outer: a, d, sides), c the constant table, o the results.
std::string functor_text(const DevChain &ch)
{
    char buf[512];
    std::string s = "struct JitFn {\n";
    snprintf(buf, sizeof(buf), "    static constexpr unsigned kSideMask = %uu;\n    static constexpr int kOut = %d;\n",
             ch.side_used, ch.n_out);
    s += buf;
    s += "    __device__ __forceinline__ static void eval(const double *in, const double *c, double *o)\n    {\n";
    for (int r = 0; r < ch.tmp_base; ++r) {
        snprintf(buf, sizeof(buf), "        const double R%d = in[%d];\n", r, r);
        s += buf;
    }
    for (int r = ch.tmp_base; r < ch.n_regs; ++r) {
        snprintf(buf, sizeof(buf), "        double R%d;\n", r);
        s += buf;
    }
    for (int k = 0; k < ch.n_ops; ++k) {
        snprintf(buf, sizeof(buf), "        R%d = ", ch.ops[k].dst);
        s += buf;
        s += op_text(ch.ops[k]) + ";\n";
    }
    for (int k = 0; k < ch.n_out; ++k) {
        snprintf(buf, sizeof(buf), "        o[%d] = ", k);
        s += buf;
        s += operand_text(ch.out[k]) + ";\n";
    }
    s += "        (void)c; (void)in;\n    }\n};\n";
    return s;
}

std::string generate_source(const DevChain &ch, const JitSpec &sp)
{
    char buf[1024];
    std::string s;
    // what the system headers and fusedops.h provide in the ahead-of-time build
    snprintf(buf, sizeof(buf),
             "typedef unsigned char uint8_t;\ntypedef int int32_t;\ntypedef unsigned int uint32_t;\n"
             "#define FO_MAX_OPS %d\n#define FO_MAX_TMPS %d\n#define FO_MAX_SIDES %d\n"
             "#define FO_MAX_SCALARS %d\n#define FO_MAX_OUT %d\n"
             "enum { FO_AT_CELL = %d, FO_AT_ROW = %d, FO_AT_COL = %d };\n"
             "enum { FO_CELL_NO_AGG = %d, FO_CELL_ROW_AGG = %d, FO_CELL_COL_AGG = %d, FO_CELL_FULL_AGG = %d };\n",
             FO_MAX_OPS, FO_MAX_TMPS, FO_MAX_SIDES, FO_MAX_SCALARS, FO_MAX_OUT, (int)FO_AT_CELL, (int)FO_AT_ROW,
             (int)FO_AT_COL, (int)FO_CELL_NO_AGG, (int)FO_CELL_ROW_AGG, (int)FO_CELL_COL_AGG, (int)FO_CELL_FULL_AGG);
    s += buf;
    if (is_outer(sp)) {
        // the Outer kernels call the functor from inside: it comes first
        s += "#define FO_JIT_OUTER 1\n";
        s += functor_text(ch);
        s += kSkeletonOuter;
        snprintf(buf, sizeof(buf),
                 "static_assert(sizeof(fo::DevChain) == %zu, \"chain layout\");\n"
                 "static_assert(sizeof(fo::OuterParams) == %zu, \"parameter layout\");\n"
                 "static_assert(sizeof(fo::DenseSplit) == %zu, \"parameter layout\");\n",
                 sizeof(DevChain), sizeof(OuterParams), sizeof(DenseSplit));
        s += buf;
        snprintf(buf, sizeof(buf),
                 "extern \"C\" __global__ void __launch_bounds__(%d, %d)\n"
                 "fo_jit_kernel(const __grid_constant__ fo::DevChain ch, const __grid_constant__ fo::OuterParams p%s)\n"
                 "{\n    ", sp.kind == kJitOuterBulk ? kBulkWarps * 32 : sp.kind == kJitOuterDense ? kDenseThreadsAll : kThreads,
                 (sp.kind == kJitOuterBulk || sp.kind == kJitOuterDense || (sp.kind == kJitOuterDirect && sp.a > 8)) ? 1 : 2,
                 sp.kind == kJitOuterDense ? ", const __grid_constant__ fo::DenseSplit sp" : "");
        s += buf;
        s += wrapper_text(ch, sp) + "\n}\n";
        return s;
    }
    if (is_row(sp)) {
        // the Row kernels call the functor from inside as well
        s += "#define FO_JIT_ROW 1\n";
        s += functor_text(ch);
        s += kSkeletonRow;
        snprintf(buf, sizeof(buf),
                 "static_assert(sizeof(fo::DevChain) == %zu, \"chain layout\");\n"
                 "static_assert(sizeof(fo::RowParams) == %zu, \"parameter layout\");\n",
                 sizeof(DevChain), sizeof(RowParams));
        s += buf;
        if (sp.kind == kJitRowDense)
            snprintf(buf, sizeof(buf), "extern \"C\" __global__ void __launch_bounds__(%d, 1)\n", kDenseBlock);
        else if (sp.kind == kJitRowNarrow)
            snprintf(buf, sizeof(buf), "extern \"C\" __global__ void __launch_bounds__(%d)\n", kThreads);
        else
            snprintf(buf, sizeof(buf), "extern \"C\" __global__ void __launch_bounds__(%d, 3)\n", kThreads);
        s += buf;
        s += "fo_jit_kernel(const __grid_constant__ fo::DevChain ch, const __grid_constant__ fo::RowParams p)\n{\n    ";
        s += wrapper_text(ch, sp) + "\n}\n";
        return s;
    }
    s += kSkeleton;
    snprintf(buf, sizeof(buf),
             "static_assert(sizeof(fo::DevChain) == %zu, \"chain layout\");\n"
             "static_assert(sizeof(fo::CellParams) == %zu, \"parameter layout\");\n"
             "static_assert(sizeof(fo::CsrCellParams) == %zu, \"parameter layout\");\n",
             sizeof(DevChain), sizeof(CellParams), sizeof(CsrCellParams));
    s += buf;
    s += functor_text(ch);
    snprintf(buf, sizeof(buf),
             "extern \"C\" __global__ void __launch_bounds__(%d)\n"
             "fo_jit_kernel(const __grid_constant__ fo::DevChain ch, const __grid_constant__ fo::%s p)\n"
             "{\n    ", kThreads, sp.kind == kJitCsr ? "CsrCellParams" : "CellParams");
    s += buf;
    s += wrapper_text(ch, sp) + "\n}\n";
    return s;
}

std::string cache_key(const DevChain &ch, const JitSpec &sp, CUcontext ctx)
{
    std::string k;
    k.append((const char *)&ctx, sizeof(ctx));
    k.append((const char *)&sp, sizeof(sp));
    k.append((const char *)&ch.n_ops, sizeof(int32_t));
    k.append((const char *)&ch.n_out, sizeof(int32_t));
    k.append((const char *)&ch.n_regs, sizeof(int32_t));
    k.append((const char *)&ch.tmp_base, sizeof(int32_t));
    k.append((const char *)&ch.side_used, sizeof(uint32_t));
    k.append((const char *)ch.out, sizeof(ch.out));
    k.append((const char *)ch.ops, sizeof(DevOp) * (size_t)ch.n_ops);
    return k;
}

// Compiles `src` for `arch`; returns the CUBIN (empty on failure, log in g_last_log).
std::vector<char> compile(const std::string &src, const std::string &arch)
{
    std::vector<char> cubin;
    Api &a = api();
    nvrtcProgram prog = nullptr;
    if (a.create(&prog, src.c_str(), "fo_jit.cu", 0, nullptr, nullptr) != 0) {
        g_last_log = "nvrtcCreateProgram failed";
        return cubin;
    }
    const std::string archopt = "--gpu-architecture=" + arch;
    const char *opts[] = {archopt.c_str(), "--std=c++17", "--fmad=false"};
    const int rc = a.compile(prog, 3, opts);
    size_t n = 0;
    if (a.log_size(prog, &n) == 0 && n > 1) {
        g_last_log.resize(n);
        a.log(prog, &g_last_log[0]);
    } else {
        g_last_log.clear();
    }
    if (rc == 0 && a.cubin_size(prog, &n) == 0 && n > 0) {
        cubin.resize(n);
        if (a.cubin(prog, cubin.data()) != 0) cubin.clear();
    }
    a.destroy(&prog);
    return cubin;
}

}  // namespace

bool jit_enabled() { return g_mode.load() != 0; }
bool jit_first_use() { return g_mode.load() == 1; }

namespace {

// The cached kernel of (ch, store) in the current context; compiles and loads it
// first if `may_compile` and it is not there yet.  nullptr if there is none.
// *status (optional): FO_OK, FO_ERR_UNSUPPORTED (no compiler / driver library /
// context) or FO_ERR_CHAIN (the compilation or the load failed).
CUfunction find_kernel(const DevChain &ch, const JitSpec &sp, bool may_compile, std::string *key_out, int *status)
{
    Api &a = api();
    if (status) *status = FO_ERR_UNSUPPORTED;
    if (!a.nvrtc_ok || !a.driver_ok) return nullptr;
    int dev = 0, major = 0, minor = 0;
    // the runtime calls make sure the primary context exists and is current
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess)
        return nullptr;
    CUcontext ctx = nullptr;
    if (a.ctx(&ctx) != 0 || !ctx) {
        if (!may_compile || cudaFree(nullptr) != cudaSuccess || a.ctx(&ctx) != 0 || !ctx) return nullptr;
    }
    CUfunction fn = nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    const std::string key = cache_key(ch, sp, ctx);
    if (key_out) *key_out = key;
    auto it = g_cache.find(key);
    if (it != g_cache.end()) {
        if (status) *status = it->second ? FO_OK : FO_ERR_CHAIN;
        return it->second;
    }
    if (!may_compile) return nullptr;
    if (status) *status = FO_ERR_CHAIN;
    auto lf = g_load_failures.find(key);
    if (lf != g_load_failures.end() && lf->second >= kLoadRetries) return nullptr;
    char arch[32];
    snprintf(arch, sizeof(arch), "sm_%d%d%s", major, minor, major >= 9 ? "a" : "");
    const std::vector<char> cubin = compile(generate_source(ch, sp), arch);
    if (cubin.empty()) {
        ++g_failures;
        g_cache.emplace(key, nullptr);        // the same source fails the same way: not compiled again
        return nullptr;
    }
    CUmodule mod = nullptr;
    if (a.load(&mod, cubin.data()) != 0 || a.getfn(&fn, mod, "fo_jit_kernel") != 0) {
        ++g_failures;
        ++g_load_failures[key];               // may be transient: tried again a few times, then given up
        return nullptr;
    }
    ++g_compiled;
    g_cache.emplace(key, fn);
    if (status) *status = FO_OK;
    return fn;
}

}  // namespace

int jit_launch(const JitSpec &sp, const DevChain &ch, const void *params, unsigned grid_x, unsigned grid_y,
               cudaStream_t st, bool may_compile, bool launch, size_t smem, const void *params2, unsigned block)
{
    const int mode = g_mode.load();
    if (mode == 0) return kJitUnavailable;
    std::string key;
    CUfunction fn = find_kernel(ch, sp, may_compile, &key, nullptr);
    if (!fn) return kJitUnavailable;
    if (!launch) return FO_OK;
    if (smem > 48u * 1024u) {
        // CU_FUNC_ATTRIBUTE_MAX_DYNAMIC_SHARED_SIZE_BYTES
        const int arc = api().setattr ? api().setattr(fn, 8, (int)smem) : 1;
        if (arc != 0) return kJitUnavailable;
    }
    void *args[3] = {(void *)&ch, (void *)params, (void *)params2};
    const int rc = api().launch(fn, grid_x, grid_y, 1, block, 1, 1, (unsigned)smem, (void *)st, args, nullptr);
    if (rc == 0) {
        std::lock_guard<std::mutex> lock(g_mutex);
        ++g_launches;
        return FO_OK;
    }
    // CUDA_ERROR_INVALID_CONTEXT (201), CUDA_ERROR_INVALID_HANDLE (400), CUDA_ERROR_NOT_FOUND (500):
    // the handle no longer belongs to a live context - forget it and let the caller interpret
    if (rc == 201 || rc == 400 || rc == 500) {
        std::lock_guard<std::mutex> lock(g_mutex);
        g_cache.erase(key);
        return kJitUnavailable;
    }
    return cuda_fail((cudaError_t)rc);        // driver and runtime share their error numbers
}

int jit_occupancy(const JitSpec &sp, const DevChain &ch)
{
    Api &a = api();
    if (g_mode.load() == 0 || !a.occupancy) return 0;
    CUfunction fn = find_kernel(ch, sp, false, nullptr, nullptr);
    int nb = 0;
    if (!fn || a.occupancy(&nb, fn, kThreads, 0) != 0) return 0;
    return nb;
}

}  // namespace fo

extern "C" {

int fo_set_jit(int mode)
{
    if (mode < 0 || mode > 2) mode = 1;
    return fo::g_mode.exchange(mode);
}

int fo_jit_prepare(const fo_chain *chain, int n_sides, int n_scalars, int store)
{
    using namespace fo;
    double scalars[FO_MAX_SCALARS] = {0};
    DevChain ch;
    const int rc = translate_chain(chain, kUseCell, n_sides, scalars, n_scalars, 1, FO_MAX_OUT, &ch);
    if (rc != FO_OK) return rc;
    if (store && ch.n_out != 1) return FO_ERR_CHAIN;
    int status = FO_ERR_UNSUPPORTED;
    const JitSpec sp = {kJitFlat, store != 0 ? 1 : 0, 0, 0};
    find_kernel(ch, sp, true, nullptr, &status);
    return status;
}

int fo_jit_stats(int *compiled, int *launches, int *failures)
{
    std::lock_guard<std::mutex> lock(fo::g_mutex);
    if (compiled) *compiled = fo::g_compiled;
    if (launches) *launches = fo::g_launches;
    if (failures) *failures = fo::g_failures;
    return (fo::api().nvrtc_ok && fo::api().driver_ok) ? 1 : 0;
}

int fo_jit_compile_check(const fo_chain *chain, int n_sides, int n_scalars, int store, char *log,
                         size_t log_bytes)
{
    using namespace fo;
    if (log && log_bytes) log[0] = 0;
    double scalars[FO_MAX_SCALARS] = {0};
    DevChain ch;
    const int rc = translate_chain(chain, kUseCell, n_sides, scalars, n_scalars, 1, FO_MAX_OUT, &ch);
    if (rc != FO_OK) return rc;
    if (!api().nvrtc_ok) return FO_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    JitSpec sp = {kJitFlat, store != 0 ? 1 : 0, 0, 0};
    if (store >= 2 && store <= 5) {     // the other skeletons over a dense input
        sp.kind = store == 5 ? kJitCols : kJitRows;
        sp.a = store == 5 ? 1 : store == 2 ? kAggRow : store == 3 ? kAggNone : kAggFull;
        sp.b = 1;
    } else if (store >= 6 && store <= 8) {     // over a CSR input: 2, 8 or 32 lanes per row
        sp.kind = kJitCsr;
        sp.a = store == 6 ? 2 : store == 7 ? 8 : 32;
    }
    const std::vector<char> cubin = compile(generate_source(ch, sp), "sm_100a");
    if (log && log_bytes) snprintf(log, log_bytes, "%s", g_last_log.c_str());
    return cubin.empty() ? FO_ERR_CHAIN : FO_OK;
}

int fo_jit_compile_check_outer(const fo_chain *chain, int n_sides, int n_scalars, int kernel, char *log,
                                size_t log_bytes)
{
    using namespace fo;
    if (log && log_bytes) log[0] = 0;
    double scalars[FO_MAX_SCALARS] = {0};
    DevChain ch;
    const int rc = translate_chain(chain, kUseOuter, n_sides, scalars, n_scalars, 1, 1, &ch);
    if (rc != FO_OK) return rc;
    if (!api().nvrtc_ok) return FO_ERR_UNSUPPORTED;
    JitSpec sp;
    switch (kernel) {
        case 0: sp = JitSpec{kJitOuterDirect, 7, kOutFull, 1}; break;
        case 1: sp = JitSpec{kJitOuterDirect, 16, kOutLeft, 0}; break;
        case 2: sp = JitSpec{kJitOuterPipe, 7, kOutFull, 0}; break;
        case 3: sp = JitSpec{kJitOuterPipe, 2, kOutRight, 0}; break;
        case 4: sp = JitSpec{kJitOuterDense, kOutFull, 0, 0}; break;
        case 5: sp = JitSpec{kJitOuterDense, kOutNone, 0, 0}; break;
        case 6: sp = JitSpec{kJitOuterBulk, 7, kOutFull, 0}; break;
        case 7: sp = JitSpec{kJitOuterBulk, 4, kOutNone, 0}; break;
        default: return FO_ERR_UNSUPPORTED;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    const std::vector<char> cubin = compile(generate_source(ch, sp), "sm_100a");
    if (log && log_bytes) snprintf(log, log_bytes, "%s", g_last_log.c_str());
    return cubin.empty() ? FO_ERR_CHAIN : FO_OK;
}

int fo_jit_compile_check_row(const fo_chain *chain, int n_sides, int n_scalars, int kernel, char *log,
                              size_t log_bytes)
{
    using namespace fo;
    if (log && log_bytes) log[0] = 0;
    double scalars[FO_MAX_SCALARS] = {0};
    DevChain ch;
    const int rc = translate_chain(chain, kUseRow, n_sides, scalars, n_scalars, 1, 1, &ch);
    if (rc != FO_OK) return rc;
    if (!api().nvrtc_ok) return FO_ERR_UNSUPPORTED;
    JitSpec sp;
    switch (kernel) {
        case 0: sp = JitSpec{kJitRowDense, 4, 4, 2, kRowColT, 1}; break;
        case 1: sp = JitSpec{kJitRowDense, 8, 16, 1, kRowNone, 0}; break;
        case 2: sp = JitSpec{kJitRowDense, 1, 1, 8, kRowRow, 1}; break;
        case 3: sp = JitSpec{kJitRowNarrow, 16, kRowColT, 1, 0, 0}; break;
        case 4: sp = JitSpec{kJitRowCsr, 2, 0, 0, 0, 0}; break;
        case 5: sp = JitSpec{kJitRowCsrReg, kRowFull, 8, 0, 0, 0}; break;
        default: return FO_ERR_UNSUPPORTED;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    const std::vector<char> cubin = compile(generate_source(ch, sp), "sm_100a");
    if (log && log_bytes) snprintf(log, log_bytes, "%s", g_last_log.c_str());
    return cubin.empty() ? FO_ERR_CHAIN : FO_OK;
}

}  // extern "C"
