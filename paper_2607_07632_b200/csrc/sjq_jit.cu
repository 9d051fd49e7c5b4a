// Run-time specialisation of the fused kernel (the CUDA analogue of the paper's
// composition-based fusion, Section 4.2: the fused pipeline of one query is
// assembled before it runs, so nothing about the query's shape is interpreted
// per row).
//
// The planner's RunParams is split in two: the *shape* (number of stages and
// levels, every stage's operation, column width, accumulator recipe and
// multipliers, the aggregation path, the modulo) is printed as a small header
// of constants, and the device source of the fused kernel is compiled for it
// with NVRTC into a module of one kernel; everything that depends on the data
// (pointers, row count, key ranges, thresholds, table sizes, payload minima)
// stays a kernel parameter, so one compiled module serves every run of the same
// query shape.  Modules are cached per process by their shape header.
//
// NVRTC is loaded with dlopen on first use; the library itself does not depend
// on it.  Without it (or without the device sources next to the library) a
// run that asks for specialisation fails with SJQ_ERR_JIT; it never falls back
// silently.
#include <dlfcn.h>

#include <cstddef>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <fstream>
#include <mutex>
#include <sstream>
#include <string>
#include <unordered_map>
#include <vector>

#include "sjq_run.cuh"

namespace sjq {

namespace {

// ---------------------------------------------------------------- NVRTC, loaded on demand
typedef struct _nvrtcProgram *nvrtcProgram;
struct Nvrtc {
    void *handle = nullptr;
    int (*CreateProgram)(nvrtcProgram *, const char *, const char *, int, const char *const *, const char *const *);
    int (*CompileProgram)(nvrtcProgram, int, const char *const *);
    int (*GetCUBINSize)(nvrtcProgram, size_t *);
    int (*GetCUBIN)(nvrtcProgram, char *);
    int (*GetProgramLogSize)(nvrtcProgram, size_t *);
    int (*GetProgramLog)(nvrtcProgram, char *);
    int (*DestroyProgram)(nvrtcProgram *);
    bool ok = false;
};

Nvrtc &nvrtc()
{
    static Nvrtc N;
    static std::once_flag once;
    std::call_once(once, [] {
        // several copies may be around (the toolkit's, one bundled with a Python package): take the newest, since
        // newer ones know more of the instruction set (256-bit loads need 12.9)
        const char *names[] = {"/usr/local/cuda/lib64/libnvrtc.so.12", "/usr/local/cuda/lib64/libnvrtc.so",
                               "libnvrtc.so.12", "libnvrtc.so"};
        int best = -1;
        for (const char *nm : names) {
            void *h = dlopen(nm, RTLD_NOW | RTLD_LOCAL);
            if (!h) continue;
            int major = 0, minor = 0;
            auto version = reinterpret_cast<int (*)(int *, int *)>(dlsym(h, "nvrtcVersion"));
            const int v = (version && version(&major, &minor) == 0) ? major * 100 + minor : 0;
            if (v > best) {
                if (N.handle) dlclose(N.handle);
                N.handle = h;
                best = v;
            } else {
                dlclose(h);
            }
        }
        if (!N.handle) return;
        bool all = true;
        auto sym = [&](const char *s) {
            void *p = dlsym(N.handle, s);
            all = all && p != nullptr;
            return p;
        };
        N.CreateProgram = reinterpret_cast<decltype(N.CreateProgram)>(sym("nvrtcCreateProgram"));
        N.CompileProgram = reinterpret_cast<decltype(N.CompileProgram)>(sym("nvrtcCompileProgram"));
        N.GetCUBINSize = reinterpret_cast<decltype(N.GetCUBINSize)>(sym("nvrtcGetCUBINSize"));
        N.GetCUBIN = reinterpret_cast<decltype(N.GetCUBIN)>(sym("nvrtcGetCUBIN"));
        N.GetProgramLogSize = reinterpret_cast<decltype(N.GetProgramLogSize)>(sym("nvrtcGetProgramLogSize"));
        N.GetProgramLog = reinterpret_cast<decltype(N.GetProgramLog)>(sym("nvrtcGetProgramLog"));
        N.DestroyProgram = reinterpret_cast<decltype(N.DestroyProgram)>(sym("nvrtcDestroyProgram"));
        N.ok = all;
    });
    return N;
}

// ---------------------------------------------------------------- device sources
// The kernel's source files sit beside the library (csrc/) and the public
// header one level up (include/); SJQ_SOURCE_DIR / SJQ_INCLUDE_DIR override.
bool read_file(const std::string &path, std::string *out)
{
    std::ifstream f(path, std::ios::binary);
    if (!f) return false;
    std::ostringstream ss;
    ss << f.rdbuf();
    *out = ss.str();
    return true;
}

std::string library_dir()
{
    Dl_info info;
    if (dladdr(reinterpret_cast<const void *>(&library_dir), &info) && info.dli_fname) {
        std::string p(info.dli_fname);
        const size_t slash = p.find_last_of('/');
        return slash == std::string::npos ? std::string(".") : p.substr(0, slash);
    }
    return ".";
}

struct Sources {
    std::string device, run, internal, api;
    bool ok = false;
    std::string error;
};

const Sources &sources()
{
    static Sources S;
    static std::once_flag once;
    std::call_once(once, [] {
        const std::string dir = library_dir();
        const char *e1 = std::getenv("SJQ_SOURCE_DIR");
        const char *e2 = std::getenv("SJQ_INCLUDE_DIR");
        const std::string src = e1 ? std::string(e1) : dir + "/csrc";
        const std::string inc = e2 ? std::string(e2) : dir + "/../include";
        S.ok = read_file(src + "/sjq_fused_device.cuh", &S.device) && read_file(src + "/sjq_run.cuh", &S.run) &&
               read_file(src + "/sjq_internal.h", &S.internal) && read_file(inc + "/sjq.h", &S.api);
        if (!S.ok) S.error = "device sources not found under " + src + " and " + inc;
    });
    return S;
}

// Stand-ins for the host headers the device source names (NVRTC has no C library headers).
const char *kStdint =
    "#ifndef SJQ_JIT_STDINT\n#define SJQ_JIT_STDINT\n"
    "typedef signed char int8_t; typedef unsigned char uint8_t; typedef short int16_t; typedef unsigned short uint16_t;\n"
    "typedef int int32_t; typedef unsigned int uint32_t; typedef long long int64_t; typedef unsigned long long uint64_t;\n"
    "typedef unsigned long uintptr_t;\n"
    "#define INT32_MIN (-2147483647 - 1)\n#define INT32_MAX 2147483647\n"
    "#define INT64_MIN (-9223372036854775807LL - 1)\n#define INT64_MAX 9223372036854775807LL\n"
    "#endif\n";
const char *kEmptyHeader = "\n";

// ---------------------------------------------------------------- the shape header
void put(std::ostringstream &o, const char *name, long long v) { o << "#define SJQ_JIT_" << name << " " << v << "LL\n"; }

} // namespace

// The shape of a run as a header of constants.  Two runs with the same text
// use the same compiled module.
std::string jit_shape_header(const RunParams &P, int agg, bool mul, bool hash, int lb_threads, int lb_blocks)
{
    std::ostringstream o;
    o << "// generated: the shape of one query\n#define SJQ_ROWS " << (P.rows == 8 ? 8 : 4) << "\n#define SJQ_SLOTS "
      << (P.slots == 4 ? 4 : 2) << "\n#define SJQ_JIT_nstages " << P.nstages << "\n//@body\n";
    o << "#define SJQ_JIT_AGG " << agg << "\n#define SJQ_JIT_MUL " << (mul ? 1 : 0) << "\n#define SJQ_JIT_HASH "
      << (hash ? 1 : 0) << "\n";
    o << "#define SJQ_LB_THREADS " << lb_threads << "\n#define SJQ_LB_BLOCKS " << lb_blocks << "\n";
    if (const char *extra = std::getenv("SJQ_JIT_EXTRA")) o << "// options: " << extra << "\n";
    o << "#define SJQ_JIT_nd0 " << P.nd0 << "\n#define SJQ_JIT_nq " << P.nq << "\n";
    o << "#define SJQ_JIT_qfold " << P.qfold << "u\n";
    o << "#define SJQ_JIT_want_count " << P.want_count << "\n#define SJQ_JIT_eager " << P.eager
      << "\n#define SJQ_JIT_has_key " << P.has_key << "\n#define SJQ_JIT_mod32 " << P.mod32
      << "\n#define SJQ_JIT_warp_agg " << P.warp_agg << "\n#define SJQ_JIT_l0_bulk " << P.l0_bulk << "\n#define SJQ_JIT_count32 " << P.count32 << "\n#define SJQ_JIT_sparse_push " << P.sparse_push
      << "\n";
    put(o, "modulo", P.modulo);
    o << "#define SJQ_JIT_modmask " << P.modmask << "ULL\n";
    o << "namespace sjq {\nnamespace {\n"
         "__device__ __forceinline__ DStage jit_stage(const RunParams &P, int s)\n{\n"
         "    DStage S = P.st[s];\n    switch (s) {\n";
    for (int s = 0; s < P.nstages; ++s) {
        const DStage &S = P.st[s];
        o << "    case " << s << ":\n        S.op = " << (int)S.op << "; S.is64 = " << (int)S.is64 << "; S.neg = " << (int)S.neg
          << "; S.never = " << (int)S.never << "; S.nset = " << (int)S.nset << "; S.set_idx = " << (int)S.set_idx
          << "; S.in_smem = " << (int)S.in_smem << "; S.kind = " << (int)S.kind << "; S.simple = " << (int)S.simple
          << "; S.acc = " << (int)S.acc << "; S.acc32 = " << S.acc32 << "; S.code_bits = " << (int)S.code_bits
          << "; S.issue_after = " << (int)S.issue_after << "; S.full = " << (int)S.full << "; S.hot = " << (int)S.hot
          << "; S.wide = " << (int)S.wide << ";\n";
        for (int i = 0; i < 9; ++i) {
            // INT64_MIN cannot be written as a literal
            if (S.mult[i] == INT64_MIN) o << "        S.mult[" << i << "] = (-9223372036854775807LL - 1);";
            else o << "        S.mult[" << i << "] = " << (long long)S.mult[i] << "LL;";
            if (S.mult32[i] == INT32_MIN) o << " S.mult32[" << i << "] = (-2147483647 - 1);\n";
            else o << " S.mult32[" << i << "] = " << S.mult32[i] << ";\n";
        }
        o << "        break;\n";
    }
    o << "    default: break;\n    }\n    return S;\n}\n} // namespace\n} // namespace sjq\n";
    return o.str();
}

namespace {

// Everything jit_shape_header prints, as bytes: cheap to build on every run; the text itself is only
// generated when the key is new.
std::string shape_key(const RunParams &P, int agg, bool mul, bool hash, int lb_threads, int lb_blocks)
{
    std::string k;
    k.reserve(64 + (size_t)P.nstages * 128);
    auto put_raw = [&](const void *p, size_t n) { k.append(static_cast<const char *>(p), n); };
    const int32_t head[] = {agg, mul ? 1 : 0, hash ? 1 : 0, lb_threads, lb_blocks, P.nstages, P.nd0, P.nq,
                            P.rows, P.want_count, P.eager, P.has_key, P.mod32, (int32_t)P.qfold, P.slots, P.warp_agg,
                            P.l0_bulk, P.count32, P.sparse_push};
    put_raw(head, sizeof(head));
    put_raw(&P.modulo, sizeof(P.modulo));
    put_raw(&P.modmask, sizeof(P.modmask));
    for (int s = 0; s < P.nstages; ++s) {
        const DStage &S = P.st[s];
        const uint8_t b[] = {S.op, S.is64, S.neg, S.never, S.nset, S.set_idx, S.in_smem, S.kind, S.simple, S.code_bits,
                             (uint8_t)S.issue_after, S.full, S.hot, S.wide};
        put_raw(b, sizeof(b));
        put_raw(&S.acc, sizeof(S.acc));
        put_raw(&S.acc32, sizeof(S.acc32));
        put_raw(S.mult, sizeof(S.mult));
        put_raw(S.mult32, sizeof(S.mult32));
    }
    if (const char *extra = std::getenv("SJQ_JIT_EXTRA")) k += extra;
    return k;
}

struct Module {
    cudaLibrary_t lib = nullptr;
    cudaKernel_t kernel = nullptr;
    int smem_set[64];  // per device: largest dynamic shared memory size the kernel has been opted in for
    std::unordered_map<uint64_t, int> occupancy; // (device, block, smem) -> blocks per SM
    Module() { for (int &v : smem_set) v = -1; }
    sjq_status status = SJQ_OK;
};

std::mutex g_mutex;
std::unordered_map<std::string, Module> g_modules;
std::string g_last_log;

sjq_status compile(const std::string &shape, std::vector<char> *cubin, std::string *log)
{
    Nvrtc &N = nvrtc();
    if (!N.ok) {
        *log = "NVRTC (libnvrtc.so.12) could not be loaded";
        return SJQ_ERR_JIT;
    }
    const Sources &S = sources();
    if (!S.ok) {
        *log = S.error;
        return SJQ_ERR_JIT;
    }
    // what precedes the //@body line of the shape text must be seen before any other header
    const size_t cut = shape.find("//@body\n");
    const std::string main_text = "#define SJQ_JIT 1\n" + shape.substr(0, cut == std::string::npos ? 0 : cut) +
                                  "#include \"sjq_fused_device.cuh\"\n";
    const std::string shape_body = cut == std::string::npos ? shape : shape.substr(cut);
    const char *main_src = main_text.c_str();
    const char *names[] = {"sjq_fused_device.cuh", "sjq_run.cuh", "sjq_internal.h", "sjq.h", "sjq_jit_shape.h",
                           "stdint.h",             "stddef.h",    "cuda_runtime.h"};
    const char *bodies[] = {S.device.c_str(), S.run.c_str(), S.internal.c_str(), S.api.c_str(), shape_body.c_str(),
                            kStdint,          kEmptyHeader,  kEmptyHeader};
    nvrtcProgram prog = nullptr;
    if (N.CreateProgram(&prog, main_src, "sjq_jit.cu", 8, bodies, names) != 0) {
        *log = "nvrtcCreateProgram failed";
        return SJQ_ERR_JIT;
    }
    // host declarations in the shared headers are harmless when read as device ones
    std::vector<const char *> opts = {"--gpu-architecture=sm_100a", "-std=c++17", "-lineinfo", "-default-device",
                                      "--disable-warnings"};
    if (std::getenv("SJQ_JIT_VERBOSE")) opts.push_back("--ptxas-options=-v");
    std::vector<std::string> extra; // experiment switches, e.g. SJQ_JIT_EXTRA="-DSJQ_PREFETCH_DIST=3"
    if (const char *e = std::getenv("SJQ_JIT_EXTRA")) {
        std::istringstream is(e);
        std::string tok;
        while (is >> tok) extra.push_back(tok);
    }
    for (const std::string &t : extra) opts.push_back(t.c_str());
    const int rc = N.CompileProgram(prog, (int)opts.size(), opts.data());
    size_t ls = 0;
    if (N.GetProgramLogSize(prog, &ls) == 0 && ls > 1) {
        log->resize(ls);
        N.GetProgramLog(prog, &(*log)[0]);
    }
    sjq_status st = SJQ_OK;
    size_t cs = 0;
    if (rc != 0 || N.GetCUBINSize(prog, &cs) != 0 || cs == 0) {
        st = SJQ_ERR_JIT;
    } else {
        cubin->resize(cs);
        if (N.GetCUBIN(prog, cubin->data()) != 0) st = SJQ_ERR_JIT;
    }
    N.DestroyProgram(&prog);
    return st;
}

// Find or build the module of a shape.  Called with g_mutex held.
sjq_status module_for(const RunParams &P, int agg, bool mul, bool hash, int lb_threads, int lb_blocks, Module **out)
{
    const std::string key = shape_key(P, agg, mul, hash, lb_threads, lb_blocks);
    auto it = g_modules.find(key);
    if (it == g_modules.end()) {
        const std::string shape = jit_shape_header(P, agg, mul, hash, lb_threads, lb_blocks);
        Module M;
        std::vector<char> cubin;
        std::string log;
        M.status = compile(shape, &cubin, &log);
        g_last_log = log;
        if (std::getenv("SJQ_JIT_VERBOSE")) std::fprintf(stderr, "[sjq jit] %s\n", log.c_str());
        if (M.status == SJQ_OK) {
            if (cudaLibraryLoadData(&M.lib, cubin.data(), nullptr, nullptr, 0, nullptr, nullptr, 0) != cudaSuccess ||
                cudaLibraryGetKernel(&M.kernel, M.lib, "sjq_jit_kernel") != cudaSuccess) {
                (void)cudaGetLastError();
                g_last_log += "\nloading the compiled module failed";
                M.status = SJQ_ERR_JIT;
            }
        }
        it = g_modules.emplace(key, M).first;
    }
    *out = &it->second;
    return it->second.status;
}

} // namespace

sjq_status jit_occupancy(const RunParams &P, int agg, bool mul, bool hash, int block, int lb_blocks, size_t smem,
                         int *ctas_per_sm)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    Module *M = nullptr;
    sjq_status st = module_for(P, agg, mul, hash, block, lb_blocks, &M);
    if (st != SJQ_OK) return st;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SJQ_ERR_CUDA;
    if ((int)smem > M->smem_set[dev]) {
        if (cudaFuncSetAttribute(reinterpret_cast<const void *>(M->kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return SJQ_ERR_CUDA;
        }
        M->smem_set[dev] = (int)smem;
    }
    const uint64_t okey = ((uint64_t)dev << 48) | ((uint64_t)block << 24) | (uint64_t)(smem & 0xFFFFFF);
    auto o = M->occupancy.find(okey);
    if (o == M->occupancy.end()) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, reinterpret_cast<const void *>(M->kernel), block, smem) !=
            cudaSuccess) {
            (void)cudaGetLastError();
            return SJQ_ERR_CUDA;
        }
        o = M->occupancy.emplace(okey, n).first;
    }
    *ctas_per_sm = o->second;
    return SJQ_OK;
}

sjq_status jit_launch(const RunParams &P, int agg, bool mul, bool hash, int grid, int block, int lb_blocks,
                      size_t smem, cudaStream_t stream)
{
    cudaKernel_t kernel;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        Module *M = nullptr;
        sjq_status st = module_for(P, agg, mul, hash, block, lb_blocks, &M);
        if (st != SJQ_OK) return st;
        kernel = M->kernel;
    }
    // the compiled kernel's parameter struct holds P.nstages stage descriptors (at least one), then the same
    // fields as RunParams: pack exactly that
    const size_t nst = (size_t)(P.nstages > 0 ? P.nstages : 1);
    const size_t tail_from = offsetof(RunParams, sets), tail_bytes = sizeof(RunParams) - tail_from;
    static_assert(offsetof(RunParams, st) == 0 && offsetof(RunParams, sets) == sizeof(DStage) * (size_t)kMaxStages,
                  "the stage descriptors lead the parameter block and the rest follows without padding");
    alignas(16) unsigned char packed[sizeof(RunParams)];
    std::memcpy(packed, P.st, nst * sizeof(DStage));
    std::memcpy(packed + nst * sizeof(DStage), reinterpret_cast<const unsigned char *>(&P) + tail_from, tail_bytes);
    void *args[] = {packed};
    if (cudaLaunchKernel(reinterpret_cast<const void *>(kernel), dim3(grid), dim3(block), args, smem, stream) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return SJQ_ERR_CUDA;
    }
    return SJQ_OK;
}

// Compile-only check (no device needed): is the shape compilable, and what did the compiler say.
sjq_status jit_compile_only(const std::string &shape, std::string *log, size_t *cubin_bytes)
{
    std::vector<char> cubin;
    sjq_status st = compile(shape, &cubin, log);
    *cubin_bytes = cubin.size();
    return st;
}

} // namespace sjq

// ---------------------------------------------------------------- C ABI
extern "C" int32_t sjq_jit_cache_clear(void)
{
    std::lock_guard<std::mutex> lock(sjq::g_mutex);
    int32_t n = 0;
    for (auto &kv : sjq::g_modules) {
        if (kv.second.lib) {
            if (cudaLibraryUnload(kv.second.lib) != cudaSuccess) (void)cudaGetLastError();
            ++n;
        }
    }
    sjq::g_modules.clear();
    return n;
}

extern "C" size_t sjq_jit_log(char *buf, size_t bytes)
{
    std::lock_guard<std::mutex> lock(sjq::g_mutex);
    if (buf && bytes) {
        const size_t n = sjq::g_last_log.size() < bytes - 1 ? sjq::g_last_log.size() : bytes - 1;
        std::memcpy(buf, sjq::g_last_log.data(), n);
        buf[n] = 0;
    }
    return sjq::g_last_log.size();
}

namespace sjq {
namespace {

// Built-in shapes for the compile-only self test: what the planner produces for typical queries.
DStage canned(uint8_t op, uint8_t kind, bool is64, uint16_t acc, uint8_t code_bits, bool in_smem)
{
    DStage S;
    std::memset(&S, 0, sizeof(S));
    S.op = op;
    S.kind = kind;
    S.is64 = is64;
    S.acc = acc;
    S.acc32 = !is64;
    S.code_bits = code_bits;
    S.in_smem = in_smem;
    for (int i = 0; i < 9; ++i) S.mult[i] = S.mult32[i] = ((acc >> i) & 1) ? (i == 3 ? 25 : 1) : 0;
    if (op == OP_LOAD && (acc == 1 || acc == 2 || acc == 4) && !is64) S.simple = (uint8_t)(acc == 1 ? 1 : acc == 2 ? 2 : 3);
    return S;
}

int canned_shape(int id, RunParams *P, int *agg, bool *mul, bool *hash)
{
    std::memset(P, 0, sizeof(*P));
    *mul = false;
    *hash = false;
    switch (id) {
    case 0: // two predicates, one filter-only join, product aggregate, scalar result
        P->st[0] = canned(OP_PRED_RANGE, ST_PRED, false, 0, 0, false);
        P->st[1] = canned(OP_PRED_RANGE, ST_PRED, false, 0, 0, false);
        P->st[2] = canned(OP_DIRECT_BITMAP, ST_PROBE, false, 0, 1, true);
        P->st[3] = canned(OP_LOAD, ST_LOAD, false, 2, 0, false);
        P->st[4] = canned(OP_LOAD, ST_LOAD, false, 4, 0, false);
        P->nstages = 5, P->nd0 = 2, P->nq = 2;
        *agg = AGG_SCALAR, *mul = true;
        return 1;
    case 1: // four joins, two group-key payloads, difference of two measures, shared-memory group table
        P->st[0] = canned(OP_DIRECT_BITMAP, ST_PROBE, false, 0, 1, false);
        P->st[1] = canned(OP_DIRECT_U8, ST_PROBE, false, 0, 8, true);
        P->st[2] = canned(OP_DIRECT_BITMAP, ST_PROBE, false, 0, 1, false);
        P->st[3] = canned(OP_DIRECT_U8, ST_PROBE, false, 8, 8, false);
        P->st[4] = canned(OP_DIRECT_U8, ST_PROBE, false, 8, 8, true);
        P->st[5] = canned(OP_LOAD, ST_LOAD, false, 2, 0, false);
        P->st[6] = canned(OP_LOAD, ST_LOAD, false, 2, 0, false);
        P->st[6].mult[1] = P->st[6].mult32[1] = -1;
        P->nstages = 7, P->nd0 = 1, P->nq = 3;
        *agg = AGG_SMEM;
        return 1;
    case 2: // 64-bit keys: presence bitmap, open-addressing probe with a payload, modulo key, global atomics, counts
        P->st[0] = canned(OP_HASHBITS, ST_PROBE, true, 0, 0, false);
        P->st[1] = canned(OP_HASH64, ST_PROBE, true, 8, 32, false);
        P->st[2] = canned(OP_LOAD, ST_LOAD, false, 2, 0, false);
        P->nstages = 3, P->nd0 = 1, P->nq = 1;
        P->modulo = 4096, P->modmask = 4095, P->mod32 = 1, P->want_count = 1;
        P->rows = 8;
        *agg = AGG_GLOBAL, *hash = true;
        return 1;
    case 3: // no queues, set predicate, 32-bit open addressing, runtime modulo, global group hash table
        P->st[0] = canned(OP_PRED_SET, ST_PRED, false, 0, 0, false);
        P->st[0].nset = 3;
        P->st[1] = canned(OP_HASH32, ST_PROBE, false, 16, 32, false);
        P->st[2] = canned(OP_LOAD, ST_LOAD, false, 1, 0, false);
        P->st[3] = canned(OP_LOAD, ST_LOAD, true, 2, 0, false);
        P->nstages = 4, P->nd0 = 0, P->nq = 0;
        P->modulo = 1000, P->mod32 = 1, P->want_count = 1;
        *agg = AGG_HASH, *hash = true;
        return 1;
    case 4: // one predicate on an int32 first column staged by bulk-asynchronous copies, one join with a 2-bit
            // payload, shared-memory group table
        P->st[0] = canned(OP_PRED_RANGE, ST_PRED, false, 0, 0, false);
        P->st[1] = canned(OP_DIRECT_U2, ST_PROBE, false, 16, 2, false);
        P->st[2] = canned(OP_LOAD, ST_LOAD, false, 1, 0, false);
        P->st[3] = canned(OP_LOAD, ST_LOAD, false, 2, 0, false);
        P->nstages = 4, P->nd0 = 1, P->nq = 1;
        P->modulo = 1000, P->mod32 = 1, P->want_count = 1;
        P->l0_bulk = 1;
        *agg = AGG_SMEM;
        return 1;
    case 5: // 64-bit first column staged by bulk-asynchronous copies, hot-key table in front of the presence bitmap
            // and of the open-addressing probe
        P->st[0] = canned(OP_HASHBITS, ST_PROBE, true, 0, 0, false);
        P->st[1] = canned(OP_HASH64, ST_PROBE, true, 8, 32, false);
        P->st[2] = canned(OP_LOAD, ST_LOAD, false, 2, 0, false);
        P->st[0].hot = 1, P->st[1].hot = 2, P->st[1].wide = 1;
        P->nstages = 3, P->nd0 = 1, P->nq = 1;
        P->modulo = 4096, P->modmask = 4095, P->mod32 = 1, P->want_count = 1;
        P->l0_bulk = 1;
        *agg = AGG_SMEM, *hash = true;
        return 1;
    default: return 0;
    }
}

} // namespace
} // namespace sjq

namespace sjq {
namespace {
// the load schedule the planner would give a final level none of whose stages drops rows
void canned_schedule(RunParams *P)
{
    if (!P->nq) return;
    const int first = P->nd0 + P->nq - 1;
    for (int t = first; t < P->nstages; ++t) P->st[t].issue_after = (int8_t)(t - 3 > first - 1 ? t - 3 : first - 1);
}
} // namespace
} // namespace sjq

extern "C" int32_t sjq_jit_selftest(int32_t shape_id, char *log, size_t log_bytes)
{
    static sjq::RunParams P; // large: keep it off the stack
    static std::mutex m;
    std::lock_guard<std::mutex> lock(m);
    int agg = 0;
    bool mul = false, hash = false;
    if (shape_id < 0) {
        int n = 0;
        while (sjq::canned_shape(n, &P, &agg, &mul, &hash)) ++n;
        return n;
    }
    if (!sjq::canned_shape(shape_id, &P, &agg, &mul, &hash)) return SJQ_ERR_INVALID_ARG;
    sjq::canned_schedule(&P);
    std::string text;
    size_t cubin = 0;
    const sjq_status st = sjq::jit_compile_only(sjq::jit_shape_header(P, agg, mul, hash, 384, 2), &text, &cubin);
    if (log && log_bytes) {
        const size_t n = text.size() < log_bytes - 1 ? text.size() : log_bytes - 1;
        std::memcpy(log, text.data(), n);
        log[n] = 0;
    }
    return st;
}
