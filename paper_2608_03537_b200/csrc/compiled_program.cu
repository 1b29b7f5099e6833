// Stage programs compiled into the fused kernel at run time (Sec. 5: the fused epilogue is generated code, not data).
//
// The interpreter of fused_pair.cuh dispatches every micro-instruction of a program on every 32-column fragment.  Here the
// same kernel source is compiled once per program with the program's structure as a constant table in front of it
// (COMFUSE_COMPILED_PROGRAM): the sweep and instruction loops unroll, every dispatch folds to the operation it selects and
// the per-row scalars live in registers.  Immediates and row-output pointers stay run-time parameters, so programs that
// differ only in constants share a kernel.  The compiler is NVRTC, loaded with dlopen when the first program asks for it;
// the kernel sources are embedded in this library at build time.  A kernel is compiled on the first call that needs it
// (seconds) and kept for the life of the process; COMFUSE_KERNEL_CACHE=<directory> also keeps the device images on disk.
#include <dlfcn.h>
#include <nvrtc.h>
#include <unistd.h>

#include <cstring>
#include <memory>
#include <mutex>
#include <string>
#include <unordered_map>
#include <vector>

#include "fused_launch.cuh"

namespace comfuse {

// written by the build: the kernel headers as text (name as it appears in an #include, contents)
extern const char* const kEmbeddedSourceNames[];
extern const char* const kEmbeddedSources[];
extern const int kEmbeddedSourceCount;

namespace {

struct Compiler {
  void* lib = nullptr;
  std::string include_dir;  // the toolkit's headers (cuda_bf16.h)
  std::string why;          // why it is unavailable, if it is
  decltype(&nvrtcCreateProgram) create = nullptr;
  decltype(&nvrtcCompileProgram) compile = nullptr;
  decltype(&nvrtcDestroyProgram) destroy = nullptr;
  decltype(&nvrtcGetProgramLogSize) log_size = nullptr;
  decltype(&nvrtcGetProgramLog) log = nullptr;
  decltype(&nvrtcGetCUBINSize) cubin_size = nullptr;
  decltype(&nvrtcGetCUBIN) cubin = nullptr;
  decltype(&nvrtcAddNameExpression) add_name = nullptr;
  decltype(&nvrtcGetLoweredName) lowered_name = nullptr;
  bool ok() const { return lib != nullptr && why.empty(); }
};

bool file_exists(const std::string& path) {
  FILE* f = std::fopen(path.c_str(), "rb");
  if (f) std::fclose(f);
  return f != nullptr;
}

const Compiler& compiler() {
  static Compiler c;
  static std::once_flag once;
  std::call_once(once, [] {
    std::vector<std::string> roots;
    for (const char* env : {"COMFUSE_CUDA_HOME", "CUDA_HOME", "CUDA_PATH"})
      if (const char* v = std::getenv(env)) roots.push_back(v);
    roots.push_back("/usr/local/cuda");
    // by full path first: a process may already hold another libnvrtc of the same soname (an older one cannot assemble
    // every instruction these kernels use)
    for (const std::string& r : roots) {
      for (const char* sub : {"/lib64/libnvrtc.so.12", "/lib/libnvrtc.so.12", "/lib64/libnvrtc.so"}) {
        if (c.lib) break;
        if (file_exists(r + sub)) c.lib = dlopen((r + sub).c_str(), RTLD_NOW | RTLD_LOCAL);
      }
      if (c.lib && c.include_dir.empty() && file_exists(r + "/include/cuda_bf16.h")) c.include_dir = r + "/include";
    }
    if (!c.lib) c.lib = dlopen("libnvrtc.so.12", RTLD_NOW | RTLD_LOCAL);
    if (!c.lib) { c.why = "libnvrtc.so.12 not found (set CUDA_HOME)"; return; }
    if (c.include_dir.empty())
      for (const std::string& r : roots)
        if (c.include_dir.empty() && file_exists(r + "/include/cuda_bf16.h")) c.include_dir = r + "/include";
    if (c.include_dir.empty()) { c.why = "the CUDA toolkit's headers were not found (set CUDA_HOME)"; return; }
#define COMFUSE_SYM(field, name)                                       \
  c.field = reinterpret_cast<decltype(c.field)>(dlsym(c.lib, #name)); \
  if (!c.field) { c.why = "libnvrtc lacks " #name; return; }
    COMFUSE_SYM(create, nvrtcCreateProgram)
    COMFUSE_SYM(compile, nvrtcCompileProgram)
    COMFUSE_SYM(destroy, nvrtcDestroyProgram)
    COMFUSE_SYM(log_size, nvrtcGetProgramLogSize)
    COMFUSE_SYM(log, nvrtcGetProgramLog)
    COMFUSE_SYM(cubin_size, nvrtcGetCUBINSize)
    COMFUSE_SYM(cubin, nvrtcGetCUBIN)
    COMFUSE_SYM(add_name, nvrtcAddNameExpression)
    COMFUSE_SYM(lowered_name, nvrtcGetLoweredName)
#undef COMFUSE_SYM
  });
  return c;
}

// The program's structure as a constant aggregate, field by field in the declaration order of StageProgram.  Immediates
// and pointers are left out (zero): the kernel reads those from its parameter.
std::string constant_table(const StageProgram& sp) {
  std::string t;
  char buf[160];
  auto put = [&](const char* fmt, auto... a) { std::snprintf(buf, sizeof(buf), fmt, a...); t += buf; };
  t += "#include \"fused_params.h\"\nnamespace comfuse {\n__device__ const StageProgram kCompiledProgram = {\n";
  put("  %d, %d, %d, %d, %d, %d, %d, {0},\n", sp.n_red, sp.n_scalar_instr, sp.n_passes, sp.terminal_pass, sp.n_row_out, sp.x_writeback,
      sp.uses_temps);
  t += "  {";
  for (int i = 0; i <= kStageMaxPasses; ++i) put("%d, ", sp.pass_off[i]);
  put("}, %d, {0, 0},\n  {", sp.n_sweeps);
  for (int i = 0; i < sp.n_sweeps; ++i) {
    const SweepStep& w = sp.sweep[i];
    put("{%d, %d, %d, %d, %d, %d, {0, 0}}, ", w.i0, w.i1, w.topk_r, w.topk_round, w.pass, w.release);
  }
  t += "},\n  {";
  const int n_code = sp.pass_off[sp.n_passes];
  for (int i = 0; i < n_code; ++i) put("{%d, %d, %d, 0.f}, ", sp.code[i].op, sp.code[i].operand, sp.code[i].index);
  t += "},\n  {";
  for (int i = 0; i < sp.n_red; ++i) {
    const StageReduction& r = sp.red[i];
    put("{%d, %d, %d, %d, %d, %d, %d, 0}, ", r.pass, r.op, r.on_terminal, r.dst, r.k, r.code_lo, r.code_hi);
  }
  t += "},\n  {";
  for (int i = 0; i < sp.n_scalar_instr; ++i) {
    const ScalarInstr& q = sp.sc[i];
    put("{%d, %d, %d, %d, %d, %d, %d, 0, 0.f, 0.f}, ", q.after_pass, q.op, q.dst, q.a_kind, q.b_kind, q.a, q.b);
  }
  t += "},\n  {";
  for (int i = 0; i < sp.n_row_out; ++i) put("{nullptr, %d, %d, %d, {0, 0, 0, 0, 0}}, ", sp.out[i].scalar, sp.out[i].is_int, sp.out[i].topk_red);
  t += "}\n};\n}  // namespace comfuse\n#define COMFUSE_COMPILED_PROGRAM 1\n#include \"fused_pair.cuh\"\n";
  return t;
}

// The device image is made without a device; it is loaded as a library (a handle valid on every device) by the first launch.
struct CompiledKernel {
  std::vector<char> image;
  std::string lowered_name;
  cudaLibrary_t library = nullptr;
  cudaKernel_t kernel = nullptr;
  std::atomic<int> max_clusters[kMaxLaunchDevices];
  CompiledKernel() { for (auto& m : max_clusters) m.store(0); }
};

// what stands in for the standard and driver headers the kernel sources name (the compiler has no host headers)
const char* const kStdintStub =
    "#pragma once\ntypedef signed char int8_t; typedef unsigned char uint8_t; typedef short int16_t; typedef unsigned short uint16_t;\n"
    "typedef int int32_t; typedef unsigned int uint32_t; typedef long long int64_t; typedef unsigned long long uint64_t;\n";
const char* const kStddefStub = "#pragma once\n";
const char* const kDriverStub =
    "#pragma once\nstruct alignas(64) CUtensorMap_st { unsigned long long opaque[16]; };\ntypedef struct CUtensorMap_st CUtensorMap;\n";

// Compiles `source` and returns the kernel named by `name_expr`, or nullptr with the reason in `why`.
std::unique_ptr<CompiledKernel> compile_kernel(const std::string& source, const std::string& name_expr, bool contract, std::string& why) {
  const Compiler& c = compiler();
  if (!c.ok()) { why = c.why; return nullptr; }
  std::vector<const char*> names, texts;
  for (int i = 0; i < kEmbeddedSourceCount; ++i) { names.push_back(kEmbeddedSourceNames[i]); texts.push_back(kEmbeddedSources[i]); }
  names.push_back("stdint.h"); texts.push_back(kStdintStub);
  names.push_back("stddef.h"); texts.push_back(kStddefStub);
  names.push_back("cuda.h"); texts.push_back(kDriverStub);
  nvrtcProgram prog = nullptr;
  if (c.create(&prog, source.c_str(), "comfuse_compiled_program.cu", static_cast<int>(names.size()), texts.data(), names.data()) != NVRTC_SUCCESS) {
    why = "nvrtcCreateProgram failed";
    return nullptr;
  }
  c.add_name(prog, name_expr.c_str());
  const std::string inc = "-I" + c.include_dir;
  std::vector<const char*> opts = {"--gpu-architecture=sm_100a", "-std=c++17", "-default-device", "-DINFINITY=__int_as_float(0x7f800000)",
                                   inc.c_str()};
#ifdef COMFUSE_CHECKED
  opts.push_back("-DCOMFUSE_CHECKED");
#endif
  if (!contract) {
    opts.push_back("--fmad=false");
    opts.push_back("-DCOMFUSE_NO_CONTRACTION");  // the packed add / multiply helpers: see sm100_primitives.cuh
  }
  if (std::getenv("COMFUSE_VERBOSE")) opts.push_back("--ptxas-options=-v");  // registers, spills and code size into the log
  const nvrtcResult r = c.compile(prog, static_cast<int>(opts.size()), opts.data());
  std::unique_ptr<CompiledKernel> out;
  if (r != NVRTC_SUCCESS || std::getenv("COMFUSE_VERBOSE")) {
    size_t n = 0;
    c.log_size(prog, &n);
    std::string log(n, ' ');
    if (n > 1) c.log(prog, &log[0]);
    if (r != NVRTC_SUCCESS) {
      why = "run-time compilation failed: " + log.substr(0, 600);
      std::fprintf(stderr, "comfuse: run-time compilation failed:\n%s\n", log.c_str());
    } else if (n > 1) {
      std::fprintf(stderr, "comfuse: run-time compiler log:\n%s\n", log.c_str());
    }
  }
  if (r == NVRTC_SUCCESS) {
    size_t nb = 0;
    const char* lowered = nullptr;
    if (c.cubin_size(prog, &nb) == NVRTC_SUCCESS && nb > 0 && c.lowered_name(prog, name_expr.c_str(), &lowered) == NVRTC_SUCCESS && lowered) {
      out.reset(new CompiledKernel);
      out->image.resize(nb);
      c.cubin(prog, out->image.data());
      out->lowered_name = lowered;
    } else {
      why = "the compiler returned no device image";
    }
  }
  c.destroy(&prog);
  return out;
}

// Optional cache of device images on disk (COMFUSE_KERNEL_CACHE=<directory>): a process finds the kernels earlier processes
// compiled.  The file name is a hash of everything the image depends on: instantiation, options, constant table, the embedded
// kernel sources and the compiler's version.  File = "comfuse-cubin-1\n" lowered-name "\n" image.  Written through a
// temporary name and renamed, so a reader never sees half a file.
uint64_t fnv1a(const std::string& text, uint64_t h = 1469598103934665603ull) {
  for (unsigned char c : text) { h ^= c; h *= 1099511628211ull; }
  return h;
}
std::string disk_cache_path(const std::string& key) {
  const char* dir = std::getenv("COMFUSE_KERNEL_CACHE");
  if (!dir || !dir[0]) return std::string();
  static const uint64_t build = [] {
    uint64_t h = 1469598103934665603ull;
    for (int i = 0; i < kEmbeddedSourceCount; ++i) h = fnv1a(kEmbeddedSources[i], h);
    int major = 0, minor = 0;
    if (auto version = reinterpret_cast<decltype(&nvrtcVersion)>(compiler().lib ? dlsym(compiler().lib, "nvrtcVersion") : nullptr))
      version(&major, &minor);
    return fnv1a(std::to_string(major) + "." + std::to_string(minor), h);
  }();
  char name[64];
  std::snprintf(name, sizeof(name), "/comfuse-%016llx.cubin", static_cast<unsigned long long>(fnv1a(key, build)));
  return std::string(dir) + name;
}
const char kDiskMagic[] = "comfuse-cubin-1\n";
std::unique_ptr<CompiledKernel> disk_cache_load(const std::string& path) {
  FILE* f = path.empty() ? nullptr : std::fopen(path.c_str(), "rb");
  if (!f) return nullptr;
  std::string all;
  char buf[1 << 16];
  for (size_t n; (n = std::fread(buf, 1, sizeof(buf), f)) > 0;) all.append(buf, n);
  std::fclose(f);
  const size_t m = sizeof(kDiskMagic) - 1;
  if (all.compare(0, m, kDiskMagic) != 0) return nullptr;
  const size_t nl = all.find('\n', m);
  if (nl == std::string::npos || nl + 1 >= all.size()) return nullptr;
  std::unique_ptr<CompiledKernel> k(new CompiledKernel);
  k->lowered_name = all.substr(m, nl - m);
  k->image.assign(all.begin() + nl + 1, all.end());
  return k;
}
void disk_cache_store(const std::string& path, const CompiledKernel& k) {
  if (path.empty()) return;
  const std::string tmp = path + ".tmp" + std::to_string(static_cast<long long>(getpid()));
  FILE* f = std::fopen(tmp.c_str(), "wb");
  if (!f) return;
  bool ok = std::fwrite(kDiskMagic, 1, sizeof(kDiskMagic) - 1, f) == sizeof(kDiskMagic) - 1;
  ok = ok && std::fwrite(k.lowered_name.data(), 1, k.lowered_name.size(), f) == k.lowered_name.size() && std::fputc('\n', f) != EOF;
  ok = ok && std::fwrite(k.image.data(), 1, k.image.size(), f) == k.image.size();
  ok = (std::fclose(f) == 0) && ok;
  if (!ok || std::rename(tmp.c_str(), path.c_str()) != 0) std::remove(tmp.c_str());
}

std::mutex g_cache_mutex;
std::unordered_map<std::string, std::unique_ptr<CompiledKernel>> g_cache;     // key: instance name + constant table
std::unordered_map<std::string, std::string> g_failed;                         // key -> reason (not retried)

}  // namespace

comfuse_status_t program_compiler_status(const char** why) {
  const Compiler& c = compiler();
  if (why) *why = c.ok() ? "" : c.why.c_str();
  return c.ok() ? COMFUSE_OK : COMFUSE_ERR_UNSUPPORTED;
}

// `launch` = false compiles (or finds) the kernel only.
cudaError_t launch_compiled_program(const GemmMaps& maps, const FusedParams& p, cudaStream_t st, bool supported_only, bool launch) {
  PairLaunchShape sh = {0, 0, 0};
  char name[160] = {0};
#define COMFUSE_CASE(n, b0, b1, cn, nst, lock)                                                                                      \
  case n: {                                                                                                                         \
    using Cfg = PairCfg<EPI_PROGRAM, b0, b1, cn, nst, lock, 2>;                                                                     \
    sh = PairLaunchShape{Cfg::kThreads, Cfg::SMEM_BYTES, 2 * cn};                                                                   \
    std::snprintf(name, sizeof(name), "comfuse::fused_pair_kernel<comfuse::EPI_PROGRAM, %d, %d, %d, %d, %d, 2>", b0, b1, cn, nst, lock); \
    break;                                                                                                                          \
  }
  switch (p.N) {
    COMFUSE_PROGRAM_INSTANCES_SMALL(COMFUSE_CASE)
    COMFUSE_PROGRAM_INSTANCES_LARGE(COMFUSE_CASE)
    COMFUSE_PROGRAM_INSTANCES_GENERATED_ONLY(COMFUSE_CASE)
    default:
      return cudaErrorInvalidValue;
  }
#undef COMFUSE_CASE
  if (supported_only) return compiler().ok() ? cudaSuccess : cudaErrorInvalidValue;
  // With the loops unrolled the compiler may contract a multiply and the add of the NEXT node into one fused multiply-add,
  // which the interpreter (a dispatch between any two nodes) never does: results then differ from the interpreter's in
  // the last bit, towards the exact value.  COMFUSE_GENERATED_FMAD=0 compiles without contraction: bit-identical results.
  const char* fmad = std::getenv("COMFUSE_GENERATED_FMAD");
  const bool contract = !(fmad && fmad[0] == '0');
  const std::string table = constant_table(p.program);
  const std::string key = std::string(name) + (contract ? "\n" : " no-contraction\n") + table;
  CompiledKernel* k = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    auto it = g_cache.find(key);
    if (it != g_cache.end()) {
      k = it->second.get();
    } else if (g_failed.count(key)) {
      return cudaErrorInvalidValue;
    } else {
      std::string why;
      const std::string on_disk = disk_cache_path(key);
      std::unique_ptr<CompiledKernel> made = disk_cache_load(on_disk);
      if (made) {
        k = made.get();
        g_cache[key] = std::move(made);
      } else {
      if (const char* dump = std::getenv("COMFUSE_GENERATED_DUMP")) {  // the generated translation unit, for inspection
        if (FILE* f = std::fopen(dump, "w")) {
          std::fprintf(f, "// %s\n%s", name, table.c_str());
          std::fclose(f);
        }
      }
      made = compile_kernel(table, name, contract, why);
      if (!made) {
        std::fprintf(stderr, "comfuse: %s\n", why.c_str());
        g_failed[key] = why;
        return cudaErrorInvalidValue;
      }
      disk_cache_store(on_disk, *made);
      k = made.get();
      g_cache[key] = std::move(made);
      }
    }
  }
  if (!launch) return cudaSuccess;
  {
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    if (!k->kernel) {
      if (cudaLibraryLoadData(&k->library, k->image.data(), nullptr, nullptr, 0, nullptr, nullptr, 0) != cudaSuccess) return cudaGetLastError();
      if (cudaLibraryGetKernel(&k->kernel, k->library, k->lowered_name.c_str()) != cudaSuccess) return cudaGetLastError();
    }
  }
  return launch_pair_kernel(reinterpret_cast<const void*>(k->kernel), k->max_clusters, sh, name, maps, p, st);
}

}  // namespace comfuse
