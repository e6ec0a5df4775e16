/* A minimal NVTX tool for the tracing tests: the NVTX loader opens this library when NVTX_INJECTION64_PATH names it,
 * and every range that a library of the process pushes or pops in a domain is written as a text line to the file that
 * SWAM_NVTX_PROBE_OUT names ("domain <name>", "push <name>", "pop"). */
#include <nvtx3/nvToolsExt.h>
#include <stdio.h>
#include <stdlib.h>

static FILE* out;

static nvtxDomainHandle_t NVTX_API on_domain_create(const char* name) {
  if (out) { fprintf(out, "domain %s\n", name); fflush(out); }
  return (nvtxDomainHandle_t)(size_t)1;
}
static int NVTX_API on_push(nvtxDomainHandle_t dom, const nvtxEventAttributes_t* a) {
  (void)dom;
  if (out) {
    fprintf(out, "push %s\n", a && a->messageType == NVTX_MESSAGE_TYPE_ASCII ? a->message.ascii : "?");
    fflush(out);
  }
  return 0;
}
static int NVTX_API on_pop(nvtxDomainHandle_t dom) {
  (void)dom;
  if (out) { fprintf(out, "pop\n"); fflush(out); }
  return 0;
}

int InitializeInjectionNvtx2(NvtxGetExportTableFunc_t get_table) {
  const NvtxExportTableCallbacks* cb = (const NvtxExportTableCallbacks*)get_table(NVTX_ETID_CALLBACKS);
  NvtxFunctionTable table = 0;
  unsigned int size = 0;
  if (!cb || !cb->GetModuleFunctionTable(NVTX_CB_MODULE_CORE2, &table, &size)) return 0;
  if (size <= NVTX_CBID_CORE2_DomainCreateA) return 0;
  if (!out) {
    const char* path = getenv("SWAM_NVTX_PROBE_OUT");
    if (path) out = fopen(path, "a");
  }
  *table[NVTX_CBID_CORE2_DomainCreateA] = (NvtxFunctionPointer)on_domain_create;
  *table[NVTX_CBID_CORE2_DomainRangePushEx] = (NvtxFunctionPointer)on_push;
  *table[NVTX_CBID_CORE2_DomainRangePop] = (NvtxFunctionPointer)on_pop;
  return 1;
}
