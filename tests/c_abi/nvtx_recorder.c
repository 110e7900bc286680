/* A minimal NVTX tool for the tests: loaded by the NVTX header code inside libef (environment
 * variable NVTX_INJECTION64_PATH), it appends every pushed range name, and a "pop" line for every
 * pop, to the file named by EF_NVTX_LOG.  Uses only the public injection interface. */
#include <stdio.h>
#include <stdlib.h>

#include <nvtx3/nvToolsExt.h>

static void record(const char* line) {
    const char* path = getenv("EF_NVTX_LOG");
    if (!path) return;
    FILE* f = fopen(path, "a");
    if (!f) return;
    fprintf(f, "%s\n", line);
    fclose(f);
}

static int NVTX_API on_push(const char* name) {
    record(name ? name : "(null)");
    return 0;
}

static int NVTX_API on_pop(void) {
    record("pop");
    return 0;
}

int InitializeInjectionNvtx2(NvtxGetExportTableFunc_t get_table) {
    const NvtxExportTableCallbacks* cb = (const NvtxExportTableCallbacks*)get_table(NVTX_ETID_CALLBACKS);
    NvtxFunctionTable table = 0;
    unsigned int size = 0;
    if (!cb || !cb->GetModuleFunctionTable(NVTX_CB_MODULE_CORE, &table, &size)) return 0;
    if (size <= NVTX_CBID_CORE_RangePop) return 0;
    *table[NVTX_CBID_CORE_RangePushA] = (NvtxFunctionPointer)on_push;
    *table[NVTX_CBID_CORE_RangePop] = (NvtxFunctionPointer)on_pop;
    return 1;
}
