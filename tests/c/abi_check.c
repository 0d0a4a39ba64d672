/* Compiles include/drk.h as plain C99 and exercises the host-only entry points through dlopen. */
#include <dlfcn.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "drk.h"

typedef void (*params_default_fn)(drk_pg_params*);
typedef size_t (*workspace_fn)(int64_t, int32_t, int32_t, int32_t, int32_t, const drk_pg_params*, int32_t);
typedef int (*chunks_fn)(int64_t, int32_t, int32_t, int32_t, const drk_pg_params*, int32_t*);
typedef const char* (*status_fn)(int);
typedef int (*version_fn)(void);
typedef void (*reward_default_fn)(drk_reward_params*);

int main(int argc, char** argv) {
  if (argc < 2) return 2;
  void* lib = dlopen(argv[1], RTLD_NOW);
  if (!lib) { fprintf(stderr, "dlopen: %s\n", dlerror()); return 3; }
  params_default_fn params_default = (params_default_fn)dlsym(lib, "drk_pg_params_default");
  workspace_fn workspace = (workspace_fn)dlsym(lib, "drk_pg_workspace_bytes");
  chunks_fn chunks = (chunks_fn)dlsym(lib, "drk_pg_bwd_chunks");
  status_fn status = (status_fn)dlsym(lib, "drk_status_string");
  version_fn version = (version_fn)dlsym(lib, "drk_version");
  reward_default_fn reward_default = (reward_default_fn)dlsym(lib, "drk_reward_params_default");
  if (!params_default || !workspace || !chunks || !status || !version || !reward_default) return 4;
  if (!dlsym(lib, "drk_trloo_advantage") || !dlsym(lib, "drk_pg_logprob_fwd") || !dlsym(lib, "drk_pg_loss_fwd_bwd") ||
      !dlsym(lib, "drk_pg_diagnostics") || !dlsym(lib, "drk_reward") || !dlsym(lib, "drk_pg_logprob_fwd_noalloc") ||
      !dlsym(lib, "drk_last_launch_count"))
    return 5;

  drk_pg_params p;
  memset(&p, 0xff, sizeof p);
  params_default(&p);
  if (fabsf(p.mrs_lo - 0.999f) > 1e-7f || fabsf(p.mrs_hi - 1.001f) > 1e-7f || fabsf(p.veto_ratio - 1e-4f) > 1e-10f) return 6;
  if (p.norm != DRK_NORM_KEPT_TOKENS || p.engine != DRK_ENGINE_AUTO || p.dw_chunk_events != NULL || p.n_dw_chunk_events != 0)
    return 7;
  drk_reward_params r;
  reward_default(&r);
  if (r.speedup_clip != 3.0f || r.prs_mode != DRK_PRS_OFF) return 8;

  const size_t fwd = workspace(32768, 5120, 151936, 32, DRK_BF16, &p, 0);
  const size_t all = workspace(32768, 5120, 151936, 32, DRK_BF16, &p, 1);
  if (fwd == 0 || all <= fwd || workspace(-1, 5120, 151936, 32, DRK_BF16, &p, 1) != 0) return 9;
  int32_t vc = 0;
  const int n = chunks(32768, 5120, 151936, DRK_BF16, &p, &vc);
  if (n < 1 || vc <= 0 || (int64_t)n * vc < 151936 || (int64_t)(n - 1) * vc >= 151936) return 10;
  if (chunks(32768, 0, 151936, DRK_BF16, &p, &vc) != DRK_ERR_INVALID_ARG) return 11;
  if (strcmp(status(DRK_OK), "ok") != 0 || version() < 100) return 12;
  printf("abi ok: workspace %zu bytes, %d chunks of %d columns\n", all, n, (int)vc);
  dlclose(lib);
  return 0;
}
