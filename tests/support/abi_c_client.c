/* A plain C99 client of the library: the header must compile as C and every entry point must
 * link.  Only the host-side calls run (no GPU needed). */
#include <stdio.h>
#include <string.h>

#include "sparseloco.h"

int main(void) {
  /* taking every entry point's address makes the linker resolve it */
  typedef void (*fn)(void);
  const fn fns[] = {(fn)sl_num_chunks, (fn)sl_codes_stride, (fn)sl_codes_bytes, (fn)sl_compress, (fn)sl_compress_batch, (fn)sl_aggregate,
                    (fn)sl_outer_apply, (fn)sl_aggregate_apply, (fn)sl_outer_step, (fn)sl_compress_batch_bf16, (fn)sl_aggregate_apply_bf16, (fn)sl_outer_apply_bf16,
                    (fn)sl_outer_step_bf16, (fn)sl_idx12_stride,
                    (fn)sl_pack_idx12, (fn)sl_unpack_idx12, (fn)sl_embed_reproject, (fn)sl_round_tf32, (fn)sl_subspace_project, (fn)sl_subspace_reconstruct,
                    (fn)sl_debug_set_wait_limit, (fn)sl_debug_bounds_selftest, (fn)sl_strerror};
  uint64_t offset[3] = {0, 4096 * 2 + 5, 4096 * 2 + 5 + 100};
  sl_layout lay;
  size_t i;
  lay.n_total = offset[2];
  lay.n_tensors = 2;
  lay.offset = offset;
  lay.cols = NULL;
  for (i = 0; i < sizeof(fns) / sizeof(fns[0]); ++i)
    if (!fns[i]) return 2;
  if (sl_num_chunks(&lay, 4096) != 4) return 3;
  if (sl_codes_stride(64, 2) != 16 || sl_idx12_stride(64) != 96) return 4;
  if (sl_codes_bytes(&lay, 4096, 64, 2) != 4 * 16 || sl_codes_bytes(&lay, 4096, 64, 3) != 0) return 7;
  if (sl_compress(NULL, NULL, NULL, &lay, 0.95f, 4096, 64, 2, NULL, NULL, NULL, NULL, NULL) != SL_ERR_INVALID_ARG) return 5;
  if (strlen(sl_strerror(SL_ERR_ALIGNMENT)) == 0) return 6;
  printf("c client ok: %d entry points\n", (int)(sizeof(fns) / sizeof(fns[0])));
  return 0;
}
