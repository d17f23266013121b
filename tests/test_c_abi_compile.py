"""The header is plain C: a C99 program that includes it compiles without warnings, links against
the library and drives the host-only scheduler (no GPU needed)."""
import os
import subprocess
import tempfile

from paper_1509_04210_b200 import binding as rb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

PROGRAM = r"""
#include <stdio.h>
#include "rudra_ps.h"

int main(void) {
  rudra_event ev[64];
  rudra_sched* s = rudra_sched_create(6, 2, RUDRA_SCHED_SOFTSYNC_ROUNDS, 42u, 0.3, 0);
  unsigned pushes = 0, steps = 0;
  int i;
  if (!s) return 1;
  if (rudra_sched_next(s, ev, 64) != 64) return 2;
  for (i = 0; i < 64; ++i) {
    if (ev[i].kind == RUDRA_EV_PUSH) { ++pushes; if (ev[i].pulled_ts > ev[i].ts) return 3; }
    if (ev[i].kind == RUDRA_EV_STEP) ++steps;
  }
  if (rudra_sched_on_pull(s, 1, 0) != 0 || rudra_sched_on_pull(s, 99, 0) != RUDRA_E_INVAL) return 7;
  if (rudra_sched_on_pull(s, 1, 1000000u) != RUDRA_E_BAD_TS) return 8;
  rudra_sched_destroy(s);
  /* learners behind a server tree: 2 leaves of 3; a fan-in that does not divide c is refused */
  s = rudra_sched_create_tree(6, 1, RUDRA_SCHED_SOFTSYNC_ROUNDS, 42u, 0.3, 0, 3);
  if (!s || rudra_sched_next(s, ev, 64) != 64) return 9;
  {
    unsigned relays = 0;
    for (i = 0; i < 64; ++i) relays += ev[i].kind == RUDRA_EV_RELAY;
    if (relays < 8) return 10;
  }
  rudra_sched_destroy(s);
  if (rudra_sched_create_tree(6, 2, RUDRA_SCHED_SOFTSYNC_ROUNDS, 42u, 0.3, 0, 2) != NULL) return 11;
  if (rudra_leaf_average(NULL, 3, RUDRA_GRAD_F32, 64, NULL, NULL) != RUDRA_E_INVAL) return 12;
  if (rudra_ps_push_group(NULL, NULL, 1, NULL, 1) != RUDRA_E_INVAL) return 13;
  /* bad arguments are refused before any device work, with a reason */
  if (rudra_ps_create(0, 4, 1, 0.1f, 0.0f, 0.0f) != NULL) return 4;
  if (rudra_ps_step(NULL) != RUDRA_E_INVAL) return 5;
  printf("%u %u %s\n", pushes, steps, rudra_last_error());
  return sizeof(rudra_event) == 40 ? 0 : 6;
}
"""


def test_c99_program_compiles_links_and_runs():
    lib = rb.library_path()
    rb.lib()
    with tempfile.TemporaryDirectory() as d:
        src, exe = os.path.join(d, "t.c"), os.path.join(d, "t")
        with open(src, "w") as f:
            f.write(PROGRAM)
        subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                               src, lib, "-Wl,-rpath," + os.path.dirname(lib), "-o", exe])
        out = subprocess.run([exe], capture_output=True, text=True, timeout=60)
        assert out.returncode == 0, (out.returncode, out.stdout, out.stderr)
        pushes, steps = (int(x) for x in out.stdout.split()[:2])
        assert pushes >= 20 and steps == pushes // 3
        assert "handle" in out.stdout
