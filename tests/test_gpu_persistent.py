"""The persistent decode-step kernel (one cooperative launch for the whole forward of a step) against the oracle.

It is an alternative schedule of the same step, switched on by an environment variable that the library reads once
per process, so every case runs in a child process: whole generations in lock step with the oracle (logits,
confidences, accept sets, jump chains, row tables: the same harness and tolerances as the separate kernels),
the separated workloads whose free runs must be bit-identical to the stored oracle traces, the ragged and
degenerate shapes, head dim 128, and the device-resident loop around it."""
import os
import subprocess
import sys

from gpu_common import engine, requires_gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _child(code, expect, timeout=900):
    engine()
    env = dict(os.environ, ODB_PERSISTENT="1")
    r = subprocess.run([sys.executable, "-c", "import sys; sys.path.insert(0, 'tests')\n" + code], cwd=ROOT, env=env,
                       capture_output=True, text=True, timeout=timeout)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-3000:]
    assert expect in r.stdout, r.stdout[-3000:]
    return r.stdout


@requires_gpu
def test_persistent_step_is_the_path_that_runs():
    """With the switch on a step is two launches of the forward (the persistent kernel and the per-row merge of
    the LM head's statistics) instead of one per projection and short kernel."""
    out = _child(
        "import synth\n"
        "from paper_2511_21759_b200 import engine as E\n"
        "shape = synth.TINY_PEAKY\n"
        "gm = E.Model.from_synth(shape, seed=0, max_batch=1, max_seq=128, max_block=16, max_copies=4)\n"
        "s = E.Session(gm); s.set_sequence(0, synth.sequence(0, 0, 64, 64, shape), 64)\n"
        "gp = E.DecodeParams(block_len=16, n_copies=4)\n"
        "s.refresh_prefill(gp, 0); s.unmask_accept(gp, True); s.profile_read()\n"
        "s.block_decode_step(gp); s.unmask_accept(gp, False)\n"
        "n = s.profile_read()[1]; assert s.status() == 0\n"
        "print('launches', n['gemm'], n['attention'], n['elementwise'], n['confidence'])\n", "launches")
    assert "launches 1 0 0 1" in out, out


@requires_gpu
def test_persistent_step_in_lockstep_and_free_running():
    _child(
        "import test_gpu_generate as t\n"
        "for wl, tol, fused in [('cfg1_tiny', 2e-2, False), ('cfg1_tiny_c4', 2e-2, False), ('peaky_c1', 4e-2, False),\n"
        "                       ('peaky_c4', 4e-2, False), ('peaky_c8', 4e-2, False), ('peaky_c8', 4e-2, True)]:\n"
        "    t.test_lockstep_generate(wl, tol, fused)\n"
        "for name in sorted(t.SEPARATED['workloads']):\n"
        "    for resident in (False, True):\n"
        "        t.test_free_run_identical_on_separated_workloads(name, resident)\n"
        "    t.test_separated_workloads_are_separated_by_the_measured_error(name)\n"
        "for copies in (1, 4, 8):\n"
        "    t.test_resident_loop_equals_call_by_call(copies)\n"
        "t.test_ragged_batch_equals_independent_runs()\n"
        "print('persistent lockstep ok')\n", "persistent lockstep ok", timeout=1500)


@requires_gpu
def test_persistent_step_on_edge_shapes():
    names = ["ragged_tail", "ragged_peaky_c8", "no_prompt", "response_of_one", "block_3_c4", "hd128_ragged", "hd128_one_tile",
             "hd128_c8_stage2", "hd128_c4_noprompt", "long_2048"]
    _child(
        "import test_gpu_edges as t\n"
        f"for c in t.CASES:\n    if c[0] in {names!r}: t.test_edge_case_in_lockstep(*c)\n"
        "t.test_an_expired_device_wait_is_reported_and_the_session_stays_usable()\n"
        "for a in (('TINY_PEAKY', 1), ('TINY_PEAKY', 8), ('TINY_HD128', 4)): t.test_poisoned_workspace_reads_nothing_unwritten(*a)\n"
        "print('persistent edges ok')\n", "persistent edges ok", timeout=1500)
