"""Do the oracle's pins have teeth?  Each case plants ONE plausible mistake in the CPU oracle (a dropped term, a wrong
sign or index, a transposed role, an off-by-one) by rewriting one line of its source in memory, and checks that the pin
named beside it then fails.  Nothing here touches the CUDA path; the mistakes live only for the duration of a test."""
import inspect
import textwrap

import numpy as np
import pytest

import test_oracle_protocol as tp
import test_oracle_update as tu
from oracle import philox, protocol as op, update as up
from paper_1902_01064_b200 import inputs


def plant(monkeypatch, owner, name, old, new):
    """Replace `old` by `new` (exactly one occurrence) in the source of owner.name and install the result."""
    fn = getattr(owner, name)
    src = textwrap.dedent(inspect.getsource(fn))
    assert src.count(old) == 1, f"{name}: expected exactly one occurrence of {old!r}"
    ns = dict(vars(inspect.getmodule(fn)))
    exec(compile(src.replace(old, new), f"<{name} with a planted mistake>", "exec"), ns)
    monkeypatch.setattr(owner, name, ns[name])


RING6 = inputs.ring(6)

PROTOCOL_CASES = [
    # (what is planted, owner, function, old text, new text, pin that must notice)
    ("Eq. 2 numerator without its +1", op, "reduce_weights",
     "nums = [v - (level - s) + 1 for v in vers]", "nums = [v - (level - s) for v in vers]",
     lambda: tp.test_weights_closed_forms()),
    ("staleness window one iteration too wide", op.HopProtocol, "_try_recv",
     ">= max(level - self.s, 0)", ">= max(level - self.s - 1, 0)",
     lambda: tp.test_staleness_window_and_gap("ring6", RING6, 2)),
    ("max_ig initial tokens instead of max_ig - 1 (Fig. alg2)", op.HopProtocol, "__init__",
     "[0] * (max_ig - 1)", "[0] * max_ig",
     lambda: tp.test_token_identity_theorem2_and_capacity("ring6", RING6, 2)),
    ("an update reduced again although an earlier Recv returned it (Fig. alg3's test)", op.HopProtocol, "_try_recv",
     "v > self.iter_reduced[(j, i)]", "v >= self.iter_reduced[(j, i)]",
     lambda: tp.test_stale_reduce_hand_worked_example()),
    ("backup workers ignored: every in-neighbour required (Fig. alg4)", op.HopProtocol, "_try_recv",
     "need = len(self.n_in[i]) - self.b[i]", "need = len(self.n_in[i])",
     lambda: tp.test_backup_prose_example_three_workers()),
    ("updates of later iterations dequeued too (Section 6 keeps them out of reach)", op.HopProtocol, "_drain",
     "if it <= level:", "if it <= level + 1:",
     lambda: tp.test_times_and_versions_match_maxplus_recurrence(2, None, False)),
    ("Send goes to the in-neighbours instead of the out-neighbours", op.HopProtocol, "__init__",
     "self.n_out[j].append(i)", "self.n_out[i].append(j)",
     lambda: tp.test_theorem1_bound_is_reached_on_a_chain()),
    ("serial approach still sends on entering the iteration (Section 3.2)", op.HopProtocol, "_enter",
     "if not self.serial:", "if True:",
     lambda: tp.test_serial_approach_with_s0_waits_for_the_neighbours_compute()),
    ("straggler test off by one: jumps past its slowest out-neighbour (Section 5)", op.HopProtocol, "_decide",
     "for j in outs) - self.max_ig - 1", "for j in outs) - self.max_ig",
     lambda: tp.test_skipping_invariants_and_progress()),
    ("a jump of several iterations pays one token (Section 5: k - k0)", op.HopProtocol, "_commit",
     "self._take_tokens(i, target - k)", "self._take_tokens(i, 1)",
     lambda: tp.test_skipping_invariants_and_progress()),
    ("token not taken on entering the next iteration", op.HopProtocol, "_commit",
     "self._take_tokens(i, 1)\n", "pass\n",
     lambda: tp.test_token_prose_example_sender_stops_at_max_ig()),
    ("NOTIFY-ACK waits for ACK(k) instead of ACK(k-1) (Table 1 row)", op.HopProtocol, "_tokens_available",
     "return k - 1 < 0 or all((k - 1) in", "return k - 2 < 0 or all((k - 2) in",
     lambda: tp.test_notify_ack_chain_reaches_both_bounds_of_table1_exactly()),
]

UPDATE_CASES = [
    ("gradient added instead of subtracted (Fig. alg0 step 3)", up, "run_updates",
     "mix = mix - lr * direction(k, i)", "mix = mix + lr * direction(k, i)",
     lambda: tu.test_standard_training_is_matrix_recursion(inputs.ring(5))),
    ("Reduce weights not normalised (Eq. 1)", up, "run_updates",
     "(float(num[t]) / float(den[k, i])) * X", "float(num[t]) * X",
     lambda: tu.test_complete_graph_is_allreduce_average()),
    ("momentum buffer damped with the gradient", up, "run_updates",
     "M[i] = momentum * M[i] + g", "M[i] = momentum * (M[i] + g)",
     lambda: tu.test_momentum_matches_torch_sgd_single_worker()),
    ("weight decay with the wrong sign", up, "run_updates",
     "g = g + weight_decay * X[(i, k)]", "g = g - weight_decay * X[(i, k)]",
     lambda: tu.test_weight_decay_and_momentum_match_torch_sgd_single_worker()),
    ("serial approach averages before it applies", up, "run_updates",
     "if o == NORMAL and not serial:", "if o == NORMAL:",
     lambda: tu.test_serial_approach_is_apply_then_average(inputs.ring(5))),
    ("a JUMP record applies a gradient", up, "run_updates",
     "if o == NORMAL and not serial:", "if o != IDLE and not serial:",
     lambda: tu.test_jump_record_has_no_gradient_and_uses_held_version()),
    ("hinge active at the kink", up, "hinge_coefficients",
     "y * margins < 1.0", "y * margins <= 1.0",
     lambda: tu.test_hinge_kink_is_inactive_and_csr_equals_dense()),
    ("hinge coefficient with the wrong sign", up, "hinge_coefficients",
     "-y / B", "y / B",
     lambda: tu.test_hinge_gradient_at_zero_closed_form()),
    ("log-loss coefficient with exp(-y m)", up, "log_coefficients",
     "np.exp(y * margins)", "np.exp(-y * margins)",
     lambda: tu.test_log_loss_gradient_matches_autograd_and_finite_differences()),
    ("CSR gradient drops the coefficient", up, "svm_gradient_csr",
     "coef[r] * val[a:e]", "val[a:e]",
     lambda: tu.test_hinge_kink_is_inactive_and_csr_equals_dense()),
    ("Philox multipliers swapped", philox, "philox4x32_10",
     "p0 = M0 * c0", "p0 = M1 * c0",
     lambda: tu.test_philox_known_answers()),
    ("Philox key not bumped between rounds", philox, "philox4x32_10",
     "k0 = (k0 + W0) & 0xFFFFFFFF", "k0 = k0 & 0xFFFFFFFF",
     lambda: tu.test_philox_known_answers()),
    ("uniform without its half-step", philox, "_uniform23",
     "+ 0.5)", "+ 0.25)",
     lambda: tu.test_box_muller_inverts_and_is_standard_normal()),
    ("Box-Muller pair swapped", philox, "box_muller",
     "return rad * np.cos(ang), rad * np.sin(ang)", "return rad * np.sin(ang), rad * np.cos(ang)",
     lambda: tu.test_box_muller_inverts_and_is_standard_normal()),
    ("gradient of the wrong stream / counter word", philox, "synthetic_gradient",
     "z = np.where(e == 0, z0, np.where(e == 1, z1, np.where(e == 2, z2, z3)))",
     "z = np.where(e == 0, z0, np.where(e == 1, z2, np.where(e == 2, z1, z3)))",
     lambda: _gradient_pairs_follow_the_definition()),
]


def _gradient_pairs_follow_the_definition():
    """Columns 4q and 4q+1 are one Box-Muller pair (words 0, 1 of the Philox block), 4q+2 and 4q+3 the other."""
    seed, sigma = 190201064, 1e-3
    g = philox.synthetic_gradient(seed, 5, 9, np.arange(64), sigma) / sigma
    r = philox.philox4x32_10(np.arange(16), np.full(16, 5), np.full(16, 9), np.full(16, philox.GRAD_STREAM), seed & 0xFFFFFFFF, seed >> 32)
    u = [((x >> np.uint32(9)).astype(np.float64) + 0.5) / 2 ** 23 for x in r]
    np.testing.assert_allclose(np.exp(-(g[0::4] ** 2 + g[1::4] ** 2) / 2), u[0], rtol=1e-9)
    np.testing.assert_allclose(np.exp(-(g[2::4] ** 2 + g[3::4] ** 2) / 2), u[2], rtol=1e-9)
    np.testing.assert_allclose(np.mod(np.arctan2(g[1::4], g[0::4]) / (2 * np.pi), 1.0), u[1], atol=1e-9)
    np.testing.assert_allclose(np.mod(np.arctan2(g[3::4], g[2::4]) / (2 * np.pi), 1.0), u[3], atol=1e-9)


def test_the_unmutated_oracle_passes_the_extra_pin():
    _gradient_pairs_follow_the_definition()


@pytest.mark.parametrize("what,owner,name,old,new,pin", PROTOCOL_CASES + UPDATE_CASES,
                         ids=[c[0] for c in PROTOCOL_CASES + UPDATE_CASES])
def test_planted_mistake_is_caught(monkeypatch, what, owner, name, old, new, pin):
    pin()                                             # the pin passes on the oracle as it stands
    plant(monkeypatch, owner, name, old, new)
    with pytest.raises((AssertionError, op.Deadlock, KeyError)):      # a failed check, a stuck protocol or a crash
        pin()
