"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's source (on the
CPU), builds it, and checks that the pin tests reject it.  The unmodified source must pass the same
battery."""
import os
import subprocess

import pytest

import oracle
from tests import test_oracle_golden as G
from tests import test_delay_guideline as D
from tests import test_oracle_invariants as I
from tests import test_oracle_sharded as S

SRC = os.path.join(os.path.dirname(oracle.__file__), "dasgd_oracle.cpp")

MUTATIONS = {
    "blend weights swapped": ("xi * wi + one_minus_xi * avg", "one_minus_xi * wi + xi * avg"),
    "weight decay dropped": ("o->decoupled_wd ? gi : gi + lambda * w_old", "gi"),
    "nesterov looks ahead with the old momentum": (
        "o->m[i] = static_cast<float>(mu * static_cast<double>(o->m[i]) + gp);\n        dir = o->nesterov ? gp + mu * static_cast<double>(o->m[i])",
        "const double m_prev = o->m[i];\n        o->m[i] = static_cast<float>(mu * static_cast<double>(o->m[i]) + gp);\n        dir = o->nesterov ? gp + mu * m_prev"),
    "nesterov ignored": ("dir = o->nesterov ? gp + mu * static_cast<double>(o->m[i]) : static_cast<double>(o->m[i]);",
                         "dir = static_cast<double>(o->m[i]);"),
    "decoupled decay also enters the gradient": ("o->decoupled_wd ? gi : gi + lambda * w_old", "gi + lambda * w_old"),
    "decoupled decay not scaled by the learning rate": ("o->decoupled_wd ? eta * lambda * w_old : 0.0", "o->decoupled_wd ? lambda * w_old : 0.0"),
    "decoupled decay dropped": ("o->decoupled_wd ? eta * lambda * w_old : 0.0", "0.0"),
    "momentum applied to the sum": ("mu * static_cast<double>(o->m[i]) + gp", "mu * (static_cast<double>(o->m[i]) + gp)"),
    "step uses the gradient instead of the momentum": (": static_cast<double>(o->m[i]);", ": gp;"),
    "sign of the step": ("w_old - decay - eta * dir", "w_old - decay + eta * dir"),
    "mean not divided": ("acc / static_cast<double>(o->K)", "acc"),
    "mean skips worker 0": ("for (int32_t k = 0; k < o->K; ++k) acc +=", "for (int32_t k = 1; k < o->K; ++k) acc +="),
    "merge fires from the start point": ("d > 0 && u - d >= tau && (u - d) % tau == 0", "d > 0 && (u - d) % tau == 0 && !o->pending.empty()"),
    "merge one step late": ("d > 0 && u - d >= tau && (u - d) % tau == 0", "d > 0 && u - d - 1 >= tau && (u - d - 1) % tau == 0"),
    "snapshot before the merge of the same step": None,   # handled below: reorder two blocks
    "snapshot one step early": ("if (u % tau == 0) {", "if ((u + 1) % tau == 0) {"),
    "bf16 truncates": ("if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1;", ""),
    "bf16 rounds ties up": ("(rest == 0x8000u && (keep & 1u))", "(rest == 0x8000u)"),
    "delta merge sign": ("wi + (avg - static_cast<double>(q.snap[i]))", "wi - (avg - static_cast<double>(q.snap[i]))"),
    "delta merge uses the current weights as the snapshot": ("static_cast<double>(q.snap[i])))", "wi))"),
    "merge takes the newest mean": ("const Pending &q = o->pending.front();", "const Pending &q = o->pending.back();"),
    "guideline: tau equals d": ("*tau = k + 1;", "*tau = k;"),
    "guideline: non-strict inequality": ("while (!(t_c < static_cast<double>(k) * t_p)) ++k;",
                                         "while (!(t_c <= static_cast<double>(k) * t_p)) ++k;"),
    "sharded mean divided by the shard's own size": ("total[p] / static_cast<double>(o->K_total)", "total[p] / static_cast<double>(o->K)"),
    "partial sum already divided": ("    sum[p] = acc;", "    sum[p] = acc / static_cast<double>(o->K);"),
    "partial sum takes the newest snapshot": (
        "  const Pending *q = nullptr;\n  for (const auto &cand : o->pending)\n    if (!cand.averaged) { q = &cand; break; }",
        "  const Pending *q = nullptr;\n  for (const auto &cand : o->pending)\n    if (!cand.averaged) { q = &cand; }"),
    "momentum averaging: blend takes the mean of the weights": ("avg_m = q.mean_m[p]", "avg_m = q.mean[p]"),
    "momentum averaging: snapshot taken from the weights": ("q.snap_m = o->m;", "q.snap_m = o->w;"),
    "momentum averaging: blend weights swapped": ("xi * mi + one_minus_xi * avg_m", "one_minus_xi * mi + xi * avg_m"),
    "momentum averaging: delta sign": ("mi + (avg_m - static_cast<double>(q.snap_m[i]))", "mi - (avg_m - static_cast<double>(q.snap_m[i]))"),
    "momentum averaging: fresh buffers instead of the snapshot": ("acc += static_cast<double>(q->snap_m[static_cast<size_t>(k) * P + p]);",
                                                                  "acc += static_cast<double>(o->m[static_cast<size_t>(k) * P + p]);"),
    "momentum averaging: switched on for everyone": ("bool average_momentum = false;", "bool average_momentum = true;"),
    "momentum merged too": ("o->pending.pop_front();\n  return ORACLE_OK;", "for (auto &x : o->m) x *= o->xi;\n  o->pending.pop_front();\n  return ORACLE_OK;"),
}


def battery():
    """A fixed list of pin tests (the same functions pytest runs), called directly."""
    for name in G.CASES:
        G.test_golden_trajectory(name)
    I.test_minibatch_sgd_equivalence()
    I.test_local_sgd_special_case()
    for tau, d in [(1, 1), (2, 1), (1, 2)]:
        I.test_xi_one_is_independent_sgd_and_matches_torch(tau, d)
    I.test_identical_replicas_stay_identical_and_mean_is_identity()
    for args in [(2, 2, 1, 0.25), (4, 1, 1, 0.25), (5, 2, 2, 0.75)]:
        I.test_mean_recursion(*args)
    for args in [(2, 2, 1, 0.25), (2, 1, 1, 0.5), (2, 1, 2, 0.25), (4, 2, 3, 0.5)]:
        I.test_against_exact_history_form(*args)
    I.test_deviation_contracts_by_xi_at_each_merge(0.25)
    I.test_delta_merge_keeps_mean_on_plain_sgd()
    I.test_momentum_closed_form_constant_gradient()
    I.test_weight_decay_closed_form_zero_gradient()
    I.test_nesterov_matches_torch()
    I.test_decoupled_weight_decay_matches_scaled_weights_then_torch(0.9, False)
    I.test_decoupled_weight_decay_matches_scaled_weights_then_torch(0.9, True)
    I.test_decoupled_weight_decay_closed_form_with_momentum()
    I.test_bf16_rounding_matches_torch_cast()
    I.test_bf16_mode_master_equals_f32_run_on_widened_gradients()
    for xi in (0.0, 0.25):
        I.test_momentum_averaging_without_delay_blends_both_halves_of_the_state(xi)
    I.test_momentum_averaging_is_a_no_op_at_xi_one(2, 1)
    for args in [(2, 1, 0.25), (1, 2, 0.25)]:
        I.test_momentum_averaging_uses_the_stale_mean_of_the_buffers(*args)
    I.test_momentum_averaging_delta_form_keeps_the_mean_buffer_on_its_plain_recursion(2, 1)
    I.test_momentum_averaging_identical_workers()
    I.test_momentum_averaging_delta_form_without_delay_equalises_the_buffers()
    I.test_momentum_averaging_mean_is_that_of_the_snapshot_not_of_later_buffers()
    S.test_mean_divides_by_the_total_number_of_workers()
    S.test_shards_in_one_process_reproduce_the_unsharded_oracle(2, 1, (3, 5))
    S.test_one_shard_holding_every_worker_is_the_unsharded_oracle_bit_for_bit()
    S.test_explicit_calls_on_shards_with_two_snapshots_in_flight()
    for row in D.table2():
        D.test_oracle_reproduces_table2(row)
    assert oracle.delay_guideline(1.0, 1.0) == (2, 3)      # Eq. 3 is strict: d > t_c / t_p
    assert oracle.delay_guideline(0.0, 1.0) == (1, 2)      # a delay of at least one step


def build_variant(tmp_path, text, tag):
    src = tmp_path / f"oracle_{tag}.cpp"
    src.write_text(text)
    lib = tmp_path / f"liboracle_{tag}.so"
    subprocess.run(["g++", "-std=c++17", "-O1", "-fPIC", "-shared", "-ffp-contract=off",
                    "-I", os.path.dirname(SRC), str(src), "-o", str(lib)], check=True)
    return oracle.bind(str(lib))


@pytest.fixture
def swap_lib():
    saved = dict(oracle._loaded)
    oracle._lib(False)
    yield lambda L: oracle._loaded.__setitem__(False, L)
    oracle._loaded.clear()
    oracle._loaded.update(saved)


def test_unmodified_source_passes_the_battery(tmp_path, swap_lib):
    swap_lib(build_variant(tmp_path, open(SRC).read(), "clean"))
    battery()


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, tmp_path, swap_lib):
    text = open(SRC).read()
    if MUTATIONS[name] is None:
        a = text.index("  if (d > 0 && u - d >= tau && (u - d) % tau == 0) {")
        b = text.index("  if (u % tau == 0) {")
        c = text.index("  return rc;\n}\n", b)
        merge_block, snap_block = text[a:b], text[b:c]
        mutated = text[:a] + snap_block + merge_block + text[c:]
    else:
        old, new = MUTATIONS[name]
        assert text.count(old) >= 1, f"mutation site not found: {old}"
        mutated = text.replace(old, new)
    assert mutated != text
    swap_lib(build_variant(tmp_path, mutated, "mut"))
    with pytest.raises((AssertionError, oracle.OracleError)):
        battery()
