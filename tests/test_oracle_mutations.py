"""Do the pins pin?  Each case plants one plausible mistake in a COPY of the oracle's source (a
dropped term, a wrong sign, an off-by-one, a swapped operand, a wrong constant), builds the copy and
runs the pin tests against it in a child process: the run must fail.  A mutant that passes would
mean that part of the oracle is checked against nothing but itself.  (The CUDA library is not
involved: the mistakes live in the oracle, on the CPU.)"""
import concurrent.futures
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "wwws_oracle.c")

# (name, text in the oracle, mutated text, pin files that must catch it)
MUTANTS = [
    ("philox_multiplier", "0xD2511F53u * c0", "0xD2511F57u * c0", ["test_oracle_rng_gossip.py", "test_oracle_create.py"]),
    ("ppm_scale", "(uint64_t)x * 1000000u) >> 32", "(uint64_t)x * 1000001u) >> 32", ["test_oracle_rng_gossip.py"]),
    ("staleness_range_one_short", "w[0], cfg->init_stale_max + 1);", "w[0], cfg->init_stale_max);", ["test_oracle_create.py"]),
    ("stale_diagonal", "uint32_t stale = (i == j) ? 0 : orc_below(", "uint32_t stale = orc_below(", ["test_oracle_create.py"]),
    ("initial_offline_bit_inverted", "pack_entry(p->ver - stale, !p->online, adv_cap_of(p), 0)", "pack_entry(p->ver - stale, p->online, adv_cap_of(p), 0)",
     ["test_oracle_create.py"]),
    ("merge_keeps_the_older", "{ return a > b ? a : b; }", "{ return a < b ? a : b; }", ["test_oracle_rng_gossip.py"]),
    ("hello_dropped", "Vn[(size_t)p * N + i] = orc_merge(Vn[(size_t)p * N + i], self[i]);", ";", ["test_oracle_rng_gossip.py"]),
    ("no_offline_mark", "row[p] = orc_merge(row[p], V[(size_t)i * N + p] | OFFBIT);", "row[p] = orc_merge(row[p], V[(size_t)i * N + p]);",
     ["test_oracle_rng_gossip.py"]),
    ("priority_window_quarter_rate", "return active ? p->cap_true / 2 : p->cap_true;", "return active ? p->cap_true / 4 : p->cap_true;",
     ["test_oracle_create.py", "test_oracle_duel_settle.py"]),
    ("drain_rate_per_ms", "(uint64_t)p->cap_eff * dt / 1000);", "(uint64_t)p->cap_eff * dt);", ["test_oracle_duel_settle.py", "test_oracle_queue.py"]),
    ("spare_sign", "spare = 1.0f - utilf;", "spare = 1.0f + utilf;", ["test_oracle_dispatch.py"]),
    ("reputation_transposed", "rep = a / b; }", "rep = b / a; }", ["test_oracle_dispatch.py"]),
    ("weight_scale", "float scaled = score * 256.0f;", "float scaled = score * 128.0f;", ["test_oracle_dispatch.py"]),
    ("interval_end_inclusive", "if (acc > r64) {", "if (acc >= r64) {", ["test_oracle_dispatch.py"]),
    ("origin_may_pick_itself", "if (id >= n->N || id == o) continue;", "if (id >= n->N) continue;", ["test_oracle_dispatch.py"]),
    ("probe_ignores_load", "if (!(util_pm(n, p) < p->accept_util_pm)) return 0;", "", ["test_oracle_dispatch.py", "test_policy_sweep.py"]),
    ("duel_threshold_swapped", "P[a].quality_fx - P[b].quality_fx) >> 1;", "P[b].quality_fx - P[a].quality_fx) >> 1;", ["test_oracle_duel_settle.py"]),
    ("majority_off_by_one", "2 * votes_a > nj ? 1 : (2 * votes_a < nj ? 2 : 3)", "2 * votes_a >= nj ? 1 : (2 * votes_a < nj ? 2 : 3)",
     ["test_oracle_duel_settle.py"]),
    ("judges_keep_the_whole_pot", "share = pot / nj;", "share = pot;", ["test_oracle_duel_settle.py"]),
    ("latency_floor", "{ return (a + b - 1) / b; }", "{ return a / b; }", ["test_oracle_duel_settle.py", "test_oracle_queue.py"]),
    ("no_version_bump", "            P[j].ver += 1;\n", "", ["test_oracle_rng_gossip.py"]),
    ("advertised_queue_in_8_token_units", "(uint64_t)P[j].backlog >> 4);", "(uint64_t)P[j].backlog >> 3);", ["test_oracle_rng_gossip.py", "test_oracle_dispatch.py"]),
    ("partner_may_be_oneself", "if (p != i && e != 0 && !(e & OFFBIT)) partner = p;", "if (e != 0 && !(e & OFFBIT)) partner = p;", ["test_oracle_rng_gossip.py"]),
    ("pull_from_believed_offline", "if (p != i && e != 0 && !(e & OFFBIT)) partner = p;", "if (p != i && e != 0) partner = p;", ["test_oracle_rng_gossip.py"]),
    ("leaver_keeps_its_queue", "{ P[j].online = 0; P[j].backlog = 0; }", "{ P[j].online = 0; }", ["test_oracle_rng_gossip.py", "test_oracle_duel_settle.py"]),
    ("offload_without_funds", "&& orc_ppm(rx.w[0]) < P[o].offload_ppm && P[o].credit >= c->reward_R;", "&& orc_ppm(rx.w[0]) < P[o].offload_ppm;",
     ["test_oracle_dispatch.py", "test_oracle_duel_settle.py"]),
    ("offline_origin_served", "if (o >= n->N || !P[o].online) { n->exec_a[x] = -3; continue; }", "if (o >= n->N) { n->exec_a[x] = -3; continue; }",
     ["test_oracle_dispatch.py", "test_oracle_duel_settle.py"]),
    ("offline_judges_allowed", "if (P[id].online) jd[nj++] = (int)id;", "jd[nj++] = (int)id;", ["test_oracle_duel_settle.py"]),
    ("noise_never_flips", "if (orc_ppm(y.w[1]) < c->p_noise_ppm) vote_a = !vote_a;", "", ["test_oracle_duel_settle.py"]),
    ("loser_not_charged", "post(n, r, (uint32_t)q, OP_PENALTY, (uint32_t)lose, -c->penalty_P);", "", ["test_oracle_duel_settle.py"]),
    ("winner_and_loser_swapped", "int win = oc == 1 ? a : b, lose = oc == 1 ? b : a;", "int win = oc == 1 ? b : a, lose = oc == 1 ? a : b;", ["test_oracle_duel_settle.py", "test_oracle_replicator.py"]),
    ("duel_pays_challenger_nothing", "post(n, r, (uint32_t)q, OP_EARN_CHALLENGER, (uint32_t)b, c->reward_R);", "", ["test_oracle_duel_settle.py"]),
    ("hop_latency_dropped", " + (a >= 0 ? c->hop_ms : 0);", ";", ["test_oracle_duel_settle.py", "test_oracle_queue.py"]),
    ("deadline_ignores_slo_factor", "(uint64_t)c->slo_num * ceil_div(work * 1000, c->cap_ref_tok_s) / c->slo_den;", "ceil_div(work * 1000, c->cap_ref_tok_s);",
     ["test_oracle_duel_settle.py", "test_oracle_queue.py"]),
    ("judge_work_like_an_execution", "(int64_t)(li + 2 * lo); ++nj;", "(int64_t)(li + lo); ++nj;", ["test_oracle_duel_settle.py", "test_oracle_queue.py"]),
    ("majority_needs_only_half", "if (2 * online <= n->N) { commit = 0;", "if (2 * online < n->N) { commit = 0;", ["test_oracle_chain.py", "test_oracle_duel_settle.py"]),
    ("fifo_ignores_earlier_requests", "uint64_t ahead = (c->flags & 16) ? (uint64_t)P[a < 0 ? o : (uint32_t)a].d_backlog : 0;", "uint64_t ahead = 0;",
     ["test_oracle_duel_settle.py", "test_oracle_queue.py"]),
    ("block_rank_not_relative_to_the_origin", "return (o / WIN + rank) % n_blk;", "return rank % n_blk;", ["test_oracle_dispatch.py"]),
    ("near_flag_never_set", "out.lane = c; out.near = m <= S / 100000;", "out.lane = c; out.near = 0;", ["test_oracle_dispatch.py"]),
    ("probe_budget_not_counted", "        ct->n_probes++;\n", "", ["test_oracle_dispatch.py", "test_oracle_duel_settle.py"]),
    ("greedy_takes_the_highest_lane_on_ties", "if (best < 0 || w->W[c] > w->W[best]) { second = best; best = c; }", "if (best < 0 || w->W[c] >= w->W[best]) { second = best; best = c; }",
     ["test_oracle_dispatch.py"]),
    ("misreport_not_advertised", "{ return (uint64_t)p->cap_eff * p->misreport_mul; }", "{ return (uint64_t)p->cap_eff; }", ["test_oracle_create.py", "test_oracle_rng_gossip.py"]),
    ("reputation_counters_not_committed", "p->credit += p->d_credit; p->wins += p->d_wins; p->duels += p->d_duels;", "p->credit += p->d_credit;",
     ["test_oracle_duel_settle.py", "test_oracle_dispatch.py"]),
    ("winner_not_counted", "P[win].d_wins += 1;", "", ["test_oracle_duel_settle.py"]),
    ("duels_counted_for_the_executor_only", "P[a].d_duels += 1; P[b].d_duels += 1;", "P[a].d_duels += 1;", ["test_oracle_duel_settle.py"]),
    ("block_id_ignores_the_parent", "orc_mix64(orc_mix64(st[S_CHAIN_HEAD] ^ chain_key(n, r)) + st[S_PENDING_DIGEST]", "orc_mix64(orc_mix64(chain_key(n, r)) + st[S_PENDING_DIGEST]",
     ["test_oracle_chain.py"]),
    ("record_hash_ignores_the_amount", "orc_mix64(orc_mix64(chain_key(n, r) ^ word) + (uint64_t)amount);", "orc_mix64(orc_mix64(chain_key(n, r) ^ word));", ["test_oracle_chain.py"]),
    ("earnings_of_the_open_block_spendable", "if (P[o].credit - P[o].blk_spent - P[o].d_spent < pay)", "if (P[o].credit + P[o].d_credit - P[o].blk_spent - P[o].d_spent < pay)",
     ["test_oracle_duel_settle.py"]),
    ("spending_forgotten_between_batches", "P[j].blk_spent = commit ? 0 : P[j].blk_spent + P[j].d_spent;", "P[j].blk_spent = 0;", ["test_oracle_duel_settle.py"]),
    ("served_not_counted", "P[a].d_backlog += (int64_t)work; P[a].served += 1; ex = (uint32_t)a;", "P[a].d_backlog += (int64_t)work; ex = (uint32_t)a;",
     ["test_oracle_duel_settle.py", "test_policy_sweep.py"]),
    ("pairwise_exchange_one_way", "for (uint32_t col = 0; col < N; ++col) pnew[col] = orc_merge(pnew[col], irow[col]);", ";", ["test_oracle_rng_gossip.py"]),
    ("stake_in_percent", "p->stake = pos * p->stake_pm / 1000;", "p->stake = pos * p->stake_pm / 100;", ["test_oracle_create.py", "test_oracle_dispatch.py"]),
]


def _run_mutant(tmp, case):
    name, old, new, files = case
    text = open(SRC).read()
    if text.count(old) != 1:
        return name, "stale", f"{text.count(old)} occurrences of the text to mutate"
    src = os.path.join(tmp, name + ".c")
    so = os.path.join(tmp, name + ".so")
    open(src, "w").write(text.replace(old, new))
    gcc = subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC", "-w", "-o", so, src],
                         capture_output=True, text=True)
    if gcc.returncode != 0:
        return name, "build", gcc.stderr[-500:]
    env = dict(os.environ, WWWS_ORACLE_LIBRARY=so)
    out = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "not gpu", "-p", "no:cacheprovider"]
                         + [os.path.join(ROOT, "tests", f) for f in files],
                         capture_output=True, text=True, timeout=900, cwd=ROOT, env=env)
    return name, ("caught" if out.returncode == 1 else "survived" if out.returncode == 0 else "error"), out.stdout[-600:]


def test_every_planted_mistake_is_caught_by_a_pin(tmp_path):
    if os.environ.get("WWWS_ORACLE_LIBRARY"):
        pytest.skip("already running against a mutated oracle")
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 2)) as pool:
        results = list(pool.map(lambda c: _run_mutant(str(tmp_path), c), MUTANTS))
    bad = [(n, what, tail) for n, what, tail in results if what != "caught"]
    assert not bad, "\n".join(f"{n}: {what}\n{tail}" for n, what, tail in bad)
