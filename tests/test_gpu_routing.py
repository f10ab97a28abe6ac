"""The library's host-side routing hook (s2d2_route with the built-in policies of Algorithm
"DoVerify" and with a user callback) against the oracle's restatement of the same policies.
Needs a context, hence a GPU, although routing itself runs on the host."""
import numpy as np
import pytest

from oracle import routing as R
from s2d2_inputs import generate_weights, get_config

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _stats(rng, seq_id, vocab, tau_conf):
    from paper_2603_25702_b200 import DraftStats
    st = DraftStats()
    n = int(rng.integers(1, 9))
    st.seq_id, st.block_start, st.first_masked, st.n_masked = seq_id, 0, 0, n
    st.span_len = int(rng.integers(1, n + 1))
    conf = rng.uniform(0.05, 1.0, size=n)
    for i in range(n):
        st.masked_idx[i] = i
        st.conf[i] = conf[i]
        st.margin[i] = float(rng.uniform(0, conf[i]))
        st.entropy[i] = float(rng.uniform(0, np.log(vocab)))
    st.n_hi = int((np.array([st.conf[i] for i in range(n)]) > tau_conf).sum())
    st.mean_conf = float(np.mean([st.conf[i] for i in range(n)]))
    return st


def test_builtin_policies_and_callback_match_the_oracle():
    from paper_2603_25702_b200 import DraftStats, Engine, RoutePolicy
    wl = get_config("t_f32")
    W = generate_weights(wl.model, seed=0)
    e = Engine(wl.model, block_size=8, max_batch=2, max_seq_len=64, kv_page_tokens=8, tau_conf=0.9,
               stream=torch.cuda.current_stream().cuda_stream)
    e.load_weights(W)
    ids = e.prefill([[1, 2, 3], [4, 5]])
    V = wl.model.vocab
    rng = np.random.default_rng(3)
    hyst = {sid: R.Hysteresis(0.8, 0.2, on=True) for sid in ids}
    for trial in range(200):
        arr = (DraftStats * 2)()
        for k, sid in enumerate(ids):
            arr[k] = _stats(rng, sid, V, 0.9)
        sts = [arr[0], arr[1]]

        def khat(st, entropy, param):
            L = st.span_len
            if entropy:
                return R.khat(R.alpha_entropy([np.float32(st.entropy[i]) for i in range(L)], param, V))
            return R.khat(R.alpha_margin([st.margin[i] for i in range(L)], np.float32(param)))

        # minimum span
        e.set_route_policy(RoutePolicy(RoutePolicy.MIN_SPAN, 3.0, 0, 0, 0, 0, 0))
        assert e.route(arr).tolist() == [int(R.min_span(s.span_len, 3)) for s in sts]
        # static and dynamic score, margin and entropy proxies
        for dyn in (0, 1):
            for ent, param in ((0, 0.1), (1, 2.0)):
                e.set_route_policy(RoutePolicy(RoutePolicy.SCORE, 0.5, 0, 0.3, dyn, ent, param))
                want = []
                for s in sts:
                    sc = R.score(khat(s, ent, param), np.float32(0.3), s.n_hi if dyn else None)
                    want.append(None if abs(sc - 0.5) < 1e-5 else int(R.score_threshold(sc, 0.5)))
                got = e.route(arr).tolist()
                assert all(w is None or w == g for w, g in zip(want, got)), (trial, dyn, ent, want, got)
        # mean confidence and never
        e.set_route_policy(RoutePolicy(RoutePolicy.MEAN_CONF, 0.6, 0, 0, 0, 0, 0))
        assert e.route(arr).tolist() == [int(R.mean_conf([s.conf[i] for i in range(s.n_masked)], np.float32(0.6))) for s in sts]
        e.set_route_policy(RoutePolicy(RoutePolicy.NEVER, 0, 0, 0, 0, 0, 0))
        assert e.route(arr).tolist() == [0, 0]
    # hysteresis keeps one state per sequence across calls
    e.set_route_policy(RoutePolicy(RoutePolicy.HYSTERESIS, 0.8, 0.2, 0.3, 0, 1, 2.0))
    for trial in range(200):
        arr = (DraftStats * 2)()
        for k, sid in enumerate(ids):
            arr[k] = _stats(rng, sid, V, 0.9)
        scores = [R.score(R.khat(R.alpha_entropy([np.float32(arr[k].entropy[i]) for i in range(arr[k].span_len)], 2.0, V)), np.float32(0.3))
                  for k in range(2)]
        if any(abs(s - 0.8) < 1e-5 or abs(s - 0.2) < 1e-5 for s in scores):
            break                                   # a threshold tie in fp32 vs fp64: state could diverge, stop here
        want = [int(hyst[sid](s)) for sid, s in zip(ids, scores)]
        assert e.route(arr).tolist() == want, trial
    # a user hook replaces the policy
    seen = []
    e.set_router(lambda st: (seen.append(st.seq_id), st.span_len >= 2)[1])
    got = e.route(arr).tolist()
    assert seen == list(ids) and got == [int(arr[k].span_len >= 2) for k in range(2)]
    e.set_router(None)
    e.close()


def test_ucb_router_follows_the_oracle_through_a_decode_run():
    """S2D2_ROUTE_UCB on the tiny fp32 workload with peaked logits, against the oracle's bandit fed with the same
    statistics and the same rewards: identical decisions at every step, and both actions occur."""
    from paper_2603_25702_b200 import Engine, RoutePolicy
    wl = get_config("t_f32", block_size=8, gen_tokens=64, model_logit_scale=12.0)
    W = generate_weights(wl.model, seed=2, gain_jitter=0.1)
    e = Engine(wl.model, block_size=8, max_batch=1, max_seq_len=128, kv_page_tokens=8, tau_conf=0.5,
               stream=torch.cuda.current_stream().cuda_stream)
    e.load_weights(W)
    sid = e.prefill([[3, 1, 4, 1, 5]])[0]
    beta = 0.7
    e.set_route_policy(RoutePolicy(RoutePolicy.UCB, beta, 0, 0, 0, 0, 0))
    orc = R.UCBRouter(beta, 8, wl.model.vocab, bins=2)
    decisions = []
    for step in range(60):
        if e.debug_seq_state(sid)["block_start"] >= 5 + 64:
            break
        st = e.draft_block([sid])
        fl = e.route(st)
        s = st[0]
        want = orc.decide(s.span_len, s.n_masked, [np.float32(s.entropy[i]) for i in range(s.span_len)])
        assert bool(fl[0]) == want, step
        e.verify_block([sid], fl)
        res = e.accept_and_commit([sid], fl)
        orc.update(res[0].n_committed)
        decisions.append(int(fl[0]))
    assert 0 in decisions and 1 in decisions and len(decisions) >= 8
    e.close()
