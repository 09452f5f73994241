"""The controller step on the GPU against the oracle, through the C-ABI: 25 decoding steps of a batch of
three sequences with a cache interval of 4.  Logits within 2e-4 of the fp64 oracle (fp32 accumulation over
12 288 features); the chosen action, the cache state, the (TT, d, k) written into the step array and the
averaged reward must be the oracle's whenever the choice has a margin above the fp32 error."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("temperature", [0.0, 1.5])
def test_controller_steps_match_the_oracle(temperature):
    import oracle
    from paper_2601_12212_b200 import binding, synth
    rng = np.random.default_rng(3)
    B, per_layer, H, N = 3, 4096, 128, 4
    F = 3 * per_layer
    actions = np.array(synth.action_space(filtered=True), np.int32)
    A = len(actions)
    w = (rng.normal(size=(H, F)) / np.sqrt(F), rng.normal(size=H) * 0.1, rng.normal(size=(H, H)) / np.sqrt(H),
         rng.normal(size=H) * 0.1, rng.normal(size=(A, H)) * 0.5, rng.normal(size=A) * 0.1)
    w = tuple(x.astype(np.float32) for x in w)
    dw = [torch.from_numpy(x).cuda() for x in w]
    d_actions = torch.from_numpy(actions).cuda()
    ctx = binding.Context(8, 2, 128, 1000, max_batch=B, max_tt=128, max_k=32, max_depth=8)
    pol = binding.make_policy(*dw, d_actions)
    i32 = dict(dtype=torch.int32, device="cuda")
    d_state = torch.zeros(B, 4, **i32)
    d_steps = torch.tensor([[1, 1, 1, 100 + s] for s in range(B)], **i32)
    d_reward = torch.full((B,), -1.0, device="cuda")
    d_logits = torch.zeros(B, A, device="cuda")
    d_action = torch.zeros(B, **i32)
    d_u = torch.zeros(B, dtype=torch.float64, device="cuda")
    states = [oracle.ControllerState() for _ in range(B)]
    prev = [(None, None)] * B
    d_alen = torch.zeros(B, **i32)
    d_secs = torch.zeros(B, device="cuda")
    asked = 0
    for step in range(25):
        hid = [synth.to_bf16_bits(rng.normal(size=(B, per_layer)).astype(np.float32).ravel()).reshape(B, per_layer)
               for _ in range(3)]
        d_hid = [torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16) for h in hid]
        u = rng.uniform(size=B)
        d_u.copy_(torch.from_numpy(u))
        binding.resps_controller_step(ctx, pol, *d_hid, per_layer, B, N, temperature, d_u,
                                      d_alen if step else None, d_secs if step else None, d_state, d_steps, d_reward,
                                      d_logits, d_action)
        assert ctx.status() == 0
        g_state, g_steps = d_state.cpu().numpy(), d_steps.cpu().numpy()
        g_reward, g_logits, g_action = d_reward.cpu().numpy(), d_logits.cpu().numpy(), d_action.cpu().numpy()
        for s in range(B):
            vec = np.concatenate([synth.bf16_bits_to_f32(h[s]) for h in hid]).astype(np.float64)
            st, act, r_avg, logits, margin = oracle.controller_step(states[s], vec, w, actions, N, temperature, u[s],
                                                                    *prev[s])
            if logits is not None:
                asked += 1
                np.testing.assert_allclose(g_logits[s], logits, atol=2e-4)
                if margin < (2e-3 if temperature == 0.0 else 1e-4):
                    st.action = int(g_action[s])        # a choice on a knife's edge: go on with the GPU's
                    act = tuple(int(x) for x in actions[st.action])
            states[s] = st
            assert g_action[s] == st.action and g_state[s, 0] == st.cache_step and g_state[s, 1] == st.action
            assert g_steps[s].tolist() == [*act, 100 + s]                   # the prefix column is not touched
            assert g_state[s, 3] == st.reward_steps
            assert g_state[s, 2:3].view(np.float32)[0] == pytest.approx(st.reward_sum, rel=1e-5)
            if r_avg is not None:
                assert g_reward[s] == pytest.approx(r_avg, rel=1e-5)
        alen = rng.integers(0, 7, size=B).astype(np.int32)
        secs = rng.uniform(4e-4, 9e-4, size=B).astype(np.float32)
        d_alen.copy_(torch.from_numpy(alen))
        d_secs.copy_(torch.from_numpy(secs))
        prev = [(int(alen[s]), float(secs[s])) for s in range(B)]
    assert asked == B * 7                                                   # steps 0, 4, ..., 24
    ctx.close()


def test_controller_host_side_errors():
    from paper_2601_12212_b200 import binding
    ctx = binding.Context(8, 2, 128, 1000, max_batch=1, max_tt=32, max_k=8, max_depth=4)
    z = torch.zeros(300 * 30, device="cuda")
    zi = torch.zeros(64, dtype=torch.int32, device="cuda")
    hid = torch.zeros(1, 10, dtype=torch.bfloat16, device="cuda")
    pol = binding.RespsPolicy(z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(),
                              zi.data_ptr(), 30, 300, 4)                    # hidden 300 > 256
    with pytest.raises(binding.RespsError) as e:
        binding.resps_controller_step(ctx, pol, hid, hid, hid, 10, 1, 4, 0.0, None, None, None, zi, zi, z[:1])
    assert e.value.code == binding.RESPS_ERR_UNSUPPORTED_SHAPE
    pol = binding.RespsPolicy(z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(),
                              zi.data_ptr(), 31, 128, 4)                    # features not a multiple of 3
    with pytest.raises(binding.RespsError) as e:
        binding.resps_controller_step(ctx, pol, hid, hid, hid, 10, 1, 4, 0.0, None, None, None, zi, zi, z[:1])
    assert e.value.code == binding.RESPS_ERR_INVALID_ARG
    ctx.close()
