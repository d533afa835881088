"""The five synthetic workloads (no arithmetic here: names and sizes only).

arch / precision / n_e / t_max / actions / updates / learning rate / terminal probability 1/term_denom.
Index 4 (n_e = 1024, Nature CNN, bf16) is the throughput configuration.
"""
CONFIGS = [
    dict(name="cfg1_nips_fp32_ne4", arch="nips", precision="fp32", n_e=4, t_max=5, n_actions=4, updates=3,
         lr=0.0028, term_denom=200),
    dict(name="cfg2_nips_fp32_ne32", arch="nips", precision="fp32", n_e=32, t_max=5, n_actions=6, updates=100,
         lr=0.0224, term_denom=200),
    dict(name="cfg3_nature_bf16_ne32", arch="nature", precision="bf16", n_e=32, t_max=5, n_actions=18, updates=100,
         lr=0.0224, term_denom=200),
    dict(name="cfg4_nature_bf16_ne256", arch="nature", precision="bf16", n_e=256, t_max=5, n_actions=18, updates=200,
         lr=0.0224, term_denom=100),
    dict(name="cfg5_nature_bf16_ne1024", arch="nature", precision="bf16", n_e=1024, t_max=5, n_actions=18,
         updates=200, lr=0.0224, term_denom=200),
]
COMMON = dict(gamma=0.99, rms_decay=0.99, rms_eps=0.1, clip_norm=40.0, entropy_beta=0.01, value_coef=1.0, seed=1)
