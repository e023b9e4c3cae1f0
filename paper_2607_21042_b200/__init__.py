"""B200-native decode step of the IndexTTS-2 Text-to-Semantic GPT behind a C-ABI library.

Importing the package is cheap and loads nothing native.  ``binding.load()`` (called by every
``TtsGpt`` constructor) opens ``libtts_gpt.so`` and raises if it is missing: there is no CPU
fallback.
"""
